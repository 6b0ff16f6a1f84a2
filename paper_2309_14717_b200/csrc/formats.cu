// Format conversions around the packed layer: dequantization of the whole weight matrix
// (Eq. 1) and the zero-point form of Algorithm 1 (W~ = alpha * (c - z)) in both directions.
// All three are element-wise and bound by HBM.
#define QALORA_TU 9
#include "common.cuh"

namespace qalora {

namespace {

constexpr int FMT_THREADS = 256;

template <typename TO> __device__ __forceinline__ void store_weight(TO* p, float v);
template <> __device__ __forceinline__ void store_weight<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void store_weight<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// One thread per (pack unit, output column): the unit's words are one 8/12/16-byte load that
// is contiguous across the columns of a warp; each of the 32 rows it writes is contiguous
// across the warp as well.
template <int BITS, typename TO>
__global__ void __launch_bounds__(FMT_THREADS)
dequantize_kernel(const uint32_t* __restrict__ codes, const float2* __restrict__ qparams, TO* __restrict__ W,
                  int N, int g, int* dbg) {
  constexpr int WORDS = BITS == 4 ? 4 : (BITS == 3 ? 3 : 2);
  const int n = blockIdx.x * FMT_THREADS + threadIdx.x;
  const int kb = blockIdx.y;
  if (n >= N) return;
  // gridDim.y = K / 32 k-block rows: the unit read, the (alpha, beta) pair and the last of the 32 rows written
  if (!QALORA_CHECK(dbg, ((size_t)kb * N + n) * WORDS + WORDS - 1, (size_t)gridDim.y * N * WORDS) ||
      !QALORA_CHECK(dbg, (size_t)(kb * 32 / g) * N + n, (size_t)(gridDim.y * 32 / g) * N) ||
      !QALORA_CHECK(dbg, ((size_t)kb * 32 + 31) * N + n, (size_t)gridDim.y * 32 * N))
    return;
  uint32_t u[WORDS];
  const uint32_t* src = codes + ((size_t)kb * N + n) * WORDS;
  if (BITS == 4) {
    const uint4 v = *reinterpret_cast<const uint4*>(src);
    u[0] = v.x; u[1] = v.y; u[2] = v.z; u[3] = v.w;
  } else if (BITS == 2) {
    const uint2 v = *reinterpret_cast<const uint2*>(src);
    u[0] = v.x; u[1] = v.y;
  } else {
#pragma unroll
    for (int i = 0; i < WORDS; ++i) u[i] = src[i];
  }
  const float2 ab = qparams[(size_t)(kb * 32 / g) * N + n];
  TO* dst = W + (size_t)kb * 32 * N + n;
#pragma unroll
  for (int j = 0; j < 32; ++j)
    store_weight<TO>(dst + (size_t)j * N, fmaf(ab.x, (float)unit_code<BITS>(u, j), ab.y));
}

// qparams[i] = (alpha[i], -alpha[i] * z[i])
__global__ void __launch_bounds__(FMT_THREADS)
from_zero_point_kernel(const float* __restrict__ alpha, const float* __restrict__ zero, float2* __restrict__ qparams, size_t n) {
  const size_t i = (size_t)blockIdx.x * FMT_THREADS + threadIdx.x;
  if (i < n) {
    const float a = alpha[i];
    qparams[i] = make_float2(a, __fmul_rn(-a, zero[i]));
  }
}

// alpha[i] = qparams[i].x;  z[i] = -qparams[i].y / qparams[i].x
__global__ void __launch_bounds__(FMT_THREADS)
to_zero_point_kernel(const float2* __restrict__ qparams, float* __restrict__ alpha, float* __restrict__ zero, size_t n) {
  const size_t i = (size_t)blockIdx.x * FMT_THREADS + threadIdx.x;
  if (i < n) {
    const float2 ab = qparams[i];
    alpha[i] = ab.x;
    zero[i] = __fdiv_rn(-ab.y, ab.x);
  }
}

template <int BITS, typename TO>
void launch_dequantize_t(const Shape& sh, const uint32_t* codes, const float2* qparams, TO* W, cudaStream_t st) {
  const dim3 grid((unsigned)((sh.N + FMT_THREADS - 1) / FMT_THREADS), (unsigned)(sh.K / 32));
  dequantize_kernel<BITS, TO><<<grid, FMT_THREADS, 0, st>>>(codes, qparams, W, sh.N, sh.g, debug_words());
}

}  // namespace

int launch_dequantize(const Shape& sh, const uint32_t* codes, const float2* qparams, void* W, bool bf16_out, cudaStream_t st) {
  if (sh.K / 32 > 65535) return QALORA_ERR_UNSUPPORTED_SHAPE;
#define QALORA_DEQ(B)                                                                                     \
  if (bf16_out) launch_dequantize_t<B, __nv_bfloat16>(sh, codes, qparams, static_cast<__nv_bfloat16*>(W), st); \
  else launch_dequantize_t<B, float>(sh, codes, qparams, static_cast<float*>(W), st)
  if (sh.bits == 4) { QALORA_DEQ(4); } else if (sh.bits == 3) { QALORA_DEQ(3); } else { QALORA_DEQ(2); }
#undef QALORA_DEQ
  count_launch();
  return cuda_status(cudaGetLastError());
}

int launch_from_zero_point(const Shape& sh, const float* alpha, const float* zero, float2* qparams, cudaStream_t st) {
  const size_t n = (size_t)sh.G * sh.N;
  from_zero_point_kernel<<<(unsigned)((n + FMT_THREADS - 1) / FMT_THREADS), FMT_THREADS, 0, st>>>(alpha, zero, qparams, n);
  count_launch();
  return cuda_status(cudaGetLastError());
}

int launch_to_zero_point(const Shape& sh, const float2* qparams, float* alpha, float* zero, cudaStream_t st) {
  const size_t n = (size_t)sh.G * sh.N;
  to_zero_point_kernel<<<(unsigned)((n + FMT_THREADS - 1) / FMT_THREADS), FMT_THREADS, 0, st>>>(qparams, alpha, zero, n);
  count_launch();
  return cuda_status(cudaGetLastError());
}

}  // namespace qalora
