// Group-wise min-max quantization + bit packing (Eq. 1 per group, Section 3.3)
// and the merge of the adapter into the zero factors (Appendix B Eq. 7).
// Both are streaming, HBM-bound kernels: one thread owns one output column of
// one quantization group, so a warp reads 128 contiguous bytes of each W row.
#define QALORA_TU 7
#include <float.h>

#include "common.cuh"
#include "ptx.cuh"

namespace qalora {

constexpr int QCOLS = 128;   // columns (threads) per block

// Each thread: two passes over its g weights.  Pass 1 finds min/max, pass 2 rounds and packs
// one 32-channel unit at a time (with g = 32 out of the registers pass 1 filled, otherwise a
// re-read that hits L1/L2).  Every floating-point step is a single IEEE fp32 operation (no FMA
// contraction), so the integer decision is reproducible bit for bit on a CPU.  The division
// t = (w - beta) / alpha is the expensive one; the code only needs rint(t), so the
// kernel first takes t' = (w - beta) * (1 / alpha), which is within 4e-6 of t for
// t in [0, 15], and falls back to the IEEE division only where t' lies within 1e-4
// of a rounding boundary (a half-integer): everywhere else rint(t') = rint(t).
// The shortcut is taken only for 1e-30 < alpha < 1e30: outside that range 1 / alpha
// overflows or is a subnormal with few significant bits (a group of nearly equal tiny
// weights, or of huge ones), and every element takes the division.
// The kernel is bound by its instruction stream, and the conversion unit (rint, float to
// int) runs at a quarter of the rate of the others, so the common path avoids it: adding
// 1.5 * 2^23 rounds t' to the nearest-even integer in the sum's low mantissa bits (exactly
// rint for 0 <= t' < 2^22), subtracting it again gives rint(t') as a float for the boundary
// test, and the code bits are taken from the sum's bit pattern with one shift and one logic
// operation per weight.  No clamp is needed: beta is the group's minimum and alpha its range
// over 2^b - 1, so 0 <= t <= (2^b - 1)(1 + 2^-22); the mask keeps a non-finite group (which is
// reported through dev_status) from spilling into its neighbours' bits.
constexpr float kRoundMagic = 12582912.0f;   // 1.5 * 2^23
#ifndef QALORA_Q_MINB
#define QALORA_Q_MINB 6
#endif

// ORs the code held in the low bits of `rbits` into position j of the unit's words.
template <int BITS>
__device__ __forceinline__ void unit_insert_bits(uint32_t* u, int j, uint32_t rbits) {
  if (BITS == 4) {
    const int e = j & 7, pos = 16 * (e & 1) + 4 * (e >> 1);
    u[j >> 3] |= (rbits << pos) & (15u << pos);
  } else if (BITS == 2) {
    const int e = j & 15, pos = 16 * (e & 1) + 2 * (e >> 1);
    u[j >> 4] |= (rbits << pos) & (3u << pos);
  } else {
    const int e = j & 15, pos = 16 * (e & 1) + 2 * (e >> 1), hpos = 16 * (j & 1) + (j >> 1);
    u[j >> 4] |= (rbits << pos) & (3u << pos);
    u[2] |= ((rbits >> 2) << hpos) & (1u << hpos);
  }
}

template <int BITS>
__global__ void __launch_bounds__(QCOLS, QALORA_Q_MINB)
quantize_kernel(const float* __restrict__ W, uint32_t* __restrict__ codes,
                float2* __restrict__ qparams, int N, int g, int G, int ntiles, int32_t* dev_status, int* dbg) {
  constexpr int WORDS = BITS == 4 ? 4 : (BITS == 3 ? 3 : 2);
  constexpr float QMAX = float((1 << BITS) - 1);
  const int q = blockIdx.x / ntiles;
  const int n = (blockIdx.x % ntiles) * QCOLS + threadIdx.x;
  if (n >= N) return;
  if (!QALORA_CHECK(dbg, ((size_t)q * g + g - 1) * N + n, (size_t)G * g * N)) return;   // the last weight this thread reads
  const float* w = W + (size_t)q * g * N + n;

  float lo = FLT_MAX, hi = -FLT_MAX;
  float nonfinite = 0.0f;                        // stays 0 unless a weight is NaN or infinite (0 * w is then NaN)
  float v[32];
  for (int k0 = 0; k0 < g; k0 += 32) {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __ldg(w + (size_t)(k0 + j) * N);
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      nonfinite = fmaf(v[j], 0.0f, nonfinite);
      lo = fminf(lo, v[j]);
      hi = fmaxf(hi, v[j]);
    }
  }
  const bool bad = !(nonfinite == 0.0f);
  const float alpha = (hi == lo) ? 1.0f : __fdiv_rn(__fsub_rn(hi, lo), QMAX);
  const float beta = lo;
  if (QALORA_CHECK(dbg, (size_t)q * N + n, (size_t)G * N)) qparams[(size_t)q * N + n] = make_float2(alpha, beta);
  if (bad && dev_status != nullptr) atomicOr(dev_status, 1);

  const bool fast = alpha > 1e-30f && alpha < 1e30f && !bad;
  const float inv_alpha = fast ? __frcp_rn(alpha) : 0.0f;
  const int kb0 = q * (g / 32);
  for (int k0 = 0; k0 < g; k0 += 32) {
    if (g > 32) {                                  // (g == 32: v still holds the group)
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = __ldg(w + (size_t)(k0 + j) * N);
    }
    uint32_t u[WORDS];
#pragma unroll
    for (int i = 0; i < WORDS; ++i) u[i] = 0u;
    // two weights per instruction (packed two-lane add / sub / mul, each lane IEEE round-to-nearest)
    const float2 beta2 = make_float2(beta, beta), inv2 = make_float2(inv_alpha, inv_alpha), magic2 = make_float2(kRoundMagic, kRoundMagic);
#pragma unroll
    for (int j = 0; j < 32; j += 2) {
      const float2 d = ptx::fsub2(make_float2(v[j], v[j + 1]), beta2);
      const float2 t = ptx::fmul2(d, inv2);
      float2 r = ptx::fadd2(t, magic2);                   // low mantissa bits: rint(t), round half to even
      const float2 c = ptx::fsub2(r, magic2);
      const float2 e = ptx::fsub2(t, c);
      if (!fast || !(fabsf(e.x) <= 0.4999f)) {            // near a boundary (or a tie, or no shortcut): exact
        float ce = rintf(__fdiv_rn(d.x, alpha));
        ce = fminf(fmaxf(ce, 0.0f), QMAX);               // (a non-finite group: any code will do, but a valid one)
        r.x = __fadd_rn(ce, kRoundMagic);
      }
      if (!fast || !(fabsf(e.y) <= 0.4999f)) {
        float ce = rintf(__fdiv_rn(d.y, alpha));
        ce = fminf(fmaxf(ce, 0.0f), QMAX);
        r.y = __fadd_rn(ce, kRoundMagic);
      }
      unit_insert_bits<BITS>(u, j, __float_as_uint(r.x));
      unit_insert_bits<BITS>(u, j + 1, __float_as_uint(r.y));
    }
    uint32_t* dst = codes + ((size_t)(kb0 + k0 / 32) * N + n) * WORDS;
    if (!QALORA_CHECK(dbg, ((size_t)(kb0 + k0 / 32) * N + n) * WORDS + WORDS - 1, (size_t)G * (g / 32) * N * WORDS)) continue;
    if (WORDS == 4) {
      *reinterpret_cast<uint4*>(dst) = make_uint4(u[0], u[1], u[2], u[3]);
    } else if (WORDS == 2) {
      *reinterpret_cast<uint2*>(dst) = make_uint2(u[0], u[1]);
    } else {
#pragma unroll
      for (int i = 0; i < WORDS; ++i) dst[i] = u[i];
    }
  }
}

int launch_quantize(const Shape& sh, const float* W, uint32_t* codes, float2* qparams,
                    int32_t* dev_status, cudaStream_t st) {
  const int ntiles = (sh.N + QCOLS - 1) / QCOLS;
  const long long blocks = (long long)sh.G * ntiles;
  if (blocks > 0x7fffffffLL) return QALORA_ERR_UNSUPPORTED_SHAPE;
  dim3 grid((unsigned)blocks), block(QCOLS);
  if (sh.bits == 4) quantize_kernel<4><<<grid, block, 0, st>>>(W, codes, qparams, sh.N, sh.g, sh.G, ntiles, dev_status, debug_words());
  else if (sh.bits == 3) quantize_kernel<3><<<grid, block, 0, st>>>(W, codes, qparams, sh.N, sh.g, sh.G, ntiles, dev_status, debug_words());
  else quantize_kernel<2><<<grid, block, 0, st>>>(W, codes, qparams, sh.N, sh.g, sh.G, ntiles, dev_status, debug_words());
  count_launch();
  return cuda_status(cudaGetLastError());
}

// beta'[q][n] = beta[q][n] + s * sum_i A[q][i] * B[i][n]; alpha is copied.
// One thread per column and MERGE_GROUPS consecutive groups: an element of B is used for all
// of them.  The kernel moves a few MB and is bound by the latency of its loads, so they are
// issued in three batches: the block's [r x 128] slice of B (16-byte loads) and its rows of A
// go to shared memory together, the thread's (alpha, beta) pairs are fetched before the sums
// start.  In-place use is safe: a thread reads only the elements it then writes.
constexpr int MERGE_GROUPS = 8;

__global__ void __launch_bounds__(QCOLS)
merge_kernel(const float2* __restrict__ qin, const __nv_bfloat16* __restrict__ A,
             const __nv_bfloat16* __restrict__ B, float2* __restrict__ qout,
             int G, int N, int r, float s, int ntiles, int* dbg) {
  extern __shared__ __align__(16) float merge_smem[];
  float* a_rows = merge_smem;                                                    // [MERGE_GROUPS][r]
  __nv_bfloat16* b_tile = reinterpret_cast<__nv_bfloat16*>(merge_smem + MERGE_GROUPS * r);   // [r][QCOLS]
  const int q0 = (blockIdx.x / ntiles) * MERGE_GROUPS;
  const int n0 = (blockIdx.x % ntiles) * QCOLS;
  const int n = n0 + threadIdx.x;
  // B slice: r rows of 128 columns = 16 pieces of 8 columns per row (N is a multiple of 8)
  for (int idx = threadIdx.x; idx < r * (QCOLS / 8); idx += QCOLS) {
    const int i = idx / (QCOLS / 8), c = (idx % (QCOLS / 8)) * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (n0 + c < N) v = __ldg(reinterpret_cast<const uint4*>(B + (size_t)i * N + n0 + c));
    *reinterpret_cast<uint4*>(b_tile + i * QCOLS + c) = v;
  }
  for (int i = threadIdx.x; i < MERGE_GROUPS * r; i += QCOLS) {
    const int q = q0 + i / r;
    a_rows[i] = q < G ? bf16_to_float(A[(size_t)q * r + i % r]) : 0.0f;
  }
  float2 p[MERGE_GROUPS];
#pragma unroll
  for (int j = 0; j < MERGE_GROUPS; ++j) {
    const int q = q0 + j;
    p[j] = make_float2(0.f, 0.f);
    if (n < N && q < G && QALORA_CHECK(dbg, (size_t)q * N + n, (size_t)G * N)) p[j] = qin[(size_t)q * N + n];
  }
  __syncthreads();
  if (n >= N) return;
  float acc[MERGE_GROUPS];
#pragma unroll
  for (int j = 0; j < MERGE_GROUPS; ++j) acc[j] = 0.0f;
  // four adapter indices per step: the rows of A come as 16-byte shared loads (the same address for
  // every lane), so that the loop is not bound by its shared-memory loads; the sums run in index order
#pragma unroll 2
  for (int i = 0; i < r; i += 4) {                 // r is a multiple of 8
    float b[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) b[k] = bf16_to_float(b_tile[(i + k) * QCOLS + threadIdx.x]);
#pragma unroll
    for (int j = 0; j < MERGE_GROUPS; ++j) {
      const float4 a = *reinterpret_cast<const float4*>(a_rows + j * r + i);
      acc[j] = fmaf(a.x, b[0], acc[j]);
      acc[j] = fmaf(a.y, b[1], acc[j]);
      acc[j] = fmaf(a.z, b[2], acc[j]);
      acc[j] = fmaf(a.w, b[3], acc[j]);
    }
  }
#pragma unroll
  for (int j = 0; j < MERGE_GROUPS; ++j) {
    const int q = q0 + j;
    if (q < G) {
      p[j].y = fmaf(s, acc[j], p[j].y);
      qout[(size_t)q * N + n] = p[j];
    }
  }
}

int launch_merge(const Shape& sh, const float2* qin, const __nv_bfloat16* A, const __nv_bfloat16* B,
                 float2* qout, cudaStream_t st) {
  const int ntiles = (sh.N + QCOLS - 1) / QCOLS;
  const long long blocks = (long long)((sh.G + MERGE_GROUPS - 1) / MERGE_GROUPS) * ntiles;
  if (blocks > 0x7fffffffLL) return QALORA_ERR_UNSUPPORTED_SHAPE;
  const size_t smem = MERGE_GROUPS * sh.r * sizeof(float) + (size_t)sh.r * QCOLS * sizeof(__nv_bfloat16);   // up to 72 KiB at rank 256
  static PerDeviceOnce smem_limit;
  if (smem_limit.run([] { return cudaFuncSetAttribute(merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024); }) != QALORA_OK)
    return QALORA_ERR_CUDA;
  merge_kernel<<<(unsigned)blocks, QCOLS, smem, st>>>(qin, A, B, qout, sh.G, sh.N, sh.r, sh.s, ntiles, debug_words());
  count_launch();
  return cuda_status(cudaGetLastError());
}

}  // namespace qalora
