// Adapter update of a fine-tuning step (Section 4.1): joint gradient norm, clipping
// coefficient and AdamW over one flat array of trained parameters.  Two launches, both
// bound by HBM: the first reads the gradients once, the second reads gradient, master
// parameter and both moments and writes parameter, moments and the bf16 copy the layers use.
#define QALORA_TU 8
#include "common.cuh"

namespace qalora {

namespace {

constexpr int OPT_THREADS = 256;
constexpr int OPT_MAX_PARTS = 1024;     // partial sums of squares (one per block of the first launch)
constexpr int OPT_BLOCKS_PER_SM = 8;

__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float sq4(float4 v) { return v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w; }

// Sum over a block in a fixed order: lanes by shuffle, then warps by one thread.
template <typename T>
__device__ __forceinline__ T block_sum(T v, T* scratch /*[OPT_THREADS / 32]*/) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  T total = 0;
#pragma unroll
  for (int w = 0; w < OPT_THREADS / 32; ++w) total += scratch[w];
  return total;
}

// parts[b] = sum of squares of block b's contiguous range of the gradient.  The ranges and the
// order of additions depend only on n and the grid, so the result is reproducible.
__global__ void __launch_bounds__(OPT_THREADS)
grad_sqnorm_kernel(const float* __restrict__ grad, size_t n, size_t per_block /*multiple of 4*/, float* __restrict__ parts,
                   int* dbg) {
  __shared__ float scratch[OPT_THREADS / 32];
  const size_t lo = (size_t)blockIdx.x * per_block;
  size_t hi = lo + per_block;
  if (hi > n) hi = n;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  if (lo < hi) {
    const size_t vec_hi = lo + ((hi - lo) & ~(size_t)3);
    size_t i = lo + (size_t)threadIdx.x * 4;
    for (; i + 3 * OPT_THREADS * 4 < vec_hi; i += 4 * OPT_THREADS * 4) {   // four independent loads in flight
      if (!QALORA_CHECK(dbg, i + 3 * OPT_THREADS * 4 + 3, n)) break;
      const float4 a = ld4(grad + i), b = ld4(grad + i + OPT_THREADS * 4), c = ld4(grad + i + 2 * OPT_THREADS * 4),
                   d = ld4(grad + i + 3 * OPT_THREADS * 4);
      acc[0] += sq4(a); acc[1] += sq4(b); acc[2] += sq4(c); acc[3] += sq4(d);
    }
    for (; i < vec_hi; i += OPT_THREADS * 4)
      if (QALORA_CHECK(dbg, i + 3, n)) acc[0] += sq4(ld4(grad + i));
    for (size_t j = vec_hi + threadIdx.x; j < hi; j += OPT_THREADS) acc[1] += grad[j] * grad[j];
  }
  const float total = block_sum((acc[0] + acc[1]) + (acc[2] + acc[3]), scratch);
  if (threadIdx.x == 0 && QALORA_CHECK(dbg, blockIdx.x, OPT_MAX_PARTS)) parts[blockIdx.x] = total;
}

struct AdamConsts {
  float decay;        // 1 - lr * weight_decay
  float beta1, beta2, one_minus_beta1, one_minus_beta2;
  float step_size;    // lr / (1 - beta1^t)
  float inv_sqrt_bc2; // 1 / sqrt(1 - beta2^t)
  float eps, max_norm;
};

__device__ __forceinline__ void adam_one(float g, float& p, float& m, float& v, float coef, const AdamConsts& k) {
  g *= coef;
  p *= k.decay;
  m = fmaf(k.beta1, m, k.one_minus_beta1 * g);
  v = fmaf(k.beta2, v, k.one_minus_beta2 * g * g);
  const float denom = fmaf(sqrtf(v), k.inv_sqrt_bc2, k.eps);
  p -= k.step_size * __fdiv_rn(m, denom);
}

// Every block adds the same partial sums in the same order (fp64), so all blocks clip by the
// same coefficient; then a grid-stride loop over groups of four parameters.
__global__ void __launch_bounds__(OPT_THREADS)
adamw_kernel(const float* __restrict__ grad, float* __restrict__ param, float* __restrict__ exp_avg,
             float* __restrict__ exp_avg_sq, __nv_bfloat16* __restrict__ param_bf16, size_t n,
             const float* __restrict__ parts, int nparts, AdamConsts k, float* __restrict__ norm_out, int* dbg) {
  __shared__ double scratch[OPT_THREADS / 32];
  double mine = 0.0;
  for (int i = threadIdx.x; i < nparts; i += OPT_THREADS) mine += (double)parts[i];
  const double sumsq = block_sum(mine, scratch);
  const float norm = (float)sqrt(sumsq);
  float coef = 1.f;
  if (k.max_norm > 0.f) coef = fminf(1.f, k.max_norm / (norm + 1e-6f));
  if (norm_out != nullptr && blockIdx.x == 0 && threadIdx.x == 0) { norm_out[0] = norm; norm_out[1] = coef; }

  const size_t nvec = n / 4, stride = (size_t)gridDim.x * OPT_THREADS;
  for (size_t q = (size_t)blockIdx.x * OPT_THREADS + threadIdx.x; q < nvec; q += stride) {
    const size_t i = q * 4;
    if (!QALORA_CHECK(dbg, i + 3, n)) break;
    const float4 g = ld4(grad + i);
    float4 p = ld4(param + i), m = ld4(exp_avg + i), v = ld4(exp_avg_sq + i);
    adam_one(g.x, p.x, m.x, v.x, coef, k); adam_one(g.y, p.y, m.y, v.y, coef, k);
    adam_one(g.z, p.z, m.z, v.z, coef, k); adam_one(g.w, p.w, m.w, v.w, coef, k);
    *reinterpret_cast<float4*>(param + i) = p;
    *reinterpret_cast<float4*>(exp_avg + i) = m;
    *reinterpret_cast<float4*>(exp_avg_sq + i) = v;
    const __nv_bfloat162 lo = __floats2bfloat162_rn(p.x, p.y), hi = __floats2bfloat162_rn(p.z, p.w);
    uint2 packed;
    packed.x = *reinterpret_cast<const uint32_t*>(&lo);
    packed.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(param_bf16 + i) = packed;
  }
  if (blockIdx.x == 0) {          // ragged tail of fewer than four
    const size_t i = nvec * 4 + threadIdx.x;
    if (i < n) {
      float p = param[i], m = exp_avg[i], v = exp_avg_sq[i];
      adam_one(grad[i], p, m, v, coef, k);
      param[i] = p; exp_avg[i] = m; exp_avg_sq[i] = v;
      param_bf16[i] = __float2bfloat16_rn(p);
    }
  }
}

}  // namespace

size_t adamw_workspace_bytes() { return OPT_MAX_PARTS * sizeof(float); }

int launch_adamw(const AdamwArgs& a, int64_t n64, const float* grad, float* param, float* exp_avg, float* exp_avg_sq,
                 __nv_bfloat16* param_bf16, float* parts, float* norm_out, cudaStream_t st) {
  const size_t n = (size_t)n64;
  if (n == 0) return QALORA_OK;
  // first launch: at most OPT_MAX_PARTS blocks, each over a contiguous range of at least 4096 values
  size_t per_block = round_up((n + OPT_MAX_PARTS - 1) / OPT_MAX_PARTS, 4);
  if (per_block < 4096) per_block = 4096;
  const int nparts = (int)((n + per_block - 1) / per_block);
  grad_sqnorm_kernel<<<nparts, OPT_THREADS, 0, st>>>(grad, n, per_block, parts, debug_words());
  AdamConsts k;
  k.decay = (float)(1.0 - (double)a.lr * a.weight_decay);
  k.beta1 = a.beta1; k.beta2 = a.beta2;
  k.one_minus_beta1 = (float)(1.0 - (double)a.beta1); k.one_minus_beta2 = (float)(1.0 - (double)a.beta2);
  k.step_size = (float)((double)a.lr / (1.0 - pow((double)a.beta1, (double)a.step)));
  k.inv_sqrt_bc2 = (float)(1.0 / sqrt(1.0 - pow((double)a.beta2, (double)a.step)));
  k.eps = a.eps; k.max_norm = a.max_grad_norm;
  const size_t want = (n / 4 + OPT_THREADS - 1) / OPT_THREADS;
  size_t blocks = (size_t)device_sm_count() * OPT_BLOCKS_PER_SM;
  if (blocks > want) blocks = want > 0 ? want : 1;
  adamw_kernel<<<(unsigned)blocks, OPT_THREADS, 0, st>>>(grad, param, exp_avg, exp_avg_sq, param_bf16, n, parts, nparts, k,
                                                         norm_out, debug_words());
  count_launch(2);
  return cuda_status(cudaGetLastError());
}

}  // namespace qalora
