// Shared device/host helpers of the QA-LoRA kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "debug.cuh"
#include "qalora.h"

namespace qalora {

// ---------------------------------------------------------------- host side --
struct Shape {
  int K, N, g, G, bits, r, words;   // words = uint32 words per pack unit
  float s;
};

__host__ __device__ inline int words_per_unit(int bits) { return bits == 4 ? 4 : (bits == 3 ? 3 : 2); }

// Validates a descriptor and fills `sh`.  Returns a qalora_status.
int check_desc(const qalora_desc* desc, Shape* sh);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Scratch layout shared by forward and backward (offsets in bytes, 256-aligned).
struct Workspace {
  size_t status;    // int32  device status word of the tensor-core kernels (first bytes of the workspace)
  size_t xp;        // float  [M][G]   pooled input                      (backward)
  size_t T;         // float  [M][r]   s * pool(x) * A                   (both)
  size_t dT;        // float  [M][r]   s * dy * B^T                      (backward)
  size_t Tb;        // bf16   [M][r]   T rounded, operand of the tensor-core path
  size_t dTb;       // bf16   [M][r]   dT rounded
  size_t partial;   // float  split-M partial sums of dA
  size_t partial_bytes;
  size_t partial_dB;   // float  split-M partial sums of dB (its own region: dB runs beside dT and dA on a second stream)
  size_t partial_dB_bytes;
  size_t dx_parts;  // float  partial results of a strip of dx tiles whose reduction is cut into parts (backward)
  size_t fwd_parts; // float  [parts][M][N] partial results of a forward reduction cut into parts (forward)
  size_t total;
  // bounds-check build only: a guard of kGuardBytes follows every region (guard[i] = its offset)
  size_t guard[12];
  int n_guard;
};
Workspace workspace_layout(const Shape& sh, int64_t m, int op);
// Bounds-check build: fill the workspace's guards / verify them (into the record words) on `st`.
// Both do nothing and return QALORA_OK in the ordinary build.
int debug_fill_guards(const Workspace& ws, void* workspace, cudaStream_t st);
int debug_verify_guards(const Workspace& ws, const void* workspace, cudaStream_t st);

// The public forward / backward in two halves (api.cu): checks that launch nothing, and the
// launches with a say on whether the workspace's status word is cleared first.
// `layout_op`: which qalora_op layout the workspace has (FORWARD, or TRAIN for a forward whose
// pooled input the backward pass of the same step reuses: `pooled`).
int forward_validate(const qalora_desc* desc, int64_t m, const void* x, const void* codes, const float* qparams,
                     const void* A, const void* B, const void* y, const void* workspace, size_t workspace_bytes,
                     int layout_op);
int forward_launch(const qalora_desc* desc, int64_t m, const void* x, const void* codes, const float* qparams,
                   const void* A, const void* B, void* y, void* workspace, void* cuda_stream, bool reset_status,
                   int layout_op);
int backward_impl(const qalora_desc* desc, int64_t m, const void* x, const void* dy, const void* codes,
                  const float* qparams, const void* A, const void* B, void* dx, float* dA, float* dB,
                  void* workspace, size_t workspace_bytes, void* cuda_stream, bool reset_status, bool pooled);

// --------------------------------------------------------------- device side --
__device__ __forceinline__ float bf16_to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// Code of position j (0..31) of a pack unit whose words are u[0..words).
template <int BITS>
__device__ __forceinline__ uint32_t unit_code(const uint32_t* u, int j) {
  if (BITS == 4) {
    const int e = j & 7;
    return (u[j >> 3] >> (16 * (e & 1) + 4 * (e >> 1))) & 15u;
  } else if (BITS == 2) {
    const int e = j & 15;
    return (u[j >> 4] >> (16 * (e & 1) + 2 * (e >> 1))) & 3u;
  } else {
    const int e = j & 15;
    const uint32_t lo = (u[j >> 4] >> (16 * (e & 1) + 2 * (e >> 1))) & 3u;
    const uint32_t hi = (u[2] >> (16 * (j & 1) + (j >> 1))) & 1u;
    return lo | (hi << 2);
  }
}

// ORs code c of position j into the unit's words.
template <int BITS>
__device__ __forceinline__ void unit_insert(uint32_t* u, int j, uint32_t c) {
  if (BITS == 4) {
    const int e = j & 7;
    u[j >> 3] |= c << (16 * (e & 1) + 4 * (e >> 1));
  } else if (BITS == 2) {
    const int e = j & 15;
    u[j >> 4] |= c << (16 * (e & 1) + 2 * (e >> 1));
  } else {
    const int e = j & 15;
    u[j >> 4] |= (c & 3u) << (16 * (e & 1) + 2 * (e >> 1));
    u[2] |= (c >> 2) << (16 * (j & 1) + (j >> 1));
  }
}

// Launch helpers implemented in the kernel files (all asynchronous on `st`).
int launch_quantize(const Shape& sh, const float* W, uint32_t* codes, float2* qparams,
                    int32_t* dev_status, cudaStream_t st);
int launch_merge(const Shape& sh, const float2* qin, const __nv_bfloat16* A, const __nv_bfloat16* B,
                 float2* qout, cudaStream_t st);
// pool + T = s*pool(x)*A.  xp may be NULL (not stored).  Tb may be NULL.
int launch_pool_T(const Shape& sh, int64_t M, const __nv_bfloat16* x, const __nv_bfloat16* A,
                  float* xp, float* T, __nv_bfloat16* Tb, cudaStream_t st);
int launch_simt_forward(const Shape& sh, int64_t M, const __nv_bfloat16* x, const uint32_t* codes,
                        const float2* qparams, const float* T, const __nv_bfloat16* B,
                        __nv_bfloat16* y, cudaStream_t st);
int launch_dT(const Shape& sh, int64_t M, const __nv_bfloat16* dy, const __nv_bfloat16* B,
              float* dT, __nv_bfloat16* dTb, cudaStream_t st);
int launch_simt_dx(const Shape& sh, int64_t M, const __nv_bfloat16* dy, const uint32_t* codes,
                   const float2* qparams, const float* dT, const __nv_bfloat16* A,
                   __nv_bfloat16* dx, cudaStream_t st);
// out[p][q] = sum_m X[m][p] * Y[m][q]   (X float [M][P]; Y bf16 or float [M][Q])
size_t atb_partial_bytes(int64_t M, int P, int Q);
int launch_atb_bf16(int64_t M, int P, int Q, const float* X, const __nv_bfloat16* Y, float* out,
                    float* partial, size_t partial_bytes, cudaStream_t st);
int launch_atb_f32(int64_t M, int P, int Q, const float* X, const float* Y, float* out,
                   float* partial, size_t partial_bytes, cudaStream_t st);

// Tensor-core paths (gemm_tc.cu).  Tb / dTb are the bf16 rank-r intermediates.
bool tc_forward_supported(const Shape& sh, int64_t M);
bool tc_dx_supported(const Shape& sh, int64_t M);
size_t tc_forward_partial_bytes(const Shape& sh, int64_t M);   // scratch for a reduction cut into parts (few tokens)
int launch_tc_forward(const Shape& sh, int64_t M, const __nv_bfloat16* x, const uint32_t* codes,
                      const float2* qparams, const __nv_bfloat16* Tb, const __nv_bfloat16* B,
                      __nv_bfloat16* y, float* partial, int* status, cudaStream_t st);
size_t tc_dx_partial_bytes(const Shape& sh, int64_t M);         // scratch for a short last wave cut into parts
int launch_tc_dx(const Shape& sh, int64_t M, const __nv_bfloat16* dy, const uint32_t* codes,
                 const float2* qparams, const __nv_bfloat16* dTb, const __nv_bfloat16* A,
                 __nv_bfloat16* dx, float* partial, int* status, cudaStream_t st);

// Forward for a few dozen to a few hundred tokens (midm_tc.cu): tokens as the MMA rows, 256
// channels per instruction.  Tb is the bf16 rank-r intermediate (ignored when r == 0).
bool midm_supported(const Shape& sh, int64_t M);
size_t midm_partial_bytes(const Shape& sh, int64_t M);
int launch_midm(const Shape& sh, int64_t M, const __nv_bfloat16* x, const uint32_t* codes, const float2* qparams,
                const __nv_bfloat16* Tb, const __nv_bfloat16* B, __nv_bfloat16* y, float* partial, int* status,
                cudaStream_t st);

// Few-token forward (gemv.cu): M <= 32.  `reset_status`: the kernel clears *status at its start.
bool gemv_supported(const Shape& sh, int64_t M);
int launch_gemv(const Shape& sh, int64_t M, const __nv_bfloat16* x, const uint32_t* codes, const float2* qparams,
                const __nv_bfloat16* Tb, const __nv_bfloat16* B, __nv_bfloat16* y, int* status, bool reset_status,
                cudaStream_t st);

void arm_few_token_wait_expiry(int stages, unsigned long long limit_ns);   // test hook, one-shot
void arm_tc_wait_expiry(int steps, unsigned long long limit_ns);           // the same for the next forward / dX tensor-core launch

// Several layers without adapter, the same M <= 16 rows each, in ONE few-token launch.
struct GemvGroupItem {
  Shape sh;
  const __nv_bfloat16* x;
  const uint32_t* codes;
  const float2* qparams;
  __nv_bfloat16* y;
};
bool gemv_group_supported(const GemvGroupItem* items, int n, int64_t M);
int launch_gemv_group(const GemvGroupItem* items, int n, int64_t M, int* status, bool reset_status, cudaStream_t st);

// out[i] = sum over splits of partial[z][i], added in a fixed order.
int launch_sum_partials(const float* partial, float* out, size_t count, int splits, cudaStream_t st);

// Tensor-core rank-r side products of the backward pass (aux_tc.cu).
bool tc_aux_supported(const Shape& sh, int64_t M);
int launch_tc_dT(const Shape& sh, int64_t M, const __nv_bfloat16* dy, const __nv_bfloat16* B,
                 float* dT, __nv_bfloat16* dTb, int* status, cudaStream_t st);
size_t tc_dB_partial_bytes(const Shape& sh, int64_t M);
int launch_tc_dB_partials(const Shape& sh, int64_t M, const __nv_bfloat16* Tb, const __nv_bfloat16* dy,
                          float* partial, int* splits_out, int* status, cudaStream_t st);

// Format conversions (formats.cu): whole-matrix dequantization and Algorithm 1's zero-point form.
int launch_dequantize(const Shape& sh, const uint32_t* codes, const float2* qparams, void* W, bool bf16_out, cudaStream_t st);
int launch_from_zero_point(const Shape& sh, const float* alpha, const float* zero, float2* qparams, cudaStream_t st);
int launch_to_zero_point(const Shape& sh, const float2* qparams, float* alpha, float* zero, cudaStream_t st);

// Adapter update (optimizer.cu): clipped AdamW over one flat array, two launches.
struct AdamwArgs { float lr, beta1, beta2, eps, weight_decay, max_grad_norm; int64_t step; };
size_t adamw_workspace_bytes();
int launch_adamw(const AdamwArgs& a, int64_t n, const float* grad, float* param, float* exp_avg, float* exp_avg_sq,
                 __nv_bfloat16* param_bf16, float* parts, float* norm_out, cudaStream_t st);

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? QALORA_OK : QALORA_ERR_CUDA; }

// ---- per-device host state ---------------------------------------------------
// A process may drive several GPUs.  Everything the library remembers about a device (its
// SM count, whether a kernel's shared-memory limit has been raised there) is kept per
// device ordinal of the device that is current at the call.
constexpr int kMaxDevices = 64;
int current_device();        // ordinal of the current device, -1 when it cannot be had or is beyond kMaxDevices
int device_sm_count();       // multiprocessors of the current device (148 when the query fails)

// One-time set-up per device, e.g. cudaFuncSetAttribute of one kernel: `run(fn)` calls
// fn() -> cudaError_t the first time it is reached with a given device current and returns
// that first outcome (as a qalora_status) from then on.  One static instance per kernel.
struct PerDeviceOnce {
  std::atomic<int> state[kMaxDevices];     // 0: not yet, 1: done, 2: failed
  PerDeviceOnce() { for (auto& s : state) s.store(0, std::memory_order_relaxed); }
  template <class Fn>
  int run(Fn fn) {
    const int dev = current_device();
    if (dev < 0) return QALORA_ERR_CUDA;
    int s = state[dev].load(std::memory_order_acquire);
    if (s == 0) {
      // two threads may both get here: the set-up is idempotent, so both just do it
      s = fn() == cudaSuccess ? 1 : 2;
      state[dev].store(s, std::memory_order_release);
    }
    return s == 1 ? QALORA_OK : QALORA_ERR_CUDA;
  }
};

// Instrumentation: launch counter and the one-shot event probe around a main kernel.
void count_launch(int n = 1);
struct MainKernelProbe {            // records the armed events around one launch
  MainKernelProbe(const char* name, cudaStream_t st);
  ~MainKernelProbe();
  cudaStream_t st;
  cudaEvent_t stop;
};

}  // namespace qalora
