// C-ABI entry points: argument checks, scratch layout and kernel dispatch.
#define QALORA_TU 1
#include <algorithm>
#include <atomic>
#include <mutex>

#include "common.cuh"

namespace qalora {

static std::atomic<uint64_t> g_launches{0};
static thread_local cudaEvent_t t_probe_start = nullptr, t_probe_stop = nullptr;
static thread_local const char* t_main_kernel = "";

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

MainKernelProbe::MainKernelProbe(const char* name, cudaStream_t s) : st(s), stop(nullptr) {
  t_main_kernel = name;
  if (t_probe_start != nullptr && t_probe_stop != nullptr) {
    cudaEventRecord(t_probe_start, st);
    stop = t_probe_stop;
  }
  t_probe_start = t_probe_stop = nullptr;
}
MainKernelProbe::~MainKernelProbe() {
  if (stop != nullptr) cudaEventRecord(stop, st);
}

int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

int device_sm_count() {
  static std::atomic<int> cached[kMaxDevices];       // zero-initialized: 0 = not asked yet
  const int dev = current_device();
  if (dev < 0) return 148;
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

// ---- bounds-check build: record words and workspace guards ---------------------------
#ifdef QALORA_DEBUG
int* debug_words() {
  static std::atomic<int*> words[kMaxDevices];        // zero-initialized
  static std::mutex mu;
  const int dev = current_device();
  if (dev < 0) return nullptr;
  int* p = words[dev].load(std::memory_order_acquire);
  if (p == nullptr) {
    std::lock_guard<std::mutex> lock(mu);
    p = words[dev].load(std::memory_order_acquire);
    if (p == nullptr) {
      if (cudaMalloc(&p, kDebugWords * sizeof(int)) != cudaSuccess) return nullptr;
      if (cudaMemset(p, 0, kDebugWords * sizeof(int)) != cudaSuccess) { cudaFree(p); return nullptr; }
      words[dev].store(p, std::memory_order_release);
    }
  }
  return p;
}

struct GuardList { unsigned long long at[12]; int n; };

// one warp per guard, two words per lane
static __global__ void guard_fill_kernel(unsigned char* ws, GuardList gl) {
  const int gi = blockIdx.x;
  unsigned* g = reinterpret_cast<unsigned*>(ws + gl.at[gi]);
  for (unsigned w = threadIdx.x; w < kGuardBytes / 4; w += blockDim.x) g[w] = kGuardPattern;
}
static __global__ void guard_verify_kernel(const unsigned char* ws, GuardList gl, int* dbg) {
  const int gi = blockIdx.x;
  const unsigned* g = reinterpret_cast<const unsigned*>(ws + gl.at[gi]);
  for (unsigned w = threadIdx.x; w < kGuardBytes / 4; w += blockDim.x) {
    if (g[w] != kGuardPattern) {
      atomicCAS(dbg + DBG_GUARD, 0, gi * 65536 + (int)w + 1);
      atomicOr(dbg + DBG_FLAGS, kDebugGuardFlag);
    }
  }
}
static GuardList guard_list(const Workspace& ws) {
  GuardList gl{};
  gl.n = ws.n_guard;
  for (int i = 0; i < ws.n_guard; ++i) gl.at[i] = ws.guard[i];
  return gl;
}
int debug_fill_guards(const Workspace& ws, void* workspace, cudaStream_t st) {
  if (ws.n_guard == 0) return QALORA_OK;
  guard_fill_kernel<<<ws.n_guard, 32, 0, st>>>(static_cast<unsigned char*>(workspace), guard_list(ws));
  return cuda_status(cudaGetLastError());
}
int debug_verify_guards(const Workspace& ws, const void* workspace, cudaStream_t st) {
  int* dbg = debug_words();
  if (ws.n_guard == 0 || dbg == nullptr) return dbg == nullptr ? QALORA_ERR_CUDA : QALORA_OK;
  guard_verify_kernel<<<ws.n_guard, 32, 0, st>>>(static_cast<const unsigned char*>(workspace), guard_list(ws), dbg);
  return cuda_status(cudaGetLastError());
}
#else
int debug_fill_guards(const Workspace&, void*, cudaStream_t) { return QALORA_OK; }
int debug_verify_guards(const Workspace&, const void*, cudaStream_t) { return QALORA_OK; }
#endif

int check_desc(const qalora_desc* d, Shape* sh) {
  if (d == nullptr) return QALORA_ERR_NULL_POINTER;
  if (d->d_in <= 0 || d->d_out <= 0 || d->group_size <= 0 || d->rank < 0) return QALORA_ERR_INVALID_ARG;
  if (d->bits != 2 && d->bits != 3 && d->bits != 4) return QALORA_ERR_INVALID_ARG;
  if (!(d->scale == d->scale) || d->scale > 3.0e38f || d->scale < -3.0e38f) return QALORA_ERR_INVALID_ARG;
  if (d->group_size % 32 != 0 || d->d_in % d->group_size != 0) return QALORA_ERR_UNSUPPORTED_SHAPE;
  if (d->d_out % 8 != 0) return QALORA_ERR_UNSUPPORTED_SHAPE;
  if (d->rank > 256 || d->rank % 8 != 0) return QALORA_ERR_UNSUPPORTED_SHAPE;
  sh->K = d->d_in; sh->N = d->d_out; sh->g = d->group_size; sh->G = d->d_in / d->group_size;
  sh->bits = d->bits; sh->r = d->rank; sh->s = d->scale; sh->words = words_per_unit(d->bits);
  return QALORA_OK;
}

// Token counts up to this take the bandwidth-bound small-M path.
static constexpr int64_t kSmallM = 16;
// The forward pass alone keeps the few-token kernel up to this many tokens (where its shapes allow).
static constexpr int64_t kFewTokenM = 32;
// Above the few-token range the forward pass takes the kernel with the tokens as the MMA rows
// (where its shapes allow): always up to 64 tokens; from 65 to 128 tokens only for layers with
// 48 to SMs - 1 channel tiles of 128, where the large-tile kernel would have to cut every tile's
// reduction into parts (measured at 65 / 96 / 128 tokens, merged, us per call, this kernel against
// the large-tile one: 22016 -> 8192: 68 / 70 / 71 against 79 / 80 / 81; 8192 -> 22016, 172 tiles:
// 72 / 79 / 86 against 75 / 76 / 77; 4096 -> 4096, 32 tiles: 20.5 / 22.4 / 23.4 against 20.3 /
// 20.4 / 20.5).
static constexpr int64_t kMidMAlways = 64, kMidM = 128;
static bool takes_midm(const Shape& sh, int64_t m) {
  if (m <= kSmallM || m > kMidM || !midm_supported(sh, m)) return false;
  if (m <= kMidMAlways) return true;
  const int tiles = sh.N / 128;
  return tiles >= 48 && tiles < device_sm_count();
}

Workspace workspace_layout(const Shape& sh, int64_t m, int op) {
  Workspace w{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off += round_up(bytes, 256);
    if (kDebugBuild) { w.guard[w.n_guard++] = off; off += kGuardBytes; }
    return at;
  };
  const size_t M = (size_t)(m > 0 ? m : 0);
  const bool train = op == QALORA_OP_TRAIN;           // one workspace for a forward + backward pair
  const bool bwd = op == QALORA_OP_BACKWARD || train;
  w.status = take(256);
  w.xp = take(bwd ? M * sh.G * sizeof(float) : 0);
  w.T = take(M * sh.r * sizeof(float));
  w.dT = take(bwd ? M * sh.r * sizeof(float) : 0);
  w.Tb = take(M * sh.r * sizeof(__nv_bfloat16));
  w.dTb = take(bwd ? M * sh.r * sizeof(__nv_bfloat16) : 0);
  size_t pa = 0, pb = 0;
  if (bwd) {
    pa = atb_partial_bytes(m, sh.G, sh.r);
    pb = atb_partial_bytes(m, sh.r, sh.N);
    if (sh.r >= 8 && sh.r <= 128) {
      const size_t c = tc_dB_partial_bytes(sh, m);
      pb = pb > c ? pb : c;
    }
  }
  w.partial_bytes = pa;
  w.partial = take(pa);
  w.partial_dB_bytes = pb;
  w.partial_dB = take(pb);
  w.dx_parts = take(bwd && m > kSmallM && tc_dx_supported(sh, m) ? tc_dx_partial_bytes(sh, m) : 0);
  // partial results of the tensor-core forward whose reduction is cut into parts; none where the
  // dispatcher takes the few-token kernel (same predicate as in forward_launch)
  const bool few = m <= kFewTokenM && gemv_supported(sh, m);
  size_t parts_bytes = 0;
  if ((!bwd || train) && !few && m > kSmallM) {
    if (takes_midm(sh, m)) parts_bytes = midm_partial_bytes(sh, m);
    else if (tc_forward_supported(sh, m)) parts_bytes = tc_forward_partial_bytes(sh, m);
  }
  w.fwd_parts = take(parts_bytes);
  w.total = off;
  return w;
}


// Argument checks of the forward pass: everything qalora_forward rejects, nothing launched.
int forward_validate(const qalora_desc* desc, int64_t m, const void* x, const void* codes, const float* qparams,
                     const void* A, const void* B, const void* y, const void* workspace, size_t workspace_bytes, int layout_op) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (m < 0 || m > QALORA_MAX_ROWS) return QALORA_ERR_INVALID_ARG;
  if (m == 0) return QALORA_OK;
  if (x == nullptr || codes == nullptr || qparams == nullptr || y == nullptr) return QALORA_ERR_NULL_POINTER;
  if (sh.r > 0 && (A == nullptr || B == nullptr)) return QALORA_ERR_NULL_POINTER;
  if (layout_op == QALORA_OP_TRAIN && sh.r == 0) return QALORA_ERR_INVALID_ARG;
  const Workspace ws = workspace_layout(sh, m, layout_op);
  if (ws.total > 0 && workspace == nullptr) return QALORA_ERR_NULL_POINTER;
  if (workspace_bytes < ws.total) return QALORA_ERR_WORKSPACE_TOO_SMALL;
  if (!aligned16(x) || !aligned16(codes) || !aligned16(qparams) || !aligned16(A) || !aligned16(B) ||
      !aligned16(y) || !aligned16(workspace))
    return QALORA_ERR_MISALIGNED;
  return QALORA_OK;
}

// The forward pass proper, on arguments forward_validate has accepted (m > 0).  The status
// word at the head of the workspace is zeroed before the first kernel that can raise it when
// `reset_status` is set (a public call); qalora_step_host zeroes it once for all its chunks
// and passes false, so that a time-out raised by an earlier chunk survives to the end.
static int forward_dispatch(const Shape& sh, const Workspace& ws, int64_t m, const void* x, const void* codes,
                            const float* qparams, const void* A, const void* B, void* y, void* workspace,
                            cudaStream_t stream, bool reset_status, int layout_op);

int forward_launch(const qalora_desc* desc, int64_t m, const void* x, const void* codes, const float* qparams,
                   const void* A, const void* B, void* y, void* workspace, void* cuda_stream, bool reset_status,
                   int layout_op) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  const Workspace ws = workspace_layout(sh, m, layout_op);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // (bounds-check build: the guards behind the workspace's regions are set before the pass and
  // looked at after its last kernel; both calls are empty otherwise)
  if ((st = debug_fill_guards(ws, workspace, stream)) != QALORA_OK) return st;
  st = forward_dispatch(sh, ws, m, x, codes, qparams, A, B, y, workspace, stream, reset_status, layout_op);
  if (st == QALORA_OK) st = debug_verify_guards(ws, workspace, stream);
  return st;
}

static int forward_dispatch(const Shape& sh, const Workspace& ws, int64_t m, const void* x, const void* codes,
                            const float* qparams, const void* A, const void* B, void* y, void* workspace,
                            cudaStream_t stream, bool reset_status, int layout_op) {
  int st = QALORA_OK;
  char* wsp = static_cast<char*>(workspace);
  float* T = reinterpret_cast<float*>(wsp + ws.T);
  __nv_bfloat16* Tb = reinterpret_cast<__nv_bfloat16*>(wsp + ws.Tb);
  int* status = reinterpret_cast<int*>(wsp + ws.status);
  const bool few = m <= kFewTokenM && gemv_supported(sh, m);
  // The few-token kernel clears the word itself (its first block, long before any wait can
  // expire): a memset node between the pooling kernel and it would undo their overlap.
  if (reset_status && !few && (st = cuda_status(cudaMemsetAsync(status, 0, sizeof(int), stream))) != QALORA_OK) return st;
  if (sh.r > 0) {
    // a forward + backward pair keeps the pooled input too: the backward pass reads it for dA
    float* xp = layout_op == QALORA_OP_TRAIN ? reinterpret_cast<float*>(wsp + ws.xp) : nullptr;
    st = launch_pool_T(sh, m, static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(A),
                       xp, T, Tb, stream);
    if (st != QALORA_OK) return st;
  }
  if (few) {
    return launch_gemv(sh, m, static_cast<const __nv_bfloat16*>(x), static_cast<const uint32_t*>(codes),
                       reinterpret_cast<const float2*>(qparams), sh.r > 0 ? Tb : nullptr,
                       static_cast<const __nv_bfloat16*>(B), static_cast<__nv_bfloat16*>(y), status, reset_status, stream);
  }
  if (takes_midm(sh, m)) {
    return launch_midm(sh, m, static_cast<const __nv_bfloat16*>(x), static_cast<const uint32_t*>(codes),
                       reinterpret_cast<const float2*>(qparams), Tb, static_cast<const __nv_bfloat16*>(B),
                       static_cast<__nv_bfloat16*>(y), reinterpret_cast<float*>(wsp + ws.fwd_parts), status, stream);
  }
  if (m > kSmallM && tc_forward_supported(sh, m)) {
    return launch_tc_forward(sh, m, static_cast<const __nv_bfloat16*>(x), static_cast<const uint32_t*>(codes),
                             reinterpret_cast<const float2*>(qparams), Tb, static_cast<const __nv_bfloat16*>(B),
                             static_cast<__nv_bfloat16*>(y), reinterpret_cast<float*>(wsp + ws.fwd_parts), status, stream);
  }
  return launch_simt_forward(sh, m, static_cast<const __nv_bfloat16*>(x), static_cast<const uint32_t*>(codes),
                             reinterpret_cast<const float2*>(qparams), T, static_cast<const __nv_bfloat16*>(B),
                             static_cast<__nv_bfloat16*>(y), stream);
}

// A second stream of the library's own, per host thread and device, for the one place where two
// HBM-bound kernels of a pass are independent (dB beside dT): forked from and joined to the
// caller's stream with events, so the caller sees one stream-ordered call.  Created on first use
// and kept; NULL when it cannot be had (the pass then runs in one stream).  During a stream
// capture of the caller's the fork/join pattern is captured like any other.
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
};
static SideStream* side_stream() {
  static thread_local SideStream per_device[kMaxDevices];
  const int dev = current_device();
  if (dev < 0) return nullptr;
  SideStream& s = per_device[dev];
  if (s.stream == nullptr) {
    cudaStream_t st = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    if (cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&a, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&b, cudaEventDisableTiming) != cudaSuccess) {
      if (a != nullptr) cudaEventDestroy(a);
      cudaStreamDestroy(st);
      return nullptr;
    }
    s.stream = st; s.fork = a; s.join = b;
  }
  return &s;
}

int backward_impl(const qalora_desc* desc, int64_t m, const void* x, const void* dy,
                  const void* codes, const float* qparams, const void* A, const void* B,
                  void* dx, float* dA, float* dB,
                  void* workspace, size_t workspace_bytes, void* cuda_stream, bool reset_status, bool pooled) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (m < 0 || m > QALORA_MAX_ROWS || sh.r == 0) return QALORA_ERR_INVALID_ARG;
  if (x == nullptr || dy == nullptr || codes == nullptr || qparams == nullptr || A == nullptr || B == nullptr)
    return QALORA_ERR_NULL_POINTER;
  // `pooled`: the workspace is the one qalora_forward_train filled for the same x, A and m; its
  // pooled input, T and bf16(T) are taken as they are
  const Workspace ws = workspace_layout(sh, m, pooled ? QALORA_OP_TRAIN : QALORA_OP_BACKWARD);
  if (ws.total > 0 && workspace == nullptr) return QALORA_ERR_NULL_POINTER;
  if (workspace_bytes < ws.total) return QALORA_ERR_WORKSPACE_TOO_SMALL;
  if (!aligned16(x) || !aligned16(dy) || !aligned16(codes) || !aligned16(qparams) || !aligned16(A) ||
      !aligned16(B) || !aligned16(dx) || !aligned16(dA) || !aligned16(dB) || !aligned16(workspace))
    return QALORA_ERR_MISALIGNED;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  char* wsp = static_cast<char*>(workspace);
  float* xp = reinterpret_cast<float*>(wsp + ws.xp);
  float* T = reinterpret_cast<float*>(wsp + ws.T);
  float* dT = reinterpret_cast<float*>(wsp + ws.dT);
  __nv_bfloat16* Tb = reinterpret_cast<__nv_bfloat16*>(wsp + ws.Tb);
  __nv_bfloat16* dTb = reinterpret_cast<__nv_bfloat16*>(wsp + ws.dTb);
  float* partial = reinterpret_cast<float*>(wsp + ws.partial);
  float* partial_dB = reinterpret_cast<float*>(wsp + ws.partial_dB);
  const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
  const __nv_bfloat16* dyb = static_cast<const __nv_bfloat16*>(dy);
  const __nv_bfloat16* Ab = static_cast<const __nv_bfloat16*>(A);
  const __nv_bfloat16* Bb = static_cast<const __nv_bfloat16*>(B);

  if (m == 0) {
    if (dA != nullptr && (st = cuda_status(cudaMemsetAsync(dA, 0, (size_t)sh.G * sh.r * sizeof(float), stream)))) return st;
    if (dB != nullptr && (st = cuda_status(cudaMemsetAsync(dB, 0, (size_t)sh.r * sh.N * sizeof(float), stream)))) return st;
    return QALORA_OK;
  }
  int* status = reinterpret_cast<int*>(wsp + ws.status);
  if (reset_status && (st = cuda_status(cudaMemsetAsync(status, 0, sizeof(int), stream))) != QALORA_OK) return st;
  // (bounds-check build: a pass on its own sets the guards; after qalora_forward_train they are already set)
  if (!pooled && (st = debug_fill_guards(ws, workspace, stream)) != QALORA_OK) return st;
  const bool aux_tc = m > kSmallM && tc_aux_supported(sh, m);
  if (!pooled && (dA != nullptr || dB != nullptr)) {
    if ((st = launch_pool_T(sh, m, xb, Ab, xp, T, Tb, stream)) != QALORA_OK) return st;
  }
  // dB = T^T dy needs only T (from the forward pass or the pooling above) and dy; dT = s dy B^T
  // needs only dy and B.  Both stream dy once at little more than half the copy rate with one
  // block per SM, so they run side by side: dB (and its fixed-order sum) on the library's second
  // stream, dT and then dA on the caller's, joined before dx, the long kernel that fills every SM.
  // A gradient of up to about the size of L2 comes from DRAM once for the two, and dx starts on a
  // warm dy.  (Few rows, where these are small CUDA-core kernels: one stream.)
  SideStream* side = (dB != nullptr && aux_tc) ? side_stream() : nullptr;
  cudaStream_t dB_stream = stream;
  if (side != nullptr) {
    if (cudaEventRecord(side->fork, stream) != cudaSuccess || cudaStreamWaitEvent(side->stream, side->fork, 0) != cudaSuccess)
      return QALORA_ERR_CUDA;
    dB_stream = side->stream;
  }
  if (dB != nullptr) {
    if (aux_tc) {
      int splits = 0;
      st = launch_tc_dB_partials(sh, m, Tb, dyb, partial_dB, &splits, status, dB_stream);
      if (st == QALORA_OK) st = launch_sum_partials(partial_dB, dB, (size_t)sh.r * sh.N, splits, dB_stream);
    } else {
      st = launch_atb_bf16(m, sh.r, sh.N, T, dyb, dB, partial_dB, ws.partial_dB_bytes, dB_stream);
    }
    if (side != nullptr && cudaEventRecord(side->join, side->stream) != cudaSuccess) st = QALORA_ERR_CUDA;
  }
  if (st == QALORA_OK) {
    if (aux_tc) st = launch_tc_dT(sh, m, dyb, Bb, dT, dTb, status, stream);
    else st = launch_dT(sh, m, dyb, Bb, dT, dTb, stream);
  }
  if (st == QALORA_OK && dA != nullptr) st = launch_atb_f32(m, sh.G, sh.r, xp, dT, dA, partial, ws.partial_bytes, stream);
  // join: everything after this point, in the call and after it, is ordered behind dB as well
  // (also when a launch above failed, so that no work of this call is left outside the caller's stream)
  if (side != nullptr && cudaStreamWaitEvent(stream, side->join, 0) != cudaSuccess) return QALORA_ERR_CUDA;
  if (st != QALORA_OK) return st;
  if (dx != nullptr && m > kSmallM && tc_dx_supported(sh, m)) {
    st = launch_tc_dx(sh, m, dyb, static_cast<const uint32_t*>(codes), reinterpret_cast<const float2*>(qparams),
                      dTb, Ab, static_cast<__nv_bfloat16*>(dx), reinterpret_cast<float*>(wsp + ws.dx_parts), status, stream);
    if (st != QALORA_OK) return st;
  } else if (dx != nullptr) {
    st = launch_simt_dx(sh, m, dyb, static_cast<const uint32_t*>(codes), reinterpret_cast<const float2*>(qparams),
                        dT, Ab, static_cast<__nv_bfloat16*>(dx), stream);
    if (st != QALORA_OK) return st;
  }
  return debug_verify_guards(ws, workspace, stream);
}

}  // namespace qalora

using namespace qalora;


extern "C" {

int qalora_version(void) { return 100 + QALORA_LAYOUT_VERSION; }

uint64_t qalora_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int qalora_profile_next_main_kernel(void* start_event, void* stop_event) {
  t_probe_start = static_cast<cudaEvent_t>(start_event);
  t_probe_stop = static_cast<cudaEvent_t>(stop_event);
  return QALORA_OK;
}

const char* qalora_main_kernel_name(void) { return t_main_kernel; }

// Test hook, deliberately not declared in the public header.  Arms the NEXT few-token
// forward launch of this process so that each of its producers stops after `stages` stages
// and its waits give up after `limit_ns` nanoseconds: the consumers' bounded waits then
// expire, the status word is raised and the kernel leaves in the ordinary way.  Nothing
// faults, traps or spins without bound.
int qalora_debug_expire_next_few_token_wait(int stages, uint64_t limit_ns) {
  if (limit_ns == 0 || limit_ns > 2000000000ull) return QALORA_ERR_INVALID_ARG;
  arm_few_token_wait_expiry(stages, limit_ns);
  return QALORA_OK;
}

// The same for the tensor-core forward / dX kernels: the next such launch of this process has
// its activation producers stop after `steps` reduction steps, and its waits give up after
// `limit_ns`.  Test hook, not declared in the public header.
int qalora_debug_expire_next_tc_wait(int steps, uint64_t limit_ns) {
  if (limit_ns == 0 || limit_ns > 2000000000ull) return QALORA_ERR_INVALID_ARG;
  arm_tc_wait_expiry(steps, limit_ns);
  return QALORA_OK;
}

int qalora_debug_checks(void) { return kDebugBuild ? 1 : 0; }

// Test hook, not declared in the public header: shows that the bounds-check build's record
// works, without any access outside a buffer.  `buf512` is 512 bytes of device memory used as
// a one-region workspace (region [0, 256), guard [256, 512)).  The guard is filled, one kernel
// then (a) asks for index 5 of an array of 4, which the check refuses and records, and (b)
// overwrites word 3 of the guard, which lies inside the buffer; the verification finds it.
// Afterwards qalora_debug_report() reads flags 6, index 5, limit 4, one failed check, guard 4.
#ifdef QALORA_DEBUG
static __global__ void debug_selftest_kernel(unsigned* buf, int* dbg) {
  if (QALORA_CHECK(dbg, 5, 4)) buf[5] = 0u;          // never taken
  buf[kGuardBytes / 4 + 3] = 0u;                      // inside the buffer: the guard's word 3
}
#endif
int qalora_debug_selftest(void* buf512, void* cuda_stream) {
#ifdef QALORA_DEBUG
  if (buf512 == nullptr) return QALORA_ERR_NULL_POINTER;
  if (!aligned16(buf512)) return QALORA_ERR_MISALIGNED;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  Workspace ws{};
  ws.guard[0] = kGuardBytes;
  ws.n_guard = 1;
  int* dbg = debug_words();
  if (dbg == nullptr) return QALORA_ERR_CUDA;
  int rc = debug_fill_guards(ws, buf512, st);
  if (rc != QALORA_OK) return rc;
  debug_selftest_kernel<<<1, 1, 0, st>>>(static_cast<unsigned*>(buf512), dbg);
  if (cudaGetLastError() != cudaSuccess) return QALORA_ERR_CUDA;
  return debug_verify_guards(ws, buf512, st);
#else
  (void)buf512; (void)cuda_stream;
  return QALORA_ERR_INVALID_ARG;
#endif
}

int qalora_debug_report(int32_t* words8) {
  if (words8 == nullptr) return QALORA_ERR_NULL_POINTER;
  for (int i = 0; i < kDebugWords; ++i) words8[i] = 0;
  if (!kDebugBuild) return QALORA_OK;
  int* dbg = debug_words();
  if (dbg == nullptr) return QALORA_ERR_CUDA;
  if (cudaDeviceSynchronize() != cudaSuccess) return QALORA_ERR_CUDA;
  if (cudaMemcpy(words8, dbg, kDebugWords * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return QALORA_ERR_CUDA;
  return cuda_status(cudaMemset(dbg, 0, kDebugWords * sizeof(int)));
}

const char* qalora_status_string(int status) {
  switch (status) {
    case QALORA_OK: return "ok";
    case QALORA_ERR_INVALID_ARG: return "invalid argument";
    case QALORA_ERR_NULL_POINTER: return "null pointer";
    case QALORA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case QALORA_ERR_MISALIGNED: return "pointer not 16-byte aligned";
    case QALORA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case QALORA_ERR_CUDA: return "CUDA error";
    case QALORA_ERR_STATIC_SCRATCH_EXCEEDED: return "request exceeds the built-in scratch of qalora_forward_static";
    default: return "unknown status";
  }
}

int qalora_packed_bytes(const qalora_desc* desc, size_t* code_bytes, size_t* qparam_bytes) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (code_bytes == nullptr || qparam_bytes == nullptr) return QALORA_ERR_NULL_POINTER;
  *code_bytes = (size_t)(sh.K / 32) * sh.N * sh.words * sizeof(uint32_t);
  *qparam_bytes = (size_t)sh.G * sh.N * 2 * sizeof(float);
  return QALORA_OK;
}

int qalora_workspace_bytes(const qalora_desc* desc, int64_t m, int op, size_t* bytes) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (bytes == nullptr) return QALORA_ERR_NULL_POINTER;
  if (m < 0 || m > QALORA_MAX_ROWS || (op != QALORA_OP_FORWARD && op != QALORA_OP_BACKWARD && op != QALORA_OP_TRAIN)) return QALORA_ERR_INVALID_ARG;
  *bytes = workspace_layout(sh, m, op).total;
  return QALORA_OK;
}

int qalora_quantize(const qalora_desc* desc, const float* W, void* codes, float* qparams,
                    int32_t* dev_status, void* cuda_stream) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (W == nullptr || codes == nullptr || qparams == nullptr) return QALORA_ERR_NULL_POINTER;
  if (!aligned16(W) || !aligned16(codes) || !aligned16(qparams)) return QALORA_ERR_MISALIGNED;
  if (dev_status != nullptr && (reinterpret_cast<uintptr_t>(dev_status) & 3u)) return QALORA_ERR_MISALIGNED;
  return launch_quantize(sh, W, static_cast<uint32_t*>(codes), reinterpret_cast<float2*>(qparams), dev_status,
                         static_cast<cudaStream_t>(cuda_stream));
}

int qalora_merge(const qalora_desc* desc, const float* qparams_in, const void* A, const void* B,
                 float* qparams_out, void* cuda_stream) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (qparams_in == nullptr || qparams_out == nullptr) return QALORA_ERR_NULL_POINTER;
  if (sh.r > 0 && (A == nullptr || B == nullptr)) return QALORA_ERR_NULL_POINTER;
  if (!aligned16(qparams_in) || !aligned16(qparams_out) || !aligned16(A) || !aligned16(B)) return QALORA_ERR_MISALIGNED;
  return launch_merge(sh, reinterpret_cast<const float2*>(qparams_in), static_cast<const __nv_bfloat16*>(A),
                      static_cast<const __nv_bfloat16*>(B), reinterpret_cast<float2*>(qparams_out),
                      static_cast<cudaStream_t>(cuda_stream));
}

int qalora_forward(const qalora_desc* desc, int64_t m, const void* x, const void* codes,
                   const float* qparams, const void* A, const void* B, void* y,
                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int st = forward_validate(desc, m, x, codes, qparams, A, B, y, workspace, workspace_bytes, QALORA_OP_FORWARD);
  if (st != QALORA_OK || m == 0) return st;
  return forward_launch(desc, m, x, codes, qparams, A, B, y, workspace, cuda_stream, /*reset_status=*/true, QALORA_OP_FORWARD);
}

int qalora_forward_train(const qalora_desc* desc, int64_t m, const void* x, const void* codes,
                         const float* qparams, const void* A, const void* B, void* y,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int st = forward_validate(desc, m, x, codes, qparams, A, B, y, workspace, workspace_bytes, QALORA_OP_TRAIN);
  if (st != QALORA_OK || m == 0) return st;
  return forward_launch(desc, m, x, codes, qparams, A, B, y, workspace, cuda_stream, /*reset_status=*/true, QALORA_OP_TRAIN);
}

int qalora_backward_train(const qalora_desc* desc, int64_t m, const void* x, const void* dy,
                          const void* codes, const float* qparams, const void* A, const void* B,
                          void* dx, float* dA, float* dB,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return backward_impl(desc, m, x, dy, codes, qparams, A, B, dx, dA, dB, workspace, workspace_bytes, cuda_stream,
                       /*reset_status=*/false, /*pooled=*/true);
}

int qalora_forward_group_workspace_bytes(const qalora_group_layer* layers, int n, int64_t m, size_t* bytes) {
  if (layers == nullptr || bytes == nullptr) return QALORA_ERR_NULL_POINTER;
  if (n < 0 || m < 0 || m > QALORA_MAX_ROWS) return QALORA_ERR_INVALID_ARG;
  size_t need = 256;                                 // the status word
  for (int i = 0; i < n; ++i) {
    Shape sh;
    int st = check_desc(&layers[i].desc, &sh);
    if (st != QALORA_OK) return st;
    const size_t w = workspace_layout(sh, m, QALORA_OP_FORWARD).total;
    need = w > need ? w : need;
  }
  *bytes = need;
  return QALORA_OK;
}

int qalora_forward_group(const qalora_group_layer* layers, int n, int64_t m,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (layers == nullptr) return QALORA_ERR_NULL_POINTER;
  if (n < 0 || m < 0 || m > QALORA_MAX_ROWS) return QALORA_ERR_INVALID_ARG;
  size_t need = 0;
  int st = qalora_forward_group_workspace_bytes(layers, n, m, &need);
  if (st != QALORA_OK) return st;
  // every layer's arguments are checked before anything is launched
  for (int i = 0; i < n; ++i) {
    const qalora_group_layer& L = layers[i];
    st = forward_validate(&L.desc, m, L.x, L.codes, L.qparams, L.A, L.B, L.y, workspace, workspace_bytes, QALORA_OP_FORWARD);
    if (st != QALORA_OK) return st;
  }
  if (n == 0 || m == 0) return QALORA_OK;
  if (workspace == nullptr) return QALORA_ERR_NULL_POINTER;
  if (workspace_bytes < need) return QALORA_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  constexpr int kMaxGroup = 8;
  GemvGroupItem items[kMaxGroup];
  bool one_launch = n <= kMaxGroup;
  for (int i = 0; i < n && one_launch; ++i) {
    check_desc(&layers[i].desc, &items[i].sh);
    items[i].x = static_cast<const __nv_bfloat16*>(layers[i].x);
    items[i].codes = static_cast<const uint32_t*>(layers[i].codes);
    items[i].qparams = reinterpret_cast<const float2*>(layers[i].qparams);
    items[i].y = static_cast<__nv_bfloat16*>(layers[i].y);
  }
  one_launch = one_launch && gemv_group_supported(items, n, m);
  if (one_launch) return launch_gemv_group(items, n, m, static_cast<int*>(workspace), /*reset_status=*/true, stream);
  // Otherwise (adapters, more than 16 rows, mixed bit widths, shapes the few-token kernel does
  // not tile, more than 8 layers): one forward pass per layer, sharing the workspace; the status
  // word is cleared once and only ever raised.
  if ((st = cuda_status(cudaMemsetAsync(workspace, 0, sizeof(int), stream))) != QALORA_OK) return st;
  for (int i = 0; i < n; ++i) {
    const qalora_group_layer& L = layers[i];
    st = forward_launch(&L.desc, m, L.x, L.codes, L.qparams, L.A, L.B, L.y, workspace, cuda_stream, /*reset_status=*/false,
                        QALORA_OP_FORWARD);
    if (st != QALORA_OK) return st;
  }
  return QALORA_OK;
}

int qalora_backward(const qalora_desc* desc, int64_t m, const void* x, const void* dy,
                    const void* codes, const float* qparams, const void* A, const void* B,
                    void* dx, float* dA, float* dB,
                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return backward_impl(desc, m, x, dy, codes, qparams, A, B, dx, dA, dB, workspace, workspace_bytes, cuda_stream,
                       /*reset_status=*/true, /*pooled=*/false);
}


namespace {
// qalora_step_host cuts the rows into chunks so that the copy of one chunk to the
// device, the kernels of another and the copy of a third back to the host run at
// the same time (the link is full duplex).  A chunk is a multiple of 256 rows and at
// least kStepChunkMin rows long, so that every chunk takes the same large-M kernels
// as the whole batch would; batches below two such chunks stay in one piece.
constexpr int kStepMaxChunks = 8;
constexpr int64_t kStepChunkMin = 1024;
int64_t step_chunk_rows(int64_t m) {
  if (m < 2 * kStepChunkMin) return m > 0 ? m : 1;
  int64_t rows = round_up((size_t)((m + kStepMaxChunks - 1) / kStepMaxChunks), 256);
  return rows < kStepChunkMin ? kStepChunkMin : rows;
}

struct StepLayout { size_t ws, x, dy, y, dx, dA, dB, dA_parts, dB_parts, total, ws_bytes; int chunks; int64_t rows; };
StepLayout step_layout(const Shape& sh, int64_t m) {
  StepLayout L{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t at = off; off += round_up(bytes, 256); return at; };
  const size_t M = (size_t)m;
  L.rows = step_chunk_rows(m);
  L.chunks = m > 0 ? (int)((m + L.rows - 1) / L.rows) : 1;
  // (a shorter last chunk may take another kernel, whose scratch can be LARGER than a full chunk's:
  // few rows have their reduction cut into parts with fp32 partial results)
  const int64_t last_rows = m > 0 ? m - (int64_t)(L.chunks - 1) * L.rows : L.rows;
  L.ws_bytes = std::max(workspace_layout(sh, L.rows, QALORA_OP_TRAIN).total, workspace_layout(sh, last_rows, QALORA_OP_TRAIN).total);
  L.ws = take(L.ws_bytes);                         // first: the status word sits at the head of the staging area
  L.x = take(M * sh.K * 2); L.dy = take(M * sh.N * 2); L.y = take(M * sh.N * 2); L.dx = take(M * sh.K * 2);
  L.dA = take((size_t)sh.G * sh.r * 4); L.dB = take((size_t)sh.r * sh.N * 4);
  L.dA_parts = take(L.chunks > 1 ? (size_t)L.chunks * sh.G * sh.r * 4 : 0);
  L.dB_parts = take(L.chunks > 1 ? (size_t)L.chunks * sh.r * sh.N * 4 : 0);
  L.total = off;
  return L;
}

// Copy streams and events of one device, made on first use and kept for the life of
// the process.  An event may be recorded again while an earlier wait on it is still
// pending: a wait refers to the record that preceded it.
struct StepPipes {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, done = nullptr;
  cudaEvent_t x[kStepMaxChunks], dy[kStepMaxChunks], fwd[kStepMaxChunks], bwd[kStepMaxChunks];
};
constexpr int kMaxDevices = 64;
std::mutex g_step_mutex;
StepPipes g_step_pipes[kMaxDevices];

StepPipes* step_pipes_locked() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  StepPipes& P = g_step_pipes[dev];
  if (P.ready) return &P;
  bool ok = cudaStreamCreateWithFlags(&P.in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&P.out, cudaStreamNonBlocking) == cudaSuccess;
  auto make = [&](cudaEvent_t* e) { ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
  make(&P.start); make(&P.done);
  for (int i = 0; i < kStepMaxChunks; ++i) { make(&P.x[i]); make(&P.dy[i]); make(&P.fwd[i]); make(&P.bwd[i]); }
  if (!ok) return nullptr;
  P.ready = true;
  return &P;
}

}  // namespace

int qalora_step_host_bytes(const qalora_desc* desc, int64_t m, size_t* bytes) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (bytes == nullptr) return QALORA_ERR_NULL_POINTER;
  if (m < 0 || m > QALORA_MAX_ROWS) return QALORA_ERR_INVALID_ARG;
  *bytes = step_layout(sh, m).total;
  return QALORA_OK;
}

int qalora_step_host(const qalora_desc* desc, int64_t m, const void* x_host, const void* dy_host,
                     const void* codes, const float* qparams, const void* A, const void* B,
                     void* y_host, void* dx_host, float* dA_host, float* dB_host,
                     void* staging, size_t staging_bytes, void* cuda_stream) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (m < 0 || m > QALORA_MAX_ROWS || sh.r == 0) return QALORA_ERR_INVALID_ARG;
  if (x_host == nullptr || dy_host == nullptr || y_host == nullptr || dx_host == nullptr || dA_host == nullptr ||
      dB_host == nullptr || staging == nullptr)
    return QALORA_ERR_NULL_POINTER;
  if (!aligned16(staging)) return QALORA_ERR_MISALIGNED;
  const StepLayout L = step_layout(sh, m);
  if (staging_bytes < L.total) return QALORA_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(staging);
  const size_t nA = (size_t)sh.G * sh.r, nB = (size_t)sh.r * sh.N;
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };

  std::lock_guard<std::mutex> lock(g_step_mutex);
  StepPipes* P = step_pipes_locked();
  if (P == nullptr) return QALORA_ERR_CUDA;
  // one status word for the whole call: cleared here, only ever raised by the chunks' kernels
  if (!ok(cudaMemsetAsync(base + L.ws, 0, sizeof(int), stream))) return QALORA_ERR_CUDA;
  // The copy streams start after everything already enqueued on the caller's stream.
  if (!ok(cudaEventRecord(P->start, stream)) || !ok(cudaStreamWaitEvent(P->in, P->start, 0)) ||
      !ok(cudaStreamWaitEvent(P->out, P->start, 0)))
    return QALORA_ERR_CUDA;
  for (int c = 0; c < L.chunks; ++c) {
    const size_t r0 = (size_t)c * L.rows;
    const int64_t rows = (int64_t)((size_t)m - r0 < (size_t)L.rows ? (size_t)m - r0 : (size_t)L.rows);
    const size_t xo = r0 * sh.K * 2, yo = r0 * sh.N * 2, xb = (size_t)rows * sh.K * 2, yb = (size_t)rows * sh.N * 2;
    float* dA_c = reinterpret_cast<float*>(base + (L.chunks > 1 ? L.dA_parts + c * nA * 4 : L.dA));
    float* dB_c = reinterpret_cast<float*>(base + (L.chunks > 1 ? L.dB_parts + c * nB * 4 : L.dB));
    if (!ok(cudaMemcpyAsync(base + L.x + xo, static_cast<const char*>(x_host) + xo, xb, cudaMemcpyHostToDevice, P->in)) ||
        !ok(cudaEventRecord(P->x[c], P->in)) ||
        !ok(cudaMemcpyAsync(base + L.dy + yo, static_cast<const char*>(dy_host) + yo, yb, cudaMemcpyHostToDevice, P->in)) ||
        !ok(cudaEventRecord(P->dy[c], P->in)) || !ok(cudaStreamWaitEvent(stream, P->x[c], 0)))
      return QALORA_ERR_CUDA;
    // (forward and backward of a chunk share the workspace: the pooled input is computed once)
    st = forward_validate(desc, rows, base + L.x + xo, codes, qparams, A, B, base + L.y + yo, base + L.ws, L.ws_bytes,
                          QALORA_OP_TRAIN);
    if (st == QALORA_OK)
      st = forward_launch(desc, rows, base + L.x + xo, codes, qparams, A, B, base + L.y + yo, base + L.ws, cuda_stream,
                          /*reset_status=*/false, QALORA_OP_TRAIN);
    if (st != QALORA_OK) return st;
    if (!ok(cudaEventRecord(P->fwd[c], stream)) || !ok(cudaStreamWaitEvent(stream, P->dy[c], 0))) return QALORA_ERR_CUDA;
    st = backward_impl(desc, rows, base + L.x + xo, base + L.dy + yo, codes, qparams, A, B, base + L.dx + xo, dA_c, dB_c,
                       base + L.ws, L.ws_bytes, cuda_stream, /*reset_status=*/false, /*pooled=*/true);
    if (st != QALORA_OK) return st;
    if (!ok(cudaEventRecord(P->bwd[c], stream)) || !ok(cudaStreamWaitEvent(P->out, P->fwd[c], 0)) ||
        !ok(cudaMemcpyAsync(static_cast<char*>(y_host) + yo, base + L.y + yo, yb, cudaMemcpyDeviceToHost, P->out)) ||
        !ok(cudaStreamWaitEvent(P->out, P->bwd[c], 0)) ||
        !ok(cudaMemcpyAsync(static_cast<char*>(dx_host) + xo, base + L.dx + xo, xb, cudaMemcpyDeviceToHost, P->out)))
      return QALORA_ERR_CUDA;
  }
  if (L.chunks > 1) {   // dA, dB = the chunks' results added in chunk order
    st = launch_sum_partials(reinterpret_cast<const float*>(base + L.dA_parts), reinterpret_cast<float*>(base + L.dA), nA,
                             L.chunks, stream);
    if (st != QALORA_OK) return st;
    st = launch_sum_partials(reinterpret_cast<const float*>(base + L.dB_parts), reinterpret_cast<float*>(base + L.dB), nB,
                             L.chunks, stream);
    if (st != QALORA_OK) return st;
  }
  if (!ok(cudaMemcpyAsync(dA_host, base + L.dA, nA * 4, cudaMemcpyDeviceToHost, stream)) ||
      !ok(cudaMemcpyAsync(dB_host, base + L.dB, nB * 4, cudaMemcpyDeviceToHost, stream)))
    return QALORA_ERR_CUDA;
  // The caller's stream ends after the last copy back to the host.
  if (!ok(cudaEventRecord(P->done, P->out)) || !ok(cudaStreamWaitEvent(stream, P->done, 0))) return QALORA_ERR_CUDA;
  return QALORA_OK;
}

int qalora_dequantize(const qalora_desc* desc, const void* codes, const float* qparams, void* W,
                      int out_bf16, void* cuda_stream) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (codes == nullptr || qparams == nullptr || W == nullptr) return QALORA_ERR_NULL_POINTER;
  if (!aligned16(codes) || !aligned16(qparams) || !aligned16(W)) return QALORA_ERR_MISALIGNED;
  return launch_dequantize(sh, static_cast<const uint32_t*>(codes), reinterpret_cast<const float2*>(qparams), W,
                           out_bf16 != 0, static_cast<cudaStream_t>(cuda_stream));
}

int qalora_qparams_from_zero_point(const qalora_desc* desc, const float* alpha, const float* zero,
                                   float* qparams, void* cuda_stream) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (alpha == nullptr || zero == nullptr || qparams == nullptr) return QALORA_ERR_NULL_POINTER;
  if (!aligned16(alpha) || !aligned16(zero) || !aligned16(qparams)) return QALORA_ERR_MISALIGNED;
  return launch_from_zero_point(sh, alpha, zero, reinterpret_cast<float2*>(qparams), static_cast<cudaStream_t>(cuda_stream));
}

int qalora_qparams_to_zero_point(const qalora_desc* desc, const float* qparams, float* alpha,
                                 float* zero, void* cuda_stream) {
  Shape sh;
  int st = check_desc(desc, &sh);
  if (st != QALORA_OK) return st;
  if (alpha == nullptr || zero == nullptr || qparams == nullptr) return QALORA_ERR_NULL_POINTER;
  if (!aligned16(alpha) || !aligned16(zero) || !aligned16(qparams)) return QALORA_ERR_MISALIGNED;
  return launch_to_zero_point(sh, reinterpret_cast<const float2*>(qparams), alpha, zero, static_cast<cudaStream_t>(cuda_stream));
}

int qalora_adamw_workspace_bytes(size_t* bytes) {
  if (bytes == nullptr) return QALORA_ERR_NULL_POINTER;
  *bytes = adamw_workspace_bytes();
  return QALORA_OK;
}

int qalora_adamw_step(const qalora_adamw_hyper* hyper, int64_t n, const float* grad, float* param,
                      float* exp_avg, float* exp_avg_sq, void* param_bf16, float* norm_out,
                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (hyper == nullptr) return QALORA_ERR_NULL_POINTER;
  auto finite_nonneg = [](float v) { return v >= 0.f && v <= 3.0e38f; };   // false for NaN
  if (n < 0 || hyper->step < 1 || !(hyper->beta1 >= 0.f && hyper->beta1 < 1.f) ||
      !(hyper->beta2 >= 0.f && hyper->beta2 < 1.f) || !finite_nonneg(hyper->lr) || !finite_nonneg(hyper->eps) ||
      !finite_nonneg(hyper->weight_decay) || !(hyper->max_grad_norm == hyper->max_grad_norm))
    return QALORA_ERR_INVALID_ARG;
  if (n == 0) return QALORA_OK;
  if (grad == nullptr || param == nullptr || exp_avg == nullptr || exp_avg_sq == nullptr || param_bf16 == nullptr ||
      workspace == nullptr)
    return QALORA_ERR_NULL_POINTER;
  if (!aligned16(grad) || !aligned16(param) || !aligned16(exp_avg) || !aligned16(exp_avg_sq) || !aligned16(param_bf16) ||
      !aligned16(workspace) || (norm_out != nullptr && (reinterpret_cast<uintptr_t>(norm_out) & 3u)))
    return QALORA_ERR_MISALIGNED;
  if (workspace_bytes < adamw_workspace_bytes()) return QALORA_ERR_WORKSPACE_TOO_SMALL;
  AdamwArgs a{hyper->lr, hyper->beta1, hyper->beta2, hyper->eps, hyper->weight_decay, hyper->max_grad_norm, hyper->step};
  return launch_adamw(a, n, grad, param, exp_avg, exp_avg_sq, static_cast<__nv_bfloat16*>(param_bf16),
                      static_cast<float*>(workspace), norm_out, static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"
