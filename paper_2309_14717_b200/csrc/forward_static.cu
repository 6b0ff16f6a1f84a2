// qalora_forward_static: the forward pass for callers that cannot allocate
// device memory.  The scratch that qalora_forward takes from a caller-owned
// workspace lives here in a fixed array inside the library's own device image.
#include <mutex>

#include "common.cuh"

namespace {

// The scratch itself.  Every GPU that loads this library carries these bytes
// from the moment its module is loaded until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[QALORA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// In host code `g_static_scratch` is only a handle for the runtime, not a device
// address; the address a kernel can use has to be asked for, once per device,
// while that device is current.
int static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return QALORA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return QALORA_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return QALORA_OK;
}

}  // namespace

extern "C" int qalora_forward_static(const qalora_desc* desc, int64_t m, const void* x, const void* codes,
                                     const float* qparams, const void* A, const void* B, void* y,
                                     void* cuda_stream) {
  size_t need = 0;
  int st = qalora_workspace_bytes(desc, m, QALORA_OP_FORWARD, &need);
  if (st != QALORA_OK) return st;
  if (need > (size_t)QALORA_STATIC_SCRATCH_BYTES) return QALORA_ERR_STATIC_SCRATCH_EXCEEDED;
  // every check of qalora_forward first, against a stand-in for the (256-byte aligned) array:
  // a rejected call must not have enqueued anything, nor touched the CUDA runtime
  alignas(16) static const char aligned_stand_in = 0;
  if ((st = qalora::forward_validate(desc, m, x, codes, qparams, A, B, y, &aligned_stand_in,
                                     (size_t)QALORA_STATIC_SCRATCH_BYTES, QALORA_OP_FORWARD)) != QALORA_OK)
    return st;
  if (m == 0) return QALORA_OK;
  void* scratch = nullptr;
  if ((st = static_scratch_address(&scratch)) != QALORA_OK) return st;
  // The array keeps whatever the previous call left in it.  The only part that has
  // to start from zero is the status word at its head; everything else is written
  // before it is read.
  if (cudaMemsetAsync(scratch, 0, 256, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return QALORA_ERR_CUDA;
  return qalora_forward(desc, m, x, codes, qparams, A, B, y, scratch, (size_t)QALORA_STATIC_SCRATCH_BYTES,
                        cuda_stream);
}
