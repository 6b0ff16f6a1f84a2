// Bounds-check build of the library (-DQALORA_DEBUG; `python -m paper_2309_14717_b200.build --debug`
// makes libqalora_debug.so beside the ordinary one).
//
// QALORA_CHECK(dbg, index, limit) guards an access whose index (an offset into a global
// array or a workspace region, a byte offset into the shared-memory window, a column of tensor
// memory, a TMA coordinate) is COMPUTED by the kernel: the access runs only when
// 0 <= index < limit.  A failed check never faults: it records the place (translation unit
// and source line), the index and the limit in the library's record words, counts itself, and
// the access is skipped.  The same build puts a guard region of 256 bytes behind every
// region of a workspace, fills it before a pass and verifies it after the pass's last kernel.
// The record is read (and cleared) with qalora_debug_report().
//
// Without the define QALORA_CHECK is constantly true, debug_words() is a null pointer
// and nothing of this costs a register or an instruction.
#pragma once
#include <cuda_runtime.h>

namespace qalora {

// Layout of the eight int32 record words.
enum DebugWord {
  DBG_FLAGS = 0,        // bit 1 (value 2): an index check failed; bit 2 (value 4): a guard word was overwritten
  DBG_SITE = 1,         // first failed check: translation unit * 100000 + source line
  DBG_INDEX_LO = 2, DBG_INDEX_HI = 3,
  DBG_LIMIT_LO = 4, DBG_LIMIT_HI = 5,
  DBG_COUNT = 6,        // failed checks in all
  DBG_GUARD = 7,        // first overwritten guard: region ordinal * 65536 + word within the guard
};
constexpr int kDebugWords = 8;
constexpr int kDebugIndexFlag = 2, kDebugGuardFlag = 4;
constexpr unsigned kGuardBytes = 256;
constexpr unsigned kGuardPattern = 0xA5C3A5C3u;

#ifdef QALORA_DEBUG
constexpr bool kDebugBuild = true;
// Device pointer to the current device's record words (allocated and zeroed on first use:
// the debug build is the one place where the library owns device memory), or NULL on failure.
int* debug_words();

__device__ __forceinline__ bool debug_in_range(int* dbg, long long index, long long limit, int site) {
  if (index >= 0 && index < limit) return true;
  if (dbg != nullptr) {
    if (atomicCAS(dbg + DBG_SITE, 0, site) == 0) {
      dbg[DBG_INDEX_LO] = (int)(index & 0xffffffffll);
      dbg[DBG_INDEX_HI] = (int)(index >> 32);
      dbg[DBG_LIMIT_LO] = (int)(limit & 0xffffffffll);
      dbg[DBG_LIMIT_HI] = (int)(limit >> 32);
    }
    atomicAdd(dbg + DBG_COUNT, 1);
    atomicOr(dbg + DBG_FLAGS, kDebugIndexFlag);
  }
  return false;
}
#define QALORA_CHECK(dbg, index, limit) \
  ::qalora::debug_in_range((dbg), (long long)(index), (long long)(limit), QALORA_TU * 100000 + __LINE__)
#else
constexpr bool kDebugBuild = false;
inline int* debug_words() { return nullptr; }
__host__ __device__ __forceinline__ bool debug_always() { return true; }   // (a call: usable as a statement without a warning)
#define QALORA_CHECK(dbg, index, limit) ::qalora::debug_always()
#endif

}  // namespace qalora
