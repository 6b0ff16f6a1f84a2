// Tensor-core kernels for the two rank-r side products of the backward pass that
// stream the whole output gradient:
//   dT[m][i]  = s * sum_n dy[m][n] * B[i][n]          (contraction over D_out)
//   dB[i][n]  =     sum_m T[m][i]  * dy[m][n]         (contraction over tokens; T holds s)
// Both are skinny (one extent is r <= 128), so they are bound by reading dy once
// from HBM.  All operands are bf16 matrices that TMA can deliver directly in the
// layouts tcgen05.mma consumes: K-major tiles for dT, and for dB -- where the
// contraction runs over rows -- MN-major tiles (a [64 rows x 128 bytes] swizzled
// box IS the MN-major swizzle atom stack).  The adapter extent is the 128-row A
// operand (rows >= r are zero), the accumulator sits in TMEM.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 2-5 = epilogue (TMEM lane quarter = warp % 4).  Waits are bounded.
#define QALORA_TU 5
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace qalora {

namespace {

constexpr int AUX_THREADS = 192;
constexpr int ROWS_A = 128;                 // MMA M: adapter index, zero padded
constexpr int STEP = 64;                    // reduction elements per stage

enum AuxMode { AUX_DT = 0, AUX_DB = 1 };

template <int MODE>
struct AuxCfg {
  static constexpr int TILE_N = MODE == AUX_DT ? 64 : 256;        // MMA N: tokens (dT) / output columns (dB)
  static constexpr int STAGES = MODE == AUX_DT ? 8 : 4;
  static constexpr uint32_t A_BYTES = ROWS_A * STEP * 2;          // 16 KiB
  static constexpr uint32_t B_BYTES = TILE_N * STEP * 2;          // 8 / 32 KiB
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr uint32_t TOTAL = STAGES * STAGE_BYTES + 256 + 1024;
  static constexpr uint32_t TMEM_COLS = TILE_N;                   // 64 or 256 (powers of two)
};

struct AuxParams {
  long long M;
  int N, r;
  float s;
  int items;              // work items
  int red_iters;          // dT: N / 64
  int n_tiles;            // dB: N tiles of 256 (last one may be ragged)
  int splits;             // dB: token splits
  long long rows_per_split;
  float* out_f32;         // dT: dT [M][r] (may be null);  dB: partial [splits][r][N]
  __nv_bfloat16* out_bf16;// dT: dTb [M][r]
  int* status;
  int* dbg;               // record words of the bounds-check build (null otherwise)
};

template <int MODE>
__global__ void __launch_bounds__(AUX_THREADS, 1)
aux_tc_kernel(const __grid_constant__ CUtensorMap a_map, const __grid_constant__ CUtensorMap b_map,
              const AuxParams p) {
  using C = AuxCfg<MODE>;
  constexpr int STAGES = C::STAGES;
  extern __shared__ uint8_t smem_raw[];
  // aligned by pointer arithmetic on the __shared__ array, so that the accesses stay shared-space loads/stores
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t smem_base = ptx::smem_u32(smem);
  uint8_t* bar_area = smem + STAGES * C::STAGE_BYTES;
  const uint32_t bar_base = smem_base + STAGES * C::STAGE_BYTES;
  auto bar_full = [&](int s) { return bar_base + 8u * s; };
  auto bar_empty = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t bar_acc_full = bar_base + 8u * (2 * STAGES);
  const uint32_t bar_acc_empty = bar_base + 8u * (2 * STAGES + 1);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_area + 8 * (2 * STAGES + 2));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_area + 8 * (2 * STAGES + 2) + 8);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const bool second_block = p.r > 64;       // dB: rows 64..127 of the adapter operand carry data

  if (MODE == AUX_DB && !second_block) {
    // rows 64..127 of every stage's A tile stay zero for the whole kernel
    for (int s = 0; s < STAGES; ++s) {
      uint4* z = reinterpret_cast<uint4*>(smem + s * C::STAGE_BYTES + 8192);
      for (int i = threadIdx.x; i < 8192 / 16; i += AUX_THREADS) z[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    ptx::fence_proxy_async();
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(bar_full(s), 1);
      ptx::mbar_init(bar_empty(s), 1);
    }
    ptx::mbar_init(bar_acc_full, 1);
    ptx::mbar_init(bar_acc_empty, 4);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&a_map);
    ptx::prefetch_tensormap(&b_map);
  }
  if (warp == 1) {
    __syncwarp();
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), C::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // work item -> (first reduction index, number of steps, output tile)
  auto item_iters = [&](int item) -> int {
    if (MODE == AUX_DT) return p.red_iters;
    const int split = item / p.n_tiles;
    const long long beg = (long long)split * p.rows_per_split;
    long long end = beg + p.rows_per_split;
    if (end > p.M) end = p.M;
    return end > beg ? (int)((end - beg + STEP - 1) / STEP) : 0;
  };

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x) {
        const int iters = item_iters(item);
        for (int i = 0; i < iters; ++i, ++it) {
          const int s = it % STAGES;
          if (!(ok = ptx::mbar_wait(bar_empty(s), ((it / STAGES) & 1) ^ 1, abort_flag))) break;
          const uint32_t stage = smem_base + s * C::STAGE_BYTES;
          // (bounds-check build: the stage lies inside the ring, the copies start inside their matrices)
          QALORA_CHECK(p.dbg, (s + 1) * C::STAGE_BYTES - 1, STAGES * C::STAGE_BYTES);
          if (MODE == AUX_DT) {
            QALORA_CHECK(p.dbg, i * STEP, p.N);
            QALORA_CHECK(p.dbg, (long long)item * C::TILE_N, p.M);
            ptx::mbar_arrive_expect_tx(bar_full(s), C::STAGE_BYTES);
            ptx::tma_load_2d(stage, &a_map, i * STEP, 0, bar_full(s));                       // B[0..127][n..n+63]
            ptx::tma_load_2d(stage + C::A_BYTES, &b_map, i * STEP, item * C::TILE_N, bar_full(s));  // dy[m..][n..]
          } else {
            const int nt = item % p.n_tiles, split = item / p.n_tiles;
            const int m = (int)((long long)split * p.rows_per_split) + i * STEP;
            QALORA_CHECK(p.dbg, m, p.M);
            QALORA_CHECK(p.dbg, nt * C::TILE_N, p.N);
            ptx::mbar_arrive_expect_tx(bar_full(s), (second_block ? 16384u : 8192u) + C::B_BYTES);
            ptx::tma_load_2d(stage, &a_map, 0, m, bar_full(s));                              // T[m..m+63][0..63]
            if (second_block) ptx::tma_load_2d(stage + 8192, &a_map, 64, m, bar_full(s));
#pragma unroll
            for (int b = 0; b < 4; ++b)                                                      // dy[m..][n..n+63], 4 blocks
              ptx::tma_load_2d(stage + C::A_BYTES + b * 8192, &b_map, nt * C::TILE_N + b * 64, m, bar_full(s));
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t IDESC = ptx::idesc_bf16(ROWS_A, C::TILE_N, MODE == AUX_DB, MODE == AUX_DB);
      uint32_t it = 0, tcount = 0;
      bool ok = true, ready = false;
      for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++tcount) {
        const int iters = item_iters(item);
        if (!(ok = ptx::mbar_wait(bar_acc_empty, (tcount & 1) ^ 1, abort_flag))) break;
        ptx::tc_fence_after();
        for (int i = 0; i < iters; ++i, ++it) {
          const int s = it % STAGES;
          // the next stage's barrier is probed inside the block that issues this stage's MMAs
          if (!ready && !(ok = ptx::mbar_wait(bar_full(s), (it / STAGES) & 1, abort_flag))) break;
          ptx::tc_fence_after();
          const uint32_t stage = smem_base + s * C::STAGE_BYTES;
          const uint32_t next_bar = bar_full((it + 1) % STAGES), next_par = ((it + 1) / STAGES) & 1;
          static_assert(STEP == 64, "the step helper issues four K = 16 MMAs");
          if (MODE == AUX_DT) {
            ready = ptx::mma4_ss_commit_probe<2, 2>(tmem_base, ptx::smem_desc(stage, 16, 1024),
                                                    ptx::smem_desc(stage + C::A_BYTES, 16, 1024), IDESC, i > 0 ? 1u : 0u,
                                                    bar_empty(s), next_bar, next_par) != 0;
          } else {   // MN-major: 64-wide blocks 8 KiB apart, 8-row groups 1 KiB apart; 2 KiB per K = 16 step
            ready = ptx::mma4_ss_commit_probe<128, 128>(tmem_base, ptx::smem_desc(stage, 8192, 1024),
                                                        ptx::smem_desc(stage + C::A_BYTES, 8192, 1024), IDESC,
                                                        i > 0 ? 1u : 0u, bar_empty(s), next_bar, next_par) != 0;
          }
        }
        if (ok) ptx::mma_commit(bar_acc_full);
      }
    }
  } else {
    const int quarter = warp % 4;
    const int row = quarter * 32 + lane;           // adapter index i
    uint32_t tcount = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++tcount) {
      const int iters = item_iters(item);
      if (!(ok = ptx::mbar_wait(bar_acc_full, tcount & 1, abort_flag))) break;
      ptx::tc_fence_after();
#pragma unroll 1
      for (int col = 0; col < C::TILE_N; col += 32) {
        uint32_t v[32];
        if (!QALORA_CHECK(p.dbg, col + 31, C::TMEM_COLS)) continue;
        ptx::tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + col, v);
        ptx::tmem_wait_ld();
        if (row >= p.r) continue;
        if (MODE == AUX_DT) {
          const long long m0 = (long long)item * C::TILE_N + col;
#pragma unroll
          for (int t = 0; t < 32; ++t) {
            if (m0 + t >= p.M) break;
            const float val = iters > 0 ? p.s * __uint_as_float(v[t]) : 0.0f;
            if (!QALORA_CHECK(p.dbg, (size_t)(m0 + t) * p.r + row, (size_t)p.M * p.r)) continue;
            if (p.out_f32 != nullptr) p.out_f32[(size_t)(m0 + t) * p.r + row] = val;
            p.out_bf16[(size_t)(m0 + t) * p.r + row] = __float2bfloat16_rn(val);
          }
        } else {
          const int nt = item % p.n_tiles, split = item / p.n_tiles;
          const int n0 = nt * C::TILE_N + col;
          float* dst = p.out_f32 + ((size_t)split * p.r + row) * p.N + n0;
#pragma unroll
          for (int t = 0; t < 32; t += 4) {
            if (n0 + t >= p.N) break;                   // N is a multiple of 8
            if (!QALORA_CHECK(p.dbg, ((size_t)split * p.r + row) * p.N + n0 + t + 3, (size_t)p.splits * p.r * p.N)) break;
            float4 o;
            o.x = iters > 0 ? __uint_as_float(v[t]) : 0.0f;
            o.y = iters > 0 ? __uint_as_float(v[t + 1]) : 0.0f;
            o.z = iters > 0 ? __uint_as_float(v[t + 2]) : 0.0f;
            o.w = iters > 0 ? __uint_as_float(v[t + 3]) : 0.0f;
            *reinterpret_cast<float4*>(dst + t) = o;
          }
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_acc_empty);
    }
  }

  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag != 0) atomicExch(p.status, 1);
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn aux_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

// bf16 [rows][cols] row-major; box = 64 columns x box_rows rows, 128-byte swizzle, zero fill
bool make_map(CUtensorMap* map, const void* base, long long rows, int cols, int box_rows) {
  EncodeTiledFn fn = aux_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int MODE>
int launch_aux(const CUtensorMap& a, const CUtensorMap& b, const AuxParams& p, cudaStream_t st) {
  using C = AuxCfg<MODE>;
  static_assert(C::TOTAL <= 232448, "shared memory budget");
  auto kern = aux_tc_kernel<MODE>;
  static PerDeviceOnce smem_limit;      // this instantiation's shared-memory limit, raised once on every device it runs on
  if (smem_limit.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::TOTAL); }) != QALORA_OK)
    return QALORA_ERR_CUDA;
  const int grid = p.items < device_sm_count() ? p.items : device_sm_count();
  kern<<<grid, AUX_THREADS, C::TOTAL, st>>>(a, b, p);
  count_launch();
  return cuda_status(cudaGetLastError());
}

}  // namespace

bool tc_aux_supported(const Shape& sh, int64_t M) {
  return sh.r >= 8 && sh.r <= 128 && sh.N % 64 == 0 && M >= 1 && M < 0x7fffffffLL - 1024 && aux_encode_fn() != nullptr;
}

// dT = s * dy * B^T  -> fp32 [M][r] (optional) and bf16 [M][r]
int launch_tc_dT(const Shape& sh, int64_t M, const __nv_bfloat16* dy, const __nv_bfloat16* B,
                 float* dT, __nv_bfloat16* dTb, int* status, cudaStream_t st) {
  CUtensorMap a, b;
  if (!make_map(&a, B, sh.r, sh.N, ROWS_A) || !make_map(&b, dy, M, sh.N, AuxCfg<AUX_DT>::TILE_N)) return QALORA_ERR_CUDA;
  AuxParams p{};
  p.M = M; p.N = sh.N; p.r = sh.r; p.s = sh.s;
  p.items = (int)((M + AuxCfg<AUX_DT>::TILE_N - 1) / AuxCfg<AUX_DT>::TILE_N);
  p.red_iters = sh.N / STEP;
  p.out_f32 = dT; p.out_bf16 = dTb; p.status = status; p.dbg = debug_words();
  return launch_aux<AUX_DT>(a, b, p, st);
}

// Number of token splits (and bytes of fp32 partials) the dB kernel uses.
int tc_dB_splits(const Shape& sh, int64_t M) {
  const int n_tiles = (sh.N + 255) / 256;
  long long splits = (device_sm_count() + n_tiles - 1) / n_tiles;
  const long long max_by_rows = (M + 511) / 512;
  if (splits > max_by_rows) splits = max_by_rows;
  return (int)(splits < 1 ? 1 : splits);
}
size_t tc_dB_partial_bytes(const Shape& sh, int64_t M) {
  return (size_t)tc_dB_splits(sh, M) * sh.r * sh.N * sizeof(float);
}

// partial[split][i][n] = sum over the split's tokens of Tb[m][i] * dy[m][n]
int launch_tc_dB_partials(const Shape& sh, int64_t M, const __nv_bfloat16* Tb, const __nv_bfloat16* dy,
                          float* partial, int* splits_out, int* status, cudaStream_t st) {
  CUtensorMap a, b;
  if (!make_map(&a, Tb, M, sh.r, STEP) || !make_map(&b, dy, M, sh.N, STEP)) return QALORA_ERR_CUDA;
  AuxParams p{};
  p.M = M; p.N = sh.N; p.r = sh.r; p.s = 1.0f;
  p.n_tiles = (sh.N + 255) / 256;
  p.splits = tc_dB_splits(sh, M);
  long long rows = (M + p.splits - 1) / p.splits;
  rows = (rows + STEP - 1) / STEP * STEP;
  p.rows_per_split = rows;
  p.splits = (int)((M + rows - 1) / rows);
  p.items = p.n_tiles * p.splits;
  p.out_f32 = partial; p.status = status; p.dbg = debug_words();
  *splits_out = p.splits;
  return launch_aux<AUX_DB>(a, b, p, st);
}

}  // namespace qalora
