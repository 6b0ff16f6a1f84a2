// Tensor-core kernels of the QA-LoRA layer for sm_100a: the forward product
// y = x * W~ (+ adapter) and the input gradient dx = dy * W~^T (+ adapter), with
// the b-bit weights dequantized on the fly.
//
// Both are computed transposed, out^T[c][m] = sum_j Wop[c][j] * act[m][j], so that
// the dequantized weights are the 128-row "A" operand of tcgen05.mma and 256
// tokens are the "N" extent: every dequantized element is reused 256 times.
//   forward : c = output channel n, j = input channel k.  A pack unit (32 input
//             channels of one column) is exactly 32 K-contiguous elements of row
//             c, so the dequantizing thread writes it straight into TENSOR
//             MEMORY (tcgen05.st) and the MMA takes A from TMEM.
//   dx      : c = input channel k, j = output channel n.  A unit is now 32
//             consecutive ROWS of one j, i.e. 64 contiguous bytes of an
//             MN-major operand: it goes to shared memory in the 128-byte
//             swizzled MN-major layout and the MMA takes A from smem.
// The same packed bytes serve both products.  The adapter is folded in as extra
// reduction steps of width r: forward appends T = s*pool(x)*A against B (a tile of
// B[r][n] as it lies in memory IS an MN-major operand: one TMA copy, no thread
// touches it), dx appends dT = s*dy*B^T against the group-expanded A.
//
// Warp roles (768 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 4-19 = four dequantizing warpgroups (each owns every fourth
// reduction step), warps 20-23 = epilogue (dx: two accumulators, so that a tile is
// drained while the next one is multiplied).  Stages are handed
// over with mbarriers; every wait is bounded and a timeout raises a status word
// instead of hanging.
#define QALORA_TU 3
#include <mutex>

#include "common.cuh"
#include "dequant.cuh"
#include "ptx.cuh"
#include "tc_host.cuh"

namespace qalora {

namespace {

constexpr int TILE_C = 128;      // out channels per tile   (MMA M)
constexpr int TILE_T = 256;      // tokens per tile         (MMA N)
constexpr int TILE_T_FEW = 64;   // tokens per tile of the forward variant for at most 64 tokens
constexpr int TILE_J = 64;       // reduction step per stage
constexpr int DQ_GROUPS = 4;     // dequantizing warpgroups
constexpr int THREADS = 128 + 128 * DQ_GROUPS + 128;
constexpr int TMEM_COLS = 512;
constexpr int ACC_COL = 0;       // accumulator: columns [0, 256); dx keeps a second one at [256, 512)
constexpr int A_COL = 256;       // forward operand ring: 8 slots of 32 columns
constexpr uint32_t ATILE_BYTES = TILE_C * TILE_J * 2;    // 16 KiB dequantized tile (dx); tile of B (forward)

enum Mode { FWD = 0, DX = 1 };

struct TcParams {
  const uint32_t* codes;
  const float2* qparams;
  const __nv_bfloat16* lora;   // FWD: B [r][N];  DX: A [G][r]
  __nv_bfloat16* out;          // FWD: y [M][N];  DX: dx [M][K]
  long long M;
  int K, N, g, r;
  int ld_out;                  // N (FWD) or K (DX)
  int c_tiles, m_tiles;        // tiles along out channels / tokens that this launch works on
  int c_tile0;                 // its first channel tile (a launch may cover a strip of the channel tiles)
  int red_iters, lora_iters;   // main / adapter reduction steps per tile
  int qp_rows;                 // rows of (alpha, beta) per code stage: 128 / g
  int tile_count;              // c_tiles * m_tiles
  int ksplit;                  // parts the reduction of a tile is cut into (1: none)
  int tile_t;                  // tokens per tile: TILE_T, or TILE_T_FEW (forward, M <= 64; always with parts)
  float* partial;              // parts: fp32 partial results [ksplit][part_rows][part_ld] of the output rectangle that
  int part_rows, part_ld;      //        starts at row part_row0, channel part_col0 (the whole output: M, ld_out, 0, 0)
  int part_row0, part_col0;
  int beside_pool;             // host side: launch beside the few-row pooling kernel before this one (forward with adapter)
  int* status;                 // device word: set to 1 when a wait timed out
  int* dbg;                    // record words of the bounds-check build (null otherwise)
  int stop_after_steps;        // normally INT_MAX; a test makes every activation producer stop early, so that waits expire
  unsigned long long wait_limit_ns;
};

// Work item of a block: part `sp` of tile `tile`, i.e. the main steps mb .. mb + n_main - 1
// and, for the last part, the adapter steps; n_steps in all.  Parts begin on even steps (a
// forward code stage feeds two).
struct TcSegment {
  int tile, sp, mb, n_main, n_steps;
};
template <bool PARTS>
__device__ __forceinline__ TcSegment tc_segment(const TcParams& p, int vt) {
  TcSegment g;
  g.tile = PARTS ? vt / p.ksplit : vt;
  g.sp = PARTS ? vt % p.ksplit : 0;
  if (!PARTS) {
    g.mb = 0;
    g.n_main = p.red_iters;
    g.n_steps = p.red_iters + p.lora_iters;
  } else {
    const long long pairs = p.red_iters / 2;
    g.mb = 2 * (int)(pairs * g.sp / p.ksplit);
    g.n_main = 2 * (int)(pairs * (g.sp + 1) / p.ksplit) - g.mb;
    g.n_steps = g.n_main + (g.sp == p.ksplit - 1 ? p.lora_iters : 0);
  }
  return g;
}
// j-th step of a segment -> step index of the tile (main steps 0 .. red_iters - 1, then the adapter steps)
template <bool PARTS>
__device__ __forceinline__ int tc_step(const TcParams& p, const TcSegment& g, int j) {
  if (!PARTS) return j;
  return j < g.n_main ? g.mb + j : p.red_iters + (j - g.n_main);
}

// Rings, decoupled so that each covers its own latency:
//   NX activation tiles (TMA, 32 KiB each);
//   NB operand slots written by the dequantizers (TMEM columns for forward: eight, so that
//      a warpgroup can fill its next slot while its last one is still being multiplied;
//      16 KiB of smem each for dx: four), each with a "ready" and a "free" barrier that
//      step it uses at index it % NB; the step's activation tile completes the same "ready"
//      barrier, and one tcgen05.commit per step frees the slot AND the tile;
//   NC code stages (two tiled TMA copies each: 4 k-block rows of pack units and the
//      rows of (alpha, beta) they need; a forward stage feeds two reduction steps)
//      that run further ahead.
// NB and NC are multiples of DQ_GROUPS, so a ring slot always belongs to the same
// dequantizing warpgroup and its barrier phases are waited on in order.
template <int BITS, int MODE, int TT = TILE_T>   // TT: tokens per tile (MMA N): 256, or 64 for the few-token variant
struct Smem {
  static constexpr uint32_t ACT_BYTES = TT * TILE_J * 2;                         // activation tile: 32 KiB (8 KiB)
  static constexpr int WORDS = BITS == 4 ? 4 : (BITS == 3 ? 3 : 2);
  static constexpr int NX = 4;
  static constexpr int NB = MODE == FWD ? 8 : 4;
  static constexpr int NC = TT == TILE_T ? 4 : 12;                               // small activation tiles leave room for a deep code ring
  static constexpr int IPS = MODE == FWD ? 2 : 1;                                // reduction steps per code stage
  static constexpr int TILE_NC = MODE == FWD ? TILE_C : TILE_J;                  // columns of a code stage
  static constexpr int NOUT = MODE == FWD ? 2 : 1;                               // epilogue staging buffers
  // Accumulators in tensor memory.  The forward product keeps its operand ring in the upper 256
  // columns, so it has one; dx takes its operand from shared memory and alternates between two,
  // so that the epilogue drains one tile while the next one is being multiplied.  (A forward
  // kernel with the operand in shared memory and two accumulators was built too: 5-8 % slower
  // than the operand in tensor memory, 0.665 against 0.615 ms for 4096 -> 11008 at 8192 tokens.)
  static constexpr int NACC = MODE == DX ? 2 : 1;
  // a code stage = 4 k-block rows x TILE_NC columns of pack units + up to 4 rows of (alpha, beta)
  static constexpr uint32_t CODE_BYTES = 4 * TILE_NC * WORDS * 4;
  static constexpr uint32_t QP_ROW_BYTES = TILE_NC * 8;
  static constexpr uint32_t QP_BYTES = 4 * QP_ROW_BYTES;
  static constexpr uint32_t CSTAGE_BYTES = ((CODE_BYTES + QP_BYTES + 127) / 128) * 128;
  static constexpr uint32_t OUT_BYTES = 32 * TILE_C * 2;                         // 32 tokens x 128 channels bf16
  static constexpr uint32_t OFF_X = 0;
  static constexpr uint32_t OFF_A = NX * ACT_BYTES;                              // dx: operand ring; forward: the adapter's tile of B
  static constexpr uint32_t OFF_C = OFF_A + (MODE == DX ? NX * ATILE_BYTES : ATILE_BYTES);
  static constexpr uint32_t OFF_OUT = OFF_C + NC * CSTAGE_BYTES;
  static constexpr uint32_t OFF_BARS = OFF_OUT + NOUT * OUT_BYTES;
  static constexpr int NBARS = 2 * NB + 2 * NC + 2 * NACC + 1;                   // + "tile of B free" (forward)
  static constexpr uint32_t TOTAL = OFF_BARS + 8 * NBARS + 64 + 1024;            // + alignment slack
};

// PARTS: every tile's reduction is cut into p.ksplit parts.  TT: tokens per tile.
template <int BITS, int MODE, bool PARTS, int TT>
__global__ void __launch_bounds__(THREADS, 1)
qalora_tc_kernel(const __grid_constant__ CUtensorMap act_map, const __grid_constant__ CUtensorMap lora_map,
                 const __grid_constant__ CUtensorMap lb_map, const __grid_constant__ CUtensorMap out_map,
                 const __grid_constant__ CUtensorMap codes_map, const __grid_constant__ CUtensorMap qp_map,
                 const TcParams p) {
  using S = Smem<BITS, MODE, TT>;
  constexpr int WORDS = S::WORDS;
  constexpr int NX = S::NX, NB = S::NB, NC = S::NC;
  constexpr uint32_t ACT_BYTES = S::ACT_BYTES;
  extern __shared__ uint8_t smem_raw[];
  // aligned by pointer arithmetic on the __shared__ array, so that the accesses stay shared-space loads/stores
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t smem_base = ptx::smem_u32(smem);
  const uint32_t bar_base = smem_base + S::OFF_BARS;
  auto bar_full_x = [&](int s) { return bar_base + 8u * s; };
  auto bar_empty_x = [&](int s) { return bar_base + 8u * (NB + s); };
  auto bar_full_c = [&](int s) { return bar_base + 8u * (2 * NB + s); };
  auto bar_empty_c = [&](int s) { return bar_base + 8u * (2 * NB + NC + s); };
  constexpr int NACC = S::NACC;
  auto bar_acc_full = [&](int b) { return bar_base + 8u * (2 * NB + 2 * NC + b); };
  auto bar_acc_empty = [&](int b) { return bar_base + 8u * (2 * NB + 2 * NC + NACC + b); };
  const uint32_t bar_lb_empty = bar_base + 8u * (2 * NB + 2 * NC + 2 * NACC);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + S::OFF_BARS + 8 * S::NBARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::OFF_BARS + 8 * S::NBARS + 8);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    // full_x: the activation tile has landed (producer's arrive + its bytes) AND the four
    // dequantizer warps have written the operand slot: one wait per step for the MMA issuer
    for (int s = 0; s < NB; ++s) { ptx::mbar_init(bar_full_x(s), 1 + 4); ptx::mbar_init(bar_empty_x(s), 1); }
    for (int s = 0; s < NC; ++s) { ptx::mbar_init(bar_full_c(s), 1); ptx::mbar_init(bar_empty_c(s), 4 * S::IPS); }
    for (int b = 0; b < NACC; ++b) { ptx::mbar_init(bar_acc_full(b), 1); ptx::mbar_init(bar_acc_empty(b), 4); }
    ptx::mbar_init(bar_lb_empty, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&act_map);
    if (p.lora_iters > 0) ptx::prefetch_tensormap(&lora_map);
    if (MODE == FWD && p.lora_iters > 0) ptx::prefetch_tensormap(&lb_map);
    ptx::prefetch_tensormap(&out_map);
    ptx::prefetch_tensormap(&codes_map);
    ptx::prefetch_tensormap(&qp_map);
  }
  if (warp == 1) {
    __syncwarp();
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int total_tiles = p.tile_count * (PARTS ? p.ksplit : 1);               // work items: (tile, part)

  if (warp == 0) {
    // ------------------------------------------------- activation producer ----
    if (lane == 0) {
      uint32_t it = 0, nlb = 0;                      // steps / adapter steps so far
      bool ok = true;
      for (int vt = blockIdx.x; vt < total_tiles && ok; vt += gridDim.x) {
        const TcSegment sg = tc_segment<PARTS>(p, vt);
        const int m0 = (sg.tile / p.c_tiles) * TT;
        const int c0 = (sg.tile % p.c_tiles + p.c_tile0) * TILE_C;
        for (int j = 0; j < sg.n_steps; ++j, ++it) {
          if (it >= (uint32_t)p.stop_after_steps) { ok = false; break; }     // (test hook: the tiles stop coming)
          const int i = tc_step<PARTS>(p, sg, j);
          const int s = it % NX, sb = it % NB;
          // the tile slot was last used by step it - NX: wait until that step has been multiplied
          if (it >= (uint32_t)NX && !(ok = ptx::mbar_wait(bar_empty_x((it - NX) % NB), ((it - NX) / NB) & 1, abort_flag, p.wait_limit_ns))) break;
          // (bounds-check build: the tile lies inside its ring and the copy starts inside the matrix)
          QALORA_CHECK(p.dbg, S::OFF_X + (s + 1) * ACT_BYTES - 1, S::OFF_A);
          QALORA_CHECK(p.dbg, m0, p.M);
          if (i < p.red_iters) {
            QALORA_CHECK(p.dbg, i * TILE_J, MODE == FWD ? p.K : p.N);
            ptx::mbar_arrive_expect_tx(bar_full_x(sb), ACT_BYTES);
            ptx::tma_load_2d(smem_base + S::OFF_X + s * ACT_BYTES, &act_map, i * TILE_J, m0, bar_full_x(sb));
          } else if (MODE == FWD) {
            // adapter step: the tile of T and, as the other operand, rows r0 .. r0 + 63 of B for the
            // tile's 128 channels (two boxes of 64 channels; rows beyond r arrive as zeros).  The one
            // buffer is free once the adapter step before this one has been multiplied.
            const int r0 = (i - p.red_iters) * TILE_J;
            QALORA_CHECK(p.dbg, r0, p.r);
            QALORA_CHECK(p.dbg, c0 + TILE_C - 1, p.N);
            if (!(ok = ptx::mbar_wait(bar_lb_empty, (nlb & 1) ^ 1, abort_flag, p.wait_limit_ns))) break;
            ++nlb;
            ptx::mbar_arrive_expect_tx(bar_full_x(sb), ACT_BYTES + ATILE_BYTES);
            // T is written by the pooling kernel, beside which this kernel may have started
            // (programmatic dependent launch): wait for it only here, before T is fetched (a
            // no-op without such a launch, or once that kernel has finished)
            asm volatile("griddepcontrol.wait;" ::: "memory");
            ptx::tma_load_2d(smem_base + S::OFF_X + s * ACT_BYTES, &lora_map, r0, m0, bar_full_x(sb));
            ptx::tma_load_2d(smem_base + S::OFF_A, &lb_map, c0, r0, bar_full_x(sb));
            ptx::tma_load_2d(smem_base + S::OFF_A + ATILE_BYTES / 2, &lb_map, c0 + 64, r0, bar_full_x(sb));
          } else {
            ptx::mbar_arrive_expect_tx(bar_full_x(sb), ACT_BYTES);
            ptx::tma_load_2d(smem_base + S::OFF_X + s * ACT_BYTES, &lora_map, (i - p.red_iters) * TILE_J, m0, bar_full_x(sb));
          }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------- code producer ----
    if (lane == 0) {
      uint32_t cit = 0;                              // code stages issued so far
      bool ok = true;
      for (int vt = blockIdx.x; vt < total_tiles && ok; vt += gridDim.x) {
        const TcSegment sg = tc_segment<PARTS>(p, vt);
        const int c0 = (sg.tile % p.c_tiles + p.c_tile0) * TILE_C;
        const int cs_end = (sg.mb + sg.n_main) / S::IPS;
        for (int cs = sg.mb / S::IPS; cs < cs_end; ++cs, ++cit) {
          const int s = cit % NC;
          if (!(ok = ptx::mbar_wait(bar_empty_c(s), ((cit / NC) & 1) ^ 1, abort_flag, p.wait_limit_ns))) break;
          const uint32_t stage = smem_base + S::OFF_C + s * S::CSTAGE_BYTES;
          // forward: k-blocks 4 cs .. 4 cs + 3 of columns c0 ..; dx: the tile's 4 k-blocks, columns 64 cs ..
          const int kb0 = MODE == FWD ? cs * 4 : c0 / 32;
          const int col0 = MODE == FWD ? c0 : cs * TILE_J;
          QALORA_CHECK(p.dbg, S::OFF_C + (s + 1) * S::CSTAGE_BYTES - 1, S::OFF_OUT);
          QALORA_CHECK(p.dbg, kb0 + 3, p.K / 32);
          QALORA_CHECK(p.dbg, col0 + S::TILE_NC - 1, p.N);
          ptx::mbar_arrive_expect_tx(bar_full_c(s), S::CODE_BYTES + p.qp_rows * S::QP_ROW_BYTES);
          ptx::tma_load_2d(stage, &codes_map, col0 * WORDS / 2, kb0, bar_full_c(s));
          ptx::tma_load_2d(stage + S::CODE_BYTES, &qp_map, 2 * col0, kb0 * 32 / p.g, bar_full_c(s));
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer ----
    if (lane == 0) {
      constexpr uint32_t IDESC_MAIN = ptx::idesc_bf16(TILE_C, TT, MODE == DX, false);
      constexpr uint32_t IDESC_LORA = ptx::idesc_bf16(TILE_C, TT, MODE == FWD, false);   // forward: the tile of B is MN-major
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      // Issuing one tcgen05.mma costs this thread about 110 cycles and the four MMAs of a step
      // keep the tensor pipe busy for 512, so everything else in this loop has to stay short:
      // per step one fence and one block of instructions that probes the NEXT step's barrier,
      // issues the four MMAs and the commit and then reads the probe (whose latency thus hides
      // behind the issue); the blocking wait runs only when the probe said "not yet".
      static_assert(TILE_J == 64, "the step helpers issue four K = 16 MMAs");
      bool ready = false;
      for (int vt = blockIdx.x; vt < total_tiles && ok; vt += gridDim.x, ++tcount) {
        const TcSegment sg = tc_segment<PARTS>(p, vt);
        const int ab = tcount % NACC;                 // accumulator of this tile
        const uint32_t acc_tmem = tmem_base + ACC_COL + ab * TILE_T;
        QALORA_CHECK(p.dbg, ACC_COL + ab * TILE_T + TT - 1, MODE == FWD ? A_COL : TMEM_COLS);
        if (!(ok = ptx::mbar_wait(bar_acc_empty(ab), ((tcount / NACC) & 1) ^ 1, abort_flag, p.wait_limit_ns))) break;
        ptx::tc_fence_after();
        for (int j = 0; j < sg.n_steps; ++j, ++it) {
          const int sx = it % NX, sb = it % NB;
          const uint32_t ph = (it / NB) & 1;
          if (!ready && !(ok = ptx::mbar_wait(bar_full_x(sb), ph, abort_flag, p.wait_limit_ns))) break;
          ptx::tc_fence_after();
          const uint32_t xs = smem_base + S::OFF_X + sx * ACT_BYTES;
          const uint32_t as = smem_base + S::OFF_A + sb * ATILE_BYTES;     // dx: NB == NX
          const uint64_t bdesc = ptx::smem_desc(xs, 16, 1024);             // + 32 bytes per K = 16 step
          const uint32_t next_bar = bar_full_x((it + 1) % NB), next_par = ((it + 1) / NB) & 1;
          const uint32_t acc = j > 0 ? 1u : 0u;
          // the commit frees the activation tile AND the operand slot
          if (MODE == FWD && j < sg.n_main) {
            ready = ptx::mma4_ts_commit_probe<2>(acc_tmem, tmem_base + A_COL + sb * 32, bdesc, IDESC_MAIN, acc,
                                                 bar_empty_x(sb), next_bar, next_par) != 0;
          } else if (MODE == FWD) {
            // adapter step: 64-channel blocks of B 8 KiB apart (LBO), 8-row groups 1 KiB apart (SBO); 2 KiB per K = 16
            ready = ptx::mma4_ss_commit_probe<128, 2>(acc_tmem, ptx::smem_desc(smem_base + S::OFF_A, 8192, 1024), bdesc,
                                                      IDESC_LORA, acc, bar_empty_x(sb), next_bar, next_par) != 0;
            ptx::mma_commit(bar_lb_empty);
          } else if (j < sg.n_main) {
            // MN-major A: 64-channel blocks 8 KiB apart (LBO), 8-column groups 1 KiB apart (SBO); 2 KiB per step
            ready = ptx::mma4_ss_commit_probe<128, 2>(acc_tmem, ptx::smem_desc(as, 8192, 1024), bdesc, IDESC_MAIN,
                                                      acc, bar_empty_x(sb), next_bar, next_par) != 0;
          } else {
            ready = ptx::mma4_ss_commit_probe<2, 2>(acc_tmem, ptx::smem_desc(as, 16, 1024), bdesc, IDESC_LORA, acc,
                                                    bar_empty_x(sb), next_bar, next_par) != 0;
          }
        }
        if (ok) ptx::mma_commit(bar_acc_full(ab));
      }
    }
  } else if (warp >= 4 && warp < 4 + 4 * DQ_GROUPS) {
    // -------------------------------------------------------- dequantizers ----
    // Warpgroup w owns the reduction steps with it % DQ_GROUPS == w and dequantizes
    // the whole step (two pack units per thread); the groups work on different
    // steps at once and hide each other's latencies.
    const int wg = (warp - 4) / 4;
    const int tw = threadIdx.x - 128 - wg * 128;  // 0..127 inside the warpgroup
    const int quarter = warp % 4;                // TMEM lane quarter of this warp
    const DqConsts dk = dq_consts<BITS>();
    uint32_t it = 0, mit0 = 0;                    // reduction steps / main steps before this tile
    bool ok = true;
    const int qsh = p.g == 32 ? 0 : (p.g == 64 ? 1 : 2);   // k-block -> (alpha, beta) row of the stage
    for (int vt = blockIdx.x; vt < total_tiles && ok; vt += gridDim.x) {
      const TcSegment sg = tc_segment<PARTS>(p, vt);
      const int c0 = (sg.tile % p.c_tiles + p.c_tile0) * TILE_C;
      for (int j = 0; j < sg.n_steps; ++j, ++it) {
        if ((int)(it % DQ_GROUPS) != wg) continue;
        const int i = tc_step<PARTS>(p, sg, j);
        const int sa = it % NB;
        // operand slot first: once it is free every earlier step has been multiplied, so
        // the code ring's previous phase has certainly completed
        if (!(ok = ptx::mbar_wait(bar_empty_x(sa), ((it / NB) & 1) ^ 1, abort_flag, p.wait_limit_ns))) break;
        const uint32_t cst = (mit0 + j) / S::IPS;  // code stage counter (main steps only; mit0 stays even)
        const int sc = cst % NC;
        const int kb_base = MODE == FWD ? ((mit0 + j) % S::IPS) * 2 : 0;   // first k-block row of this step
        if (i < p.red_iters && !(ok = ptx::mbar_wait(bar_full_c(sc), (cst / NC) & 1, abort_flag, p.wait_limit_ns))) break;
        const uint8_t* cstage = smem + S::OFF_C + sc * S::CSTAGE_BYTES;
        if (MODE == FWD) {
          // (an adapter step needs nothing from this group: its operands both come by TMA; the
          // group still owns the step's slot of the ring and signs it off below)
          if (i < p.red_iters) {
            ptx::tc_fence_after();
            const int row = quarter * 32 + lane;   // out channel within the tile = TMEM lane
#pragma unroll
            for (int half = 0; half < 2; ++half) { // the two 32-channel blocks of the step
              uint32_t v[16];
              const int kbl = kb_base + half;
              const uint32_t* cw = reinterpret_cast<const uint32_t*>(cstage) + (kbl * TILE_C + row) * WORDS;
              if (!QALORA_CHECK(p.dbg, (kbl * TILE_C + row) * WORDS + WORDS - 1, S::CODE_BYTES / 4) ||
                  !QALORA_CHECK(p.dbg, (kbl >> qsh) * TILE_C + row, p.qp_rows * TILE_C) ||
                  !QALORA_CHECK(p.dbg, A_COL + sa * 32 + half * 16 + 15, TMEM_COLS))
                continue;
              uint32_t w[WORDS];
              load_unit<WORDS>(cw, w);
              const float2 ab = reinterpret_cast<const float2*>(cstage + S::CODE_BYTES)[(kbl >> qsh) * TILE_C + row];
              dequant_unit<BITS>(w, ab, dk, v);
              ptx::tmem_st16(tmem_base + ((uint32_t)(quarter * 32) << 16) + A_COL + sa * 32 + half * 16, v);
            }
            ptx::tmem_wait_st();
            ptx::tc_fence_before();
          }
        } else {
          uint8_t* atile = smem + S::OFF_A + sa * ATILE_BYTES;
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int dq = tw + 128 * h;         // 0..255: unit (main steps) / half-row (adapter steps)
            if (i < p.red_iters) {
              uint32_t v[16];
              const int kbl = dq / TILE_J, nl = dq % TILE_J;       // 32-channel block, column
              const uint32_t* cw = reinterpret_cast<const uint32_t*>(cstage) + (kbl * TILE_J + nl) * WORDS;
              if (!QALORA_CHECK(p.dbg, (kbl * TILE_J + nl) * WORDS + WORDS - 1, S::CODE_BYTES / 4) ||
                  !QALORA_CHECK(p.dbg, (kbl >> qsh) * TILE_J + nl, p.qp_rows * TILE_J) ||
                  !QALORA_CHECK(p.dbg, S::OFF_A + sa * ATILE_BYTES + (kbl / 2) * 8192 + (nl / 8) * 1024 + (nl % 8) * 128 + 127, S::OFF_C))
                continue;
              uint32_t w[WORDS];
              load_unit<WORDS>(cw, w);
              const float2 ab = reinterpret_cast<const float2*>(cstage + S::CODE_BYTES)[(kbl >> qsh) * TILE_J + nl];
              dequant_unit<BITS>(w, ab, dk, v);
              // MN-major, 128-byte swizzle: row = column nl (128 bytes = 64 channels),
              // this unit fills chunks (kbl%2)*4 .. +3 of block kbl/2
              uint8_t* rowp = atile + (kbl / 2) * 8192 + (nl / 8) * 1024 + (nl % 8) * 128;
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const int chunk = ((kbl % 2) * 4 + q) ^ (nl % 8);
                *reinterpret_cast<uint4*>(rowp + chunk * 16) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
              }
            } else {
              // adapter step, K-major rows: row c holds A[(c0 + c) / g][r0 .. r0 + 63]
              const int row = dq / 2, halfrow = dq % 2;
              const int r0 = (i - p.red_iters) * TILE_J + halfrow * 32;
              const __nv_bfloat16* ap = p.lora + (size_t)((c0 + row) / p.g) * p.r + r0;
              uint8_t* rowp = atile + (row / 8) * 1024 + (row % 8) * 128;
              if (!QALORA_CHECK(p.dbg, (c0 + row) / p.g, p.K / p.g) ||
                  !QALORA_CHECK(p.dbg, S::OFF_A + sa * ATILE_BYTES + (row / 8) * 1024 + (row % 8) * 128 + 127, S::OFF_C))
                continue;
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                uint4 t = make_uint4(0u, 0u, 0u, 0u);
                if (r0 + q * 8 < p.r) t = *reinterpret_cast<const uint4*>(ap + q * 8);   // r is a multiple of 8
                const int chunk = (halfrow * 4 + q) ^ (row % 8);
                *reinterpret_cast<uint4*>(rowp + chunk * 16) = t;
              }
            }
          }
          ptx::fence_proxy_async();              // make the generic-proxy writes visible to the MMA
        }
        __syncwarp();
        if (lane == 0) {
          ptx::mbar_arrive(bar_full_x(sa));
          if (i < p.red_iters) ptx::mbar_arrive(bar_empty_c(sc));
        }
      }
      mit0 += sg.n_main;
    }
  } else if (warp >= 4 + 4 * DQ_GROUPS) {
    // ------------------------------------------------------------ epilogue ----
    // Each thread owns one out channel (its TMEM lane) and reads 32 tokens at a
    // time; the bf16 values are transposed through a [32 tokens][128 channels]
    // staging tile and leave with one TMA store per chunk (rows beyond M are
    // clipped by the tensor map).  The accumulator is released as soon as its
    // last column has been read.
    const int quarter = warp % 4;
    const int et = threadIdx.x - (128 + 128 * DQ_GROUPS);    // 0..127
    const int ch = quarter * 32 + lane;
    uint32_t tcount = 0, chunk = 0;
    bool ok = true;
    for (int vt = blockIdx.x; vt < total_tiles && ok; vt += gridDim.x, ++tcount) {
      const int tile = PARTS ? vt / p.ksplit : vt, sp = PARTS ? vt % p.ksplit : 0;
      const int ct = tile % p.c_tiles + p.c_tile0, mt = tile / p.c_tiles;
      const int ab = tcount % NACC;
      // The four warps meet at barriers below, so they must agree on leaving: a thread whose wait
      // gave up (the abort flag was raised elsewhere) and a thread that saw the phase complete in
      // the same instant would otherwise part ways.
      ok = ptx::mbar_wait(bar_acc_full(ab), (tcount / NACC) & 1, abort_flag, p.wait_limit_ns);
      if (!(ok = ptx::named_barrier_and(3, 128, ok))) break;
      ptx::tc_fence_after();
#pragma unroll 1
      for (int col = 0; col < TT; col += 32, ++chunk) {
        uint32_t v[32];
        if (QALORA_CHECK(p.dbg, ACC_COL + ab * TILE_T + col + 31, MODE == FWD ? A_COL : TMEM_COLS))
          ptx::tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + ACC_COL + ab * TILE_T + col, v);
        ptx::tmem_wait_ld();
        if (col == TT - 32) {                     // all columns read: hand the accumulator back
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar_acc_empty(ab));
        }
        if constexpr (PARTS) {
          // a part of the reduction: fp32 partial results [part][token][channel], added up by
          // sum_parts_kernel; a warp writes 32 neighbouring channels of one token per store
          const long long prow = (long long)mt * TT + col - p.part_row0;       // row and column inside the rectangle
          const int pcol = ct * TILE_C + ch - p.part_col0;
          float* dst = p.partial + ((size_t)sp * p.part_rows + prow) * p.part_ld + pcol;
#pragma unroll
          for (int t = 0; t < 32; ++t)
            if ((long long)mt * TT + col + t < p.M &&
                QALORA_CHECK(p.dbg, ((size_t)sp * p.part_rows + prow + t) * p.part_ld + pcol, (size_t)p.ksplit * p.part_rows * p.part_ld) &&
                QALORA_CHECK(p.dbg, pcol, p.part_ld) && QALORA_CHECK(p.dbg, prow + t, p.part_rows))
              dst[(size_t)t * p.part_ld] = __uint_as_float(v[t]);
          continue;
        }
        uint8_t* stg = smem + S::OFF_OUT + (chunk % S::NOUT) * S::OUT_BYTES;
        ptx::named_barrier(1, 128);               // the staging tile's previous store has been read out
#pragma unroll
        for (int t = 0; t < 32; ++t)
          reinterpret_cast<__nv_bfloat16*>(stg)[t * TILE_C + ch] = __float2bfloat16_rn(__uint_as_float(v[t]));
        ptx::fence_proxy_async();
        ptx::named_barrier(2, 128);
        if (et == 0 && (long long)mt * TT + col < p.M && QALORA_CHECK(p.dbg, ct * TILE_C + TILE_C - 1, p.ld_out) &&
            QALORA_CHECK(p.dbg, S::OFF_OUT + (chunk % S::NOUT + 1) * S::OUT_BYTES - 1, S::OFF_BARS)) {
          ptx::tma_store_2d(&out_map, ct * TILE_C, mt * TT + col, ptx::smem_u32(stg));
          ptx::bulk_commit_group();
          ptx::bulk_wait_group_read<S::NOUT - 1>();
        }
      }
    }
    if (et == 0) ptx::bulk_wait_group<0>();
  }

  // ---------------------------------------------------------------- teardown ----
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag != 0) atomicExch(p.status, 1);
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace

// ------------------------------------------------------------------ host side --
// (tensor-map builders and the sum of parts are shared with midm_tc.cu: tc_host.cuh)
EncodeTiledFn encode_fn() {
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

// bf16 matrix [rows][cols] row-major, box = 64 columns x `box_rows` rows, 128-byte swizzle;
// out-of-range rows and columns read as zero.
bool make_act_map(CUtensorMap* map, const void* base, long long rows, int cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {TILE_J, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 output [rows][cols] row-major, box = 128 columns x 32 rows, no swizzle (store side)
bool make_out_map(CUtensorMap* map, void* base, long long rows, int cols) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {TILE_C, 32};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// packed codes [K/32][N][words] uint32 seen as a 2-D matrix of 8-byte elements, so that one
// box row is the whole contiguous run of tile_cols pack units; box = kb_rows k-block rows
bool make_codes_map(CUtensorMap* map, const uint32_t* codes, int K, int N, int bits, int tile_cols, int kb_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  const int words = words_per_unit(bits);
  cuuint64_t dims[2] = {(cuuint64_t)N * words / 2, (cuuint64_t)(K / 32)};
  cuuint64_t strides[1] = {(cuuint64_t)N * words * 4};
  cuuint32_t box[2] = {(cuuint32_t)(tile_cols * words / 2), (cuuint32_t)kb_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<uint32_t*>(codes), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// (alpha, beta) float32 [G][2N]; box = 2 * tile_cols floats x rows
bool make_qp_map(CUtensorMap* map, const float2* qp, int G, int N, int tile_cols, int rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)N * 2, (cuuint64_t)G};
  cuuint64_t strides[1] = {(cuuint64_t)N * 8};
  cuuint32_t box[2] = {(cuuint32_t)(2 * tile_cols), (cuuint32_t)rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float2*>(qp), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// out[i] = bf16(sum over parts of partial[part][i]), added in part order; 8 elements per thread
static __global__ void __launch_bounds__(256)
sum_parts_kernel(const float* __restrict__ partial, __nv_bfloat16* __restrict__ out, size_t count, int parts) {
  const size_t i0 = ((size_t)blockIdx.x * 256 + threadIdx.x) * 8;
  if (i0 >= count) return;                                   // count is a multiple of 8
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int s = 0; s < parts; ++s) {
    const float4 a = *reinterpret_cast<const float4*>(partial + (size_t)s * count + i0);
    const float4 b = *reinterpret_cast<const float4*>(partial + (size_t)s * count + i0 + 4);
    acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
    acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
  }
  uint4 o;
  o.x = pack_bf16x2(acc[0], acc[1]); o.y = pack_bf16x2(acc[2], acc[3]);
  o.z = pack_bf16x2(acc[4], acc[5]); o.w = pack_bf16x2(acc[6], acc[7]);
  *reinterpret_cast<uint4*>(out + i0) = o;
}

// The same for a rectangle of the output: out[(row0 + r) * out_ld + col0 + c] = bf16(sum over parts of
// partial[(part * part_rows + r) * cols + c]), r < rows, c < cols (cols a multiple of 8); 8 elements per thread
static __global__ void __launch_bounds__(256)
sum_parts_rect_kernel(const float* __restrict__ partial, __nv_bfloat16* __restrict__ out, int rows, int cols, int parts,
                      int part_rows, long long out_ld, long long row0, int col0) {
  const size_t i0 = ((size_t)blockIdx.x * 256 + threadIdx.x) * 8;
  if (i0 >= (size_t)rows * cols) return;
  const size_t r = i0 / cols, c = i0 % cols;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int s = 0; s < parts; ++s) {
    const float* src = partial + ((size_t)s * part_rows + r) * cols + c;
    const float4 a = *reinterpret_cast<const float4*>(src);
    const float4 b = *reinterpret_cast<const float4*>(src + 4);
    acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
    acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
  }
  uint4 o;
  o.x = pack_bf16x2(acc[0], acc[1]); o.y = pack_bf16x2(acc[2], acc[3]);
  o.z = pack_bf16x2(acc[4], acc[5]); o.w = pack_bf16x2(acc[6], acc[7]);
  *reinterpret_cast<uint4*>(out + (row0 + (long long)r) * out_ld + col0 + c) = o;
}

int launch_sum_parts_bf16(const float* partial, __nv_bfloat16* out, size_t count, int parts, cudaStream_t st) {
  sum_parts_kernel<<<(unsigned)((count / 8 + 255) / 256), 256, 0, st>>>(partial, out, count, parts);
  count_launch();
  return cuda_status(cudaGetLastError());
}

namespace {

template <int BITS, int MODE, bool PARTS, int TT>
int launch_tc_t(const CUtensorMap& act, const CUtensorMap& lora, const TcParams& p, cudaStream_t st) {
  using S = Smem<BITS, MODE, TT>;
  CUtensorMap out, cmap, qmap, lb = act;
  // forward with adapter: B [r][N] in boxes of 64 channels x 64 rows (rows beyond r read as zero)
  if (MODE == FWD && p.r > 0 && !make_act_map(&lb, p.lora, p.r, p.N, TILE_J)) return QALORA_ERR_CUDA;
  if (!make_out_map(&out, p.out, p.M, p.ld_out)) return QALORA_ERR_CUDA;
  if (!make_codes_map(&cmap, p.codes, p.K, p.N, BITS, S::TILE_NC, 4)) return QALORA_ERR_CUDA;
  if (!make_qp_map(&qmap, p.qparams, p.K / p.g, p.N, S::TILE_NC, p.qp_rows)) return QALORA_ERR_CUDA;
  static_assert(S::TOTAL <= 232448, "shared memory budget");
  auto kern = qalora_tc_kernel<BITS, MODE, PARTS, TT>;
  static PerDeviceOnce smem_limit;      // this instantiation's shared-memory limit, raised once on every device it runs on
  if (smem_limit.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S::TOTAL); }) != QALORA_OK)
    return QALORA_ERR_CUDA;
  const int tiles = p.tile_count * p.ksplit;
  const int grid = tiles < device_sm_count() ? tiles : device_sm_count();
  {
    MainKernelProbe probe(MODE == FWD ? "qalora_tc_kernel<fwd>" : "qalora_tc_kernel<dx>", st);
    // p.beside_pool: the kernel before this one in the stream is the few-row pooling kernel that
    // writes T and lets its successor start at once; this kernel then starts beside it and waits
    // for it only before an adapter step fetches T (x, the weights and the status word are final:
    // the pooling kernel itself started after them).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = S::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (MODE == FWD && p.beside_pool != 0) ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kern, act, lora, lb, out, cmap, qmap, p) != cudaSuccess) return QALORA_ERR_CUDA;
  }
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return QALORA_ERR_CUDA;
  if (PARTS && p.part_ld == p.ld_out && p.part_rows == p.M) return launch_sum_parts_bf16(p.partial, p.out, (size_t)p.M * p.ld_out, p.ksplit, st);
  if (PARTS) {   // the parts cover a rectangle of the output (the tiles of a last, short wave)
    const long long left = p.M - p.part_row0;
    const int rows = (int)(left < p.part_rows ? left : p.part_rows);
    const size_t count = (size_t)rows * p.part_ld;
    sum_parts_rect_kernel<<<(unsigned)((count / 8 + 255) / 256), 256, 0, st>>>(p.partial, p.out, rows, p.part_ld, p.ksplit, p.part_rows,
                                                                             p.ld_out, p.part_row0, p.part_col0);
    count_launch();
    return cuda_status(cudaGetLastError());
  }
  return QALORA_OK;
}

template <int BITS, int MODE>
int launch_tc(const CUtensorMap& act, const CUtensorMap& lora, const TcParams& p, cudaStream_t st) {
  if (MODE == FWD && p.tile_t == TILE_T_FEW) return launch_tc_t<BITS, FWD, true, TILE_T_FEW>(act, lora, p, st);
  if (p.ksplit > 1) return launch_tc_t<BITS, MODE, true, TILE_T>(act, lora, p, st);
  return launch_tc_t<BITS, MODE, false, TILE_T>(act, lora, p, st);
}

}  // namespace

// Test hook (qalora_debug_expire_next_tc_wait in api.cu): when armed, the activation producers
// of the next forward or dX launch stop after `steps` reduction steps and the launch's waits give
// up after `limit_ns`: every role's bounded wait runs out, the status word is raised and the
// blocks leave through their ordinary teardown (tensor memory released).  One-shot.
static std::atomic<int> g_tc_expire_after_steps{0x7fffffff};
static std::atomic<unsigned long long> g_tc_expire_limit_ns{ptx::WAIT_LIMIT_NS};
void arm_tc_wait_expiry(int steps, unsigned long long limit_ns) {
  g_tc_expire_limit_ns.store(limit_ns);
  g_tc_expire_after_steps.store(steps < 0 ? 0 : steps);
}
static void take_expiry(TcParams* p) {
  p->stop_after_steps = g_tc_expire_after_steps.exchange(0x7fffffff);
  p->wait_limit_ns = p->stop_after_steps != 0x7fffffff ? g_tc_expire_limit_ns.load() : ptx::WAIT_LIMIT_NS;
}

static bool tc_group_ok(int g) { return g == 32 || g == 64 || g == 128; }

bool tc_forward_supported(const Shape& sh, int64_t M) {
  return tc_group_ok(sh.g) && sh.N % TILE_C == 0 && sh.K % (2 * TILE_J) == 0 && M >= 1 && M <= 0x7fffffffLL / 2 && encode_fn() != nullptr;
}
bool tc_dx_supported(const Shape& sh, int64_t M) {
  return tc_group_ok(sh.g) && sh.K % TILE_C == 0 && sh.N % TILE_J == 0 && M >= 1 && M <= 0x7fffffffLL / 2 && encode_fn() != nullptr;
}

// Parts the forward reduction is cut into.  With few tokens a layer has fewer (or not many
// more) 128 x 256 tiles than the GPU has SMs; cutting every tile's reduction into parts fills
// the SMs and evens out the last wave.  The parts meet as fp32 partial results in scratch.
int tc_forward_parts(const Shape& sh, int64_t M) {
  if (M > 512) return 1;
  if (M <= TILE_T_FEW && sh.K / TILE_J >= 8) {
    // the 64-token variant always writes partial results; as many parts as fill the SMs evenly
    const long long tiles = sh.N / TILE_C;
    const int steps = sh.K / TILE_J, sms = device_sm_count();
    int best = 1;
    double best_cost = 1e30;
    for (int ks = 1; ks <= 8; ++ks) {
      if (ks > 1 && steps / ks < 8) break;
      const double cost = (double)((tiles * ks + sms - 1) / sms) / ks + 0.02 * ks;
      if (cost < best_cost - 1e-9) { best_cost = cost; best = ks; }
    }
    return -best;                                              // negative: the 64-token variant
  }
  const long long tiles = (long long)(sh.N / TILE_C) * ((M + TILE_T - 1) / TILE_T);
  const int steps = sh.K / TILE_J, sms = device_sm_count();
  if (tiles >= sms) return 1;             // at least one full wave (a short LAST wave is cut into parts on its own, see below)
  // Fewer tiles than SMs: parts fill the idle SMs.  Cost in units of one tile's time: waves of
  // work items over the parts, a start-up share per part, and the parts' fp32 partial results
  // (written and read again: 8 bytes per output and part) at the HBM rate against the tile's
  // steps x 512 tensor cycles.
  const double tile_us = steps * 0.27, out_mb = (double)M * sh.N * 8e-6;
  int best = 1;
  double best_cost = 1.0;
  for (int ks = 2; ks <= 8; ++ks) {
    if (steps / ks < 8) break;
    if ((size_t)ks * M * sh.N * sizeof(float) > ((size_t)256 << 20)) break;
    const double cost = (double)((tiles * ks + sms - 1) / sms) / ks + 0.02 * ks + ks * out_mb / 6.0 / tile_us;
    if (cost < best_cost - 1e-9) { best_cost = cost; best = ks; }
  }
  return best;
}
// A layer with a few waves of tiles whose last wave is short: a strip of its channel tiles (all
// token tiles of the last `strip_c` channel tiles, about as many tiles as that wave holds) is
// cut into parts, in a second launch, so that it costs 1 / parts of a tile's time instead of a
// whole wave; e.g. 172 tiles on 148 SMs are one wave of 148 whole tiles and one of 24 x 6 parts,
// 640 tiles (40 x 16) are four waves of 37 x 16 whole tiles and one of 3 x 16 x 3 parts.  The
// parts' fp32 partial results cover only that strip of the output.
struct TcTail { int strip_c, ks; };
static TcTail tc_tail(long long c_tiles, long long m_tiles, int steps) {
  TcTail t{0, 1};
  const long long tiles = c_tiles * m_tiles;
  const int sms = device_sm_count();
  if (tiles <= sms || tiles >= 6LL * sms) return t;               // one wave, or so many that the last one hardly matters
  const int rem = (int)(tiles % sms);
  if (rem == 0 || rem * 2 > sms) return t;
  const long long strip_c = (rem + m_tiles - 1) / m_tiles, strip = strip_c * m_tiles;
  if (strip_c >= c_tiles || strip > sms) return t;
  int ks = (int)(sms / strip);
  if (ks > 8) ks = 8;
  if (ks > steps / 8) ks = steps / 8;
  if (ks < 2) return t;
  t.strip_c = (int)strip_c; t.ks = ks;
  return t;
}
static TcTail tc_forward_tail(const Shape& sh, int64_t M) {
  if (tc_forward_parts(sh, M) != 1) return TcTail{0, 1};          // already cut into parts as a whole
  return tc_tail(sh.N / TILE_C, (M + TILE_T - 1) / TILE_T, sh.K / TILE_J);
}
// the same for dx (channel tiles along K, reduction over N; parts begin on even steps, so N must be a multiple of 128)
#ifndef QALORA_TC_DX_TAIL
#define QALORA_TC_DX_TAIL 1
#endif
static TcTail tc_dx_tail(const Shape& sh, int64_t M) {
  if (!QALORA_TC_DX_TAIL || sh.N % (2 * TILE_J) != 0) return TcTail{0, 1};
  return tc_tail(sh.K / TILE_C, (M + TILE_T - 1) / TILE_T, sh.N / TILE_J);
}
size_t tc_dx_partial_bytes(const Shape& sh, int64_t M) {
  const TcTail tail = tc_dx_tail(sh, M);
  return tail.strip_c > 0 ? (size_t)tail.ks * M * tail.strip_c * TILE_C * sizeof(float) : 0;
}
size_t tc_forward_partial_bytes(const Shape& sh, int64_t M) {
  const int ks = tc_forward_parts(sh, M);
  if (ks < 0) return (size_t)(-ks) * M * sh.N * sizeof(float);
  if (ks > 1) return (size_t)ks * M * sh.N * sizeof(float);
  const TcTail tail = tc_forward_tail(sh, M);
  return tail.strip_c > 0 ? (size_t)tail.ks * M * tail.strip_c * TILE_C * sizeof(float) : 0;
}

#ifndef QALORA_TC_BESIDE_POOL_ROWS
#define QALORA_TC_BESIDE_POOL_ROWS 512
#endif
// y = x * W~ + Tb * B with Tb = bf16(s * pool(x) * A) precomputed ([M][r]).
// `partial`: tc_forward_partial_bytes() of scratch.
int launch_tc_forward(const Shape& sh, int64_t M, const __nv_bfloat16* x, const uint32_t* codes,
                      const float2* qparams, const __nv_bfloat16* Tb, const __nv_bfloat16* B,
                      __nv_bfloat16* y, float* partial, int* status, cudaStream_t st) {
  const int parts = tc_forward_parts(sh, M);
  const int tile_t = parts < 0 ? TILE_T_FEW : TILE_T;
  CUtensorMap act, lora;
  if (!make_act_map(&act, x, M, sh.K, tile_t)) return QALORA_ERR_CUDA;
  lora = act;
  if (sh.r > 0 && !make_act_map(&lora, Tb, M, sh.r, tile_t)) return QALORA_ERR_CUDA;
  TcParams p{};
  p.codes = codes; p.qparams = qparams; p.lora = B; p.out = y;
  p.M = M; p.K = sh.K; p.N = sh.N; p.g = sh.g; p.r = sh.r; p.ld_out = sh.N;
  p.c_tiles = sh.N / TILE_C; p.m_tiles = (int)((M + tile_t - 1) / tile_t);
  p.red_iters = sh.K / TILE_J; p.lora_iters = (sh.r + TILE_J - 1) / TILE_J;
  p.status = status; p.qp_rows = 128 / sh.g; p.dbg = debug_words();
  take_expiry(&p);
  p.ksplit = parts < 0 ? -parts : parts; p.tile_t = tile_t; p.partial = partial;
  p.c_tile0 = 0; p.tile_count = p.c_tiles * p.m_tiles;
  p.part_rows = (int)M; p.part_ld = sh.N; p.part_row0 = 0; p.part_col0 = 0;
  // (below 512 rows the pooling kernel is the few-row one, which releases its successor at its start)
  p.beside_pool = (sh.r > 0 && M < QALORA_TC_BESIDE_POOL_ROWS) ? 1 : 0;
  const TcTail tail = tc_forward_tail(sh, M);
  if (tail.strip_c > 0) {
    // whole tiles of the other channel tiles first, then the strip cut into parts (same stream: one after the other)
    TcParams pa = p;
    pa.c_tiles = p.c_tiles - tail.strip_c;
    pa.tile_count = pa.c_tiles * p.m_tiles;
    int st_a = sh.bits == 4 ? launch_tc<4, FWD>(act, lora, pa, st) : (sh.bits == 3 ? launch_tc<3, FWD>(act, lora, pa, st) : launch_tc<2, FWD>(act, lora, pa, st));
    if (st_a != QALORA_OK) return st_a;
    TcParams pb = p;
    pb.c_tiles = tail.strip_c; pb.c_tile0 = pa.c_tiles; pb.tile_count = tail.strip_c * p.m_tiles; pb.ksplit = tail.ks;
    pb.part_rows = (int)M; pb.part_ld = tail.strip_c * TILE_C; pb.part_row0 = 0; pb.part_col0 = pa.c_tiles * TILE_C;
    pb.beside_pool = 0;                              // its predecessor is the kernel above
    if (sh.bits == 4) return launch_tc<4, FWD>(act, lora, pb, st);
    if (sh.bits == 3) return launch_tc<3, FWD>(act, lora, pb, st);
    return launch_tc<2, FWD>(act, lora, pb, st);
  }
  if (sh.bits == 4) return launch_tc<4, FWD>(act, lora, p, st);
  if (sh.bits == 3) return launch_tc<3, FWD>(act, lora, p, st);
  return launch_tc<2, FWD>(act, lora, p, st);
}

// dx = dy * W~^T + dTb * expand(A)^T with dTb = bf16(s * dy * B^T) precomputed ([M][r]).
int launch_tc_dx(const Shape& sh, int64_t M, const __nv_bfloat16* dy, const uint32_t* codes,
                 const float2* qparams, const __nv_bfloat16* dTb, const __nv_bfloat16* A,
                 __nv_bfloat16* dx, float* partial, int* status, cudaStream_t st) {
  CUtensorMap act, lora;
  if (!make_act_map(&act, dy, M, sh.N, TILE_T)) return QALORA_ERR_CUDA;
  lora = act;
  if (sh.r > 0 && !make_act_map(&lora, dTb, M, sh.r, TILE_T)) return QALORA_ERR_CUDA;
  TcParams p{};
  p.codes = codes; p.qparams = qparams; p.lora = A; p.out = dx;
  p.M = M; p.K = sh.K; p.N = sh.N; p.g = sh.g; p.r = sh.r; p.ld_out = sh.K;
  p.c_tiles = sh.K / TILE_C; p.m_tiles = (int)((M + TILE_T - 1) / TILE_T);
  p.red_iters = sh.N / TILE_J; p.lora_iters = (sh.r + TILE_J - 1) / TILE_J;
  p.status = status; p.qp_rows = 128 / sh.g; p.dbg = debug_words();
  take_expiry(&p);
  p.ksplit = 1; p.tile_t = TILE_T; p.partial = nullptr;
  p.c_tile0 = 0; p.tile_count = p.c_tiles * p.m_tiles;
  p.part_rows = (int)M; p.part_ld = sh.K; p.part_row0 = 0; p.part_col0 = 0;
  const TcTail tail = tc_dx_tail(sh, M);
  if (tail.strip_c > 0 && partial != nullptr) {
    // whole tiles of the other channel tiles first, then the strip of a short last wave cut into parts
    TcParams pa = p;
    pa.c_tiles = p.c_tiles - tail.strip_c;
    pa.tile_count = pa.c_tiles * p.m_tiles;
    int st_a = sh.bits == 4 ? launch_tc<4, DX>(act, lora, pa, st) : (sh.bits == 3 ? launch_tc<3, DX>(act, lora, pa, st) : launch_tc<2, DX>(act, lora, pa, st));
    if (st_a != QALORA_OK) return st_a;
    TcParams pb = p;
    pb.c_tiles = tail.strip_c; pb.c_tile0 = pa.c_tiles; pb.tile_count = tail.strip_c * p.m_tiles; pb.ksplit = tail.ks;
    pb.partial = partial;
    pb.part_rows = (int)M; pb.part_ld = tail.strip_c * TILE_C; pb.part_row0 = 0; pb.part_col0 = pa.c_tiles * TILE_C;
    if (sh.bits == 4) return launch_tc<4, DX>(act, lora, pb, st);
    if (sh.bits == 3) return launch_tc<3, DX>(act, lora, pb, st);
    return launch_tc<2, DX>(act, lora, pb, st);
  }
  if (sh.bits == 4) return launch_tc<4, DX>(act, lora, p, st);
  if (sh.bits == 3) return launch_tc<3, DX>(act, lora, p, st);
  return launch_tc<2, DX>(act, lora, p, st);
}

}  // namespace qalora
