// Forward product for a few dozen to 128 tokens (17 <= M <= 128 where the few-token kernel does not run):
//     y[m][n] = sum_k x[m][k] * W~[k][n]  (+ adapter),
// in the orientation in which the TOKENS are the 128 rows of the tcgen05 MMA and 256 output
// channels are its N extent.
//
// Why a kernel of its own.  With this few tokens every code byte is used once per token tile,
// so the forward pass is bound by how fast the codes can be dequantized and by the cost of
// ISSUING MMAs, not by the tensor pipe: one tcgen05.mma costs its issuing thread about 110
// cycles whatever its N extent is.  The large-M kernel (gemm_tc.cu) makes the dequantized
// weights the 128-row operand, i.e. 128 channels x 16 reduction indices per instruction; with
// 64 tokens as its N extent that is 2048 weights per 110 cycles and SM.  Here one instruction
// takes 256 channels x 16 indices, twice as many weights, and the 128-row operand is the
// activation tile (rows beyond M are zero-filled by the tensor copy and cost no traffic).
//
// Work item = (256-channel tile, 128-token tile, part of the reduction); a persistent block
// takes items in turn.  (With more than one token tile every weight would be dequantized once
// per tile: the kernel is used for one tile, M <= 128.)  Parts leave fp32 partial results [part][M][N] in the workspace, added in
// part order afterwards (deterministic); a layer cut into one part writes bf16 directly.
//
// Warp roles (768 threads, 1 block per SM):
//   warp 0     activation producer: x tiles [128 or 64 tokens x 64 k] (TMA, 128-byte swizzle), ring of 3 or 6
//   warp 1     MMA issuer and owner of tensor memory (two 256-column fp32 accumulators)
//   warp 2     code producer: stages of 2 k-block rows x 256 columns of pack units + their
//              (alpha, beta) rows (two tiled copies of 128 columns each per kind), ring of 4
//   warps 4-19 two dequantizing groups of 256 threads; group g owns the steps with
//              step % 2 == g: thread = one channel row, two pack units (64 reduction indices)
//              per step, written as a K-major, 128-byte-swizzled operand row into one of 4 slots
//   warps 20-23 epilogue: tcgen05.ld of 32 channels per token row, stored straight to global
//              memory (fp32 partial results or bf16), 128 / 64 contiguous bytes per thread
// The adapter is folded in as extra reduction steps of the last part: bf16(s pool(x) A) tiles
// against rows of B gathered from global memory.
// Every wait is bounded; a wait that gives up raises the status word and the block unwinds.
#define QALORA_TU 4
#include "common.cuh"
#include "dequant.cuh"
#include "ptx.cuh"
#include "tc_host.cuh"

namespace qalora {

namespace {

constexpr int MM_TOK = 128;       // token rows per tile (MMA M)
constexpr int MM_CH = 256;        // channels per tile   (MMA N)
constexpr int MM_J = 64;          // reduction indices per step
constexpr int MM_GROUPS = 2;      // dequantizing groups
constexpr int MM_THREADS = 128 + 256 * MM_GROUPS + 128;
constexpr int MM_NB = 4, MM_NC = 4, MM_NACC = 2;
constexpr uint32_t MM_X_RING = 48 * 1024;               // activation tiles: 3 of 128 rows or 6 of 64 rows
constexpr uint32_t MM_B_BYTES = MM_CH * MM_J * 2;       // 32 KiB

struct MmParams {
  const __nv_bfloat16* lora_B;  // B [r][N]
  __nv_bfloat16* y;             // [M][N]
  float* partial;               // parts > 1: fp32 [parts][M][N]
  long long M;
  int K, N, g, r;
  int n_tiles, m_tiles, parts;
  int red_iters, lora_iters;    // main / adapter reduction steps of a whole tile
  int qp_rows;                  // rows of (alpha, beta) per code stage: 64 / g, at least one
  int* status;
  int* dbg;                     // record words of the bounds-check build (null otherwise)
};

// XROWS: token rows an activation tile brings (64 for M <= 64, else 128).  The MMA always reads
// 128 rows; with 64-row tiles rows 64 .. 127 of its operand are whatever follows in shared
// memory (the next tile), and the accumulator rows they produce are never stored.  Half-size
// tiles double the ring's depth, which is what bounds the kernel: a tile's slot is free only
// when the step that used it has been multiplied, and the copy then takes a microsecond.
template <int BITS, int XROWS>
struct MmSmem {
  static constexpr int WORDS = BITS == 4 ? 4 : (BITS == 3 ? 3 : 2);
  static constexpr uint32_t X_BYTES = XROWS * MM_J * 2;
  static constexpr int NX = MM_X_RING / X_BYTES;
  static constexpr uint32_t CODE_HALF = 2 * 128 * WORDS * 4;        // 2 k-block rows x 128 columns of units
  static constexpr uint32_t CODE_BYTES = 2 * CODE_HALF;              // 256 columns
  static constexpr uint32_t QP_HALF_ROW = 128 * 8;
  static constexpr uint32_t QP_BYTES = 2 * 2 * QP_HALF_ROW;          // up to 2 rows x 256 columns
  static constexpr uint32_t CSTAGE_BYTES = ((CODE_BYTES + QP_BYTES + 127) / 128) * 128;
  static constexpr uint32_t OFF_X = 0;
  static constexpr uint32_t OFF_B = MM_X_RING;
  static constexpr uint32_t OFF_C = OFF_B + MM_NB * MM_B_BYTES;
  static constexpr uint32_t OFF_BARS = OFF_C + MM_NC * CSTAGE_BYTES;
  static constexpr int NBARS = 2 * NX + 2 * MM_NB + 2 * MM_NC + 2 * MM_NACC;
  static constexpr uint32_t TOTAL = OFF_BARS + 8 * NBARS + 64 + 1024;   // + alignment slack
};

struct MmItem {
  int nt, mt, sp, mb, n_main, n_steps;
};
// Work item vt -> (channel tile, token tile, part) and its steps: main steps mb .. mb + n_main - 1,
// then, for the last part, the adapter steps.
__device__ __forceinline__ MmItem mm_item(const MmParams& p, int vt) {
  MmItem w;
  w.sp = vt % p.parts;
  const int tile = vt / p.parts;
  w.nt = tile % p.n_tiles;
  w.mt = tile / p.n_tiles;
  w.mb = (int)((long long)p.red_iters * w.sp / p.parts);
  w.n_main = (int)((long long)p.red_iters * (w.sp + 1) / p.parts) - w.mb;
  w.n_steps = w.n_main + (w.sp == p.parts - 1 ? p.lora_iters : 0);
  return w;
}

template <int BITS, int XROWS>
__global__ void __launch_bounds__(MM_THREADS, 1)
qalora_midm_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap t_map,
                   const __grid_constant__ CUtensorMap lb_map, const __grid_constant__ CUtensorMap codes_map,
                   const __grid_constant__ CUtensorMap qp_map, const MmParams p) {
  using S = MmSmem<BITS, XROWS>;
  constexpr int WORDS = S::WORDS;
  constexpr int MM_NX = S::NX;
  constexpr uint32_t MM_X_BYTES = S::X_BYTES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t smem_base = ptx::smem_u32(smem);
  const uint32_t bar_base = smem_base + S::OFF_BARS;
  auto bar_full_x = [&](int s) { return bar_base + 8u * s; };
  auto bar_empty_x = [&](int s) { return bar_base + 8u * (MM_NX + s); };
  auto bar_full_b = [&](int s) { return bar_base + 8u * (2 * MM_NX + s); };
  auto bar_empty_b = [&](int s) { return bar_base + 8u * (2 * MM_NX + MM_NB + s); };
  auto bar_full_c = [&](int s) { return bar_base + 8u * (2 * MM_NX + 2 * MM_NB + s); };
  auto bar_empty_c = [&](int s) { return bar_base + 8u * (2 * MM_NX + 2 * MM_NB + MM_NC + s); };
  auto bar_acc_full = [&](int s) { return bar_base + 8u * (2 * MM_NX + 2 * MM_NB + 2 * MM_NC + s); };
  auto bar_acc_empty = [&](int s) { return bar_base + 8u * (2 * MM_NX + 2 * MM_NB + 2 * MM_NC + MM_NACC + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + S::OFF_BARS + 8 * S::NBARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::OFF_BARS + 8 * S::NBARS + 8);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    for (int s = 0; s < MM_NX; ++s) { ptx::mbar_init(bar_full_x(s), 1); ptx::mbar_init(bar_empty_x(s), 1); }
    for (int s = 0; s < MM_NB; ++s) { ptx::mbar_init(bar_full_b(s), 8); ptx::mbar_init(bar_empty_b(s), 1); }
    for (int s = 0; s < MM_NC; ++s) { ptx::mbar_init(bar_full_c(s), 1); ptx::mbar_init(bar_empty_c(s), 8); }
    for (int s = 0; s < MM_NACC; ++s) { ptx::mbar_init(bar_acc_full(s), 1); ptx::mbar_init(bar_acc_empty(s), 4); }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&x_map);
    if (p.lora_iters > 0) { ptx::prefetch_tensormap(&t_map); ptx::prefetch_tensormap(&lb_map); }
    ptx::prefetch_tensormap(&codes_map);
    ptx::prefetch_tensormap(&qp_map);
  }
  if (warp == 1) {
    __syncwarp();
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int total_items = p.n_tiles * p.m_tiles * p.parts;

  if (warp == 0) {
    // ------------------------------------------------- activation producer ----
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int vt = blockIdx.x; vt < total_items && ok; vt += gridDim.x) {
        const MmItem w = mm_item(p, vt);
        const int m0 = w.mt * MM_TOK;
        for (int j = 0; j < w.n_steps; ++j, ++it) {
          const int s = it % MM_NX;
          if (!(ok = ptx::mbar_wait(bar_empty_x(s), ((it / MM_NX) & 1) ^ 1, abort_flag))) break;
          // (bounds-check build: the tile lies inside its ring, the copy starts inside the matrix)
          QALORA_CHECK(p.dbg, S::OFF_X + (s + 1) * MM_X_BYTES - 1, S::OFF_B);
          QALORA_CHECK(p.dbg, m0, p.M);
          QALORA_CHECK(p.dbg, j < w.n_main ? (w.mb + j) * MM_J : (j - w.n_main) * MM_J, j < w.n_main ? p.K : p.r);
          ptx::mbar_arrive_expect_tx(bar_full_x(s), MM_X_BYTES);
          if (j < w.n_main)
            ptx::tma_load_2d(smem_base + S::OFF_X + s * MM_X_BYTES, &x_map, (w.mb + j) * MM_J, m0, bar_full_x(s));
          else {
            // T is written by the pooling kernel, beside which this kernel may have started
            // (programmatic dependent launch): wait for it only here, before T is fetched (a
            // no-op when the launch carried no such attribute or the kernel has long finished)
            asm volatile("griddepcontrol.wait;" ::: "memory");
            ptx::tma_load_2d(smem_base + S::OFF_X + s * MM_X_BYTES, &t_map, (j - w.n_main) * MM_J, m0, bar_full_x(s));
          }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------- code producer ----
    if (lane == 0) {
      uint32_t cit = 0;
      bool ok = true;
      for (int vt = blockIdx.x; vt < total_items && ok; vt += gridDim.x) {
        const MmItem w = mm_item(p, vt);
        const int c0 = w.nt * MM_CH;
        for (int j = 0; j < w.n_main; ++j, ++cit) {
          const int s = cit % MM_NC;
          if (!(ok = ptx::mbar_wait(bar_empty_c(s), ((cit / MM_NC) & 1) ^ 1, abort_flag))) break;
          const uint32_t stage = smem_base + S::OFF_C + s * S::CSTAGE_BYTES;
          const int kb0 = (w.mb + j) * 2, q0 = kb0 * 32 / p.g;
          QALORA_CHECK(p.dbg, S::OFF_C + (s + 1) * S::CSTAGE_BYTES - 1, S::OFF_BARS);
          QALORA_CHECK(p.dbg, kb0 + 1, p.K / 32);
          QALORA_CHECK(p.dbg, q0, p.K / p.g);
          QALORA_CHECK(p.dbg, c0 + MM_CH - 1, p.N);
          ptx::mbar_arrive_expect_tx(bar_full_c(s), S::CODE_BYTES + 2 * p.qp_rows * S::QP_HALF_ROW);
#pragma unroll
          for (int h = 0; h < 2; ++h) {          // a tiled copy spans at most 256 elements: 128 columns each
            ptx::tma_load_2d(stage + h * S::CODE_HALF, &codes_map, (c0 + 128 * h) * WORDS / 2, kb0, bar_full_c(s));
            ptx::tma_load_2d(stage + S::CODE_BYTES + h * 2 * S::QP_HALF_ROW, &qp_map, 2 * (c0 + 128 * h), q0, bar_full_c(s));
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer ----
    if (lane == 0) {
      constexpr uint32_t IDESC = ptx::idesc_bf16(MM_TOK, MM_CH, false, false);   // both operands K-major
      constexpr uint32_t IDESC_LORA = ptx::idesc_bf16(MM_TOK, MM_CH, false, true); // adapter step: the tile of B is MN-major
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      uint32_t ready = 0;                          // bit 0: operand slot of the coming step, bit 1: its activation tile
      for (int vt = blockIdx.x; vt < total_items && ok; vt += gridDim.x, ++tcount) {
        const MmItem w = mm_item(p, vt);
        const int ab = tcount % MM_NACC;
        const uint32_t acc_tmem = tmem_base + ab * MM_CH;
        QALORA_CHECK(p.dbg, ab * MM_CH + MM_CH - 1, 512);
        if (!(ok = ptx::mbar_wait(bar_acc_empty(ab), ((tcount / MM_NACC) & 1) ^ 1, abort_flag))) break;
        ptx::tc_fence_after();
        for (int j = 0; j < w.n_steps; ++j, ++it) {
          const int sx = it % MM_NX, sb = it % MM_NB;
          // Both barriers of this step were probed in the instruction block of the step before (a
          // probe answers after some 200 cycles even for a phase long complete: issued first and
          // read last, that latency hides behind the MMA issue); a blocking wait runs only after a
          // "not yet".
          if (!(ready & 1u) && !(ok = ptx::mbar_wait(bar_full_b(sb), (it / MM_NB) & 1, abort_flag))) break;
          if (!(ready & 2u) && !(ok = ptx::mbar_wait(bar_full_x(sx), (it / MM_NX) & 1, abort_flag))) break;
          ptx::tc_fence_after();
          // rows of 128 bytes (64 reduction indices), 8-row groups 1 KiB apart; + 32 bytes per K = 16
          const uint64_t adesc = ptx::smem_desc(smem_base + S::OFF_X + sx * MM_X_BYTES, 16, 1024);
          const uint64_t bdesc = ptx::smem_desc(smem_base + S::OFF_B + sb * MM_B_BYTES, 16, 1024);
          // one block: the probes for the NEXT step, four MMAs, the two commits (the tile and the
          // operand slot are free once these MMAs are done), then the probes' answers
          if (j < w.n_main) {
            ready = ptx::mma4_ss_commit2_probe2<2, 2>(acc_tmem, adesc, bdesc, IDESC, j > 0 ? 1u : 0u, bar_empty_x(sx),
                                                      bar_empty_b(sb), bar_full_b((it + 1) % MM_NB), ((it + 1) / MM_NB) & 1,
                                                      bar_full_x((it + 1) % MM_NX), ((it + 1) / MM_NX) & 1);
          } else {
            // adapter step: rows r0 .. r0 + 63 of B as they lie in memory: 64-channel blocks 8 KiB apart
            // (LBO), 8-row groups 1 KiB apart (SBO), 2 KiB per K = 16
            const uint64_t lbdesc = ptx::smem_desc(smem_base + S::OFF_B + sb * MM_B_BYTES, 8192, 1024);
            ready = ptx::mma4_ss_commit2_probe2<2, 128>(acc_tmem, adesc, lbdesc, IDESC_LORA, j > 0 ? 1u : 0u, bar_empty_x(sx),
                                                        bar_empty_b(sb), bar_full_b((it + 1) % MM_NB), ((it + 1) / MM_NB) & 1,
                                                        bar_full_x((it + 1) % MM_NX), ((it + 1) / MM_NX) & 1);
          }
        }
        if (ok) ptx::mma_commit(bar_acc_full(ab));
      }
    }
  } else if (warp >= 4 && warp < 4 + 8 * MM_GROUPS) {
    // -------------------------------------------------------- dequantizers ----
    const int grp = (warp - 4) / 8;
    const int row = threadIdx.x - 128 - grp * 256;        // channel row of the tile: 0..255
    const DqConsts dk = dq_consts<BITS>();
    const int qsh = p.g == 32 ? 0 : (p.g == 64 ? 1 : 2);  // k-block of the stage -> its (alpha, beta) row (two k-blocks per stage)
    const int half_col = row / 128, col_in_half = row % 128;
    uint32_t it = 0, mit = 0;
    bool ok = true;
    for (int vt = blockIdx.x; vt < total_items && ok; vt += gridDim.x) {
      const MmItem w = mm_item(p, vt);
      const int c0 = w.nt * MM_CH;
      for (int j = 0; j < w.n_steps; ++j, ++it) {
        const bool main_step = j < w.n_main;
        const uint32_t cst = mit + (main_step ? j : 0);
        if ((int)(it % MM_GROUPS) != grp) continue;
        const int sb = it % MM_NB, sc = cst % MM_NC;
        if (!(ok = ptx::mbar_wait(bar_empty_b(sb), ((it / MM_NB) & 1) ^ 1, abort_flag))) break;
        if (main_step && !(ok = ptx::mbar_wait(bar_full_c(sc), (cst / MM_NC) & 1, abort_flag))) break;
        if (!main_step) {
          // adapter step: the operand is a tile of B itself, rows r0 .. r0 + 63 for the tile's 256
          // channels, brought by four tiled copies (64 channels each; rows beyond r arrive as zeros)
          // straight into the operand slot.  No thread touches it: the group's first thread asks for
          // the copies, every warp signs the slot off.
          if (row == 0) {
            const int r0 = (j - w.n_main) * MM_J;
            QALORA_CHECK(p.dbg, r0, p.r);
            QALORA_CHECK(p.dbg, c0 + MM_CH - 1, p.N);
            ptx::mbar_arrive_expect_tx(bar_full_b(sb), MM_B_BYTES);
#pragma unroll
            for (int h = 0; h < 4; ++h)
              ptx::tma_load_2d(smem_base + S::OFF_B + sb * MM_B_BYTES + h * 8192, &lb_map, c0 + 64 * h, r0, bar_full_b(sb));
          } else if (lane == 0) {
            ptx::mbar_arrive(bar_full_b(sb));
          }
          continue;
        }
        const uint8_t* cstage = smem + S::OFF_C + sc * S::CSTAGE_BYTES;
        uint8_t* rowp = smem + S::OFF_B + sb * MM_B_BYTES + (row / 8) * 1024 + (row % 8) * 128;
        if (!QALORA_CHECK(p.dbg, S::OFF_B + sb * MM_B_BYTES + (row / 8) * 1024 + (row % 8) * 128 + 127, S::OFF_C)) continue;
#pragma unroll
        for (int half = 0; half < 2; ++half) {   // the two 32-index blocks of the step
          uint32_t v[16];
          const uint32_t* cw = reinterpret_cast<const uint32_t*>(cstage + half_col * S::CODE_HALF) + (half * 128 + col_in_half) * WORDS;
          if (!QALORA_CHECK(p.dbg, half_col * S::CODE_HALF / 4 + (half * 128 + col_in_half) * WORDS + WORDS - 1, S::CODE_BYTES / 4) ||
              !QALORA_CHECK(p.dbg, half_col * 2 * 128 + (half >> qsh) * 128 + col_in_half, S::QP_BYTES / 8))
            continue;
          uint32_t wd[WORDS];
          load_unit<WORDS>(cw, wd);
          const float2 ab = reinterpret_cast<const float2*>(cstage + S::CODE_BYTES + half_col * 2 * S::QP_HALF_ROW)[(half >> qsh) * 128 + col_in_half];
          dequant_unit<BITS>(wd, ab, dk, v);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int chunk = (half * 4 + q) ^ (row % 8);
            *reinterpret_cast<uint4*>(rowp + chunk * 16) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
          }
        }
        ptx::fence_proxy_async();                // make the generic-proxy writes visible to the MMA
        __syncwarp();
        if (lane == 0) {
          ptx::mbar_arrive(bar_full_b(sb));
          if (main_step) ptx::mbar_arrive(bar_empty_c(sc));
        }
      }
      mit += w.n_main;
    }
  } else if (warp >= 4 + 8 * MM_GROUPS) {
    // ------------------------------------------------------------ epilogue ----
    // A thread owns one token row (its TMEM lane) and reads 32 channels at a time.
    const int quarter = warp % 4;
    uint32_t tcount = 0;
    bool ok = true;
    for (int vt = blockIdx.x; vt < total_items && ok; vt += gridDim.x, ++tcount) {
      const MmItem w = mm_item(p, vt);
      const int ab = tcount % MM_NACC;
      if (!(ok = ptx::mbar_wait(bar_acc_full(ab), (tcount / MM_NACC) & 1, abort_flag))) break;
      ptx::tc_fence_after();
      const long long token = (long long)w.mt * MM_TOK + quarter * 32 + lane;
      const size_t out_off = (size_t)(token < p.M ? token : 0) * p.N + (size_t)w.nt * MM_CH;
      float* pdst = p.parts > 1 ? p.partial + (size_t)w.sp * p.M * p.N + out_off : nullptr;
      __nv_bfloat16* ydst = p.y + out_off;
#pragma unroll 1
      for (int col = 0; col < MM_CH; col += 32) {
        uint32_t v[32];
        if (QALORA_CHECK(p.dbg, ab * MM_CH + col + 31, 512))
          ptx::tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + ab * MM_CH + col, v);
        ptx::tmem_wait_ld();
        if (col == MM_CH - 32) {                  // all columns read: hand the accumulator back
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar_acc_empty(ab));
        }
        if (token < p.M && QALORA_CHECK(p.dbg, out_off + col + 31, (size_t)p.M * p.N) &&
            QALORA_CHECK(p.dbg, w.sp, p.parts)) {
          if (p.parts > 1) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              *reinterpret_cast<uint4*>(pdst + col + 4 * q) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
          } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              uint4 o;
              o.x = pack_bf16x2(__uint_as_float(v[8 * q]), __uint_as_float(v[8 * q + 1]));
              o.y = pack_bf16x2(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3]));
              o.z = pack_bf16x2(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5]));
              o.w = pack_bf16x2(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7]));
              *reinterpret_cast<uint4*>(ydst + col + 8 * q) = o;
            }
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown ----
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag != 0) atomicExch(p.status, 1);
  if (warp == 1) {
    __syncwarp();
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Parts the reduction is cut into: as many as fill the SMs evenly, each at least 4 steps long.
int mm_parts(const Shape& sh, int64_t M) {
  const long long tiles = (long long)(sh.N / MM_CH) * ((M + MM_TOK - 1) / MM_TOK);
  const int steps = sh.K / MM_J, sms = device_sm_count();
  int best = 1;
  double best_cost = 1e30;
  for (int ps = 1; ps <= 8; ++ps) {
    if (ps > 1 && steps / ps < 4) break;
    const double cost = (double)((tiles * ps + sms - 1) / sms) / ps + 0.02 * ps;    // waves x share of a tile + per-part start-up
    if (cost < best_cost - 1e-9) { best_cost = cost; best = ps; }
  }
  return best;
}

#ifndef QALORA_MM_PDL
#define QALORA_MM_PDL 1
#endif
template <int BITS, int XROWS>
int launch_midm_t(const CUtensorMap& xm, const CUtensorMap& tm, const MmParams& p, const uint32_t* codes,
                  const float2* qparams, cudaStream_t st) {
  using S = MmSmem<BITS, XROWS>;
  static_assert(S::TOTAL <= 232448, "shared memory budget");
  CUtensorMap cm, qm, lb = xm;
  // with adapter: B [r][N] in boxes of 64 channels x 64 rows (rows beyond r read as zero)
  if (p.r > 0 && !make_act_map(&lb, p.lora_B, p.r, p.N, MM_J)) return QALORA_ERR_CUDA;
  if (!make_codes_map(&cm, codes, p.K, p.N, BITS, 128, 2)) return QALORA_ERR_CUDA;
  if (!make_qp_map(&qm, qparams, p.K / p.g, p.N, 128, p.qp_rows)) return QALORA_ERR_CUDA;
  auto kern = qalora_midm_kernel<BITS, XROWS>;
  static PerDeviceOnce smem_limit;
  if (smem_limit.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S::TOTAL); }) != QALORA_OK)
    return QALORA_ERR_CUDA;
  const int items = p.n_tiles * p.m_tiles * p.parts;
  const int grid = items < device_sm_count() ? items : device_sm_count();
  {
    MainKernelProbe probe("qalora_midm_kernel", st);
    // With an adapter the kernel before this one in the stream is the few-row pooling kernel that
    // writes T (it lets its successor start at once): this kernel starts beside it, streams and
    // multiplies the weights, and waits for it only before the adapter step fetches T.  x, the
    // weights and the status word are final by then: the pooling kernel itself started after them.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(MM_THREADS);
    cfg.dynamicSmemBytes = S::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (QALORA_MM_PDL && p.r > 0) ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kern, xm, tm, lb, cm, qm, p) != cudaSuccess) return QALORA_ERR_CUDA;
  }
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return QALORA_ERR_CUDA;
  if (p.parts > 1) return launch_sum_parts_bf16(p.partial, p.y, (size_t)p.M * p.N, p.parts, st);
  return QALORA_OK;
}

}  // namespace

bool midm_supported(const Shape& sh, int64_t M) {
  return (sh.g == 32 || sh.g == 64 || sh.g == 128) && sh.N % MM_CH == 0 && sh.K % MM_J == 0 && sh.K / MM_J >= 4 &&
         M >= 1 && M <= MM_TOK && encode_fn() != nullptr;
}

size_t midm_partial_bytes(const Shape& sh, int64_t M) {
  const int ps = mm_parts(sh, M);
  return ps > 1 ? (size_t)ps * M * sh.N * sizeof(float) : 0;
}

// y = x * W~ + Tb * B with Tb = bf16(s * pool(x) * A) precomputed ([M][r]; ignored when r == 0).
// `partial`: midm_partial_bytes() of scratch.
int launch_midm(const Shape& sh, int64_t M, const __nv_bfloat16* x, const uint32_t* codes, const float2* qparams,
                const __nv_bfloat16* Tb, const __nv_bfloat16* B, __nv_bfloat16* y, float* partial, int* status,
                cudaStream_t st) {
  const int xrows = M <= 64 ? 64 : MM_TOK;                // rows an activation tile brings
  CUtensorMap xm, tm;
  if (!make_act_map(&xm, x, M, sh.K, xrows)) return QALORA_ERR_CUDA;
  tm = xm;
  if (sh.r > 0 && !make_act_map(&tm, Tb, M, sh.r, xrows)) return QALORA_ERR_CUDA;
  MmParams p{};
  p.lora_B = B; p.y = y; p.partial = partial;
  p.M = M; p.K = sh.K; p.N = sh.N; p.g = sh.g; p.r = sh.r;
  p.n_tiles = sh.N / MM_CH; p.m_tiles = (int)((M + MM_TOK - 1) / MM_TOK); p.parts = mm_parts(sh, M);
  p.red_iters = sh.K / MM_J; p.lora_iters = (sh.r + MM_J - 1) / MM_J;
  p.qp_rows = MM_J / sh.g > 0 ? MM_J / sh.g : 1;
  p.status = status; p.dbg = debug_words();
#define QALORA_MM(BITS) (xrows == 64 ? launch_midm_t<BITS, 64>(xm, tm, p, codes, qparams, st) : launch_midm_t<BITS, 128>(xm, tm, p, codes, qparams, st))
  if (sh.bits == 4) return QALORA_MM(4);
  if (sh.bits == 3) return QALORA_MM(3);
  return QALORA_MM(2);
#undef QALORA_MM
}

}  // namespace qalora
