// Few-token forward (M <= 32): y = x * W~ (+ T * B), bound by streaming the packed
// codes and the (alpha, beta) pairs from HBM exactly once.
//
// Design
//  * One block (eight consumer warps in two sets that take two k-blocks of a stage each, plus
//    one producer warp) owns 128 output columns and a slice of the input channels; the
//    slices of one column tile form a thread-block CLUSTER, and the partial sums
//    are added through distributed shared memory in a fixed order (no atomics,
//    no second kernel, no scratch).
//  * A single thread streams codes, qparams and the x slice into a shared-memory
//    ring with three tiled TMA copies per 128-channel stage, so that many tens of
//    KiB per SM are in flight without using registers.
//  * The products run on mma.sync.m16n8k16 (bf16 in, fp32 accumulate) with 16
//    columns of W as the rows and 8 tokens as the columns: a lane's 32-bit words
//    of packed codes ARE its A fragments after one shift and one mask per pair
//    (the code is OR-ed into the mantissa of bf16 128.0, no conversion; with 4-bit
//    codes one ldmatrix fetches the four words a lane needs for a k-block), and its
//    16-byte load of x is its B fragments.  The products x * (128 + c) are exact
//    in fp32; the two MMAs of a 32-channel block give D = sum (128 + c) x, and the
//    block is folded as
//        acc += alpha * D + (beta - 128 alpha) * xp,
//    where xp (the group sum of x, which the paper's pooling also needs) comes from one
//    more MMA with ones as the A operand (independent of the code MMAs).  alpha and beta
//    stay fp32.  With group sizes 64 and 128 a set's two k-blocks share (alpha, beta):
//    they go into one accumulator chain and are folded once.
//  * The same reduction step adds the adapter term T * B (T = s * pool(x) * A is
//    computed by the pooling kernel) and rounds to bf16.
//  * Launches of the layer without adapter carry the programmatic-dependent-launch
//    attribute: the kernel lets its successor start at once and itself starts as soon
//    as its predecessor allows, streams the first ring of codes and (alpha, beta) -
//    weights, which no kernel of a forward pass writes - and waits for the
//    predecessor's completion (griddepcontrol.wait) only before it fetches x; y is
//    written after every stage, hence every x slice, has been consumed.
//    Back-to-back layers of a decoding step thus overlap one layer's tail with the
//    next one's start.
#define QALORA_TU 2
#include <cooperative_groups.h>

#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace cg = cooperative_groups;

namespace qalora {

namespace {

constexpr int GV_COLS = 128;        // columns per block
constexpr int GV_SETS = 2;          // consumer warp sets; set s takes the k-blocks b with b % 2 == s
constexpr int GV_WARPS = 4 * GV_SETS;   // consumer warps: 4 per set, 32 columns each
constexpr int GV_THREADS = (GV_WARPS + 1) * 32;   // + 1 producer warp
constexpr int GV_KBS = 4;           // 32-channel blocks per stage (128 channels)
constexpr int GV_ROWS = 32;         // most token rows

template <int BITS, int NTS>      // NTS: sets of 8 token rows (1, 2 or 4)
struct GvSmem {
  static constexpr int ROWS = 8 * NTS;                                  // token rows held in shared memory
  static constexpr int STAGES = NTS == 1 ? 4 : 3;                       // three blocks per SM (two with 32 rows)
  static constexpr int WORDS = BITS == 4 ? 4 : (BITS == 3 ? 3 : 2);
  static constexpr uint32_t CODE_ROW = GV_COLS * WORDS * 4;             // one k-block row of units
  static constexpr uint32_t QP_ROW = GV_COLS * 8;
  static constexpr uint32_t X_BYTES = ROWS * GV_KBS * 32 * 2;           // rows x 128 channels bf16
  static constexpr uint32_t OFF_CODES = 0;
  static constexpr uint32_t OFF_QP = GV_KBS * CODE_ROW;
  static constexpr uint32_t OFF_X = OFF_QP + GV_KBS * QP_ROW;
  static constexpr uint32_t STAGE_BYTES = ((OFF_X + X_BYTES + 127) / 128) * 128;
  static constexpr uint32_t RING_BYTES = STAGES * STAGE_BYTES;
  // fp32 partial sums [sets][rows][128]: written after the last stage has been consumed,
  // over the ring's memory
  static constexpr uint32_t PARTIAL_BYTES = GV_SETS * ROWS * GV_COLS * 4;
  static constexpr uint32_t OFF_PARTIAL = 0;
  static_assert(PARTIAL_BYTES <= RING_BYTES, "the partial sums reuse the ring");
  static constexpr uint32_t OFF_BARS = RING_BYTES;
  static constexpr uint32_t TOTAL = OFF_BARS + 128 + 128;               // + alignment slack
};

struct GvParams {
  const uint32_t* codes;
  const float2* qparams;
  const __nv_bfloat16* Tb;      // bf16 [M][r], T = s * pool(x) * A, or null
  const __nv_bfloat16* B;       // [r][N]
  __nv_bfloat16* y;             // [M][N]
  int M, K, N, g, r;
  int total_stages;             // K / 128
  int* status;
  int reset_status;             // the first block clears *status before any wait can expire
  int pdl_wait;                 // launched beside its predecessor: the producer waits for it before it fetches x
  int stop_after_stages;        // normally INT_MAX; a test makes every producer stop early, so that waits expire
  unsigned long long wait_limit_ns;
  int* dbg;                     // record words of the bounds-check build (null otherwise)
};

// (not volatile: a pure function of its operands, so that independent MMAs can be interleaved)
__device__ __forceinline__ void mma16816(float* d, const uint32_t* a, uint32_t b0, uint32_t b1, const float* c) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}

// The four bf16x2 fragments (128 + c) of the 8 positions 8t .. 8t+7 of a unit, t = lane % 4.
// `lo` is the word that holds the (low) code bits of those positions, already shifted so
// that they start at bit 0 of each half-word; `hi` (3-bit codes only) the third-bit word
// shifted likewise.
//
// The logic/shift pipe is what this kernel runs out of first, so the extraction is spelled
// out: the constants live in registers (FragConsts; a LOP3 takes one immediate at most, and
// with two it becomes two instructions) and "(a & mask) | magic" is one LOP3.  (Shifting by
// mul.hi on the multiplier pipe instead was measured slower.)
struct FragConsts {
  uint32_t mask, magic;
};
template <int BITS>
__device__ __forceinline__ FragConsts frag_consts() {
  FragConsts c;
  // asm volatile: the values stay opaque, so that they are not turned back into immediates
  asm volatile("mov.b32 %0, %1;" : "=r"(c.mask) : "n"(BITS == 4 ? 0x000f000f : 0x00030003));
  asm volatile("mov.b32 %0, 0x43004300;" : "=r"(c.magic));
  return c;
}
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {   // (a & b) | c
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
template <int BITS>
__device__ __forceinline__ void code_fragments(uint32_t lo, uint32_t hi, const FragConsts& k, uint32_t* f) {
  constexpr int W = BITS == 4 ? 4 : 2;          // field width of the (low) code bits
#pragma unroll
  for (int i = 0; i < 4; ++i) f[i] = and_or(lo >> (W * i), k.mask, k.magic);
  if (BITS == 3) {
#pragma unroll
    for (int i = 0; i < 4; ++i) f[i] |= ((hi >> i) & 0x00010001u) << 2;
  }
}

// The fold of one k-block (or chain of two) into the running sums of a 16-column group:
// acc += alpha * D + (beta - 128 alpha) * xp for the fragment's (column gq | gq + 8) x (token
// 2t | 2t + 1), as packed two-lane FMAs.  With one token row the odd token column of the
// fragment is all padding and only the two columns of token 2t are folded (one packed pair).
#ifndef QALORA_GV_FFMA2
#define QALORA_GV_FFMA2 1
#endif
template <bool ONE>
__device__ __forceinline__ void fold(float* acc, const float* D, const float* xp, float2 q0, float2 q1) {
#if QALORA_GV_FFMA2
  if constexpr (ONE) {
    const float2 r = ptx::ffma2(make_float2(q0.x, q1.x), make_float2(D[0], D[2]),
                                ptx::ffma2(make_float2(q0.y, q1.y), make_float2(xp[0], xp[0]), make_float2(acc[0], acc[2])));
    acc[0] = r.x; acc[2] = r.y;
  } else {
    const float2 xp2 = make_float2(xp[0], xp[1]);
    const float2 r0 = ptx::ffma2(make_float2(q0.x, q0.x), make_float2(D[0], D[1]),
                                 ptx::ffma2(make_float2(q0.y, q0.y), xp2, make_float2(acc[0], acc[1])));
    const float2 r1 = ptx::ffma2(make_float2(q1.x, q1.x), make_float2(D[2], D[3]),
                                 ptx::ffma2(make_float2(q1.y, q1.y), xp2, make_float2(acc[2], acc[3])));
    acc[0] = r0.x; acc[1] = r0.y; acc[2] = r1.x; acc[3] = r1.y;
  }
#else
  acc[0] = fmaf(q0.x, D[0], fmaf(q0.y, xp[0], acc[0]));
  if constexpr (!ONE) acc[1] = fmaf(q0.x, D[1], fmaf(q0.y, xp[1], acc[1]));
  acc[2] = fmaf(q1.x, D[2], fmaf(q1.y, xp[0], acc[2]));
  if constexpr (!ONE) acc[3] = fmaf(q1.x, D[3], fmaf(q1.y, xp[1], acc[3]));
#endif
}

// NTS: sets of 8 token rows in use (M <= 8 NTS).  CHAIN: the group size is 64 or 128, so the two
// k-blocks a warp set takes from a stage share (alpha, beta) and are folded together.
// The work of one block: `block` is its index among the blocks of the layer described by p
// (a layer's blocks are consecutive in the grid, a whole number of clusters).
template <int BITS, int NTS, bool CHAIN, bool ONE = false>   // ONE: a single token row (M == 1; NTS == 1)
__device__ __forceinline__ void gemv_block(const CUtensorMap& x_map, const CUtensorMap& codes_map,
                                           const CUtensorMap& qp_map, const GvParams& p, const int block) {
  using S = GvSmem<BITS, NTS>;
  constexpr int WORDS = S::WORDS;
  constexpr int GV_STAGES = S::STAGES;
  extern __shared__ uint8_t smem_raw[];
  // aligned by pointer arithmetic on the __shared__ array, so that the accesses stay shared-space loads/stores
  uint8_t* smem = smem_raw + ((128u - (ptx::smem_u32(smem_raw) & 127u)) & 127u);
  const uint32_t smem_base = ptx::smem_u32(smem);
  auto bar_full = [&](int s) { return smem_base + S::OFF_BARS + 8u * s; };
  auto bar_empty = [&](int s) { return smem_base + S::OFF_BARS + 8u * (GV_STAGES + s); };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::OFF_BARS + 8 * (2 * GV_STAGES));
  float* partial = reinterpret_cast<float*>(smem + S::OFF_PARTIAL);

  cg::cluster_group cluster = cg::this_cluster();
  const int splits = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int n0 = (block / splits) * GV_COLS;
  const int st_beg = (int)((long long)p.total_stages * rank / splits);
  const int st_end = (int)((long long)p.total_stages * (rank + 1) / splits);
  const int n_stages = st_end - st_beg;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    for (int s = 0; s < GV_STAGES; ++s) {
      ptx::mbar_init(bar_full(s), 1);
      ptx::mbar_init(bar_empty(s), GV_WARPS);
    }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&x_map);
    ptx::prefetch_tensormap(&codes_map);
    ptx::prefetch_tensormap(&qp_map);
    if (block == 0 && p.reset_status) *p.status = 0;     // a wait gives up only after seconds: no block can have raised it yet
    // the next kernel in the stream may start (it waits for this one's completion before it
    // reads or writes anything this one touches)
    asm volatile("griddepcontrol.launch_dependents;");
  }
  __syncthreads();

  if (warp == GV_WARPS) {
    // ------------------------------------------------------------ producer ----
    if (lane == 0) {
      const int n_issue = n_stages < p.stop_after_stages ? n_stages : p.stop_after_stages;
      const int qrows = (GV_KBS * 32) / p.g;
      const uint32_t stage_tx = GV_KBS * S::CODE_ROW + qrows * S::QP_ROW + S::X_BYTES;
      // three tiled copies per stage: 4 k-block rows of pack units, the rows of
      // (alpha, beta) they need (128 / g of them) and the x slice.  The first ring of
      // weights goes out at once; x follows when the predecessor kernel is complete.
      const int first = n_issue < GV_STAGES ? n_issue : GV_STAGES;
      // (bounds-check build: the block's last stage and its columns lie inside the matrices)
      QALORA_CHECK(p.dbg, (long long)st_end * GV_KBS - 1, p.K / 32);
      QALORA_CHECK(p.dbg, n0 + GV_COLS - 1, p.N);
      QALORA_CHECK(p.dbg, st_end * GV_KBS * 32 / p.g - 1, p.K / p.g);
      if (p.pdl_wait) {
        for (int it = 0; it < first; ++it) {
          const int st = st_beg + it;
          const uint32_t stage = smem_base + it * S::STAGE_BYTES;
          ptx::mbar_arrive_expect_tx(bar_full(it), stage_tx);
          ptx::tma_load_2d(stage + S::OFF_CODES, &codes_map, n0 * WORDS / 2, st * GV_KBS, bar_full(it));
          ptx::tma_load_2d(stage + S::OFF_QP, &qp_map, 2 * n0, st * GV_KBS * 32 / p.g, bar_full(it));
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int it = 0; it < first; ++it)
          ptx::tma_load_2d(smem_base + it * S::STAGE_BYTES + S::OFF_X, &x_map, (st_beg + it) * GV_KBS * 32, 0, bar_full(it));
      } else {
        for (int it = 0; it < first; ++it) {      // no predecessor to wait for: each stage's three copies together
          const int st = st_beg + it;
          const uint32_t stage = smem_base + it * S::STAGE_BYTES;
          ptx::mbar_arrive_expect_tx(bar_full(it), stage_tx);
          ptx::tma_load_2d(stage + S::OFF_CODES, &codes_map, n0 * WORDS / 2, st * GV_KBS, bar_full(it));
          ptx::tma_load_2d(stage + S::OFF_QP, &qp_map, 2 * n0, st * GV_KBS * 32 / p.g, bar_full(it));
          ptx::tma_load_2d(stage + S::OFF_X, &x_map, st * GV_KBS * 32, 0, bar_full(it));
        }
      }
      bool ok = true;
      int s = 0;
      uint32_t ph = 0;                              // phase of bar_empty(s) the refill of slot s waits for
      for (int it = first; it < n_issue && ok; ++it) {
        const int st = st_beg + it;
        if (!(ok = ptx::mbar_wait(bar_empty(s), ph, abort_flag, p.wait_limit_ns))) break;
        const uint32_t stage = smem_base + s * S::STAGE_BYTES;
        ptx::mbar_arrive_expect_tx(bar_full(s), stage_tx);
        ptx::tma_load_2d(stage + S::OFF_CODES, &codes_map, n0 * WORDS / 2, st * GV_KBS, bar_full(s));
        ptx::tma_load_2d(stage + S::OFF_QP, &qp_map, 2 * n0, st * GV_KBS * 32 / p.g, bar_full(s));
        ptx::tma_load_2d(stage + S::OFF_X, &x_map, st * GV_KBS * 32, 0, bar_full(s));
        if (++s == GV_STAGES) { s = 0; ph ^= 1; }
      }
    }
  } else {
    // ----------------------------------------------------------- consumers ----
    // Warp w of set s owns columns 32 (w % 4) .. + 31 and the k-blocks b of each stage
    // with b / 2 == s.  The weights are the A operand (16 columns x 16 channels per
    // MMA) and the tokens the B operand (8 token columns), so that a lane's fragments of x
    // are the register pairs its 16-byte load delivered and the code fragments are built
    // in place.  Every k-block is folded on its own (the fold is linear, so the k-blocks
    // of one quantization group may be folded separately with the same alpha and beta).
    const int set = warp / 4, wcol = (warp % 4) * 32;
    const int qsh = p.g == 32 ? 0 : (p.g == 64 ? 1 : 2);   // k-block of the stage -> its (alpha, beta) row
    const int gq = lane / 4, t = lane % 4;        // fragment row (column of W, token), quad lane

    // per-thread byte offsets inside a stage; everything else is a compile-time constant
    const uint32_t x_off = S::OFF_X + gq * (GV_KBS * 64) + t * 16 + set * (GV_KBS / GV_SETS) * 64;
    const uint32_t lo_word = BITS == 4 ? t : (t >> 1);
    const uint32_t lo_shift = BITS == 4 ? 0 : 8 * (t & 1);
    const uint32_t c_off = S::OFF_CODES + set * (GV_KBS / GV_SETS) * S::CODE_ROW + ((wcol + gq) * WORDS + lo_word) * 4;
    const uint32_t h_off = S::OFF_CODES + set * (GV_KBS / GV_SETS) * S::CODE_ROW + ((wcol + gq) * WORDS + 2) * 4;   // 3-bit codes: third-bit word
    // 4-bit codes: ldmatrix row address of this lane (matrix lane / 8 = 8-column group, row lane % 8:
    // the unit of column wcol + lane); thread (gq, t) then holds word t of the units of columns
    // wcol + gq, + 8, + 16, + 24
    const uint32_t m_off = S::OFF_CODES + set * (GV_KBS / GV_SETS) * S::CODE_ROW + (wcol + lane) * 16;
    const uint32_t q_off = S::OFF_QP + (wcol + gq) * 8;
    float acc[2][NTS][4];                         // [16-column group][token set][(col gq | gq + 8) x (token 2t | 2t + 1)]
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
      for (int ts = 0; ts < NTS; ++ts)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[c][ts][i] = 0.f;
    const float zero4[4] = {0.f, 0.f, 0.f, 0.f};
    const FragConsts fk = frag_consts<BITS>();
    constexpr uint32_t ONES = 0x3f803f80u;        // bf16x2 (1, 1)
    const uint32_t ones4[4] = {ONES, ONES, ONES, ONES};
    bool ok = true;
    // (bounds-check build: the last byte this thread reads of a stage's x slice, code rows and (alpha, beta) rows)
    ok = QALORA_CHECK(p.dbg, x_off + (GV_KBS / GV_SETS - 1) * 64 + (NTS - 1) * 8 * (GV_KBS * 64) + 15, S::OFF_X + S::X_BYTES) &&
         QALORA_CHECK(p.dbg, (BITS == 4 ? m_off + 15 : (BITS == 3 ? h_off : c_off) + 24 * WORDS * 4 + 3) + (GV_KBS / GV_SETS - 1) * S::CODE_ROW,
                      S::OFF_CODES + GV_KBS * S::CODE_ROW) &&
         QALORA_CHECK(p.dbg, q_off + ((GV_KBS - 1) >> qsh) * S::QP_ROW + 24 * 8 + 7, S::OFF_QP + ((GV_KBS * 32) / p.g) * S::QP_ROW);
    int s = 0;
    uint32_t ph = 0;
    for (int it = 0; it < n_stages && ok; ++it) {
      if (!(ok = ptx::mbar_wait(bar_full(s), ph, abort_flag, p.wait_limit_ns))) break;
      const uint8_t* stage = smem + s * S::STAGE_BYTES;
      // words of the codes of a k-block: w[2 cg + j] = this lane's word of column wcol + 16 cg + 8 j + gq
      auto load_words = [&](int bb, uint32_t* w, uint32_t* hi) {
        if constexpr (BITS == 4) {
          const uint32_t addr = smem_base + s * S::STAGE_BYTES + m_off + bb * S::CODE_ROW;
          asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                       : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr));
          hi[0] = hi[1] = hi[2] = hi[3] = 0u;
        } else {
#pragma unroll
          for (int m = 0; m < 4; ++m) {
            const uint32_t coff = bb * S::CODE_ROW + (m * 8) * WORDS * 4;
            w[m] = *reinterpret_cast<const uint32_t*>(stage + c_off + coff) >> lo_shift;
            hi[m] = BITS == 3 ? *reinterpret_cast<const uint32_t*>(stage + h_off + coff) >> (4 * t) : 0u;
          }
        }
      };
      if constexpr (CHAIN) {
        // the set's two k-blocks lie in one quantization group: one accumulator chain over
        // both (four MMAs per 16 columns), one fold, one (alpha, beta) load
        uint4 xs[2][NTS];
        float xp[NTS][2];
#pragma unroll
        for (int ts = 0; ts < NTS; ++ts) {
#pragma unroll
          for (int bb = 0; bb < 2; ++bb)
            xs[bb][ts] = *reinterpret_cast<const uint4*>(stage + x_off + bb * 64 + ts * 8 * (GV_KBS * 64));
          // xp of the tokens over both k-blocks (ones as the A operand: every row of the product holds the sums)
          float pool[4];
          mma16816(pool, ones4, xs[0][ts].x, xs[0][ts].y, zero4);
          mma16816(pool, ones4, xs[0][ts].z, xs[0][ts].w, pool);
          mma16816(pool, ones4, xs[1][ts].x, xs[1][ts].y, pool);
          mma16816(pool, ones4, xs[1][ts].z, xs[1][ts].w, pool);
          xp[ts][0] = pool[0];
          xp[ts][1] = pool[1];
        }
        uint32_t w[2][4], hi[2][4];
        load_words(0, w[0], hi[0]);
        load_words(1, w[1], hi[1]);
        const uint8_t* qrow = stage + q_off + (((set * (GV_KBS / GV_SETS)) >> qsh) * S::QP_ROW);
#pragma unroll
        for (int cg = 0; cg < 2; ++cg) {
          float D[NTS][4];
#pragma unroll
          for (int bb = 0; bb < 2; ++bb) {
            uint32_t f[2][4];
#pragma unroll
            for (int j = 0; j < 2; ++j) code_fragments<BITS>(w[bb][2 * cg + j], hi[bb][2 * cg + j], fk, f[j]);
            const uint32_t a0[4] = {f[0][0], f[1][0], f[0][1], f[1][1]};
            const uint32_t a1[4] = {f[0][2], f[1][2], f[0][3], f[1][3]};
#pragma unroll
            for (int ts = 0; ts < NTS; ++ts) {
              mma16816(D[ts], a0, xs[bb][ts].x, xs[bb][ts].y, bb == 0 ? zero4 : D[ts]);
              mma16816(D[ts], a1, xs[bb][ts].z, xs[bb][ts].w, D[ts]);
            }
          }
          float2 q0 = *reinterpret_cast<const float2*>(qrow + (cg * 16) * 8);
          float2 q1 = *reinterpret_cast<const float2*>(qrow + (cg * 16 + 8) * 8);
          q0.y = fmaf(-128.f, q0.x, q0.y);      // D holds sum (128 + c) x: the offset goes into the xp term
          q1.y = fmaf(-128.f, q1.x, q1.y);
#pragma unroll
          for (int ts = 0; ts < NTS; ++ts) {
            fold<ONE>(acc[cg][ts], D[ts], xp[ts], q0, q1);
          }
        }
      } else {
#pragma unroll
        for (int bb = 0; bb < GV_KBS / GV_SETS; ++bb) {
          // this set's k-block b = 2 set + bb; B fragments: x[token gq (+ 8)][32 b + 8 t .. + 7]:
          // the lane's k slots (2t, 2t+1 | 2t+8, 2t+9) of MMA 0 are channels 8t .. 8t+3, those of MMA 1 8t+4 .. 8t+7
          uint4 xs[NTS];
          float xp[NTS][2];
#pragma unroll
          for (int ts = 0; ts < NTS; ++ts) {
            xs[ts] = *reinterpret_cast<const uint4*>(stage + x_off + bb * 64 + ts * 8 * (GV_KBS * 64));
            // xp of the tokens (ones as the A operand: every row of the product holds the sums)
            float pool[4];
            mma16816(pool, ones4, xs[ts].x, xs[ts].y, zero4);
            mma16816(pool, ones4, xs[ts].z, xs[ts].w, pool);
            xp[ts][0] = pool[0];
            xp[ts][1] = pool[1];
          }
          uint32_t w[4], hi[4];
          load_words(bb, w, hi);
          const uint8_t* qrow = stage + q_off + (((set * (GV_KBS / GV_SETS) + bb) >> qsh) * S::QP_ROW);
#pragma unroll
          for (int cg = 0; cg < 2; ++cg) {
            // columns wcol + 16 cg + gq (fragment rows 0..7) and + 8 (rows 8..15)
            uint32_t f[2][4];
#pragma unroll
            for (int j = 0; j < 2; ++j) code_fragments<BITS>(w[2 * cg + j], hi[2 * cg + j], fk, f[j]);
            float2 q0 = *reinterpret_cast<const float2*>(qrow + (cg * 16) * 8);
            float2 q1 = *reinterpret_cast<const float2*>(qrow + (cg * 16 + 8) * 8);
            q0.y = fmaf(-128.f, q0.x, q0.y);    // D holds sum (128 + c) x: the offset goes into the xp term
            q1.y = fmaf(-128.f, q1.x, q1.y);
            const uint32_t a0[4] = {f[0][0], f[1][0], f[0][1], f[1][1]};
            const uint32_t a1[4] = {f[0][2], f[1][2], f[0][3], f[1][3]};
#pragma unroll
            for (int ts = 0; ts < NTS; ++ts) {
              float D[4];
              mma16816(D, a0, xs[ts].x, xs[ts].y, zero4);
              mma16816(D, a1, xs[ts].z, xs[ts].w, D);
              fold<ONE>(acc[cg][ts], D, xp[ts], q0, q1);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar_empty(s));
      if (++s == GV_STAGES) { s = 0; ph ^= 1; }
    }
    // every consumer warp has left the ring before the partial sums overwrite it
    ptx::named_barrier(1, GV_WARPS * 32);
    if (p.r > 0 && rank == 0) {
      // Adapter term T * B, once per column tile (by the cluster's first block), as more MMAs
      // into the same accumulators: rows = columns of B (A operand: B transposed, two 2-byte
      // loads per register, from L2), columns = tokens (B operand: T in bf16, as the
      // tensor-core kernel takes it).  The sets take alternate 16-row steps of the rank;
      // rows beyond it read as zero.  T is written by the pooling kernel, which this kernel
      // is allowed to overtake (programmatic stream serialization): wait for it only now (a
      // no-op when the launch carried no such attribute).
      asm volatile("griddepcontrol.wait;" ::: "memory");
      const unsigned short* Bu = reinterpret_cast<const unsigned short*>(p.B);
      const unsigned short* Tu = reinterpret_cast<const unsigned short*>(p.Tb);
      auto pair = [](const unsigned short* base, size_t stride, int i, int r) -> uint32_t {   // (base[i], base[i + 1]) along stride
        const uint32_t lo = i < r ? base[(size_t)i * stride] : 0u;
        const uint32_t hi = i + 1 < r ? base[(size_t)(i + 1) * stride] : 0u;
        return lo | (hi << 16);
      };
      const int ksteps = (p.r + 15) / 16;
      for (int ks = set; ks < ksteps; ks += GV_SETS) {
        const int i0 = ks * 16 + 2 * t;
        uint32_t tb[NTS][2];
#pragma unroll
        for (int ts = 0; ts < NTS; ++ts) {
          const int token = ts * 8 + gq;
          const bool live = token < p.M;
          const unsigned short* Tr = Tu + (size_t)(live ? token : 0) * p.r;
          QALORA_CHECK(p.dbg, (size_t)(live ? token : 0) * p.r, (size_t)p.M * p.r);
          tb[ts][0] = live ? pair(Tr, 1, i0, p.r) : 0u;
          tb[ts][1] = live ? pair(Tr, 1, i0 + 8, p.r) : 0u;
        }
#pragma unroll
        for (int cg = 0; cg < 2; ++cg) {
          const unsigned short* c0 = Bu + n0 + wcol + cg * 16 + gq;
          if (!QALORA_CHECK(p.dbg, n0 + wcol + cg * 16 + gq + 8, p.N)) continue;
          const uint32_t a[4] = {pair(c0, p.N, i0, p.r), pair(c0 + 8, p.N, i0, p.r),
                                 pair(c0, p.N, i0 + 8, p.r), pair(c0 + 8, p.N, i0 + 8, p.r)};
#pragma unroll
          for (int ts = 0; ts < NTS; ++ts) mma16816(acc[cg][ts], a, tb[ts][0], tb[ts][1], acc[cg][ts]);
        }
      }
    }
    // partial sums of this warp set: [16 token rows][128 columns]
    float* mine = partial + set * (S::ROWS * GV_COLS);
#pragma unroll
    for (int cg = 0; cg < 2; ++cg)
#pragma unroll
      for (int ts = 0; ts < NTS; ++ts) {
        const int col = wcol + cg * 16 + gq, row = ts * 8 + 2 * t;
        if (!QALORA_CHECK(p.dbg, (set * S::ROWS + row + 1) * GV_COLS + col + 8, S::PARTIAL_BYTES / 4)) continue;
        mine[row * GV_COLS + col] = acc[cg][ts][0];
        mine[(row + 1) * GV_COLS + col] = acc[cg][ts][1];
        mine[row * GV_COLS + col + 8] = acc[cg][ts][2];
        mine[(row + 1) * GV_COLS + col + 8] = acc[cg][ts][3];
      }
  }

  // ---- add the slices in rank order through distributed shared memory ---------
  cluster.sync();
  {
    const int col_beg = GV_COLS * rank / splits, col_end = GV_COLS * (rank + 1) / splits;
    const int cols_per = col_end - col_beg;
    const int outs = p.M * cols_per;
    for (int o = threadIdx.x; o < outs; o += GV_THREADS) {
      const int row = o / cols_per, col = col_beg + o % cols_per;
      float v = 0.f;
      for (int rk = 0; rk < splits; ++rk) {
        const float* remote = cluster.map_shared_rank(partial, rk);
#pragma unroll
        for (int sset = 0; sset < GV_SETS; ++sset) v += remote[sset * (S::ROWS * GV_COLS) + row * GV_COLS + col];
      }
      if (QALORA_CHECK(p.dbg, (size_t)row * p.N + n0 + col, (size_t)p.M * p.N)) p.y[(size_t)row * p.N + n0 + col] = __float2bfloat16_rn(v);
    }
  }
  cluster.sync();
  if (threadIdx.x == 0 && *abort_flag != 0) atomicExch(p.status, 1);
}

template <int BITS, int NTS, bool CHAIN, bool ONE = false>
__global__ void __launch_bounds__(GV_THREADS, NTS == 4 ? 2 : 3)
qalora_gemv_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap codes_map,
                   const __grid_constant__ CUtensorMap qp_map, const GvParams p) {
  gemv_block<BITS, NTS, CHAIN, ONE>(x_map, codes_map, qp_map, p, (int)blockIdx.x);
}

// Several layers in ONE launch (the projections of a transformer block that read finished
// inputs: q, k, v; gate, up; or any set of independent layers): block b works for the layer l
// with first_block[l] <= b < first_block[l + 1].  Launch, cluster set-up and the first bytes'
// latency are paid once for all of them.
constexpr int GV_GROUP_MAX = 8;
struct GvGroup {
  CUtensorMap x_map[GV_GROUP_MAX], codes_map[GV_GROUP_MAX], qp_map[GV_GROUP_MAX];
  GvParams p[GV_GROUP_MAX];
  int first_block[GV_GROUP_MAX + 1];
  int n;
};

template <int BITS, int NTS, bool CHAIN>
__global__ void __launch_bounds__(GV_THREADS, NTS == 4 ? 2 : 3)
qalora_gemv_group_kernel(const __grid_constant__ GvGroup grp) {
  int l = 0;
  while (l + 1 < grp.n && (int)blockIdx.x >= grp.first_block[l + 1]) ++l;      // the same for every thread of a cluster
  gemv_block<BITS, NTS, CHAIN>(grp.x_map[l], grp.codes_map[l], grp.qp_map[l], grp.p[l], (int)blockIdx.x - grp.first_block[l]);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn gv_encode_fn() {
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

// Tensor maps of a layer's weights: packed codes [K/32][N][words] uint32 seen as a 2-D matrix of
// 8-byte elements, so that one box row is the whole contiguous run of 128 pack units (2 KiB at
// 4 bits), and (alpha, beta) float32 [G][2N] with a box of 256 floats x (128 / g) rows.
bool make_weight_maps(const GvParams& p, int words, CUtensorMap* cm, CUtensorMap* qm) {
  EncodeTiledFn fn = gv_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)p.N * words / 2, (cuuint64_t)(p.K / 32)};
  cuuint64_t strides[1] = {(cuuint64_t)p.N * words * 4};
  cuuint32_t box[2] = {(cuuint32_t)(GV_COLS * words / 2), GV_KBS};
  cuuint32_t estr[2] = {1, 1};
  if (fn(cm, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<uint32_t*>(p.codes), dims, strides, box, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  cuuint64_t qdims[2] = {(cuuint64_t)p.N * 2, (cuuint64_t)(p.K / p.g)};
  cuuint64_t qstrides[1] = {(cuuint64_t)p.N * 8};
  cuuint32_t qbox[2] = {2 * GV_COLS, (cuuint32_t)((GV_KBS * 32) / p.g)};
  cuuint32_t qestr[2] = {1, 1};
  return fn(qm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float2*>(p.qparams), qdims, qstrides, qbox, qestr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// x bf16 [M][K]; box = 128 channels x the token rows the kernel keeps (8, 16 or 32; rows beyond M read as zero)
bool make_x_map(const __nv_bfloat16* x, int K, int64_t M, CUtensorMap* xm) {
  EncodeTiledFn fn = gv_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {GV_KBS * 32, (cuuint32_t)(M > 16 ? 32 : (M > 8 ? 16 : 8))};
  cuuint32_t estr[2] = {1, 1};
  return fn(xm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Launch configuration shared by the single-layer and the grouped kernel: `blocks` blocks in
// clusters of `splits`; with `programmatic` the launch carries programmatic stream serialization.
template <class Kernel, class... Args>
cudaError_t launch_clustered(Kernel kern, unsigned blocks, int splits, size_t smem, bool programmatic, cudaStream_t st,
                             const char* probe_name, const Args&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(GV_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic ? 2 : 1;
  cudaError_t e;
  {
    MainKernelProbe probe(probe_name, st);
    e = cudaLaunchKernelEx(&cfg, kern, args...);
  }
  count_launch();
  return e;
}

template <int BITS, int NTS, bool CHAIN, bool ONE = false>
int launch_gemv_t(const CUtensorMap& xm, const GvParams& p, int splits, cudaStream_t st) {
  using S = GvSmem<BITS, NTS>;
  CUtensorMap cm, qm;
  if (!make_weight_maps(p, S::WORDS, &cm, &qm)) return QALORA_ERR_CUDA;
  auto kern = qalora_gemv_kernel<BITS, NTS, CHAIN, ONE>;
  static PerDeviceOnce smem_limit;      // this instantiation's shared-memory limit, raised once on every device it runs on
  if (smem_limit.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S::TOTAL); }) != QALORA_OK)
    return QALORA_ERR_CUDA;
  // Programmatic stream serialization lets this kernel start before its predecessor in the
  // stream has finished.  Without adapter (p.pdl_wait) that is always wanted: the kernel
  // streams its first ring of weights at once and waits for the predecessor only before it
  // fetches x.  With an adapter the predecessor is the pooling kernel that writes T, which
  // is read only after the last stage: the kernel starts beside it.  With more than 8 token
  // rows the pooling kernel is larger, and beside a short main loop the overlap measured
  // slower (4096 x 4096, 16 rows: 15.7 against 14.8 us), beside a long one faster
  // (8192 x 22016: 56 against 63 us): there it is used from 64 Mi weights on.
  const bool programmatic = p.pdl_wait != 0 || (p.Tb != nullptr && (NTS == 1 || (long long)p.K * p.N >= (64ll << 20)));
  return cuda_status(launch_clustered(kern, (unsigned)((p.N / GV_COLS) * splits), splits, S::TOTAL, programmatic, st,
                                      "qalora_gemv_kernel", xm, cm, qm, p));
}

template <int BITS, int NTS, bool CHAIN>
int launch_gemv_group_t(const GvGroup& grp, int splits, bool programmatic, cudaStream_t st) {
  using S = GvSmem<BITS, NTS>;
  auto kern = qalora_gemv_group_kernel<BITS, NTS, CHAIN>;
  static PerDeviceOnce smem_limit;
  if (smem_limit.run([&] { return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S::TOTAL); }) != QALORA_OK)
    return QALORA_ERR_CUDA;
  return cuda_status(launch_clustered(kern, (unsigned)grp.first_block[grp.n], splits, S::TOTAL, programmatic, st,
                                      "qalora_gemv_group_kernel", grp));
}

}  // namespace

// Test hook (see qalora_debug_expire_next_few_token_wait in api.cu): when armed, the producers
// of the next few-token launch stop after `stages` stages of their slice and its waits give up
// after `limit_ns`, so that the consumers' waits run out: the bounded-wait path (status word,
// orderly exit) can be exercised without a fault and without a kernel that hangs.
std::atomic<int> g_expire_after_stages{0x7fffffff};
std::atomic<unsigned long long> g_expire_limit_ns{ptx::WAIT_LIMIT_NS};
void arm_few_token_wait_expiry(int stages, unsigned long long limit_ns) {
  g_expire_limit_ns.store(limit_ns);
  g_expire_after_stages.store(stages < 0 ? 0 : stages);
}

// Slices per column tile (= cluster size): the count among {1,2,3,4,6,8} that brings the
// grid closest to two blocks per SM.  Three blocks fit on an SM, so the grid stays one
// wave with room for imbalance, while a block still streams enough bytes to amortize its
// fixed cost (launch, barrier set-up, first-byte latency, two cluster barriers).  With more
// than 16 token rows only two blocks fit on an SM: there the grid must not exceed two blocks
// per SM, or a second wave would follow.
static int gv_slices(const Shape& sh, int64_t M) {
  const int tiles = sh.N / GV_COLS, total_stages = sh.K / (GV_KBS * 32), target = 2 * device_sm_count();
  const bool capped = M > 16;
  int splits = 1, best = 1 << 30;
  for (int sp : {1, 2, 3, 4, 6, 8}) {
    if (sp > total_stages) break;
    if (capped && sp > 1 && tiles * sp > target) break;
    const int miss = tiles * sp > target ? tiles * sp - target : target - tiles * sp;
    if (miss < best) { best = miss; splits = sp; }
  }
  return splits;
}

bool gemv_supported(const Shape& sh, int64_t M) {
  if (!(M >= 1 && M <= GV_ROWS && sh.N % GV_COLS == 0 && sh.K % (GV_KBS * 32) == 0 &&
        (sh.g == 32 || sh.g == 64 || sh.g == 128) && gv_encode_fn() != nullptr))
    return false;
  if (M > 16) {
    // 17..32 rows: the tensor-pipe work per code grows with the rows and only two blocks fit
    // on an SM, so this kernel beats the 64-token tensor-core tile only where its grid fills
    // the SMs evenly (measured, merged layers: 15 against 20 us for a 4096 x 4096 layer whose
    // 256 blocks fill 86 % of two per SM; 116 against 88 us for 8192 x 22016, whose 172 blocks
    // fill 58 %).  Layers with and without adapter alike: the adapter term is a few more MMAs
    // into the same accumulators.
    const int sms = device_sm_count();
    const long long blocks = (long long)(sh.N / GV_COLS) * gv_slices(sh, M);
    const long long waves = (blocks + sms - 1) / sms;
    if (blocks > sms && (waves > 2 || blocks * 4 < waves * sms * 3)) return false;
  }
  return true;
}

// Programmatic dependent launch (a merged layer's kernel starts beside its predecessor in the
// stream and streams its first ring of weights at once) pays only with small clusters: with two
// blocks per cluster the one-token forward of 8192 -> 22016 gains 2.6 us per call in a replay of
// back-to-back layers, with clusters of 4 to 8 the same replay LOSES 1.5 to 8 us per call
// (22016 -> 8192: 29.7 us without, 37.4 us with; 8192 -> 8192: 14.3 / 17.4; 4096 -> 11008: 11.6 / 13.1).
#ifndef QALORA_GV_PDL_MAX_SPLITS
#define QALORA_GV_PDL_MAX_SPLITS 2
#endif
#ifndef QALORA_GV_GROUP_PDL_MAX_SPLITS
#define QALORA_GV_GROUP_PDL_MAX_SPLITS 2
#endif
// y = x * W~ + T * B for M <= 32 rows; Tb is T = s * pool(x) * A in bf16 [M][r] (null when r == 0).
int launch_gemv(const Shape& sh, int64_t M, const __nv_bfloat16* x, const uint32_t* codes, const float2* qparams,
                const __nv_bfloat16* Tb, const __nv_bfloat16* B, __nv_bfloat16* y, int* status, bool reset_status,
                cudaStream_t st) {
  CUtensorMap xm;
  if (!make_x_map(x, sh.K, M, &xm)) return QALORA_ERR_CUDA;
  GvParams p{};
  p.codes = codes; p.qparams = qparams; p.Tb = Tb; p.B = B; p.y = y; p.dbg = debug_words();
  p.M = (int)M; p.K = sh.K; p.N = sh.N; p.g = sh.g; p.r = sh.r;
  p.total_stages = sh.K / (GV_KBS * 32);
  p.status = status;
  p.reset_status = reset_status ? 1 : 0;
  p.stop_after_stages = g_expire_after_stages.exchange(0x7fffffff);     // one-shot: the next launch only
  p.wait_limit_ns = p.stop_after_stages != 0x7fffffff ? g_expire_limit_ns.load() : ptx::WAIT_LIMIT_NS;
  const int splits = gv_slices(sh, M);
  p.pdl_wait = (Tb == nullptr && splits <= QALORA_GV_PDL_MAX_SPLITS) ? 1 : 0;
  const int nts = M > 16 ? 4 : (M > 8 ? 2 : 1);
  const bool chain = sh.g >= 64;
#define QALORA_GV_N(BITS, NTS) (chain ? launch_gemv_t<BITS, NTS, true>(xm, p, splits, st) : launch_gemv_t<BITS, NTS, false>(xm, p, splits, st))
// (32 rows: the per-k-block fold for every group size; the chained form runs out of registers there)
#define QALORA_GV_1(BITS) (chain ? launch_gemv_t<BITS, 1, true, true>(xm, p, splits, st) : launch_gemv_t<BITS, 1, false, true>(xm, p, splits, st))
#define QALORA_GV(BITS) (nts == 4 ? launch_gemv_t<BITS, 4, false>(xm, p, splits, st) : (nts == 2 ? QALORA_GV_N(BITS, 2) : (M == 1 ? QALORA_GV_1(BITS) : QALORA_GV_N(BITS, 1))))
  if (sh.bits == 4) return QALORA_GV(4);
  if (sh.bits == 3) return QALORA_GV(3);
  return QALORA_GV(2);
#undef QALORA_GV
#undef QALORA_GV_1
#undef QALORA_GV_N
}


// Slices per column tile for a group of layers (one cluster size for the whole launch): the
// count that brings the grid closest to three blocks per SM and that every layer can be cut into.
static int gv_group_slices(const GemvGroupItem* items, int n) {
  long long tiles = 0;
  int min_stages = 1 << 30;
  for (int i = 0; i < n; ++i) {
    tiles += items[i].sh.N / GV_COLS;
    const int stages = items[i].sh.K / (GV_KBS * 32);
    min_stages = stages < min_stages ? stages : min_stages;
  }
  // (three blocks per SM here, two for a single layer: measured on the five projections of a 7B
  // block, 268 column tiles: 29.8 us with one slice per tile, 25.5 us with two; single layers were
  // slower with the higher target, e.g. 8192 -> 22016 32.2 against 30.6 us)
  const long long target = 3ll * device_sm_count();
  int splits = 1;
  long long best = 1ll << 60;
  for (int sp : {1, 2, 3, 4, 6, 8}) {
    if (sp > min_stages) break;
    const long long miss = tiles * sp > target ? tiles * sp - target : target - tiles * sp;
    if (miss < best) { best = miss; splits = sp; }
  }
  return splits;
}

bool gemv_group_supported(const GemvGroupItem* items, int n, int64_t M) {
  if (n < 1 || n > GV_GROUP_MAX || M < 1 || M > 16) return false;
  for (int i = 0; i < n; ++i) {
    const Shape& sh = items[i].sh;
    if (sh.r != 0 || sh.bits != items[0].sh.bits || (sh.g >= 64) != (items[0].sh.g >= 64) || !gemv_supported(sh, M)) return false;
  }
  return true;
}

// y_l = x_l * W~_l for the layers of a group (no adapters), M <= 16 rows each, in one launch.
int launch_gemv_group(const GemvGroupItem* items, int n, int64_t M, int* status, bool reset_status, cudaStream_t st) {
  GvGroup grp{};
  grp.n = n;
  const int splits = gv_group_slices(items, n);
  const bool pdl = splits <= QALORA_GV_GROUP_PDL_MAX_SPLITS;   // see launch_gemv
  const int words = words_per_unit(items[0].sh.bits);
  int blocks = 0;
  for (int i = 0; i < n; ++i) {
    const Shape& sh = items[i].sh;
    GvParams& p = grp.p[i];
    p.codes = items[i].codes; p.qparams = items[i].qparams; p.Tb = nullptr; p.B = nullptr; p.y = items[i].y; p.dbg = debug_words();
    p.M = (int)M; p.K = sh.K; p.N = sh.N; p.g = sh.g; p.r = 0;
    p.total_stages = sh.K / (GV_KBS * 32);
    p.status = status;
    p.reset_status = (reset_status && i == 0) ? 1 : 0;
    p.pdl_wait = pdl ? 1 : 0;
    p.stop_after_stages = 0x7fffffff;
    p.wait_limit_ns = ptx::WAIT_LIMIT_NS;
    if (!make_x_map(items[i].x, sh.K, M, &grp.x_map[i]) || !make_weight_maps(p, words, &grp.codes_map[i], &grp.qp_map[i]))
      return QALORA_ERR_CUDA;
    grp.first_block[i] = blocks;
    blocks += (sh.N / GV_COLS) * splits;
  }
  grp.first_block[n] = blocks;
  const bool two_sets = M > 8, chain = items[0].sh.g >= 64;
#define QALORA_GVG(BITS) (two_sets ? (chain ? launch_gemv_group_t<BITS, 2, true>(grp, splits, pdl, st) : launch_gemv_group_t<BITS, 2, false>(grp, splits, pdl, st)) \
                                   : (chain ? launch_gemv_group_t<BITS, 1, true>(grp, splits, pdl, st) : launch_gemv_group_t<BITS, 1, false>(grp, splits, pdl, st)))
  if (items[0].sh.bits == 4) return QALORA_GVG(4);
  if (items[0].sh.bits == 3) return QALORA_GVG(3);
  return QALORA_GVG(2);
#undef QALORA_GVG
}

}  // namespace qalora
