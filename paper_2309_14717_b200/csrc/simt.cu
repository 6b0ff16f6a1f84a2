// General-shape CUDA-core kernels of the QA-LoRA layer.  They accept every
// supported shape and serve (a) shapes the tensor-core kernels do not tile and
// (b) the small rank-r side products.  fp32 accumulation throughout.
#define QALORA_TU 6
#include "common.cuh"

namespace qalora {

// ------------------------------------------------------------ pool and T -----
// One token row per blockIdx.x: xp[q] = sum of the g channels of group q
// (Appendix B Eq. 3), then T[i] = s * sum_q xp[q] * A[q][i] for the 32 adapter
// columns of blockIdx.y (every block pools the row again: it is a few KiB).
// The kernel is short and bound by the latency of its loads, so they are issued in
// batches: the block's 32-column slice of A goes to shared memory first (its loads are
// independent of everything else), the row of x is read four 16-byte pieces per lane at a
// time before any of them is reduced.
constexpr int POOL_THREADS = 256;
constexpr size_t kPoolASliceMax = 40 * 1024;          // the slice of A is kept in shared memory up to this size

__global__ void __launch_bounds__(POOL_THREADS)
pool_T_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ A,
              float* __restrict__ xp_out, float* __restrict__ T, __nv_bfloat16* __restrict__ Tb,
              int K, int g, int G, int r, float s, int a_in_smem, int* dbg) {
  extern __shared__ __align__(16) uint8_t pool1_smem[];
  float* xp = reinterpret_cast<float*>(pool1_smem);                                        // [G]
  __nv_bfloat16* As = reinterpret_cast<__nv_bfloat16*>(pool1_smem + ((size_t)G * 4 + 15) / 16 * 16);   // [G][32] when a_in_smem
  // The few-token forward kernel that follows needs T only at its very end: let it start now
  // (it waits for this grid before it reads T).  Without such a dependent launch this does nothing.
  asm volatile("griddepcontrol.launch_dependents;");
  const size_t m = blockIdx.x;
  const int i0 = blockIdx.y * 32;
  if (a_in_smem) {
    // rows of 32 columns = 4 pieces of 8 (r is a multiple of 8: a piece lies inside the rank or beyond it)
    for (int idx = threadIdx.x; idx < G * 4; idx += POOL_THREADS) {
      const int q = idx / 4, c = idx % 4;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (i0 + c * 8 < r) v = __ldg(reinterpret_cast<const uint4*>(A + (size_t)q * r + i0 + c * 8));
      if (QALORA_CHECK(dbg, q * 32 + c * 8 + 7, G * 32)) *reinterpret_cast<uint4*>(As + (size_t)q * 32 + c * 8) = v;
    }
  }
  const __nv_bfloat16* xr = x + m * (size_t)K;
  // four lanes per group, 8 channels (16 bytes) per lane and step; g is a multiple of 32.
  // Groups q0 + 64 u + tid / 4, u = 0..3, are handled together: their loads first, then the sums.
  const int lane4 = threadIdx.x & 3;
  for (int q0 = 0; q0 < G; q0 += POOL_THREADS) {       // uniform trip count: the shuffles see whole warps
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k = lane4 * 8; k < g; k += 32) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int q = q0 + u * (POOL_THREADS / 4) + threadIdx.x / 4;
        v[u] = make_uint4(0u, 0u, 0u, 0u);
        if (q < G && QALORA_CHECK(dbg, (long long)q * g + k + 7, K)) v[u] = __ldg(reinterpret_cast<const uint4*>(xr + (size_t)q * g + k));
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v[u]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(h[i]);
          acc[u] += f.x + f.y;
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int q = q0 + u * (POOL_THREADS / 4) + threadIdx.x / 4;
      float a = acc[u];
      a += __shfl_xor_sync(0xffffffffu, a, 1);
      a += __shfl_xor_sync(0xffffffffu, a, 2);
      if (lane4 == 0 && q < G) {
        xp[q] = a;
        if (xp_out != nullptr && blockIdx.y == 0 && QALORA_CHECK(dbg, m * (size_t)G + q, (size_t)gridDim.x * G))
          xp_out[m * (size_t)G + q] = a;
      }
    }
  }
  __syncthreads();
  // this block's 32 adapter columns (blockIdx.y); 8 threads share a column, each taking
  // every eighth group
  __shared__ float part[8][33];
  const int il = threadIdx.x % 32, pr = threadIdx.x / 32;
  const int i = i0 + il;
  float acc = 0.0f;
  if (i < r) {
    if (a_in_smem) {
#pragma unroll 4
      for (int q = pr; q < G; q += 8) acc = fmaf(xp[q], bf16_to_float(As[(size_t)q * 32 + il]), acc);
    } else {
#pragma unroll 4
      for (int q = pr; q < G; q += 8) acc = fmaf(xp[q], bf16_to_float(A[(size_t)q * r + i]), acc);
    }
  }
  part[pr][il] = acc;
  __syncthreads();
  if (pr == 0 && i < r) {
    float t = 0.0f;
#pragma unroll
    for (int k = 0; k < 8; ++k) t += part[k][il];
    t *= s;
    if (QALORA_CHECK(dbg, m * (size_t)r + i, (size_t)gridDim.x * r)) {
      T[m * (size_t)r + i] = t;
      if (Tb != nullptr) Tb[m * (size_t)r + i] = __float2bfloat16_rn(t);
    }
  }
}

// Streaming version for many rows and a group size of 32, 64 or 128: sixteen rows per block.
// The group sums themselves run on the tensor cores: with an all-ones B operand,
// mma.sync.m16n8k16 adds up the 16 reduction slots of each A row whatever their order, so a
// lane feeds the 16 bytes it loaded (8 channels) straight in as A registers, two MMAs cover
// 16 groups x 32 channels, and the fp32 group sums come out in the accumulator: four instructions per KiB of x instead of converting and adding element by
// element, which had left the kernel bound by its instruction stream at half the copy rate.
// A warp takes one row of x at a time and lets 16 consecutive GROUPS of it be the MMA's 16
// rows, so that (g = 32) each of its load instructions reads 512 contiguous bytes.
// T = xp * A then runs on mma.sync.m16n8k16 with the block's 16 rows as the MMA rows
// and the groups as the reduction dimension; xp enters as a bf16 pair hi + lo
// (hi = xp rounded, lo = the remainder rounded: 16 significant bits together), so that
// T keeps fp32-like accuracy although the operands are bf16.
constexpr int POOL16_ROWS = 16;
#ifndef QALORA_POOL16_WARPS
#define QALORA_POOL16_WARPS 8
#endif
constexpr int POOL16_WARPS = QALORA_POOL16_WARPS;     // warps per block; several blocks per SM, so that one block's T phase hides behind the others' streaming

__device__ __forceinline__ void mma_bf16_16816(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Row stride (in 32-bit words) of the bf16 [16][Gp] arrays in shared memory: at least
// Gp / 2 and = 4 mod 32, so that the eight rows x four words of a fragment load fall into
// 32 different banks.
__host__ __device__ inline int pool16_stride_words(int G) {
  const int gp = (G + 15) / 16 * 16;
  int w = gp / 2;
  w += (4 - (w % 32) + 32) % 32;
  return w;
}

template <int LANES_PER_GROUP>   // g / 8: 4, 8 or 16
__global__ void __launch_bounds__(POOL16_WARPS * 32, 1024 / (POOL16_WARPS * 32))
pool_T_rows_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ A,
                   float* __restrict__ xp_out, float* __restrict__ T, __nv_bfloat16* __restrict__ Tb,
                   long long M, int K, int G, int r, float s, int smem_words, int* dbg) {
  extern __shared__ __align__(16) uint32_t pool_smem[];
  const int SW = pool16_stride_words(G);                 // row stride of the two bf16 arrays, in words
  __nv_bfloat16* xhi = reinterpret_cast<__nv_bfloat16*>(pool_smem);                 // [16][2 SW]
  __nv_bfloat16* xlo = reinterpret_cast<__nv_bfloat16*>(pool_smem + POOL16_ROWS * SW);
  float* part = reinterpret_cast<float*>(pool_smem + 2 * POOL16_ROWS * SW);        // [ksplit][16][r]
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int Gp = (G + 15) / 16 * 16;
  const long long row0 = (long long)blockIdx.x * POOL16_ROWS;
  // the padding groups G .. Gp - 1 count as zero (rows beyond M load zeros below)
  for (int i = threadIdx.x; i < POOL16_ROWS * (Gp - G); i += POOL16_WARPS * 32) {
    const int row = i / (Gp - G), q = G + i % (Gp - G);
    xhi[row * 2 * SW + q] = __float2bfloat16_rn(0.f);
    xlo[row * 2 * SW + q] = __float2bfloat16_rn(0.f);
  }
  {
    constexpr int CPG = LANES_PER_GROUP / 4;              // 32-channel chunks (64 bytes) per group
    constexpr int UNR = 4 / CPG;                          // sets of 16 groups whose loads are in flight together (8 x 16 bytes per lane)
    constexpr uint32_t ONES = 0x3f803f80u;                // bf16x2 (1, 1)
    // The 16 "rows" of the MMA are 16 consecutive GROUPS of one row of x: lanes 4v .. 4v + 3
    // hold the 64 bytes of a chunk of group v (a0, a2) and of group v + 8 (a1, a3), so with
    // g = 32 a load instruction of the warp reads 512 contiguous bytes.
    const int v = lane / 4, t4 = lane % 4;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    for (int rr = warp; rr < POOL16_ROWS; rr += POOL16_WARPS) {
      const long long m = row0 + rr;
      if (m >= M) {                                       // rows beyond M count as zero
        for (int q = lane; q < G; q += 32) {
          xhi[rr * 2 * SW + q] = __float2bfloat16_rn(0.f);
          xlo[rr * 2 * SW + q] = __float2bfloat16_rn(0.f);
        }
        continue;
      }
      const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)m * K) + t4;   // + 4 per chunk
      for (int qb = 0; qb < G; qb += 16 * UNR) {
        uint4 va[UNR][CPG], vb[UNR][CPG];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
          const int qa = qb + 16 * u + v, qh = qa + 8;    // this lane's two groups of the set
#pragma unroll
          for (int c = 0; c < CPG; ++c) {
            va[u][c] = qa < G && QALORA_CHECK(dbg, ((size_t)qa * CPG + c) * 32 + t4 * 8 + 7, K) ? __ldg(xr + ((size_t)qa * CPG + c) * 4) : zero;
            vb[u][c] = qh < G && QALORA_CHECK(dbg, ((size_t)qh * CPG + c) * 32 + t4 * 8 + 7, K) ? __ldg(xr + ((size_t)qh * CPG + c) * 4) : zero;
          }
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
          const int qa = qb + 16 * u + v, qh = qa + 8;
          float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int c = 0; c < CPG; ++c) {
            const uint32_t a0[4] = {va[u][c].x, vb[u][c].x, va[u][c].y, vb[u][c].y};
            const uint32_t a1[4] = {va[u][c].z, vb[u][c].z, va[u][c].w, vb[u][c].w};
            mma_bf16_16816(d, a0, ONES, ONES);
            mma_bf16_16816(d, a1, ONES, ONES);
          }
          // every column of the product holds the sums: d[0] for group qa, d[2] for group qh
          if (t4 == 0) {
            if (qa < G && QALORA_CHECK(dbg, rr * 2 * SW + qa, POOL16_ROWS * 2 * SW)) {
              const __nv_bfloat16 h = __float2bfloat16_rn(d[0]);
              xhi[rr * 2 * SW + qa] = h;
              xlo[rr * 2 * SW + qa] = __float2bfloat16_rn(d[0] - __bfloat162float(h));
              if (xp_out != nullptr && QALORA_CHECK(dbg, (size_t)m * G + qa, (size_t)M * G)) xp_out[(size_t)m * G + qa] = d[0];
            }
            if (qh < G && QALORA_CHECK(dbg, rr * 2 * SW + qh, POOL16_ROWS * 2 * SW)) {
              const __nv_bfloat16 h = __float2bfloat16_rn(d[2]);
              xhi[rr * 2 * SW + qh] = h;
              xlo[rr * 2 * SW + qh] = __float2bfloat16_rn(d[2] - __bfloat162float(h));
              if (xp_out != nullptr && QALORA_CHECK(dbg, (size_t)m * G + qh, (size_t)M * G)) xp_out[(size_t)m * G + qh] = d[2];
            }
          }
        }
      }
    }
  }
  __syncthreads();
  // T tile of 16 rows x 8 adapter columns per job; with few column tiles the groups are split
  // over several warps (ksplit parts), whose sums meet in shared memory
  const int ntiles = r / 8;                               // r is a multiple of 8
  int ksplit = 1;
  while (ksplit * 2 * ntiles <= POOL16_WARPS) ksplit *= 2;
  const int gq = lane / 4, t = lane % 4;
  const uint32_t* hi32 = pool_smem;
  const uint32_t* lo32 = pool_smem + POOL16_ROWS * SW;
  const uint16_t* A16 = reinterpret_cast<const uint16_t*>(A);
  for (int job = warp; job < ntiles * ksplit; job += POOL16_WARPS) {
    const int nt = job % ntiles, part_i = job / ntiles;
    const int n = nt * 8 + gq;                            // this lane's column of A
    float d[4] = {0.f, 0.f, 0.f, 0.f};
    for (int ks = part_i; ks < Gp / 16; ks += ksplit) {
      const int k0 = ks * 16 + 2 * t;                     // groups k0, k0 + 1 | k0 + 8, k0 + 9
      uint32_t bw[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int q = k0 + (e & 1) + 8 * (e >> 1);
        bw[e] = q < G ? A16[(size_t)q * r + n] : 0u;
      }
      const uint32_t b0 = bw[0] | (bw[1] << 16), b1 = bw[2] | (bw[3] << 16);
      const int w0 = ks * 8 + t;                          // word of (k0, k0 + 1) in a row
      const uint32_t ah[4] = {hi32[gq * SW + w0], hi32[(gq + 8) * SW + w0], hi32[gq * SW + w0 + 4], hi32[(gq + 8) * SW + w0 + 4]};
      const uint32_t al[4] = {lo32[gq * SW + w0], lo32[(gq + 8) * SW + w0], lo32[gq * SW + w0 + 4], lo32[(gq + 8) * SW + w0 + 4]};
      mma_bf16_16816(d, ah, b0, b1);
      mma_bf16_16816(d, al, b0, b1);
    }
    float* pp = part + (size_t)part_i * POOL16_ROWS * r;
    const int col = nt * 8 + 2 * t;
    // the last element this lane writes must lie inside the block's shared memory
    if (QALORA_CHECK(dbg, 2 * POOL16_ROWS * SW + (part_i * POOL16_ROWS + gq + 8) * r + col + 1, smem_words)) {
      pp[gq * r + col] = d[0];
      pp[gq * r + col + 1] = d[1];
      pp[(gq + 8) * r + col] = d[2];
      pp[(gq + 8) * r + col + 1] = d[3];
    }
  }
  __syncthreads();
  for (int o = threadIdx.x; o < POOL16_ROWS * r; o += POOL16_WARPS * 32) {
    const long long mm = (long long)blockIdx.x * POOL16_ROWS + o / r;
    float v = 0.f;
    for (int pi = 0; pi < ksplit; ++pi) v += part[(size_t)pi * POOL16_ROWS * r + o];
    v *= s;
    if (mm < M && QALORA_CHECK(dbg, (size_t)mm * r + o % r, (size_t)M * r)) {
      T[(size_t)mm * r + o % r] = v;
      if (Tb != nullptr) Tb[(size_t)mm * r + o % r] = __float2bfloat16_rn(v);
    }
  }
}

// shared memory of pool_T_rows_kernel (up to kPool16MaxSmem)
constexpr size_t kPool16MaxSmem = 96 * 1024;
static size_t pool16_smem_bytes(int G, int r) {
  const int ntiles = r / 8;
  int ksplit = 1;
  while (ksplit * 2 * ntiles <= POOL16_WARPS) ksplit *= 2;
  return (size_t)2 * POOL16_ROWS * pool16_stride_words(G) * 4 + (size_t)ksplit * POOL16_ROWS * r * 4;
}

int launch_pool_T(const Shape& sh, int64_t M, const __nv_bfloat16* x, const __nv_bfloat16* A,
                  float* xp, float* T, __nv_bfloat16* Tb, cudaStream_t st) {
  if (M == 0) return QALORA_OK;
  const size_t smem = sh.r >= 8 ? pool16_smem_bytes(sh.G, sh.r) : 0;
  const bool rows_path = M >= 512 && (sh.g == 32 || sh.g == 64 || sh.g == 128) && sh.K % 256 == 0 &&
                         sh.r >= 8 && smem <= kPool16MaxSmem;
  if (rows_path) {
    static PerDeviceOnce smem_limit;                     // once per device: allow more than the default 48 KiB
    const int attr_st = smem_limit.run([] {
      cudaError_t e = cudaFuncSetAttribute(pool_T_rows_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPool16MaxSmem);
      if (e == cudaSuccess) e = cudaFuncSetAttribute(pool_T_rows_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPool16MaxSmem);
      if (e == cudaSuccess) e = cudaFuncSetAttribute(pool_T_rows_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPool16MaxSmem);
      return e;
    });
    if (attr_st != QALORA_OK) return attr_st;
    const unsigned grid = (unsigned)((M + POOL16_ROWS - 1) / POOL16_ROWS);
    if (sh.g == 32) pool_T_rows_kernel<4><<<grid, POOL16_WARPS * 32, smem, st>>>(x, A, xp, T, Tb, M, sh.K, sh.G, sh.r, sh.s, (int)(smem / 4), debug_words());
    else if (sh.g == 64) pool_T_rows_kernel<8><<<grid, POOL16_WARPS * 32, smem, st>>>(x, A, xp, T, Tb, M, sh.K, sh.G, sh.r, sh.s, (int)(smem / 4), debug_words());
    else pool_T_rows_kernel<16><<<grid, POOL16_WARPS * 32, smem, st>>>(x, A, xp, T, Tb, M, sh.K, sh.G, sh.r, sh.s, (int)(smem / 4), debug_words());
  } else {
    dim3 grid((unsigned)M, (unsigned)((sh.r + 31) / 32 > 0 ? (sh.r + 31) / 32 : 1));
    const size_t xp_bytes = ((size_t)sh.G * sizeof(float) + 15) / 16 * 16, a_bytes = (size_t)sh.G * 32 * sizeof(__nv_bfloat16);
    const int a_in_smem = (sh.r > 0 && a_bytes <= kPoolASliceMax) ? 1 : 0;
    pool_T_kernel<<<grid, POOL_THREADS, xp_bytes + (a_in_smem ? a_bytes : 0), st>>>(x, A, xp, T, Tb, sh.K, sh.g, sh.G, sh.r, sh.s,
                                                                                    a_in_smem, debug_words());
  }
  count_launch();
  return cuda_status(cudaGetLastError());
}

// ------------------------------------------------------------- dT ------------
// dT[m][i] = s * sum_n dy[m][n] * B[i][n]; one block per row, one warp per i.
constexpr int DT_THREADS = 256;

__global__ void __launch_bounds__(DT_THREADS)
dT_kernel(const __nv_bfloat16* __restrict__ dy, const __nv_bfloat16* __restrict__ B,
          float* __restrict__ dT, __nv_bfloat16* __restrict__ dTb, int N, int r, float s, int* dbg) {
  const size_t m = blockIdx.x;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const __nv_bfloat16* dyr = dy + m * (size_t)N;
  for (int i = warp; i < r; i += DT_THREADS / 32) {
    const __nv_bfloat16* br = B + (size_t)i * N;
    float acc = 0.0f;
    for (int n = lane * 8; n < N; n += 256) {            // N is a multiple of 8
      const uint4 a = *reinterpret_cast<const uint4*>(dyr + n);
      const uint4 b = *reinterpret_cast<const uint4*>(br + n);
      const __nv_bfloat162* ha = reinterpret_cast<const __nv_bfloat162*>(&a);
      const __nv_bfloat162* hb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 fa = __bfloat1622float2(ha[j]), fb = __bfloat1622float2(hb[j]);
        acc = fmaf(fa.x, fb.x, acc);
        acc = fmaf(fa.y, fb.y, acc);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
      acc *= s;
      if (QALORA_CHECK(dbg, m * (size_t)r + i, (size_t)gridDim.x * r)) {
        dT[m * (size_t)r + i] = acc;
        if (dTb != nullptr) dTb[m * (size_t)r + i] = __float2bfloat16_rn(acc);
      }
    }
  }
}

int launch_dT(const Shape& sh, int64_t M, const __nv_bfloat16* dy, const __nv_bfloat16* B,
              float* dT, __nv_bfloat16* dTb, cudaStream_t st) {
  if (M == 0) return QALORA_OK;
  dT_kernel<<<(unsigned)M, DT_THREADS, 0, st>>>(dy, B, dT, dTb, sh.N, sh.r, sh.s, debug_words());
  count_launch();
  return cuda_status(cudaGetLastError());
}

// ------------------------------------------------------ tiled main products --
// 64 x 64 output tile, 256 threads, 4 x 4 outputs per thread, 32-deep steps.
constexpr int TM = 64, TN = 64, TK = 32, SIMT_THREADS = 256;

// y[m][n] = sum_k x[m][k] * W~[k][n] + sum_i T[m][i] * B[i][n]
template <int BITS>
__global__ void __launch_bounds__(SIMT_THREADS)
simt_forward_kernel(const __nv_bfloat16* __restrict__ x, const uint32_t* __restrict__ codes,
                    const float2* __restrict__ qparams, const float* __restrict__ T,
                    const __nv_bfloat16* __restrict__ B, __nv_bfloat16* __restrict__ y,
                    long long M, int K, int N, int g, int r, int* dbg) {
  constexpr int WORDS = BITS == 4 ? 4 : (BITS == 3 ? 3 : 2);
  __shared__ __align__(16) float xs[TK][TM + 4];
  __shared__ __align__(16) float ws[TK][TN + 4];
  const int tid = threadIdx.x;
  const long long m0 = (long long)blockIdx.y * TM;
  const int n0 = blockIdx.x * TN;
  const int ty = tid / 16, tx = tid % 16;
  float acc[4][4] = {};

  const int lrow = tid / 4, lseg = (tid % 4) * 8;       // x loader: row, 8-channel segment
  const int un = tid % 64, uj = (tid / 64) * 8;         // W loader: column, first position
  for (int k0 = 0; k0 < K; k0 += TK) {
    {
      float v[8] = {};
      if (m0 + lrow < M && QALORA_CHECK(dbg, (size_t)(m0 + lrow) * K + k0 + lseg + 7, (size_t)M * K)) {
        const uint4 raw = *reinterpret_cast<const uint4*>(x + (size_t)(m0 + lrow) * K + k0 + lseg);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(h[i]);
          v[2 * i] = f.x; v[2 * i + 1] = f.y;
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) xs[lseg + i][lrow] = v[i];
    }
    {
      const int n = n0 + un;
      if (n < N && QALORA_CHECK(dbg, ((size_t)(k0 / 32) * N + n) * WORDS + WORDS - 1, (size_t)(K / 32) * N * WORDS) &&
          QALORA_CHECK(dbg, (size_t)(k0 / g) * N + n, (size_t)(K / g) * N)) {
        const uint32_t* u = codes + ((size_t)(k0 / 32) * N + n) * WORDS;
        uint32_t w[WORDS];
#pragma unroll
        for (int i = 0; i < WORDS; ++i) w[i] = __ldg(u + i);
        const float2 ab = __ldg(qparams + (size_t)(k0 / g) * N + n);
#pragma unroll
        for (int i = 0; i < 8; ++i) ws[uj + i][un] = fmaf(ab.x, (float)unit_code<BITS>(w, uj + i), ab.y);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) ws[uj + i][un] = 0.0f;
      }
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < TK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&xs[kk][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&ws[kk][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  // adapter term and store
  const int nb = n0 + tx * 4;
  if (nb >= N) return;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long m = m0 + ty * 4 + i;
    if (m >= M) continue;
    for (int t = 0; t < r; ++t) {
      const float tv = __ldg(T + (size_t)m * r + t);
      const uint2 raw = *reinterpret_cast<const uint2*>(B + (size_t)t * N + nb);
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
      const float2 b0 = __bfloat1622float2(h[0]), b1 = __bfloat1622float2(h[1]);
      acc[i][0] = fmaf(tv, b0.x, acc[i][0]); acc[i][1] = fmaf(tv, b0.y, acc[i][1]);
      acc[i][2] = fmaf(tv, b1.x, acc[i][2]); acc[i][3] = fmaf(tv, b1.y, acc[i][3]);
    }
    __nv_bfloat162 o[2] = {__floats2bfloat162_rn(acc[i][0], acc[i][1]), __floats2bfloat162_rn(acc[i][2], acc[i][3])};
    if (QALORA_CHECK(dbg, (size_t)m * N + nb + 3, (size_t)M * N)) *reinterpret_cast<uint2*>(y + (size_t)m * N + nb) = *reinterpret_cast<uint2*>(o);
  }
}

int launch_simt_forward(const Shape& sh, int64_t M, const __nv_bfloat16* x, const uint32_t* codes,
                        const float2* qparams, const float* T, const __nv_bfloat16* B,
                        __nv_bfloat16* y, cudaStream_t st) {
  if (M == 0) return QALORA_OK;
  const long long mt = (M + TM - 1) / TM;
  if (mt > 65535) return QALORA_ERR_UNSUPPORTED_SHAPE;
  dim3 grid((sh.N + TN - 1) / TN, (unsigned)mt), block(SIMT_THREADS);
#define QALORA_FWD(BITS) simt_forward_kernel<BITS><<<grid, block, 0, st>>>(x, codes, qparams, T, B, y, M, sh.K, sh.N, sh.g, sh.r, debug_words())
  {
    MainKernelProbe probe("simt_forward_kernel", st);
    if (sh.bits == 4) QALORA_FWD(4); else if (sh.bits == 3) QALORA_FWD(3); else QALORA_FWD(2);
  }
  count_launch();
#undef QALORA_FWD
  return cuda_status(cudaGetLastError());
}

// dx[m][k] = sum_n dy[m][n] * W~[k][n] + sum_i dT[m][i] * A[k/g][i]
template <int BITS>
__global__ void __launch_bounds__(SIMT_THREADS)
simt_dx_kernel(const __nv_bfloat16* __restrict__ dy, const uint32_t* __restrict__ codes,
               const float2* __restrict__ qparams, const float* __restrict__ dT,
               const __nv_bfloat16* __restrict__ A, __nv_bfloat16* __restrict__ dx,
               long long M, int K, int N, int g, int r, int* dbg) {
  constexpr int WORDS = BITS == 4 ? 4 : (BITS == 3 ? 3 : 2);
  __shared__ __align__(16) float ds[TK][TM + 4];        // [n][m]
  __shared__ __align__(16) float ws[TK][TN + 4];        // [n][k]
  const int tid = threadIdx.x;
  const long long m0 = (long long)blockIdx.y * TM;
  const int k0 = blockIdx.x * TN;                       // 64 output channels = 2 k-blocks
  const int ty = tid / 16, tx = tid % 16;
  float acc[4][4] = {};

  const int lrow = tid / 4, lseg = (tid % 4) * 8;
  const int un = tid % 32, ukb = (tid / 32) % 2, uj = (tid / 64) * 8;
  for (int n0 = 0; n0 < N; n0 += TK) {
    {
      float v[8] = {};
      if (m0 + lrow < M && n0 + lseg < N && QALORA_CHECK(dbg, (size_t)(m0 + lrow) * N + n0 + lseg + 7, (size_t)M * N)) {
        const uint4 raw = *reinterpret_cast<const uint4*>(dy + (size_t)(m0 + lrow) * N + n0 + lseg);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(h[i]);
          v[2 * i] = f.x; v[2 * i + 1] = f.y;
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) ds[lseg + i][lrow] = v[i];
    }
    {
      const int n = n0 + un, k = k0 + ukb * 32;
      if (n < N && k < K && QALORA_CHECK(dbg, ((size_t)(k / 32) * N + n) * WORDS + WORDS - 1, (size_t)(K / 32) * N * WORDS) &&
          QALORA_CHECK(dbg, (size_t)(k / g) * N + n, (size_t)(K / g) * N)) {
        const uint32_t* u = codes + ((size_t)(k / 32) * N + n) * WORDS;
        uint32_t w[WORDS];
#pragma unroll
        for (int i = 0; i < WORDS; ++i) w[i] = __ldg(u + i);
        const float2 ab = __ldg(qparams + (size_t)(k / g) * N + n);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          ws[un][ukb * 32 + uj + i] = fmaf(ab.x, (float)unit_code<BITS>(w, uj + i), ab.y);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) ws[un][ukb * 32 + uj + i] = 0.0f;
      }
    }
    __syncthreads();
#pragma unroll 8
    for (int nn = 0; nn < TK; ++nn) {
      const float4 a = *reinterpret_cast<const float4*>(&ds[nn][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&ws[nn][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  const int kc = k0 + tx * 4;
  if (kc >= K) return;
  const int q = kc / g;                                 // 4 consecutive channels share a group
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long m = m0 + ty * 4 + i;
    if (m >= M) continue;
    float lora = 0.0f;
    for (int t = 0; t < r; ++t)
      lora = fmaf(__ldg(dT + (size_t)m * r + t), bf16_to_float(A[(size_t)q * r + t]), lora);
    __nv_bfloat162 o[2] = {__floats2bfloat162_rn(acc[i][0] + lora, acc[i][1] + lora),
                           __floats2bfloat162_rn(acc[i][2] + lora, acc[i][3] + lora)};
    if (QALORA_CHECK(dbg, (size_t)m * K + kc + 3, (size_t)M * K)) *reinterpret_cast<uint2*>(dx + (size_t)m * K + kc) = *reinterpret_cast<uint2*>(o);
  }
}

int launch_simt_dx(const Shape& sh, int64_t M, const __nv_bfloat16* dy, const uint32_t* codes,
                   const float2* qparams, const float* dT, const __nv_bfloat16* A,
                   __nv_bfloat16* dx, cudaStream_t st) {
  if (M == 0) return QALORA_OK;
  const long long mt = (M + TM - 1) / TM;
  if (mt > 65535) return QALORA_ERR_UNSUPPORTED_SHAPE;
  dim3 grid((sh.K + TN - 1) / TN, (unsigned)mt), block(SIMT_THREADS);
#define QALORA_DX(BITS) simt_dx_kernel<BITS><<<grid, block, 0, st>>>(dy, codes, qparams, dT, A, dx, M, sh.K, sh.N, sh.g, sh.r, debug_words())
  {
    MainKernelProbe probe("simt_dx_kernel", st);
    if (sh.bits == 4) QALORA_DX(4); else if (sh.bits == 3) QALORA_DX(3); else QALORA_DX(2);
  }
  count_launch();
#undef QALORA_DX
  return cuda_status(cudaGetLastError());
}

// ----------------------------------------------- X^T * Y reductions over M ---
// out[p][q] = sum_m X[m][p] * Y[m][q].  The token range is split over
// blockIdx.z; each split writes its own partial tile and a second kernel adds
// the partials in a fixed order, so the result does not depend on scheduling.
template <typename TY> __device__ __forceinline__ float load_as_float(const TY* p);
template <> __device__ __forceinline__ float load_as_float<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float load_as_float<__nv_bfloat16>(const __nv_bfloat16* p) { return bf16_to_float(*p); }

template <typename TY>
__global__ void __launch_bounds__(SIMT_THREADS)
atb_partial_kernel(const float* __restrict__ X, const TY* __restrict__ Y, float* __restrict__ partial,
                   long long M, int P, int Q, long long rows_per_split, int* dbg) {
  __shared__ __align__(16) float xs[TK][TM + 4];
  __shared__ __align__(16) float ys[TK][TN + 4];
  const int tid = threadIdx.x;
  const int p0 = blockIdx.y * TM, q0 = blockIdx.x * TN;
  const int ty = tid / 16, tx = tid % 16;
  const long long mbeg = (long long)blockIdx.z * rows_per_split;
  const long long mend = min(M, mbeg + rows_per_split);
  float acc[4][4] = {};
  // The block's share of rows is short (a few 32-row steps), so the kernel is bound by the
  // latency of its loads: the next step's elements are fetched into registers while the
  // current step is multiplied out of shared memory.
  constexpr int PER = TK * TM / SIMT_THREADS;             // elements of each tile per thread
  float xr[PER], yr[PER];
  auto fetch = [&](long long m0) {
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int e = tid + i * SIMT_THREADS;
      const int mm = e / TM, c = e % TM;
      const long long m = m0 + mm;
      xr[i] = (m < mend && p0 + c < P) ? __ldg(X + (size_t)m * P + p0 + c) : 0.0f;
      yr[i] = (m < mend && q0 + c < Q) ? load_as_float<TY>(Y + (size_t)m * Q + q0 + c) : 0.0f;
    }
  };
  if (mbeg < mend) fetch(mbeg);
  for (long long m0 = mbeg; m0 < mend; m0 += TK) {
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int e = tid + i * SIMT_THREADS;
      xs[e / TM][e % TM] = xr[i];
      ys[e / TM][e % TM] = yr[i];
    }
    __syncthreads();
    if (m0 + TK < mend) fetch(m0 + TK);
#pragma unroll 8
    for (int mm = 0; mm < TK; ++mm) {
      const float4 a = *reinterpret_cast<const float4*>(&xs[mm][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&ys[mm][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* dst = partial + (size_t)blockIdx.z * P * Q;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int p = p0 + ty * 4 + i, q = q0 + tx * 4 + j;
      if (p < P && q < Q && QALORA_CHECK(dbg, ((size_t)blockIdx.z * P + p) * Q + q, (size_t)gridDim.z * P * Q)) dst[(size_t)p * Q + q] = acc[i][j];
    }
}

__global__ void sum_partials_kernel(const float* __restrict__ partial, float* __restrict__ out,
                                    size_t count, int splits) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  float acc = 0.0f;
  for (int z = 0; z < splits; ++z) acc += partial[(size_t)z * count + i];
  out[i] = acc;
}

static long long atb_splits(int64_t M, int P, int Q) {
  const int tiles = ((P + TM - 1) / TM) * ((Q + TN - 1) / TN);
  long long splits = (2 * 148 + tiles - 1) / tiles;        // about two blocks per SM
  const long long max_by_rows = (M + 4 * TK - 1) / (4 * TK);
  if (splits > max_by_rows) splits = max_by_rows;
  return splits < 1 ? 1 : splits;
}

size_t atb_partial_bytes(int64_t M, int P, int Q) {
  const size_t count = (size_t)P * Q;
  if (count == 0 || M <= 0) return 0;
  return (size_t)atb_splits(M, P, Q) * count * sizeof(float);
}

template <typename TY>
static int launch_atb(int64_t M, int P, int Q, const float* X, const TY* Y, float* out,
                      float* partial, size_t partial_bytes, cudaStream_t st) {
  const size_t count = (size_t)P * Q;
  if (count == 0) return QALORA_OK;
  if (M == 0) return cuda_status(cudaMemsetAsync(out, 0, count * sizeof(float), st));
  long long splits = atb_splits(M, P, Q);
  const long long max_by_space = (long long)(partial_bytes / (count * sizeof(float)));
  if (splits > max_by_space) splits = max_by_space;
  if (splits < 1) return QALORA_ERR_WORKSPACE_TOO_SMALL;
  long long rows = (M + splits - 1) / splits;
  rows = (rows + TK - 1) / TK * TK;
  splits = (M + rows - 1) / rows;
  dim3 grid((Q + TN - 1) / TN, (P + TM - 1) / TM, (unsigned)splits);
  atb_partial_kernel<TY><<<grid, SIMT_THREADS, 0, st>>>(X, Y, partial, M, P, Q, rows, debug_words());
  sum_partials_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(partial, out, count, (int)splits);
  count_launch(2);
  return cuda_status(cudaGetLastError());
}

int launch_sum_partials(const float* partial, float* out, size_t count, int splits, cudaStream_t st) {
  if (count == 0) return QALORA_OK;
  sum_partials_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(partial, out, count, splits);
  count_launch();
  return cuda_status(cudaGetLastError());
}

int launch_atb_bf16(int64_t M, int P, int Q, const float* X, const __nv_bfloat16* Y, float* out,
                    float* partial, size_t partial_bytes, cudaStream_t st) {
  return launch_atb<__nv_bfloat16>(M, P, Q, X, Y, out, partial, partial_bytes, st);
}
int launch_atb_f32(int64_t M, int P, int Q, const float* X, const float* Y, float* out,
                   float* partial, size_t partial_bytes, cudaStream_t st) {
  return launch_atb<float>(M, P, Q, X, Y, out, partial, partial_bytes, st);
}

}  // namespace qalora
