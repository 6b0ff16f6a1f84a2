// Dequantization of one pack unit (32 input channels of one output column) to 16 bf16x2
// registers, shared by the tensor-core kernels.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "ptx.cuh"

namespace qalora {

// ---- dequantization of one pack unit to 16 bf16x2 registers ------------------
// The two codes of a pair sit at the same bit offset of the two half-words, so one shift
// and one LOP3 turn them into the bf16 pair (128 + c0, 128 + c1): the code is OR-ed into
// the mantissa of bf16 128.0, no int-to-float conversion.  Widening each half to fp32 is
// one more logic op, then W~ = alpha * (128 + c) + (beta - 128 alpha) is ONE fp32 FMA per
// element, and the pair is rounded once to bf16x2.  alpha and beta stay in fp32, so the
// only rounding that matters is that of the final weight (rounding alpha or beta
// themselves would put a common error on all channels of a group, which the pooled input
// amplifies).
// The logic/shift pipe is the busiest one in these kernels.  A LOP3 takes at most one
// immediate, so the masks live in registers (DqConsts, made opaque to the compiler):
// "(a & mask) | magic" then is one instruction instead of two.
struct DqConsts {
  uint32_t mask, magic, himask, third, nibbles, magic32;
};
template <int BITS>
__device__ __forceinline__ DqConsts dq_consts() {
  DqConsts c;
  asm volatile("mov.b32 %0, %1;" : "=r"(c.mask) : "n"(BITS == 4 ? 0x000f000f : 0x00030003));
  asm volatile("mov.b32 %0, 0x43004300;" : "=r"(c.magic));
  asm volatile("mov.b32 %0, 0xffff0000;" : "=r"(c.himask));
  asm volatile("mov.b32 %0, 0x00040004;" : "=r"(c.third));
  asm volatile("mov.b32 %0, 0x0f0f0f0f;" : "=r"(c.nibbles));
  asm volatile("mov.b32 %0, 0x43000000;" : "=r"(c.magic32));
  return c;
}
__device__ __forceinline__ uint32_t lop_and_or(uint32_t a, uint32_t b, uint32_t c) {   // (a & b) | c
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t lop_and(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("and.b32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
template <int SHIFT>   // positive: shift left
__device__ __forceinline__ uint32_t shift_to(uint32_t w) {
  if constexpr (SHIFT >= 0) return w << SHIFT; else return w >> (-SHIFT);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&t);
}

template <int WORDS>
__device__ __forceinline__ void load_unit(const uint32_t* cw, uint32_t* w) {
  if constexpr (WORDS == 4) {
    const uint4 t = *reinterpret_cast<const uint4*>(cw);
    w[0] = t.x; w[1] = t.y; w[2] = t.z; w[3] = t.w;
  } else if constexpr (WORDS == 2) {
    const uint2 t = *reinterpret_cast<const uint2*>(cw);
    w[0] = t.x; w[1] = t.y;
  } else {
#pragma unroll
    for (int q = 0; q < WORDS; ++q) w[q] = cw[q];
  }
}

#ifndef QALORA_DQ_FFMA2
#define QALORA_DQ_FFMA2 1
#endif
// alpha * (v0, v1) + b for a pair of codes: one packed two-lane FMA (fma.rn.f32x2; each lane an
// ordinary IEEE fused multiply-add), then one conversion of the pair to bf16x2
__device__ __forceinline__ uint32_t dq_fma_pair(float v0, float v1, float a, float b) {
#if QALORA_DQ_FFMA2
  const float2 r = ptx::ffma2(make_float2(a, a), make_float2(v0, v1), make_float2(b, b));
  return pack_bf16x2(r.x, r.y);
#else
  return pack_bf16x2(fmaf(a, v0, b), fmaf(a, v1, b));
#endif
}

// pair P of word I: positions (2P, 2P+1) of that word's codes
template <int BITS, int I, int P>
__device__ __forceinline__ uint32_t dq_pair(const uint32_t* w, float a, float b, const DqConsts& k) {
  constexpr int W = BITS == 4 ? 4 : 2;             // width of the (low) code bits
  uint32_t pr = lop_and_or(w[I] >> (W * P), k.mask, k.magic);
  if constexpr (BITS == 3) {
    // third bits of the pair: bits PH and 16 + PH of word 2, PH = 8 I + P; they go to bit 2 of each half
    constexpr int PH = 8 * I + P;
    pr = lop_and_or(shift_to<2 - PH>(w[2]), k.third, pr);
  }
  const float v0 = __uint_as_float(pr << 16), v1 = __uint_as_float(lop_and(pr, k.himask));   // 128 + c, exactly
  return dq_fma_pair(v0, v1, a, b);
}

template <int BITS, int I, int P>
__device__ __forceinline__ void dq_all(const uint32_t* w, float a, float b, const DqConsts& k, uint32_t* out) {
  constexpr int PAIRS = BITS == 4 ? 4 : 8;          // pairs per word
  constexpr int NWORDS = BITS == 4 ? 4 : 2;         // words that carry the (low) code bits
  out[I * PAIRS + P] = dq_pair<BITS, I, P>(w, a, b, k);
  if constexpr (P + 1 < PAIRS) dq_all<BITS, I, P + 1>(w, a, b, k, out);
  else if constexpr (I + 1 < NWORDS) dq_all<BITS, I + 1, 0>(w, a, b, k, out);
}

// 4-bit codes, a cheaper route to the same values.  One AND gives the word's four even nibbles
// as the low nibbles of its four bytes, one shift and one AND the four odd ones; a byte
// permute then drops such a byte straight into mantissa bits 16-19 of the fp32 number 128.0
// (0x43000000), i.e. it makes fp32 (128 + c) in ONE instruction per code: 11 logic-pipe
// instructions per word of eight codes instead of 15.  Byte B of the even (odd) word holds the
// code of position e with (e & 1, e >> 1) = (B >> 1, 2 (B & 1)) (+ 1 for the odd word).
template <int B>
__device__ __forceinline__ float dq4_byte(uint32_t nib, uint32_t magic32) {
  uint32_t d;                                          // bytes (3, 2, 1, 0) = (0x43, byte B of nib, 0, 0)
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(nib), "r"(magic32), "n"(0x7044 | (B << 8)));
  return __uint_as_float(d);
}
__device__ __forceinline__ void dq4_word(uint32_t w, float a, float b, const DqConsts& k, uint32_t* out4) {
  const uint32_t ev = lop_and(w, k.nibbles), od = lop_and(w >> 4, k.nibbles);
  // pairs (positions 2P, 2P + 1): P = 0 and 2 from the even nibbles, P = 1 and 3 from the odd ones
  out4[0] = dq_fma_pair(dq4_byte<0>(ev, k.magic32), dq4_byte<2>(ev, k.magic32), a, b);
  out4[1] = dq_fma_pair(dq4_byte<0>(od, k.magic32), dq4_byte<2>(od, k.magic32), a, b);
  out4[2] = dq_fma_pair(dq4_byte<1>(ev, k.magic32), dq4_byte<3>(ev, k.magic32), a, b);
  out4[3] = dq_fma_pair(dq4_byte<1>(od, k.magic32), dq4_byte<3>(od, k.magic32), a, b);
}

// out[q] = bf16x2 of positions (2q, 2q+1) of the unit, q = 0..15
template <int BITS>
__device__ __forceinline__ void dequant_unit(const uint32_t* w, float2 ab, const DqConsts& k, uint32_t* out) {
  const float b = fmaf(-128.f, ab.x, ab.y);
  if constexpr (BITS == 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i) dq4_word(w[i], ab.x, b, k, out + 4 * i);
    return;
  }
  dq_all<BITS, 0, 0>(w, ab.x, b, k, out);
}

}  // namespace qalora
