// Dequantization of one pack unit (32 input channels of one output column) to 16 bf16x2
// registers, shared by the tensor-core kernels.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "ptx.cuh"

namespace qalora {

// ---- dequantization of one pack unit to 16 bf16x2 registers ------------------
// A code is brought into a byte of its own (masks and shifts on whole words, four codes at a
// time), a byte permute drops that byte into mantissa bits 16.. of the fp32 number 128.0
// (0x43000000 | c << 16 = 128 + c exactly: no int-to-float conversion), then
// W~ = alpha * (128 + c) + (beta - 128 alpha) is one fp32 FMA per element, two elements per
// packed instruction, and the pair is rounded once to bf16x2.  alpha and beta stay in fp32, so
// the only rounding that matters is that of the final weight (rounding alpha or beta
// themselves would put a common error on all channels of a group, which the pooled input
// amplifies).
// The logic/shift pipe is the busiest one in these kernels.  A LOP3 takes at most one
// immediate, so the masks live in registers (DqConsts, made opaque to the compiler):
// "(a & mask) | x" then is one instruction instead of two.
struct DqConsts {
  uint32_t nibbles, magic32, twobits, third_a, third_b;
};
template <int BITS>
__device__ __forceinline__ DqConsts dq_consts() {
  DqConsts c;
  asm volatile("mov.b32 %0, 0x0f0f0f0f;" : "=r"(c.nibbles));
  asm volatile("mov.b32 %0, 0x43000000;" : "=r"(c.magic32));
  asm volatile("mov.b32 %0, 0x03030303;" : "=r"(c.twobits));
  asm volatile("mov.b32 %0, 0x00040004;" : "=r"(c.third_a));
  asm volatile("mov.b32 %0, 0x04000400;" : "=r"(c.third_b));
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

// 2- and 3-bit codes by the same route.  A word of the low code bits holds 16 codes, two bits
// each: the even positions e = 2k in its low half-word at bit 2k, the odd ones in the high
// half-word at the same offset.  Shifted right by 2 ss (ss = 0..3) and masked with 0x03030303 it
// leaves one code in each byte: positions 2 ss | 8 + 2 ss | 2 ss + 1 | 9 + 2 ss in bytes 0..3, i.e.
// the pairs k = ss (bytes 0, 2) and k = 4 + ss (bytes 1, 3).  The third bit of position j of the
// unit sits in word 2 at bit 16 (j & 1) + (j >> 1); for those four positions of word I that is
// b0, b0 + 4, b0 + 16, b0 + 20 with b0 = 8 I + ss, so two shifts bring them to bit 2 of bytes
// 0 and 2 and of bytes 1 and 3.  Then one byte permute per code, one packed FMA and one
// conversion per pair: 2.4 (3.4) instructions per 2-bit (3-bit) code instead of 3 (4).
template <int BITS, int I, int SS>
__device__ __forceinline__ void dq23_quad(const uint32_t* w, float a, float b, const DqConsts& k, uint32_t* out) {
  uint32_t nib = lop_and(SS == 0 ? w[I] : (w[I] >> (2 * SS)), k.twobits);
  if constexpr (BITS == 3) {
    constexpr int B0 = 8 * I + SS;
    nib = lop_and_or(shift_to<2 - B0>(w[2]), k.third_a, nib);
    nib = lop_and_or(shift_to<6 - B0>(w[2]), k.third_b, nib);
  }
  out[8 * I + SS] = dq_fma_pair(dq4_byte<0>(nib, k.magic32), dq4_byte<2>(nib, k.magic32), a, b);
  out[8 * I + 4 + SS] = dq_fma_pair(dq4_byte<1>(nib, k.magic32), dq4_byte<3>(nib, k.magic32), a, b);
}

// out[q] = bf16x2 of positions (2q, 2q+1) of the unit, q = 0..15
template <int BITS>
__device__ __forceinline__ void dequant_unit(const uint32_t* w, float2 ab, const DqConsts& k, uint32_t* out) {
  const float b = fmaf(-128.f, ab.x, ab.y);
  if constexpr (BITS == 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i) dq4_word(w[i], ab.x, b, k, out + 4 * i);
  } else {
    dq23_quad<BITS, 0, 0>(w, ab.x, b, k, out); dq23_quad<BITS, 0, 1>(w, ab.x, b, k, out);
    dq23_quad<BITS, 0, 2>(w, ab.x, b, k, out); dq23_quad<BITS, 0, 3>(w, ab.x, b, k, out);
    dq23_quad<BITS, 1, 0>(w, ab.x, b, k, out); dq23_quad<BITS, 1, 1>(w, ab.x, b, k, out);
    dq23_quad<BITS, 1, 2>(w, ab.x, b, k, out); dq23_quad<BITS, 1, 3>(w, ab.x, b, k, out);
  }
}

}  // namespace qalora
