// Exact RoPE arithmetic in fp32 (Sec. 3.1 "Parallel attention": positions restart in every chunk; pairs
// (t, t + d/2), angle p * theta^(-2t/d)).
//
// The rotated value must equal the fp64 rotation rounded ONCE to bf16, bit for bit, but fp64 arithmetic (a
// small fraction of the fp32 rate) is almost never executed.  Three levels:
//   1. fp32 with the fp32 heads of the table entries.  Its error is below 2^-22 (|x1| + |x2|); when
//      y - tol and y + tol round to the same bf16 value, that value is the correctly rounded one.
//   2. otherwise (about one output in a few thousand) the value is re-evaluated as an unevaluated sum of two
//      fp32 numbers (products with their exact FMA residuals, the fp32 tails of the table entries), good to
//      2^-43 (|x1| + |x2|), and rounded from there;
//   3. if that is still too close to a rounding boundary (practically never), fp64 on the fp64 table.
#pragma once
#include "pc_sm100.cuh"

namespace pc {

// one output y = a * c - b * s from (c, s) = (ch + cl, sh + sl); returns the bf16 bits, or 0xFFFFFFFF when
// the value is too close to a rounding boundary to decide
__device__ __forceinline__ uint32_t rope_out_dd(float a, float b, float ch, float sh, float cl, float sl) {
  const float p = __fmul_rn(a, ch), pe = __fmaf_rn(a, ch, -p);          // a * ch = p + pe exactly
  const float q = __fmul_rn(b, sh), qe = __fmaf_rn(b, sh, -q);
  const float nq = -q;
  const float s1 = __fadd_rn(p, nq);                                     // p - q = s1 + e1 exactly (two-sum)
  const float bb = __fsub_rn(s1, p);
  const float e1 = __fadd_rn(__fsub_rn(p, __fsub_rn(s1, bb)), __fsub_rn(nq, bb));
  const float small = __fadd_rn(__fsub_rn(pe, qe), __fmaf_rn(a, cl, -__fmul_rn(b, sl)));
  const float lo = __fadd_rn(small, e1);
  float z = __fadd_rn(s1, lo);                                           // s1 + lo = z + dl exactly
  const float zz = __fsub_rn(z, s1);
  float dl = __fadd_rn(__fsub_rn(s1, __fsub_rn(z, zz)), __fsub_rn(lo, zz));
  const float mag = fabsf(a) + fabsf(b);
  const float tol = 1.1368684e-13f * mag;                                // 2^-43 (|a| + |b|)
  if (!(fabsf(z) > 3.8146973e-6f * mag)) return (z == 0.0f && mag == 0.0f) ? 0u : 0xFFFFFFFFu;   // heavy cancellation
  uint32_t u = __float_as_uint(z);
  const uint32_t sign = u & 0x80000000u;
  if (sign) dl = -dl;                                                    // work on the magnitude
  u &= 0x7FFFFFFFu;
  const uint32_t low = u & 0xFFFFu, base = u >> 16;
  uint32_t r;
  if (low != 0x8000u) r = (u + 0x7FFFu + (base & 1u)) >> 16;             // not a midpoint of two bf16 values
  else if (dl > tol) r = base + 1u;
  else if (dl < -tol) r = base;
  else return 0xFFFFFFFFu;
  return r | (sign >> 16);
}

// Table layout of the fp32 heads and tails: one float4 per TWO consecutive pairs (2i, 2i + 1) of a position,
// (cos_2i, cos_2i+1, sin_2i, sin_2i+1), so that the packed fp32 instructions find their operands in register pairs.
//
// Levels 2 and 3 for ONE output y = a * c - b * s (pass (b, -a) for the second output of a pair, b c + a s) at
// table entry `pair` of a position's row: heads in hi_row, tails in lo_row (float4 per two pairs), fp64 (cos, sin)
// in d_row.  Returns the bf16 bits.
__device__ __forceinline__ uint32_t rope_one_exact(float a, float b, int pair, const float4* __restrict__ hi_row,
                                                   const float4* __restrict__ lo_row, const double2* __restrict__ d_row) {
  const float* h = reinterpret_cast<const float*>(hi_row + (pair >> 1));
  const float* l = reinterpret_cast<const float*>(lo_row + (pair >> 1));
  const int e = pair & 1;
  uint32_t r = rope_out_dd(a, b, __ldg(h + e), __ldg(h + 2 + e), __ldg(l + e), __ldg(l + 2 + e));
  if (r == 0xFFFFFFFFu) {
    const double2 t = __ldg(d_row + pair);
    r = f64_to_bf16_rne((double)a * t.x - (double)b * t.y);
  }
  return r;
}

// Two pairs through level 1 (packed fp32 arithmetic).  x1w / x2w: the two bf16 of x1 (first half of the row) and of
// x2 (second half) as they sit in memory; same layout on return.  Returns non-zero when one of the four outputs is
// too close to a rounding boundary for level 1 to decide (that output is then not valid yet).
__device__ __forceinline__ uint32_t rope_two_pairs_fast(uint32_t x1w, uint32_t x2w, float4 hi, uint32_t& lo_out,
                                                        uint32_t& up_out) {
  const float a0 = __uint_as_float(x1w << 16), a1 = __uint_as_float(x1w & 0xFFFF0000u);
  const float b0 = __uint_as_float(x2w << 16), b1 = __uint_as_float(x2w & 0xFFFF0000u);
  const uint64_t A = pack_f32x2(a0, a1), B = pack_f32x2(b0, b1), NB = pack_f32x2(-b0, -b1);
  const uint64_t C = pack_f32x2(hi.x, hi.y), S = pack_f32x2(hi.z, hi.w);
  const uint64_t Y1 = fma_f32x2(NB, S, mul_f32x2(A, C));                 // a c - b s
  const uint64_t Y2 = fma_f32x2(A, S, mul_f32x2(B, C));                  // b c + a s
  const float m0 = fabsf(a0) + fabsf(b0), m1 = fabsf(a1) + fabsf(b1);
  const uint64_t T = pack_f32x2(2.3841858e-7f * m0, 2.3841858e-7f * m1);     // 2^-22 (|a| + |b|)
  const uint64_t NT = pack_f32x2(-2.3841858e-7f * m0, -2.3841858e-7f * m1);
  float p, q;
  unpack_f32x2(add_f32x2(Y1, NT), p, q);
  lo_out = pack_bf16x2(p, q);
  unpack_f32x2(add_f32x2(Y1, T), p, q);
  const uint32_t lo_up = pack_bf16x2(p, q);
  unpack_f32x2(add_f32x2(Y2, NT), p, q);
  up_out = pack_bf16x2(p, q);
  unpack_f32x2(add_f32x2(Y2, T), p, q);
  const uint32_t up_up = pack_bf16x2(p, q);
  return (lo_out ^ lo_up) | (up_out ^ up_up);
}

}  // namespace pc
