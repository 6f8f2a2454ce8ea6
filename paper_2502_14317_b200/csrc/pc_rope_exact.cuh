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
// Levels 2 and 3 for the two pairs (a0, b0), (a1, b1) at the table entry `hi` (heads), `lo_p` (tails), `d_p` (fp64,
// (cos, sin) per pair).  Returns the bf16 bits: y1 = a c - b s of both pairs in lo_out, y2 = b c + a s in up_out.
__device__ __noinline__ static void rope_pairs_exact(float a0, float a1, float b0, float b1, float4 hi,
                                                     const float4* __restrict__ lo_p, const double2* __restrict__ d_p,
                                                     uint32_t& lo_out, uint32_t& up_out) {
  const float4 lo = __ldg(lo_p);
  uint32_t y1a = rope_out_dd(a0, b0, hi.x, hi.z, lo.x, lo.z), y2a = rope_out_dd(b0, -a0, hi.x, hi.z, lo.x, lo.z);
  uint32_t y1b = rope_out_dd(a1, b1, hi.y, hi.w, lo.y, lo.w), y2b = rope_out_dd(b1, -a1, hi.y, hi.w, lo.y, lo.w);
  if ((y1a | y2a | y1b | y2b) == 0xFFFFFFFFu) {
    const double2 t0 = __ldg(d_p), t1 = __ldg(d_p + 1);
    const double da0 = (double)a0, da1 = (double)a1, db0 = (double)b0, db1 = (double)b1;
    if (y1a == 0xFFFFFFFFu) y1a = f64_to_bf16_rne(da0 * t0.x - db0 * t0.y);
    if (y2a == 0xFFFFFFFFu) y2a = f64_to_bf16_rne(db0 * t0.x + da0 * t0.y);
    if (y1b == 0xFFFFFFFFu) y1b = f64_to_bf16_rne(da1 * t1.x - db1 * t1.y);
    if (y2b == 0xFFFFFFFFu) y2b = f64_to_bf16_rne(db1 * t1.x + da1 * t1.y);
  }
  lo_out = y1a | (y1b << 16);
  up_out = y2a | (y2b << 16);
}

// Two pairs through level 1 (packed fp32 arithmetic); falls back to rope_pairs_exact.  x1w / x2w: the two bf16 of
// x1 (first half of the row) and of x2 (second half) as they sit in memory; same layout on return.
__device__ __forceinline__ void rope_two_pairs(uint32_t x1w, uint32_t x2w, float4 hi, const float4* __restrict__ lo_p,
                                               const double2* __restrict__ d_p, uint32_t& lo_out, uint32_t& up_out) {
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
  const uint32_t lo_dn = pack_bf16x2(p, q);
  unpack_f32x2(add_f32x2(Y1, T), p, q);
  const uint32_t lo_up = pack_bf16x2(p, q);
  unpack_f32x2(add_f32x2(Y2, NT), p, q);
  const uint32_t up_dn = pack_bf16x2(p, q);
  unpack_f32x2(add_f32x2(Y2, T), p, q);
  const uint32_t up_up = pack_bf16x2(p, q);
  lo_out = lo_dn;
  up_out = up_dn;
  if (((lo_dn ^ lo_up) | (up_dn ^ up_up)) != 0u) rope_pairs_exact(a0, a1, b0, b1, hi, lo_p, d_p, lo_out, up_out);
}

}  // namespace pc
