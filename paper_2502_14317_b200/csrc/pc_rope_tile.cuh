// RoPE of query rows inside a shared-memory tile (Sec. 3.1 "Parallel attention": positions restart in
// every chunk; pairs (t, t + d/2), angle p * theta^(-2t/d)), head size 128.
//
// The result is the fp64 rotation rounded ONCE to bf16, bit for bit, but fp64 arithmetic is almost never
// executed.  Three levels:
//   1. fp32 with the fp32 heads of the table entries.  Its error is below 2^-22 (|x1| + |x2|); when
//      y - tol and y + tol round to the same bf16 value, that value is the correctly rounded one.
//   2. otherwise (about one output in 4000) the value is re-evaluated as an unevaluated sum of two fp32
//      numbers (products with their exact FMA residuals, the fp32 tails of the table entries), good to
//      2^-43 (|x1| + |x2|), and rounded from there;
//   3. if that is still too close to a rounding boundary (practically never), fp64 on the fp64 table.
// Levels 2 and 3 are out-of-line so that the fast path stays small.
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

// the four outputs of one lane and row again, exactly.  t0, t1: table entries (c_hi, s_hi, c_lo, s_lo) of the
// pairs 2l and 2l + 1; tab_row: fp64 entries of the same two pairs.
static __device__ __noinline__ void rope_pairs_exact(float a0, float a1, float b0, float b1, float4 t0, float4 t1,
                                              const double2* __restrict__ tab_row, uint32_t& rl, uint32_t& rh) {
  uint32_t l0 = rope_out_dd(a0, b0, t0.x, t0.y, t0.z, t0.w), h0 = rope_out_dd(b0, -a0, t0.x, t0.y, t0.z, t0.w);
  uint32_t l1 = rope_out_dd(a1, b1, t1.x, t1.y, t1.z, t1.w), h1 = rope_out_dd(b1, -a1, t1.x, t1.y, t1.z, t1.w);
  if ((l0 | h0 | l1 | h1) == 0xFFFFFFFFu) {
    const double2 d0 = __ldg(tab_row), d1 = __ldg(tab_row + 1);
    const double da0 = (double)a0, da1 = (double)a1, db0 = (double)b0, db1 = (double)b1;
    if (l0 == 0xFFFFFFFFu) l0 = f64_to_bf16_rne(da0 * d0.x - db0 * d0.y);
    if (h0 == 0xFFFFFFFFu) h0 = f64_to_bf16_rne(db0 * d0.x + da0 * d0.y);
    if (l1 == 0xFFFFFFFFu) l1 = f64_to_bf16_rne(da1 * d1.x - db1 * d1.y);
    if (h1 == 0xFFFFFFFFu) h1 = f64_to_bf16_rne(db1 * d1.x + da1 * d1.y);
  }
  rl = l0 | (l1 << 16);
  rh = h0 | (h1 << 16);
}

// RoPE of 16 rows of a 128-byte-swizzled [128 x 128] bf16 tile (two atoms of 64 columns, the second 16384
// bytes after the first) by one warp: rows row0 .. row0 + 15, row i at position pos_of(i) (negative: leave the
// row alone).  Lane l takes the pairs (t, t + 64) for t = 2l, 2l + 1 of a row, so a warp reads a row of the
// table as one contiguous block.  Rows go in two batches of eight: all table and tile reads of a batch are
// issued before the first use (the empty asm statement pins that order: left alone, the compiler interleaves
// loads and arithmetic row by row and the warp pays the L2 latency of the table sixteen times, not twice).
template <typename PosOf>
__device__ __forceinline__ void rope_rows_warp(uint8_t* tile, int row0, int lane, const float4* __restrict__ tab4,
                                               const double2* __restrict__ tab, PosOf pos_of) {
  constexpr int HALF = 64;                                   // pairs per row
  uint8_t* const lo_base = tile + (lane & 3) * 4;
#pragma unroll
  for (int r0 = 0; r0 < 16; r0 += 8) {
    float4 t0[8], t1[8];
    uint32_t lo[8], hi[8];
    int pos[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      pos[i] = pos_of(row0 + r0 + i);
      const float4* e = tab4 + (size_t)(pos[i] < 0 ? 0 : pos[i]) * HALF + 2 * lane;
      t0[i] = __ldg(e);
      t1[i] = __ldg(e + 1);
      const uint8_t* lo_p = lo_base + sw128_offset(row0 + r0 + i, lane >> 2);
      lo[i] = *reinterpret_cast<const uint32_t*>(lo_p);
      hi[i] = *reinterpret_cast<const uint32_t*>(lo_p + 16384);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i)
      asm volatile("" : "+f"(t0[i].x), "+f"(t0[i].y), "+f"(t1[i].x), "+f"(t1[i].y), "+r"(lo[i]), "+r"(hi[i]));
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float a0 = __uint_as_float(lo[i] << 16), a1 = __uint_as_float(lo[i] & 0xFFFF0000u);   // x1 of pairs 2l, 2l + 1
      const float b0 = __uint_as_float(hi[i] << 16), b1 = __uint_as_float(hi[i] & 0xFFFF0000u);   // x2
      const float c0 = t0[i].x, s0 = t0[i].y, c1 = t1[i].x, s1 = t1[i].y;
      const float yl0 = fmaf(-b0, s0, a0 * c0), yh0 = fmaf(a0, s0, b0 * c0);
      const float yl1 = fmaf(-b1, s1, a1 * c1), yh1 = fmaf(a1, s1, b1 * c1);
      const float tol0 = 2.3841858e-7f * (fabsf(a0) + fabsf(b0)), tol1 = 2.3841858e-7f * (fabsf(a1) + fabsf(b1));   // 2^-22
      uint32_t rl = pack_bf16x2(yl0 - tol0, yl1 - tol1), rh = pack_bf16x2(yh0 - tol0, yh1 - tol1);
      const uint32_t rl_up = pack_bf16x2(yl0 + tol0, yl1 + tol1), rh_up = pack_bf16x2(yh0 + tol0, yh1 + tol1);
      if ((rl != rl_up || rh != rh_up) && pos[i] >= 0)
        rope_pairs_exact(a0, a1, b0, b1, t0[i], t1[i], tab + (size_t)pos[i] * HALF + 2 * lane, rl, rh);
      lo[i] = rl;
      hi[i] = rh;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (pos[i] < 0) continue;
      uint8_t* lo_p = lo_base + sw128_offset(row0 + r0 + i, lane >> 2);
      *reinterpret_cast<uint32_t*>(lo_p) = lo[i];
      *reinterpret_cast<uint32_t*>(lo_p + 16384) = hi[i];
    }
  }
}

}  // namespace pc
