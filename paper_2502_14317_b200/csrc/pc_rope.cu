// RoPE with position reuse (Sec. 3.1 "Parallel attention": positions restart in every
// chunk).  Pairs (t, t + d/2), angle p * theta^(-2t/d).  Queries and keys are rotated once,
// before the attention kernel, by a bandwidth-bound pass: the result is the fp64 rotation
// rounded once to bf16 (see pc_rope_exact.cuh for how fp32 arithmetic gets there), so rotated
// keys - an output that the gather copies - are reproducible to the bit.
#include "pc_kernels.h"
#include "pc_rope_exact.cuh"

namespace pc {

// tab: (cos, sin) per (position, pair), fp64.  tab_hi / tab_lo: fp32 heads / tails of the same values, one float4
// per two consecutive pairs (cos_2i, cos_2i+1, sin_2i, sin_2i+1); value = head + tail to 2^-48.
__global__ void rope_table_kernel(double2* __restrict__ tab, float4* __restrict__ tab_hi, float4* __restrict__ tab_lo, int n_pos,
                                  int half, double theta, int pos0) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;      // one thread per two pairs
  if (i >= n_pos * (half / 2)) return;
  const int p = i / (half / 2), t = 2 * (i % (half / 2));
  double c[2], s[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const double inv_freq = pow(theta, -2.0 * (double)(t + e) / (double)(2 * half));
    sincos((double)(pos0 + p) * inv_freq, &s[e], &c[e]);
    tab[(size_t)p * half + t + e] = make_double2(c[e], s[e]);
  }
  if (tab_hi != nullptr) {
    const float c0 = (float)c[0], c1 = (float)c[1], s0 = (float)s[0], s1 = (float)s[1];
    tab_hi[i] = make_float4(c0, c1, s0, s1);
    tab_lo[i] = make_float4((float)(c[0] - (double)c0), (float)(c[1] - (double)c1), (float)(s[0] - (double)s0),
                            (float)(s[1] - (double)s1));
  }
}

void launch_rope_table(double2* tab, float4* tab_hi, float4* tab_lo, int n_pos, int d, double theta, int pos0, cudaStream_t st) {
  const int n = n_pos * (d / 4);
  note_launch();
  rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(tab, tab_hi, tab_lo, n_pos, d / 2, theta, pos0);
}

// y[c,p,h,:] = bf16( RoPE(x[c,p,h,:], position p) ).  One warp owns one position: a lane holds 8 consecutive
// pairs (t .. t+7) and takes every (32 / (d/16))-th head, so one pass of the warp reads and writes a contiguous
// piece of the token's row (1 KB for d = 128), and a block of 8 warps streams 8 adjacent rows: the DRAM pages
// are walked front to back, as a copy would.  The table entries of (position, pairs) stay in registers across
// the heads and across the chunks of the block's slice.
// Outputs that the fp32 arithmetic cannot decide (about one in 1300) are redone exactly by the whole warp: the
// sixteen outputs of an undecided lane go to sixteen lanes, one each, and are patched into the row after the
// vector store.  (Handling them in the lane that found them would make a third of the warp's passes wait for one
// lane's slow path.)
__global__ void __launch_bounds__(256, 4) rope_rows_kernel(const uint16_t* __restrict__ x, long long s_chunk, long long s_tok,
                                                           long long s_head, uint16_t* __restrict__ y,
                                                           const float4* __restrict__ tab_hi, const float4* __restrict__ tab_lo,
                                                           const double2* __restrict__ tab, int C, int L, int H, int d) {
  const int half = d / 2;
  const int groups = half / 8;                              // 16-byte groups per half row (4 or 8)
  const int lane = threadIdx.x & 31;
  const int p = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (p >= L) return;                                       // whole warps leave together
  const int g = lane % groups, h_first = lane / groups, h_step = 32 / groups;
  const size_t row0 = (size_t)p * half;                     // first pair of this position in the tables
  const float4* hi_row = tab_hi + row0 / 2;
  const float4* lo_row = tab_lo + row0 / 2;
  const double2* d_row = tab + row0;
  float4 hi[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) hi[i] = __ldg(hi_row + g * 4 + i);
  const int zs = gridDim.z;                                 // small inputs: the head passes are dealt out over grid.z
  const long long step_src = (long long)h_step * zs * s_head;
  const size_t step_dst = (size_t)h_step * zs * d;
  const int n_pass = (H + h_step - 1) / h_step;
  const int h_mine = h_first + (int)blockIdx.z * h_step;    // this thread's head in its first pass
  for (int c = blockIdx.y; c < C; c += gridDim.y) {
    const uint16_t* src = x + (long long)c * s_chunk + (long long)p * s_tok + (long long)h_mine * s_head + g * 8;
    uint16_t* const dst_tok = y + ((size_t)c * L + p) * H * d;
    uint16_t* dst = dst_tok + (size_t)h_mine * d + g * 8;
    uint4 n1 = make_uint4(0, 0, 0, 0), n2 = make_uint4(0, 0, 0, 0);
    if (h_mine < H) {
      n1 = __ldg(reinterpret_cast<const uint4*>(src));
      n2 = __ldg(reinterpret_cast<const uint4*>(src + half));
    }
#pragma unroll 1
    for (int ps = blockIdx.z; ps < n_pass; ps += zs, src += step_src, dst += step_dst) {
      const bool active = h_first + ps * h_step < H;
      const uint4 x1 = n1, x2 = n2;
      if (ps + zs < n_pass && h_first + (ps + zs) * h_step < H) {                // the next pass's row is in flight during this one's arithmetic
        n1 = __ldg(reinterpret_cast<const uint4*>(src + step_src));
        n2 = __ldg(reinterpret_cast<const uint4*>(src + step_src + half));
      } else {
        n1 = make_uint4(0, 0, 0, 0); n2 = make_uint4(0, 0, 0, 0);
      }
      uint4 y1, y2;
      uint32_t amb = rope_two_pairs_fast(x1.x, x2.x, hi[0], y1.x, y2.x);
      amb |= rope_two_pairs_fast(x1.y, x2.y, hi[1], y1.y, y2.y);
      amb |= rope_two_pairs_fast(x1.z, x2.z, hi[2], y1.z, y2.z);
      amb |= rope_two_pairs_fast(x1.w, x2.w, hi[3], y1.w, y2.w);
      if (active) {
        *reinterpret_cast<uint4*>(dst) = y1;
        *reinterpret_cast<uint4*>(dst + half) = y2;
      }
      unsigned todo = __ballot_sync(0xFFFFFFFFu, active && amb != 0u);
      if (todo != 0u) {                                     // warp-uniform
        __syncwarp();                                       // the vector stores above precede the patches below
        const int t = (lane >> 1) & 7, second = lane & 1;   // lanes 0..15: pair t of the undecided lane, first / second output
        do {
          const int srcl = __ffs(todo) - 1;
          todo &= todo - 1;
          const uint32_t w1[4] = {__shfl_sync(0xFFFFFFFFu, x1.x, srcl), __shfl_sync(0xFFFFFFFFu, x1.y, srcl),
                                  __shfl_sync(0xFFFFFFFFu, x1.z, srcl), __shfl_sync(0xFFFFFFFFu, x1.w, srcl)};
          const uint32_t w2[4] = {__shfl_sync(0xFFFFFFFFu, x2.x, srcl), __shfl_sync(0xFFFFFFFFu, x2.y, srcl),
                                  __shfl_sync(0xFFFFFFFFu, x2.z, srcl), __shfl_sync(0xFFFFFFFFu, x2.w, srcl)};
          if (lane < 16) {
            const int wsel = t >> 1;
            const uint32_t u1 = wsel == 0 ? w1[0] : wsel == 1 ? w1[1] : wsel == 2 ? w1[2] : w1[3];
            const uint32_t u2 = wsel == 0 ? w2[0] : wsel == 1 ? w2[1] : wsel == 2 ? w2[2] : w2[3];
            const float a = __uint_as_float((t & 1) ? (u1 & 0xFFFF0000u) : (u1 << 16));
            const float b = __uint_as_float((t & 1) ? (u2 & 0xFFFF0000u) : (u2 << 16));
            const int sg = srcl % groups, sh = srcl / groups + ps * h_step;      // pair group and head of that lane
            const int pair = sg * 8 + t;
            const uint32_t r = second ? rope_one_exact(b, -a, pair, hi_row, lo_row, d_row)
                                      : rope_one_exact(a, b, pair, hi_row, lo_row, d_row);
            dst_tok[(size_t)sh * d + (second ? half : 0) + pair] = (uint16_t)r;
          }
        } while (todo != 0u);
        __syncwarp();
      }
    }
  }
}

void launch_rope_rows(const void* x, const long long x_stride[3], void* y, const double2* tab, const float4* tab_hi,
                      const float4* tab_lo, int C, int L, int H, int d, cudaStream_t st) {
  const int bx = (L + 7) / 8;                               // 8 positions per block
  // a slice of the chunks per block: the table entries are reused over the slice; enough blocks to fill the GPU
  int ny = (4736 + bx - 1) / bx;
  ny = ny < 1 ? 1 : (ny > C ? C : ny);
  // a few positions and chunks only (the query window of one sequence): the passes over the heads, which a warp
  // would otherwise walk one after the other, become blocks of their own
  const int n_pass = (H + 32 / (d / 16) - 1) / (32 / (d / 16));
  int nz = bx * ny < 592 ? 592 / (bx * ny) : 1;
  nz = nz > n_pass ? n_pass : (nz < 1 ? 1 : nz);
  dim3 grid((unsigned)bx, (unsigned)ny, (unsigned)nz);
  note_launch();
  rope_rows_kernel<<<grid, 256, 0, st>>>((const uint16_t*)x, x_stride[0], x_stride[1], x_stride[2], (uint16_t*)y, tab_hi,
                                         tab_lo, tab, C, L, H, d);
}

// Rows behind the end of a chunk that is shorter than L (per-chunk lengths): outputs read as zero there.
__global__ void zero_chunk_tails_kernel(const int* __restrict__ chunk_len, int L, int w, int Hq, int Hkv, int d,
                                        uint16_t* __restrict__ o, long long so_chunk, long long so_tok, long long so_head,
                                        float* __restrict__ lse, float* __restrict__ win_score) {
  const int c = blockIdx.y;
  int len = chunk_len[c];
  len = len > L ? L : (len <= w ? w + 1 : len);
  const int n_tail = L - len;
  const long long per_tok = (long long)Hq * (d / 8);        // 16-byte pieces of an output row over all heads
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < (long long)n_tail * per_tok;
       i += (long long)gridDim.x * blockDim.x) {
    const int p = len + (int)(i / per_tok), rest = (int)(i % per_tok), h = rest / (d / 8), piece = rest % (d / 8);
    *reinterpret_cast<uint4*>(o + (long long)c * so_chunk + (long long)p * so_tok + (long long)h * so_head + piece * 8) =
        make_uint4(0, 0, 0, 0);
  }
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < (long long)n_tail * (Hq + Hkv);
       i += (long long)gridDim.x * blockDim.x) {
    const int row = (int)(i / n_tail), p = len + (int)(i % n_tail);
    if (row < Hq) { if (lse != nullptr) lse[((size_t)c * Hq + row) * L + p] = 0.0f; }
    else win_score[((size_t)c * Hkv + (row - Hq)) * L + p] = 0.0f;
  }
}

void launch_zero_chunk_tails(const int* chunk_len, int C, int L, int w, int Hq, int Hkv, int d, void* o,
                             const long long o_stride[3], float* lse, float* win_score, cudaStream_t st) {
  note_launch();
  zero_chunk_tails_kernel<<<dim3(64, (unsigned)C), 256, 0, st>>>(chunk_len, L, w, Hq, Hkv, d, (uint16_t*)o, o_stride[0],
                                                                o_stride[1], o_stride[2], lse, win_score);
}

}  // namespace pc
