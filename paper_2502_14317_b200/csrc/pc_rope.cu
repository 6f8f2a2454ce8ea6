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
__global__ void __launch_bounds__(256, 4) rope_rows_kernel(const uint16_t* __restrict__ x, long long s_chunk, long long s_tok,
                                                           long long s_head, uint16_t* __restrict__ y,
                                                           const float4* __restrict__ tab_hi, const float4* __restrict__ tab_lo,
                                                           const double2* __restrict__ tab, int C, int L, int H, int d) {
  const int half = d / 2;
  const int groups = half / 8;                              // 16-byte groups per half row (4 or 8)
  const int lane = threadIdx.x & 31;
  const int p = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (p >= L) return;
  const int g = lane % groups, h_first = lane / groups, h_step = 32 / groups;
  const size_t e0 = (size_t)p * half + g * 8;               // first pair of this thread in the tables
  float4 hi[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) hi[i] = __ldg(tab_hi + e0 / 2 + i);
  for (int c = blockIdx.y; c < C; c += gridDim.y) {
    const uint16_t* src_c = x + (long long)c * s_chunk + (long long)p * s_tok + g * 8;
    uint16_t* dst_c = y + ((size_t)c * L + p) * H * d + g * 8;
#pragma unroll 1
    for (int h = h_first; h < H; h += h_step) {
      const uint16_t* src = src_c + (long long)h * s_head;
      uint16_t* dst = dst_c + (size_t)h * d;
      const uint4 x1 = __ldg(reinterpret_cast<const uint4*>(src));
      const uint4 x2 = __ldg(reinterpret_cast<const uint4*>(src + half));
      uint4 y1, y2;
      rope_two_pairs(x1.x, x2.x, hi[0], tab_lo + e0 / 2 + 0, tab + e0 + 0, y1.x, y2.x);
      rope_two_pairs(x1.y, x2.y, hi[1], tab_lo + e0 / 2 + 1, tab + e0 + 2, y1.y, y2.y);
      rope_two_pairs(x1.z, x2.z, hi[2], tab_lo + e0 / 2 + 2, tab + e0 + 4, y1.z, y2.z);
      rope_two_pairs(x1.w, x2.w, hi[3], tab_lo + e0 / 2 + 3, tab + e0 + 6, y1.w, y2.w);
      *reinterpret_cast<uint4*>(dst) = y1;
      *reinterpret_cast<uint4*>(dst + half) = y2;
    }
  }
}

void launch_rope_rows(const void* x, const long long x_stride[3], void* y, const double2* tab, const float4* tab_hi,
                      const float4* tab_lo, int C, int L, int H, int d, cudaStream_t st) {
  const int bx = (L + 7) / 8;                               // 8 positions per block
  // a slice of the chunks per block: the table entries are reused over the slice; enough blocks to fill the GPU
  int ny = (4736 + bx - 1) / bx;
  ny = ny < 1 ? 1 : (ny > C ? C : ny);
  dim3 grid((unsigned)bx, (unsigned)ny);
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
