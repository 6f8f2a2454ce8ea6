// RoPE with position reuse (Sec. 3.1 "Parallel attention": positions restart in every
// chunk).  Pairs (t, t + d/2), angle p * theta^(-2t/d).  The rotation is evaluated in
// fp64 and rounded once to bf16, so rotated keys are reproducible to the bit.
#include "pc_kernels.h"
#include "pc_sm100.cuh"
#include "pc_rope_tile.cuh"

namespace pc {

__global__ void rope_table_kernel(double2* __restrict__ tab, float4* __restrict__ tab4, int n_pos, int half, double theta,
                                  int pos0) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_pos * half) return;
  const int p = i / half, t = i % half;
  const double inv_freq = pow(theta, -2.0 * (double)t / (double)(2 * half));
  const double phi = (double)(pos0 + p) * inv_freq;
  double s, c;
  sincos(phi, &s, &c);
  tab[i] = make_double2(c, s);
  if (tab4 != nullptr) {                                  // the same entries as fp32 head + fp32 tail: c = c_hi + c_lo to 2^-48
    const float ch = (float)c, sh = (float)s;
    tab4[i] = make_float4(ch, sh, (float)(c - (double)ch), (float)(s - (double)sh));
  }
}

void launch_rope_table(double2* tab, float4* tab4, int n_pos, int d, double theta, int pos0, cudaStream_t st) {
  const int n = n_pos * (d / 2);
  rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(tab, tab4, n_pos, d / 2, theta, pos0);
}

// One thread owns 8 consecutive pairs (t..t+7) of one position and walks all heads and a
// slice of chunks, so its 8 table entries are read once.
__global__ void __launch_bounds__(256) rope_keys_kernel(const uint16_t* __restrict__ k, long long s_chunk,
                                                        long long s_tok, long long s_head,
                                                        uint16_t* __restrict__ k_rot, const double2* __restrict__ tab,
                                                        int C, int L, int Hkv, int d) {
  const int half = d / 2;
  const int groups = half / 8;                              // 16-byte groups per half row
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= (long long)L * groups) return;
  const int p = (int)(gid / groups), g = (int)(gid % groups);
  double2 cs[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) cs[i] = tab[(size_t)p * half + g * 8 + i];
  for (int c = blockIdx.y; c < C; c += gridDim.y) {
    for (int h = 0; h < Hkv; ++h) {
      const uint16_t* src = k + (long long)c * s_chunk + (long long)p * s_tok + (long long)h * s_head;
      uint16_t* dst = k_rot + (((size_t)c * L + p) * Hkv + h) * d;
      const uint4 lo = *reinterpret_cast<const uint4*>(src + g * 8);
      const uint4 hi = *reinterpret_cast<const uint4*>(src + half + g * 8);
      const uint32_t lo_w[4] = {lo.x, lo.y, lo.z, lo.w}, hi_w[4] = {hi.x, hi.y, hi.z, hi.w};
      uint32_t out_lo[4], out_hi[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t rl = 0, rh = 0;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const double x1 = (double)__uint_as_float(((lo_w[i] >> (16 * e)) & 0xFFFFu) << 16);
          const double x2 = (double)__uint_as_float(((hi_w[i] >> (16 * e)) & 0xFFFFu) << 16);
          const double2 t = cs[2 * i + e];
          rl |= (uint32_t)f64_to_bf16_rne(x1 * t.x - x2 * t.y) << (16 * e);
          rh |= (uint32_t)f64_to_bf16_rne(x2 * t.x + x1 * t.y) << (16 * e);
        }
        out_lo[i] = rl;
        out_hi[i] = rh;
      }
      *reinterpret_cast<uint4*>(dst + g * 8) = make_uint4(out_lo[0], out_lo[1], out_lo[2], out_lo[3]);
      *reinterpret_cast<uint4*>(dst + half + g * 8) = make_uint4(out_hi[0], out_hi[1], out_hi[2], out_hi[3]);
    }
  }
}

void launch_rope_keys(const void* k, const long long k_stride[3], void* k_rot, const double2* tab, int C, int L,
                      int Hkv, int d, cudaStream_t st) {
  const long long n = (long long)L * (d / 16);
  dim3 grid((unsigned)((n + 255) / 256), (unsigned)(C < 64 ? C : 64));
  rope_keys_kernel<<<grid, 256, 0, st>>>((const uint16_t*)k, k_stride[0], k_stride[1], k_stride[2], (uint16_t*)k_rot,
                                         tab, C, L, Hkv, d);
}

// RoPE of whole [128 rows x 128] tiles with the routine the attention kernel applies to its query tiles:
// a tile is staged in shared memory in the 128-byte-swizzled layout the tensor cores read, rotated by eight
// warps of 16 rows, and written back.  x, y: [C, L, H, 128] contiguous.
__global__ void __launch_bounds__(256) rope_tiles_kernel(const uint4* __restrict__ x, uint4* __restrict__ y,
                                                         const float4* __restrict__ tab4, const double2* __restrict__ tab,
                                                         int L, int H, int tiles_per_chunk) {
  __shared__ __align__(1024) uint8_t tile[32768];
  const int tix = blockIdx.x % tiles_per_chunk, h = (blockIdx.x / tiles_per_chunk) % H, c = blockIdx.x / (tiles_per_chunk * H);
  const int tok0 = tix * 128;
  for (int i = threadIdx.x; i < 128 * 16; i += blockDim.x) {          // 16-byte pieces: row, piece (8 per 64-column atom)
    const int row = i >> 4, piece = i & 15;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (tok0 + row < L) v = x[(((size_t)c * L + tok0 + row) * H + h) * 16 + piece];
    *reinterpret_cast<uint4*>(tile + (piece >> 3) * 16384 + sw128_offset(row, piece & 7)) = v;
  }
  __syncthreads();
  rope_rows_warp(tile, (threadIdx.x >> 5) * 16, threadIdx.x & 31, tab4, tab,
                 [=](int row) { return tok0 + row < L ? tok0 + row : -1; });
  __syncthreads();
  for (int i = threadIdx.x; i < 128 * 16; i += blockDim.x) {
    const int row = i >> 4, piece = i & 15;
    if (tok0 + row < L)
      y[(((size_t)c * L + tok0 + row) * H + h) * 16 + piece] =
          *reinterpret_cast<const uint4*>(tile + (piece >> 3) * 16384 + sw128_offset(row, piece & 7));
  }
}

void launch_rope_tiles(const void* x, void* y, const float4* tab4, const double2* tab, int C, int L, int H, cudaStream_t st) {
  const int tiles = (L + 127) / 128;
  rope_tiles_kernel<<<C * H * tiles, 256, 0, st>>>((const uint4*)x, (uint4*)y, tab4, tab, L, H, tiles);
}

}  // namespace pc
