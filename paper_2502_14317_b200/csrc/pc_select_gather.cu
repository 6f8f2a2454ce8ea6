// Ranking and gather kernels: chunk top-m (Eq. 3-4), token top-k per kv-head (Eq. 7),
// compressed-cache gather (Eq. 7, Eq. 9), and the single-layer stand-in for the chunk
// self-information.  All HBM- or latency-bound; no tensor cores here on purpose.
#include "pc_kernels.h"

namespace pc {

// Monotone map float -> uint32 with "larger key = better".  NaN ranks worst, -0 == +0.
__device__ __forceinline__ uint32_t rank_key(float f, bool lower_is_better) {
  if (f != f) return 0u;
  if (lower_is_better) f = -f;
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;                       // -0 -> +0
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return u == 0u ? 1u : u;                            // keep 0 for NaN only (-NaN patterns never reach here)
}

// ------------------------------------------------------------------ chunk score stand-in
__global__ void chunk_score_kernel(const float* __restrict__ win_lse, int n_per_chunk, float* __restrict__ score) {
  __shared__ double part[256];
  const int c = blockIdx.x;
  double acc = 0.0;
  for (int i = threadIdx.x; i < n_per_chunk; i += blockDim.x) acc += (double)win_lse[(size_t)c * n_per_chunk + i];
  part[threadIdx.x] = acc;
  __syncthreads();
  for (int s = blockDim.x / 2; s > 0; s >>= 1) {       // fixed tree: deterministic
    if (threadIdx.x < s) part[threadIdx.x] += part[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) score[c] = (float)(-part[0] / (double)n_per_chunk);
}

void launch_chunk_score(const float* win_lse, int C, int n_per_chunk, float* score, cudaStream_t st) {
  chunk_score_kernel<<<C, 256, 0, st>>>(win_lse, n_per_chunk, score);
}

// ------------------------------------------------------------------ chunk top-m
// One block; thread i ranks chunk i against all others (C <= 1024).
__global__ void select_chunks_kernel(const float* __restrict__ score, int C, int m, int lower_is_better,
                                     int* __restrict__ kept) {
  __shared__ uint32_t key[1024];
  __shared__ int flag[1024];
  const int i = threadIdx.x;
  if (i < C) key[i] = rank_key(score[i], lower_is_better != 0);
  __syncthreads();
  int sel = 0;
  if (i < C) {
    const uint32_t mine = key[i];
    int rank = 0;
    for (int j = 0; j < C; ++j) rank += (key[j] > mine) || (key[j] == mine && j < i);
    sel = rank < m;
  }
  flag[i] = sel;
  __syncthreads();
  if (sel) {
    int pos = 0;
    for (int j = 0; j < i; ++j) pos += flag[j];
    kept[pos] = i;
  }
}

void launch_select_chunks(const float* score, int C, int m, int lower_is_better, int* kept, cudaStream_t st) {
  select_chunks_kernel<<<1, 1024, 0, st>>>(score, C, m, lower_is_better, kept);
}

// ------------------------------------------------------------------ token top-k
// One CTA per (kept chunk, kv-head) row.  The row's keys sit in shared memory; an
// 8-bit-digit radix search finds the k-th largest key T, then one ordered sweep emits
// the positions with key > T plus the first (k - count_gt) positions with key == T,
// so ties go to the lower position and the output is ascending.
constexpr int SEL_THREADS = 1024;
constexpr int SEL_WARPS = SEL_THREADS / 32;

__global__ void __launch_bounds__(SEL_THREADS) select_tokens_kernel(const float* __restrict__ win_score,
                                                                    const int* __restrict__ kept, int Hkv, int L,
                                                                    int n_cand, int k, int* __restrict__ idx) {
  extern __shared__ uint32_t sel_smem[];
  uint32_t* keys = sel_smem;                                   // [n_cand]
  uint32_t* hist = sel_smem + ((n_cand + 31) & ~31);           // [SEL_WARPS][256]
  __shared__ uint32_t tot[256];
  __shared__ uint32_t s_prefix, s_remaining;
  __shared__ int2 scan[SEL_THREADS];

  const int row = blockIdx.x;                 // r * Hkv + hkv
  const int r = row / Hkv, hk = row % Hkv;
  const int c = kept[r];
  const float* src = win_score + ((size_t)c * Hkv + hk) * L;
  int* out = idx + (size_t)row * k;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (k >= n_cand) {                          // nothing to evict: identity, then -1 padding
    for (int j = tid; j < k; j += SEL_THREADS) out[j] = j < n_cand ? j : -1;
    return;
  }
  for (int j = tid; j < n_cand; j += SEL_THREADS) keys[j] = rank_key(src[j], false);
  if (tid == 0) { s_prefix = 0u; s_remaining = (uint32_t)k; }
  __syncthreads();

  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int b = tid; b < SEL_WARPS * 256; b += SEL_THREADS) hist[b] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t himask = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
    uint32_t* myhist = hist + warp * 256;
    const int n_round = (n_cand + SEL_THREADS - 1) / SEL_THREADS * SEL_THREADS;
    for (int j = tid; j < n_round; j += SEL_THREADS) {
      const bool active = j < n_cand && ((keys[j < n_cand ? j : 0] & himask) == prefix);
      const uint32_t digit = active ? ((keys[j] >> shift) & 0xFFu) : 0x100u;
      const uint32_t peers = __match_any_sync(0xFFFFFFFFu, digit);
      if (active && lane == (__ffs(peers) - 1)) myhist[digit] += __popc(peers);   // one writer per digit per warp
      __syncwarp();
    }
    __syncthreads();
    if (tid < 256) {
      uint32_t s = 0;
      for (int wv = 0; wv < SEL_WARPS; ++wv) s += hist[wv * 256 + tid];
      tot[tid] = s;
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t remaining = s_remaining, above = 0;
      int b = 255;
      for (; b > 0; --b) {
        if (above + tot[b] >= remaining) break;
        above += tot[b];
      }
      s_remaining = remaining - above;
      s_prefix = prefix | ((uint32_t)b << shift);
    }
    __syncthreads();
  }
  const uint32_t T = s_prefix;
  const int need_eq = (int)s_remaining;        // how many keys equal to T are taken (lowest positions first)

  // ordered emission: contiguous segment per thread, block scan of (count_gt, count_eq)
  const int seg = (n_cand + SEL_THREADS - 1) / SEL_THREADS;
  const int j0 = tid * seg, j1 = min(j0 + seg, n_cand);
  int gt = 0, eq = 0;
  for (int j = j0; j < j1; ++j) { gt += keys[j] > T; eq += keys[j] == T; }
  scan[tid] = make_int2(gt, eq);
  __syncthreads();
  for (int off = 1; off < SEL_THREADS; off <<= 1) {            // Hillis-Steele inclusive scan
    int2 v = scan[tid];
    if (tid >= off) { int2 u = scan[tid - off]; v.x += u.x; v.y += u.y; }
    __syncthreads();
    scan[tid] = v;
    __syncthreads();
  }
  int gt_before = scan[tid].x - gt, eq_before = scan[tid].y - eq;
  for (int j = j0; j < j1; ++j) {
    const uint32_t key = keys[j];
    if (key > T) {
      out[gt_before + min(eq_before, need_eq)] = j;
      ++gt_before;
    } else if (key == T) {
      if (eq_before < need_eq) out[gt_before + eq_before] = j;
      ++eq_before;
    }
  }
}

cudaError_t launch_select_tokens(const float* win_score, const int* kept, int m, int Hkv, int L, int n_cand, int k,
                                 int* idx, cudaStream_t st) {
  const size_t smem = ((size_t)((n_cand + 31) & ~31) + SEL_WARPS * 256) * sizeof(uint32_t);
  static size_t configured = 0;
  if (smem > 48 * 1024 && smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(select_tokens_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  select_tokens_kernel<<<m * Hkv, SEL_THREADS, smem, st>>>(win_score, kept, Hkv, L, n_cand, k, idx);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ gather
// One row of d bf16 (2d bytes) per (kv-head, slot); LPR lanes move one row with 16-byte
// accesses, K and V in the same thread so both copies are in flight together.
template <int D>
__global__ void __launch_bounds__(256) gather_kv_kernel(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src,
                                                        long long s_chunk, long long s_tok, long long s_head,   // in uint4 units
                                                        const int* __restrict__ kept, const int* __restrict__ idx, int m,
                                                        int Hkv, int k, uint4* __restrict__ k_out,
                                                        uint4* __restrict__ v_out, int* __restrict__ pos_out) {
  constexpr int LPR = D / 8;                                   // lanes per row
  const long long n_rows = (long long)Hkv * m * k;
  const long long gthreads = (long long)gridDim.x * blockDim.x;
  const int sub = threadIdx.x % LPR;
  for (long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) / LPR; row < n_rows; row += gthreads / LPR) {
    const int hk = (int)(row / ((long long)m * k));
    const int slot = (int)(row % ((long long)m * k));
    const int r = slot / k, t = slot % k;
    const int j = idx[((size_t)r * Hkv + hk) * k + t];
    uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
    if (j >= 0) {
      const long long off = (long long)kept[r] * s_chunk + (long long)j * s_tok + (long long)hk * s_head + sub;
      kv = __ldg(k_src + off);
      vv = __ldg(v_src + off);
    }
    k_out[row * LPR + sub] = kv;
    v_out[row * LPR + sub] = vv;
    if (pos_out != nullptr && sub == 0) pos_out[row] = j;
  }
}

cudaError_t launch_gather_kv(const void* k_src, const void* v_src, const long long stride_elems[3], const int* kept,
                             const int* idx, int m, int Hkv, int k, int d, void* k_out, void* v_out, int* pos_out,
                             int sm_count, cudaStream_t st) {
  const long long n_rows = (long long)Hkv * m * k;
  const int lpr = d / 8;
  long long want = (n_rows * lpr + 255) / 256;
  int blocks = (int)(want < (long long)sm_count * 8 ? want : (long long)sm_count * 8);
  if (blocks < 1) blocks = 1;
  const long long sc = stride_elems[0] / 8, stok = stride_elems[1] / 8, sh = stride_elems[2] / 8;
  if (d == 128)
    gather_kv_kernel<128><<<blocks, 256, 0, st>>>((const uint4*)k_src, (const uint4*)v_src, sc, stok, sh, kept, idx, m,
                                                  Hkv, k, (uint4*)k_out, (uint4*)v_out, pos_out);
  else
    gather_kv_kernel<64><<<blocks, 256, 0, st>>>((const uint4*)k_src, (const uint4*)v_src, sc, stok, sh, kept, idx, m,
                                                 Hkv, k, (uint4*)k_out, (uint4*)v_out, pos_out);
  return cudaGetLastError();
}

}  // namespace pc
