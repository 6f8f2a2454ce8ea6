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
// One CTA per (kept chunk, kv-head) row, 32 candidates per thread held in REGISTERS.
//   1. The row is read once with coalesced 16-byte loads into shared memory (padded by one
//      word per 32 so that the next step is free of bank conflicts); every thread then takes
//      the 32 consecutive positions [32 tid, 32 tid + 32) as order-preserving uint32 keys and
//      transposes its 32 x 32 bit matrix in registers: word b then holds bit b of all 32 keys.
//   2. The k-th largest key T is found bit by bit, most significant first.  On the bit slices a
//      round is three instructions per thread (and, popc, add) plus one redux per warp, one
//      shared-memory atomic per warp and one barrier: 32 rounds whatever the distribution of
//      the scores, no histogram hot spots, and the masks of the keys > T and == T fall out.
//   3. One block scan of (count > T, count == T) gives every thread its output offset; positions
//      with key > T plus the first (k - count_gt) positions with key == T are staged in shared
//      memory in ascending order (ties go to the lower position) and written out coalesced.
// HBM traffic: the row once (4 B per candidate) + 4 B per kept index.
constexpr int SEL_KPT = 32;                                    // keys per thread
constexpr int SEL_MAX_THREADS = 1024;                          // n_cand <= 32768

__device__ __forceinline__ int sel_pad(int p) { return p + (p >> 5); }

// Attention calibration (Eq. 8): a candidate whose score exceeds the threshold of its region (first n_s
// positions / last n_r positions / the rest) is evicted before the ranking.  +inf switches a region off.
struct SelCalib {
  int on, n_s, n_r;
  float lam_s, lam_m, lam_r;
};

__global__ void __launch_bounds__(SEL_MAX_THREADS) select_tokens_kernel(const float* __restrict__ win_score,
                                                                        const int* __restrict__ kept, int Hkv, int L,
                                                                        int n_cand, int k, int* __restrict__ idx,
                                                                        const SelCalib cal) {
  extern __shared__ uint32_t sel_smem[];                       // [n_pad] keys, later reused for the staged output
  __shared__ int s_cnt[32];                                    // per bit: keys of the row >= the candidate threshold
  __shared__ int2 s_scan[32];

  const int row = blockIdx.x;                                  // r * Hkv + hkv
  const int r = row / Hkv, hk = row % Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  int* out = idx + (size_t)row * k;

  if (tid < 32) s_cnt[tid] = 0;                                // visible after the barrier that follows the row load
  if (k >= n_cand && !cal.on) {                                // nothing to evict: identity, then -1 padding
    for (int j = tid; j < k; j += blockDim.x) out[j] = j < n_cand ? j : -1;
    return;
  }
  const int k_out = k;
  if (k > n_cand) k = n_cand;                                  // calibrated: rank all candidates, pad the rest
  const int c = kept[r];
  const float* src = win_score + ((size_t)c * Hkv + hk) * L;

  // keys: NaN ranks below every number (1); evicted candidates and the padding rank below NaN (0) and are
  // never emitted
  auto key_of = [&](float v, int p) -> uint32_t {
    uint32_t kk = rank_key(v, false);
    kk = kk == 0u ? 1u : kk;
    if (cal.on) {
      const float lam = p < cal.n_s ? cal.lam_s : (p >= n_cand - cal.n_r ? cal.lam_r : cal.lam_m);
      if (v > lam) kk = 0u;
    }
    return kk;
  };
  // ---- 1. row -> shared memory (coalesced), -> registers (32 consecutive positions per thread)
  if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
    const float4* src4 = reinterpret_cast<const float4*>(src);
    const int n4 = n_cand >> 2;
    for (int i = tid; i < n4; i += blockDim.x) {
      const float4 v = __ldg(src4 + i);
      const int p = 4 * i;                                     // 4 consecutive positions never straddle a pad slot
      uint32_t* d = sel_smem + sel_pad(p);
      d[0] = key_of(v.x, p); d[1] = key_of(v.y, p + 1); d[2] = key_of(v.z, p + 2); d[3] = key_of(v.w, p + 3);
    }
    for (int p = (n4 << 2) + tid; p < n_cand; p += blockDim.x) sel_smem[sel_pad(p)] = key_of(__ldg(src + p), p);
  } else {
    for (int p = tid; p < n_cand; p += blockDim.x) sel_smem[sel_pad(p)] = key_of(__ldg(src + p), p);
  }
  __syncthreads();
  uint32_t key[SEL_KPT];
  const int p0 = tid * SEL_KPT;
#pragma unroll
  for (int i = 0; i < SEL_KPT; ++i) key[i] = (p0 + i < n_cand) ? sel_smem[p0 + i + tid] : 0u;   // pad(p0 + i) = p0 + i + tid; 0 ranks below every candidate

  // in-register transpose of the 32 x 32 bit matrix: afterwards key[31 - b] holds bit b of every
  // key, the key at position p0 + i sitting at bit 31 - i
  {
    uint32_t m = 0x0000FFFFu;
#pragma unroll
    for (int j = 16; j != 0; j >>= 1, m ^= (m << j)) {
#pragma unroll
      for (int q = 0; q < 32; q = (q + j + 1) & ~j) {
        const uint32_t t = (key[q] ^ (key[q + j] >> j)) & m;
        key[q] ^= t;
        key[q + j] ^= (t << j);
      }
    }
  }

  // ---- 2. k-th largest key, bit by bit.  active: keys equal to T on the bits decided so far;
  // above: keys already known to be larger than T.
  uint32_t active = 0xFFFFFFFFu, above = 0u, T = 0u;
  int n_above = 0;
#pragma unroll
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t ones = active & key[31 - bit];
    int cnt = n_above + __popc(ones);                          // keys >= (T | 1 << bit)
    cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
    if (lane == 0) atomicAdd(&s_cnt[bit], cnt);
    __syncthreads();
    if (s_cnt[bit] >= k) {                                     // at least k keys are that large: the k-th largest has this bit
      T |= 1u << bit;
      active = ones;
    } else {
      above |= ones;
      n_above += __popc(ones);
      active &= ~key[31 - bit];
    }
  }
  // active = keys == T.  T == 0 only when fewer than k candidates survived calibration: the keys equal to 0
  // are evicted candidates and padding, none of which is emitted

  // ---- 3. ordered emission
  const int gt = n_above, eq = __popc(active);
  int sgt = gt, seq = eq;                                      // inclusive warp scan of both counts
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int a = __shfl_up_sync(0xFFFFFFFFu, sgt, off), b2 = __shfl_up_sync(0xFFFFFFFFu, seq, off);
    if (lane >= off) { sgt += a; seq += b2; }
  }
  if (lane == 31) s_scan[warp] = make_int2(sgt, seq);
  __syncthreads();                                             // also: every thread is done reading the keys from shared memory
  int gt_before = sgt - gt, eq_before = seq - eq, gt_total = 0;
  for (int wv = 0; wv < nwarps; ++wv) {
    const int2 t = s_scan[wv];
    if (wv < warp) { gt_before += t.x; eq_before += t.y; }
    gt_total += t.x;
  }
  const int need_eq = T == 0u ? 0 : k - gt_total;              // keys equal to T that are taken (lowest positions first)
  const int n_emit = gt_total + need_eq;
  int* stage = reinterpret_cast<int*>(sel_smem);               // [k]
#pragma unroll
  for (int i = 0; i < SEL_KPT; ++i) {
    const uint32_t sel_bit = 0x80000000u >> i;
    if (above & sel_bit) {
      stage[gt_before + min(eq_before, need_eq)] = p0 + i;
      ++gt_before;
    } else if (active & sel_bit) {
      if (eq_before < need_eq) stage[gt_before + eq_before] = p0 + i;
      ++eq_before;
    }
  }
  __syncthreads();
  for (int j = tid; j < k_out; j += blockDim.x) out[j] = j < n_emit ? stage[j] : -1;
}

cudaError_t launch_select_tokens(const float* win_score, const int* kept, int m, int Hkv, int L, int n_cand, int k,
                                 int* idx, const float* calib /* null or {n_s, n_r, lam_s, lam_m, lam_r} */,
                                 cudaStream_t st) {
  int threads = ((n_cand + SEL_KPT - 1) / SEL_KPT + 31) / 32 * 32;
  if (threads < 32) threads = 32;
  if (threads > SEL_MAX_THREADS) return cudaErrorInvalidValue;
  const size_t words = (size_t)n_cand + (n_cand >> 5) + 1;
  SelCalib cal = {0, 0, 0, 0.f, 0.f, 0.f};
  if (calib) cal = SelCalib{1, (int)calib[0], (int)calib[1], calib[2], calib[3], calib[4]};
  const size_t stage = (k < n_cand || cal.on) ? (size_t)(k < n_cand ? k : n_cand) : 0;   // uncalibrated k >= n_cand writes the identity directly
  const size_t smem = (words > stage ? words : stage) * sizeof(uint32_t);
  static size_t configured = 0;
  if (smem > 48 * 1024 && smem > configured) {
    cudaError_t e = cudaFuncSetAttribute(select_tokens_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  select_tokens_kernel<<<m * Hkv, threads, smem, st>>>(win_score, kept, Hkv, L, n_cand, k, idx, cal);
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
