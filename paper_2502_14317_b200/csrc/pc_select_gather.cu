// Ranking and gather kernels: chunk top-m (Eq. 3-4), token top-k per kv-head (Eq. 7),
// compressed-cache gather (Eq. 7, Eq. 9), and the single-layer stand-in for the chunk
// self-information.  All HBM- or latency-bound; no tensor cores here on purpose.
#include "pc_kernels.h"
#include "pc_rank.cuh"

namespace pc {

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
  note_launch();
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

// Stand-in score and chunk top-m in ONE launch (C <= 64): four groups of 256 threads reduce the chunks' window
// log-sum-exp in the order of chunk_score_kernel (same bits), then the block ranks them.
__global__ void __launch_bounds__(1024) score_select_chunks_kernel(const float* __restrict__ win_lse, int n_per_chunk, int C,
                                                                   int m, int lower_is_better, float* __restrict__ score,
                                                                   int* __restrict__ kept) {
  __shared__ double part[4][256];
  __shared__ uint32_t key[64];
  __shared__ int flag[64];
  const int grp = threadIdx.x >> 8, t = threadIdx.x & 255;
  for (int c0 = 0; c0 < C; c0 += 4) {                        // the barriers inside are reached by every thread
    const int c = c0 + grp;
    double acc = 0.0;
    if (c < C)
      for (int i = t; i < n_per_chunk; i += 256) acc += (double)win_lse[(size_t)c * n_per_chunk + i];
    part[grp][t] = acc;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
      if (t < s) part[grp][t] += part[grp][t + s];
      __syncthreads();
    }
    if (t == 0 && c < C) {
      const float sc = (float)(-part[grp][0] / (double)n_per_chunk);
      score[c] = sc;
      key[c] = rank_key(sc, lower_is_better != 0);
    }
    __syncthreads();
  }
  const int i = threadIdx.x;
  int sel = 0;
  if (i < C) {
    const uint32_t mine = key[i];
    int rank = 0;
    for (int j = 0; j < C; ++j) rank += (key[j] > mine) || (key[j] == mine && j < i);
    sel = rank < m;
    flag[i] = sel;
  }
  __syncthreads();
  if (sel) {
    int pos = 0;
    for (int j = 0; j < i; ++j) pos += flag[j];
    kept[pos] = i;
  }
}

void launch_score_select_chunks(const float* win_lse, int C, int n_per_chunk, int m, int lower_is_better, float* score,
                                int* kept, cudaStream_t st) {
  if (C <= 64) {
    note_launch();
    score_select_chunks_kernel<<<1, 1024, 0, st>>>(win_lse, n_per_chunk, C, m, lower_is_better, score, kept);
  } else {
    launch_chunk_score(win_lse, C, n_per_chunk, score, st);
    launch_select_chunks(score, C, m, lower_is_better, kept, st);
  }
}

void launch_select_chunks(const float* score, int C, int m, int lower_is_better, int* kept, cudaStream_t st) {
  note_launch();
  select_chunks_kernel<<<1, 1024, 0, st>>>(score, C, m, lower_is_better, kept);
}

// ------------------------------------------------------------------ token top-k
// One CTA per (kept chunk, kv-head) row, 32 candidates per thread held in REGISTERS, no staging
// of the row in shared memory.
//   1. Warp w owns the 1024 positions [1024 w, 1024 w + 1024).  Lane l reads them as 8 coalesced
//      16-byte loads (chunk j = positions 1024 w + 128 j + 4 l + 0..3), turns every score into an
//      order-preserving uint32 key and transposes its 32 x 32 bit matrix in registers: word b then
//      holds bit b of all 32 keys (byte permutes for the 16- and 8-bit stages).
//   2. The k-th largest key T is found bit by bit, most significant first.  On the bit slices a
//      round is three instructions per thread (and, popc, redux), one count per warp in shared memory,
//      one barrier and one redux over the warps' counts, whatever the distribution of the scores (no
//      atomics, no histogram hot spots); the masks of the keys
//      > T and == T fall out.  The search stops as soon as every key still undecided belongs to
//      the top k (with distinct scores after about log2(n_cand) rounds past their common prefix).
//   3. One block scan over the per-chunk counts (eight counts packed in two words) gives every
//      thread the output rank of its kept positions, which are put in ascending order in shared memory
//      and written out coalesced (straight to the index row when k is too large to stage).  Only when the keys equal to T cannot all be kept does a second scan rank
//      them first (ties go to the lower position).
// HBM traffic: the row once (4 B per candidate) + 4 B per kept index.
constexpr int SEL_KPT = 32;                                    // keys per thread
constexpr int SEL_SPAN = 32 * SEL_KPT;                         // positions per warp
constexpr int SEL_MAX_THREADS = 1024;                          // n_cand <= 32768
constexpr int SEL_SMALL_CTAS = 5;                              // resident CTAs per SM asked for by the narrow variant

// Attention calibration (Eq. 8): a candidate whose score exceeds the threshold of its region (first n_s
// positions / last n_r positions / the rest) is evicted before the ranking.  +inf switches a region off.
struct SelCalib {
  int on, n_s, n_r;
  float lam_s, lam_m, lam_r;
};

// 4 nibbles of a 16-bit value -> 4 bytes
__device__ __forceinline__ uint32_t sel_spread_nibbles(uint32_t h) {
  const uint32_t t = (h | (h << 8)) & 0x00FF00FFu;
  return (t | (t << 4)) & 0x0F0F0F0Fu;
}

// Ranks in position order.  Bit 31 - i of x belongs to key i of the thread (chunk j = i / 4).  On return
// offs[j] is the number of set bits of the whole block at positions before this thread's chunk j; the
// return value is the number of set bits of the block.  Contains one block barrier.
__device__ __forceinline__ int sel_ordered_offsets(uint32_t x, int lane, int warp, int nwarps, int* s_tot,
                                                   int (&offs)[8]) {
  uint32_t n = x - ((x >> 1) & 0x55555555u);
  n = (n & 0x33333333u) + ((n >> 2) & 0x33333333u);            // per nibble: its population count
  const uint32_t own_hi = sel_spread_nibbles(n >> 16);         // byte 3 - j: chunk j (j < 4)
  const uint32_t own_lo = sel_spread_nibbles(n & 0xFFFFu);     // byte 7 - j: chunk j (j >= 4)
  uint32_t hi = own_hi, lo = own_lo;                           // inclusive scan over the lanes; a byte holds at most 128
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t a = __shfl_up_sync(0xFFFFFFFFu, hi, off), b = __shfl_up_sync(0xFFFFFFFFu, lo, off);
    if (lane >= off) { hi += a; lo += b; }
  }
  const uint32_t t_hi = __shfl_sync(0xFFFFFFFFu, hi, 31), t_lo = __shfl_sync(0xFFFFFFFFu, lo, 31);
  const uint32_t e_hi = hi - own_hi, e_lo = lo - own_lo;
  int run = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int sh = 8 * (3 - (j & 3));
    offs[j] = run + (int)(((j < 4 ? e_hi : e_lo) >> sh) & 0xFFu);
    run += (int)(((j < 4 ? t_hi : t_lo) >> sh) & 0xFFu);
  }
  if (lane == 0) s_tot[warp] = run;
  __syncthreads();
  const int v = lane < nwarps ? s_tot[lane] : 0;
  const int base = __reduce_add_sync(0xFFFFFFFFu, lane < warp ? v : 0);
  const int total = __reduce_add_sync(0xFFFFFFFFu, v);
#pragma unroll
  for (int j = 0; j < 8; ++j) offs[j] += base;
  return total;
}

// Copy of the kept rows by the block that ranked them (online chunk queue: a chunk that enters the queue is
// ranked and compacted in one launch; chunks that do not enter are not ranked at all).
struct SelGather {
  const uint4* k_src; const uint4* v_src;                      // [Cb,L,Hkv,d] through strides in 16-byte units
  long long s_chunk, s_tok, s_head;
  uint4* k_out; uint4* v_out; int* pos_out;                    // slot storage [Hkv, m*k, d] x 2, [Hkv, m*k]
  int lpr;                                                     // 16-byte pieces (= lanes) per row, d / 8
};

// STAGE: the kept positions are first put in order in shared memory (k words) and written out coalesced;
// otherwise (k too large for that) they are stored straight to the index row.
// SMALL: rows of at most 8192 candidates (256 threads), compiled for five CTAs per SM.
// GATHER (with STAGE): kept[r] is the batch chunk that moves into queue slot r (-1: the slot keeps its contents and
// the block returns); positions go to pos_out[hkv, r*k + t] and the rows k_src / v_src[kept[r], pos, hkv] to slot r.
template <bool CAL, bool STAGE, bool SMALL, bool GATHER = false>
__global__ void __launch_bounds__(SMALL ? 256 : SEL_MAX_THREADS, SMALL ? SEL_SMALL_CTAS : 1) select_tokens_kernel(const float* __restrict__ win_score,
                                                                        const int* __restrict__ kept, int Hkv, int L,
                                                                        int n_cand, int k, int* __restrict__ idx,
                                                                        const SelCalib cal, const SelGather ga = SelGather()) {
  extern __shared__ int sel_stage[];                           // STAGE: [min(k, n_cand)]
  __shared__ int s_part[2][32];                                // [round parity][warp]: undecided keys of the warp with the bit set
  __shared__ int s_tot[2][32];

  const int row = blockIdx.x;                                  // r * Hkv + hkv
  const int r = row / Hkv, hk = row % Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int n_slots = gridDim.x / Hkv;
  int* out = GATHER ? ga.pos_out + ((size_t)hk * n_slots + r) * k : idx + (size_t)row * k;
  if (GATHER && kept[r] < 0) return;                           // nothing moves into this slot

  if (!GATHER && !CAL && k >= n_cand) {                        // nothing to evict: identity, then -1 padding
    for (int j = tid; j < k; j += blockDim.x) out[j] = j < n_cand ? j : -1;
    return;
  }
  const int k_out = k;
  if (k > n_cand) k = n_cand;                                  // rank all candidates, pad the rest
  const int c = kept[r];
  const float* src = win_score + ((size_t)c * Hkv + hk) * L;

  // ---- 1. the row -> registers
  const int pbase = warp * SEL_SPAN + 4 * lane;
  const bool vec = (reinterpret_cast<uintptr_t>(src) & 15u) == 0;
  float val[SEL_KPT];
  uint32_t valid = 0u;                                         // bit 31 - i: key i is a candidate
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int p = pbase + 128 * j;
    if (vec && p + 3 < n_cand) {
      const float4 t = __ldg(reinterpret_cast<const float4*>(src + p));
      val[4 * j] = t.x; val[4 * j + 1] = t.y; val[4 * j + 2] = t.z; val[4 * j + 3] = t.w;
      valid |= 0xF0000000u >> (4 * j);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool in = p + e < n_cand;
        val[4 * j + e] = in ? __ldg(src + p + e) : 0.0f;
        if (in) valid |= 0x80000000u >> (4 * j + e);
      }
    }
  }

  // Keys.  The order-preserving image of a score with bit pattern u is u ^ 0x80000000 for u >= 0 and ~u for
  // u < 0; the exclusive-or is applied to the bit slices inside the search (one operand more of a logic
  // instruction there), so the registers keep u itself.  -0 ranks as +0 (the addition turns it into +0);
  // NaN ranks below every number (image 1 = pattern 0xFFFFFFFE); positions that are not candidates rank
  // below NaN (image 0 = pattern 0xFFFFFFFF) and are never emitted.
  uint32_t key[SEL_KPT];
  float nan_probe = 0.0f;                                      // NaN if any score is (or after inf - inf: checked exactly below)
#pragma unroll
  for (int i = 0; i < SEL_KPT; ++i) {
    const float f = __fadd_rn(val[i], 0.0f);
    nan_probe = __fadd_rn(nan_probe, f);
    key[i] = __float_as_uint(f);
    if (CAL) {
      const int p = pbase + 128 * (i >> 2) + (i & 3);
      const float lam = p < cal.n_s ? cal.lam_s : (p >= n_cand - cal.n_r ? cal.lam_r : cal.lam_m);
      if (val[i] > lam) valid &= ~(0x80000000u >> i);
    }
  }
  if (nan_probe != nan_probe) {                                // rare
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i)
      if ((key[i] & 0x7FFFFFFFu) > 0x7F800000u) key[i] = 0xFFFFFFFEu;
  }
  if (valid != 0xFFFFFFFFu) {
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i)
      if (!(valid & (0x80000000u >> i))) key[i] = 0xFFFFFFFFu;
  }

  // in-register transpose of the 32 x 32 bit matrix: afterwards key[31 - b] holds bit b of every
  // pattern, key i sitting at bit 31 - i
#pragma unroll
  for (int q = 0; q < 16; ++q) {                               // exchange 16-bit halves
    const uint32_t a = key[q], b = key[q + 16];
    key[q] = __byte_perm(a, b, 0x3276);                        // (a & 0xFFFF0000) | (b >> 16)
    key[q + 16] = __byte_perm(a, b, 0x1054);                   // (b & 0x0000FFFF) | (a << 16)
  }
#pragma unroll
  for (int q = 0; q < 32; ++q) {                               // exchange bytes
    if (q & 8) continue;
    const uint32_t a = key[q], b = key[q + 8];
    key[q] = __byte_perm(a, b, 0x3715);                        // (a & 0xFF00FF00) | ((b >> 8) & 0x00FF00FF)
    key[q + 8] = __byte_perm(a, b, 0x2604);                    // (b & 0x00FF00FF) | ((a << 8) & 0xFF00FF00)
  }
  {
    uint32_t m = 0x0F0F0F0Fu;
#pragma unroll
    for (int j = 4; j != 0; j >>= 1, m ^= (m << j)) {
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        if (q & j) continue;
        const uint32_t a = key[q], b = key[q + j];
        key[q] = (a & ~m) | ((b >> j) & m);
        key[q + j] = (b & m) | ((a << j) & ~m);
      }
    }
  }

  // ---- 2. k-th largest key, bit by bit.  active: keys equal to T on the bits decided so far (n_active of
  // them in the row, of which the `need` largest are kept); above: keys already known to be larger than T.
  uint32_t active = 0xFFFFFFFFu, above = 0u;
  int n_active = SEL_KPT * blockDim.x, need = k;
  const uint32_t neg = key[0];                                 // sign bits: the slices below bit 31 are inverted for these keys
#pragma unroll
  for (int bit = 31; bit >= 0; --bit) {
    if (n_active == need) break;                               // every undecided key is kept
    const uint32_t slice = bit == 31 ? ~neg : key[31 - bit] ^ neg;   // this bit of the order-preserving images
    const uint32_t ones = active & slice;
    const int cnt = __reduce_add_sync(0xFFFFFFFFu, __popc(ones));
    int* const part = s_part[bit & 1];                         // per-warp counts, double-buffered over the rounds
    if (lane == 0) part[warp] = cnt;
    __syncthreads();
    const int tot = __reduce_add_sync(0xFFFFFFFFu, lane < nwarps ? part[lane] : 0);   // undecided keys with this bit set
    const bool take = tot >= need;                             // the k-th largest has this bit
    above |= take ? 0u : ones;
    active = take ? ones : (active & ~slice);
    need -= take ? 0 : tot;
    n_active = take ? tot : n_active - tot;
  }

  // ---- 3. ordered emission
  uint32_t taken;
  if (n_active == need) {
    taken = (above | active) & valid;
  } else {
    // all 32 bits decided and more keys equal T than are needed: the lowest positions win.  (When T is 0
    // the keys equal to it are no candidates, and nothing more is taken.)
    const uint32_t eq = active & valid;
    int eq_before[8];
    sel_ordered_offsets(eq, lane, warp, nwarps, s_tot[1], eq_before);
    uint32_t pick = 0u;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) {
      const uint32_t sel_bit = 0x80000000u >> i;
      if (eq & sel_bit) {
        if (eq_before[i >> 2] < need) pick |= sel_bit;
        ++eq_before[i >> 2];
      }
    }
    taken = (above & valid) | pick;
  }
  int offs[8];
  const int n_emit = sel_ordered_offsets(taken, lane, warp, nwarps, s_tot[0], offs);
  if (STAGE) {
    const uint32_t stage_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(sel_stage));
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      uint32_t addr = stage_u32 + 4u * offs[j];
#pragma unroll
      for (int e = 0; e < 4; ++e) {                            // predicated store and advance: no branch per key
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %1, 0;\n\t@p st.shared.u32 [%0], %2;\n\t@p add.u32 %0, %0, 4;\n\t}"
            : "+r"(addr)
            : "r"(taken & (0x80000000u >> (4 * j + e))), "r"(pbase + 128 * j + e)
            : "memory");
      }
    }
    __syncthreads();
    for (int j = tid; j < k_out; j += blockDim.x) out[j] = j < n_emit ? sel_stage[j] : -1;
    if (GATHER) {                                              // rows of the kept positions, lpr lanes per row, K and V together
      const int rows_per_warp = 32 / ga.lpr, piece = lane % ga.lpr;
      for (int j0 = warp * rows_per_warp; j0 < k_out; j0 += nwarps * rows_per_warp) {
        const int j = j0 + lane / ga.lpr;
        if (j >= k_out) continue;
        const int pos = j < n_emit ? sel_stage[j] : -1;
        uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
        if (pos >= 0) {
          const long long off = (long long)c * ga.s_chunk + (long long)pos * ga.s_tok + (long long)hk * ga.s_head + piece;
          kv = __ldg(ga.k_src + off);
          vv = __ldg(ga.v_src + off);
        }
        const size_t dst = (((size_t)hk * n_slots + r) * k_out + j) * ga.lpr + piece;
        ga.k_out[dst] = kv;
        ga.v_out[dst] = vv;
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) {
      const bool t = (taken & (0x80000000u >> i)) != 0u;
      if (t) out[offs[i >> 2]] = pbase + 128 * (i >> 2) + (i & 3);
      offs[i >> 2] += t ? 1 : 0;
    }
    for (int j = n_emit + tid; j < k_out; j += blockDim.x) out[j] = -1;
  }
}

cudaError_t launch_select_tokens(const float* win_score, const int* kept, int m, int Hkv, int L, int n_cand, int k,
                                 int* idx, const SelCalibArgs* calib, cudaStream_t st) {
  int threads = (n_cand + SEL_SPAN - 1) / SEL_SPAN * 32;
  if (threads < 32) threads = 32;
  if (threads > SEL_MAX_THREADS) return cudaErrorInvalidValue;
  // region sizes beyond the row mean "the whole row": clamp them on the host (they are compared with positions)
  const SelCalib cal = calib ? SelCalib{1, calib->n_s < n_cand ? calib->n_s : n_cand, calib->n_r < n_cand ? calib->n_r : n_cand,
                                        calib->lam_s, calib->lam_m, calib->lam_r}
                             : SelCalib{0, 0, 0, 0.f, 0.f, 0.f};
  const size_t stage_bytes = sizeof(int) * (size_t)(k < n_cand ? k : n_cand);
  const bool stage = stage_bytes <= 40 * 1024;                 // within the default dynamic shared-memory limit
  const int grid = m * Hkv;
#define PC_SELECT(C, S)                                                                                               \
  do {                                                                                                                \
    note_launch();                                                                                                    \
    if (threads <= 256)                                                                                               \
      select_tokens_kernel<C, S, true><<<grid, threads, S ? stage_bytes : 0, st>>>(win_score, kept, Hkv, L, n_cand, k, \
                                                                                    idx, cal);                        \
    else                                                                                                              \
      select_tokens_kernel<C, S, false><<<grid, threads, S ? stage_bytes : 0, st>>>(win_score, kept, Hkv, L, n_cand,   \
                                                                                     k, idx, cal);                    \
  } while (0)
  if (calib) {
    if (stage) PC_SELECT(true, true); else PC_SELECT(true, false);
  } else {
    if (stage) PC_SELECT(false, true); else PC_SELECT(false, false);
  }
#undef PC_SELECT
  return cudaGetLastError();
}

// Ranking and compaction of the chunks that enter the online queue, one launch.  Returns cudaErrorNotSupported when
// the kept positions of a row do not fit the staging buffer (the caller then ranks and gathers in two launches).
cudaError_t launch_select_gather_slots(const float* win_score, const int* slot_src, int m, int Hkv, int L, int n_cand,
                                       int k, const void* k_src, const void* v_src, const long long stride_elems[3],
                                       int d, void* q_k, void* q_v, int* q_pos, cudaStream_t st) {
  int threads = (n_cand + SEL_SPAN - 1) / SEL_SPAN * 32;
  if (threads < 32) threads = 32;
  if (threads > SEL_MAX_THREADS) return cudaErrorInvalidValue;
  const size_t stage_bytes = sizeof(int) * (size_t)(k < n_cand ? k : n_cand);
  if (stage_bytes > 40 * 1024) return cudaErrorNotSupported;
  const SelCalib cal{0, 0, 0, 0.f, 0.f, 0.f};
  SelGather ga;
  ga.k_src = (const uint4*)k_src; ga.v_src = (const uint4*)v_src;
  ga.s_chunk = stride_elems[0] / 8; ga.s_tok = stride_elems[1] / 8; ga.s_head = stride_elems[2] / 8;
  ga.k_out = (uint4*)q_k; ga.v_out = (uint4*)q_v; ga.pos_out = q_pos;
  ga.lpr = d / 8;
  note_launch();
  if (threads <= 256)
    select_tokens_kernel<false, true, true, true><<<m * Hkv, threads, stage_bytes, st>>>(win_score, slot_src, Hkv, L, n_cand, k,
                                                                                        nullptr, cal, ga);
  else
    select_tokens_kernel<false, true, false, true><<<m * Hkv, threads, stage_bytes, st>>>(win_score, slot_src, Hkv, L, n_cand, k,
                                                                                         nullptr, cal, ga);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ gather
// One row of d bf16 (2d bytes) per (kv-head, slot); LPR lanes move one row with 16-byte
// accesses, K and V in the same thread so both copies are in flight together.
// BY_SLOT (online chunk queue): kept[r] is the chunk that moves into slot r of the output, or -1 for a slot
// that keeps its contents; the index rows are then those of the source chunk, idx[kept[r], hkv, :].
template <int D, bool BY_SLOT>
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
    const int c = kept[r];
    if (BY_SLOT && c < 0) continue;
    const int j = idx[((size_t)(BY_SLOT ? c : r) * Hkv + hk) * k + t];
    uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
    if (j >= 0) {
      const long long off = (long long)c * s_chunk + (long long)j * s_tok + (long long)hk * s_head + sub;
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
                             int sm_count, bool by_slot, cudaStream_t st) {
  const long long n_rows = (long long)Hkv * m * k;
  const int lpr = d / 8;
  long long want = (n_rows * lpr + 255) / 256;
  int blocks = (int)(want < (long long)sm_count * 8 ? want : (long long)sm_count * 8);
  if (blocks < 1) blocks = 1;
  const long long sc = stride_elems[0] / 8, stok = stride_elems[1] / 8, sh = stride_elems[2] / 8;
#define PC_GATHER(D, S)                                                                                              \
  gather_kv_kernel<D, S><<<blocks, 256, 0, st>>>((const uint4*)k_src, (const uint4*)v_src, sc, stok, sh, kept, idx, m, \
                                                 Hkv, k, (uint4*)k_out, (uint4*)v_out, pos_out)
  note_launch();
  if (d == 128) {
    if (by_slot) PC_GATHER(128, true); else PC_GATHER(128, false);
  } else {
    if (by_slot) PC_GATHER(64, true); else PC_GATHER(64, false);
  }
#undef PC_GATHER
  return cudaGetLastError();
}

// Append the w new (key, value) rows of every sequence behind the Nk valid entries of caches stored with
// room to grow: cache[b, hkv, Nk + i, :] = win[b, i, hkv, :].  One 16-byte piece per thread.
__global__ void append_kv_kernel(const uint4* __restrict__ k_win, const uint4* __restrict__ v_win, int B, int w, int Hkv,
                                 int lpr, long long Nk, long long Nk_cap, uint4* __restrict__ k_cache,
                                 uint4* __restrict__ v_cache) {
  const long long n = (long long)B * w * Hkv * lpr;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int piece = (int)(i % lpr);
    long long x = i / lpr;
    const int hkv = (int)(x % Hkv); x /= Hkv;
    const int t = (int)(x % w);
    const long long b = x / w;
    const long long dst = ((b * Hkv + hkv) * Nk_cap + Nk + t) * lpr + piece;
    k_cache[dst] = __ldg(k_win + i);
    v_cache[dst] = __ldg(v_win + i);
  }
}

cudaError_t launch_append_kv(const void* k_win, const void* v_win, int B, int w, int Hkv, int d, long long Nk,
                             long long Nk_cap, void* k_cache, void* v_cache, cudaStream_t st) {
  const int lpr = d / 8;
  const long long n = (long long)B * w * Hkv * lpr;
  const int blocks = (int)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184);
  note_launch();
  append_kv_kernel<<<blocks < 1 ? 1 : blocks, 256, 0, st>>>((const uint4*)k_win, (const uint4*)v_win, B, w, Hkv, lpr, Nk, Nk_cap,
                                                        (uint4*)k_cache, (uint4*)v_cache);
  return cudaGetLastError();
}

}  // namespace pc
