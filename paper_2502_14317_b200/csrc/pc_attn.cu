// Attention kernels for sm_100a: chunk-local causal attention with fused query-window
// scores (Eq. 1-2, Eq. 5-6) and parallel attention over the compressed cache (Eq. 9-11).
//
// One persistent CTA per SM, 12 warps in 3 warpgroups:
//   warps 0-3  softmax group 0   (one 128-row query block, thread = row = TMEM lane)
//   warps 4-7  softmax group 1   (a second 128-row block sharing the same K/V tiles)
//   warp  8    TMA producer      (Q tiles, K/V ring)
//   warp  9    tcgen05 issuer for block 0 (owns the TMEM allocation)
//   warp 10    tcgen05 issuer for block 1
//   warp 11    idle
// Two issuers, not one: a tcgen05.mma issue blocks while the tensor pipe is busy, and every
// barrier wait or commit between two batches costs the issuing thread ~100 cycles during
// which a single issuer lets the pipe run dry.  With one issuer per block the waits of one
// overlap the issue of the other.
// Per 128-key tile:  S_b = Q_b K^T  (SS MMA, fp32 in TMEM)  ->  softmax group b turns S_b
// into bf16 P_b in place in TMEM  ->  O_b += P_b V  (TS MMA, V as N-major smem operand).
// While group 0 runs its softmax the tensor core works for group 1 and vice versa.
// The running maximum is only raised when it grows by more than 2^8 (lazy rescale), so
// the accumulator is rarely touched between tiles.
// Queries and keys arrive rotated (the RoPE pre-pass of pc_rope.cu runs before these kernels).
// In the parallel attention an item whose rows fill one block only (a decoding step) is run by
// BOTH groups on alternate key tiles and merged afterwards, like two key splits.
//
// Window scores (prefill only): the item that owns the last query tiles of a
// (chunk, kv-head) group runs them for all G q-heads, keeps the window rows' final
// log-sum-exp in shared memory, then sweeps the keys once more computing the transposed
// product K_j Qw^T (keys on TMEM lanes, the G*w window rows on columns), so the column
// sum of Eq. 6 is a per-thread sum in a fixed order: deterministic, no atomics.
#include "pc_kernels.h"
#include "pc_attn.h"
#include "pc_sm100.cuh"


namespace pc {

namespace {

constexpr int TILE = 128;
constexpr int NUM_THREADS = 384;               // 3 warpgroups: softmax 0, softmax 1, {producer, two issuers, one idle warp}
constexpr int WARP_PRODUCER = 8;
constexpr int WARP_MMA = 9;                 // issuer of block 0; WARP_MMA + 1 issues block 1
constexpr int NS = 4;                       // K/V ring stages
constexpr float LAZY_RESCALE = 8.0f;        // log2 units
constexpr int ITEM_DONE = -1;

// where-codes stored in the status word when a wait gives up
enum { W_ITEM = 101, W_QFULL, W_QROT /* unused, keeps the later codes */, W_QFREE, W_KVFULL, W_KVFREE, W_SFULL, W_PFULL, W_OFULL, W_ACCFREE, W_TFULL, W_TFREE, W_TURN, W_PHALF };

struct __align__(16) Misc {
  uint64_t q_full[2], q_free[2];
  uint64_t kv_full[NS], kv_free[NS];
  uint64_t s_full[2], p_half[2], p_full[2], o_full[2], acc_free[2];
  uint64_t item_full[2], item_empty[2];
  uint64_t t_full[2], t_free[2];
  uint64_t turn[2];                        // issue token passed between the two tcgen05 issuers
  uint64_t mma_done;                       // every tensor-core operation of both issuers has completed (teardown)
  int item_slot[2];
  uint32_t tmem_base;
  int abort_flag;                          // these two words stay adjacent: bounded waits read the limit through the
  int wait_kcycles;                        // flag's address
  float lse2[1024];                        // window-row log-sum-exp (log2 domain), G * w <= 1024
  float xch[2][TILE];
};

template <int D>
struct Cfg {
  static constexpr int TILE_BYTES = TILE * D * 2;
  static constexpr int ATOMS = D / 64;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_RING = 2 * TILE_BYTES;
  static constexpr int OFF_MISC = OFF_RING + NS * TILE_BYTES;
  static constexpr int SMEM_BYTES = OFF_MISC + (int)sizeof(Misc) + 1024;   // + alignment slack
};

// One pair of 128-row query blocks that share K/V tiles.
struct SubItem {
  int hA, tA, hB, tB;        // q-head and query tile of block A / B; hB < 0: block B absent
};

// ------------------------------------------------------------------ item decoding (prefill)
// With per-chunk lengths the query tiles of a shorter chunk are numbered from the END: slot v of the static
// decomposition (v = T - 1 is the last tile of a full-length chunk) is tile v - (T - T_c) of a chunk with T_c
// tiles; slots below T - T_c are empty.  The window then always sits in the last two slots, which the tail item
// of the group owns together with the score sweep.
struct Sched {
  int T, t_w, ntt, G, P, hp_mode, ipg, n_lp;
  int wp, hb, Gs, n_pass;                    // score sweep: operand rows per head (w rounded up to 8), heads per 128-row
                                             // block, heads per pass, passes
};

// length of chunk c in tokens (window included), clamped to (w, L]
__device__ __forceinline__ int chunk_length(const PrefillParams& p, int c) {
  if (p.chunk_len == nullptr) return p.L;
  int len = __ldg(p.chunk_len + c);
  len = len > p.L ? p.L : len;
  return len <= p.w ? p.w + 1 : len;
}

__device__ __forceinline__ Sched make_sched(const PrefillParams& p) {
  Sched s;
  s.T = (p.L + TILE - 1) / TILE;
  s.G = p.Hq / p.Hkv;
  s.hp_mode = (s.G % 2 == 0);
  s.P = s.G / 2;
  s.wp = (p.w + 7) & ~7;
  s.hb = TILE / s.wp;
  s.Gs = 2 * s.hb < s.G ? 2 * s.hb : s.G;
  s.n_pass = (s.G + s.Gs - 1) / s.Gs;
  if (s.hp_mode) {
    // tail slots: the tiles that can hold window rows (two with per-chunk lengths: the window of some chunk may
    // straddle two tiles even where that of a full-length chunk does not)
    s.ntt = (p.chunk_len != nullptr) ? (p.w > 1 ? 2 : 1) : s.T - (p.L - p.w) / TILE;
    if (s.ntt > s.T) s.ntt = s.T;
    s.t_w = s.T - s.ntt;
    s.n_lp = 0;
    s.ipg = 1 + s.t_w * s.P;
  } else {
    s.ntt = s.T >= 2 ? 2 : 1;
    s.t_w = s.T - s.ntt;
    s.n_lp = (s.t_w + 1) / 2;                // tile pairs below the tail, from the top
    s.ipg = 1 + s.n_lp * s.G;
  }
  return s;
}

// score sweep: q-heads whose window rows sit in block b (0 / 1) of pass u
__device__ __forceinline__ int sweep_heads(const Sched& s, int u, int b) {
  const int heads = (s.G - u * s.Gs) < s.Gs ? (s.G - u * s.Gs) : s.Gs;
  const int first = heads < s.hb ? heads : s.hb;
  return b ? heads - first : first;
}

// number of sub-items of item `within` (0 = tail item of the group)
__device__ __forceinline__ int n_subitems(const Sched& s, int within) {
  if (within != 0) return 1;
  return s.hp_mode ? s.P * s.ntt : s.G;
}

// len: length of the sub-item's chunk.  Returns hA < 0 for an empty sub-item (every role skips it).
__device__ __forceinline__ SubItem decode_sub(const Sched& s, int hkv, int within, int sub, int len) {
  SubItem it;
  const int h0 = hkv * s.G;
  if (s.hp_mode) {
    int pair, tile;
    if (within == 0) { pair = sub / s.ntt; tile = s.T - 1 - (sub % s.ntt); }
    else { const int x = within - 1; tile = s.t_w - 1 - x / s.P; pair = x % s.P; }
    it.hA = h0 + 2 * pair; it.hB = it.hA + 1; it.tA = tile; it.tB = tile;
  } else {
    int g, hi;
    if (within == 0) { g = sub; hi = s.T - 1; }
    else { const int x = within - 1; g = x % s.G; hi = s.t_w - 1 - 2 * (x / s.G); }
    if (hi >= 1) { it.hA = h0 + g; it.tA = hi - 1; it.hB = h0 + g; it.tB = hi; }
    else { it.hA = h0 + g; it.tA = hi; it.hB = -1; it.tB = 0; }
  }
  const int shift = s.T - (len + TILE - 1) / TILE;          // empty slots of a shorter chunk
  if (shift > 0) {
    it.tA -= shift;
    it.tB -= shift;
    if (it.hB >= 0 && it.tB < 0) it.hB = -1;
    if (it.tA < 0) {
      if (it.hB >= 0 && s.hp_mode == 0) { it.tA = it.tB; it.hB = -1; it.tB = 0; }   // only the upper tile of the pair exists
      else { it.hA = -1; it.hB = -1; }
    }
  }
  return it;
}

// One arrival for a whole warp (an arrival per thread costs the barrier 32 serialised shared-memory operations).
__device__ __forceinline__ void warp_arrive(uint64_t* bar) {
  __syncwarp();
  if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

// ------------------------------------------------------------------ softmax of one tile (thread = row)
// Reads the 128 fp32 logits of this thread's row from TMEM, updates the running
// (m, l), rescales the accumulator when the maximum moved by more than 2^LAZY_RESCALE,
// and writes bf16 probabilities back over the logits.  `vis` = visible columns (<= 0: none).
// The first half of the probabilities (keys 0..63) is published on `p_half_bar` as soon as it
// is in TMEM, so that the first half of P V runs under the exponentials of the second half.
template <int D>
__device__ __forceinline__ void softmax_tile(uint32_t s_taddr, uint32_t o_taddr, int vis, bool first_tile,
                                             float scale_log2, float& m_used, float& l_run, uint64_t* p_half_bar) {
  uint32_t s[4][32];
#pragma unroll
  for (int q = 0; q < 4; ++q) tmem_ld32(s_taddr + q * 32, s[q]);
  tmem_wait_ld();
  if (vis < TILE) {
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (q * 32 + j >= vis) s[q][j] = 0xFF800000u;              // -inf
  }
  // row maximum: four independent chains of 3-input max
  float mq[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    float a = fmax3(__uint_as_float(s[q][0]), __uint_as_float(s[q][1]), __uint_as_float(s[q][2]));
#pragma unroll
    for (int j = 3; j < 31; j += 2) a = fmax3(a, __uint_as_float(s[q][j]), __uint_as_float(s[q][j + 1]));
    mq[q] = fmaxf(a, __uint_as_float(s[q][31]));
  }
  const float m_tile = fmaxf(fmaxf(mq[0], mq[1]), fmaxf(mq[2], mq[3])) * scale_log2;   // -inf if nothing visible
  float alpha = 1.0f;
  const bool raise = first_tile || (m_tile > m_used + LAZY_RESCALE);
  if (raise) {
    const float m_new = fmaxf(m_used, m_tile);
    alpha = (m_used == -INFINITY) ? 0.0f : fast_exp2(m_used - m_new);
    m_used = m_new;
  }
  if (!first_tile && __any_sync(0xFFFFFFFFu, raise)) {           // warp-uniform: each warp owns its 32 lanes of O
#pragma unroll 1
    for (int q = 0; q < D / 8; ++q) {                             // rare path: small chunks keep registers free
      uint32_t o[8];
      tmem_ld8(o_taddr + q * 8, o);
      tmem_wait_ld();
#pragma unroll
      for (int j = 0; j < 8; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
      tmem_st8(o_taddr + q * 8, o);
    }
  }
  const float neg_m = (m_used == -INFINITY) ? 0.0f : -m_used;     // fully masked row so far: exp2(-inf) = 0
  const uint64_t scale2 = pack_f32x2(scale_log2, scale_log2), negm2 = pack_f32x2(neg_m, neg_m);
  uint64_t sum2[2] = {0ull, 0ull};                                // four partial row sums (two packed pairs)
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint32_t packed[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(s[q][2 * j]), __uint_as_float(s[q][2 * j + 1])), scale2, negm2);
      float x0, x1, p0, p1;
      unpack_f32x2(x2, x0, x1);
      p0 = fast_exp2(x0);                                         // MUFU pipe
      p1 = fast_exp2(x1);
      sum2[j & 1] = add_f32x2(sum2[j & 1], pack_f32x2(p0, p1));
      packed[j] = pack_bf16x2(p0, p1);
    }
    tmem_st16(s_taddr + q * 16, packed);                          // P aliases the first 64 columns of S
    if (q == 1) {                                                 // keys 0..63 of P are final: the issuer may start P V on them
      tmem_wait_st();
      tc_fence_before_sync();
      warp_arrive(p_half_bar);
    }
  }
  float a0, a1, a2, a3;
  unpack_f32x2(sum2[0], a0, a1);
  unpack_f32x2(sum2[1], a2, a3);
  l_run = l_run * alpha + ((a0 + a1) + (a2 + a3));
  tmem_wait_st();
}

// ------------------------------------------------------------------ tensor-core issue helpers (one thread)
template <int D>
__device__ __forceinline__ void issue_qk(uint32_t d_tmem, uint32_t q_smem, uint32_t k_smem, int n_cols) {
  const uint32_t idesc = make_idesc_bf16_f32(TILE, n_cols, false, false);
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    const uint32_t off = (ks / 4) * 16384 + (ks % 4) * 32;
    mma_ss(d_tmem, make_smem_desc_sw128(q_smem + off, 16, 1024), make_smem_desc_sw128(k_smem + off, 16, 1024), idesc,
           ks > 0);
  }
}
// transposed product for the score sweep: D[keys, rows] = K_tile * Qw^T
template <int D>
__device__ __forceinline__ void issue_kq(uint32_t d_tmem, uint32_t k_smem, uint32_t q_smem, int n_cols) {
  issue_qk<D>(d_tmem, k_smem, q_smem, n_cols);
}
// k-steps [ks0, ks1) of O += P V (16 keys per step)
template <int D>
__device__ __forceinline__ void issue_pv(uint32_t o_tmem, uint32_t p_tmem, uint32_t v_smem, bool accumulate, int ks0,
                                         int ks1) {
  constexpr uint32_t idesc = make_idesc_bf16_f32(TILE, D, false, true);
#pragma unroll
  for (int ks = ks0; ks < ks1; ++ks) {
    mma_ts(o_tmem, p_tmem + ks * 8, make_smem_desc_sw128(v_smem + ks * 2048, 16384, 1024), idesc,
           accumulate || ks > 0);
  }
}

// ------------------------------------------------------------------ per-role state
struct Waits {                                 // how many times each barrier has been used by this role
  uint32_t q[2] = {0, 0};                      // q_full / q_free (one use per block load)
  uint32_t kv = 0;                             // ring position (monotone)
  uint32_t s[2] = {0, 0}, p[2] = {0, 0}, o[2] = {0, 0}, acc[2] = {0, 0};   // p counts p_half and p_full alike
  uint32_t t[2] = {0, 0};
  uint32_t turn = 0;                           // batches issued so far by this issuer
  uint32_t item = 0;
};
__device__ __forceinline__ uint32_t full_par(uint32_t n) { return n & 1u; }          // n-th use of a "full" barrier
__device__ __forceinline__ uint32_t free_par(uint32_t n) { return (n & 1u) ^ 1u; }   // before the n-th use of a resource

// ------------------------------------------------------------------ shared pieces of the three roles
struct Ctx {
  Misc* mi;
  uint8_t* sQ[2];
  uint8_t* ring;
  uint32_t tmem;
  volatile int* abort_flag;
  int* status;
};

__device__ __forceinline__ void init_barriers(Misc& mi, int wait_kcycles) {
#pragma unroll
  for (int b = 0; b < 2; ++b) {
    mbar_init(&mi.q_full[b], 1); mbar_init(&mi.q_free[b], 1);
    mbar_init(&mi.s_full[b], 1); mbar_init(&mi.p_half[b], 4); mbar_init(&mi.p_full[b], 4); mbar_init(&mi.o_full[b], 1);
    mbar_init(&mi.acc_free[b], 4);
    mbar_init(&mi.item_full[b], 1); mbar_init(&mi.item_empty[b], 10);      // 8 softmax warps + 2 issuer threads
    mbar_init(&mi.t_full[b], 2); mbar_init(&mi.t_free[b], 8);
    mbar_init(&mi.turn[b], 1);
  }
  for (int s = 0; s < NS; ++s) { mbar_init(&mi.kv_full[s], 1); mbar_init(&mi.kv_free[s], 2); }   // both issuers release a stage
  mbar_init(&mi.mma_done, 2);
  mi.abort_flag = 0;
  mi.wait_kcycles = wait_kcycles;
  fence_mbar_init();
}

// producer: publish the next work item (dynamic queue); returns it
// skip_final: test hook - the "no more work" message is written but never signalled, so that the consumers' wait for
// it runs out.  Nothing is in flight at that point: every copy has been consumed and every accumulator read out.
__device__ __forceinline__ int producer_next_item(const Ctx& cx, Waits& wt, int* counter, int n_items, bool skip_final = false) {
  Misc& mi = *cx.mi;
  const int slot = wt.item & 1;
  mbar_wait(&mi.item_empty[slot], free_par(wt.item >> 1), cx.abort_flag, cx.status, W_ITEM);
  int item = atomicAdd(counter, 1);
  if (item >= n_items || *cx.abort_flag) item = ITEM_DONE;
  mi.item_slot[slot] = item;
  if (!(skip_final && item == ITEM_DONE)) mbar_arrive(&mi.item_full[slot]);
  ++wt.item;
  return item;
}
// consumers: read the next work item
// whole_warp: called by all 32 threads of a softmax warp (one arrival for the warp); else by a single issuer thread
__device__ __forceinline__ int consumer_next_item(const Ctx& cx, Waits& wt, bool whole_warp) {
  Misc& mi = *cx.mi;
  const int slot = wt.item & 1;
  if (!mbar_wait(&mi.item_full[slot], full_par(wt.item >> 1), cx.abort_flag, cx.status, W_ITEM)) return ITEM_DONE;   // aborted: stop
  const int item = mi.item_slot[slot];
  if (whole_warp) warp_arrive(&mi.item_empty[slot]); else mbar_arrive(&mi.item_empty[slot]);
  ++wt.item;
  return item;
}

// producer: one 128 x D tile into the next ring stage; (c1, c2, c3) are the outer TMA coordinates
template <int D>
__device__ __forceinline__ void producer_ring_tile(const Ctx& cx, Waits& wt, const CUtensorMap* tmap, int c1, int c2,
                                                   int c3) {
  using C = Cfg<D>;
  Misc& mi = *cx.mi;
  if (*cx.abort_flag) return;                  // a wait has run out: no copy is issued into a ring that nobody drains
  const int st = wt.kv % NS;
  if (!mbar_wait(&mi.kv_free[st], free_par(wt.kv / NS), cx.abort_flag, cx.status, W_KVFREE)) return;
  mbar_arrive_expect_tx(&mi.kv_full[st], C::TILE_BYTES);
  for (int a = 0; a < C::ATOMS; ++a)
    tma_load_4d(cx.ring + st * C::TILE_BYTES + a * 16384, tmap, &mi.kv_full[st], a * 64, c1, c2, c3);
  ++wt.kv;
}

// producer: before exit, every copy it issued must have landed
__device__ __forceinline__ void producer_drain(const Ctx& cx, const Waits& wt) {
  Misc& mi = *cx.mi;
  for (uint32_t i = (wt.kv > NS ? wt.kv - NS : 0); i < wt.kv; ++i) mbar_wait_drain(&mi.kv_full[i % NS], full_par(i / NS), cx.abort_flag);
#pragma unroll
  for (int b = 0; b < 2; ++b)
    if (wt.q[b] > 0) mbar_wait_drain(&mi.q_full[b], full_par(wt.q[b] - 1), cx.abort_flag);
}

// The two issuers take turns: the tensor pipe then runs the batch of one block to its end
// before the other block's batch, which keeps the two softmax groups half a period apart
// (while one group computes, the pipe works for the other).  Issuer 0 goes first.
__device__ __forceinline__ void turn_take(const Ctx& cx, Waits& wt, int b) {
  Misc& mi = *cx.mi;
  mbar_wait(&mi.turn[b], b == 0 ? free_par(wt.turn) : full_par(wt.turn), cx.abort_flag, cx.status, W_TURN);
}
__device__ __forceinline__ void turn_pass(const Ctx& cx, Waits& wt, int b) {
  mbar_arrive(&cx.mi->turn[b ^ 1]);
  ++wt.turn;
}

// issuer of block b: the flash loop over the n K/V tiles of the ring (order K0, V0, K1, V1, ...).
// Block b takes part in its first nb_b tiles - or, with `alternate` (the two blocks hold the SAME query rows and
// share the key tiles of the item between them), in the tiles of parity b.  The issuer of an absent or shorter block
// still walks the ring, takes its turns and releases the stages it does not use, so that both issuers arrive once
// on every kv_free barrier and the token keeps alternating.
template <int D>
__device__ __forceinline__ void mma_flash_block(const Ctx& cx, Waits& wt, int b, bool has_b, int nb_b, int n,
                                                bool alternate = false) {
  using C = Cfg<D>;
  Misc& mi = *cx.mi;
  const uint32_t ring_u32 = smem_u32(cx.ring);
  const uint32_t q_u32 = smem_u32(cx.sQ[b]);
  const uint32_t tS = cx.tmem + b * 128, tO = cx.tmem + 256 + b * 128;
  auto takes_part = [&](int j) { return has_b && j < n && (alternate ? ((j & 1) == b) : (j < nb_b)); };
  const int last = alternate ? (((n - 1) & 1) == b ? n - 1 : n - 2) : nb_b - 1;     // last tile of this block
  if (has_b) {
    // accumulator and score buffers of earlier work must have been read out
    mbar_wait(&mi.acc_free[b], free_par(wt.acc[b]), cx.abort_flag, cx.status, W_ACCFREE);
#pragma unroll
    for (int e = 0; e < 2; ++e) mbar_wait(&mi.t_free[e], free_par(wt.t[e]), cx.abort_flag, cx.status, W_TFREE);
    // the query block (rotated by the pre-pass, in global memory) is ready as soon as its copy has landed
    mbar_wait(&mi.q_full[b], full_par(wt.q[b]), cx.abort_flag, cx.status, W_QFULL);
    ++wt.q[b];
  }
  {  // S(0)
    const int st = wt.kv % NS;
    mbar_wait(&mi.kv_full[st], full_par(wt.kv / NS), cx.abort_flag, cx.status, W_KVFULL);
    ++wt.kv;
    turn_take(cx, wt, b);
    if (takes_part(0)) {
      tc_fence_after_sync();
      issue_qk<D>(tS, q_u32, ring_u32 + st * C::TILE_BYTES, TILE);
      mma_commit(&mi.s_full[b]);
      turn_pass(cx, wt, b);
      mma_commit(&mi.kv_free[st]);
    } else {
      turn_pass(cx, wt, b);
      mbar_arrive(&mi.kv_free[st]);
    }
  }
  bool first = true;                           // no P V of this block issued yet: the first one overwrites the accumulator
  for (int j = 0; j < n; ++j) {
    const int st_v = wt.kv % NS;
    mbar_wait(&mi.kv_full[st_v], full_par(wt.kv / NS), cx.abort_flag, cx.status, W_KVFULL);
    ++wt.kv;
    int st_k = 0;
    const bool more = j + 1 < n;
    if (more) {
      st_k = wt.kv % NS;
      mbar_wait(&mi.kv_full[st_k], full_par(wt.kv / NS), cx.abort_flag, cx.status, W_KVFULL);
      ++wt.kv;
    }
    const bool pv_now = takes_part(j), qk_next = takes_part(j + 1);
    if (pv_now || qk_next) {
      if (pv_now) {
        // first half of P V as soon as keys 0..63 of P are in TMEM (no token: it is not on the
        // other block's critical path for long, and the pipe is in order)
        mbar_wait(&mi.p_half[b], full_par(wt.p[b]), cx.abort_flag, cx.status, W_PHALF);
        tc_fence_after_sync();
        issue_pv<D>(tO, tS, ring_u32 + st_v * C::TILE_BYTES, !first, 0, TILE / 32);
        mbar_wait(&mi.p_full[b], full_par(wt.p[b]), cx.abort_flag, cx.status, W_PFULL);
        ++wt.p[b];
      }
      turn_take(cx, wt, b);
      tc_fence_after_sync();
      if (pv_now) {
        issue_pv<D>(tO, tS, ring_u32 + st_v * C::TILE_BYTES, true, TILE / 32, TILE / 16);
        first = false;
        if (j == last) mma_commit(&mi.o_full[b]);
      }
      // S of this block's next tile overwrites S / P of its previous one: the pipe runs the P V above first
      if (qk_next) { issue_qk<D>(tS, q_u32, ring_u32 + st_k * C::TILE_BYTES, TILE); mma_commit(&mi.s_full[b]); }
      turn_pass(cx, wt, b);
      mma_commit(&mi.kv_free[st_v]);
      if (more) mma_commit(&mi.kv_free[st_k]);
    } else {                                   // stages this block never reads
      turn_take(cx, wt, b);
      turn_pass(cx, wt, b);
      mbar_arrive(&mi.kv_free[st_v]);
      if (more) mbar_arrive(&mi.kv_free[st_k]);
    }
  }
  if (has_b) ++wt.acc[b];
}

// softmax group: online softmax over the key tiles of this block (all n, or with `alternate` those of parity b)
// for this thread's row; vis(j) = visible columns of tile j.  Leaves (m_used, l_run); the accumulator O_b stays
// in TMEM.
template <int D, class VisFn>
__device__ __forceinline__ void wg_flash_loop(const Ctx& cx, uint32_t& n_s, uint32_t& n_o, int b, uint32_t tS,
                                              uint32_t tO, int n, float scale_log2, VisFn vis, float& m_used,
                                              float& l_run, bool alternate = false) {
  Misc& mi = *cx.mi;
  m_used = -INFINITY;
  l_run = 0.0f;
  const int j0 = alternate ? b : 0, step = alternate ? 2 : 1;
  for (int j = j0; j < n; j += step) {
    mbar_wait(&mi.s_full[b], full_par(n_s), cx.abort_flag, cx.status, W_SFULL);
    ++n_s;
    tc_fence_after_sync();
    softmax_tile<D>(tS, tO, vis(j), j == j0, scale_log2, m_used, l_run, &mi.p_half[b]);
    tc_fence_before_sync();
    warp_arrive(&mi.p_full[b]);
  }
  mbar_wait(&mi.o_full[b], full_par(n_o), cx.abort_flag, cx.status, W_OFULL);
  ++n_o;
  tc_fence_after_sync();
}

}  // namespace

// ====================================================================================
//                                   PREFILL KERNEL
// ====================================================================================
template <int D>
__global__ void __launch_bounds__(NUM_THREADS, 1)
prefill_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                    const __grid_constant__ CUtensorMap tm_qw, const __grid_constant__ PrefillParams prm) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  Misc& mi = *reinterpret_cast<Misc*>(smem + C::OFF_MISC);
  Ctx cx;
  cx.mi = &mi;
  cx.sQ[0] = smem + C::OFF_Q;
  cx.sQ[1] = smem + C::OFF_Q + C::TILE_BYTES;
  cx.ring = smem + C::OFF_RING;
  cx.abort_flag = &mi.abort_flag;
  cx.status = prm.status;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const Sched sch = make_sched(prm);
  const int n_items = prm.C * prm.Hkv * sch.ipg;
  const int n_pass = sch.n_pass;

  if (tid == 0) init_barriers(mi, prm.wait_kcycles);
  if (warp == WARP_MMA) tmem_alloc(&mi.tmem_base, 512);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  cx.tmem = mi.tmem_base;

  Waits wt;

  if (warp == WARP_PRODUCER) {
    // ================================================================ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); tma_prefetch_desc(&tm_qw);
      while (true) {
        const int item = producer_next_item(cx, wt, prm.counter, n_items, prm.skip_final_publication != 0);
        if (item == ITEM_DONE) break;
        const int group = item / sch.ipg, within = item % sch.ipg;
        const int c = group / prm.Hkv, hkv = group % prm.Hkv;
        const int nsub = n_subitems(sch, within);
        const int len = chunk_length(prm, c);
        const int T_c = (len + TILE - 1) / TILE;
        for (int sub = 0; sub < nsub; ++sub) {
          const SubItem it = decode_sub(sch, hkv, within, sub, len);
          if (it.hA < 0) continue;
#pragma unroll
          for (int b = 0; b < 2; ++b) {
            const int h = b ? it.hB : it.hA, t = b ? it.tB : it.tA;
            if (h < 0) continue;
            mbar_wait(&mi.q_free[b], free_par(wt.q[b]), cx.abort_flag, cx.status, W_QFREE);
            mbar_arrive_expect_tx(&mi.q_full[b], C::TILE_BYTES);
            for (int a = 0; a < C::ATOMS; ++a)
              tma_load_4d(cx.sQ[b] + a * 16384, &tm_q, &mi.q_full[b], a * 64, h, t * TILE, c);
            ++wt.q[b];
          }
          const int n = (it.hB >= 0 ? it.tB : it.tA) + 1;
          for (int j = 0; j < n; ++j) {
            producer_ring_tile<D>(cx, wt, &tm_k, hkv, j * TILE, c);
            producer_ring_tile<D>(cx, wt, &tm_v, hkv, j * TILE, c);
          }
        }
        if (within == 0) {
          // ---- score sweep: window queries of Gs heads per pass, then all key tiles.  A head's rows in the operand
          // are the wp tokens that end with the chunk (wp = w rounded up to 8: the first wp - w of them are not
          // window rows and are left out of the sums; a start before token 0 reads zeros)
          for (int u = 0; u < n_pass; ++u) {
#pragma unroll
            for (int b = 0; b < 2; ++b) {
              const int heads_b = sweep_heads(sch, u, b);
              if (heads_b == 0) continue;
              mbar_wait(&mi.q_free[b], free_par(wt.q[b]), cx.abort_flag, cx.status, W_QFREE);
              mbar_arrive_expect_tx(&mi.q_full[b], heads_b * sch.wp * D * 2);
              for (int ih = 0; ih < heads_b; ++ih) {
                const int g = u * sch.Gs + b * sch.hb + ih;
                for (int a = 0; a < C::ATOMS; ++a)
                  tma_load_4d(cx.sQ[b] + a * 16384 + ih * sch.wp * 128, &tm_qw, &mi.q_full[b], a * 64, hkv * sch.G + g,
                              len - sch.wp, c);
              }
              ++wt.q[b];
            }
            for (int j = 0; j < T_c; ++j) producer_ring_tile<D>(cx, wt, &tm_k, hkv, j * TILE, c);
          }
        }
      }
      producer_drain(cx, wt);
    }
    __syncwarp();
  } else if (warp == WARP_MMA || warp == WARP_MMA + 1) {
    // ================================================================ tcgen05 issuers (one per block)
    if (lane == 0) {
      const int b = warp - WARP_MMA;
      const uint32_t ring_u32 = smem_u32(cx.ring);
      const uint32_t q_u32 = smem_u32(cx.sQ[b]);
      while (true) {
        const int item = consumer_next_item(cx, wt, false);
        if (item == ITEM_DONE) break;
        const int group = item / sch.ipg, within = item % sch.ipg;
        const int hkv = group % prm.Hkv;
        const int nsub = n_subitems(sch, within);
        const int len = chunk_length(prm, group / prm.Hkv);
        const int T_c = (len + TILE - 1) / TILE;
        for (int sub = 0; sub < nsub; ++sub) {
          const SubItem it = decode_sub(sch, hkv, within, sub, len);
          if (it.hA < 0) continue;
          const bool has_b = (b == 0) || it.hB >= 0;
          const int nb_b = (b == 0) ? it.tA + 1 : (it.hB >= 0 ? it.tB + 1 : 0);
          const int n = (it.hB >= 0 ? it.tB : it.tA) + 1;
          mma_flash_block<D>(cx, wt, b, has_b, nb_b, n);
        }
        if (within == 0) {
          // ---- score sweep: this issuer computes the columns of its own block (window rows b*128..)
          mbar_wait(&mi.acc_free[b], free_par(wt.acc[b]), cx.abort_flag, cx.status, W_ACCFREE);
          for (int u = 0; u < n_pass; ++u) {
            const int rows_b = sweep_heads(sch, u, b) * sch.wp;
            if (rows_b > 0) { mbar_wait(&mi.q_full[b], full_par(wt.q[b]), cx.abort_flag, cx.status, W_QROT); ++wt.q[b]; }
            for (int j = 0; j < T_c; ++j) {
              const int e = j & 1;
              mbar_wait(&mi.t_free[e], free_par(wt.t[e]), cx.abort_flag, cx.status, W_TFREE);
              const int st = wt.kv % NS;
              mbar_wait(&mi.kv_full[st], full_par(wt.kv / NS), cx.abort_flag, cx.status, W_KVFULL);
              ++wt.kv;
              if (rows_b > 0) {
                tc_fence_after_sync();
                issue_kq<D>(cx.tmem + e * 256 + b * 128, ring_u32 + st * C::TILE_BYTES, q_u32, (rows_b + 15) & ~15);
                mma_commit(&mi.t_full[e]);
                mma_commit(&mi.kv_free[st]);
              } else {
                mbar_arrive(&mi.t_full[e]);
                mbar_arrive(&mi.kv_free[st]);
              }
              ++wt.t[e];
            }
          }
        }
      }
      mma_commit(&mi.mma_done);                              // teardown waits for everything this thread issued
    }
    __syncwarp();
  } else if (warp < 8) {
    // ================================================================ softmax groups
    const int b = warp >> 2;                                 // block / group index
    const int r = tid & 127;                                 // row in the block = TMEM lane
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = cx.tmem + b * 128 + lane_sel, tO = cx.tmem + 256 + b * 128 + lane_sel;
    const float scale_log2 = prm.scale_log2;
    uint8_t* const myQ = b ? cx.sQ[1] : cx.sQ[0];
    uint32_t n_s = 0, n_o = 0, n_t0 = 0, n_t1 = 0;            // barrier use counts of this group
    while (true) {
      const int item = consumer_next_item(cx, wt, true);
      if (item == ITEM_DONE) break;
      const int group = item / sch.ipg, within = item % sch.ipg;
      const int c = group / prm.Hkv, hkv = group % prm.Hkv;
      const int nsub = n_subitems(sch, within);
      const int len = chunk_length(prm, c);
      const int T_c = (len + TILE - 1) / TILE;
      for (int sub = 0; sub < nsub; ++sub) {
        const SubItem it = decode_sub(sch, hkv, within, sub, len);
        const int h = b ? it.hB : it.hA, t = b ? it.tB : it.tA;
        if (h < 0) continue;
        const int token = t * TILE + r;
        // ---- main loop over key tiles (causal: keys <= token; only the diagonal tile is masked)
        float m_used, l_run;
        const int n = t + 1;
        wg_flash_loop<D>(cx, n_s, n_o, b, tS, tO, n, scale_log2,
                         [&](int j) { return (j == n - 1) ? (token - j * TILE + 1) : TILE; }, m_used, l_run);
        // ---- epilogue: normalise, stage bf16 rows in the (now idle) Q buffer, TMA store
        const float inv_l = 1.0f / l_run;
        const bool in_chunk = token < len;                   // rows behind the end of the chunk are written as zeros
#pragma unroll
        for (int q = 0; q < D / 32; ++q) {
          uint32_t o[32];
          tmem_ld32(tO + q * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int g4 = 0; g4 < 4; ++g4) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              pk[e] = in_chunk ? pack_bf16x2(__uint_as_float(o[g4 * 8 + 2 * e]) * inv_l, __uint_as_float(o[g4 * 8 + 2 * e + 1]) * inv_l) : 0u;
            const int col = q * 32 + g4 * 8;
            *reinterpret_cast<uint4*>(myQ + (col / 64) * 16384 + sw128_offset(r, (col % 64) / 8)) =
                make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
        tc_fence_before_sync();
        warp_arrive(&mi.acc_free[b]);
        const float lse2 = m_used + log2f(l_run);
        if (in_chunk) {
          if (prm.lse) prm.lse[((size_t)c * prm.Hq + h) * prm.L + token] = lse2 * 0.6931471805599453f;
          const int wi = token - (len - prm.w);
          if (wi >= 0) {
            prm.win_lse[((size_t)c * prm.Hq + h) * prm.w + wi] = lse2 * 0.6931471805599453f;
            if (within == 0) mi.lse2[(h - hkv * sch.G) * prm.w + wi] = lse2;
          }
        }
        fence_proxy_async_smem();
        named_barrier_sync(1 + b, 128);
        if (r == 0) {
          for (int a = 0; a < C::ATOMS; ++a) tma_store_4d(&tm_o, myQ + a * 16384, a * 64, h, t * TILE, c);
          tma_store_commit();
          tma_store_wait_read();
          mbar_arrive(&mi.q_free[b]);
        }
      }
      if (within == 0) {
        // ---- score sweep: this thread owns key (j * 128 + r); columns are the window rows
        named_barrier_sync(3, 256);                           // lse2 complete and visible to both groups
        const int w0 = len - prm.w;                           // first window token of this chunk
        for (int u = 0; u < n_pass; ++u) {
          const int heads_b = sweep_heads(sch, u, b);          // heads whose rows sit in this group's columns
          const int rows_b = heads_b * sch.wp;
          const float* lse_rows = mi.lse2 + (u * sch.Gs + b * sch.hb) * prm.w;   // log-sum-exp of this group's first head
          for (int j = 0; j < T_c; ++j) {
            const int e = j & 1;
            mbar_wait(&mi.t_full[e], full_par(e ? n_t1 : n_t0), cx.abort_flag, cx.status, W_TFULL);
            if (e) ++n_t1; else ++n_t0;
            tc_fence_after_sync();
            const int key = j * TILE + r;
            const bool need_mask = (j * TILE + TILE - 1) > w0;
            float part = 0.0f;
            const uint32_t tT = cx.tmem + e * 256 + b * 128 + lane_sel;
            for (int ih = 0; ih < heads_b; ++ih) {             // a head has wp columns, the last w of them are window rows
              for (int col = 0; col < sch.wp; col += 8) {
                uint32_t sv[8];
                tmem_ld8(tT + ih * sch.wp + col, sv);
                tmem_wait_ld();
                const int wi0 = col - (sch.wp - prm.w);        // window row of the first of these columns (negative: none)
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) {
                  const int wi = wi0 + jj;
                  float pv = fast_exp2(fmaf(__uint_as_float(sv[jj]), scale_log2, -lse_rows[ih * prm.w + (wi < 0 ? 0 : wi)]));
                  if (wi < 0 || (need_mask && key > w0 + wi)) pv = 0.0f;
                  part += pv;
                }
              }
            }
            tc_fence_before_sync();
            warp_arrive(&mi.t_free[e]);
            if (b == 1) mi.xch[e][r] = part;
            named_barrier_sync(3, 256);
            if (b == 0 && key < len) {
              float* dst = prm.win_score + ((size_t)c * prm.Hkv + hkv) * prm.L + key;
              const float total = part + mi.xch[e][r];
              *dst = (u == 0) ? total : (*dst + total);
            }
          }
          if (rows_b > 0) {
            named_barrier_sync(1 + b, 128);                   // every thread of the group is past its last use of sQ[b]
            if (r == 0) mbar_arrive(&mi.q_free[b]);
          }
        }
      }
    }
    if (r == 0) tma_store_wait_all();
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == WARP_MMA) {
    // no tensor-core operation may still be running when its accumulators are freed: both issuers ended with a
    // commit to mma_done.  Immediate in a clean run; after an abort this is what makes the exit safe (the wait
    // ignores the abort flag and is bounded).
    mbar_wait_drain(&mi.mma_done, 0, cx.abort_flag);
    tc_fence_after_sync();
    tmem_dealloc(cx.tmem, 512);
  }
}

// ====================================================================================
//                          PARALLEL (GLOBAL) ATTENTION KERNEL
// ====================================================================================
// Queries arrive rotated (RoPE pre-pass).  Item = (sequence, kv-head, row group, key split).
// When the rows of an item fill one block only (G * w <= 128, e.g. a decoding step), both blocks hold those
// rows and take alternate key tiles, each with its own running maximum, sum and accumulator: two softmax
// streams per CTA instead of one, merged afterwards like two key splits.  The rows of an item are the w window
// queries of up to 256/w q-heads of one kv-head, packed head-major into the two 128-row
// blocks; both blocks stream the same cache tiles, and the last split appends the
// window's own keys (causal inside the window).
template <int D>
__global__ void __launch_bounds__(NUM_THREADS, 1)
parallel_attn_kernel(const __grid_constant__ CUtensorMap tm_qw, const __grid_constant__ CUtensorMap tm_kc,
                     const __grid_constant__ CUtensorMap tm_vc, const __grid_constant__ CUtensorMap tm_kw,
                     const __grid_constant__ CUtensorMap tm_vw, const __grid_constant__ ParallelParams prm) {
  using C = Cfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  Misc& mi = *reinterpret_cast<Misc*>(smem + C::OFF_MISC);
  Ctx cx;
  cx.mi = &mi;
  cx.sQ[0] = smem + C::OFF_Q;
  cx.sQ[1] = smem + C::OFF_Q + C::TILE_BYTES;
  cx.ring = smem + C::OFF_RING;
  cx.abort_flag = &mi.abort_flag;
  cx.status = prm.status;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = prm.Hq / prm.Hkv;
  const int n_items = prm.B * prm.Hkv * prm.n_rg * prm.n_split;

  if (tid == 0) init_barriers(mi, prm.wait_kcycles);
  if (warp == WARP_MMA) tmem_alloc(&mi.tmem_base, 512);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  cx.tmem = mi.tmem_base;

  Waits wt;

  // item -> (seq, hkv, rg, split) and its tile range / row counts
  struct Dec { int seq, hkv, g0, split, rows[2], j0, n_cache, n; };
  auto decode = [&](int item) {
    Dec d;
    d.split = item % prm.n_split;
    int x = item / prm.n_split;
    const int rg = x % prm.n_rg; x /= prm.n_rg;
    d.hkv = x % prm.Hkv;
    d.seq = x / prm.Hkv;
    d.g0 = rg * prm.Gs;
    const int heads = (G - d.g0) < prm.Gs ? (G - d.g0) : prm.Gs;
    const int rows_total = heads * prm.w;
    d.rows[0] = rows_total < TILE ? rows_total : TILE;
    d.rows[1] = rows_total > TILE ? rows_total - TILE : 0;
    if (prm.alt) d.rows[1] = d.rows[0];           // one block of rows: both blocks hold it and share the key tiles
    d.j0 = d.split * prm.tiles_per_split;
    const int j1 = (d.j0 + prm.tiles_per_split) < prm.n_cache_tiles ? (d.j0 + prm.tiles_per_split) : prm.n_cache_tiles;
    d.n_cache = j1 - d.j0;
    d.n = d.n_cache + (d.split == prm.n_split - 1 ? 1 : 0);
    return d;
  };

  if (warp == WARP_PRODUCER) {
    if (lane == 0) {
      tma_prefetch_desc(&tm_qw); tma_prefetch_desc(&tm_kc); tma_prefetch_desc(&tm_vc);
      while (true) {
        const int item = producer_next_item(cx, wt, prm.counter, n_items);
        if (item == ITEM_DONE) break;
        const Dec d = decode(item);
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          if (d.rows[b] == 0) continue;
          mbar_wait(&mi.q_free[b], free_par(wt.q[b]), cx.abort_flag, cx.status, W_QFREE);
          mbar_arrive_expect_tx(&mi.q_full[b], d.rows[b] * D * 2);
          for (int r0 = 0; r0 < d.rows[b]; r0 += prm.w) {
            const int g = d.g0 + ((prm.alt ? 0 : b * TILE) + r0) / prm.w;
            for (int a = 0; a < C::ATOMS; ++a)
              tma_load_4d(cx.sQ[b] + a * 16384 + r0 * 128, &tm_qw, &mi.q_full[b], a * 64, d.hkv * G + g, 0, d.seq);
          }
          ++wt.q[b];
        }
        for (int jj = 0; jj < d.n; ++jj) {
          if (jj < d.n_cache) {
            producer_ring_tile<D>(cx, wt, &tm_kc, (d.j0 + jj) * TILE, d.hkv, d.seq);
            producer_ring_tile<D>(cx, wt, &tm_vc, (d.j0 + jj) * TILE, d.hkv, d.seq);
          } else {
            producer_ring_tile<D>(cx, wt, &tm_kw, d.hkv, 0, d.seq);
            producer_ring_tile<D>(cx, wt, &tm_vw, d.hkv, 0, d.seq);
          }
        }
      }
      producer_drain(cx, wt);
    }
    __syncwarp();
  } else if (warp == WARP_MMA || warp == WARP_MMA + 1) {
    if (lane == 0) {
      const int b = warp - WARP_MMA;
      while (true) {
        const int item = consumer_next_item(cx, wt, false);
        if (item == ITEM_DONE) break;
        const Dec d = decode(item);
        const bool has_b = d.rows[b] > 0;
        mma_flash_block<D>(cx, wt, b, has_b, has_b ? d.n : 0, d.n, prm.alt != 0);
      }
      mma_commit(&mi.mma_done);
    }
    __syncwarp();
  } else if (warp < 8) {
    const int b = warp >> 2;
    const int r = tid & 127;
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = cx.tmem + b * 128 + lane_sel, tO = cx.tmem + 256 + b * 128 + lane_sel;
    uint32_t n_s = 0, n_o = 0;
    const int wi = r % prm.w;                                 // window index of this row (128 % w == 0)
    while (true) {
      const int item = consumer_next_item(cx, wt, true);
      if (item == ITEM_DONE) break;
      const Dec d = decode(item);
      const int rows_b = b ? d.rows[1] : d.rows[0];
      if (rows_b == 0) continue;
      float m_used, l_run;
      wg_flash_loop<D>(cx, n_s, n_o, b, tS, tO, d.n, prm.scale_log2,
                       [&](int jj) {
                         if (jj >= d.n_cache) return wi + 1;                       // window tile: causal
                         const int left = prm.Nk - (d.j0 + jj) * TILE;             // ragged last cache tile
                         return left < TILE ? left : TILE;
                       },
                       m_used, l_run, prm.alt != 0);
      if (r == 0) mbar_arrive(&mi.q_free[b]);                 // all MMAs that read sQ[b] have completed
      const int g = d.g0 + ((prm.alt ? 0 : b * TILE) + r) / prm.w;
      const int h = d.hkv * G + g;
      const bool valid = r < rows_b;
      if (prm.n_part == 1) {
        const float inv_l = 1.0f / l_run;
        uint4* dst = reinterpret_cast<uint4*>(prm.out + (((size_t)d.seq * prm.w + wi) * prm.Hq + h) * D);
#pragma unroll
        for (int q = 0; q < D / 32; ++q) {
          uint32_t o[32];
          tmem_ld32(tO + q * 32, o);
          tmem_wait_ld();
          if (valid) {
#pragma unroll
            for (int g4 = 0; g4 < 4; ++g4) {
              uint32_t pk[4];
#pragma unroll
              for (int e = 0; e < 4; ++e)
                pk[e] = pack_bf16x2(__uint_as_float(o[g4 * 8 + 2 * e]) * inv_l, __uint_as_float(o[g4 * 8 + 2 * e + 1]) * inv_l);
              dst[q * 4 + g4] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
          }
        }
        if (valid && prm.lse_out)
          prm.lse_out[((size_t)d.seq * prm.Hq + h) * prm.w + wi] = (m_used + log2f(l_run)) * 0.6931471805599453f;
      } else {
        const int part = prm.alt ? 2 * d.split + b : d.split;   // partial result of this block
        const size_t prow = (((size_t)d.seq * prm.Hq + h) * prm.n_part + part) * prm.w + wi;
        uint4* dst = reinterpret_cast<uint4*>(prm.part_o + prow * D);
#pragma unroll
        for (int q = 0; q < D / 32; ++q) {
          uint32_t o[32];
          tmem_ld32(tO + q * 32, o);
          tmem_wait_ld();
          if (valid) {
#pragma unroll
            for (int g4 = 0; g4 < 8; ++g4) dst[q * 8 + g4] = make_uint4(o[g4 * 4], o[g4 * 4 + 1], o[g4 * 4 + 2], o[g4 * 4 + 3]);
          }
        }
        if (valid) reinterpret_cast<float2*>(prm.part_ml)[prow] = make_float2(m_used, l_run);
      }
      tc_fence_before_sync();
      warp_arrive(&mi.acc_free[b]);
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == WARP_MMA) {
    // no tensor-core operation may still be running when its accumulators are freed: both issuers ended with a
    // commit to mma_done.  Immediate in a clean run; after an abort this is what makes the exit safe (the wait
    // ignores the abort flag and is bounded).
    mbar_wait_drain(&mi.mma_done, 0, cx.abort_flag);
    tc_fence_after_sync();
    tmem_dealloc(cx.tmem, 512);
  }
}

// Merge of the key splits: out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s.  One warp per output row.
template <int D>
__global__ void __launch_bounds__(256) parallel_merge_kernel(const float* __restrict__ part_o,
                                                             const float* __restrict__ part_ml, int n_rows_bh, int w,
                                                             int Hq, int n_split, __nv_bfloat16* __restrict__ out,
                                                             float* __restrict__ lse_out) {
  const int row = blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5);      // (seq * Hq + h) * w + i
  const int lane = threadIdx.x & 31;
  if (row >= n_rows_bh * w) return;
  const int bh = row / w, i = row % w;
  const int seq = bh / Hq, h = bh % Hq;
  float M = -INFINITY;
  for (int s = 0; s < n_split; ++s) M = fmaxf(M, part_ml[(((size_t)bh * n_split + s) * w + i) * 2]);
  float denom = 0.0f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < n_split; ++s) {
    const size_t prow = ((size_t)bh * n_split + s) * w + i;
    const float wgt = exp2f(part_ml[prow * 2] - M);
    denom += wgt * part_ml[prow * 2 + 1];
    if (lane < D / 4) {
      const float4 o = reinterpret_cast<const float4*>(part_o + prow * D)[lane];
      acc.x += wgt * o.x; acc.y += wgt * o.y; acc.z += wgt * o.z; acc.w += wgt * o.w;
    }
  }
  const float inv = 1.0f / denom;
  if (lane < D / 4) {
    uint2 pk;
    pk.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    pk.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    reinterpret_cast<uint2*>(out + (((size_t)seq * w + i) * Hq + h) * D)[lane] = pk;
  }
  if (lane == 0 && lse_out) lse_out[(size_t)bh * w + i] = (M + log2f(denom)) * 0.6931471805599453f;
}

// ====================================================================================
//                                   host launchers
// ====================================================================================
template <int D>
static cudaError_t launch_prefill_t(const CUtensorMap* maps, const PrefillParams& prm, int grid, cudaStream_t st) {
  // the opt-in to large dynamic shared memory is a per-device attribute of the function: set it on every call
  // (a host-side call of a few hundred nanoseconds) rather than remember which devices have it
  if (cudaError_t e = cudaFuncSetAttribute(prefill_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Cfg<D>::SMEM_BYTES); e != cudaSuccess) return e;
  note_launch();
  prefill_attn_kernel<D><<<grid, NUM_THREADS, Cfg<D>::SMEM_BYTES, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], prm);
  return cudaGetLastError();
}

cudaError_t launch_prefill_attn(const CUtensorMap* maps, const PrefillParams& prm, int d, int grid, cudaStream_t st) {
  return d == 128 ? launch_prefill_t<128>(maps, prm, grid, st) : launch_prefill_t<64>(maps, prm, grid, st);
}

template <int D>
static cudaError_t launch_parallel_t(const CUtensorMap* maps, const ParallelParams& prm, int grid, cudaStream_t st) {
  // the opt-in to large dynamic shared memory is a per-device attribute of the function: set it on every call
  // (a host-side call of a few hundred nanoseconds) rather than remember which devices have it
  if (cudaError_t e = cudaFuncSetAttribute(parallel_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Cfg<D>::SMEM_BYTES); e != cudaSuccess) return e;
  note_launch();
  parallel_attn_kernel<D><<<grid, NUM_THREADS, Cfg<D>::SMEM_BYTES, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], prm);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (prm.n_part > 1) {
    const int rows = prm.B * prm.Hq * prm.w;
    note_launch();
    parallel_merge_kernel<D><<<(rows + 7) / 8, 256, 0, st>>>(prm.part_o, prm.part_ml, prm.B * prm.Hq, prm.w, prm.Hq,
                                                            prm.n_part, prm.out, prm.lse_out);
    e = cudaGetLastError();
  }
  return e;
}

cudaError_t launch_parallel_attn(const CUtensorMap* maps, const ParallelParams& prm, int d, int grid, cudaStream_t st) {
  return d == 128 ? launch_parallel_t<128>(maps, prm, grid, st) : launch_parallel_t<64>(maps, prm, grid, st);
}

}  // namespace pc
