// Chunk-local causal attention with fused query-window scores (Eq. 1-2, Eq. 5-6) for head
// size 128 on CTA pairs.
//
// Two CTAs of a cluster work as one unit (tcgen05 cta_group::2).  Each CTA owns ONE 128-row
// query block; the two blocks of a pair read the same K/V (two q-heads of one kv-head at the
// same query tile, or two adjacent query tiles of one head), so every 128-key tile is split
// between the two shared memories: each CTA stages 64 keys of K and 64 head-dim columns of V
// and the tensor cores of both SMs read both halves.  That halves the shared-memory traffic
// per MMA, which is what limits a single CTA with two blocks at this head size.
//
// Per CTA, TMEM holds two S buffers (one per softmax warpgroup, 128 columns each), two P buffers
// (64 columns of bf16 each) and one accumulator (128 columns).  Two softmax warpgroups take
// alternate key tiles (thread = query row), chained only through the short per-row decision on the
// running maximum.  As soon as a warpgroup has S(j) in registers, Q K^T of its next tile S(j+2)
// may run into the same buffer, so that S is waiting when the warpgroup comes back; P(j) goes to
// the warpgroup's P buffer once P V of its previous tile has run.
//
// Warps (12 per CTA): 0-3 softmax of even tiles, 4-7 softmax of odd tiles (both: epilogue and score
// sweep split by halves),
// 8 TMA producer, 9 issuer of Q K^T, 10 and 11 issuers of P V for even / odd tiles (issuers run in
// the leader CTA only).  Several issuers because a tcgen05.mma issue blocks while the pipe is busy
// and every barrier wait or commit of an issuing thread costs it about a hundred cycles.
//
// Window scores: the pair that runs the last query tiles of a (chunk, kv-head) group keeps the
// window rows' log-sum-exp in both shared memories, then sweeps the keys once more with the
// transposed product K_j Qw^T (each CTA takes every other key tile; keys on TMEM lanes, window
// rows on columns), so Eq. 6 is a per-thread sum in a fixed order: deterministic, fp32, no atomics.
#include "pc_kernels.h"
#include "pc_attn.h"
#include "pc_sm100.cuh"

namespace pc {

namespace {

constexpr int TILE = 128;
constexpr int D = 128;
constexpr int NT2 = 384;                     // threads per CTA
constexpr int WARP_PRODUCER = 8, WARP_QK = 9, WARP_PV = 10;
constexpr int NKS = 4, NVS = 4;              // K / V ring stages (16 KB each)
constexpr int NSB = 2;                       // S buffers in TMEM (one per warpgroup); P has buffers of its own
constexpr uint32_t TM_P = 256;               // two P buffers of 64 columns (128 bf16 keys each), one per warpgroup
constexpr int HALF_BYTES = 16384;            // 64 keys x 128 d of K, or 128 keys x 64 d of V
constexpr int Q_BYTES = 32768;
constexpr uint32_t TM_O = 384;               // accumulator columns
constexpr float LAZY_RESCALE = 8.0f;         // log2 units

enum { W2_QFULL = 201, W2_QFREE, W2_KFULL, W2_KFREE, W2_VFULL, W2_VFREE, W2_SFULL, W2_PA, W2_PB,
       W2_PVDONE, W2_OFULL, W2_ACCFREE, W2_LSE, W2_TFULL, W2_TFREE, W2_MPUB, W2_TURN };

struct __align__(16) Misc2 {
  uint64_t q_full[2], q_free[2];             // q_full: leader only, counts the bytes of both CTAs' query tiles
  uint64_t k_full[NKS], k_free[NKS], v_full[NVS], v_free[NVS];
  uint64_t s_full[2][NSB];                   // [owning warpgroup][buffer]: a waiter must see every phase of its barrier
  uint64_t p_a[2][NSB], p_b[2][NSB];         // [owning warpgroup = P V issuer][buffer]
  uint64_t s_read[NSB];                      // leader only: S of the tile in this buffer is in registers (8 warps of the pair)
  uint64_t pv_turn[2];                       // leader only: issue token of the two P V issuers
  uint64_t o_full, acc_free, lse_ready;
  uint64_t t_full[2], t_free[2];
  uint64_t m_pub[2][4];                      // [owner warpgroup][warp]: its reference maxima of a tile are in mref
  uint64_t mma_done;                         // every tensor-core operation of the three issuers has completed (teardown)
  uint32_t tmem_base;
  int abort_flag;                            // the two words after tmem_base stay adjacent: bounded waits read the limit
  int wait_kcycles;                          // through the flag's address
  float lse2[1024];                          // window-row log-sum-exp (log2 units) of all G heads, G * w <= 1024
  float mref[2][TILE];                       // [tile parity][row]: reference maximum (log2 units) after that tile
  float xl[2][TILE];                         // [key half][row]: half-row sums
  float xs[2][2][TILE];                      // [buffer][column half][key]: partial window scores
};

constexpr int OFF_Q = 0;
constexpr int OFF_RK = 2 * Q_BYTES;
constexpr int OFF_RV = OFF_RK + NKS * HALF_BYTES;
constexpr int OFF_MISC = OFF_RV + NVS * HALF_BYTES;
constexpr int SMEM2_BYTES = OFF_MISC + (int)sizeof(Misc2) + 1024;

__device__ __forceinline__ uint32_t full_par(uint32_t n) { return n & 1u; }           // n-th completion of a barrier
__device__ __forceinline__ uint32_t free_par(uint32_t n) { return (n & 1u) ^ 1u; }    // completion n-1 (passes for n = 0)

// ------------------------------------------------------------------ work decomposition
// Groups = (chunk, kv-head); the items of a group are ordered heaviest first; item 0 of a
// group (the tail item) holds the query tiles with window rows for all G heads, then the sweep.
// The two CTAs of a pair take the same query tile of two q-heads of the kv-head, so G must be even (an odd
// group size would leave a pair with two different query tiles of one head, one of them walking a masked
// key tile; such shapes run on the single-CTA kernel instead).
// Division of n < 2^31 by a fixed divisor as a multiplication (round-up method with a 32-bit multiplier).
struct FastDiv {
  uint32_t d, mul, shr;
  __device__ __forceinline__ void init(uint32_t div) {
    d = div;
    uint32_t l = 0;
    while ((1u << l) < div) ++l;                           // ceil(log2(div))
    shr = 31u + l;
    mul = static_cast<uint32_t>(((1ull << shr) + div - 1) / div);
  }
  __device__ __forceinline__ int quot(int n) const {
    return static_cast<int>((static_cast<uint64_t>(static_cast<uint32_t>(n)) * mul) >> shr);
  }
  __device__ __forceinline__ void divmod(int n, int& q, int& r) const {
    q = quot(n);
    r = n - q * static_cast<int>(d);
  }
};

// With per-chunk lengths the query tiles of a shorter chunk are numbered from the END: slot v of the static
// decomposition (v = T - 1 is the last tile of a full-length chunk) is tile v - (T - T_c) of a chunk with T_c tiles,
// and slots below T - T_c are empty.  The window then always sits in the last one or two slots, which the tail item
// of the group owns together with the score sweep.
struct Sched2 {
  int T, t_w, ntt, G, P, ipg, hp, n_pass, wp;
  FastDiv d_ipg, d_hkv, d_ntt, d_P;
};
__device__ __forceinline__ Sched2 make_sched2(const PrefillParams& p) {
  Sched2 s;
  s.T = (p.L + TILE - 1) / TILE;
  s.G = p.Hq / p.Hkv;
  s.P = s.G / 2;
  // slots of the tail item: the tiles that can hold window rows (with per-chunk lengths the window of some chunk
  // may straddle two tiles even where that of a full-length chunk does not)
  s.ntt = (p.chunk_len != nullptr) ? (p.w > 1 ? 2 : 1) : s.T - (p.L - p.w) / TILE;
  if (s.ntt > s.T) s.ntt = s.T;
  s.t_w = s.T - s.ntt;
  s.ipg = 1 + s.t_w * s.P;
  s.wp = (p.w + 7) & ~7;                                  // window rows of a head in the sweep operand (multiple of 8)
  const int cap = TILE / s.wp, want = s.G / 2;
  s.hp = cap < want ? cap : want;                         // window heads per CTA and sweep pass
  s.n_pass = (s.G + 2 * s.hp - 1) / (2 * s.hp);
  s.d_ipg.init(s.ipg); s.d_hkv.init(p.Hkv); s.d_ntt.init(s.ntt); s.d_P.init(s.P);
  return s;
}
__device__ __forceinline__ int n_subitems2(const Sched2& s, int within) {
  if (within != 0) return 1;
  return s.P * s.ntt;
}
struct Blk {
  int h;       // q-head of this CTA's block
  int t;       // query tile of this CTA's block
  int n;       // key tiles the pair walks
};
// length of chunk c in tokens (window included), clamped to (w, L]
__device__ __forceinline__ int chunk_length(const PrefillParams& p, int c) {
  if (p.chunk_len == nullptr) return p.L;
  int len = __ldg(p.chunk_len + c);
  len = len > p.L ? p.L : len;
  return len <= p.w ? p.w + 1 : len;
}
// len: length of the block's chunk.  b.n == 0: an empty slot, every role skips the block.
__device__ __forceinline__ Blk decode_blk(const Sched2& s, int rank, int hkv, int within, int sub, int len) {
  Blk b;
  const int h0 = hkv * s.G;
  int pair, tile;
  if (within == 0) { int rem; s.d_ntt.divmod(sub, pair, rem); tile = s.T - 1 - rem; }
  else { int q; s.d_P.divmod(within - 1, q, pair); tile = s.t_w - 1 - q; }
  tile -= s.T - (len + TILE - 1) / TILE;
  b.h = h0 + 2 * pair + rank;
  b.t = tile;
  b.n = tile < 0 ? 0 : tile + 1;
  return b;
}

struct Ctx2 {
  Misc2* mi;
  uint8_t* sQ[2];
  uint8_t* rK;
  uint8_t* rV;
  uint32_t tmem;
  uint32_t rank;
  volatile int* abort_flag;
  int* status;
};

// waits of the single-thread service roles (long pause between polls) / of the softmax warps
#define WAIT2(bar, par, code) mbar_wait_ns<SERVICE_BACKOFF_NS>((bar), (par), cx.abort_flag, cx.status, (code))
#define WAIT2S(bar, par, code) mbar_wait((bar), (par), cx.abort_flag, cx.status, (code))

// wait whose completion also makes the peer CTA's earlier shared-memory writes visible
__device__ __forceinline__ void mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status,
                                                  int where) {
  if (mbar_try_wait_cluster(bar, parity)) return;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait_cluster(bar, parity)) {
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return;
      if (clock64() - t0 > (static_cast<long long>(abort_flag[1]) << 10)) {
        *abort_flag = 1;
        if (status) atomicCAS(status, 0, where);
        return;
      }
    }
  }
}

__device__ __forceinline__ void init_barriers2(Misc2& mi, int wait_kcycles) {
  for (int b = 0; b < 2; ++b) {
    mbar_init(&mi.q_full[b], 1); mbar_init(&mi.q_free[b], 1);
    mbar_init(&mi.t_full[b], 1); mbar_init(&mi.t_free[b], 16);
  }
  for (int s = 0; s < NKS; ++s) { mbar_init(&mi.k_full[s], 1); mbar_init(&mi.k_free[s], 1); }
  for (int s = 0; s < NVS; ++s) { mbar_init(&mi.v_full[s], 1); mbar_init(&mi.v_free[s], 1); }
  for (int s = 0; s < NSB; ++s) {
    mbar_init(&mi.s_full[0][s], 1); mbar_init(&mi.s_full[1][s], 1); mbar_init(&mi.s_read[s], 8);
    for (int g = 0; g < 2; ++g) { mbar_init(&mi.p_a[g][s], 8); mbar_init(&mi.p_b[g][s], 8); }   // 4 warps of the owning warpgroup in each CTA
  }
  mbar_init(&mi.pv_turn[0], 1); mbar_init(&mi.pv_turn[1], 1);
  mbar_init(&mi.o_full, 1); mbar_init(&mi.acc_free, 16); mbar_init(&mi.lse_ready, 16);
  for (int w = 0; w < 4; ++w) { mbar_init(&mi.m_pub[0][w], 1); mbar_init(&mi.m_pub[1][w], 1); }   // warp to warp (same rows)
  mbar_init(&mi.mma_done, 3);
  mi.abort_flag = 0;
  mi.wait_kcycles = wait_kcycles;
  fence_mbar_init();
}

}  // namespace

// ====================================================================================
//                                   KERNEL
// ====================================================================================
// tensor maps: tm_q (box 64 d x 128 tokens), tm_kh (rotated keys, box 64 d x 64 tokens),
// tm_k (rotated keys, box 64 d x 128 tokens), tm_v (box 64 d x 128 tokens), tm_o (store,
// box 64 d x 128 tokens), tm_qw (box 64 d x w tokens)
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NT2, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kh,
                    const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    const __grid_constant__ CUtensorMap tm_o, const __grid_constant__ CUtensorMap tm_qw,
                    const __grid_constant__ PrefillParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  Misc2& mi = *reinterpret_cast<Misc2*>(smem + OFF_MISC);
  Ctx2 cx;
  cx.mi = &mi;
  cx.sQ[0] = smem + OFF_Q;
  cx.sQ[1] = smem + OFF_Q + Q_BYTES;
  cx.rK = smem + OFF_RK;
  cx.rV = smem + OFF_RV;
  cx.abort_flag = &mi.abort_flag;
  cx.status = prm.status;
  cx.rank = cluster_ctarank();

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cx.rank;
  const bool leader = (rank == 0);
  const Sched2 sch = make_sched2(prm);
  const int n_items = prm.C * prm.Hkv * sch.ipg;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int rows_half = sch.hp * sch.wp;                 // sweep operand rows per CTA and pass (B operand half)

  if (tid == 0) init_barriers2(mi, prm.wait_kcycles);
  if (warp == WARP_QK) tmem_alloc_pair(&mi.tmem_base, 512);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                    // both CTAs' barriers exist before any remote arrive
  tc_fence_after_sync();
  cx.tmem = mi.tmem_base;

  if (warp == WARP_PRODUCER) {
    // ================================================================ TMA producer (both CTAs)
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_kh); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v);
      tma_prefetch_desc(&tm_qw);
      uint32_t cQ = 0, cK = 0, cV = 0;
      // Once a wait has run out (abort flag) no new work is started: every role leaves its loops at the next item,
      // this one also at the next tile, so that no copy is issued into a ring that nobody drains any more.
      for (int item = pair_id; item < n_items && !*cx.abort_flag; item += n_pairs) {
        int group, within, c, hkv;
        sch.d_ipg.divmod(item, group, within);
        sch.d_hkv.divmod(group, c, hkv);
        const int nsub = n_subitems2(sch, within);
        const int len = chunk_length(prm, c);
        for (int sub = 0; sub < nsub; ++sub) {
          const Blk bk = decode_blk(sch, rank, hkv, within, sub, len);
          if (bk.n == 0) continue;
          {
            const int qb = cQ & 1;
            WAIT2(&mi.q_free[qb], free_par(cQ >> 1), W2_QFREE);
            if (leader) mbar_arrive_expect_tx(&mi.q_full[qb], 2 * Q_BYTES);
            const uint32_t bar = map_to_cta(&mi.q_full[qb], 0);
            for (int a = 0; a < 2; ++a) tma_load_4d_pair(cx.sQ[qb] + a * 16384, &tm_q, bar, a * 64, bk.h, bk.t * TILE, c);
            ++cQ;
          }
          for (int j = 0; j < bk.n && !*cx.abort_flag; ++j) {
            {
              const int s = cK % NKS;
              WAIT2(&mi.k_free[s], free_par(cK / NKS), W2_KFREE);
              if (leader) mbar_arrive_expect_tx(&mi.k_full[s], 2 * HALF_BYTES);
              const uint32_t bar = map_to_cta(&mi.k_full[s], 0);
              for (int a = 0; a < 2; ++a)
                tma_load_4d_pair(cx.rK + s * HALF_BYTES + a * 8192, &tm_kh, bar, a * 64, hkv, j * TILE + (int)rank * 64, c);
              ++cK;
            }
            {
              const int s = cV % NVS;
              WAIT2(&mi.v_free[s], free_par(cV / NVS), W2_VFREE);
              if (leader) mbar_arrive_expect_tx(&mi.v_full[s], 2 * HALF_BYTES);
              tma_load_4d_pair(cx.rV + s * HALF_BYTES, &tm_v, map_to_cta(&mi.v_full[s], 0), (int)rank * 64, hkv, j * TILE, c);
              ++cV;
            }
          }
        }
        if (within == 0) {
          // ---- score sweep: window queries of hp heads per CTA and pass, then this CTA's key tiles.  A head's rows
          // in the operand are the wp tokens that end with the chunk (wp = w rounded up to 8: the first wp - w rows
          // are not window rows and are left out of the sums; a start before token 0 reads zeros)
          const int n_sweep_tiles = ((len + TILE - 1) / TILE + 1) / 2;
          for (int u = 0; u < sch.n_pass; ++u) {
            const int qb = cQ & 1;
            WAIT2(&mi.q_free[qb], free_par(cQ >> 1), W2_QFREE);
            if (leader) mbar_arrive_expect_tx(&mi.q_full[qb], 2 * rows_half * D * 2);
            const uint32_t bar = map_to_cta(&mi.q_full[qb], 0);
            for (int i = 0; i < sch.hp; ++i) {
              int g = u * 2 * sch.hp + (int)rank * sch.hp + i;
              if (g >= sch.G) g = sch.G - 1;              // filler rows: loaded, never summed
              for (int a = 0; a < 2; ++a)
                tma_load_4d_pair(cx.sQ[qb] + a * 16384 + i * sch.wp * 128, &tm_qw, bar, a * 64, hkv * sch.G + g,
                                 len - sch.wp, c);
            }
            ++cQ;
            if (cK & 1) {                                 // a full key tile takes an even-aligned pair of stages
              const int s = cK % NKS;
              WAIT2(&mi.k_free[s], free_par(cK / NKS), W2_KFREE);
              if (leader) mbar_arrive(&mi.k_full[s]);
              ++cK;
            }
            for (int jj = 0; jj < n_sweep_tiles && !*cx.abort_flag; ++jj) {
              const int tile = 2 * jj + (int)rank;
              for (int a = 0; a < 2; ++a) {
                const int s = cK % NKS;
                WAIT2(&mi.k_free[s], free_par(cK / NKS), W2_KFREE);
                if (leader) mbar_arrive_expect_tx(&mi.k_full[s], 2 * HALF_BYTES);
                tma_load_4d_pair(cx.rK + s * HALF_BYTES, &tm_k, map_to_cta(&mi.k_full[s], 0), a * 64, hkv, tile * TILE, c);
                ++cK;
              }
            }
          }
        }
      }
      // Every copy issued must have landed before a CTA may exit.  In a run without a timed-out wait that follows
      // from the last uses of the rings having been consumed (the teardown below waits for every tensor-core
      // operation).  After an abort nothing is consumed any more: the leader, whose barriers count the bytes of both
      // CTAs' copies, waits on them (ignoring the abort flag, bounded); the peer cannot observe the completion of
      // its own last copies and lets a fixed pause pass that outlasts any copy in flight.
      if (*cx.abort_flag) {
        if (leader) {
          for (uint32_t i = (cK > NKS ? cK - NKS : 0); i < cK; ++i) mbar_wait_drain(&mi.k_full[i % NKS], full_par(i / NKS), cx.abort_flag);
          for (uint32_t i = (cV > NVS ? cV - NVS : 0); i < cV; ++i) mbar_wait_drain(&mi.v_full[i % NVS], full_par(i / NVS), cx.abort_flag);
          for (uint32_t i = (cQ > 2 ? cQ - 2 : 0); i < cQ; ++i) mbar_wait_drain(&mi.q_full[i & 1], full_par(i >> 1), cx.abort_flag);
        }
        abort_grace_pause(cx.abort_flag);
      }
    }
    __syncwarp();
  } else if (warp == WARP_QK) {
    // ================================================================ issuer of S = Q K^T (leader CTA)
    if (lane == 0 && leader) {
      const uint32_t idesc_qk = make_idesc_bf16_f32(256, TILE, false, false);
      const uint32_t idesc_sw = make_idesc_bf16_f32(256, 2 * rows_half, false, false);
      const uint32_t rk_u32 = smem_u32(cx.rK);
      uint32_t cQ = 0, cK = 0, cS = 0, cT = 0, n_done = 0;
      for (int item = pair_id; item < n_items && !*cx.abort_flag; item += n_pairs) {
        int group, within, c, hkv;
        sch.d_ipg.divmod(item, group, within);
        sch.d_hkv.divmod(group, c, hkv);
        const int nsub = n_subitems2(sch, within);
        const int len = chunk_length(prm, c);
        for (int sub = 0; sub < nsub; ++sub) {
          const Blk bk = decode_blk(sch, rank, hkv, within, sub, len);
          if (bk.n == 0) continue;
          const int qb = cQ & 1;
          WAIT2(&mi.q_full[qb], full_par(cQ >> 1), W2_QFULL);           // the query tiles of both CTAs have landed
          ++cQ;
          const uint32_t q_u32 = smem_u32(cx.sQ[qb]);
          for (int j = 0; j < bk.n; ++j) {
            const int sb = cS % NSB;
            // S(t) of a warpgroup overwrites its S(t-2): wait until that is in registers.  (P lives elsewhere.)
            WAIT2(&mi.s_read[sb], free_par(cS / NSB), W2_PVDONE);
            const int s = cK % NKS;
            WAIT2(&mi.k_full[s], full_par(cK / NKS), W2_KFULL);
            tc_fence_after_sync();
            const uint32_t k_u32 = rk_u32 + s * HALF_BYTES;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks)
              mma_ss_pair(cx.tmem + sb * TILE, make_smem_desc_sw128(q_u32 + (ks / 4) * 16384 + (ks % 4) * 32, 16, 1024),
                          make_smem_desc_sw128(k_u32 + (ks / 4) * 8192 + (ks % 4) * 32, 16, 1024), idesc_qk, ks > 0);
            mma_commit_pair(&mi.s_full[cS & 1][sb]);   // tile cS belongs to warpgroup cS & 1
            mma_commit_pair(&mi.k_free[s]);
            ++cK;
            ++cS;
          }
          ++n_done;
        }
        if (within == 0) {
          // ---- score sweep.  Its two [128 keys x 256 rows] buffers overlay all of TMEM: every S/P
          // buffer is consumed and the accumulator has been read out once acc_free completes.
          WAIT2(&mi.acc_free, free_par(n_done), W2_ACCFREE);
          const int n_sweep_tiles = ((len + TILE - 1) / TILE + 1) / 2;
          for (int u = 0; u < sch.n_pass; ++u) {
            const int qb = cQ & 1;
            WAIT2(&mi.q_full[qb], full_par(cQ >> 1), W2_QFULL);
            ++cQ;
            const uint32_t q_u32 = smem_u32(cx.sQ[qb]);
            if (cK & 1) {
              const int s = cK % NKS;
              WAIT2(&mi.k_full[s], full_par(cK / NKS), W2_KFULL);
              mma_commit_pair(&mi.k_free[s]);
              ++cK;
            }
            for (int jj = 0; jj < n_sweep_tiles; ++jj) {
              const int e = cT & 1;
              WAIT2(&mi.t_free[e], free_par(cT >> 1), W2_TFREE);
              const int s = cK % NKS;
              WAIT2(&mi.k_full[s], full_par(cK / NKS), W2_KFULL);
              WAIT2(&mi.k_full[s + 1], full_par((cK + 1) / NKS), W2_KFULL);
              tc_fence_after_sync();
              const uint32_t k_u32 = rk_u32 + s * HALF_BYTES;
#pragma unroll
              for (int ks = 0; ks < D / 16; ++ks)
                mma_ss_pair(cx.tmem + e * 256, make_smem_desc_sw128(k_u32 + (ks / 4) * 16384 + (ks % 4) * 32, 16, 1024),
                            make_smem_desc_sw128(q_u32 + (ks / 4) * 16384 + (ks % 4) * 32, 16, 1024), idesc_sw, ks > 0);
              mma_commit_pair(&mi.t_full[e]);
              mma_commit_pair(&mi.k_free[s]);
              mma_commit_pair(&mi.k_free[s + 1]);
              cK += 2;
              ++cT;
            }
          }
          // the next item's S buffers overlay the sweep buffers: wait until both were read
          WAIT2(&mi.t_free[0], free_par((cT + 1) >> 1), W2_TFREE);
          WAIT2(&mi.t_free[1], free_par(cT >> 1), W2_TFREE);
        }
      }
      mma_commit_pair(&mi.mma_done);                         // teardown waits for everything this thread issued
    }
    __syncwarp();
  } else if (warp == WARP_PV || warp == WARP_PV + 1) {
    // ================================================================ issuers of O += P V (leader CTA)
    // Two threads take alternate tiles: the barrier waits and commits of one (a few hundred cycles
    // per tile, during which a blocked-issue pipe would run dry) overlap the issue of the other.
    // A token keeps the accumulation in tile order, so the result does not depend on timing.
    if (lane == 0 && leader) {
      const int me = warp - WARP_PV;
      constexpr uint32_t idesc_pv = make_idesc_bf16_f32(256, D, false, true);
      const uint32_t rv_u32 = smem_u32(cx.rV);
      uint32_t cS = 0, n_done = 0, n_turn = 0;
      for (int item = pair_id; item < n_items && !*cx.abort_flag; item += n_pairs) {
        int group, within, c, hkv;
        sch.d_ipg.divmod(item, group, within);
        sch.d_hkv.divmod(group, c, hkv);
        const int nsub = n_subitems2(sch, within);
        const int len = chunk_length(prm, c);
        for (int sub = 0; sub < nsub; ++sub) {
          const Blk bk = decode_blk(sch, rank, hkv, within, sub, len);
          if (bk.n == 0) continue;
          WAIT2(&mi.acc_free, free_par(n_done), W2_ACCFREE);                   // accumulator of the previous block read out
          for (int j = 0; j < bk.n; ++j, ++cS) {
            if ((int)(cS & 1) != me) continue;
            const int sb = cS % NSB;
            const int s = cS % NVS;                                            // one V stage per tile
            WAIT2(&mi.v_full[s], full_par(cS / NVS), W2_VFULL);
            const uint32_t v_u32 = rv_u32 + s * HALF_BYTES;
            const uint32_t tP = cx.tmem + TM_P + (cS & 1) * 64;
            WAIT2(&mi.p_a[me][sb], full_par(cS / NSB), W2_PA);           // keys 0..63 of P
            WAIT2(&mi.pv_turn[me], me == 0 ? free_par(n_turn) : full_par(n_turn), W2_TURN);   // P V of tile cS-1 issued
            tc_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              mma_ts_pair(cx.tmem + TM_O, tP + ks * 8, make_smem_desc_sw128(v_u32 + ks * 2048, 16384, 1024), idesc_pv,
                          j > 0 || ks > 0);
            WAIT2(&mi.p_b[me][sb], full_par(cS / NSB), W2_PB);           // keys 64..127
            tc_fence_after_sync();
#pragma unroll
            for (int ks = 4; ks < 8; ++ks)
              mma_ts_pair(cx.tmem + TM_O, tP + ks * 8, make_smem_desc_sw128(v_u32 + ks * 2048, 16384, 1024), idesc_pv, true);
            tc_fence_before_sync();
            mbar_arrive(&mi.pv_turn[me ^ 1]);
            ++n_turn;
            mma_commit_pair(&mi.v_free[s]);
            if (j == bk.n - 1) mma_commit_pair(&mi.o_full);
          }
          ++n_done;
        }
      }
      mma_commit_pair(&mi.mma_done);
    }
    __syncwarp();
  } else if (warp < 8) {
    // ================================================================ softmax: two threads per query row
    const int r = tid & 127;                                 // row of the block = TMEM lane
    const int hlf = tid >> 7;                                // which 64 keys of every tile / which 64 head-dim columns
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const float scale_log2 = prm.scale_log2;
    const uint32_t a_acc_free = map_to_cta(&mi.acc_free, 0);
    uint32_t cQ = 0, cS = 0, cT = 0, n_done = 0, n_tail = 0;
    uint32_t n_pub_mine = 0, n_pub_other = 0;                // publications made by this warpgroup / seen from the other
    // The output tile is stored from the block's Q buffer.  The thread that issued the store does not wait for
    // it there (its warp would reach the next block's first tile a few thousand cycles after the others, and a
    // tile is only as fast as its slowest warp): it waits, and hands the buffer back to the producer, after its
    // first tile of the next block, when the store has long been read.
    int store_pending = -1;                                  // thread 0: Q buffer of a store that may still be reading it
    auto finish_store = [&]() {
      if (tid == 0 && store_pending >= 0) {
        tma_store_wait_read();
        mbar_arrive(&mi.q_free[store_pending]);
        store_pending = -1;
      }
    };
    for (int item = pair_id; item < n_items && !*cx.abort_flag; item += n_pairs) {
      int group, within, c, hkv;
      sch.d_ipg.divmod(item, group, within);
      sch.d_hkv.divmod(group, c, hkv);
      const int nsub = n_subitems2(sch, within);
      const int len = chunk_length(prm, c);
      for (int sub = 0; sub < nsub; ++sub) {
        const Blk bk = decode_blk(sch, rank, hkv, within, sub, len);
        if (bk.n == 0) continue;
        const int token = bk.t * TILE + r;
        const int qb = cQ & 1;                               // this block's query buffer (its output is staged there)
        ++cQ;
        uint8_t* const myQ = cx.sQ[qb];
        // ---- key tiles: the two warpgroups take alternate tiles (whole rows, one thread per row), so the
        // load / maximum phase of one tile runs under the exponentials of the other.  The running
        // maximum is decided tile by tile in order: the owner of tile j waits for the owner of tile
        // j-1 to publish its per-row reference maximum, decides (lazy rescale) and publishes its own.
        float m_seen = -INFINITY, l_run = 0.0f;                // l_run: sum over this thread's tiles, relative to m_seen
        for (int j = 0; j < bk.n; ++j, ++cS) {
          const int owner = cS & 1;
          if (owner != hlf) continue;
          const int sb = cS % NSB;
          WAIT2S(&mi.s_full[owner][sb], full_par(cS / NSB), W2_SFULL);
          tc_fence_after_sync();
          const uint32_t tS = cx.tmem + sb * TILE + lane_sel;
          uint32_t s[4][32];
#pragma unroll
          for (int q = 0; q < 4; ++q) tmem_ld32(tS + q * 32, s[q]);
          tmem_wait_ld();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(map_to_cta(&mi.s_read[sb], 0));   // Q K^T of this warpgroup's next tile may start
          const int vis = token - j * TILE + 1;                // visible columns (causal); >= 128: all
          if (vis < TILE) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (q * 32 + i >= vis) s[q][i] = 0xFF800000u;            // -inf
          }
          float mq[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            float a = fmax3(__uint_as_float(s[q][0]), __uint_as_float(s[q][1]), __uint_as_float(s[q][2]));
#pragma unroll
            for (int i = 3; i < 31; i += 2) a = fmax3(a, __uint_as_float(s[q][i]), __uint_as_float(s[q][i + 1]));
            mq[q] = fmaxf(a, __uint_as_float(s[q][31]));
          }
          const float m_tile = fmaxf(fmaxf(mq[0], mq[1]), fmaxf(mq[2], mq[3])) * scale_log2;   // -inf: nothing visible
          // reference maximum after tile j-1 (published by the other warpgroup)
          float m_prev = -INFINITY;
          if (j > 0) {                                         // the partner's publication of tile j-1
            WAIT2S(&mi.m_pub[hlf ^ 1][warp & 3], full_par(n_pub_other), W2_MPUB);
            ++n_pub_other;
            m_prev = mi.mref[(j - 1) & 1][r];
          }
          const bool first_tile = (j == 0);
          const bool raise = first_tile || (m_tile > m_prev + LAZY_RESCALE);
          const float m_new = raise ? fmaxf(m_prev, m_tile) : m_prev;
          mi.mref[j & 1][r] = m_new;
          __syncwarp();
          if (lane == 0) mbar_arrive(&mi.m_pub[hlf][warp & 3]);   // the warp with the same rows may decide tile j+1
          ++n_pub_mine;
          if (m_new != m_seen) {                               // bring this thread's partial sum to the new reference
            l_run *= (m_seen == -INFINITY) ? 0.0f : fast_exp2(m_seen - m_new);
            m_seen = m_new;
          }
          if (!first_tile && __any_sync(0xFFFFFFFFu, raise)) {
            // rare: rescale the accumulator rows of this warp.  P V of tile j-1 may still be running
            // (it is not ordered before this tile's S): wait for it; P V of tile j cannot start before
            // this thread publishes P.
            const float alpha = (m_prev == -INFINITY) ? 0.0f : fast_exp2(m_prev - m_new);
            const uint32_t prev = cS - 1;
            WAIT2S(&mi.v_free[prev % NVS], full_par(prev / NVS), W2_PVDONE);   // committed after P V of tile `prev`
            tc_fence_after_sync();
            const uint32_t tO = cx.tmem + TM_O + lane_sel;
#pragma unroll 1
            for (int q = 0; q < D / 8; ++q) {
              uint32_t o[8];
              tmem_ld8(tO + q * 8, o);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              tmem_st8(tO + q * 8, o);
            }
          }
          if (cS >= 2) {
            // the P buffer of this warpgroup is free once P V of its previous tile has run; this wait also keeps
            // the softmax at most one own tile ahead of the P V issuer, whose barriers have one phase bit
            const uint32_t prev2 = cS - 2;
            WAIT2S(&mi.v_free[prev2 % NVS], full_par(prev2 / NVS), W2_PVDONE);
            tc_fence_after_sync();
          }
          const float neg_m = (m_new == -INFINITY) ? 0.0f : -m_new;
          const uint64_t scale2 = pack_f32x2(scale_log2, scale_log2), negm2 = pack_f32x2(neg_m, neg_m);
          uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t packed[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(s[q][2 * i]), __uint_as_float(s[q][2 * i + 1])), scale2, negm2);
              float x0, x1, p0, p1;
              unpack_f32x2(x2, x0, x1);
              p0 = fast_exp2(x0);                                // MUFU pipe
              p1 = fast_exp2(x1);
              sum2[i & 1] = add_f32x2(sum2[i & 1], pack_f32x2(p0, p1));
              packed[i] = pack_bf16x2(p0, p1);
            }
            tmem_st16(cx.tmem + TM_P + hlf * 64 + q * 16 + lane_sel, packed);   // P: 64 bf16 columns
            if (q == 1) {                                      // keys 0..63 are final: P V may start on them
              tmem_wait_st();
              tc_fence_before_sync();
              __syncwarp();
              if (lane == 0) mbar_arrive_remote(map_to_cta(&mi.p_a[hlf][sb], 0));
            }
          }
          float a0, a1, a2, a3;
          unpack_f32x2(sum2[0], a0, a1);
          unpack_f32x2(sum2[1], a2, a3);
          l_run += (a0 + a1) + (a2 + a3);
          tmem_wait_st();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(map_to_cta(&mi.p_b[hlf][sb], 0));
          finish_store();
        }
        // the warpgroup that did not own the last tile consumes its owner's publication; then both
        // bring their partial sums to the final reference maximum
        {
          const int last_owner = (cS - 1) & 1;
          if (hlf != last_owner) {
            WAIT2S(&mi.m_pub[hlf ^ 1][warp & 3], full_par(n_pub_other), W2_MPUB);
            ++n_pub_other;
          }
          const float m_fin = mi.mref[(bk.n - 1) & 1][r];
          if (m_fin != m_seen) {
            l_run *= (m_seen == -INFINITY) ? 0.0f : fast_exp2(m_seen - m_fin);
            m_seen = m_fin;
          }
        }
        const float m_used = m_seen;
        finish_store();
        // ---- epilogue: combine the two half-row sums, normalise, stage bf16 rows in this block's
        // (now idle) Q buffer, TMA store
        WAIT2S(&mi.o_full, full_par(n_done), W2_OFULL);
        ++n_done;
        tc_fence_after_sync();
        mi.xl[hlf][r] = l_run;
        named_barrier_sync(1, 256);
        const float l_tot = mi.xl[0][r] + mi.xl[1][r];
        const float inv_l = token < len ? 1.0f / l_tot : 0.0f;   // rows behind the end of the chunk are written as zeros
        {
          const uint32_t tO = cx.tmem + TM_O + hlf * 64 + lane_sel;
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            uint32_t o[32];
            tmem_ld32(tO + q * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int g4 = 0; g4 < 4; ++g4) {
              uint32_t pk[4];
#pragma unroll
              for (int e = 0; e < 4; ++e)
                pk[e] = token < len ? pack_bf16x2(__uint_as_float(o[g4 * 8 + 2 * e]) * inv_l, __uint_as_float(o[g4 * 8 + 2 * e + 1]) * inv_l) : 0u;
              *reinterpret_cast<uint4*>(myQ + hlf * 16384 + sw128_offset(r, q * 4 + g4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(a_acc_free);
        if (hlf == 0 && token < len) {
          const float lse2 = m_used + log2f(l_tot);
          if (prm.lse) prm.lse[((size_t)c * prm.Hq + bk.h) * prm.L + token] = lse2 * 0.6931471805599453f;
          const int wi = token - (len - prm.w);
          if (wi >= 0) {
            prm.win_lse[((size_t)c * prm.Hq + bk.h) * prm.w + wi] = lse2 * 0.6931471805599453f;
            if (within == 0) {                               // the sweep of both CTAs needs it
              float* slot = &mi.lse2[(bk.h - hkv * sch.G) * prm.w + wi];
              *slot = lse2;
              st_shared_cluster_f32(map_to_cta(slot, rank ^ 1u), lse2);
            }
          }
        }
        fence_proxy_async_smem();
        named_barrier_sync(1, 256);
        if (tid == 0) {
          if (bk.t * TILE < prm.L) {
            for (int a = 0; a < 2; ++a) tma_store_4d(&tm_o, myQ + a * 16384, a * 64, bk.h, bk.t * TILE, c);
            tma_store_commit();
          }
          store_pending = qb;                                // released by finish_store() once the store has read it
        }
      }
      if (within == 0) {
        finish_store();                                      // a later sweep pass loads window queries into that buffer
        // ---- score sweep.  First make the window rows' log-sum-exp of all heads visible in both CTAs.
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster(map_to_cta(&mi.lse_ready, 0));
          mbar_arrive_cluster(map_to_cta(&mi.lse_ready, 1));
        }
        mbar_wait_cluster(&mi.lse_ready, full_par(n_tail), cx.abort_flag, cx.status, W2_LSE);
        ++n_tail;
        const int n_sweep_tiles = ((len + TILE - 1) / TILE + 1) / 2;
        const int w0 = len - prm.w;                          // first window token of this chunk
        for (int u = 0; u < sch.n_pass; ++u) {
          const int qb = cQ & 1;                             // window queries of this pass (loaded and consumed by other warps)
          ++cQ;
          // this thread sums the columns of the heads that CTA `hlf` loaded: local head i = ncol / w
          const int g_base = u * 2 * sch.hp + hlf * sch.hp;
          for (int jj = 0; jj < n_sweep_tiles; ++jj) {
            const int e = cT & 1;
            WAIT2S(&mi.t_full[e], full_par(cT >> 1), W2_TFULL);
            tc_fence_after_sync();
            const int key = (2 * jj + (int)rank) * TILE + r;
            const bool need_mask = (2 * jj + (int)rank) * TILE + TILE - 1 > w0;
            const uint32_t tT = cx.tmem + e * 256 + hlf * rows_half + lane_sel;
            float part = 0.0f;
            for (int ih = 0; ih < sch.hp; ++ih) {            // heads of this column half; a head has wp columns, the last w are window rows
              const int g = g_base + ih;
              if (g >= sch.G) break;                         // filler head
              const float* lse_head = mi.lse2 + g * prm.w;
              for (int col = 0; col < sch.wp; col += 8) {
                uint32_t sv[8];
                tmem_ld8(tT + ih * sch.wp + col, sv);
                tmem_wait_ld();
                const int wi0 = col - (sch.wp - prm.w);      // window row of the first of these 8 columns (negative: not a window row)
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const int wi = wi0 + i;
                  float pv = fast_exp2(fmaf(__uint_as_float(sv[i]), scale_log2, -lse_head[wi < 0 ? 0 : wi]));
                  if (wi < 0 || (need_mask && key > w0 + wi)) pv = 0.0f;
                  part += pv;
                }
              }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(map_to_cta(&mi.t_free[e], 0));
            mi.xs[e][hlf][r] = part;
            named_barrier_sync(1, 256);
            if (hlf == 0 && key < len) {
              float* dst = prm.win_score + ((size_t)c * prm.Hkv + hkv) * prm.L + key;
              const float total = part + mi.xs[e][1][r];
              *dst = (u == 0) ? total : (*dst + total);
            }
            ++cT;
          }
          named_barrier_sync(1, 256);                        // everyone is past its last use of sQ[qb]
          if (tid == 0) mbar_arrive(&mi.q_free[qb]);
        }
      }
    }
    finish_store();
    if (tid == 0) tma_store_wait_all();
  }

  // ---- teardown: no CTA may exit while its peer can still signal it or read its shared memory
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == WARP_QK) {
    // no tensor-core operation may still be running when its accumulators are freed: every issuer ended with a
    // commit to mma_done (three arrivals in both CTAs).  Immediate in a clean run; after an abort this is what
    // makes the exit safe.  The wait ignores the abort flag and is bounded.
    mbar_wait_drain(&mi.mma_done, 0, cx.abort_flag);
    tc_fence_after_sync();
    tmem_dealloc_pair(cx.tmem, 512);
  }
}

// ====================================================================================
//                                   host launcher
// ====================================================================================
// maps: 0 q (box 64 x 128 tokens), 1 rotated keys (64 x 128), 2 v (64 x 128), 3 o (store), 4 q with a
// w-token box, 5 rotated keys with a 64-token box.  The grid is a whole number of CTA pairs.
cudaError_t launch_prefill_pair(const CUtensorMap* maps, const PrefillParams& prm, int sm_count, cudaStream_t st) {
  // the opt-in to large dynamic shared memory is a per-device attribute of the function: set it on every call
  // (a host-side call of a few hundred nanoseconds) rather than remember which devices have it
  if (cudaError_t e = cudaFuncSetAttribute(prefill_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES); e != cudaSuccess) return e;
  const int grid = (sm_count / 2) * 2;
  if (grid < 2) return cudaErrorInvalidConfiguration;
  if ((prm.Hq / prm.Hkv) % 2 != 0) return cudaErrorInvalidValue;   // the pair kernel takes even group sizes
  note_launch();
  prefill_pair_kernel<<<grid, NT2, SMEM2_BYTES, st>>>(maps[0], maps[5], maps[1], maps[2], maps[3], maps[4], prm);
  return cudaGetLastError();
}

}  // namespace pc
