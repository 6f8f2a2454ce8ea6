// Parallel (global) attention of the query window over the compressed cache (Sec. 3.1 "Global attention",
// Eq. 9-11) for head size 128 on CTA pairs, for batches in which every (sequence, kv-head) brings a whole
// number of 256-row groups: G * w a multiple of 256.
//
// The machinery is that of the chunk-local pair kernel (tcgen05 cta_group::2: each CTA of a cluster owns one
// 128-row query block, every 128-key tile is split between the two shared memories - 64 keys of K and 64
// head-dim columns of V per CTA - which halves the shared-memory traffic per MMA; two softmax warpgroups
// per CTA take alternate key tiles and meet only in the per-row decision on the running maximum).
// What differs: the 256 rows of a pair are the w window queries of 256 / w q-heads of one kv-head (they
// all read the same cache, so a pair streams each cache tile once for all of them and no key split or
// merge pass is needed once the batch has a few groups per pair); there is no causal structure except
// inside the last tile, which holds the window's own keys; a ragged last cache tile is masked by count.
// Queries arrive rotated (the bandwidth-bound RoPE pass runs before this kernel).
//
// Warps (12 per CTA): 0-3 softmax of even tiles, 4-7 softmax of odd tiles, 8 TMA producer, 9 issuer of
// Q K^T, 10 and 11 issuers of P V for even / odd tiles (issuers run in the leader CTA only).
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

enum { W3_QFULL = 301, W3_QFREE, W3_KFULL, W3_KFREE, W3_VFULL, W3_VFREE, W3_SFULL, W3_PA, W3_PB,
       W3_PVDONE, W3_OFULL, W3_ACCFREE, W3_MPUB, W3_TURN };

struct __align__(16) Misc3 {
  uint64_t q_full[2], q_free[2];             // q_full: leader only, counts the bytes of both CTAs' query tiles
  uint64_t k_full[NKS], k_free[NKS], v_full[NVS], v_free[NVS];
  uint64_t s_full[2][NSB];                   // [owning warpgroup][buffer]
  uint64_t p_a[2][NSB], p_b[2][NSB];         // [owning warpgroup = P V issuer][buffer]
  uint64_t s_read[NSB];                      // leader only: S of the tile in this buffer is in registers (8 warps of the pair)
  uint64_t pv_turn[2];                       // leader only: issue token of the two P V issuers
  uint64_t o_full, acc_free;
  uint64_t m_pub[2][4];                      // [owner warpgroup][warp]: its reference maxima of a tile are in mref
  uint64_t mma_done;                         // every tensor-core operation of the three issuers has completed (teardown)
  uint32_t tmem_base;
  int abort_flag;                            // the two words after tmem_base stay adjacent: bounded waits read the limit
  int wait_kcycles;                          // through the flag's address
  float mref[2][TILE];                       // [tile parity][row]: reference maximum (log2 units) after that tile
  float xl[2][TILE];                         // [warpgroup][row]: partial row sums
};

constexpr int OFF_Q = 0;
constexpr int OFF_RK = 2 * Q_BYTES;
constexpr int OFF_RV = OFF_RK + NKS * HALF_BYTES;
constexpr int OFF_MISC = OFF_RV + NVS * HALF_BYTES;
constexpr int SMEM3_BYTES = OFF_MISC + (int)sizeof(Misc3) + 1024;

__device__ __forceinline__ uint32_t full_par(uint32_t n) { return n & 1u; }           // n-th completion of a barrier
__device__ __forceinline__ uint32_t free_par(uint32_t n) { return (n & 1u) ^ 1u; }    // completion n-1 (passes for n = 0)

struct Ctx3 {
  Misc3* mi;
  uint8_t* sQ[2];
  uint8_t* rK;
  uint8_t* rV;
  uint32_t tmem;
  uint32_t rank;
  volatile int* abort_flag;
  int* status;
};

// waits of the single-thread service roles (long pause between polls) / of the softmax warps
#define WAIT3(bar, par, code) mbar_wait_ns<SERVICE_BACKOFF_NS>((bar), (par), cx.abort_flag, cx.status, (code))
#define WAIT3S(bar, par, code) mbar_wait((bar), (par), cx.abort_flag, cx.status, (code))

__device__ __forceinline__ void init_barriers3(Misc3& mi, int wait_kcycles) {
  for (int b = 0; b < 2; ++b) { mbar_init(&mi.q_full[b], 1); mbar_init(&mi.q_free[b], 1); }
  for (int s = 0; s < NKS; ++s) { mbar_init(&mi.k_full[s], 1); mbar_init(&mi.k_free[s], 1); }
  for (int s = 0; s < NVS; ++s) { mbar_init(&mi.v_full[s], 1); mbar_init(&mi.v_free[s], 1); }
  for (int s = 0; s < NSB; ++s) {
    mbar_init(&mi.s_full[0][s], 1); mbar_init(&mi.s_full[1][s], 1); mbar_init(&mi.s_read[s], 8);
    for (int g = 0; g < 2; ++g) { mbar_init(&mi.p_a[g][s], 8); mbar_init(&mi.p_b[g][s], 8); }   // 4 warps of the owning warpgroup in each CTA
  }
  mbar_init(&mi.pv_turn[0], 1); mbar_init(&mi.pv_turn[1], 1);
  mbar_init(&mi.o_full, 1); mbar_init(&mi.acc_free, 16);
  for (int w = 0; w < 4; ++w) { mbar_init(&mi.m_pub[0][w], 1); mbar_init(&mi.m_pub[1][w], 1); }   // warp to warp (same rows)
  mbar_init(&mi.mma_done, 3);
  mi.abort_flag = 0;
  mi.wait_kcycles = wait_kcycles;
  fence_mbar_init();
}

// item -> (sequence, kv-head, row group); the pair's rows are the windows of the 2 * hpc heads from h0 on,
// CTA `rank` holds heads h0 + rank * hpc .. + hpc - 1, head-major (row = local head * w + window index)
struct Item3 {
  int seq, hkv, h0;
};
__device__ __forceinline__ Item3 decode_item3(const ParallelPairParams& p, int item) {
  Item3 it;
  const int rg = item % p.n_rg;
  const int x = item / p.n_rg;
  it.hkv = x % p.Hkv;
  it.seq = x / p.Hkv;
  it.h0 = it.hkv * (p.Hq / p.Hkv) + rg * 2 * p.hpc;
  return it;
}

}  // namespace

// tensor maps: tm_q (rotated window queries [B,w,Hq,d], box 64 d x 1 head x w tokens), tm_o (output, same
// shape and box, store), tm_kc (cache keys [B,Hkv,Nk,d], box 64 d x 64 keys), tm_vc (cache values, box 64 d x
// 128 keys), tm_kw (window keys [B,w,Hkv,d], box 64 d x 1 head x 64 tokens), tm_vw (window values, box 64 d x
// 1 head x 128 tokens).  Rows of a box that lie behind the end of the tensor read as zeros; the softmax masks
// those keys by count.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NT2, 1)
parallel_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_o,
                     const __grid_constant__ CUtensorMap tm_kc, const __grid_constant__ CUtensorMap tm_vc,
                     const __grid_constant__ CUtensorMap tm_kw, const __grid_constant__ CUtensorMap tm_vw,
                     const __grid_constant__ ParallelPairParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  Misc3& mi = *reinterpret_cast<Misc3*>(smem + OFF_MISC);
  Ctx3 cx;
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
  const int n_items = prm.B * prm.Hkv * prm.n_rg;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_cache = (prm.Nk + TILE - 1) / TILE;          // cache tiles; the window tile follows them
  const int n_tiles = n_cache + 1;

  if (tid == 0) init_barriers3(mi, prm.wait_kcycles);
  if (warp == WARP_QK) tmem_alloc_pair(&mi.tmem_base, 512);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                    // both CTAs' barriers exist before any remote arrive
  tc_fence_after_sync();
  cx.tmem = mi.tmem_base;

  if (warp == WARP_PRODUCER) {
    // ================================================================ TMA producer (both CTAs)
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_kc); tma_prefetch_desc(&tm_vc); tma_prefetch_desc(&tm_kw);
      tma_prefetch_desc(&tm_vw);
      uint32_t cQ = 0, cK = 0, cV = 0;
      // Once a wait has run out (abort flag) no new work is started: every role leaves its loops at the next item,
      // this one also at the next tile, so that no copy is issued into a ring that nobody drains any more.
      for (int item = pair_id; item < n_items && !*cx.abort_flag; item += n_pairs) {
        const Item3 it = decode_item3(prm, item);
        {
          const int qb = cQ & 1;
          WAIT3(&mi.q_free[qb], free_par(cQ >> 1), W3_QFREE);
          if (leader) mbar_arrive_expect_tx(&mi.q_full[qb], 2 * Q_BYTES);
          const uint32_t bar = map_to_cta(&mi.q_full[qb], 0);
          for (int i = 0; i < prm.hpc; ++i)
            for (int a = 0; a < 2; ++a)
              tma_load_4d_pair(cx.sQ[qb] + a * 16384 + i * prm.w * 128, &tm_q, bar, a * 64, it.h0 + (int)rank * prm.hpc + i, 0,
                               it.seq);
          ++cQ;
        }
        for (int j = 0; j < n_tiles && !*cx.abort_flag; ++j) {
          {
            const int s = cK % NKS;
            WAIT3(&mi.k_free[s], free_par(cK / NKS), W3_KFREE);
            if (leader) mbar_arrive_expect_tx(&mi.k_full[s], 2 * HALF_BYTES);
            const uint32_t bar = map_to_cta(&mi.k_full[s], 0);
            for (int a = 0; a < 2; ++a) {
              uint8_t* dst = cx.rK + s * HALF_BYTES + a * 8192;
              if (j < n_cache) tma_load_4d_pair(dst, &tm_kc, bar, a * 64, j * TILE + (int)rank * 64, it.hkv, it.seq);
              else tma_load_4d_pair(dst, &tm_kw, bar, a * 64, it.hkv, (int)rank * 64, it.seq);
            }
            ++cK;
          }
          {
            const int s = cV % NVS;
            WAIT3(&mi.v_free[s], free_par(cV / NVS), W3_VFREE);
            if (leader) mbar_arrive_expect_tx(&mi.v_full[s], 2 * HALF_BYTES);
            const uint32_t bar = map_to_cta(&mi.v_full[s], 0);
            if (j < n_cache) tma_load_4d_pair(cx.rV + s * HALF_BYTES, &tm_vc, bar, (int)rank * 64, j * TILE, it.hkv, it.seq);
            else tma_load_4d_pair(cx.rV + s * HALF_BYTES, &tm_vw, bar, (int)rank * 64, it.hkv, 0, it.seq);
            ++cV;
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
      const uint32_t rk_u32 = smem_u32(cx.rK);
      uint32_t cQ = 0, cK = 0, cS = 0;
      for (int item = pair_id; item < n_items && !*cx.abort_flag; item += n_pairs) {
        const int qb = cQ & 1;
        WAIT3(&mi.q_full[qb], full_par(cQ >> 1), W3_QFULL);             // the query tiles of both CTAs have landed
        ++cQ;
        const uint32_t q_u32 = smem_u32(cx.sQ[qb]);
        for (int j = 0; j < n_tiles; ++j) {
          const int sb = cS % NSB;
          // S(t) of a warpgroup overwrites its S(t-2): wait until that is in registers.  (P lives elsewhere.)
          WAIT3(&mi.s_read[sb], free_par(cS / NSB), W3_PVDONE);
          const int s = cK % NKS;
          WAIT3(&mi.k_full[s], full_par(cK / NKS), W3_KFULL);
          tc_fence_after_sync();
          const uint32_t k_u32 = rk_u32 + s * HALF_BYTES;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            mma_ss_pair(cx.tmem + sb * TILE, make_smem_desc_sw128(q_u32 + (ks / 4) * 16384 + (ks % 4) * 32, 16, 1024),
                        make_smem_desc_sw128(k_u32 + (ks / 4) * 8192 + (ks % 4) * 32, 16, 1024), idesc_qk, ks > 0);
          mma_commit_pair(&mi.s_full[cS & 1][sb]);     // tile cS belongs to warpgroup cS & 1
          mma_commit_pair(&mi.k_free[s]);
          ++cK;
          ++cS;
        }
      }
      mma_commit_pair(&mi.mma_done);                         // teardown waits for everything this thread issued
    }
    __syncwarp();
  } else if (warp == WARP_PV || warp == WARP_PV + 1) {
    // ================================================================ issuers of O += P V (leader CTA)
    // Two threads take alternate tiles; a token keeps the accumulation in tile order, so the result does not
    // depend on timing.
    if (lane == 0 && leader) {
      const int me = warp - WARP_PV;
      constexpr uint32_t idesc_pv = make_idesc_bf16_f32(256, D, false, true);
      const uint32_t rv_u32 = smem_u32(cx.rV);
      uint32_t cS = 0, n_done = 0, n_turn = 0;
      for (int item = pair_id; item < n_items && !*cx.abort_flag; item += n_pairs) {
        WAIT3(&mi.acc_free, free_par(n_done), W3_ACCFREE);                     // accumulator of the previous item read out
        for (int j = 0; j < n_tiles; ++j, ++cS) {
          if ((int)(cS & 1) != me) continue;
          const int sb = cS % NSB;
          const int s = cS % NVS;                                              // one V stage per tile
          WAIT3(&mi.v_full[s], full_par(cS / NVS), W3_VFULL);
          const uint32_t v_u32 = rv_u32 + s * HALF_BYTES;
          const uint32_t tP = cx.tmem + TM_P + (cS & 1) * 64;
          WAIT3(&mi.p_a[me][sb], full_par(cS / NSB), W3_PA);             // keys 0..63 of P
          WAIT3(&mi.pv_turn[me], me == 0 ? free_par(n_turn) : full_par(n_turn), W3_TURN);   // P V of tile cS-1 issued
          tc_fence_after_sync();
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            mma_ts_pair(cx.tmem + TM_O, tP + ks * 8, make_smem_desc_sw128(v_u32 + ks * 2048, 16384, 1024), idesc_pv,
                        j > 0 || ks > 0);
          WAIT3(&mi.p_b[me][sb], full_par(cS / NSB), W3_PB);             // keys 64..127
          tc_fence_after_sync();
#pragma unroll
          for (int ks = 4; ks < 8; ++ks)
            mma_ts_pair(cx.tmem + TM_O, tP + ks * 8, make_smem_desc_sw128(v_u32 + ks * 2048, 16384, 1024), idesc_pv, true);
          tc_fence_before_sync();
          mbar_arrive(&mi.pv_turn[me ^ 1]);
          ++n_turn;
          mma_commit_pair(&mi.v_free[s]);
          if (j == n_tiles - 1) mma_commit_pair(&mi.o_full);
        }
        ++n_done;
      }
      mma_commit_pair(&mi.mma_done);
    }
    __syncwarp();
  } else if (warp < 8) {
    // ================================================================ softmax: the two warpgroups take alternate tiles
    const int r = tid & 127;                                 // row of the block = TMEM lane
    const int hlf = tid >> 7;                                // warpgroup: owner of the tiles of this parity
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const float scale_log2 = prm.scale_log2;
    const uint32_t a_acc_free = map_to_cta(&mi.acc_free, 0);
    const int wi = r % prm.w;                                // window index of this row
    const int h_local = r / prm.w;
    uint32_t cQ = 0, cS = 0, n_done = 0;
    uint32_t n_pub_mine = 0, n_pub_other = 0;                // publications made by this warpgroup / seen from the other
    int store_pending = -1;                                  // thread 0: Q buffer of a store that may still be reading it
    auto finish_store = [&]() {
      if (tid == 0 && store_pending >= 0) {
        tma_store_wait_read();
        mbar_arrive(&mi.q_free[store_pending]);
        store_pending = -1;
      }
    };
    for (int item = pair_id; item < n_items && !*cx.abort_flag; item += n_pairs) {
      const Item3 it = decode_item3(prm, item);
      const int h = it.h0 + (int)rank * prm.hpc + h_local;
      const int qb = cQ & 1;                                 // this item's query buffer (its output is staged there)
      ++cQ;
      uint8_t* const myQ = cx.sQ[qb];
      float m_seen = -INFINITY, l_run = 0.0f;                // l_run: sum over this thread's tiles, relative to m_seen
      for (int j = 0; j < n_tiles; ++j, ++cS) {
        const int owner = cS & 1;
        if (owner != hlf) continue;
        const int sb = cS % NSB;
        WAIT3S(&mi.s_full[owner][sb], full_par(cS / NSB), W3_SFULL);
        tc_fence_after_sync();
        const uint32_t tS = cx.tmem + sb * TILE + lane_sel;
        uint32_t s[4][32];
#pragma unroll
        for (int q = 0; q < 4; ++q) tmem_ld32(tS + q * 32, s[q]);
        tmem_wait_ld();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(map_to_cta(&mi.s_read[sb], 0));   // Q K^T of this warpgroup's next tile may start
        // visible keys of this tile: all but the tail of the last cache tile; the window tile is causal
        const int vis = j < n_cache ? prm.Nk - j * TILE : wi + 1;
        if (vis < TILE) {
#pragma unroll
          for (int q = 0; q < 4; ++q)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (q * 32 + i >= vis) s[q][i] = 0xFF800000u;              // -inf
        }
        float mq[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float a = fmax3(__uint_as_float(s[q][0]), __uint_as_float(s[q][1]), __uint_as_float(s[q][2]));
#pragma unroll
          for (int i = 3; i < 31; i += 2) a = fmax3(a, __uint_as_float(s[q][i]), __uint_as_float(s[q][i + 1]));
          mq[q] = fmaxf(a, __uint_as_float(s[q][31]));
        }
        const float m_tile = fmaxf(fmaxf(mq[0], mq[1]), fmaxf(mq[2], mq[3])) * scale_log2;
        float m_prev = -INFINITY;
        if (j > 0) {                                           // the partner's publication of tile j-1
          WAIT3S(&mi.m_pub[hlf ^ 1][warp & 3], full_par(n_pub_other), W3_MPUB);
          ++n_pub_other;
          m_prev = mi.mref[(j - 1) & 1][r];
        }
        const bool first_tile = (j == 0);
        const bool raise = first_tile || (m_tile > m_prev + LAZY_RESCALE);
        const float m_new = raise ? fmaxf(m_prev, m_tile) : m_prev;
        mi.mref[j & 1][r] = m_new;
        __syncwarp();
        if (lane == 0) mbar_arrive(&mi.m_pub[hlf][warp & 3]);     // the warp with the same rows may decide tile j+1
        ++n_pub_mine;
        if (m_new != m_seen) {                                 // bring this thread's partial sum to the new reference
          l_run *= (m_seen == -INFINITY) ? 0.0f : fast_exp2(m_seen - m_new);
          m_seen = m_new;
        }
        if (!first_tile && __any_sync(0xFFFFFFFFu, raise)) {
          // rare: rescale the accumulator rows of this warp.  P V of tile j-1 may still be running: wait for it;
          // P V of tile j cannot start before this thread publishes P.
          const float alpha = (m_prev == -INFINITY) ? 0.0f : fast_exp2(m_prev - m_new);
          const uint32_t prev = cS - 1;
          WAIT3S(&mi.v_free[prev % NVS], full_par(prev / NVS), W3_PVDONE);   // committed after P V of tile `prev`
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
          WAIT3S(&mi.v_free[prev2 % NVS], full_par(prev2 / NVS), W3_PVDONE);
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
            p0 = fast_exp2(x0);                                  // MUFU pipe
            p1 = fast_exp2(x1);
            sum2[i & 1] = add_f32x2(sum2[i & 1], pack_f32x2(p0, p1));
            packed[i] = pack_bf16x2(p0, p1);
          }
          tmem_st16(cx.tmem + TM_P + hlf * 64 + q * 16 + lane_sel, packed);   // P: 64 bf16 columns
          if (q == 1) {                                        // keys 0..63 are final: P V may start on them
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
      // the warpgroup that did not own the last tile consumes its owner's publication; then both bring
      // their partial sums to the final reference maximum
      {
        const int last_owner = (cS - 1) & 1;
        if (hlf != last_owner) {
          WAIT3S(&mi.m_pub[hlf ^ 1][warp & 3], full_par(n_pub_other), W3_MPUB);
          ++n_pub_other;
        }
        const float m_fin = mi.mref[(n_tiles - 1) & 1][r];
        if (m_fin != m_seen) {
          l_run *= (m_seen == -INFINITY) ? 0.0f : fast_exp2(m_seen - m_fin);
          m_seen = m_fin;
        }
      }
      finish_store();
      // ---- epilogue: combine the two partial row sums, normalise, stage bf16 rows in this item's (now idle)
      // Q buffer, TMA store (one box per head: its w window rows)
      WAIT3S(&mi.o_full, full_par(n_done), W3_OFULL);
      ++n_done;
      tc_fence_after_sync();
      mi.xl[hlf][r] = l_run;
      named_barrier_sync(1, 256);
      const float l_tot = mi.xl[0][r] + mi.xl[1][r];
      const float inv_l = 1.0f / l_tot;
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
              pk[e] = pack_bf16x2(__uint_as_float(o[g4 * 8 + 2 * e]) * inv_l, __uint_as_float(o[g4 * 8 + 2 * e + 1]) * inv_l);
            *reinterpret_cast<uint4*>(myQ + hlf * 16384 + sw128_offset(r, q * 4 + g4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(a_acc_free);
      if (hlf == 0 && prm.lse_out)
        prm.lse_out[((size_t)it.seq * prm.Hq + h) * prm.w + wi] = (m_seen + log2f(l_tot)) * 0.6931471805599453f;
      fence_proxy_async_smem();
      named_barrier_sync(1, 256);
      if (tid == 0) {
        for (int i = 0; i < prm.hpc; ++i)
          for (int a = 0; a < 2; ++a)
            tma_store_4d(&tm_o, myQ + a * 16384 + i * prm.w * 128, a * 64, it.h0 + (int)rank * prm.hpc + i, 0, it.seq);
        tma_store_commit();
        store_pending = qb;                                  // released by finish_store() once the store has read it
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
    // commit to mma_done (three arrivals in both CTAs).  The wait ignores the abort flag and is bounded.
    mbar_wait_drain(&mi.mma_done, 0, cx.abort_flag);
    tc_fence_after_sync();
    tmem_dealloc_pair(cx.tmem, 512);
  }
}

// maps: 0 rotated q (box 64 x 1 head x w), 1 out (same box, store), 2 cache keys (64 x 64 keys), 3 cache values
// (64 x 128 keys), 4 window keys (64 x 1 head x 64 tokens), 5 window values (64 x 1 head x 128 tokens).
cudaError_t launch_parallel_pair(const CUtensorMap* maps, const ParallelPairParams& prm, int sm_count, cudaStream_t st) {
  if (cudaError_t e = cudaFuncSetAttribute(parallel_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM3_BYTES); e != cudaSuccess) return e;
  if (prm.hpc < 1 || prm.hpc * prm.w != TILE || prm.n_rg < 1) return cudaErrorInvalidValue;
  const long long n_items = (long long)prm.B * prm.Hkv * prm.n_rg;
  long long pairs = sm_count / 2;
  if (pairs > n_items) pairs = n_items;
  if (pairs < 1) return cudaErrorInvalidConfiguration;
  note_launch();
  parallel_pair_kernel<<<(unsigned)(2 * pairs), NT2, SMEM3_BYTES, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], prm);
  return cudaGetLastError();
}

}  // namespace pc
