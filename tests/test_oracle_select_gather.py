"""Pins for the oracle's ranking (Eq. 3-4, Eq. 7), gather (Eq. 9), global attention
(Eq. 10-11) and the whole path (CPU only)."""
import math

import numpy as np
import pytest

import pc_inputs
from oracle import parallelcomp_oracle as orc


def _rand_bits(rng, shape):
    return pc_inputs.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


# --------------------------------------------------------------------------- chunk ranking
def _brute_topm(scores, m, lower=True):
    # selection by repeated scan: pick the best remaining, lowest id on ties
    left = list(range(len(scores)))
    chosen = []
    for _ in range(m):
        best = None
        for c in left:
            s = scores[c]
            if math.isnan(s):
                continue
            if best is None or (s < scores[best] if lower else s > scores[best]):
                best = c
        if best is None:
            best = left[0]
        chosen.append(best)
        left.remove(best)
    return sorted(chosen)


def test_select_chunks_bruteforce_ties_and_streaming():
    rng = np.random.default_rng(0)
    for C, m in ((16, 8), (32, 12), (32, 4), (5, 5), (7, 1)):
        s = rng.standard_normal(C).astype(np.float32)
        assert orc.select_chunks(s, m).tolist() == _brute_topm(s.tolist(), m)
        assert orc.select_chunks(s, m, lower_is_better=False).tolist() == _brute_topm(s.tolist(), m, lower=False)
        for batch in (1, 3, C):
            assert np.array_equal(orc.select_chunks_streaming(s, m, batch), orc.select_chunks(s, m))
    # all equal -> the lowest ids
    assert orc.select_chunks(np.zeros(9, np.float32), 4).tolist() == [0, 1, 2, 3]
    # quantised scores: many ties
    s = (rng.integers(0, 3, size=20)).astype(np.float32)
    assert orc.select_chunks(s, 7).tolist() == _brute_topm(s.tolist(), 7)
    assert np.array_equal(orc.select_chunks_streaming(s, 7, 4), orc.select_chunks(s, 7))
    # NaN ranks worst; -0.0 ties with +0.0
    s = np.array([np.nan, 1.0, -0.0, 0.0, np.nan, -1.0], dtype=np.float32)
    assert orc.select_chunks(s, 3).tolist() == [2, 3, 5]
    assert orc.select_chunks(s, 2).tolist() == [2, 5]
    assert orc.select_chunks(s, 5).tolist() == [0, 1, 2, 3, 5]


# --------------------------------------------------------------------------- token ranking
def _brute_topk_row(row, k):
    chosen = []
    left = list(range(len(row)))
    for _ in range(min(k, len(row))):
        best = None
        for j in left:
            if math.isnan(row[j]):
                continue
            if best is None or row[j] > row[best]:
                best = j
        if best is None:
            best = left[0]
        chosen.append(best)
        left.remove(best)
    return sorted(chosen)


def test_select_tokens_bruteforce_identity_ties_padding():
    rng = np.random.default_rng(1)
    C, Hkv, L, w = 5, 3, 40, 6
    S = rng.random((C, Hkv, L)).astype(np.float32)
    kept = np.array([1, 3, 4], dtype=np.int32)
    idx = orc.select_tokens(S, kept, L - w, 10)
    assert idx.shape == (3, Hkv, 10) and idx.dtype == np.int32
    for r, c in enumerate(kept):
        for hk in range(Hkv):
            assert idx[r, hk].tolist() == _brute_topk_row(S[c, hk, :L - w].tolist(), 10)
            assert np.all(np.diff(idx[r, hk]) > 0)
    # window keys are never candidates even if their scores are the largest
    S2 = S.copy()
    S2[:, :, L - w:] = 100.0
    assert np.array_equal(orc.select_tokens(S2, kept, L - w, 10), idx)
    # k = n_cand -> identity
    full = orc.select_tokens(S, kept, L - w, L - w)
    assert np.array_equal(full, np.broadcast_to(np.arange(L - w, dtype=np.int32), full.shape))
    # ties -> lowest positions
    Sq = np.floor(S * 4).astype(np.float32)
    idq = orc.select_tokens(Sq, kept, L - w, 9)
    for r, c in enumerate(kept):
        for hk in range(Hkv):
            assert idq[r, hk].tolist() == _brute_topk_row(Sq[c, hk, :L - w].tolist(), 9)
    # k > n_cand -> all candidates then -1
    pad = orc.select_tokens(S, kept, L - w, L - w + 3)
    assert np.array_equal(pad[..., :L - w], full) and np.all(pad[..., L - w:] == -1)
    # NaN worst, zeros of either sign tie
    row = np.array([[[0.0, np.nan, -0.0, 0.5, np.nan, 0.0]]], dtype=np.float32)
    assert orc.select_tokens(row, np.array([0]), 6, 3)[0, 0].tolist() == [0, 2, 3]
    assert orc.select_tokens(row, np.array([0]), 6, 5)[0, 0].tolist() == [0, 1, 2, 3, 5]


# --------------------------------------------------------------------------- gather
def test_gather_identity_and_indexing():
    rng = np.random.default_rng(2)
    C, L, Hkv, d, w = 3, 10, 2, 4, 2
    ctx = L - w
    k_rot = rng.integers(0, 65536, size=(C, L, Hkv, d)).astype(np.uint16)
    v = rng.integers(0, 65536, size=(C, L, Hkv, d)).astype(np.uint16)
    kept = np.arange(C, dtype=np.int32)
    idx = np.broadcast_to(np.arange(ctx, dtype=np.int32), (C, Hkv, ctx)).copy()
    Kc, Vc, pos = orc.gather_kv(k_rot, v, kept, idx)
    # keep everything: the cache is the context part of K, head-major
    assert np.array_equal(Kc, k_rot[:, :ctx].transpose(2, 0, 1, 3).reshape(Hkv, C * ctx, d))
    assert np.array_equal(Vc, v[:, :ctx].transpose(2, 0, 1, 3).reshape(Hkv, C * ctx, d))
    assert np.array_equal(pos, np.tile(np.arange(ctx), (Hkv, C)))
    # explicit entries, different per head
    kept = np.array([2, 0], dtype=np.int32)
    idx = np.array([[[1, 5], [0, 7]], [[3, 4], [2, -1]]], dtype=np.int32)
    Kc, Vc, pos = orc.gather_kv(k_rot, v, kept, idx)
    assert np.array_equal(Kc[0, 0], k_rot[2, 1, 0]) and np.array_equal(Kc[0, 1], k_rot[2, 5, 0])
    assert np.array_equal(Kc[1, 1], k_rot[2, 7, 1]) and np.array_equal(Vc[0, 3], v[0, 4, 0])
    assert np.array_equal(Vc[1, 2], v[0, 2, 1])
    assert np.all(Kc[1, 3] == 0) and np.all(Vc[1, 3] == 0) and pos[1, 3] == -1
    assert pos.tolist() == [[1, 5, 3, 4], [0, 7, 2, -1]]


# --------------------------------------------------------------------------- global attention
def test_single_chunk_keep_all_equals_full_causal_attention():
    rng = np.random.default_rng(3)
    C, L, Hq, Hkv, d, w = 1, 24, 4, 2, 8, 5
    q, k, v = _rand_bits(rng, (C, L, Hq, d)), _rand_bits(rng, (C, L, Hkv, d)), _rand_bits(rng, (C, L, Hkv, d))
    out = orc.hot_path(q, k, v, w=w, theta=10000.0, m=1, k=L - w)
    assert np.allclose(out["Fg"], out["O"][0, L - w:], atol=1e-13)
    assert np.allclose(out["LSEg"], out["LSE"][0, :, L - w:], atol=1e-13)
    assert np.allclose(out["O_win"], out["O"][:, L - w:], atol=1e-13)


def test_parallel_attention_invariants():
    rng = np.random.default_rng(4)
    B, w, Hq, Hkv, d, Nk = 2, 4, 4, 2, 8, 19
    qw = _rand_bits(rng, (B, w, Hq, d))
    kc, vc = _rand_bits(rng, (B, Hkv, Nk, d)), _rand_bits(rng, (B, Hkv, Nk, d))
    kw, vw = _rand_bits(rng, (B, w, Hkv, d)), _rand_bits(rng, (B, w, Hkv, d))
    Fg, LSE = orc.parallel_attention(qw, 100, 10000.0, None, kc, vc, kw, vw)
    # permuting cache entries changes nothing
    perm = rng.permutation(Nk)
    Fg2, LSE2 = orc.parallel_attention(qw, 100, 10000.0, None, kc[:, :, perm], vc[:, :, perm], kw, vw)
    assert np.allclose(Fg, Fg2, atol=1e-13) and np.allclose(LSE, LSE2, atol=1e-13)
    # all values equal -> output is that value
    vconst = np.broadcast_to(vc[:, :, :1], vc.shape).copy()
    vwconst = np.broadcast_to(vc[:, :, 0][:, None], vw.shape).copy()
    Fg3, _ = orc.parallel_attention(qw, 100, 10000.0, None, kc, vconst, kw, vwconst)
    G = Hq // Hkv
    for h in range(Hq):
        assert np.allclose(Fg3[:, :, h], orc.bf16_to_f64(vc[:, h // G, 0])[:, None, :], atol=1e-13)
    # first window row sees the whole cache plus itself only: explicit softmax
    b, h = 1, 3
    qr = orc.bf16_to_f64(orc.rope_bf16(qw, 10000.0, pos0=100))[b, 0, h]
    keys = np.concatenate([orc.bf16_to_f64(kc[b, h // G]), orc.bf16_to_f64(kw[b, :1, h // G])])
    vals = np.concatenate([orc.bf16_to_f64(vc[b, h // G]), orc.bf16_to_f64(vw[b, :1, h // G])])
    logit = keys @ qr / math.sqrt(d)
    p = np.exp(logit - logit.max())
    p /= p.sum()
    assert np.allclose(Fg[b, 0, h], p @ vals, atol=1e-13)
    # splitting the cache into ranges and merging partial results by their LSE gives the same answer
    cut = 7
    empty_k = np.zeros((B, 0, Hkv, d), np.uint16)
    Fa, La = orc.parallel_attention(qw, 100, 10000.0, None, kc[:, :, :cut], vc[:, :, :cut], empty_k, empty_k)
    Fb, Lb = orc.parallel_attention(qw, 100, 10000.0, None, kc[:, :, cut:], vc[:, :, cut:], kw, vw)
    wa = np.exp(La - np.logaddexp(La, Lb)).transpose(0, 2, 1)[..., None]
    assert np.allclose(wa * Fa + (1 - wa) * Fb, Fg, atol=1e-13)
    assert np.allclose(np.logaddexp(La, Lb), LSE, atol=1e-13)
    # n_valid masks padded cache entries
    Fm, _ = orc.parallel_attention(qw, 100, 10000.0, None, kc, vc, kw, vw, n_valid=np.full((B, Hkv), cut))
    Fc, _ = orc.parallel_attention(qw, 100, 10000.0, None, kc[:, :, :cut], vc[:, :, :cut], kw, vw)
    assert np.allclose(Fm, Fc, atol=1e-13)


# --------------------------------------------------------------------------- whole path
def test_eviction_order_commutes_and_chunk_permutation(cfg0_inputs, cfg0_oracle):
    cfg, inp = cfg0_inputs
    a = cfg0_oracle
    b = orc.hot_path(inp["q"], inp["k"], inp["v"], w=cfg.w, theta=cfg.rope_theta, m=cfg.m, k=cfg.k,
                     tokens_first=True, full_local=False)
    for key in ("kept", "idx", "Kc", "Vc", "pos"):
        assert np.array_equal(a[key], b[key]), key
    assert np.allclose(a["Fg"], b["Fg"], atol=0)
    # the global output does not depend on the order in which chunks were laid out
    perm = np.array([2, 0, 3, 1])
    c = orc.hot_path(inp["q"][perm], inp["k"][perm], inp["v"][perm], w=cfg.w, theta=cfg.rope_theta,
                     m=cfg.m, k=cfg.k, full_local=False)
    assert sorted(perm[c["kept"]].tolist()) == a["kept"].tolist()
    assert np.allclose(c["Fg"], a["Fg"], atol=1e-12)


def test_cfg0_structure(cfg0_inputs, cfg0_oracle):
    cfg, inp = cfg0_inputs
    out = cfg0_oracle
    G = cfg.G
    assert np.allclose(out["S"].sum(-1), G * cfg.w, atol=1e-10)
    assert out["idx"].shape == (cfg.m, cfg.Hkv, cfg.k)
    # planted chunk is kept and every planted key survives token eviction (a property of the generator)
    assert inp["planted_chunks"] == [2]
    assert 2 in out["kept"].tolist()
    r = out["kept"].tolist().index(2)
    for hk in range(cfg.Hkv):
        assert set(inp["planted_pos"][0, hk].tolist()) <= set(out["idx"][r, hk].tolist())
        # the sink key is kept in every kept chunk
        for rr in range(cfg.m):
            assert out["idx"][rr, hk, 0] == 0
    # window replicated: every chunk carries the same window tokens
    assert np.array_equal(inp["q"][0, cfg.ctx:], inp["q"][3, cfg.ctx:])
    assert np.array_equal(out["k_rot"][0, cfg.ctx:], out["k_rot"][1, cfg.ctx:])


def test_select_tokens_calibrated_pins():
    """Eq. 8 + Eq. 7.  Pins: thresholds at +inf reduce to Eq. 7; a brute-force loop; hand-made rows with the
    three regions; survivors fewer than k are padded with -1; NaN is never 'above the threshold'."""
    rng = np.random.default_rng(21)
    C, Hkv, L, w = 3, 2, 60, 4
    S = rng.random((C, Hkv, L)).astype(np.float32)
    kept = np.array([0, 2], dtype=np.int32)
    inf = float("inf")
    assert np.array_equal(orc.select_tokens_calibrated(S, kept, L - w, 9, 5, 7, inf, inf, inf),
                          orc.select_tokens(S, kept, L - w, 9))
    # brute force: per row, loop over positions, drop those above their region's threshold, take the k largest
    n_cand, k, n_s, n_r, ls, lm, lr = L - w, 12, 5, 7, 0.5, 0.8, 0.3
    got = orc.select_tokens_calibrated(S, kept, n_cand, k, n_s, n_r, ls, lm, lr)
    for r, c in enumerate(kept):
        for hk in range(Hkv):
            alive = []
            for j in range(n_cand):
                lam = ls if j < n_s else (lr if j >= n_cand - n_r else lm)
                if not (S[c, hk, j] > np.float32(lam)):
                    alive.append(j)
            best = sorted(alive, key=lambda j: (-float(S[c, hk, j]), j))[:k]
            exp = sorted(best) + [-1] * (k - len(best))
            assert got[r, hk].tolist() == exp
    # hand-made row: positions 0..9, n_s = 2, n_r = 3 -> regions s = {0,1}, m = {2..6}, r = {7,8,9}
    row = np.array([[[9.0, 0.1, 5.0, 0.2, 0.3, 6.0, 0.4, 7.0, 0.5, 0.6]]], dtype=np.float32)
    one = np.array([0])
    assert orc.select_tokens_calibrated(row, one, 10, 3, 2, 3, inf, inf, inf)[0, 0].tolist() == [0, 5, 7]
    assert orc.select_tokens_calibrated(row, one, 10, 3, 2, 3, 1.0, inf, inf)[0, 0].tolist() == [2, 5, 7]     # sink evicted
    assert orc.select_tokens_calibrated(row, one, 10, 3, 2, 3, inf, 5.5, inf)[0, 0].tolist() == [0, 2, 7]     # middle peak evicted
    assert orc.select_tokens_calibrated(row, one, 10, 3, 2, 3, inf, inf, 0.55)[0, 0].tolist() == [0, 2, 5]    # recency peaks evicted
    assert orc.select_tokens_calibrated(row, one, 10, 3, 2, 3, 0.0, 0.0, 0.0)[0, 0].tolist() == [-1, -1, -1]  # everything evicted
    few = orc.select_tokens_calibrated(row, one, 10, 6, 2, 3, 0.05, 0.25, 0.45)[0, 0].tolist()
    assert few == [3, -1, -1, -1, -1, -1]                                                                    # only 0.2 survives
    # equality with the threshold is kept (strictly greater is evicted); NaN is kept and ranks last
    row2 = np.array([[[0.5, np.nan, 0.7, 0.5]]], dtype=np.float32)
    assert orc.select_tokens_calibrated(row2, one, 4, 4, 0, 0, inf, 0.5, inf)[0, 0].tolist() == [0, 1, 3, -1]
    assert orc.select_tokens_calibrated(row2, one, 4, 2, 0, 0, inf, 0.5, inf)[0, 0].tolist() == [0, 3]
