"""GPU parity: ranking and gather kernels are bit-exact against the oracle on the same inputs."""
import numpy as np
import pytest
import torch

import pc_inputs
from oracle import parallelcomp_oracle as orc
from tests.gpu_util import to_dev, to_bits

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("C,m", [(4, 2), (16, 8), (32, 12), (32, 4), (1, 1), (1000, 37), (1024, 1024)])
def test_select_chunks(C, m):
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(C + m)
    for trial in range(3):
        s = rng.standard_normal(C).astype(np.float32)
        if trial == 1:
            s = np.round(s * 2) / 2                              # many ties
        if trial == 2 and C > 4:
            s[rng.integers(0, C, size=3)] = np.nan
            s[0] = -0.0
            s[1] = 0.0
        for lower in (True, False):
            got = pc.select_chunks(_dev(s), m, lower).cpu().numpy()
            assert np.array_equal(got, orc.select_chunks(s, m, lower)), (C, m, trial, lower)


def test_chunk_score_from_lse():
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(0)
    lse = rng.standard_normal((16, 32, 64)).astype(np.float32) * 3 + 5
    got = pc.chunk_score_from_lse(_dev(lse)).cpu().numpy()
    ref = orc.chunk_score_from_lse(lse)
    assert np.allclose(got, ref, rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("C,Hkv,L,w,k,m", [
    (4, 2, 256, 16, 64, 2),          # cfg0 shape
    (3, 8, 8192, 64, 2048, 2),       # cfg1 row shape
    (3, 4, 4096, 64, 1024, 3),       # cfg2 row shape
    (2, 2, 8192, 64, 512, 1),        # cfg3 row shape
    (2, 3, 1000, 8, 1, 2),           # k = 1
    (2, 1, 777, 8, 768, 2),          # k = n_cand - 1
    (2, 2, 300, 16, 284, 2),         # k = n_cand: identity
    (1, 2, 100, 4, 120, 1),          # k > n_cand: padding with -1
    (1, 1, 32768, 8, 5000, 1),       # largest supported row
    (2, 2, 20000, 64, 12000, 2),     # k too large for the staged output: direct ordered stores
    (1, 1, 32768, 8, 32000, 1),      # the same at the largest row
])
def test_select_tokens(C, Hkv, L, w, k, m):
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(L + k)
    n_cand = L - w
    kept = np.sort(rng.choice(C, size=m, replace=False)).astype(np.int32)
    for trial in range(4):
        S = rng.random((C, Hkv, L)).astype(np.float32) ** 8              # peaky, like attention mass
        if trial == 1:
            S = (np.floor(S * 16) / 16).astype(np.float32)               # heavy ties, many exact zeros
        if trial == 2:
            S[:] = 0.25                                                  # all equal -> lowest positions
        if trial == 3:
            S[:, :, ::97] = np.nan
            S[:, :, 5::101] = -0.0
            S[:, :, 7::103] = np.inf
            S[:, :, 9::107] = -1.0
        got = pc.select_tokens(_dev(S), _dev(kept), n_cand, k).cpu().numpy()
        ref = orc.select_tokens(S, kept, n_cand, k)
        assert np.array_equal(got, ref), (trial, np.argwhere(got != ref)[:5])


@pytest.mark.parametrize("C,L,Hkv,d,m,k", [(4, 256, 2, 64, 2, 64), (3, 1024, 8, 128, 2, 300), (2, 130, 3, 128, 2, 7)])
def test_gather(C, L, Hkv, d, m, k):
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(L)
    k_rot = rng.integers(0, 65536, size=(C, L, Hkv, d)).astype(np.uint16)
    v = rng.integers(0, 65536, size=(C, L, Hkv, d)).astype(np.uint16)
    kept = np.sort(rng.choice(C, size=m, replace=False)).astype(np.int32)
    idx = np.stack([[np.sort(rng.choice(L - 8, size=k, replace=False)) for _ in range(Hkv)] for _ in range(m)]).astype(np.int32)
    idx[-1, -1, -2:] = -1                                                  # padded entries
    kc, vc, pos = pc.gather_kv(to_dev(k_rot), to_dev(v), _dev(kept), _dev(idx))
    Kc, Vc, P = orc.gather_kv(k_rot, v, kept, idx)
    assert np.array_equal(to_bits(kc), Kc) and np.array_equal(to_bits(vc), Vc)
    assert np.array_equal(pos.cpu().numpy(), P)
    # head-major source through strides
    kh = to_dev(k_rot).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vh = to_dev(v).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    kc2, vc2, _ = pc.gather_kv(kh, vh, _dev(kept), _dev(idx))
    assert np.array_equal(to_bits(kc), to_bits(kc2)) and np.array_equal(to_bits(vc), to_bits(vc2))   # bits: random patterns include NaN


def test_keep_all_gather_is_a_reshape():
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(5)
    C, L, Hkv, d, w = 3, 200, 2, 64, 8
    ctx = L - w
    k_rot = rng.integers(0, 65536, size=(C, L, Hkv, d)).astype(np.uint16)
    S = rng.random((C, Hkv, L)).astype(np.float32)
    kept = pc.select_chunks(_dev(np.zeros(C, np.float32)), C, True)
    idx = pc.select_tokens(_dev(S), kept, ctx, ctx)
    kc, vc, pos = pc.gather_kv(to_dev(k_rot), to_dev(k_rot), kept, idx)
    assert np.array_equal(to_bits(kc), k_rot[:, :ctx].transpose(2, 0, 1, 3).reshape(Hkv, C * ctx, d))


@pytest.mark.parametrize("C,m,L,w,k,Hkv,n_s,n_r,lams", [
    (3, 2, 600, 8, 100, 2, 100, 100, (0.6, 0.9, 0.4)),          # all three regions active
    (2, 2, 300, 16, 284, 2, 10, 20, (0.5, 0.5, 0.5)),           # k = n_cand: survivors only, -1 padding
    (2, 1, 8192, 64, 2048, 8, 100, 100, (float("inf"), 0.97, float("inf"))),   # workload row shape, middle peaks only
    (1, 1, 200, 8, 50, 1, 150, 150, (0.2, 0.3, 0.4)),           # overlapping regions: the sink region wins
    (2, 2, 400, 8, 30, 2, 100, 100, (0.0, 0.0, 0.0)),           # everything above the thresholds: all -1
    (1, 1, 16000, 64, 11000, 2, 100, 100, (0.9, 0.95, 0.9)),    # k too large for the staged output
    (2, 2, 500, 12, 80, 2, 10 ** 6, 7, (0.7, 0.2, 0.3)),         # sink region larger than the row: it is the whole row
    (1, 1, 300, 8, 40, 2, 3, 2 ** 31 - 1, (0.5, 0.2, 0.6)),      # recency region 'everything' (largest int32)
])
def test_select_tokens_calibrated(C, m, L, w, k, Hkv, n_s, n_r, lams):
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(L + k)
    S = rng.random((C, Hkv, L)).astype(np.float32)
    S[:, :, 0] = 50.0                                            # a sink peak
    S[:, :, 5] = np.float32(lams[0]) if np.isfinite(lams[0]) else 0.5   # exactly at the threshold: kept
    S[0, 0, 7] = np.nan
    kept = np.sort(rng.choice(C, size=m, replace=False)).astype(np.int32)
    got = pc.select_tokens_calibrated(torch.from_numpy(S).cuda(), torch.from_numpy(kept).cuda(), L - w, k, n_s=n_s,
                                      n_r=n_r, lambda_s=lams[0], lambda_m=lams[1], lambda_r=lams[2])
    torch.cuda.synchronize()
    ref = orc.select_tokens_calibrated(S, kept, L - w, k, n_s, n_r, *lams)
    assert np.array_equal(got.cpu().numpy(), ref)
    # thresholds at +inf: the calibrated entry point is pc_select_tokens
    inf = float("inf")
    a = pc.select_tokens_calibrated(torch.from_numpy(S).cuda(), torch.from_numpy(kept).cuda(), L - w, k, n_s=n_s, n_r=n_r,
                                    lambda_s=inf, lambda_m=inf, lambda_r=inf)
    b = pc.select_tokens(torch.from_numpy(S).cuda(), torch.from_numpy(kept).cuda(), L - w, k)
    assert torch.equal(a, b)


@pytest.mark.parametrize("C,Hq,w,m", [(16, 32, 64, 8), (4, 4, 16, 2), (64, 8, 24, 17), (7, 3, 5, 7), (100, 4, 8, 30)])
def test_score_and_chunk_ranking_in_one_call(C, Hq, w, m):
    """pc_score_select_chunks = pc_chunk_score_from_lse + pc_select_chunks, bit for bit (one launch up to 64 chunks,
    two beyond), and the oracle's selection on that score."""
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(C * 31 + w)
    lse = rng.standard_normal((C, Hq, w)).astype(np.float32) * 3 + 7
    if C > 4:
        lse[3] = lse[1]                                          # a tie between two chunks
    d = _dev(lse)
    score_a = pc.chunk_score_from_lse(d)
    kept_a = pc.select_chunks(score_a, m, True)
    n0 = pc.launch_count()
    score_b, kept_b = pc.score_select_chunks(d, m, True)
    assert pc.launch_count() - n0 == (1 if C <= 64 else 2)
    torch.cuda.synchronize()
    assert torch.equal(score_a.view(torch.int32), score_b.view(torch.int32)) and torch.equal(kept_a, kept_b)
    assert np.array_equal(kept_b.cpu().numpy(), orc.select_chunks(score_b.cpu().numpy(), m, True))
