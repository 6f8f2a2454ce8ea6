"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot run the bulk attention of a 128K workload in seconds, so bulk outputs are checked on
sampled rows the oracle computes one by one; everything on the window path (scores, ranking, gather,
global attention) is checked in full or through properties that hold at any size.
"""
import numpy as np
import pytest
import torch

import pc_inputs
from oracle import parallelcomp_oracle as orc
from tests.gpu_util import to_dev, to_bits, to_f64, check_attention_output, check_scores

pytestmark = pytest.mark.gpu


def _check_prefill_workload(name, n_row_samples=48, n_groups=2):
    import paper_2502_14317_b200 as pc
    cfg = pc_inputs.get_config(name)
    inp = pc_inputs.make_prefill_inputs(cfg)
    q, k, v = inp["q"], inp["k"], inp["v"]
    C, L, w, G, d = cfg.C, cfg.L, cfg.w, cfg.G, cfg.d
    dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
    res = pc.hot_path(dq, dk, dv, w=w, rope_theta=cfg.rope_theta, m=cfg.m, k_keep=cfg.k)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 0
    scale = 1.0 / np.sqrt(d)
    rng = np.random.default_rng(1234)

    # --- Eq. 6 invariant on every (chunk, kv-head): G*w softmax rows, each summing to 1
    S_gpu = res["win_score"].cpu().numpy()
    assert np.allclose(S_gpu.sum(-1), G * w, rtol=2e-4)
    assert (S_gpu >= 0).all()

    # --- sampled groups: rotated keys (bit-exact), bulk rows, window scores, LSE
    k_rot_gpu = to_bits(res["k_rot"])
    o_gpu = res["o"]
    win_lse_gpu = res["win_lse"].cpu().numpy()
    groups = [(int(rng.integers(C)), int(rng.integers(cfg.Hkv))) for _ in range(n_groups)]
    groups.append((inp["planted_chunks"][0], 0))
    for (c, hk) in groups:
        qs = q[c:c + 1, :, hk * G:(hk + 1) * G]
        ks, vs = k[c:c + 1, :, hk:hk + 1], v[c:c + 1, :, hk:hk + 1]
        q_rot, k_rot = orc.rope_bf16(qs, cfg.rope_theta), orc.rope_bf16(ks, cfg.rope_theta)
        assert np.array_equal(k_rot_gpu[c, :, hk], k_rot[0, :, 0]), "rotated keys differ"
        S, O_win, LSE_win = orc.window_scores(q_rot, k_rot, vs, w, scale)
        check_scores(S_gpu[c, hk], S[0, 0], G, w, L)
        assert np.abs(win_lse_gpu[c, hk * G:(hk + 1) * G] - LSE_win[0]).max() <= 2e-3
        check_attention_output(to_f64(o_gpu[c, L - w:, hk * G:(hk + 1) * G]), O_win[0], "O window rows")
        # bulk rows: tile edges, the first rows and random rows
        rows = np.unique(np.concatenate([[0, 1, 127, 128, 129, L - w - 1, L - 1],
                                         rng.integers(0, L, size=n_row_samples)]))
        for g in range(G):
            _, O_rows, _ = orc.local_attention_rows(q_rot, k_rot, vs, 0, g, rows, scale)
            got = to_f64(o_gpu[c, torch.from_numpy(rows).cuda(), hk * G + g])
            check_attention_output(got, O_rows, "O sampled rows")

    # --- ranking: bit-exact given the tensors the GPU ranked (all rows)
    score_gpu = res["chunk_score"].cpu().numpy()
    assert np.allclose(score_gpu, orc.chunk_score_from_lse(win_lse_gpu), rtol=1e-5, atol=1e-5)
    kept = orc.select_chunks(score_gpu, cfg.m)
    assert np.array_equal(res["kept"].cpu().numpy(), kept)
    idx = orc.select_tokens(S_gpu, kept, cfg.ctx, cfg.k)
    assert np.array_equal(res["idx"].cpu().numpy(), idx)
    # planted keys survive eviction in every planted chunk that was kept (generator property)
    for pi, pc_ in enumerate(inp["planted_chunks"]):
        if pc_ in kept.tolist():
            r = kept.tolist().index(pc_)
            for hk in range(cfg.Hkv):
                assert set(inp["planted_pos"][pi, hk].tolist()) <= set(idx[r, hk].tolist())

    # --- gather: bit copy of K_rot / V rows (vectorised restatement of the oracle's indexing, checked against
    #     the oracle's own loop on a slice)
    kc, vc, pos = to_bits(res["kc"]), to_bits(res["vc"]), res["pos"].cpu().numpy()
    for r in range(cfg.m):
        for hk in range(cfg.Hkv):
            sl = slice(r * cfg.k, (r + 1) * cfg.k)
            assert np.array_equal(kc[hk, sl], k_rot_gpu[kept[r], idx[r, hk], hk])
            assert np.array_equal(vc[hk, sl], v[kept[r], idx[r, hk], hk])
            assert np.array_equal(pos[hk, sl], idx[r, hk])
    Kc_o, Vc_o, _ = orc.gather_kv(k_rot_gpu, v, kept[:1], idx[:1, :1, :64])
    assert np.array_equal(kc[:1, :64], Kc_o) and np.array_equal(vc[:1, :64], Vc_o)

    # --- global attention over the cache the GPU built, all heads and rows
    Fg, _ = orc.parallel_attention(q[0:1, L - w:], L - w, cfg.rope_theta, None, kc[None], vc[None],
                                   k_rot_gpu[0:1, L - w:], v[0:1, L - w:])
    check_attention_output(to_f64(res["fg"]), Fg, "Fg")


def test_cfg1_llama3_128k():
    _check_prefill_workload("cfg1")


def test_cfg2_llama2_mha_128k():
    _check_prefill_workload("cfg2", n_row_samples=32)


def test_cfg3_stress_256k():
    _check_prefill_workload("cfg3", n_row_samples=24, n_groups=1)


def test_paper_hyperparameters_w8_half_kept():
    """Second workload shape: the paper's own settings (window of 8 tokens, half of each chunk kept, 3 chunks kept)."""
    _check_prefill_workload("paper_w8", n_row_samples=24, n_groups=1)


def test_position_reuse_6k_budget_24k():
    """Second workload shape: 6K chunks (48 key tiles, not a power of two) with a 24K compressed cache."""
    _check_prefill_workload("reuse6k", n_row_samples=24, n_groups=1)


def test_cfg4_batch_of_compressed_caches():
    import paper_2502_14317_b200 as pc
    cfg = pc_inputs.get_config("cfg4")
    inp = pc_inputs.make_parallel_attn_inputs(cfg)
    res = pc.parallel_attn(to_dev(inp["q_win"]), to_dev(inp["k_cache"]), to_dev(inp["v_cache"]), to_dev(inp["k_win"]),
                           to_dev(inp["v_win"]), q_pos0=cfg.q_pos0, rope_theta=cfg.rope_theta, want_lse=True)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 0
    out = to_f64(res["out"])
    lse = res["lse"].cpu().numpy()
    assert np.isfinite(out).all()
    for b in (0, 37, 63):
        s = slice(b, b + 1)
        Fg, LSE = orc.parallel_attention(inp["q_win"][s], cfg.q_pos0, cfg.rope_theta, None, inp["k_cache"][s],
                                         inp["v_cache"][s], inp["k_win"][s], inp["v_win"][s])
        check_attention_output(out[s], Fg, f"Fg seq {b}")
        assert np.abs(lse[s] - LSE).max() <= 2e-3


def test_cfg4_decoding_step_over_the_full_batch():
    """One generation step over the same 64 compressed caches (one query token per sequence, 4.3 GB of K/V): the
    launch configuration the bench times (two key splits, two softmax streams per CTA, merge), every sequence
    against the oracle; then the same step through pc_parallel_attn_append on caches with spare room."""
    import paper_2502_14317_b200 as pc
    cfg = pc_inputs.get_config("cfg4")
    inp = pc_inputs.make_parallel_attn_inputs(cfg)
    q1 = np.ascontiguousarray(inp["q_win"][:, :1])
    k1, v1 = np.ascontiguousarray(inp["k_win"][:, :1]), np.ascontiguousarray(inp["v_win"][:, :1])
    kc, vc = to_dev(inp["k_cache"]), to_dev(inp["v_cache"])
    res = pc.parallel_attn(to_dev(q1), kc, vc, to_dev(k1), to_dev(v1), q_pos0=cfg.q_pos0, rope_theta=cfg.rope_theta,
                           want_lse=True)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 0
    Fg, LSE = orc.parallel_attention(q1, cfg.q_pos0, cfg.rope_theta, None, inp["k_cache"], inp["v_cache"], k1, v1)
    check_attention_output(to_f64(res["out"]), Fg, "Fg, decoding step, 64 sequences")
    assert np.abs(res["lse"].cpu().numpy() - LSE).max() <= 2e-3
    B, Hkv, Nk, d = inp["k_cache"].shape
    cap = Nk + 8
    kcap = torch.zeros((B, Hkv, cap, d), dtype=torch.bfloat16, device="cuda")
    vcap = torch.zeros((B, Hkv, cap, d), dtype=torch.bfloat16, device="cuda")
    kcap[:, :, :Nk].copy_(kc)
    vcap[:, :, :Nk].copy_(vc)
    res2 = pc.parallel_attn_append(to_dev(q1), kcap, vcap, Nk, to_dev(k1), to_dev(v1), q_pos0=cfg.q_pos0,
                                   rope_theta=cfg.rope_theta)
    torch.cuda.synchronize()
    assert int(res2["status"].item()) == 0
    assert torch.equal(res2["out"], res["out"]), "same step, caches with spare room"
    assert np.array_equal(to_bits(kcap[:, :, Nk]), k1[:, 0]) and np.array_equal(to_bits(vcap[:, :, Nk]), v1[:, 0])
    assert int(kcap[:, :, Nk + 1:].abs().max().item()) == 0
