"""GPU parity: pc_parallel_attn (Eq. 9-11) and the chained five-call path against the oracle."""
import numpy as np
import pytest
import torch

import pc_inputs
from oracle import parallelcomp_oracle as orc
from tests.gpu_util import to_dev, to_bits, to_f64, check_attention_output, check_scores

pytestmark = pytest.mark.gpu


def _bits(rng, shape):
    return pc_inputs.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


@pytest.mark.parametrize("B,w,Hq,Hkv,d,Nk,q_pos0,theta", [
    (2, 16, 4, 2, 64, 128, 240, 1e4),         # cfg0-like compressed cache
    (1, 64, 8, 2, 128, 1000, 8128, 5e5),      # ragged last cache tile, G*w = 256 rows (both blocks)
    (1, 64, 32, 8, 128, 4096, 8128, 5e5),     # B = 1: keys split across CTAs + merge kernel
    (3, 8, 2, 2, 64, 300, 4088, 1e4),         # MHA, smallest window, one block
    (1, 64, 8, 1, 128, 700, 8128, 5e5),       # G*w = 512 rows: two row groups per kv-head
    (2, 128, 2, 1, 64, 77, 0, 1e4),           # cache shorter than one tile, widest window
    (1, 32, 6, 2, 128, 2049, 100, 1e4),       # G = 3, one key past a tile boundary
    (2, 1, 8, 2, 128, 3000, 8191, 5e5),       # decoding step: one query token over the cache (+ its own key)
    (3, 2, 4, 4, 64, 500, 4094, 1e4),         # two query tokens, MHA
    (1, 4, 32, 8, 128, 16384, 8188, 5e5),     # four query tokens over a 16K cache, Llama-3 heads
    (2, 4, 8, 2, 128, 50, 77, 1e4),           # rows fill one block: two streams; one cache tile to one, the window tile to the other
    (5, 1, 4, 4, 64, 128, 4095, 1e4),         # decoding, MHA, head size 64, cache of exactly one tile
    (1, 16, 8, 2, 128, 5000, 300, 5e5),       # 64 rows per kv-head, 40 cache tiles split over the CTAs, two streams each
    # batches whose 256-row groups fill the CTA pairs (head size 128, G*w a multiple of 256): the pair kernel
    (8, 64, 32, 8, 128, 300, 8128, 5e5),      # 64 groups, ragged last cache tile
    (15, 64, 32, 8, 128, 256, 8128, 5e5),     # 120 groups: two rounds per pair, cache of whole tiles
    (28, 32, 16, 2, 128, 520, 100, 1e4),      # G = 8, w = 32: four heads per CTA
    (16, 128, 8, 2, 128, 130, 0, 1e4),        # G*w = 512: two groups per kv-head, one head per CTA, two keys in the last tile
    (60, 8, 32, 1, 128, 129, 5, 1e4),         # smallest window of that kernel: sixteen heads per CTA
])
def test_parallel_attn_shapes(B, w, Hq, Hkv, d, Nk, q_pos0, theta):
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(Nk + w)
    qw = _bits(rng, (B, w, Hq, d))
    kc, vc = _bits(rng, (B, Hkv, Nk, d)), _bits(rng, (B, Hkv, Nk, d))
    kw, vw = _bits(rng, (B, w, Hkv, d)), _bits(rng, (B, w, Hkv, d))
    kc[:, :, 0] = pc_inputs.f32_to_bf16_bits(pc_inputs.bf16_bits_to_f32(kc[:, :, 0]) * np.float32(4.0))
    res = pc.parallel_attn(to_dev(qw), to_dev(kc), to_dev(vc), to_dev(kw), to_dev(vw), q_pos0=q_pos0,
                           rope_theta=theta, want_lse=True)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 0
    Fg, LSE = orc.parallel_attention(qw, q_pos0, theta, None, kc, vc, kw, vw)
    check_attention_output(to_f64(res["out"]), Fg, "Fg")
    assert np.abs(res["lse"].cpu().numpy() - LSE).max() <= 2e-3


@pytest.mark.parametrize("B,Hq,Hkv,d,Nk0,cap,steps", [
    (2, 8, 2, 128, 250, 260, (1, 1, 4, 1)),   # crosses a tile boundary of the cache (256) while generating
    (3, 4, 4, 64, 40, 48, (1, 2, 1)),         # MHA, head size 64
])
def test_generation_steps_append_to_the_cache(B, Hq, Hkv, d, Nk0, cap, steps):
    """pc_parallel_attn_append in a loop: every step attends over the entries valid so far (oracle on the same prefix)
    and leaves its new keys / values behind them; entries further back stay as they were."""
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(cap)
    kc, vc = _bits(rng, (B, Hkv, cap, d)), _bits(rng, (B, Hkv, cap, d))    # entries >= Nk0: junk that must never be read
    k_dev, v_dev = to_dev(kc), to_dev(vc)
    n, pos, theta = Nk0, 1000, 1e4
    for w in steps:
        qw = _bits(rng, (B, w, Hq, d))
        kw, vw = _bits(rng, (B, w, Hkv, d)), _bits(rng, (B, w, Hkv, d))
        res = pc.parallel_attn_append(to_dev(qw), k_dev, v_dev, n, to_dev(kw), to_dev(vw), q_pos0=pos, rope_theta=theta,
                                      want_lse=True)
        torch.cuda.synchronize()
        assert int(res["status"].item()) == 0
        Fg, LSE = orc.parallel_attention(qw, pos, theta, None, np.ascontiguousarray(kc[:, :, :n]),
                                         np.ascontiguousarray(vc[:, :, :n]), kw, vw)
        check_attention_output(to_f64(res["out"]), Fg, f"Fg over {n} entries, {w} new")
        assert np.abs(res["lse"].cpu().numpy() - LSE).max() <= 2e-3
        kc[:, :, n:n + w] = kw.transpose(0, 2, 1, 3)
        vc[:, :, n:n + w] = vw.transpose(0, 2, 1, 3)
        assert np.array_equal(to_bits(k_dev), kc) and np.array_equal(to_bits(v_dev), vc), "cache after the append"
        n += w
        pos += w
    # a step that does not fit is refused before anything is launched
    lib = pc.load_library()
    assert lib.pc_parallel_attn_append(B, 1, Hq, Hkv, d, cap, cap, None, 0, 1e4, 0.0, None, None, None, None, None, None,
                                       None, None, 0, None) == -1


def test_cfg4_slice():
    """The batch-of-compressed-caches workload at a size the oracle finishes in seconds: 2 of the 64
    sequences, full Nk = 16384 (128 key tiles), same generator."""
    import paper_2502_14317_b200 as pc
    cfg = pc_inputs.get_config("cfg4")
    inp = pc_inputs.make_parallel_attn_inputs(cfg, B=2)
    res = pc.parallel_attn(to_dev(inp["q_win"]), to_dev(inp["k_cache"]), to_dev(inp["v_cache"]), to_dev(inp["k_win"]),
                           to_dev(inp["v_win"]), q_pos0=cfg.q_pos0, rope_theta=cfg.rope_theta, want_lse=True)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 0
    Fg, LSE = orc.parallel_attention(inp["q_win"], cfg.q_pos0, cfg.rope_theta, None, inp["k_cache"], inp["v_cache"],
                                     inp["k_win"], inp["v_win"])
    check_attention_output(to_f64(res["out"]), Fg, "Fg")
    assert np.abs(res["lse"].cpu().numpy() - LSE).max() <= 2e-3


def test_cfg0_whole_path(cfg0_inputs, cfg0_oracle):
    """All five calls chained on one stream; every stage compared with the oracle."""
    import paper_2502_14317_b200 as pc
    cfg, inp = cfg0_inputs
    ref = cfg0_oracle
    q, k, v = to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"])
    res = pc.hot_path(q, k, v, w=cfg.w, rope_theta=cfg.rope_theta, m=cfg.m, k_keep=cfg.k)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 0
    check_attention_output(to_f64(res["o"]), ref["O"])
    S_gpu = res["win_score"].cpu().numpy()
    check_scores(S_gpu, ref["S"], cfg.G, cfg.w, cfg.L)
    assert np.array_equal(to_bits(res["k_rot"]), ref["k_rot"])
    score_gpu = res["chunk_score"].cpu().numpy()
    assert np.allclose(score_gpu, ref["chunk_score"], atol=2e-3)
    # ranking and gather: bit-exact given the tensors the GPU ranked
    kept = orc.select_chunks(score_gpu, cfg.m)
    assert np.array_equal(res["kept"].cpu().numpy(), kept)
    idx = orc.select_tokens(S_gpu, kept, cfg.ctx, cfg.k)
    assert np.array_equal(res["idx"].cpu().numpy(), idx)
    Kc, Vc, pos = orc.gather_kv(ref["k_rot"], inp["v"], kept, idx)
    assert np.array_equal(to_bits(res["kc"]), Kc) and np.array_equal(to_bits(res["vc"]), Vc)
    assert np.array_equal(res["pos"].cpu().numpy(), pos)
    # global attention over the cache the GPU built
    L, w = cfg.L, cfg.w
    Fg, _ = orc.parallel_attention(inp["q"][0:1, L - w:], L - w, cfg.rope_theta, None, Kc[None], Vc[None],
                                   ref["k_rot"][0:1, L - w:], inp["v"][0:1, L - w:])
    check_attention_output(to_f64(res["fg"])[0], Fg[0], "Fg")
    # end to end the oracle made the same eviction decisions on this input
    assert np.array_equal(kept, ref["kept"])
    assert np.array_equal(idx, ref["idx"])
    check_attention_output(to_f64(res["fg"])[0], ref["Fg"], "Fg end-to-end")
    # planted keys survive (generator property)
    r = kept.tolist().index(2)
    for hk in range(cfg.Hkv):
        assert set(inp["planted_pos"][0, hk].tolist()) <= set(idx[r, hk].tolist())


def test_single_chunk_keep_all_equals_local_attention():
    """C = 1, keep everything: the global output equals the window rows of the local attention."""
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(11)
    C, L, Hq, Hkv, d, w = 1, 400, 4, 2, 64, 16
    q, k, v = _bits(rng, (C, L, Hq, d)), _bits(rng, (C, L, Hkv, d)), _bits(rng, (C, L, Hkv, d))
    res = pc.hot_path(to_dev(q), to_dev(k), to_dev(v), w=w, rope_theta=1e4, m=1, k_keep=L - w)
    torch.cuda.synchronize()
    o_win = to_f64(res["o"])[0, L - w:]
    fg = to_f64(res["fg"])[0]
    assert np.abs(o_win - fg).max() <= 1e-2          # two bf16 roundings of the same quantity
    O, _, _ = orc.local_attention(q, k, v, 1e4)
    check_attention_output(fg, O[0, L - w:], "Fg vs full causal attention")


def test_hot_path_from_host_matches_device_path(cfg0_inputs):
    """Uploading the chunks in groups on a copy stream must give exactly what the all-on-device path gives."""
    import paper_2502_14317_b200 as pc
    cfg, inp = cfg0_inputs
    pin = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    hq, hk, hv = pin(inp["q"]), pin(inp["k"]), pin(inp["v"])
    ref = pc.hot_path(hq.cuda(), hk.cuda(), hv.cuda(), w=cfg.w, rope_theta=cfg.rope_theta, m=cfg.m, k_keep=cfg.k)
    buffers = {}
    for _ in range(2):                                            # second call reuses buffers, streams and events
        got = pc.hot_path_from_host(hq, hk, hv, w=cfg.w, rope_theta=cfg.rope_theta, m=cfg.m, k_keep=cfg.k, n_groups=3,
                                    buffers=buffers)
        torch.cuda.synchronize()
        assert int(got["status"].item()) == 0
        for key in ("o", "k_rot", "win_score", "win_lse", "kept", "idx", "kc", "vc", "fg"):
            assert torch.equal(got[key], ref[key]), key
