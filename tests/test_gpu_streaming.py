"""GPU parity of the online chunk queue (Sec. 3.1 "Chunk eviction") and of the path that streams chunk batches.

The oracle's definition is the offline one - the m best chunks over ALL chunks, then token eviction and
gather on those - plus its own slow online queue; the streamed CUDA path must give the same chunks, the same
indices and the same compressed cache bit for bit, whatever the batch size.
"""
import numpy as np
import pytest
import torch

import pc_inputs
from oracle import parallelcomp_oracle as orc
from tests.gpu_util import to_dev, to_bits, to_f64, check_attention_output

pytestmark = pytest.mark.gpu


def _stream_scores(scores: np.ndarray, m: int, batch: int):
    """Push `scores` through pc_queue_update in batches; returns the final (chunk ids by slot, scores by slot) and
    the per-batch slot_src arrays."""
    import paper_2502_14317_b200 as pc
    st = pc.queue_init(m, 1, 1, 64, torch.device("cuda:0"))
    srcs = []
    for c0 in range(0, len(scores), batch):
        s = torch.from_numpy(scores[c0:c0 + batch].copy()).cuda()
        before = st["q_chunk"].clone()
        pc.queue_update(st, s, c0, True)
        srcs.append((c0, before.cpu().numpy(), st["slot_src"].cpu().numpy().copy(), st["q_chunk"].cpu().numpy().copy()))
    torch.cuda.synchronize()
    return st["q_chunk"].cpu().numpy(), st["q_score"].cpu().numpy(), srcs


@pytest.mark.parametrize("C,m,batch", [(16, 8, 4), (37, 5, 7), (64, 12, 64), (9, 9, 2), (40, 3, 1), (1000, 24, 500)])
def test_queue_update_matches_oracle(C, m, batch):
    rng = np.random.default_rng(C * 131 + m)
    scores = rng.standard_normal(C).astype(np.float32)
    scores[rng.integers(0, C, size=max(1, C // 5))] = scores[0]          # ties
    if C > 10:
        scores[[3, C - 2]] = np.nan                                       # NaN ranks worst
        scores[5] = -0.0
        scores[6] = 0.0
    q_chunk, q_score, steps = _stream_scores(scores, m, batch)
    want = orc.select_chunks_streaming(scores, m, batch)
    assert np.array_equal(np.sort(q_chunk), want)
    assert np.array_equal(want, orc.select_chunks(scores, m))
    # every slot carries the score of its chunk
    assert np.array_equal(q_score.view(np.uint32), scores[q_chunk].view(np.uint32))
    # slot discipline: a chunk that stays keeps its slot; a slot that changes names the batch chunk that moved in
    for c0, before, slot_src, after in steps:
        for s in range(m):
            if slot_src[s] < 0:
                assert after[s] == before[s]
            else:
                assert after[s] == c0 + slot_src[s] and after[s] != before[s]
        moved = slot_src[slot_src >= 0]
        assert len(set(moved.tolist())) == len(moved)
        assert np.all(np.diff(moved) > 0)                                 # ascending chunks into ascending freed slots


def test_queue_with_fewer_chunks_than_slots():
    import paper_2502_14317_b200 as pc
    scores = np.array([0.5, np.nan, -1.0], dtype=np.float32)
    q_chunk, _, _ = _stream_scores(scores, 5, 2)
    assert sorted(q_chunk.tolist()) == [-1, -1, 0, 1, 2]
    # emit: ids ascending, empty places last with zero rows and position -1
    st = pc.queue_init(4, 2, 3, 64, torch.device("cuda:0"))
    pc.queue_update(st, torch.tensor([2.0, 1.0], device="cuda"), 10, True)
    k_src = torch.randn((2, 8, 2, 64), device="cuda").bfloat16()
    v_src = torch.randn((2, 8, 2, 64), device="cuda").bfloat16()
    idx = torch.tensor([[[0, 2, 5], [1, 2, 3]], [[4, 6, 7], [0, 1, -1]]], dtype=torch.int32, device="cuda")
    pc.queue_gather(st, k_src, v_src, idx)
    kept, kc, vc, pos = pc.queue_emit(st)
    torch.cuda.synchronize()
    assert kept.tolist() == [10, 11, -1, -1]
    Kc, Vc, P = orc.gather_kv(to_bits(k_src), to_bits(v_src), np.array([0, 1]), idx.cpu().numpy())
    assert np.array_equal(to_bits(kc)[:, :6], Kc) and np.array_equal(to_bits(vc)[:, :6], Vc)
    assert np.array_equal(pos.cpu().numpy()[:, :6], P)
    assert not to_bits(kc)[:, 6:].any() and not to_bits(vc)[:, 6:].any()
    assert (pos.cpu().numpy()[:, 6:] == -1).all()


def _check_streaming(cfg, inp, batch, chunk_score=None, check_fg=True):
    import paper_2502_14317_b200 as pc
    q, k, v = inp["q"], inp["k"], inp["v"]
    dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
    L, w = cfg.L, cfg.w
    cs = None if chunk_score is None else torch.from_numpy(chunk_score).cuda()
    # the tensors the GPU ranks (all chunks at once), for the oracle to rank as well
    full = pc.hot_path(dq, dk, dv, w=w, rope_theta=cfg.rope_theta, m=cfg.m, k_keep=cfg.k, chunk_score=cs)
    torch.cuda.synchronize()
    score = full["chunk_score"].cpu().numpy()
    S = full["win_score"].cpu().numpy()
    k_rot = to_bits(full["k_rot"])
    kept_o = orc.select_chunks_streaming(score, cfg.m, batch)
    assert np.array_equal(kept_o, orc.select_chunks(score, cfg.m))
    idx_o = orc.select_tokens(S, kept_o, cfg.ctx, cfg.k)

    buffers = {}
    for _ in range(2):                                                    # the second pass reuses queue and buffers
        got = pc.hot_path_streaming(dq, dk, dv, w=w, rope_theta=cfg.rope_theta, m=cfg.m, k_keep=cfg.k, batch=batch,
                                    chunk_score=cs, buffers=buffers)
        torch.cuda.synchronize()
        assert int(got["status"].item()) == 0
        assert np.array_equal(got["kept"].cpu().numpy(), kept_o)
        kc, vc, pos = to_bits(got["kc"]), to_bits(got["vc"]), got["pos"].cpu().numpy()
        for r in range(cfg.m):
            for hk in range(cfg.Hkv):
                sl = slice(r * cfg.k, (r + 1) * cfg.k)
                assert np.array_equal(pos[hk, sl], idx_o[r, hk])
                assert np.array_equal(kc[hk, sl], k_rot[kept_o[r], idx_o[r, hk], hk])
                assert np.array_equal(vc[hk, sl], v[kept_o[r], idx_o[r, hk], hk])
        Kc_o, Vc_o, _ = orc.gather_kv(k_rot, v, kept_o[:1], idx_o[:1, :1, :32])
        assert np.array_equal(kc[:1, :32], Kc_o) and np.array_equal(vc[:1, :32], Vc_o)
        if check_fg:
            Fg, _ = orc.parallel_attention(q[0:1, L - w:], L - w, cfg.rope_theta, None, kc[None], vc[None],
                                           k_rot[0:1, L - w:], v[0:1, L - w:])
            check_attention_output(to_f64(got["fg"]), Fg, "Fg (streamed)")
        # and identical to the path that holds all chunks at once
        for key in ("kept", "kc", "vc", "pos", "fg"):
            assert torch.equal(got[key], full[key]), key


@pytest.mark.parametrize("batch", [1, 2, 3, 4])
def test_streaming_path_cfg0(cfg0_inputs, batch):
    cfg, inp = cfg0_inputs
    _check_streaming(cfg, inp, batch)


def test_streaming_path_cfg0_late_chunks_push_out_early_ones(cfg0_inputs):
    cfg, inp = cfg0_inputs
    _check_streaming(cfg, inp, 1, chunk_score=np.array([4.0, 3.0, 2.0, 1.0], dtype=np.float32))
    _check_streaming(cfg, inp, 2, chunk_score=np.array([1.0, 1.0, 1.0, 1.0], dtype=np.float32))    # ties: lower ids stay


def test_streaming_path_cfg1_batches_of_4():
    cfg = pc_inputs.get_config("cfg1")
    inp = pc_inputs.make_prefill_inputs(cfg)
    rng = np.random.default_rng(7)
    # scores that make every batch change the queue
    _check_streaming(cfg, inp, 4, chunk_score=rng.permutation(cfg.C).astype(np.float32), check_fg=True)


def test_streaming_with_a_shorter_last_chunk(cfg0_inputs):
    """An input whose length is not a multiple of the chunk length: three chunks of 256 tokens and a last one of
    200 (window included).  The short chunk is a batch of its own; its window sits right behind its context, at
    positions 184..199.  The oracle is composed per chunk length from the same pinned pieces."""
    import dataclasses
    import paper_2502_14317_b200 as pc
    cfg, inp = cfg0_inputs
    w, m, kk, theta = cfg.w, 2, cfg.k, cfg.rope_theta
    La, Lb = cfg.L, 200
    scale = 1.0 / np.sqrt(cfg.d)
    cfg_b = dataclasses.replace(cfg, name="tail", C=1, L=Lb, n_planted_chunks=0, seed=cfg.seed + 77, planted_chunks=())
    tail = pc_inputs.make_prefill_inputs(cfg_b)
    qa, ka, va = inp["q"][:3], inp["k"][:3], inp["v"][:3]
    qb, kb, vb = tail["q"].copy(), tail["k"].copy(), tail["v"].copy()
    qb[:, Lb - w:], kb[:, Lb - w:], vb[:, Lb - w:] = qa[:1, La - w:], ka[:1, La - w:], va[:1, La - w:]   # same query tokens
    host = [(qa, ka, va), (qb, kb, vb)]
    dev = [tuple(to_dev(t) for t in b) for b in host]

    # per-batch tensors of the CUDA path, checked against the oracle, then ranked by the oracle as they are
    S_all, krot_all, score_all = [], [], []
    for (q, k, v), (dq, dk, dv) in zip(host, dev):
        L = q.shape[1]
        pre = pc.chunk_prefill_attn(dq, dk, dv, w=w, rope_theta=theta)
        sc = pc.chunk_score_from_lse(pre["win_lse"])
        torch.cuda.synchronize()
        assert int(pre["status"].item()) == 0
        q_rot, k_rot = orc.rope_bf16(q, theta), orc.rope_bf16(k, theta)
        assert np.array_equal(to_bits(pre["k_rot"]), k_rot)
        S, _, LSE_win = orc.window_scores(q_rot, k_rot, v, w, scale)
        S_gpu = pre["win_score"].cpu().numpy()
        d = np.abs(S_gpu - S)
        assert np.all(d <= 1e-3 * np.maximum(S, cfg.G * w / L))
        assert np.allclose(sc.cpu().numpy(), orc.chunk_score_from_lse(LSE_win), atol=2e-3)
        S_all.append(S_gpu)
        krot_all.append(k_rot)
        score_all.append(sc.cpu().numpy())

    for forced in (None, np.array([3.0, 1.0, 4.0, 0.5], dtype=np.float32)):     # second case: the short chunk is kept
        score = np.concatenate(score_all) if forced is None else forced
        kept_o = orc.select_chunks(score, m)
        Kc_o, Vc_o, pos_o = [], [], []
        for c in kept_o:
            bi, local = (0, int(c)) if c < 3 else (1, 0)
            n_cand = host[bi][0].shape[1] - w
            idx = orc.select_tokens(S_all[bi], np.array([local]), n_cand, kk)
            K1, V1, P1 = orc.gather_kv(krot_all[bi], host[bi][2], np.array([local]), idx)
            Kc_o.append(K1); Vc_o.append(V1); pos_o.append(P1)
        Kc_o, Vc_o, pos_o = (np.concatenate(x, axis=1) for x in (Kc_o, Vc_o, pos_o))
        got = pc.hot_path_streaming([b[0] for b in dev], [b[1] for b in dev], [b[2] for b in dev], w=w, rope_theta=theta,
                                    m=m, k_keep=kk, chunk_score=None if forced is None else torch.from_numpy(forced).cuda())
        torch.cuda.synchronize()
        assert int(got["status"].item()) == 0
        assert np.array_equal(got["kept"].cpu().numpy(), kept_o)
        assert np.array_equal(got["pos"].cpu().numpy(), pos_o)
        assert np.array_equal(to_bits(got["kc"]), Kc_o) and np.array_equal(to_bits(got["vc"]), Vc_o)
        Fg, _ = orc.parallel_attention(qa[0:1, La - w:], La - w, theta, None, Kc_o[None], Vc_o[None],
                                       krot_all[0][0:1, La - w:], va[0:1, La - w:])
        check_attention_output(to_f64(got["fg"]), Fg, "Fg (ragged)")
    if forced is not None:
        assert 3 in kept_o.tolist()


@pytest.mark.parametrize("Cb,L,w,Hkv,d,k,m", [(4, 256, 16, 2, 64, 64, 3), (3, 1100, 64, 2, 128, 300, 5), (2, 300, 24, 3, 128, 500, 2)])
def test_rank_and_compact_in_one_launch_equals_the_two_calls(Cb, L, w, Hkv, d, k, m):
    """pc_queue_select_gather = pc_select_tokens on the batch + pc_queue_gather, bit for bit: positions, keys and
    values of the slots that take a chunk; slots that keep their contents are not touched.  (k above the number of
    candidates in the last case: the tail of a slot is padded with position -1 and zero rows.)"""
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(Cb * 100 + k)
    score = torch.from_numpy(rng.random((Cb, Hkv, L)).astype(np.float32)).cuda()
    ksrc = torch.from_numpy(rng.integers(0, 2 ** 15, size=(Cb, L, Hkv, d)).astype(np.int16)).cuda().view(torch.bfloat16)
    vsrc = torch.from_numpy(rng.integers(0, 2 ** 15, size=(Cb, L, Hkv, d)).astype(np.int16)).cuda().view(torch.bfloat16)
    slot_src = torch.full((m,), -1, dtype=torch.int32, device="cuda")
    slot_src[0] = Cb - 1
    if m > 2:
        slot_src[2] = 0
    states = []
    for fused in (False, True):
        st = pc.queue_init(m, Hkv, k, d, "cuda")
        for key in ("q_k", "q_v"):
            st[key].view(torch.int16).fill_(0x1234)                   # untouched slots must keep this
        st["q_pos"].fill_(-7)
        st["slot_src"].copy_(slot_src)
        if fused:
            n0 = pc.launch_count()
            pc.queue_select_gather(st, score, ksrc, vsrc, L - w)
            assert pc.launch_count() - n0 == 1
        else:
            idx = pc.select_tokens(score, torch.arange(Cb, dtype=torch.int32, device="cuda"), L - w, k)
            pc.queue_gather(st, ksrc, vsrc, idx)
        torch.cuda.synchronize()
        states.append(st)
    for key in ("q_k", "q_v"):
        assert torch.equal(states[0][key].view(torch.int16), states[1][key].view(torch.int16)), key
    assert torch.equal(states[0]["q_pos"], states[1]["q_pos"])
    assert int((states[1]["q_pos"][:, k:2 * k] == -7).all()) == 1     # slot 1 keeps its contents
