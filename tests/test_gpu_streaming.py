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
