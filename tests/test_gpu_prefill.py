"""GPU parity: pc_chunk_prefill_attn against the CPU oracle, element by element (through the C ABI)."""
import numpy as np
import pytest
import torch

import pc_inputs
from oracle import parallelcomp_oracle as orc
from tests.gpu_util import to_dev, to_bits, to_f64, check_attention_output, check_scores

pytestmark = pytest.mark.gpu


def _run_and_compare(q, k, v, w, theta, want_lse=True, sharp=False):
    import paper_2502_14317_b200 as pc
    C, L, Hq, d = q.shape
    Hkv = k.shape[2]
    G = Hq // Hkv
    res = pc.chunk_prefill_attn(to_dev(q), to_dev(k), to_dev(v), w=w, rope_theta=theta, want_lse=want_lse)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 0, f"device wait ran out, code {int(res['status'].item())}"
    O, LSE, k_rot = orc.local_attention(q, k, v, theta)
    scale = 1.0 / np.sqrt(d)
    S, O_win, LSE_win = orc.window_scores(orc.rope_bf16(q, theta), k_rot, v, w, scale)
    # rotated keys: the rotation is evaluated in fp64 on both sides -> same bits
    assert np.array_equal(to_bits(res["k_rot"]), k_rot), "k_rot differs from the oracle"
    check_attention_output(to_f64(res["o"]), O, sharp=sharp)
    lse = res["lse"].cpu().numpy().astype(np.float64)
    assert np.abs(lse - LSE).max() <= 2e-3, f"LSE max err {np.abs(lse - LSE).max():.3e}"
    win_lse = res["win_lse"].cpu().numpy().astype(np.float64)
    assert np.abs(win_lse - LSE_win).max() <= 2e-3
    got_S = res["win_score"].cpu().numpy()
    check_scores(got_S, S, G, w, L)
    assert np.allclose(got_S.sum(-1), G * w, rtol=1e-4)        # Eq. 6: G*w softmax rows, each summing to 1
    return res


def test_cfg0_full(cfg0_inputs):
    cfg, inp = cfg0_inputs
    _run_and_compare(inp["q"], inp["k"], inp["v"], cfg.w, cfg.rope_theta)


@pytest.mark.parametrize("C,L,w,Hq,Hkv,d,theta", [
    (2, 384, 64, 4, 1, 128, 500000.0),     # GQA G=4 (two head pairs), d=128, three query tiles
    (2, 300, 16, 2, 2, 64, 10000.0),       # MHA (tile-pair mode), ragged last tile (300 = 2*128 + 44)
    (1, 200, 128, 2, 1, 64, 10000.0),      # window spans two tiles, ragged
    (3, 520, 8, 3, 3, 128, 10000.0),       # MHA, odd tile count (5 tiles), smallest window
    (1, 100, 32, 8, 1, 64, 10000.0),       # single ragged tile, G*w = 256 window rows
    (1, 640, 64, 8, 1, 128, 500000.0),     # G*w = 512 window rows: two score passes
    (1, 130, 64, 1, 1, 64, 10000.0),       # single head, MHA, two tiles with a 2-token tail
    # head size 128 runs on CTA pairs: two q-heads (or two adjacent query tiles) per pair
    (2, 300, 16, 2, 1, 128, 10000.0),      # G=2: one head pair, ragged last tile
    (1, 100, 32, 1, 1, 128, 10000.0),      # MHA, a single ragged tile: the second CTA of the pair has no block
    (1, 256, 128, 4, 2, 128, 500000.0),    # widest window = exactly the last tile, two kv-heads
    (2, 1100, 64, 6, 2, 128, 10000.0),     # G=3 (odd): tile-pair mode, 9 tiles, ragged
    (1, 1024, 8, 2, 2, 128, 10000.0),      # MHA, even tile count, smallest window
    (1, 200, 128, 8, 1, 128, 10000.0),     # G*w = 1024 window rows: four score passes, window over two tiles
    # windows that are no power of two (the sweep pads a head's rows to a multiple of 8 and leaves the pad out)
    (2, 400, 24, 4, 2, 128, 10000.0),      # CTA pairs, w = 24
    (1, 700, 100, 4, 1, 128, 500000.0),    # CTA pairs, w = 100 (the region size of App. C), window over two tiles
    (1, 300, 5, 2, 1, 128, 10000.0),       # CTA pairs, w = 5 < 8
    (1, 260, 1, 4, 2, 128, 10000.0),       # CTA pairs, a single query token
    (2, 400, 24, 3, 3, 128, 10000.0),      # multi-head (single-CTA kernel, tile-pair mode), w = 24
    (1, 520, 100, 6, 2, 128, 10000.0),     # G = 3, w = 100
    (2, 300, 24, 4, 2, 64, 10000.0),       # head size 64, w = 24
    (1, 333, 100, 2, 1, 64, 10000.0),      # head size 64, w = 100
    (1, 140, 3, 8, 2, 64, 10000.0),        # head size 64, w = 3
])
def test_shapes(C, L, w, Hq, Hkv, d, theta):
    rng = np.random.default_rng(L * 7 + Hq)
    q = pc_inputs.f32_to_bf16_bits(rng.standard_normal((C, L, Hq, d)).astype(np.float32))
    k = pc_inputs.f32_to_bf16_bits(rng.standard_normal((C, L, Hkv, d)).astype(np.float32))
    v = pc_inputs.f32_to_bf16_bits(rng.standard_normal((C, L, Hkv, d)).astype(np.float32))
    k[:, 0] = pc_inputs.f32_to_bf16_bits(pc_inputs.bf16_bits_to_f32(k[:, 0]) * np.float32(4.0))
    _run_and_compare(q, k, v, w, theta)


@pytest.mark.parametrize("d", [64, 128])
def test_growing_logits_rescale_path(d):
    """Keys whose norm grows along the chunk make the running row maximum jump by more than the lazy
    threshold again and again, so the accumulator is rescaled in most tiles (rare otherwise)."""
    rng = np.random.default_rng(99 + d)
    C, L, Hq, Hkv, w = 1, 700, 4, 2, 32
    q = rng.standard_normal((C, L, Hq, d)).astype(np.float32)
    k = rng.standard_normal((C, L, Hkv, d)).astype(np.float32)
    v = rng.standard_normal((C, L, Hkv, d)).astype(np.float32)
    k *= np.linspace(1.0, 40.0, L, dtype=np.float32)[None, :, None, None]
    bits = [pc_inputs.f32_to_bf16_bits(x) for x in (q, k, v)]
    _run_and_compare(bits[0], bits[1], bits[2], w, 10000.0, sharp=True)


@pytest.mark.parametrize("Hq,Hkv", [(4, 2), (2, 2), (6, 2)])
def test_growing_logits_many_tiles(Hq, Hkv):
    """The same stress over 13 key tiles, two chunks, even and odd group sizes: the softmax warpgroups, the three
    issuing threads and the TMEM buffers go through many rounds in which a warpgroup stalls in the rescale path
    while the other runs ahead, including across query blocks and the score sweep."""
    rng = np.random.default_rng(7 + Hq)
    C, L, w, d = 2, 1600, 64, 128
    q = rng.standard_normal((C, L, Hq, d)).astype(np.float32)
    k = rng.standard_normal((C, L, Hkv, d)).astype(np.float32)
    v = rng.standard_normal((C, L, Hkv, d)).astype(np.float32)
    k *= np.linspace(1.0, 60.0, L, dtype=np.float32)[None, :, None, None]
    bits = [pc_inputs.f32_to_bf16_bits(x) for x in (q, k, v)]
    _run_and_compare(bits[0], bits[1], bits[2], w, 10000.0, sharp=True)


def test_deterministic_and_strided(cfg0_inputs):
    import paper_2502_14317_b200 as pc
    cfg, inp = cfg0_inputs
    q, k, v = to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"])
    a = pc.chunk_prefill_attn(q, k, v, w=cfg.w, rope_theta=cfg.rope_theta)
    b = pc.chunk_prefill_attn(q, k, v, w=cfg.w, rope_theta=cfg.rope_theta)
    # head-major storage viewed token-major: same numbers through explicit strides
    qh = q.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    kh = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vh = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    c = pc.chunk_prefill_attn(qh, kh, vh, w=cfg.w, rope_theta=cfg.rope_theta)
    torch.cuda.synchronize()
    for key in ("o", "k_rot", "win_score", "win_lse"):
        assert torch.equal(a[key], b[key]), f"{key} not reproducible run to run"
        assert torch.equal(a[key], c[key]), f"{key} differs for strided inputs"


def test_deterministic_head_size_128():
    """The CTA-pair kernel (two issuing threads, two softmax warpgroups on alternate tiles) must give the same
    bits run to run: accumulation order and score sums are fixed by construction."""
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(5)
    q = to_dev(pc_inputs.f32_to_bf16_bits(rng.standard_normal((2, 900, 8, 128)).astype(np.float32)))
    k = to_dev(pc_inputs.f32_to_bf16_bits(rng.standard_normal((2, 900, 2, 128)).astype(np.float32)))
    v = to_dev(pc_inputs.f32_to_bf16_bits(rng.standard_normal((2, 900, 2, 128)).astype(np.float32)))
    runs = [pc.chunk_prefill_attn(q, k, v, w=64, rope_theta=5e5, want_lse=True) for _ in range(3)]
    torch.cuda.synchronize()
    for key in ("o", "win_score", "win_lse", "lse"):
        assert torch.equal(runs[0][key], runs[1][key]) and torch.equal(runs[0][key], runs[2][key]), key


def test_argument_errors():
    import paper_2502_14317_b200 as pc
    q = torch.zeros((1, 256, 4, 64), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((1, 256, 2, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pc.PcError, match="unsupported"):
        pc.chunk_prefill_attn(q, k, k, w=129, rope_theta=1e4)          # window wider than a tile
    with pytest.raises(pc.PcError, match="invalid"):
        pc.chunk_prefill_attn(q, k, k, w=256, rope_theta=1e4)          # window >= L
    q96 = torch.zeros((1, 256, 4, 96), dtype=torch.bfloat16, device="cuda")
    k96 = torch.zeros((1, 256, 2, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pc.PcError, match="unsupported"):
        pc.chunk_prefill_attn(q96, k96, k96, w=16, rope_theta=1e4)     # head size
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    lib = pc.load_library()
    import ctypes
    from paper_2502_14317_b200.binding import _make_desc, _ptr
    o = torch.empty_like(q)
    desc = _make_desc(q, k, k, o, 16, 1e4, 0.0)
    ws = torch.empty(64, dtype=torch.uint8, device="cuda")
    S = torch.empty((1, 2, 256), dtype=torch.float32, device="cuda")
    Lw = torch.empty((1, 4, 16), dtype=torch.float32, device="cuda")
    rc = lib.pc_chunk_prefill_attn(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(k), None, _ptr(o), None, None, _ptr(S), _ptr(Lw),
                                   None, _ptr(ws), ws.numel(), None)
    assert rc == -3                                                     # PC_ERR_WORKSPACE
    rc = lib.pc_chunk_prefill_attn(ctypes.byref(desc), None, _ptr(k), _ptr(k), None, _ptr(o), None, None, _ptr(S), _ptr(Lw),
                                   None, _ptr(ws), ws.numel(), None)
    assert rc == -1                                                     # PC_ERR_INVALID_ARG


@pytest.mark.parametrize("C,L,H,d,theta", [
    (2, 8192, 4, 128, 500000.0),           # the routine of the tile prologue, positions up to 8191 (angles up to 8191 rad)
    (1, 4096, 8, 128, 10000.0),
    (3, 333, 2, 128, 10000.0),             # ragged last tile
    (2, 1000, 3, 64, 10000.0),             # head size 64: the fp64 pre-pass kernel
])
def test_rope_position_reuse_equals_fp64_rotation_rounded_once(C, L, H, d, theta):
    """The query rotation of the tile prologue is fp32 with two exact fallbacks; its bits must be those of the
    oracle's fp64 rotation.  Mixed magnitudes so that many outputs sit near a bf16 rounding boundary; with
    millions of outputs the second level (about 1 in 4000) runs thousands of times."""
    import paper_2502_14317_b200 as pc
    rng = np.random.default_rng(5 + L + d)
    x = rng.standard_normal((C, L, H, d)).astype(np.float32) * np.exp2(rng.integers(-6, 7, size=(C, L, H, 1))).astype(np.float32)
    x[0, :, 0, : d // 2] = np.float32(1.0)                    # exact cosines / sines of the table reach the output
    x[0, :, 0, d // 2:] = np.float32(0.0)
    bits = pc_inputs.f32_to_bf16_bits(x)
    got = to_bits(pc.rope_position_reuse(to_dev(bits), rope_theta=theta))
    torch.cuda.synchronize()
    ref = orc.rope_bf16(bits, theta)
    bad = np.argwhere(got != ref)
    assert bad.shape[0] == 0, f"{bad.shape[0]} of {ref.size} rotated values differ from the fp64 rotation, first at {bad[0]}"


@pytest.mark.parametrize("L,w,Hq,Hkv,d,lens", [
    (640, 64, 4, 2, 128, [640, 500, 129, 65, 384]),      # CTA pairs: full, ragged, two tiles, one tile, tile-aligned
    (520, 24, 4, 1, 128, [300, 520, 25, 256]),           # w = 24, the shortest chunk has a single context token
    (640, 64, 3, 3, 128, [640, 333, 130, 65]),           # multi-head, single-CTA kernel (tile-pair mode)
    (400, 16, 4, 2, 64, [400, 17, 250, 128]),            # head size 64
    (300, 100, 2, 2, 64, [101, 300, 229]),               # head size 64, multi-head, w = 100
])
def test_chunks_of_different_lengths_in_one_call(L, w, Hq, Hkv, d, lens):
    """Sec. 3.1: chunks of AT MOST the trained length.  chunk_len[c] tokens of chunk c count (window included, the
    window directly behind the context); every chunk must equal the oracle run on that chunk alone, and everything
    at or behind its end reads as zero."""
    import paper_2502_14317_b200 as pc
    C = len(lens)
    rng = np.random.default_rng(L + w + Hq + d)
    q = pc_inputs.f32_to_bf16_bits(rng.standard_normal((C, L, Hq, d)).astype(np.float32))
    k = pc_inputs.f32_to_bf16_bits(rng.standard_normal((C, L, Hkv, d)).astype(np.float32))
    v = pc_inputs.f32_to_bf16_bits(rng.standard_normal((C, L, Hkv, d)).astype(np.float32))
    k[:, 0] = pc_inputs.f32_to_bf16_bits(pc_inputs.bf16_bits_to_f32(k[:, 0]) * np.float32(4.0))
    theta, G = 10000.0, Hq // Hkv
    cl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    nan = float("nan")
    res = pc.chunk_prefill_attn(to_dev(q), to_dev(k), to_dev(v), w=w, rope_theta=theta, want_lse=True, chunk_len=cl,
                                out=torch.full((C, L, Hq, d), nan, dtype=torch.bfloat16, device="cuda"),
                                win_score=torch.full((C, Hkv, L), nan, dtype=torch.float32, device="cuda"),
                                lse=torch.full((C, Hq, L), nan, dtype=torch.float32, device="cuda"))
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 0
    got_o, got_S = to_f64(res["o"]), res["win_score"].cpu().numpy()
    got_lse, got_wl = res["lse"].cpu().numpy().astype(np.float64), res["win_lse"].cpu().numpy().astype(np.float64)
    assert np.array_equal(to_bits(res["k_rot"]), orc.rope_bf16(k, theta))
    scale = 1.0 / np.sqrt(d)
    for c, n in enumerate(lens):
        qc, kc, vc = q[c:c + 1, :n], k[c:c + 1, :n], v[c:c + 1, :n]
        O, LSE, k_rot = orc.local_attention(qc, kc, vc, theta)
        S, _, LSE_win = orc.window_scores(orc.rope_bf16(qc, theta), k_rot, vc, w, scale)
        check_attention_output(got_o[c:c + 1, :n], O, f"O of chunk {c} ({n} tokens)")
        assert np.abs(got_lse[c:c + 1, :, :n] - LSE).max() <= 2e-3
        assert np.abs(got_wl[c:c + 1] - LSE_win).max() <= 2e-3
        check_scores(got_S[c:c + 1, :, :n], S, G, w, n)
        assert np.allclose(got_S[c, :, :n].sum(-1), G * w, rtol=1e-4)
        assert np.all(got_o[c, n:] == 0.0) and np.all(got_S[c, :, n:] == 0.0) and np.all(got_lse[c, :, n:] == 0.0)


def test_a_wait_that_runs_out_returns_a_status_and_leaves_the_device_usable(cfg0_inputs):
    """Every device-side wait is bounded.  Here one is made to run out without faulting anything: the producer
    warp of the single-CTA kernel (head size 64) leaves out the data-free "no more work" signal after the last
    work item, when no copy and no tensor-core operation is in flight; the consumer warps wait for it for about a
    millisecond (limit set through the test hook), store the code of that wait in the status word, drain and
    return.  The outputs of that call are complete, and the next call on the same stream is bit-identical to a
    clean run."""
    import paper_2502_14317_b200 as pc
    cfg, inp = cfg0_inputs
    q, k, v = to_dev(inp["q"]), to_dev(inp["k"]), to_dev(inp["v"])
    lib = pc.load_library()

    def run():
        r = pc.chunk_prefill_attn(q, k, v, w=cfg.w, rope_theta=cfg.rope_theta, want_lse=True)
        torch.cuda.synchronize()
        return r

    clean = run()
    assert int(clean["status"].item()) == 0
    assert lib.pc_debug_bounded_wait_test(2_000_000, 1) == 0          # waits give up after 2e6 cycles (about 1 ms)
    try:
        hit = run()
    finally:
        assert lib.pc_debug_bounded_wait_test(0, 0) == 0
    code = int(hit["status"].item())
    assert code == 101, f"expected the code of the work-item wait in the status word, got {code}"
    for key in ("o", "win_score", "win_lse", "lse", "k_rot"):
        assert torch.equal(hit[key], clean[key]), key                 # all work was done before the missing signal
    again = run()
    assert int(again["status"].item()) == 0
    for key in ("o", "win_score", "win_lse", "lse", "k_rot"):
        assert torch.equal(again[key], clean[key]), key
