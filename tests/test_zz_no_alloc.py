"""pc_parallel_attn_static: the entry point for callers that are not allowed to allocate device memory
(its scratch is a fixed array inside the library).  It must give what pc_parallel_attn gives, also on a
second call that finds the first call's leftovers in the shared scratch.

Collected last on purpose: a failure here cannot hide any other test behind `-x`.
"""
import numpy as np
import pytest
import torch

import pc_inputs
from oracle import parallelcomp_oracle as orc
from tests.gpu_util import to_dev, to_bits, to_f64, check_attention_output


def _bits(rng, shape):
    return pc_inputs.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


def _case(seed, B, w, Hq, Hkv, d, Nk):
    rng = np.random.default_rng(seed)
    t = {"q_win": _bits(rng, (B, w, Hq, d)), "k_cache": _bits(rng, (B, Hkv, Nk, d)),
         "v_cache": _bits(rng, (B, Hkv, Nk, d)), "k_win": _bits(rng, (B, w, Hkv, d)),
         "v_win": _bits(rng, (B, w, Hkv, d))}
    return {k: to_dev(v) for k, v in t.items()}


@pytest.mark.gpu
def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row():
    import paper_2502_14317_b200 as pc
    limit = pc.parallel_attn_static_scratch_bytes()
    assert limit == 16 << 20
    # two different shapes back to back: the second call starts from a scratch full of the first
    # call's counter, table and partial results.  Both shapes split the keys (merge kernel runs).
    shapes = [(2, 16, 4, 2, 64, 1024, 240, 1e4), (1, 64, 8, 2, 128, 3000, 8128, 5e5)]
    for rep, (B, w, Hq, Hkv, d, Nk, q_pos0, theta) in enumerate(shapes):
        need = pc.parallel_attn_workspace_bytes(B, w, Hq, Hkv, d, Nk)
        assert 65536 < need <= limit, need                      # key splits in use, and it fits
        t = _case(100 + rep, B, w, Hq, Hkv, d, Nk)
        ref = pc.parallel_attn(t["q_win"], t["k_cache"], t["v_cache"], t["k_win"], t["v_win"], q_pos0=q_pos0,
                               rope_theta=theta, want_lse=True)
        out = torch.full((B, w, Hq, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((B, Hq, w), float("nan"), dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        if rep == 0:
            # the set-up call of this device: it looks the array's address up, and with CUDA's lazy module loading
            # that is also the moment the driver binds the array's 16 MiB (the library image's own data, no
            # allocation call); every later call must leave the device's memory exactly as it finds it
            pc.parallel_attn_static(t["q_win"], t["k_cache"], t["v_cache"], t["k_win"], t["v_win"], out,
                                    q_pos0=q_pos0, rope_theta=theta, lse_out=lse, status=status)
        for call in range(2):                                    # same shape twice as well
            out.fill_(float("nan"))
            # the reason this entry point exists: no device memory is taken while it runs - neither through
            # torch's caching allocator nor behind its back (the driver's free-memory figure)
            torch.cuda.synchronize()
            before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
            pc.parallel_attn_static(t["q_win"], t["k_cache"], t["v_cache"], t["k_win"], t["v_win"], out,
                                    q_pos0=q_pos0, rope_theta=theta, lse_out=lse, status=status)
            torch.cuda.synchronize()
            after = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
            assert after[0] == before[0] and after[1] == before[1] and after[2] >= before[2], (before, after)
            assert int(status.item()) == 0 and int(ref["status"].item()) == 0
            # same kernels and the same split plan: the tolerance of the attention outputs is met with room
            # to spare (in fact the two agree bit for bit)
            check_attention_output(to_f64(out), to_f64(ref["out"]), f"static call {call} of shape {rep}")
            assert torch.equal(out.view(torch.int16), ref["out"].view(torch.int16))
            assert np.abs(lse.cpu().numpy() - ref["lse"].cpu().numpy()).max() <= 2e-3
        # and against the oracle, through this entry point (not only against the other CUDA entry)
        bits = {k_: to_bits(v_) for k_, v_ in t.items()}
        Fg, LSEg = orc.parallel_attention(bits["q_win"], q_pos0, theta, None, bits["k_cache"], bits["v_cache"],
                                          bits["k_win"], bits["v_win"])
        check_attention_output(to_f64(out), Fg, f"static entry vs oracle, shape {rep}")
        assert np.abs(lse.cpu().numpy().astype(np.float64) - LSEg).max() <= 2e-3


@pytest.mark.gpu
def test_static_scratch_entry_refuses_what_does_not_fit():
    import paper_2502_14317_b200 as pc
    lib = pc.load_library()
    B, w, Hq, Hkv, d, Nk = 1, 64, 32, 8, 128, 16384             # one sequence, widely split keys: 64 MiB of partials
    assert pc.parallel_attn_workspace_bytes(B, w, Hq, Hkv, d, Nk) > pc.parallel_attn_static_scratch_bytes()
    x = torch.zeros(16, dtype=torch.uint8, device="cuda")
    p = x.data_ptr()
    rc = lib.pc_parallel_attn_static(B, w, Hq, Hkv, d, Nk, p, 8128, 5e5, 0.0, p, p, p, p, p, None, None, None)
    assert rc == -6 and "scratch" in pc.status_string(rc)
    with pytest.raises(pc.PcError, match="bytes of scratch"):
        t = _case(7, 1, 64, 32, 8, 128, 16384)
        pc.parallel_attn_static(t["q_win"], t["k_cache"], t["v_cache"], t["k_win"], t["v_win"],
                                torch.empty((1, 64, 32, 128), dtype=torch.bfloat16, device="cuda"),
                                q_pos0=8128, rope_theta=5e5)
