"""Pins for the oracle's RoPE, chunk-local attention and window scores (CPU only).

Each test checks the oracle against something fixed outside it: a closed form,
an invariant of Eq. 1-2 / Eq. 6, a library routine used as a special case
(torch SDPA in fp64), or a scalar Python loop over the definition.
"""
import math

import numpy as np
import pytest
import torch

import pc_inputs
from oracle import parallelcomp_oracle as orc
from tests import brute


def _rand_bits(rng, shape, scale=1.0):
    return pc_inputs.f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32))


# --------------------------------------------------------------------------- bf16 conversion
def test_bf16_roundtrip_and_ties():
    # every finite bf16 pattern survives widening + rounding
    bits = np.arange(0, 0x10000, dtype=np.uint32).astype(np.uint16)
    finite = (bits & 0x7F80) != 0x7F80
    bits = bits[finite]
    assert np.array_equal(orc.f64_to_bf16(orc.bf16_to_f64(bits)), bits)
    # ties go to the even mantissa: 1 + 2^-8 is halfway between 1.0 (even) and 1 + 2^-7
    assert orc.f64_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
    assert orc.f64_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82
    # just above the tie rounds up (a float32 detour would lose this bit)
    assert orc.f64_to_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 0x3F81
    # agrees with torch's conversion on fp32 inputs
    x = np.random.default_rng(0).standard_normal(4096).astype(np.float32)
    t = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.f64_to_bf16(x.astype(np.float64)), t)
    assert np.array_equal(pc_inputs.f32_to_bf16_bits(x), t)
    # and with the exact rational rounding used by the scalar brute force
    for v in (0.1, -2.71828, 3.0e-5, 123.456):
        assert int(orc.f64_to_bf16(np.array([v]))[0]) == brute.float_to_bf16_bits(v)


# --------------------------------------------------------------------------- RoPE
def test_rope_closed_form_d2():
    # d = 2: one pair, inv_freq = 1, so position p rotates (x1, x2) by p radians
    x = np.array([[[1.0, 0.0]], [[0.25, -2.0]], [[3.0, 4.0]]])      # [tokens=3, heads=1, d=2]
    out = orc.rope_rotate(x, np.array([0, 1, 5]), theta=10000.0)
    assert np.allclose(out[0, 0], [1.0, 0.0], atol=0)
    assert np.allclose(out[1, 0], [0.25 * math.cos(1) + 2.0 * math.sin(1), -2.0 * math.cos(1) + 0.25 * math.sin(1)], atol=1e-15)
    assert np.allclose(out[2, 0], [3 * math.cos(5) - 4 * math.sin(5), 4 * math.cos(5) + 3 * math.sin(5)], atol=1e-14)


def test_rope_frequencies_and_pairing():
    d, theta, p = 8, 500000.0, 7
    # a unit vector in slot t must land in slots (t, t + d/2) with angle p * theta^(-2t/d)
    for t in range(d // 2):
        x = np.zeros((1, 1, d))
        x[0, 0, t] = 1.0
        out = orc.rope_rotate(x, np.array([p]), theta)[0, 0]
        phi = p * theta ** (-2.0 * t / d)
        expect = np.zeros(d)
        expect[t], expect[t + d // 2] = math.cos(phi), math.sin(phi)
        assert np.allclose(out, expect, atol=1e-15)


def test_rope_matches_rotate_half_formulation():
    # the "x*cos + rotate_half(x)*sin" statement used by Llama-family models, written with torch ops
    rng = np.random.default_rng(1)
    L, H, d, theta = 37, 3, 16, 10000.0
    x = rng.standard_normal((L, H, d))
    inv = 1.0 / (theta ** (torch.arange(0, d, 2, dtype=torch.float64) / d))
    freqs = torch.outer(torch.arange(L, dtype=torch.float64), inv)
    emb = torch.cat([freqs, freqs], dim=-1)
    xt = torch.from_numpy(x)
    rot_half = torch.cat([-xt[..., d // 2:], xt[..., :d // 2]], dim=-1)
    expect = xt * emb.cos()[:, None, :] + rot_half * emb.sin()[:, None, :]
    assert np.allclose(orc.rope_rotate(x, np.arange(L), theta), expect.numpy(), atol=1e-13)


def test_rope_norm_and_shift_invariance():
    rng = np.random.default_rng(2)
    L, d, theta = 64, 32, 10000.0
    q = rng.standard_normal((L, 1, d))
    k = rng.standard_normal((L, 1, d))
    pos = np.arange(L)
    q0, k0 = orc.rope_rotate(q, pos, theta), orc.rope_rotate(k, pos, theta)
    assert np.allclose(np.linalg.norm(q0, axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-13)
    # position 0 is the identity
    assert np.array_equal(q0[0], q[0])
    # logits depend only on the position difference
    shift = 1234
    q1, k1 = orc.rope_rotate(q, pos + shift, theta), orc.rope_rotate(k, pos + shift, theta)
    s0 = q0[:, 0] @ k0[:, 0].T
    s1 = q1[:, 0] @ k1[:, 0].T
    assert np.allclose(s0, s1, atol=1e-10)


# --------------------------------------------------------------------------- Eq. 1-2
def _tiny_case(seed=3, C=2, L=12, Hq=4, Hkv=2, d=8):
    rng = np.random.default_rng(seed)
    return (_rand_bits(rng, (C, L, Hq, d)), _rand_bits(rng, (C, L, Hkv, d)), _rand_bits(rng, (C, L, Hkv, d)))


def test_local_attention_vs_scalar_loops():
    q, k, v = _tiny_case()
    theta = 10000.0
    scale = 1.0 / math.sqrt(q.shape[-1])
    O, LSE, k_rot = orc.local_attention(q, k, v, theta)
    for c, h in ((0, 0), (1, 3), (0, 2)):
        A_b, O_b, LSE_b = brute.causal_attention_loops(q.tolist(), k.tolist(), v.tolist(), c, h, theta, scale)
        assert np.allclose(O[c, :, h], np.array(O_b), atol=1e-12)
        assert np.allclose(LSE[c, h], np.array(LSE_b), atol=1e-12)
    # rotated keys agree with the scalar rotation + exact rounding
    for (c, j, hk) in ((0, 5, 1), (1, 11, 0)):
        expect = [brute.float_to_bf16_bits(x) for x in
                  brute.rope_scalar([brute.bf16_to_float(b) for b in k[c, j, hk]], j, theta)]
        assert k_rot[c, j, hk].tolist() == expect


def test_local_attention_vs_torch_sdpa_fp64():
    q, k, v = _tiny_case(seed=4, C=2, L=33, Hq=4, Hkv=2, d=16)
    theta = 500000.0
    O, LSE, k_rot = orc.local_attention(q, k, v, theta)
    q_rot = orc.rope_bf16(q, theta)
    G = q.shape[2] // k.shape[2]
    tq = torch.from_numpy(orc.bf16_to_f64(q_rot)).permute(0, 2, 1, 3)                       # [C,Hq,L,d]
    tk = torch.from_numpy(orc.bf16_to_f64(k_rot)).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
    tv = torch.from_numpy(orc.bf16_to_f64(v)).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    assert np.allclose(O, ref.permute(0, 2, 1, 3).numpy(), atol=1e-12)


def test_local_attention_invariants():
    q, k, v = _tiny_case(seed=5, C=1, L=20, Hq=2, Hkv=1, d=8)
    theta = 10000.0
    scale = 1.0 / math.sqrt(8)
    q_rot, k_rot = orc.rope_bf16(q, theta), orc.rope_bf16(k, theta)
    A, O, LSE = orc.local_attention_rows(q_rot, k_rot, v, 0, 1, np.arange(20), scale)
    assert np.allclose(A.sum(axis=1), 1.0, atol=1e-14)
    assert np.all(np.triu(A, 1) == 0.0)                       # causal
    assert np.allclose(O[0], orc.bf16_to_f64(v[0, 0, 0]), atol=1e-15)   # row 0 sees only key 0
    # all keys equal (at position 0 rotation is identity; use theta so large that rotation ~ identity is NOT assumed:
    # instead zero keys -> all logits 0) -> uniform attention -> running mean of V
    kz = np.zeros_like(k)
    A2, O2, _ = orc.local_attention_rows(q_rot, orc.rope_bf16(kz, theta), v, 0, 0, np.arange(20), scale)
    vf = orc.bf16_to_f64(v[0, :, 0])
    running_mean = np.cumsum(vf, axis=0) / np.arange(1, 21)[:, None]
    assert np.allclose(O2, running_mean, atol=1e-13)
    # LSE of uniform zero logits over i+1 keys = log(i+1)
    _, _, lse2 = orc.local_attention_rows(q_rot, orc.rope_bf16(kz, theta), v, 0, 0, np.arange(20), scale)
    assert np.allclose(lse2, np.log(np.arange(1, 21)), atol=1e-14)


def test_two_token_softmax_closed_form():
    # d=2, H=1, L=2, q = k = (1, 0) at both positions; theta irrelevant (one pair, inv_freq 1).
    # Rotated+rounded: position 0 -> (1, 0); position 1 -> (bf16(cos 1), bf16(sin 1)) = (0.5390625, 0.83984375).
    one = 0x3F80
    q = np.array([[[[one, 0]], [[one, 0]]]], dtype=np.uint16)        # [C=1, L=2, H=1, d=2]
    k = q.copy()
    v = np.array([[[[0x4000, 0]], [[0, 0x4080]]]], dtype=np.uint16)  # v0 = (2, 0), v1 = (0, 4)
    O, LSE, k_rot = orc.local_attention(q, k, v, 10000.0)
    c1, s1 = 0.5390625, 0.83984375
    assert orc.bf16_to_f64(k_rot[0, 1, 0]).tolist() == [c1, s1]
    sc = 1.0 / math.sqrt(2.0)
    l0, l1 = c1 * sc, (c1 * c1 + s1 * s1) * sc
    p0 = 1.0 / (1.0 + math.exp(l1 - l0))
    assert np.allclose(O[0, 1, 0], [2 * p0, 4 * (1 - p0)], atol=1e-15)
    assert np.allclose(O[0, 0, 0], [2.0, 0.0], atol=0)
    assert abs(LSE[0, 0, 1] - math.log(math.exp(l0) + math.exp(l1))) < 1e-15
    assert abs(LSE[0, 0, 0] - 1.0 * sc) < 1e-15


# --------------------------------------------------------------------------- Eq. 6
def test_window_score_invariants_and_loops():
    q, k, v = _tiny_case(seed=6, C=2, L=14, Hq=4, Hkv=2, d=8)
    theta, w = 10000.0, 5
    L, G = 14, 2
    scale = 1.0 / math.sqrt(8)
    q_rot, k_rot = orc.rope_bf16(q, theta), orc.rope_bf16(k, theta)
    S, O_win, LSE_win = orc.window_scores(q_rot, k_rot, v, w, scale)
    assert S.shape == (2, 2, L)
    assert np.all(S >= 0)
    assert np.allclose(S.sum(axis=-1), G * w, atol=1e-12)          # G*w softmax rows, each summing to 1
    # brute force: explicit loops over heads, window rows and keys
    for c in range(2):
        for hk in range(2):
            acc = [0.0] * L
            for g in range(G):
                A_b, O_b, LSE_b = brute.causal_attention_loops(q.tolist(), k.tolist(), v.tolist(), c, hk * G + g, theta, scale)
                for i in range(L - w, L):
                    for j in range(L):
                        acc[j] += A_b[i][j]
                assert np.allclose(O_win[c, :, hk * G + g], np.array(O_b[L - w:]), atol=1e-12)
                assert np.allclose(LSE_win[c, hk * G + g], np.array(LSE_b[L - w:]), atol=1e-12)
            assert np.allclose(S[c, hk], np.array(acc), atol=1e-12)
    # the last key is seen by the last row only
    A_last, _, _ = orc.local_attention_rows(q_rot, k_rot, v, 0, 0, np.array([L - 1]), scale)
    A_last1, _, _ = orc.local_attention_rows(q_rot, k_rot, v, 0, 1, np.array([L - 1]), scale)
    assert abs(S[0, 0, L - 1] - (A_last[0, L - 1] + A_last1[0, L - 1])) < 1e-14


def test_window_score_w1_is_last_softmax_row():
    q, k, v = _tiny_case(seed=7, C=1, L=9, Hq=1, Hkv=1, d=4)
    scale = 0.5
    q_rot, k_rot = orc.rope_bf16(q, 10000.0), orc.rope_bf16(k, 10000.0)
    S, _, _ = orc.window_scores(q_rot, k_rot, v, 1, scale)
    A, _, _ = orc.local_attention_rows(q_rot, k_rot, v, 0, 0, np.array([8]), scale)
    assert np.allclose(S[0, 0], A[0], atol=0)


def test_chunk_score_surrogate_orders_by_match_strength():
    # chunk 1's keys are aligned with the window queries -> larger LSE -> lower (better) score
    lse = np.array([[[1.0, 2.0], [3.0, 4.0]], [[5.0, 6.0], [7.0, 8.0]]])
    assert np.allclose(orc.chunk_score_from_lse(lse), [-2.5, -6.5])
