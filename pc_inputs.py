"""Seeded synthetic inputs for the ParallelComp attention hot path.

This module only DRAWS inputs (random tensors with the paper's shapes and a
planted structure).  It holds none of the method's arithmetic: no RoPE, no
softmax, no ranking.  Both the CUDA path and the CPU oracle consume the arrays
produced here; neither is imported from here.

All tensors are bf16, carried as numpy ``uint16`` bit patterns (numpy has no
bf16 dtype).  ``f32_to_bf16_bits`` is a plain dtype conversion (round to
nearest even), the same conversion ``torch.Tensor.to(torch.bfloat16)`` does.

Workload shapes follow the paper's setting (Sec. 3.1, App. C): a long input is
cut into C chunks whose length L *including* the w-token query window equals
the model's trained context (4K for Llama-2, 8K for Llama-3); the same query
window is appended to every chunk.  Total context 128K-256K.
"""
from __future__ import annotations

from dataclasses import dataclass, field, asdict
import numpy as np

__all__ = [
    "PrefillConfig", "ParallelAttnConfig", "CONFIGS", "get_config",
    "f32_to_bf16_bits", "bf16_bits_to_f32", "make_prefill_inputs",
    "make_parallel_attn_inputs", "PLANT_GAIN", "SINK_GAIN",
]

SINK_GAIN = 4.0    # key 0 of every chunk is scaled by this (attention sink)
PLANT_GAIN = 4.0   # planted keys: gain * (0.8 * unit-RMS mean window query + 0.2 * noise)
BASE_SEED = 0x5043


@dataclass(frozen=True)
class PrefillConfig:
    """One chunked-prefill workload: C chunks of L tokens (ctx = L - w context + w window)."""
    name: str
    C: int
    L: int
    w: int
    Hq: int
    Hkv: int
    d: int
    rope_theta: float
    m: int            # chunks kept
    k: int            # tokens kept per (kept chunk, kv-head)
    n_planted_chunks: int
    n_planted_keys: int
    seed: int
    planted_chunks: tuple = ()   # fixed choice; () -> drawn from the seed

    @property
    def ctx(self) -> int:
        return self.L - self.w

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    def as_dict(self):
        return asdict(self)


@dataclass(frozen=True)
class ParallelAttnConfig:
    """Parallel attention over already-compressed caches: B sequences, Nk kept keys each."""
    name: str
    B: int
    Nk: int
    w: int
    Hq: int
    Hkv: int
    d: int
    rope_theta: float
    q_pos0: int       # chunk-local position of the first window token (= L - w)
    seg: int          # kept tokens per kept chunk; one sink entry per segment
    seed: int

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    def as_dict(self):
        return asdict(self)


CONFIGS = {
    # tiny gate case: the oracle runs in full in seconds
    "cfg0": PrefillConfig("cfg0", C=4, L=256, w=16, Hq=4, Hkv=2, d=64, rope_theta=1.0e4,
                          m=2, k=64, n_planted_chunks=1, n_planted_keys=8,
                          seed=BASE_SEED + 0, planted_chunks=(2,)),
    # Llama-3-8B attention shape, 128K = 16 x 8K
    "cfg1": PrefillConfig("cfg1", C=16, L=8192, w=64, Hq=32, Hkv=8, d=128, rope_theta=5.0e5,
                          m=8, k=2048, n_planted_chunks=3, n_planted_keys=32, seed=BASE_SEED + 1),
    # Llama-2-7B attention shape (MHA), 128K = 32 x 4K
    "cfg2": PrefillConfig("cfg2", C=32, L=4096, w=64, Hq=32, Hkv=32, d=128, rope_theta=1.0e4,
                          m=12, k=1024, n_planted_chunks=4, n_planted_keys=32, seed=BASE_SEED + 2),
    # 256K stress, aggressive eviction
    "cfg3": PrefillConfig("cfg3", C=32, L=8192, w=64, Hq=32, Hkv=8, d=128, rope_theta=5.0e5,
                          m=4, k=512, n_planted_chunks=2, n_planted_keys=32, seed=BASE_SEED + 3),
    # the paper's own hyper-parameters (App. C) on the Llama-3 shape: query window = last 8 tokens, half of
    # every chunk kept, 3 chunks kept; 32K context to keep the test short
    "paper_w8": PrefillConfig("paper_w8", C=4, L=8192, w=8, Hq=32, Hkv=8, d=128, rope_theta=5.0e5,
                              m=3, k=4092, n_planted_chunks=1, n_planted_keys=32, seed=BASE_SEED + 5),
    # 6K position reuse under a 24K KV budget (the Llama-3.1 / Qwen2.5 setting): chunks of 6144, Nk = 4 x 6016
    "reuse6k": PrefillConfig("reuse6k", C=6, L=6144, w=64, Hq=32, Hkv=8, d=128, rope_theta=5.0e5,
                             m=4, k=6016, n_planted_chunks=1, n_planted_keys=32, seed=BASE_SEED + 6),
    # parallel attention only, batch of compressed caches
    "cfg4": ParallelAttnConfig("cfg4", B=64, Nk=16384, w=64, Hq=32, Hkv=8, d=128, rope_theta=5.0e5,
                               q_pos0=8128, seg=2048, seed=BASE_SEED + 4),
}


def get_config(name: str):
    return CONFIGS[name]


# --------------------------------------------------------------------------- dtype conversion
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even.  Inputs here are finite."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_bf16(rng: np.random.Generator, shape) -> np.ndarray:
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))


# --------------------------------------------------------------------------- prefill workloads
def make_prefill_inputs(cfg: PrefillConfig, C: int | None = None, seed: int | None = None):
    """Draw Q [C,L,Hq,d], K,V [C,L,Hkv,d] as bf16 bit patterns (pre-RoPE), token-major.

    Structure, stated in the same terms as the workload description:
      * Q, K, V ~ N(0,1) i.i.d.
      * The query window (last w tokens) is drawn once and copied into every
        chunk (the same query tokens follow every chunk).
      * Key 0 of every chunk is multiplied by SINK_GAIN (attention sink).
      * In ``n_planted_chunks`` chunks, ``n_planted_keys`` context keys per
        kv-head are overwritten with
        PLANT_GAIN * (0.8 * u + 0.2 * noise), u = mean of that kv-head group's
        window queries rescaled to unit RMS.  (Built in the stored, pre-RoPE
        space; no rotation is applied here.)

    Returns a dict with q, k, v (uint16), planted_chunks (list[int]) and
    planted_pos (int array [n_planted_chunks, Hkv, n_planted_keys]).
    ``C`` overrides the number of chunks (used to draw a bounded sample of a
    large workload with the same recipe).
    """
    C = cfg.C if C is None else int(C)
    L, w, Hq, Hkv, d = cfg.L, cfg.w, cfg.Hq, cfg.Hkv, cfg.d
    ctx = L - w
    rng = np.random.default_rng(cfg.seed if seed is None else seed)

    q = np.empty((C, L, Hq, d), dtype=np.uint16)
    k = np.empty((C, L, Hkv, d), dtype=np.uint16)
    v = np.empty((C, L, Hkv, d), dtype=np.uint16)
    for c in range(C):                       # chunk at a time keeps the fp32 temporaries small
        q[c] = _normal_bf16(rng, (L, Hq, d))
        k[c] = _normal_bf16(rng, (L, Hkv, d))
        v[c] = _normal_bf16(rng, (L, Hkv, d))
    # one query window, replicated
    qw = _normal_bf16(rng, (w, Hq, d))
    kw = _normal_bf16(rng, (w, Hkv, d))
    vw = _normal_bf16(rng, (w, Hkv, d))
    q[:, ctx:] = qw
    k[:, ctx:] = kw
    v[:, ctx:] = vw

    # attention sink: key 0 of every chunk
    k[:, 0] = f32_to_bf16_bits(bf16_bits_to_f32(k[:, 0]) * np.float32(SINK_GAIN))

    # planted keys
    n_pc = min(cfg.n_planted_chunks, C)
    if cfg.planted_chunks and all(pc < C for pc in cfg.planted_chunks):
        planted_chunks = list(cfg.planted_chunks)[:n_pc]
    else:
        planted_chunks = sorted(rng.choice(C, size=n_pc, replace=False).tolist())
    G = Hq // Hkv
    qw_f = bf16_bits_to_f32(qw).reshape(w, Hkv, G, d)
    planted_pos = np.zeros((n_pc, Hkv, cfg.n_planted_keys), dtype=np.int64)
    for pi, pc in enumerate(planted_chunks):
        for hk in range(Hkv):
            u = qw_f[:, hk].reshape(-1, d).mean(axis=0)
            u = u / np.sqrt(np.mean(u * u))
            pos = np.sort(rng.choice(np.arange(1, ctx), size=cfg.n_planted_keys, replace=False))
            noise = rng.standard_normal((cfg.n_planted_keys, d), dtype=np.float32)
            planted = np.float32(PLANT_GAIN) * (np.float32(0.8) * u[None, :] + np.float32(0.2) * noise)
            k[pc, pos, hk] = f32_to_bf16_bits(planted.astype(np.float32))
            planted_pos[pi, hk] = pos
    return {"q": q, "k": k, "v": v, "planted_chunks": planted_chunks, "planted_pos": planted_pos}


# --------------------------------------------------------------------------- parallel-attention workloads
def make_parallel_attn_inputs(cfg: ParallelAttnConfig, B: int | None = None, Nk: int | None = None,
                              seed: int | None = None):
    """Draw one batch for the parallel (global) attention call.

    q_win [B,w,Hq,d] pre-RoPE; k_cache, v_cache [B,Hkv,Nk,d] (keys are taken as
    already rotated: N(0,1) is rotation-invariant in distribution);
    k_win, v_win [B,w,Hkv,d].  One x SINK_GAIN key at the start of each
    ``seg``-token segment of the cache.
    """
    B = cfg.B if B is None else int(B)
    Nk = cfg.Nk if Nk is None else int(Nk)
    w, Hq, Hkv, d = cfg.w, cfg.Hq, cfg.Hkv, cfg.d
    rng = np.random.default_rng(cfg.seed if seed is None else seed)
    q_win = _normal_bf16(rng, (B, w, Hq, d))
    k_win = _normal_bf16(rng, (B, w, Hkv, d))
    v_win = _normal_bf16(rng, (B, w, Hkv, d))
    k_cache = np.empty((B, Hkv, Nk, d), dtype=np.uint16)
    v_cache = np.empty((B, Hkv, Nk, d), dtype=np.uint16)
    for b in range(B):
        k_cache[b] = _normal_bf16(rng, (Hkv, Nk, d))
        v_cache[b] = _normal_bf16(rng, (Hkv, Nk, d))
    seg = max(1, min(cfg.seg, Nk))
    sink = np.arange(0, Nk, seg)
    k_cache[:, :, sink] = f32_to_bf16_bits(bf16_bits_to_f32(k_cache[:, :, sink]) * np.float32(SINK_GAIN))
    return {"q_win": q_win, "k_cache": k_cache, "v_cache": v_cache, "k_win": k_win, "v_win": v_win}
