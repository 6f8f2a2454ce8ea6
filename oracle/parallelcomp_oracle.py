"""CPU oracle for the ParallelComp attention hot path (arXiv 2502.14317, Sec. 3.1).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 numpy statement of what
each step of the path computes.  It shares no code with the CUDA library and is
imported only by the tests, by ``__graft_entry__.smoke()`` and by the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``.  The product path
never routes through it.

Every function is the textbook definition written out (no tiling, no online
softmax, no fusion).  ``numpy.matmul`` / ``numpy.sort`` serve as library steps.

Conventions (the paper is silent on each; the same readings bind the kernels):
  * bf16 tensors travel as uint16 bit patterns; arithmetic is fp64.
  * RoPE pairs element t with t + d/2 ("rotate-half"), angle p * theta^(-2t/d),
    positions restart at 0 in every chunk (position reuse, Sec. 3.1
    "Parallel attention").  Rotated q and k are rounded to bf16 (round to
    nearest even) because the tensor-core path consumes bf16 operands;
    everything after that rounding stays fp64.
  * Local attention is causal (decoder models), Eq. 1-2.
  * The window score of Eq. 6 sums the softmax probabilities of the last w rows
    over rows and over the G q-heads that share one kv-head.
  * Chunk ranking keeps the m chunks with the lowest self-information (Eq. 3-4);
    token ranking keeps the k highest window scores (Eq. 7); ties go to the
    lower index; outputs are listed in ascending index order.
  * The compressed cache (Eq. 9) concatenates the kept K/V of the kept chunks;
    the window's own K/V follow once.  Global attention is Eq. 10-11.

Pins (tests/test_oracle_*.py): closed forms for d=2 RoPE and two-token softmax,
row sums, shift invariance, a pure-Python triple loop, torch SDPA in fp64 as a
library special case, C=1 keep-all == full causal attention, brute-force sort,
k = ctx identity gather.  No function here is "parity unpinned" against those
definitions; what cannot be pinned is agreement with the authors' own code on
the conventions listed above (the paper prints no worked example).
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------- bf16 <-> fp64


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def f64_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 to the nearest bf16 (ties to even); returns uint16 bit patterns.

    Done directly on the fp64 value (not via fp32) so there is a single rounding.
    bf16 keeps 8 significant bits: scale the value so that its ulp is 1, round
    half to even with numpy.rint, scale back; the result is exactly representable
    in fp32, so the final cast is exact.
    """
    x = np.asarray(x, dtype=np.float64)
    mant, expo = np.frexp(x)                  # x = mant * 2**expo, 0.5 <= |mant| < 1
    # normal bf16 numbers: 8 significant bits -> ulp = 2**(expo-8); subnormals
    # (expo < -125) share the fixed ulp 2**-133
    e_ulp = np.maximum(expo - 8, -133)
    r = np.rint(np.ldexp(x, -e_ulp))          # ties to even
    y = np.ldexp(r, e_ulp).astype(np.float32)
    return (y.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# --------------------------------------------------------------------------- RoPE (position reuse)


def rope_angles(positions: np.ndarray, d: int, theta: float) -> np.ndarray:
    """phi[p, t] = p * theta**(-2t/d), t < d/2."""
    t = np.arange(d // 2, dtype=np.float64)
    inv_freq = np.float64(theta) ** (-2.0 * t / d)
    return np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]


def rope_rotate(x: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotate x[..., token, head, d] (fp64) by its token's position; pairs (t, t+d/2)."""
    d = x.shape[-1]
    h = d // 2
    phi = rope_angles(positions, d, theta)                    # [tokens, d/2]
    cos = np.cos(phi)[:, None, :]
    sin = np.sin(phi)[:, None, :]
    x1, x2 = x[..., :h], x[..., h:]
    out = np.empty_like(x)
    out[..., :h] = x1 * cos - x2 * sin
    out[..., h:] = x2 * cos + x1 * sin
    return out


def rope_bf16(bits: np.ndarray, theta: float, pos0: int = 0) -> np.ndarray:
    """bf16 in, bf16 out: rotate tokens at positions pos0, pos0+1, ... along axis -3."""
    n_tok = bits.shape[-3]
    pos = np.arange(pos0, pos0 + n_tok)
    return f64_to_bf16(rope_rotate(bf16_to_f64(bits), pos, theta))


# --------------------------------------------------------------------------- Eq. 1-2: chunk-local attention


def _softmax_rows(s: np.ndarray):
    """Plain softmax over the last axis; also returns log-sum-exp (natural log)."""
    mx = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - mx)
    z = np.sum(e, axis=-1, keepdims=True)
    return e / z, (mx + np.log(z))[..., 0]


def local_attention_rows(q_rot: np.ndarray, k_rot: np.ndarray, v: np.ndarray, c: int, h: int,
                         rows: np.ndarray, scale: float):
    """Eq. 1-2 for chunk c, q-head h, the given query rows (chunk-local indices).

    q_rot [C,L,Hq,d], k_rot/v [C,L,Hkv,d] are bf16 bit patterns, q/k already
    rotated.  Returns (A [len(rows), L] with zeros above the diagonal,
    O [len(rows), d], LSE [len(rows)]), all fp64.
    """
    Hq, Hkv = q_rot.shape[2], k_rot.shape[2]
    L = k_rot.shape[1]
    hk = h // (Hq // Hkv)
    rows = np.asarray(rows, dtype=np.int64)
    qf = bf16_to_f64(q_rot[c, rows, h])           # [R, d]
    kf = bf16_to_f64(k_rot[c, :, hk])             # [L, d]
    vf = bf16_to_f64(v[c, :, hk])
    s = (qf @ kf.T) * scale                       # [R, L]
    visible = np.arange(L)[None, :] <= rows[:, None]
    s = np.where(visible, s, -np.inf)
    a, lse = _softmax_rows(s)
    return a, a @ vf, lse


def local_attention(q_bits, k_bits, v_bits, theta: float, scale: float | None = None):
    """Full chunk-local causal attention of Eq. 1-2 with position reuse.

    q_bits [C,L,Hq,d], k_bits/v_bits [C,L,Hkv,d] bf16 patterns, pre-RoPE.
    Returns O [C,L,Hq,d] fp64, LSE [C,Hq,L] fp64, k_rot bits [C,L,Hkv,d].
    """
    C, L, Hq, d = q_bits.shape
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    q_rot = rope_bf16(q_bits, theta)
    k_rot = rope_bf16(k_bits, theta)
    O = np.empty((C, L, Hq, d), dtype=np.float64)
    LSE = np.empty((C, Hq, L), dtype=np.float64)
    rows = np.arange(L)
    for c in range(C):
        for h in range(Hq):
            _, o, lse = local_attention_rows(q_rot, k_rot, v_bits, c, h, rows, scale)
            O[c, :, h] = o
            LSE[c, h] = lse
    return O, LSE, k_rot


# --------------------------------------------------------------------------- Eq. 5-6: query-window score


def window_scores(q_rot, k_rot, v_bits, w: int, scale: float):
    """S[c,hkv,j] = sum over the G q-heads of kv-head hkv and the last w rows i of A[c,h,i,j].

    Also returns the window rows' outputs O_win [C,w,Hq,d] and LSE_win [C,Hq,w]
    (by-products of the same softmax rows).
    """
    C, L, Hq, d = q_rot.shape
    Hkv = k_rot.shape[2]
    G = Hq // Hkv
    rows = np.arange(L - w, L)
    S = np.zeros((C, Hkv, L), dtype=np.float64)
    O_win = np.empty((C, w, Hq, d), dtype=np.float64)
    LSE_win = np.empty((C, Hq, w), dtype=np.float64)
    for c in range(C):
        for h in range(Hq):
            a, o, lse = local_attention_rows(q_rot, k_rot, v_bits, c, h, rows, scale)
            S[c, h // G] += a.sum(axis=0)
            O_win[c, :, h] = o
            LSE_win[c, h] = lse
    return S, O_win, LSE_win


def chunk_score_from_lse(lse_win: np.ndarray) -> np.ndarray:
    """Single-layer stand-in for the self-information I_c of Eq. 3.

    The true I_c = -log P(X^q | X^c) needs the whole model and its LM head.  The
    stand-in is minus the mean, over q-heads and window rows, of the log-sum-exp
    of the window's attention logits: the more strongly the query window matches
    a chunk's keys, the lower the score.  lse_win [C,Hq,w] -> [C].
    """
    return -np.mean(np.asarray(lse_win, dtype=np.float64), axis=(1, 2))


# --------------------------------------------------------------------------- Eq. 3-4 / Eq. 7: ranking


def _rank_key_desc(x: np.ndarray) -> np.ndarray:
    """Key such that ascending stable sort lists the best (largest) first, NaN last."""
    x = np.asarray(x, dtype=np.float64)
    key = -x                                  # -0.0 and +0.0 both compare equal
    return np.where(np.isnan(x), np.inf, key)


def select_chunks(chunk_score: np.ndarray, m: int, lower_is_better: bool = True) -> np.ndarray:
    """Keep the m best chunks (Eq. 3-4: lowest self-information); ties -> lower id; ids ascending."""
    s = np.asarray(chunk_score, dtype=np.float32).astype(np.float64)
    key = _rank_key_desc(-s if lower_is_better else s)
    order = np.argsort(key, kind="stable")
    return np.sort(order[:m]).astype(np.int32)


def select_tokens(win_score: np.ndarray, kept: np.ndarray, n_cand: int, k: int) -> np.ndarray:
    """Eq. 7: per kept chunk and kv-head keep the k highest-scored context tokens.

    win_score [C,Hkv,L] float32 (the tensor handed over is ranked as it is),
    candidates are positions j < n_cand.  Returns idx [m,Hkv,k] int32, ascending
    positions; if k > n_cand the tail is padded with -1.
    """
    S = np.asarray(win_score, dtype=np.float32)
    _, Hkv, _ = S.shape
    m = len(kept)
    idx = np.full((m, Hkv, k), -1, dtype=np.int32)
    kk = min(k, n_cand)
    for r, c in enumerate(kept):
        for hk in range(Hkv):
            key = _rank_key_desc(S[c, hk, :n_cand])
            order = np.argsort(key, kind="stable")
            idx[r, hk, :kk] = np.sort(order[:kk])
    return idx


def select_tokens_calibrated(win_score: np.ndarray, kept: np.ndarray, n_cand: int, k: int, n_s: int, n_r: int,
                             lam_s: float, lam_m: float, lam_r: float) -> np.ndarray:
    """Eq. 8 (attention calibration) followed by Eq. 7: in every kept chunk and kv-head, first evict the
    candidates whose cumulative score EXCEEDS the threshold of their region, then keep the k highest-scored
    of the rest.  Regions (App. C): R_s = the first n_s candidate positions, R_r = the last n_r candidate
    positions, R_m = the remaining ones; a threshold of +inf switches a region off (the paper evicts one
    token type per layer range).  The comparison is taken on the float32 score against the float32
    threshold.  Returns idx [m,Hkv,k] int32, ascending positions, padded with -1 where fewer than k survive.
    """
    S = np.asarray(win_score, dtype=np.float32)
    _, Hkv, _ = S.shape
    lam = np.empty(n_cand, dtype=np.float32)
    lam[:] = np.float32(lam_m)
    lam[max(0, n_cand - n_r):] = np.float32(lam_r)
    lam[:min(n_s, n_cand)] = np.float32(lam_s)                  # the sink region wins where the two overlap
    idx = np.full((len(kept), Hkv, k), -1, dtype=np.int32)
    for r, c in enumerate(kept):
        for hk in range(Hkv):
            row = S[c, hk, :n_cand]
            alive = np.flatnonzero(~(row > lam))                 # NaN is not "greater": it stays (and ranks worst)
            order = alive[np.argsort(_rank_key_desc(row[alive]), kind="stable")]
            kk = min(k, len(order))
            idx[r, hk, :kk] = np.sort(order[:kk])
    return idx


def select_chunks_streaming(chunk_score: np.ndarray, m: int, batch: int) -> np.ndarray:
    """The paper's online fixed-size priority queue: chunks arrive in batches, the queue
    keeps the m lowest scores seen so far (ties -> lower id).  Must equal select_chunks."""
    s = np.asarray(chunk_score, dtype=np.float32).astype(np.float64)
    queue: list[tuple[float, int]] = []
    for start in range(0, len(s), batch):
        for c in range(start, min(start + batch, len(s))):
            queue.append((np.inf if np.isnan(s[c]) else s[c], c))
        queue.sort()
        del queue[m:]
    return np.sort(np.array([c for _, c in queue], dtype=np.int32))


# --------------------------------------------------------------------------- Eq. 7 + Eq. 9: compressed cache


def gather_kv(k_rot: np.ndarray, v_bits: np.ndarray, kept: np.ndarray, idx: np.ndarray):
    """Kc[hkv, r*k+t] = k_rot[kept[r], idx[r,hkv,t], hkv] (same for V); pos = idx.

    Padded entries (idx < 0) give zero rows and position -1.
    Returns (Kc, Vc) uint16 [Hkv, m*k, d] and pos int32 [Hkv, m*k].
    """
    m, Hkv, k = idx.shape
    d = k_rot.shape[-1]
    Kc = np.zeros((Hkv, m * k, d), dtype=np.uint16)
    Vc = np.zeros((Hkv, m * k, d), dtype=np.uint16)
    pos = np.full((Hkv, m * k), -1, dtype=np.int32)
    for r in range(m):
        for hk in range(Hkv):
            for t in range(k):
                j = int(idx[r, hk, t])
                if j < 0:
                    continue
                Kc[hk, r * k + t] = k_rot[kept[r], j, hk]
                Vc[hk, r * k + t] = v_bits[kept[r], j, hk]
                pos[hk, r * k + t] = j
    return Kc, Vc, pos


# --------------------------------------------------------------------------- Eq. 9-11: global attention


def parallel_attention(q_win_bits, q_pos0: int, theta: float, scale: float | None,
                       k_cache, v_cache, k_win, v_win, n_valid=None):
    """Global attention of the query window over the compressed cache.

    q_win_bits [B,w,Hq,d] pre-RoPE (rotated here at positions q_pos0..q_pos0+w-1,
    then rounded to bf16); k_cache/v_cache [B,Hkv,Nk,d] with keys already rotated
    (every kept key sits before the window, so all of them are visible to every
    query); k_win/v_win [B,w,Hkv,d], keys already rotated at the window's
    positions, causal among themselves.  ``n_valid`` (optional [B,Hkv]) masks
    cache entries >= n_valid (padding).  Returns Fg [B,w,Hq,d], LSE [B,Hq,w].
    """
    B, w, Hq, d = q_win_bits.shape
    Hkv, Nk = k_cache.shape[1], k_cache.shape[2]
    G = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    q_rot = rope_bf16(q_win_bits, theta, pos0=q_pos0)
    Fg = np.empty((B, w, Hq, d), dtype=np.float64)
    LSE = np.empty((B, Hq, w), dtype=np.float64)
    wk = k_win.shape[1]                       # window keys present (w, or 0 for a cache-only partial)
    causal = np.arange(wk)[None, :] <= np.arange(w)[:, None]
    for b in range(B):
        for h in range(Hq):
            hk = h // G
            qf = bf16_to_f64(q_rot[b, :, h])
            keys = np.concatenate([bf16_to_f64(k_cache[b, hk]), bf16_to_f64(k_win[b, :, hk])], axis=0)
            vals = np.concatenate([bf16_to_f64(v_cache[b, hk]), bf16_to_f64(v_win[b, :, hk])], axis=0)
            s = (qf @ keys.T) * scale
            vis = np.ones((w, Nk), dtype=bool)
            if n_valid is not None:
                vis = np.broadcast_to(np.arange(Nk)[None, :] < int(n_valid[b, hk]), (w, Nk))
            s = np.where(np.concatenate([vis, causal], axis=1), s, -np.inf)
            a, lse = _softmax_rows(s)
            Fg[b, :, h] = a @ vals
            LSE[b, h] = lse
    return Fg, LSE


# --------------------------------------------------------------------------- whole path


def hot_path(q_bits, k_bits, v_bits, *, w: int, theta: float, m: int, k: int,
             scale: float | None = None, chunk_score=None, tokens_first: bool = False,
             full_local: bool = True):
    """One pass of the whole path over one batch of chunks, in the order of Sec. 3.1.

    ``full_local`` False skips the bulk rows of Eq. 1-2 (only the window rows,
    which everything downstream depends on, are computed).  ``tokens_first``
    ranks tokens in every chunk before ranking chunks (the order of the paper's
    overview figure); the two orders must give the same cache.
    """
    C, L, Hq, d = q_bits.shape
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out = {}
    q_rot = rope_bf16(q_bits, theta)
    k_rot = rope_bf16(k_bits, theta)
    out["k_rot"] = k_rot
    if full_local:
        O, LSE, _ = local_attention(q_bits, k_bits, v_bits, theta, scale)
        out["O"], out["LSE"] = O, LSE
    S, O_win, LSE_win = window_scores(q_rot, k_rot, v_bits, w, scale)
    out["S"], out["O_win"], out["LSE_win"] = S, O_win, LSE_win
    score = chunk_score_from_lse(LSE_win) if chunk_score is None else np.asarray(chunk_score)
    out["chunk_score"] = score.astype(np.float32)
    S32 = S.astype(np.float32)
    if tokens_first:
        all_idx = select_tokens(S32, np.arange(C), L - w, k)
        kept = select_chunks(out["chunk_score"], m)
        idx = all_idx[kept]
    else:
        kept = select_chunks(out["chunk_score"], m)
        idx = select_tokens(S32, kept, L - w, k)
    out["kept"], out["idx"] = kept, idx
    Kc, Vc, pos = gather_kv(k_rot, v_bits, kept, idx)
    out["Kc"], out["Vc"], out["pos"] = Kc, Vc, pos
    # the window is the same in every chunk; take its copy from chunk kept[0]
    c0 = int(kept[0])
    Fg, LSEg = parallel_attention(q_bits[c0:c0 + 1, L - w:], L - w, theta, scale,
                                  Kc[None], Vc[None], k_rot[c0:c0 + 1, L - w:], v_bits[c0:c0 + 1, L - w:])
    out["Fg"], out["LSEg"] = Fg[0], LSEg[0]
    return out
