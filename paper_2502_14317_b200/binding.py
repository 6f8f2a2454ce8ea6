"""ctypes binding for libpc.so.  Same names as the C entry points, minus the ``pc_`` prefix.

Tensors are torch CUDA tensors; bf16 data is ``torch.bfloat16``.  Outputs and
workspaces are allocated here with torch (device memory only) unless passed in.
All calls enqueue on torch's current stream and do not synchronise.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_float, c_int32, c_int64, c_size_t, c_void_p, c_char_p, POINTER, Structure

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class PcError(RuntimeError):
    pass


class _PrefillDesc(Structure):
    _fields_ = [("C", c_int32), ("L", c_int32), ("w", c_int32), ("Hq", c_int32), ("Hkv", c_int32), ("d", c_int32),
                ("rope_theta", c_float), ("softmax_scale", c_float),
                ("q_stride", c_int64 * 3), ("k_stride", c_int64 * 3), ("v_stride", c_int64 * 3),
                ("o_stride", c_int64 * 3)]


def lib_path() -> str:
    return os.path.join(_HERE, "libpc.so")


def load_library():
    """Load libpc.so (built in-tree by ``python -m paper_2502_14317_b200.build``).  Fails loudly if absent."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = lib_path()
    if not os.path.exists(path):
        raise PcError(f"{path} not found: build it with `python -m paper_2502_14317_b200.build` "
                      "(there is no fallback path)")
    lib = ctypes.CDLL(path)
    lib.pc_status_string.restype = c_char_p
    lib.pc_status_string.argtypes = [c_int32]
    lib.pc_version.restype = c_int32
    lib.pc_chunk_prefill_attn_workspace_bytes.restype = c_size_t
    lib.pc_chunk_prefill_attn_workspace_bytes.argtypes = [POINTER(_PrefillDesc)]
    lib.pc_chunk_prefill_attn.restype = c_int32
    lib.pc_chunk_prefill_attn.argtypes = [POINTER(_PrefillDesc)] + [c_void_p] * 11 + [c_size_t, c_void_p]
    lib.pc_rope_position_reuse_workspace_bytes.restype = c_size_t
    lib.pc_rope_position_reuse_workspace_bytes.argtypes = [c_int32, c_int32]
    lib.pc_rope_position_reuse.restype = c_int32
    lib.pc_rope_position_reuse.argtypes = [c_void_p] + [c_int32] * 4 + [c_float, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.pc_debug_bounded_wait_test.restype = c_int32
    lib.pc_debug_bounded_wait_test.argtypes = [c_int64, c_int32]
    lib.pc_launch_count.restype = ctypes.c_uint64
    lib.pc_launch_count.argtypes = []
    lib.pc_chunk_score_from_lse.restype = c_int32
    lib.pc_chunk_score_from_lse.argtypes = [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p]
    lib.pc_score_select_chunks.restype = c_int32
    lib.pc_score_select_chunks.argtypes = [c_void_p] + [c_int32] * 5 + [c_void_p, c_void_p, c_void_p]
    lib.pc_select_chunks.restype = c_int32
    lib.pc_select_chunks.argtypes = [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p]
    lib.pc_select_tokens.restype = c_int32
    lib.pc_select_tokens.argtypes = [c_void_p, c_void_p] + [c_int32] * 6 + [c_void_p, c_void_p]
    lib.pc_select_tokens_calibrated.restype = c_int32
    lib.pc_select_tokens_calibrated.argtypes = [c_void_p, c_void_p] + [c_int32] * 8 + [c_float] * 3 + [c_void_p, c_void_p]
    lib.pc_gather_kv.restype = c_int32
    lib.pc_gather_kv.argtypes = [c_void_p, c_void_p, POINTER(c_int64), c_void_p, c_void_p] + [c_int32] * 4 + \
                                [c_void_p, c_void_p, c_void_p, c_void_p]
    lib.pc_queue_init.restype = c_int32
    lib.pc_queue_init.argtypes = [c_int32, c_void_p, c_void_p, c_void_p]
    lib.pc_queue_update.restype = c_int32
    lib.pc_queue_update.argtypes = [c_void_p] + [c_int32] * 4 + [c_void_p] * 4
    lib.pc_queue_gather.restype = c_int32
    lib.pc_queue_gather.argtypes = [c_void_p, c_void_p, POINTER(c_int64), c_void_p, c_void_p] + [c_int32] * 4 + \
        [c_void_p] * 4
    lib.pc_queue_select_gather.restype = c_int32
    lib.pc_queue_select_gather.argtypes = [c_void_p, c_void_p, c_void_p, POINTER(c_int64), c_void_p] + [c_int32] * 6 + [c_void_p] * 4
    lib.pc_queue_emit.restype = c_int32
    lib.pc_queue_emit.argtypes = [c_void_p] + [c_int32] * 4 + [c_void_p] * 9
    lib.pc_parallel_attn_workspace_bytes.restype = c_size_t
    lib.pc_parallel_attn_workspace_bytes.argtypes = [c_int32] * 6
    lib.pc_parallel_attn.restype = c_int32
    lib.pc_parallel_attn.argtypes = [c_int32] * 6 + [c_void_p, c_int32, c_float, c_float] + [c_void_p] * 8 + \
                                    [c_size_t, c_void_p]
    lib.pc_parallel_attn_append.restype = c_int32
    lib.pc_parallel_attn_append.argtypes = [c_int32] * 7 + [c_void_p, c_int32, c_float, c_float] + [c_void_p] * 8 + \
                                           [c_size_t, c_void_p]
    lib.pc_parallel_attn_static_scratch_bytes.restype = c_size_t
    lib.pc_parallel_attn_static_scratch_bytes.argtypes = []
    lib.pc_parallel_attn_static.restype = c_int32
    lib.pc_parallel_attn_static.argtypes = [c_int32] * 6 + [c_void_p, c_int32, c_float, c_float] + [c_void_p] * 8
    _LIB = lib
    return lib


def version() -> int:
    return int(load_library().pc_version())


def launch_count() -> int:
    """pc_launch_count: kernels launched by the library in this process so far."""
    return int(load_library().pc_launch_count())


def status_string(code: int) -> str:
    return load_library().pc_status_string(int(code)).decode()


def _check(rc: int, what: str):
    if rc != 0:
        raise PcError(f"{what} failed: {status_string(rc)} ({rc})")


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _need_cuda(*tensors):
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise PcError("tensors must live on a CUDA device")


def _make_desc(q, k, v, o, w, rope_theta, softmax_scale):
    C, L, Hq, d = q.shape
    Hkv = k.shape[2]
    desc = _PrefillDesc(C, L, w, Hq, Hkv, d, float(rope_theta), float(softmax_scale))
    for name, t in (("q_stride", q), ("k_stride", k), ("v_stride", v), ("o_stride", o)):
        if t.stride(3) != 1:
            raise PcError("head dimension must be contiguous")
        getattr(desc, name)[0], getattr(desc, name)[1], getattr(desc, name)[2] = t.stride(0), t.stride(1), t.stride(2)
    return desc


def chunk_prefill_attn_workspace_bytes(C, L, w, Hq, Hkv, d, k_rot_in_workspace=False) -> int:
    desc = _PrefillDesc(C, L, w, Hq, Hkv, d, 10000.0, 0.0)
    need = int(load_library().pc_chunk_prefill_attn_workspace_bytes(ctypes.byref(desc)))
    if need and k_rot_in_workspace:                           # rotated keys in the workspace (k_rot = NULL in the call)
        need += (C * L * Hkv * d * 2 + 255) // 256 * 256
    return need


def chunk_prefill_attn(q, k, v, *, w, rope_theta, softmax_scale=0.0, want_lse=False, out=None, k_rot=None,
                       win_score=None, win_lse=None, lse=None, status=None, workspace=None, chunk_len=None):
    """pc_chunk_prefill_attn: q [C,L,Hq,d], k/v [C,L,Hkv,d] bf16 (pre-RoPE); chunk_len: int32 [C] device tensor
    (tokens per chunk, window included) or None for full chunks.

    Returns dict(o, k_rot, win_score, win_lse, lse, status, workspace).
    """
    lib = load_library()
    _need_cuda(q, k, v)
    C, L, Hq, d = q.shape
    Hkv = k.shape[2]
    dev = q.device
    o = torch.empty((C, L, Hq, d), dtype=torch.bfloat16, device=dev) if out is None else out
    if k_rot is None:
        k_rot = torch.empty((C, L, Hkv, d), dtype=torch.bfloat16, device=dev)
    if win_score is None:
        win_score = torch.empty((C, Hkv, L), dtype=torch.float32, device=dev)
    if win_lse is None:
        win_lse = torch.empty((C, Hq, w), dtype=torch.float32, device=dev)
    if lse is None and want_lse:
        lse = torch.empty((C, Hq, L), dtype=torch.float32, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    desc = _make_desc(q, k, v, o, w, rope_theta, softmax_scale)
    need = int(lib.pc_chunk_prefill_attn_workspace_bytes(ctypes.byref(desc)))
    if workspace is None or workspace.numel() < need:          # need == 0: a bad descriptor, which the call below names
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    if chunk_len is not None and (chunk_len.dtype != torch.int32 or chunk_len.numel() != C or not chunk_len.is_cuda):
        raise PcError("chunk_len must be an int32 CUDA tensor with one entry per chunk")
    rc = lib.pc_chunk_prefill_attn(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(chunk_len), _ptr(o), _ptr(k_rot),
                                   _ptr(lse), _ptr(win_score), _ptr(win_lse), _ptr(status), _ptr(workspace),
                                   workspace.numel(), _stream())
    _check(rc, "pc_chunk_prefill_attn")
    return {"o": o, "k_rot": k_rot, "win_score": win_score, "win_lse": win_lse, "lse": lse, "status": status,
            "workspace": workspace}


def rope_position_reuse(x, *, rope_theta, out=None, workspace=None):
    """pc_rope_position_reuse: x [C,L,H,d] bf16 contiguous -> the rotated tensor (positions 0..L-1 in every chunk)."""
    lib = load_library()
    _need_cuda(x)
    if not x.is_contiguous():
        raise PcError("pc_rope_position_reuse takes a contiguous tensor")
    C, L, H, d = x.shape
    out = torch.empty_like(x) if out is None else out
    need = int(lib.pc_rope_position_reuse_workspace_bytes(L, d))
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=x.device)
    _check(lib.pc_rope_position_reuse(_ptr(x), C, L, H, d, float(rope_theta), _ptr(out), _ptr(workspace), workspace.numel(),
                                      _stream()), "pc_rope_position_reuse")
    return out


def chunk_score_from_lse(win_lse, out=None):
    """pc_chunk_score_from_lse: win_lse [C,Hq,w] fp32 -> [C] fp32."""
    lib = load_library()
    _need_cuda(win_lse)
    C, Hq, w = win_lse.shape
    out = torch.empty(C, dtype=torch.float32, device=win_lse.device) if out is None else out
    _check(lib.pc_chunk_score_from_lse(_ptr(win_lse), C, Hq, w, _ptr(out), _stream()), "pc_chunk_score_from_lse")
    return out


def select_chunks(chunk_score, m, lower_is_better=True, out=None):
    """pc_select_chunks: chunk_score [C] fp32 -> kept [m] int32 (ascending ids)."""
    lib = load_library()
    _need_cuda(chunk_score)
    C = chunk_score.numel()
    out = torch.empty(m, dtype=torch.int32, device=chunk_score.device) if out is None else out
    _check(lib.pc_select_chunks(_ptr(chunk_score), C, int(m), int(bool(lower_is_better)), _ptr(out), _stream()),
           "pc_select_chunks")
    return out


def score_select_chunks(win_lse, m, lower_is_better=True, score_out=None, kept_out=None):
    """pc_score_select_chunks: win_lse [C,Hq,w] fp32 -> (chunk_score [C] fp32, kept [m] int32), one launch for C <= 64."""
    lib = load_library()
    _need_cuda(win_lse)
    C, Hq, w = win_lse.shape
    score = torch.empty(C, dtype=torch.float32, device=win_lse.device) if score_out is None else score_out
    kept = torch.empty(m, dtype=torch.int32, device=win_lse.device) if kept_out is None else kept_out
    _check(lib.pc_score_select_chunks(_ptr(win_lse), C, Hq, w, int(m), int(bool(lower_is_better)), _ptr(score), _ptr(kept),
                                      _stream()), "pc_score_select_chunks")
    return score, kept


def select_tokens(win_score, kept, n_cand, k, out=None):
    """pc_select_tokens: win_score [C,Hkv,L] fp32, kept [m] int32 -> idx [m,Hkv,k] int32."""
    lib = load_library()
    _need_cuda(win_score, kept)
    C, Hkv, L = win_score.shape
    m = kept.numel()
    out = torch.empty((m, Hkv, k), dtype=torch.int32, device=win_score.device) if out is None else out
    _check(lib.pc_select_tokens(_ptr(win_score), _ptr(kept), C, m, Hkv, L, int(n_cand), int(k), _ptr(out), _stream()),
           "pc_select_tokens")
    return out


def select_tokens_calibrated(win_score, kept, n_cand, k, *, n_s=100, n_r=100, lambda_s=float("inf"),
                             lambda_m=float("inf"), lambda_r=float("inf"), out=None):
    """pc_select_tokens_calibrated: Eq. 8 eviction of over-attended tokens per region, then the top-k of Eq. 7."""
    lib = load_library()
    _need_cuda(win_score, kept)
    C, Hkv, L = win_score.shape
    m = kept.numel()
    out = torch.empty((m, Hkv, k), dtype=torch.int32, device=win_score.device) if out is None else out
    _check(lib.pc_select_tokens_calibrated(_ptr(win_score), _ptr(kept), C, m, Hkv, L, int(n_cand), int(k), int(n_s),
                                           int(n_r), float(lambda_s), float(lambda_m), float(lambda_r), _ptr(out),
                                           _stream()), "pc_select_tokens_calibrated")
    return out


def gather_kv(k_src, v_src, kept, idx, k_out=None, v_out=None, pos_out=None, want_pos=True):
    """pc_gather_kv: k_src/v_src [C,L,Hkv,d] bf16 -> (k_out, v_out [Hkv, m*k, d], pos [Hkv, m*k])."""
    lib = load_library()
    _need_cuda(k_src, v_src, kept, idx)
    C, L, Hkv, d = k_src.shape
    m, _, k = idx.shape
    dev = k_src.device
    if k_src.stride() != v_src.stride() or k_src.stride(3) != 1:
        raise PcError("k_src and v_src must share strides with a contiguous head dimension")
    k_out = torch.empty((Hkv, m * k, d), dtype=torch.bfloat16, device=dev) if k_out is None else k_out
    v_out = torch.empty((Hkv, m * k, d), dtype=torch.bfloat16, device=dev) if v_out is None else v_out
    if pos_out is None and want_pos:
        pos_out = torch.empty((Hkv, m * k), dtype=torch.int32, device=dev)
    strides = (c_int64 * 3)(k_src.stride(0), k_src.stride(1), k_src.stride(2))
    _check(lib.pc_gather_kv(_ptr(k_src), _ptr(v_src), strides, _ptr(kept), _ptr(idx), m, Hkv, k, d, _ptr(k_out),
                            _ptr(v_out), _ptr(pos_out), _stream()), "pc_gather_kv")
    return k_out, v_out, pos_out


def queue_init(m, Hkv, k, d, device):
    """pc_queue_init: an empty online chunk queue of m slots with its slot storage.

    Returns the state dict {q_score [m] f32, q_chunk [m] i32, q_k, q_v [Hkv, m*k, d] bf16, q_pos [Hkv, m*k] i32,
    slot_src [m] i32}."""
    lib = load_library()
    st = {"q_score": torch.empty(m, dtype=torch.float32, device=device),
          "q_chunk": torch.empty(m, dtype=torch.int32, device=device),
          "q_k": torch.empty((Hkv, m * k, d), dtype=torch.bfloat16, device=device),
          "q_v": torch.empty((Hkv, m * k, d), dtype=torch.bfloat16, device=device),
          "q_pos": torch.empty((Hkv, m * k), dtype=torch.int32, device=device),
          "slot_src": torch.empty(m, dtype=torch.int32, device=device),
          "m": m, "Hkv": Hkv, "k": k, "d": d}
    _need_cuda(st["q_score"])
    _check(lib.pc_queue_init(m, _ptr(st["q_score"]), _ptr(st["q_chunk"]), _stream()), "pc_queue_init")
    return st


def queue_update(state, chunk_score, chunk_id0, lower_is_better=True):
    """pc_queue_update: push the scores of a batch of chunks (ids chunk_id0, chunk_id0 + 1, ...); fills state['slot_src']."""
    lib = load_library()
    _need_cuda(chunk_score)
    if chunk_score.dtype != torch.float32 or not chunk_score.is_contiguous():
        raise PcError("chunk_score must be contiguous float32")
    _check(lib.pc_queue_update(_ptr(chunk_score), chunk_score.numel(), int(chunk_id0), 1 if lower_is_better else 0,
                               state["m"], _ptr(state["q_score"]), _ptr(state["q_chunk"]), _ptr(state["slot_src"]),
                               _stream()), "pc_queue_update")
    return state["slot_src"]


def queue_gather(state, k_src, v_src, idx):
    """pc_queue_gather: move the compressed caches of the chunks that entered the queue into their slots.

    k_src/v_src [Cb,L,Hkv,d] bf16 (rotated keys, values of the batch), idx [Cb,Hkv,k] from select_tokens on all chunks."""
    lib = load_library()
    _need_cuda(k_src, v_src, idx)
    Cb, L, Hkv, d = k_src.shape
    if idx.shape != (Cb, Hkv, state["k"]) or Hkv != state["Hkv"] or d != state["d"]:
        raise PcError("idx must be [Cb, Hkv, k] for the queue's k; Hkv and d must match the queue")
    if k_src.stride() != v_src.stride() or k_src.stride(3) != 1:
        raise PcError("k_src and v_src must share strides with a contiguous head dimension")
    strides = (c_int64 * 3)(k_src.stride(0), k_src.stride(1), k_src.stride(2))
    _check(lib.pc_queue_gather(_ptr(k_src), _ptr(v_src), strides, _ptr(state["slot_src"]), _ptr(idx), state["m"], Hkv,
                               state["k"], d, _ptr(state["q_k"]), _ptr(state["q_v"]), _ptr(state["q_pos"]), _stream()),
           "pc_queue_gather")


def queue_select_gather(state, win_score, k_src, v_src, n_cand):
    """pc_queue_select_gather: rank the tokens of the chunks that entered the queue and move their kept rows into
    their slots, one launch.  win_score [Cb,Hkv,L] fp32, k_src/v_src [Cb,L,Hkv,d] bf16 of the batch."""
    lib = load_library()
    _need_cuda(win_score, k_src, v_src)
    Cb, L, Hkv, d = k_src.shape
    if Hkv != state["Hkv"] or d != state["d"] or win_score.shape != (Cb, Hkv, L) or not win_score.is_contiguous():
        raise PcError("win_score must be contiguous [Cb, Hkv, L]; Hkv and d must match the queue")
    if k_src.stride() != v_src.stride() or k_src.stride(3) != 1:
        raise PcError("k_src and v_src must share strides with a contiguous head dimension")
    strides = (c_int64 * 3)(k_src.stride(0), k_src.stride(1), k_src.stride(2))
    _check(lib.pc_queue_select_gather(_ptr(win_score), _ptr(k_src), _ptr(v_src), strides, _ptr(state["slot_src"]), state["m"],
                                      Hkv, L, int(n_cand), state["k"], d, _ptr(state["q_k"]), _ptr(state["q_v"]),
                                      _ptr(state["q_pos"]), _stream()), "pc_queue_select_gather")


def queue_emit(state, k_out=None, v_out=None, pos_out=None, kept_out=None):
    """pc_queue_emit: the surviving chunks in ascending id order -> (kept [m], k_out, v_out [Hkv, m*k, d], pos [Hkv, m*k])."""
    lib = load_library()
    m, Hkv, k, d = state["m"], state["Hkv"], state["k"], state["d"]
    dev = state["q_k"].device
    k_out = torch.empty((Hkv, m * k, d), dtype=torch.bfloat16, device=dev) if k_out is None else k_out
    v_out = torch.empty((Hkv, m * k, d), dtype=torch.bfloat16, device=dev) if v_out is None else v_out
    pos_out = torch.empty((Hkv, m * k), dtype=torch.int32, device=dev) if pos_out is None else pos_out
    kept_out = torch.empty(m, dtype=torch.int32, device=dev) if kept_out is None else kept_out
    order = state.setdefault("slot_order", torch.empty(m, dtype=torch.int32, device=dev))
    _check(lib.pc_queue_emit(_ptr(state["q_chunk"]), m, Hkv, k, d, _ptr(state["q_k"]), _ptr(state["q_v"]),
                             _ptr(state["q_pos"]), _ptr(kept_out), _ptr(order), _ptr(k_out), _ptr(v_out), _ptr(pos_out),
                             _stream()), "pc_queue_emit")
    return kept_out, k_out, v_out, pos_out


def parallel_attn_workspace_bytes(B, w, Hq, Hkv, d, Nk) -> int:
    return int(load_library().pc_parallel_attn_workspace_bytes(B, w, Hq, Hkv, d, Nk))


def parallel_attn(q_win, k_cache, v_cache, k_win, v_win, *, q_pos0, rope_theta, softmax_scale=0.0, out=None,
                  lse_out=None, want_lse=False, status=None, workspace=None):
    """pc_parallel_attn: q_win [B,w,Hq,d] (pre-RoPE), k_cache/v_cache [B,Hkv,Nk,d], k_win/v_win [B,w,Hkv,d]."""
    lib = load_library()
    _need_cuda(q_win, k_cache, v_cache, k_win, v_win)
    B, w, Hq, d = q_win.shape
    Hkv, Nk = k_cache.shape[1], k_cache.shape[2]
    dev = q_win.device
    for t in (q_win, k_cache, v_cache, k_win, v_win):
        if not t.is_contiguous():
            raise PcError("pc_parallel_attn takes contiguous tensors")
    out = torch.empty((B, w, Hq, d), dtype=torch.bfloat16, device=dev) if out is None else out
    if lse_out is None and want_lse:
        lse_out = torch.empty((B, Hq, w), dtype=torch.float32, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    need = parallel_attn_workspace_bytes(B, w, Hq, Hkv, d, Nk)
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    rc = lib.pc_parallel_attn(B, w, Hq, Hkv, d, Nk, _ptr(q_win), int(q_pos0), float(rope_theta), float(softmax_scale),
                              _ptr(k_cache), _ptr(v_cache), _ptr(k_win), _ptr(v_win), _ptr(out), _ptr(lse_out),
                              _ptr(status), _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "pc_parallel_attn")
    return {"out": out, "lse": lse_out, "status": status, "workspace": workspace}


def parallel_attn_append(q_win, k_cache, v_cache, n_valid, k_win, v_win, *, q_pos0, rope_theta, softmax_scale=0.0,
                         out=None, lse_out=None, want_lse=False, status=None, workspace=None):
    """pc_parallel_attn_append: as parallel_attn over the first ``n_valid`` entries of k_cache / v_cache
    [B,Hkv,Nk_cap,d]; afterwards k_win, v_win are written to entries n_valid .. n_valid + w - 1 of the caches."""
    lib = load_library()
    _need_cuda(q_win, k_cache, v_cache, k_win, v_win)
    B, w, Hq, d = q_win.shape
    Hkv, cap = k_cache.shape[1], k_cache.shape[2]
    dev = q_win.device
    for t in (q_win, k_cache, v_cache, k_win, v_win):
        if not t.is_contiguous():
            raise PcError("pc_parallel_attn_append takes contiguous tensors")
    out = torch.empty((B, w, Hq, d), dtype=torch.bfloat16, device=dev) if out is None else out
    if lse_out is None and want_lse:
        lse_out = torch.empty((B, Hq, w), dtype=torch.float32, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    need = parallel_attn_workspace_bytes(B, w, Hq, Hkv, d, int(n_valid))
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    rc = lib.pc_parallel_attn_append(B, w, Hq, Hkv, d, int(n_valid), cap, _ptr(q_win), int(q_pos0), float(rope_theta),
                                     float(softmax_scale), _ptr(k_cache), _ptr(v_cache), _ptr(k_win), _ptr(v_win),
                                     _ptr(out), _ptr(lse_out), _ptr(status), _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "pc_parallel_attn_append")
    return {"out": out, "lse": lse_out, "status": status, "workspace": workspace}


def parallel_attn_static_scratch_bytes() -> int:
    return int(load_library().pc_parallel_attn_static_scratch_bytes())


def parallel_attn_static(q_win, k_cache, v_cache, k_win, v_win, out, *, q_pos0, rope_theta, softmax_scale=0.0,
                         lse_out=None, status=None):
    """pc_parallel_attn_static: pc_parallel_attn for callers that may not allocate device memory.

    Nothing is allocated here either: ``out`` (and ``lse_out`` / ``status`` if wanted) must be passed in, and
    the scratch is the fixed array inside the library.  Shapes that need more scratch than that array
    holds are refused.  Calls on one device share the array, so keep them on one stream.
    """
    lib = load_library()
    _need_cuda(q_win, k_cache, v_cache, k_win, v_win, out)
    B, w, Hq, d = q_win.shape
    Hkv, Nk = k_cache.shape[1], k_cache.shape[2]
    for t in (q_win, k_cache, v_cache, k_win, v_win, out):
        if not t.is_contiguous():
            raise PcError("pc_parallel_attn_static takes contiguous tensors")
    need, have = parallel_attn_workspace_bytes(B, w, Hq, Hkv, d, Nk), parallel_attn_static_scratch_bytes()
    if need > have:
        raise PcError(f"pc_parallel_attn_static: this shape needs {need} bytes of scratch, the built-in array holds "
                      f"{have}; use pc_parallel_attn with a workspace instead")
    rc = lib.pc_parallel_attn_static(B, w, Hq, Hkv, d, Nk, _ptr(q_win), int(q_pos0), float(rope_theta),
                                     float(softmax_scale), _ptr(k_cache), _ptr(v_cache), _ptr(k_win), _ptr(v_win),
                                     _ptr(out), _ptr(lse_out), _ptr(status), _stream())
    _check(rc, "pc_parallel_attn_static")
    return out


def hot_path(q, k, v, *, w, rope_theta, m, k_keep, softmax_scale=0.0, chunk_score=None, buffers=None):
    """One pass of the whole path on the current stream: the five C-ABI calls chained, no host sync.

    ``chunk_score`` (device fp32 [C]) stands for the self-information of Eq. 3; if None the
    single-layer stand-in computed from the window log-sum-exp is used.
    ``buffers`` (dict) lets repeated calls reuse outputs and workspaces.
    """
    b = {} if buffers is None else buffers
    C, L, Hq, d = q.shape
    pre = chunk_prefill_attn(q, k, v, w=w, rope_theta=rope_theta, softmax_scale=softmax_scale, out=b.get("o"),
                             k_rot=b.get("k_rot"), win_score=b.get("win_score"), win_lse=b.get("win_lse"),
                             status=b.get("status"), workspace=b.get("ws_prefill"))
    if chunk_score is not None:
        score, kept = chunk_score, select_chunks(chunk_score, m, True, out=b.get("kept"))
    else:
        score, kept = score_select_chunks(pre["win_lse"], m, True, score_out=b.get("chunk_score"), kept_out=b.get("kept"))
    idx = select_tokens(pre["win_score"], kept, L - w, k_keep, out=b.get("idx"))
    kc, vc, pos = gather_kv(pre["k_rot"], v, kept, idx, k_out=b.get("kc"), v_out=b.get("vc"), pos_out=b.get("pos"))
    # the window is the same in every chunk: take it from chunk 0 (views, no copy)
    q_win = q[0:1, L - w:].contiguous() if not q[0:1, L - w:].is_contiguous() else q[0:1, L - w:]
    k_win = pre["k_rot"][0:1, L - w:]
    v_win = v[0:1, L - w:]
    if not v_win.is_contiguous():
        v_win = v_win.contiguous()
    pa = parallel_attn(q_win, kc.unsqueeze(0), vc.unsqueeze(0), k_win, v_win, q_pos0=L - w, rope_theta=rope_theta,
                       softmax_scale=softmax_scale, out=b.get("fg"), status=pre["status"], workspace=b.get("ws_par"))
    res = {"o": pre["o"], "k_rot": pre["k_rot"], "win_score": pre["win_score"], "win_lse": pre["win_lse"],
           "chunk_score": score, "kept": kept, "idx": idx, "kc": kc, "vc": vc, "pos": pos, "fg": pa["out"],
           "status": pre["status"], "ws_prefill": pre["workspace"], "ws_par": pa["workspace"]}
    if buffers is not None:
        buffers.update({"o": res["o"], "k_rot": res["k_rot"], "win_score": res["win_score"], "win_lse": res["win_lse"],
                        "chunk_score": score if chunk_score is None else b.get("chunk_score"), "kept": kept, "idx": idx,
                        "kc": kc, "vc": vc, "pos": pos, "fg": res["fg"], "status": res["status"],
                        "ws_prefill": res["ws_prefill"], "ws_par": res["ws_par"]})
    return res


def hot_path_streaming(q, k, v, *, w, rope_theta, m, k_keep, batch=None, softmax_scale=0.0, chunk_score=None,
                       buffers=None):
    """The whole path with the chunks taken one batch at a time through the online chunk queue.

    Per batch: chunk-local attention, queue update, then the chunks that entered the queue are ranked per kv-head
    and their kept rows copied into their slots (one launch; a chunk that does not enter is dropped whole); the batch's outputs
    (attention output, rotated keys, window scores) live in buffers of batch size that the next batch
    overwrites, so device memory beyond the inputs is O(batch + m) chunks whatever C is.  After the last batch
    the queue is emitted in chunk order and the window attends over it.  Same results as :func:`hot_path`
    (kept chunks, indices and compressed cache bit for bit).

    q, k, v are either whole device tensors [C,L,*,d], cut into batches of ``batch`` chunks, or lists of
    per-batch tensors [Cb,L_b,*,d].  In a list the chunk length may differ from batch to batch (a shorter
    last chunk is a batch of its own: its window directly follows its context, and only the k_keep tokens it
    contributes persist); every L_b - w must be at least k_keep.  The query window of the global attention is
    taken from the first chunk of the first batch.  A caller that streams from elsewhere makes the same calls
    on its own batches.
    """
    b = {} if buffers is None else buffers
    if isinstance(q, (list, tuple)):
        batches = list(zip(q, k, v))
    else:
        if batch is None:
            raise PcError("hot_path_streaming needs a batch size for whole tensors")
        batches = [(q[c0:c0 + batch], k[c0:c0 + batch], v[c0:c0 + batch]) for c0 in range(0, q.shape[0], batch)]
    q0, k0, v0 = batches[0]
    _, L0, Hq, d = q0.shape
    Hkv = k0.shape[2]
    dev = q0.device
    n_max = max(bq.shape[0] for bq, _, _ in batches)
    if "queue" not in b:
        b["queue"] = queue_init(m, Hkv, k_keep, d, dev)
    else:
        lib = load_library()
        _check(lib.pc_queue_init(m, _ptr(b["queue"]["q_score"]), _ptr(b["queue"]["q_chunk"]), _stream()), "pc_queue_init")
    if "ids" not in b or b["ids"].numel() < n_max:
        b["ids"] = torch.arange(n_max, dtype=torch.int32, device=dev)
    qu = b["queue"]
    c0 = 0
    k_win = None
    for bq, bk, bv in batches:
        n, L = bq.shape[0], bq.shape[1]
        if L - w < k_keep:
            raise PcError("a chunk of %d tokens has fewer than k_keep = %d context tokens" % (L, k_keep))
        pb = b.setdefault("pre_%dx%d" % (n, L), {})            # buffers per batch shape
        pre = chunk_prefill_attn(bq, bk, bv, w=w, rope_theta=rope_theta, softmax_scale=softmax_scale,
                                 out=pb.get("o"), k_rot=pb.get("k_rot"), win_score=pb.get("win_score"),
                                 win_lse=pb.get("win_lse"), status=b.get("status"), workspace=pb.get("workspace"))
        b["status"] = pre["status"]
        pb.update({"o": pre["o"], "k_rot": pre["k_rot"], "win_score": pre["win_score"], "win_lse": pre["win_lse"],
                   "workspace": pre["workspace"]})
        if chunk_score is not None:
            score = chunk_score[c0:c0 + n]
        else:
            score = chunk_score_from_lse(pre["win_lse"], out=pb.get("score"))
            pb["score"] = score
        queue_update(qu, score, c0, True)
        if k_keep <= 10240:                                    # rank and compact the chunks that entered, one launch
            queue_select_gather(qu, pre["win_score"], pre["k_rot"], bv, L - w)
        else:
            idx = select_tokens(pre["win_score"], b["ids"][:n], L - w, k_keep, out=pb.get("idx"))
            pb["idx"] = idx
            queue_gather(qu, pre["k_rot"], bv, idx)
        if k_win is None:                                      # the window is the same in every chunk: keep the first
            k_win = b.get("k_win")
            if k_win is None or k_win.shape != (1, w, Hkv, d):
                k_win = torch.empty((1, w, Hkv, d), dtype=torch.bfloat16, device=dev)
            k_win.copy_(pre["k_rot"][0:1, L - w:])
            b["k_win"] = k_win
        c0 += n
    kept, kc, vc, pos = queue_emit(qu, k_out=b.get("kc"), v_out=b.get("vc"), pos_out=b.get("pos"), kept_out=b.get("kept"))
    b.update({"kc": kc, "vc": vc, "pos": pos, "kept": kept})
    q_win = q0[0:1, L0 - w:]
    q_win = q_win if q_win.is_contiguous() else q_win.contiguous()
    v_win = v0[0:1, L0 - w:]
    v_win = v_win if v_win.is_contiguous() else v_win.contiguous()
    pa = parallel_attn(q_win, kc.unsqueeze(0), vc.unsqueeze(0), k_win, v_win, q_pos0=L0 - w, rope_theta=rope_theta,
                       softmax_scale=softmax_scale, out=b.get("fg"), status=b["status"], workspace=b.get("ws_par"))
    b.update({"fg": pa["out"], "ws_par": pa["workspace"]})
    return {"kept": kept, "kc": kc, "vc": vc, "pos": pos, "fg": pa["out"], "status": b["status"]}


def hot_path_from_host(hq, hk, hv, *, w, rope_theta, m, k_keep, softmax_scale=0.0, n_groups=4, buffers=None):
    """The whole path for inputs that live in pinned HOST memory (hq [C,L,Hq,d], hk/hv [C,L,Hkv,d], bf16).

    Chunks are independent until the chunk ranking, so they are uploaded in ``n_groups`` groups on a copy
    stream while the attention of the previous group runs on the current stream; the ranking, gather and
    parallel attention follow once all groups are done.  ``buffers`` (dict) keeps the device tensors,
    streams and events between calls.  Returns the same dict as :func:`hot_path` (device tensors).
    """
    b = {} if buffers is None else buffers
    C, L, Hq, d = hq.shape
    Hkv = hk.shape[2]
    dev = torch.device("cuda", torch.cuda.current_device())
    if "q" not in b:
        b["q"] = torch.empty(hq.shape, dtype=torch.bfloat16, device=dev)
        b["k"] = torch.empty(hk.shape, dtype=torch.bfloat16, device=dev)
        b["v"] = torch.empty(hv.shape, dtype=torch.bfloat16, device=dev)
        b["o"] = torch.empty(hq.shape, dtype=torch.bfloat16, device=dev)
        b["k_rot"] = torch.empty(hk.shape, dtype=torch.bfloat16, device=dev)
        b["win_score"] = torch.empty((C, Hkv, L), dtype=torch.float32, device=dev)
        b["win_lse"] = torch.empty((C, Hq, w), dtype=torch.float32, device=dev)
        b["status"] = torch.zeros(1, dtype=torch.int32, device=dev)
        b["copy_stream"] = torch.cuda.Stream(device=dev)
        b["uploaded"] = [torch.cuda.Event() for _ in range(n_groups)]
        b["consumed"] = torch.cuda.Event()
    q, k, v = b["q"], b["k"], b["v"]
    main, copy = torch.cuda.current_stream(), b["copy_stream"]
    copy.wait_stream(main)                       # the previous call may still read q, k, v
    bounds = [(g * C) // n_groups for g in range(n_groups + 1)]
    for g in range(n_groups):
        c0, c1 = bounds[g], bounds[g + 1]
        if c1 == c0:
            continue
        with torch.cuda.stream(copy):
            q[c0:c1].copy_(hq[c0:c1], non_blocking=True)
            k[c0:c1].copy_(hk[c0:c1], non_blocking=True)
            v[c0:c1].copy_(hv[c0:c1], non_blocking=True)
            b["uploaded"][g].record(copy)
        main.wait_event(b["uploaded"][g])
        pre = chunk_prefill_attn(q[c0:c1], k[c0:c1], v[c0:c1], w=w, rope_theta=rope_theta, softmax_scale=softmax_scale,
                                 out=b["o"][c0:c1], k_rot=b["k_rot"][c0:c1], win_score=b["win_score"][c0:c1],
                                 win_lse=b["win_lse"][c0:c1], status=b["status"], workspace=b.get("ws_prefill"))
        b["ws_prefill"] = pre["workspace"]
    score, kept = score_select_chunks(b["win_lse"], m, True, score_out=b.get("chunk_score"), kept_out=b.get("kept"))
    idx = select_tokens(b["win_score"], kept, L - w, k_keep, out=b.get("idx"))
    kc, vc, pos = gather_kv(b["k_rot"], v, kept, idx, k_out=b.get("kc"), v_out=b.get("vc"), pos_out=b.get("pos"))
    pa = parallel_attn(q[0:1, L - w:], kc.unsqueeze(0), vc.unsqueeze(0), b["k_rot"][0:1, L - w:], v[0:1, L - w:],
                       q_pos0=L - w, rope_theta=rope_theta, softmax_scale=softmax_scale, out=b.get("fg"),
                       status=b["status"], workspace=b.get("ws_par"))
    b.update(chunk_score=score, kept=kept, idx=idx, kc=kc, vc=vc, pos=pos, fg=pa["out"], ws_par=pa["workspace"])
    return {"o": b["o"], "k_rot": b["k_rot"], "win_score": b["win_score"], "win_lse": b["win_lse"], "chunk_score": score,
            "kept": kept, "idx": idx, "kc": kc, "vc": vc, "pos": pos, "fg": pa["out"], "status": b["status"]}
