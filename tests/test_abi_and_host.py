"""CPU-only checks of the boundary and host logic: the library loads and exports every symbol that
include/pc.h declares; host-side argument validation; bench.py's replica aggregation over gloo."""
import ctypes
import json
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_14317_b200 import build, binding
    build.build_library()
    return binding.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "pc.h")).read()
    return sorted(set(re.findall(r"PC_API\s+[\w\s\*]+?\b(pc_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert set(names) >= {"pc_chunk_prefill_attn", "pc_select_chunks", "pc_select_tokens", "pc_gather_kv",
                          "pc_parallel_attn", "pc_chunk_prefill_attn_workspace_bytes",
                          "pc_parallel_attn_workspace_bytes", "pc_chunk_score_from_lse", "pc_status_string",
                          "pc_version"}
    for n in names:
        assert hasattr(lib, n), f"{n} declared in pc.h but not exported by libpc.so"


def test_status_strings_and_version(lib):
    from paper_2502_14317_b200 import binding
    assert binding.version() >= 1000
    assert binding.status_string(0) == "ok"
    texts = {binding.status_string(c) for c in (-1, -2, -3, -4, -5)}
    assert len(texts) == 5 and "unknown status" not in texts
    assert binding.status_string(-99) == "unknown status"


def test_workspace_queries_are_host_only(lib):
    from paper_2502_14317_b200 import binding
    # cfg1: 256 B counter + fp64 cos/sin table L * d/2 * 16 B + its fp32 head and tail copies 2 * L * d/2 * 8 B
    # + the rotated queries C * L * Hq * d * 2 B
    tables = lambda L, d: 256 + L * (d // 2) * 16 + L * (d // 2) * 16
    assert binding.chunk_prefill_attn_workspace_bytes(16, 8192, 64, 32, 8, 128) == tables(8192, 128) + 16 * 8192 * 32 * 128 * 2
    assert binding.chunk_prefill_attn_workspace_bytes(4, 256, 16, 4, 2, 64) == tables(256, 64) + 4 * 256 * 4 * 64 * 2
    with_krot = binding.chunk_prefill_attn_workspace_bytes(16, 8192, 64, 32, 8, 128, k_rot_in_workspace=True)
    assert with_krot == tables(8192, 128) + 16 * 8192 * 32 * 128 * 2 + 16 * 8192 * 8 * 128 * 2
    # unsupported shapes give 0
    assert binding.chunk_prefill_attn_workspace_bytes(1, 256, 24, 4, 2, 64) > 0        # any window up to 128 tokens
    assert binding.chunk_prefill_attn_workspace_bytes(1, 256, 129, 4, 2, 64) == 0      # wider than a tile
    assert binding.chunk_prefill_attn_workspace_bytes(1, 64, 64, 4, 2, 64) == 0        # no context token left
    assert binding.chunk_prefill_attn_workspace_bytes(1, 256, 16, 4, 2, 96) == 0       # head size
    assert binding.chunk_prefill_attn_workspace_bytes(1, 256, 16, 4, 3, 64) == 0       # Hq % Hkv
    # a batch whose 256-row groups fill the CTA pairs: counter, the three cos/sin tables of the window and the rotated
    # window queries; no per-split partial results
    assert binding.parallel_attn_workspace_bytes(64, 64, 32, 8, 128, 16384) == 256 + 64 * 64 * 16 + 2 * 64 * 32 * 16 + 64 * 64 * 32 * 128 * 2
    # one sequence: keys split over the CTAs (16 splits of 8 tiles: one item per SM), fp32 partial outputs and
    # (max, sum) per split besides the tables and the rotated queries
    fixed = 256 + 64 * 64 * 16 + 2 * 64 * 32 * 16 + 1 * 64 * 32 * 128 * 2
    assert binding.parallel_attn_workspace_bytes(1, 64, 32, 8, 128, 16384) == fixed + 16 * 32 * 64 * (128 + 2) * 4
    # a decoding step (one query token per sequence): the four rows of a kv-head fill one block only, so both blocks of
    # a CTA take alternate key tiles and every one of the 2 key splits leaves two partial results per (sequence, q-head)
    fixed = 256 + 1 * 64 * 16 + 2 * 1 * 32 * 16 + 64 * 1 * 32 * 128 * 2
    assert binding.parallel_attn_workspace_bytes(64, 1, 32, 8, 128, 16384) == fixed + 4 * 64 * 32 * 1 * (128 + 2) * 4
    assert binding.parallel_attn_workspace_bytes(64, 64, 32, 8, 100, 16384) == 0


def test_host_side_argument_errors_need_no_gpu(lib):
    # null pointers / bad sizes are rejected before any CUDA call
    assert lib.pc_select_chunks(None, 4, 2, 1, None, None) == -1
    buf = (ctypes.c_float * 4)()
    out = (ctypes.c_int32 * 4)()
    p, o = ctypes.cast(buf, ctypes.c_void_p), ctypes.cast(out, ctypes.c_void_p)
    assert lib.pc_select_chunks(p, 4, 5, 1, o, None) == -1          # m > C
    assert lib.pc_select_chunks(p, 2000, 5, 1, o, None) == -2       # C > 1024
    assert lib.pc_select_tokens(p, o, 4, 2, 2, 256, 300, 64, o, None) == -1    # n_cand > L
    st = (ctypes.c_int64 * 3)(256 * 2 * 96, 2 * 96, 96)
    assert lib.pc_gather_kv(p, p, st, o, o, 2, 2, 64, 96, p, p, None, None) == -2   # head size
    assert lib.pc_gather_kv(p, p, None, o, o, 2, 2, 64, 64, p, p, None, None) == -1  # no strides
    assert lib.pc_parallel_attn(1, 24, 4, 2, 64, 128, p, 0, 1e4, 0.0, p, p, p, p, p, None, None, None, 0, None) == -2
    assert lib.pc_select_tokens_calibrated(p, o, 4, 2, 2, 256, 200, 64, -1, 0, 1.0, 1.0, 1.0, o, None) == -1   # n_s < 0
    assert lib.pc_queue_init(0, p, o, None) == -1                    # no slots
    assert lib.pc_queue_update(p, 4, -1, 1, 2, p, o, o, None) == -1  # negative chunk id
    assert lib.pc_queue_update(p, 1000, 0, 1, 100, p, o, o, None) == -2   # slots + batch > 1024
    assert lib.pc_queue_gather(p, p, st, o, o, 2, 2, 64, 96, p, p, o, None) == -2   # head size
    assert lib.pc_queue_emit(o, 2, 2, 64, 128, p, p, o, o, None, p, p, None, None) == -1    # no slot_order array


def test_binding_fails_loudly_without_library(tmp_path, monkeypatch):
    from paper_2502_14317_b200 import binding
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "lib_path", lambda: str(tmp_path / "missing.so"))
    with pytest.raises(binding.PcError, match="no fallback"):
        binding.load_library()


_WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=2)
rank = dist.get_rank()
total_ms, e2e_ms = bench.max_over_ranks([10.0 + 5.0 * rank, 40.0 - 3.0 * rank], dist)
value = bench.replica_throughput(131072, dist.get_world_size(), total_ms / 1)
if rank == 0:
    print(json.dumps({{"total_ms": total_ms, "e2e_ms": e2e_ms, "value": value}}))
dist.barrier()
dist.destroy_process_group()
"""


def test_replica_aggregation_world_size_2_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29577")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["total_ms"] == 15.0 and res["e2e_ms"] == 40.0           # slowest rank on each clock
    assert abs(res["value"] - 2 * 131072 / 15e-3) < 1e-6               # all ranks' tokens / slowest time


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_launcher_makes_one_environment_per_gpu():
    sys.path.insert(0, ROOT)
    import bench
    envs = bench.worker_environments(4, 29611, base_env={"KEEP": "1"})
    assert len(envs) == 4 and all(e["KEEP"] == "1" for e in envs)
    assert [e["RANK"] for e in envs] == ["0", "1", "2", "3"] == [e["LOCAL_RANK"] for e in envs]
    assert {e["WORLD_SIZE"] for e in envs} == {"4"} and {e["MASTER_ADDR"] for e in envs} == {"127.0.0.1"}
    assert {e["MASTER_PORT"] for e in envs} == {"29611"}


def test_bench_without_launcher_starts_its_own_ranks():
    # `bench.py --gpus 2` with no WORLD_SIZE in the environment must start two ranks itself; on the reference
    # arm rank 1 exits at once and rank 0 would time the oracle, so a tiny stand-in command is spawned instead
    sys.path.insert(0, ROOT)
    import bench
    code = "import os, sys; sys.exit(0 if os.environ['WORLD_SIZE'] == '2' and os.environ['RANK'] in '01' else 7)"
    assert bench.spawn_workers([sys.executable, "-c", code], 2) == 0
    assert bench.spawn_workers([sys.executable, "-c", "import os, sys; sys.exit(5 * int(os.environ['RANK']))"], 2) == 5


def _params(name):
    """Parameter names of the prototype of `name` in include/pc.h, in order."""
    text = open(os.path.join(ROOT, "include", "pc.h")).read()
    m = re.search(r"PC_API\s+[\w\s\*]+?\b" + name + r"\s*\(([^;]*?)\)\s*;", text, re.S)
    assert m, name
    out = []
    for piece in m.group(1).replace("\n", " ").split(","):
        piece = piece.strip()
        if piece in ("void", ""):
            continue
        out.append(re.sub(r"\[\d*\]$", "", piece).split()[-1].lstrip("*"))
    return out


def test_boundary_has_the_argument_lists_of_the_scope_table():
    """The five calls of the path: argument names and order as the scope table lists them.  Two documented
    additions: the optional full log-sum-exp output `lse` of the prefill call, and `Hkv` in the parallel-attention
    workspace query (the split plan depends on the number of kv-heads)."""
    assert _params("pc_chunk_prefill_attn_workspace_bytes") == ["desc"]
    assert _params("pc_chunk_prefill_attn") == ["desc", "q", "k", "v", "chunk_len", "o", "k_rot", "lse", "win_score",
                                                "win_lse", "status_word", "workspace", "workspace_bytes", "stream"]
    assert _params("pc_select_chunks") == ["chunk_score", "C", "m", "lower_is_better", "kept", "stream"]
    assert _params("pc_select_tokens") == ["win_score", "kept", "C", "m", "Hkv", "L", "n_cand", "k", "idx", "stream"]
    assert _params("pc_gather_kv") == ["k_src", "v_src", "kv_stride", "kept", "idx", "m", "Hkv", "k", "d", "k_out",
                                       "v_out", "pos_out", "stream"]
    assert _params("pc_parallel_attn_workspace_bytes") == ["B", "w", "Hq", "Hkv", "d", "Nk"]
    assert _params("pc_parallel_attn") == ["B", "w", "Hq", "Hkv", "d", "Nk", "q_win", "q_pos0", "rope_theta",
                                           "softmax_scale", "k_cache", "v_cache", "k_win", "v_win", "out", "lse_out",
                                           "status_word", "workspace", "workspace_bytes", "stream"]


def test_header_is_plain_c(tmp_path):
    """include/pc.h is the boundary for C callers: it must compile as C99 on its own, without warnings."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler here")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "use_pc.c"
    src.write_text('#include "pc.h"\nint main(void) { return (int)sizeof(pc_prefill_desc) == 0; }\n')
    r = subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only",
                        "-I", os.path.join(root, "include"), str(src)], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
