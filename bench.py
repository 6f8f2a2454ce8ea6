#!/usr/bin/env python
"""Benchmark of the ParallelComp attention hot path on B200.

One step = one pass of the whole path (chunk prefill attention with fused window scores,
chunk ranking, token ranking, KV gather, parallel attention over the compressed cache)
over one 128K batch of seeded synthetic input.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1] [--impl reference]

N > 1 runs N independent replicas (the path has no exchange step): launch with
torch.distributed.run; rank 0 prints the line, value = tokens of all ranks / max time.
`--impl reference` times the CPU oracle (fp64 numpy) on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import re
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import pc_inputs  # noqa: E402

METRIC = "chunked_prefill_tokens_per_s_per_layer"
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def choose_bf16_peak(peaks: dict, clocks: dict | None, timed_region_s: float) -> tuple[float, str]:
    """The bf16 roofline denominator that fits this run: the burst cuBLAS figure unless the run's own clock
    record shows the power-managed regime of the sustained figure (a timed region of a second or more whose
    median SM clock sits more than 5 % below the maximum)."""
    sm, mx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    power_managed = bool(sm and mx and sm < 0.95 * mx)
    if timed_region_s >= 1.0 and power_managed:
        return peaks["bf16_tflops_sustained"], (f"{peaks['source']} cuBLAS bf16, sustained: timed region {timed_region_s:.2f} s at a "
                                                f"median SM clock of {sm:.0f} of {mx:.0f} MHz")
    why = f"timed region {timed_region_s:.2f} s" + (f", median SM clock {sm:.0f} of {mx:.0f} MHz" if sm and mx else ", no clock samples")
    return peaks["bf16_tflops"], f"{peaks['source']} cuBLAS bf16, burst: {why}"


def recorded_traffic(kernel_sources: list[str], profile: str, scale: float):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary `profile` (a line
    `dram_bytes_captured: N` and a line `kernel_source_sha256: H` over the listed source files).  Returns
    (bytes scaled to this launch, note), or (None, why) when the kernel sources changed since the capture."""
    import hashlib
    path = os.path.join(ROOT, "profiles", profile)
    try:
        text = open(path).read()
        captured = float(re.search(r"dram_bytes_captured:\s*([0-9.eE+]+)", text).group(1))
        want = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text).group(1)
    except Exception:
        return None, f"no machine-readable traffic record in profiles/{profile}"
    h = hashlib.sha256()
    for f in kernel_sources:
        with open(os.path.join(ROOT, "paper_2502_14317_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    if h.hexdigest() != want:
        return None, f"kernel sources changed since the capture in profiles/{profile}"
    return captured * scale, f"ncu dram__bytes_read+write of the capture in profiles/{profile} ({captured / 1e6:.2f} MB) x {scale:g}"


def prefill_flops(cfg) -> float:
    """Algorithmic FLOPs of the chunk-local attention: 4 d per visible (query, key) pair per q-head."""
    return 2.0 * cfg.d * cfg.L * (cfg.L + 1) * cfg.Hq * cfg.C


def workload_description(cfg) -> dict:
    return {"workload": f"{cfg.name}: C={cfg.C} chunks x L={cfg.L} (ctx {cfg.ctx} + window w={cfg.w}), Hq={cfg.Hq}, "
                        f"Hkv={cfg.Hkv}, d={cfg.d}, rope_theta={cfg.rope_theta:g}, keep m={cfg.m} chunks x k={cfg.k} "
                        f"tokens per kv-head",
            "tokens_per_step": cfg.C * cfg.L, "l2": "inputs (1.6 GB) larger than L2, no flush needed",
            "parallelism": "single GPU (replicas only for N > 1)"}


# --------------------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(cfg, threads_hint=None):
    """Time the oracle, as it stands, on a bounded sample of the workload: one chunk and a
    quarter of the head groups, full chunk length, the whole path.  Returns (tokens/s equivalent,
    seconds, description)."""
    from oracle import parallelcomp_oracle as orc
    hkv_s = max(1, cfg.Hkv // 4)
    sub = dataclasses.replace(cfg, C=1, Hq=hkv_s * cfg.G, Hkv=hkv_s, m=1, n_planted_chunks=1, planted_chunks=())
    inp = pc_inputs.make_prefill_inputs(sub)
    t0 = time.perf_counter()
    orc.hot_path(inp["q"], inp["k"], inp["v"], w=sub.w, theta=sub.rope_theta, m=1, k=min(sub.k, sub.ctx))
    dt = time.perf_counter() - t0
    frac = (1.0 / cfg.C) * (hkv_s / cfg.Hkv)
    tokens_equiv = cfg.C * cfg.L * frac
    desc = (f"whole path on 1 of {cfg.C} chunks x {hkv_s} of {cfg.Hkv} kv-head groups at full L={cfg.L} "
            f"({frac:.4g} of the step); tokens/s = {tokens_equiv:.0f} token-equivalents / {dt:.1f} s")
    return tokens_equiv / dt, dt, desc


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return len(os.sched_getaffinity(0))


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, secs, desc = [], [], ""
    for _ in range(args.warmup_ref):
        oracle_sample(cfg)
    for _ in range(args.steps_ref):
        v, s, desc = oracle_sample(cfg)
        vals.append(v)
        secs.append(s)
    value = statistics.mean(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps_ref, "warmup": args.warmup_ref, "ms_per_step": 1e3 * statistics.mean(secs),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_description(cfg),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0,
            "note": "steps and warmup are capped at 3 and 1 for this arm (one oracle sample takes about ten seconds); "
                    "the GPU arm runs the step counts it was given"}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid = uuid
        self.proc = None
        self.tmp = None

    def start(self):
        try:
            self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", self.uuid], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        rows = [r.strip().split(",") for r in self.tmp.read().strip().splitlines() if r.strip()]
        self.tmp.close()
        os.unlink(self.tmp.name)
        sm, reasons, mx, pw = [], set(), None, []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                r = [x.strip() for x in r]
                sm.append(float(r[0]))
                mx = float(r[1])
                pw.append(float(r[2]))
                for name, flag in zip(names, r[4:8]):
                    if flag.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        if sm:
            out.update({"sm_mhz": statistics.median(sm), "sm_max_mhz": mx, "reasons": sorted(reasons),
                        "samples": len(sm), "power_w_max": max(pw) if pw else None})
        return out


# --------------------------------------------------------------------------------------- replicas
def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of per-rank timings over all ranks (identity for a single process)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def replica_throughput(units_per_rank: float, world: int, max_ms_per_step: float) -> float:
    """Whole-job throughput of `world` independent replicas: all units / slowest rank's time."""
    return world * units_per_rank / (max_ms_per_step * 1e-3)


def worker_environments(n: int, port: int, base_env=None) -> list:
    """Environments of the n replica processes of one node (one process per GPU, rendezvous on 127.0.0.1)."""
    envs = []
    for r in range(n):
        e = dict(os.environ if base_env is None else base_env)
        e.update({"RANK": str(r), "LOCAL_RANK": str(r), "WORLD_SIZE": str(n), "LOCAL_WORLD_SIZE": str(n),
                  "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
        envs.append(e)
    return envs


def free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_workers(cmd: list, n: int, port=None) -> int:
    """Start `cmd` n times as ranks 0..n-1 (rank 0 inherits stdout, the others' stdout is dropped: rank 0 prints the
    line), wait for all of them, return the largest exit code."""
    port = free_port() if port is None else port
    procs = []
    for r, env in enumerate(worker_environments(n, port)):
        procs.append(subprocess.Popen(cmd, env=env, stdout=None if r == 0 else subprocess.DEVNULL))
    return max(abs(p.wait()) for p in procs)


# --------------------------------------------------------------------------------------- GPU leg
def run_gpu(args, cfg):
    import torch
    import paper_2502_14317_b200 as pc

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    pc.load_library()
    peaks = load_peaks()

    # ---- inputs: generated once on the host (same generator the parity tests use), pinned
    inp = pc_inputs.make_prefill_inputs(cfg, seed=cfg.seed + rank)

    def pinned(bits):
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).pin_memory()

    hq, hk, hv = pinned(inp["q"]), pinned(inp["k"]), pinned(inp["v"])
    q, k, v = (t.to(dev, non_blocking=True) for t in (hq, hk, hv))
    torch.cuda.synchronize()
    buffers: dict = {}
    L, w = cfg.L, cfg.w

    def step(events=None):
        """The five C-ABI calls chained on the current stream (plus the stand-in chunk score)."""
        pre = pc.chunk_prefill_attn(q, k, v, w=w, rope_theta=cfg.rope_theta, out=buffers.get("o"),
                                    k_rot=buffers.get("k_rot"), win_score=buffers.get("win_score"),
                                    win_lse=buffers.get("win_lse"), status=buffers.get("status"),
                                    workspace=buffers.get("ws_prefill"))
        if events: events[1].record()
        score, kept = pc.score_select_chunks(pre["win_lse"], cfg.m, True, score_out=buffers.get("chunk_score"),
                                             kept_out=buffers.get("kept"))
        idx = pc.select_tokens(pre["win_score"], kept, L - w, cfg.k, out=buffers.get("idx"))
        if events: events[2].record()
        kc, vc, pos = pc.gather_kv(pre["k_rot"], v, kept, idx, k_out=buffers.get("kc"), v_out=buffers.get("vc"),
                                   pos_out=buffers.get("pos"))
        if events: events[3].record()
        pa = pc.parallel_attn(q[0:1, L - w:], kc.unsqueeze(0), vc.unsqueeze(0), pre["k_rot"][0:1, L - w:],
                              v[0:1, L - w:], q_pos0=L - w, rope_theta=cfg.rope_theta, out=buffers.get("fg"),
                              status=pre["status"], workspace=buffers.get("ws_par"))
        buffers.update(o=pre["o"], k_rot=pre["k_rot"], win_score=pre["win_score"], win_lse=pre["win_lse"],
                       status=pre["status"], ws_prefill=pre["workspace"], chunk_score=score, kept=kept, idx=idx,
                       kc=kc, vc=vc, pos=pos, fg=pa["out"], ws_par=pa["workspace"])
        return pa["out"]

    # kernels of one step (counted by the library, see pc_launch_count): cos/sin table, rotation of keys and of
    # queries, chunk attention, stand-in score + chunk top-m, token top-k, gather, window cos/sin table, parallel
    # attention, merge of its key splits

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    assert int(buffers["status"].item()) == 0, "a device-side wait ran out during warm-up"

    props = torch.cuda.get_device_properties(dev)
    sampler = ClockSampler("GPU-" + str(props.uuid)) if rank == 0 else None
    if sampler: sampler.start()

    # ---- timed region: K steps, inputs resident in HBM
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    launches_before = pc.launch_count()
    t_start.record()
    for s in range(args.steps):
        ev[s][0].record()
        step(ev[s])
        ev[s][4].record()
    t_end.record()
    barrier()
    total_ms = t_start.elapsed_time(t_end)
    launches_timed = pc.launch_count() - launches_before
    clocks = sampler.stop() if sampler else None
    assert int(buffers["status"].item()) == 0, "a device-side wait ran out"

    stage_ms = {name: statistics.mean(ev[s][a].elapsed_time(ev[s][b]) for s in range(args.steps))
                for name, a, b in (("prefill_attn", 0, 1), ("score_select", 1, 2), ("gather", 2, 3), ("parallel_attn", 3, 4))}
    prefill_ms_per_step = [ev[s][0].elapsed_time(ev[s][1]) for s in range(args.steps)]

    # ---- launch floor of the ranking stage: two launches that do (next to) nothing, timed like the stage
    tiny_lse = torch.zeros((1, 1, 1), dtype=torch.float32, device=dev)
    tiny_buf = {}

    def two_tiny_launches():
        tiny_buf["s"], tiny_buf["k"] = pc.score_select_chunks(tiny_lse, 1, True, score_out=tiny_buf.get("s"), kept_out=tiny_buf.get("k"))
        tiny_buf["s"], tiny_buf["k"] = pc.score_select_chunks(tiny_lse, 1, True, score_out=tiny_buf.get("s"), kept_out=tiny_buf.get("k"))
    empty_pair_ms = _time_us(torch, two_tiny_launches, warm=3, reps=50) / 1e3

    # ---- end to end through the public API with host buffers: H2D of Q,K,V and D2H of the result every step
    e2e_steps = max(1, min(args.steps, 5))
    h_out = torch.empty((1, w, cfg.Hq, cfg.d), dtype=torch.bfloat16).pin_memory()

    e2e_buffers: dict = {}

    def e2e_step():
        # public API for host inputs: uploads the chunks in groups on a copy stream while the attention of the
        # previous group runs; every byte of Q, K, V crosses PCIe inside the timed region, and the result comes back
        res = pc.hot_path_from_host(hq, hk, hv, w=w, rope_theta=cfg.rope_theta, m=cfg.m, k_keep=cfg.k,
                                    n_groups=min(16, cfg.C), buffers=e2e_buffers)
        h_out.copy_(res["fg"], non_blocking=True)

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps

    # ---- max over ranks
    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dist, dev)
    ms_per_step = total_ms / args.steps
    tokens = cfg.C * cfg.L
    value = replica_throughput(tokens, world, ms_per_step)

    if rank == 0:
        # DRAM bytes per launch of the dominant kernel: read from the committed ncu summary (a 2-chunk launch
        # of the same shape, scaled by the chunk count); null once the kernel sources differ from the captured ones
        pair_path = cfg.d == 128 and cfg.G % 2 == 0
        traffic, traffic_note = args.traffic_bytes, "command line"
        if traffic is None:
            if pair_path and cfg.L == 8192 and cfg.Hq == 32 and cfg.Hkv == 8:
                traffic, traffic_note = recorded_traffic(["pc_prefill2.cu", "pc_sm100.cuh"],
                                                         "prefill_pair_kernel_cfg1_C2_ncu_full.md", cfg.C / 2.0)
            else:
                traffic_note = "no ncu capture of this shape"
        flops = prefill_flops(cfg)
        ach_tflops = flops / (stage_ms["prefill_attn"] * 1e-3) / 1e12
        peak_tflops, peak_note = choose_bf16_peak(peaks, clocks, total_ms * 1e-3)
        sm_count = props.multi_processor_count
        sm_mhz = (clocks or {}).get("sm_mhz")
        gather_bytes = 2.0 * (2 * cfg.Hkv * cfg.m * cfg.k * cfg.d * 2)
        sel_bytes = 4.0 * cfg.m * cfg.Hkv * (cfg.ctx + cfg.k)
        par_flops = 4.0 * cfg.d * (cfg.m * cfg.k + (w + 1) / 2) * w * cfg.Hq
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_description(cfg),
            "clocks": clocks,
            "e2e": {"value": replica_throughput(tokens, world, e2e_ms), "unit": UNIT,
                    "h2d_bytes_per_step": int(hq.numel() + hk.numel() + hv.numel()) * 2,
                    "d2h_bytes_per_step": int(h_out.numel()) * 2, "ms_per_step": e2e_ms, "steps": e2e_steps},
            "gpu_launches": launches_timed,
            "roofline": {"bound": "tensor", "kernel": ("prefill_pair_kernel" if pair_path else "prefill_attn_kernel") +
                                   " (+ RoPE table and key pre-pass inside the same call)",
                         "achieved": ach_tflops, "peak": peak_tflops, "unit": "TFLOP/s",
                         "frac": ach_tflops / peak_tflops,
                         "frac_of_burst_peak": ach_tflops / peaks["bf16_tflops"],
                         "frac_of_sustained_peak": ach_tflops / peaks["bf16_tflops_sustained"],
                         "frac_of_nominal_2250": ach_tflops / 2250.0,
                         "peak_source": peak_note,
                         "flop_per_clk_per_sm": (ach_tflops * 1e12 / (sm_mhz * 1e6 * sm_count)) if sm_mhz else None,
                         "algorithmic_flops_per_launch": flops, "ms_per_launch": stage_ms["prefill_attn"],
                         "ms_per_launch_fastest": min(prefill_ms_per_step),
                         "tflops_fastest_launch": flops / (min(prefill_ms_per_step) * 1e-3) / 1e12,
                         "ms_per_launch_by_step": [round(x, 3) for x in prefill_ms_per_step],
                         "power_note": "back-to-back launches run into the board power cap after roughly 50 ms (sw_power_cap): the "
                                       "launch time then rises by about a tenth; ms_per_launch is the mean over the timed steps, "
                                       "ms_per_launch_fastest the launch least affected",
                         "traffic": traffic, "traffic_note": traffic_note},
            "stages": {
                "prefill_attn": {"ms": stage_ms["prefill_attn"], "tflops": ach_tflops},
                "score_select": {"ms": stage_ms["score_select"], "algorithmic_bytes": sel_bytes,
                                 "gbs": sel_bytes / (stage_ms["score_select"] * 1e-3) / 1e9,
                                 "launches": 2, "launch_floor_ms": empty_pair_ms,
                                 "note": "two launches (stand-in score + chunk top-m; token top-k), latency-bound at this size; "
                                         "launch_floor_ms = two empty kernels timed the same way"},
                "gather": {"ms": stage_ms["gather"], "algorithmic_bytes": gather_bytes,
                           "gbs": gather_bytes / (stage_ms["gather"] * 1e-3) / 1e9,
                           "frac_of_measured_hbm": gather_bytes / (stage_ms["gather"] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
                "parallel_attn": {"ms": stage_ms["parallel_attn"],
                                  "tflops": par_flops / (stage_ms["parallel_attn"] * 1e-3) / 1e12},
            },
        }
        if world == 1 and not args.no_extra:
            line["extra"] = extra_measurements(pc, torch, dev, peaks)
            line["extra"]["streamed_hot_path"] = streamed_measurement(pc, torch, cfg, q, k, v, buffers)
        if not args.no_cpu_baseline and world == 1:
            v_cpu, s_cpu, desc = oracle_sample(cfg)
            line["cpu_baseline"] = {"value": v_cpu, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                    "sample": desc}
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def _time_us(torch, fn, warm=3, reps=20):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return 1e3 * e0.elapsed_time(e1) / reps


def _tensor_bytes(torch, obj) -> int:
    if isinstance(obj, torch.Tensor):
        return obj.numel() * obj.element_size()
    if isinstance(obj, dict):
        return sum(_tensor_bytes(torch, x) for x in obj.values())
    return 0


def streamed_measurement(pc, torch, cfg, q, k, v, step_buffers, batch=4) -> dict:
    """The same workload with the chunks taken `batch` at a time through the online chunk queue
    (outside the timed region): time of one pass and the device memory held beyond the inputs."""
    sb: dict = {}

    def run():
        pc.hot_path_streaming(q, k, v, w=cfg.w, rope_theta=cfg.rope_theta, m=cfg.m, k_keep=cfg.k, batch=batch, buffers=sb)
    us = _time_us(torch, run, warm=2, reps=5)
    tokens = cfg.C * cfg.L
    return {"batch_chunks": batch, "ms": us / 1e3, "tokens_per_s": tokens / (us * 1e-6),
            "intermediate_bytes": _tensor_bytes(torch, sb), "intermediate_bytes_all_chunks_at_once": _tensor_bytes(torch, step_buffers),
            "note": "pc_chunk_prefill_attn + pc_select_tokens on every chunk + pc_queue_update/gather per batch, "
                    "pc_queue_emit + pc_parallel_attn at the end; same results as the timed step"}


def _extra_prefill(pc, torch, dev, peaks, g, out):
    """pc_chunk_prefill_attn at the two other full-size shapes (one call each, random device data)."""
    for name in ("cfg2", "cfg3"):
        cfg = pc_inputs.get_config(name)
        q = torch.randn((cfg.C, cfg.L, cfg.Hq, cfg.d), device=dev, generator=g).bfloat16()
        k = torch.randn((cfg.C, cfg.L, cfg.Hkv, cfg.d), device=dev, generator=g).bfloat16()
        v = torch.randn((cfg.C, cfg.L, cfg.Hkv, cfg.d), device=dev, generator=g).bfloat16()
        buf = {}

        def run():
            r = pc.chunk_prefill_attn(q, k, v, w=cfg.w, rope_theta=cfg.rope_theta, out=buf.get("o"), k_rot=buf.get("k_rot"),
                                      win_score=buf.get("win_score"), win_lse=buf.get("win_lse"), status=buf.get("status"),
                                      workspace=buf.get("workspace"))
            buf.update(r)
        us = _time_us(torch, run, warm=3, reps=5)
        assert int(buf["status"].item()) == 0
        tf = prefill_flops(cfg) / us / 1e6
        out["prefill_" + name] = {"us": us, "tflops": tf, "frac_of_measured_bf16_burst": tf / peaks["bf16_tflops"],
                                  "kernel": "prefill_pair_kernel" if (cfg.d == 128 and cfg.G % 2 == 0) else "prefill_attn_kernel",
                                  "workload": workload_description(cfg)["workload"]}
        del q, k, v, buf
        torch.cuda.empty_cache()


def extra_measurements(pc, torch, dev, peaks, only=None, select_chunks=8192, parallel_batch=64) -> dict:
    """Single-call timings of the stages whose full-size workloads are not part of the cfg1 step
    (outside the timed region; random device data, parity is covered by the tests):
    parallel attention over a batch of compressed caches (cfg4), token top-k on enough rows to be
    bandwidth-bound, and the gather at the cfg2 size."""
    out = {}
    g = torch.Generator(device=dev).manual_seed(4)
    if only in (None, "prefill"):
        _extra_prefill(pc, torch, dev, peaks, g, out)
    if only in (None, "parallel"):
        _extra_parallel(pc, torch, dev, peaks, g, out, parallel_batch)
    if only in (None, "select"):
        _extra_select(pc, torch, dev, peaks, g, out, select_chunks)
    if only in (None, "gather"):
        _extra_gather(pc, torch, dev, peaks, g, out)
    if only in (None, "rope"):
        _extra_rope(pc, torch, dev, peaks, g, out)
    return out


def _extra_rope(pc, torch, dev, peaks, g, out):
    # ---- the RoPE pre-pass alone (pc_rope_position_reuse: table kernel + rotation pass), query and key tensors of cfg1
    for name, shape in (("rope_queries_cfg1", (16, 8192, 32, 128)), ("rope_keys_cfg1", (16, 8192, 8, 128))):
        x = torch.randn(shape, device=dev, generator=g).bfloat16()
        y = torch.empty_like(x)
        lib = pc.load_library()
        ws = torch.empty(int(lib.pc_rope_position_reuse_workspace_bytes(shape[1], shape[3])), dtype=torch.uint8, device=dev)
        us = _time_us(torch, lambda: pc.rope_position_reuse(x, rope_theta=5e5, out=y, workspace=ws), reps=10)
        nbytes = 2.0 * x.numel() * 2
        out[name] = {"us": us, "algorithmic_bytes": nbytes, "gbs": nbytes / us / 1e3,
                     "frac_of_measured_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"]}
        del x, y, ws


def _extra_parallel(pc, torch, dev, peaks, g, out, B=64):
    # ---- cfg4: B=64 sequences x (8 kept chunks x 2048 keys), 64 window queries (a smaller B for an ncu capture)
    w, Hq, Hkv, d, Nk = 64, 32, 8, 128, 16384
    qw = torch.randn((B, w, Hq, d), device=dev, generator=g).bfloat16()
    kc = torch.randn((B, Hkv, Nk, d), device=dev, generator=g).bfloat16()
    vc = torch.randn((B, Hkv, Nk, d), device=dev, generator=g).bfloat16()
    kw = torch.randn((B, w, Hkv, d), device=dev, generator=g).bfloat16()
    vw = torch.randn((B, w, Hkv, d), device=dev, generator=g).bfloat16()
    buf = {}

    def run_par():
        r = pc.parallel_attn(qw, kc, vc, kw, vw, q_pos0=8128, rope_theta=5e5, out=buf.get("out"), status=buf.get("status"),
                             workspace=buf.get("workspace"))
        buf.update(r)
    us = _time_us(torch, run_par, reps=10)
    flops = 4.0 * d * (Nk + (w + 1) / 2) * w * Hq * B
    kv_bytes = 2.0 * B * Hkv * Nk * d * 2
    out["parallel_attn_cfg4" if B == 64 else "parallel_attn_cfg4_B%d" % B] = {"us": us, "tflops": flops / us / 1e6, "kv_gbs": kv_bytes / us / 1e3,
                                 "frac_of_measured_bf16_burst": flops / us / 1e6 / peaks["bf16_tflops"],
                                 "frac_of_measured_hbm": kv_bytes / us / 1e3 / peaks["hbm_gbs"],
                                 "flops": flops, "kv_bytes": kv_bytes, "l2": "%.1f GB of K/V per call, larger than L2" % (kv_bytes / 1e9),
                                 "note": "runs unsplit on CTA pairs when the batch fills them (else key splits + merge)"}
    # ---- decoding step over the same caches: one query token per sequence (w = 1), HBM-bound
    q1 = torch.randn((B, 1, Hq, d), device=dev, generator=g).bfloat16()
    k1 = torch.randn((B, 1, Hkv, d), device=dev, generator=g).bfloat16()
    v1 = torch.randn((B, 1, Hkv, d), device=dev, generator=g).bfloat16()
    buf1 = {}

    def run_dec():
        r = pc.parallel_attn(q1, kc, vc, k1, v1, q_pos0=8191, rope_theta=5e5, out=buf1.get("out"), status=buf1.get("status"),
                             workspace=buf1.get("workspace"))
        buf1.update(r)
    us = _time_us(torch, run_dec, reps=10)
    # ---- the same step as a generation loop runs it: caches stored with spare room, the step's key / value appended
    cap = Nk + 64
    kcap = torch.empty((B, Hkv, cap, d), device=dev, dtype=torch.bfloat16)
    vcap = torch.empty((B, Hkv, cap, d), device=dev, dtype=torch.bfloat16)
    kcap[:, :, :Nk].copy_(kc)
    vcap[:, :, :Nk].copy_(vc)
    buf2 = {}

    def run_gen():
        r = pc.parallel_attn_append(q1, kcap, vcap, Nk, k1, v1, q_pos0=8191, rope_theta=5e5, out=buf2.get("out"),
                                    status=buf2.get("status"), workspace=buf2.get("workspace"))
        buf2.update(r)
    us_gen = _time_us(torch, run_gen, reps=10)
    del kcap, vcap
    out["decode_step_with_append"] = {"us": us_gen, "kv_gbs": kv_bytes / us_gen / 1e3,
                                      "frac_of_measured_hbm": kv_bytes / us_gen / 1e3 / peaks["hbm_gbs"],
                                      "note": "pc_parallel_attn_append, w = 1, B = %d, %d valid of %d entries" % (B, Nk, cap)}
    out["decode_step_cfg4_caches"] = {"us": us, "kv_gbs": kv_bytes / us / 1e3,
                                      "frac_of_measured_hbm": kv_bytes / us / 1e3 / peaks["hbm_gbs"],
                                      "kv_bytes": kv_bytes, "note": "pc_parallel_attn with w = 1, B = %d, Nk = %d" % (B, Nk)}


def _extra_select(pc, torch, dev, peaks, g, out, n_chunks):
    # ---- token top-k, cfg1 row shape (8128 candidates -> 2048) on 8 rows per chunk (65536 rows = 2.1 GB of scores)
    C, Hk, L, n_cand, k = n_chunks, 8, 8192, 8128, 2048
    score = torch.rand((C, Hk, L), device=dev, generator=g)
    kept = torch.arange(C, device=dev, dtype=torch.int32)
    idx = torch.empty((C, Hk, k), device=dev, dtype=torch.int32)
    us = _time_us(torch, lambda: pc.select_tokens(score, kept, n_cand, k, out=idx), reps=5)
    sel_bytes = 4.0 * C * Hk * (n_cand + k)
    out["select_tokens_%d_rows" % (C * Hk)] = {"us": us, "algorithmic_bytes": sel_bytes, "gbs": sel_bytes / us / 1e3,
                                       "frac_of_measured_hbm": sel_bytes / us / 1e3 / peaks["hbm_gbs"]}


def _extra_gather(pc, torch, dev, peaks, g, out):
    # ---- gather at the cfg2 size: 12 kept chunks x 1024 tokens x 32 heads (201 MB read + 201 MB written)
    d = 128
    C2, L2, H2, m2, k2 = 32, 4096, 32, 12, 1024
    ksrc = torch.randn((C2, L2, H2, d), device=dev, generator=g).bfloat16()
    vsrc = torch.randn((C2, L2, H2, d), device=dev, generator=g).bfloat16()
    kept2 = torch.arange(0, 2 * m2, 2, device=dev, dtype=torch.int32)
    idx2 = torch.sort(torch.rand((m2, H2, L2 - 64), device=dev, generator=g).argsort(-1)[..., :k2], -1).values.to(torch.int32)
    gb = {}

    def run_gather():
        gb["k"], gb["v"], gb["p"] = pc.gather_kv(ksrc, vsrc, kept2, idx2, k_out=gb.get("k"), v_out=gb.get("v"), pos_out=gb.get("p"))
    us = _time_us(torch, run_gather, reps=20)
    g_bytes = 2.0 * (2 * H2 * m2 * k2 * d * 2)
    out["gather_cfg2"] = {"us": us, "algorithmic_bytes": g_bytes, "gbs": g_bytes / us / 1e3,
                          "frac_of_measured_hbm": g_bytes / us / 1e3 / peaks["hbm_gbs"],
                          "l2": "sources 2 x 1.07 GB, larger than L2"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg1", choices=["cfg0", "cfg1", "cfg2", "cfg3"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the single-call timings of cfg4 / scaled select / cfg2 gather")
    ap.add_argument("--parallel-batch", type=int, default=64,
                    help="sequences of the parallel-attention measurement (smaller for an ncu capture)")
    ap.add_argument("--extra-only", default=None, choices=["parallel", "select", "gather", "prefill", "rope"],
                    help="run only that single-call measurement and print it (no step loop; e.g. for an ncu capture)")
    ap.add_argument("--select-chunks", type=int, default=8192,
                    help="rows / 8 of the scaled token top-k measurement (smaller for an ncu capture)")
    ap.add_argument("--chunks", type=int, default=None,
                    help="override the number of chunks (smaller case of the same workload, e.g. for an ncu capture)")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="dram bytes per launch of the dominant kernel from an ncu capture (see profiles/)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = pc_inputs.get_config(args.workload)
    if args.chunks is not None:
        cfg = dataclasses.replace(cfg, name=f"{cfg.name}[C={args.chunks}]", C=args.chunks, m=min(cfg.m, args.chunks),
                                  n_planted_chunks=min(cfg.n_planted_chunks, args.chunks))
    if args.extra_only:
        import torch
        import paper_2502_14317_b200 as pc
        dev = torch.device("cuda:0")
        torch.cuda.set_device(dev)
        print(json.dumps({"extra": extra_measurements(pc, torch, dev, load_peaks(), only=args.extra_only,
                                                      select_chunks=args.select_chunks, parallel_batch=args.parallel_batch)}))
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: become the launcher of --gpus replicas, one process per GPU
        sys.exit(spawn_workers([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus))
    if args.impl == "reference":
        # the oracle takes ~20 s per sample: bound the run to a few minutes whatever K and W say
        args.steps_ref = max(1, min(args.steps, 3))
        args.warmup_ref = max(0, min(args.warmup, 1))
        run_reference(args, cfg)
    else:
        run_gpu(args, cfg)


if __name__ == "__main__":
    main()
