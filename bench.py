#!/usr/bin/env python
"""Benchmark of the KVSwap decode hot path (predictor + sparse decode attention) on B200.

A *step* is one decode step over all L layers of the workload through kvswap_decode_step: per
layer the predictor (low-rank scoring -> head sum -> group max -> top-k) and the sparse decode
attention (gather + split-K online-softmax attention + combine), the predictor one layer ahead of
the attention (what a model allows whose layer-l prediction is formed from the input of layer l-1).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 5] [--meta joint|per_head]
    python bench.py --impl reference ...      # the CPU oracle timed on the host cores

Prints ONE JSON line (rank 0).  `value` is decode steps/s with every input resident in HBM;
`e2e` is the same step driven through kvswap_decode_step_host with the step's queries in pinned
host memory and its outputs read back, both copies inside the timed region.  Beside them:
`roofline` (the attention call against the measured HBM peak, with the in-run read-only probe),
`roofline_score_select`, `secondary` (the same two figures on config 5 with per-head metadata and
on config 4), `growing_context` (a token appended per layer before every step), `reuse_buffer`
(hit rate and phase costs with the slow tier in pinned host memory, and the tiered step),
`prefill`, `cpu_baseline` (the C++/OpenMP twin of the oracle on one full layer).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2511_11907_b200 import workloads as W  # noqa: E402

METRIC = "decode_steps_per_sec"
UNIT = "steps/s"

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the split-K sparse-decode
# kernel from one ncu capture at the workload's full shapes on three layers (the traffic of a launch
# does not depend on the layer count).  None for workloads that were not captured, or whose kernel
# has changed since.  Key: (config, metadata layout, scope).
NCU_TRAFFIC = {(5, "joint", "kv_head"): 134451029 + 3957163, (5, "per_head", "kv_head"): 134451029 + 3957163}


def esz_of(dtype: int) -> int:
    return 4 if dtype == 0 else 2


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", type=int, default=5, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--meta", choices=["joint", "per_head"], default="joint")
    ap.add_argument("--scope", choices=["kv_head", "all_heads"], default="kv_head")
    ap.add_argument("--layers", type=int, default=None, help="override L (debugging only; reported)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the config-5-per-head and config-4 legs")
    ap.add_argument("--min-calls", type=int, default=None,
                    help="launches per per-call figure (default 2000; fewer only for runs under a profiler)")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def workload_name(wl, args):
    n = {W.F32: "fp32", W.BF16: "bf16", W.F16: "fp16"}
    return (f"config{wl.config}: L={wl.layers} B={wl.batch} N={wl.n_ctx} Hq/Hkv={wl.n_q_heads}/{wl.n_kv_heads} "
            f"d={wl.head_dim} r={wl.rank} G={wl.group_size} M={wl.top_k} kv={n[wl.kv_dtype]} meta={n[wl.meta_dtype]} "
            f"layout={args.meta} scope={args.scope}")


# --------------------------------------------------------------------------------------------
# Clock sampling during the timed region
# --------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            import torch
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            ident = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            ident = str(device_index)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50", "-i", ident],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t_begin: float, t_end: float):
        """Summary of the samples taken in [t_begin, t_end] (wall clock); if the region was too
        short to catch any, of all samples taken while the GPU ran the same step loop."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        rows = []
        for line in self.file:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                ts = time.mktime(time.strptime(parts[0].split(".")[0], "%Y/%m/%d %H:%M:%S")) + float("0." + parts[0].split(".")[1])
                rows.append((ts, float(parts[1]), float(parts[2]), parts[4:8]))
            except Exception:
                continue
        self.file.close()
        os.unlink(self.file.name)
        inside = [r for r in rows if t_begin - 0.05 <= r[0] <= t_end + 0.05]
        used, where = (inside, "timed region") if inside else (rows, "whole step loop (timed region shorter than one sample)")
        if not used:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in used for n, v in zip(names, r[3]) if v == "Active"})
        return {"sm_mhz": statistics.median(r[1] for r in used), "sm_max_mhz": max(r[2] for r in used),
                "reasons": reasons, "samples": len(used), "window": where}


# --------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and the --impl reference arm): the C++/OpenMP twin of the
# oracle (oracle/kvswap_oracle_omp.cpp; the numpy oracle it is checked against stays the parity
# authority) on one full layer of the workload -- all B sequences -- scaled to L layers.
# --------------------------------------------------------------------------------------------
def cpu_model():
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def oracle_layer_seconds(K, V, q, proj, meta, wl, scope_name):
    """Seconds the OpenMP twin needs for one layer (all sequences): score_select then attend."""
    from oracle import omp_twin as T
    t0 = time.perf_counter()
    idx, _ = T.score_select(q, proj, meta, wl.group_size, wl.top_k, scope_name)
    T.attend(q, K, V, idx, wl.group_size, scope_name)
    return time.perf_counter() - t0


def host_layer_inputs(wl, layer, meta_heads):
    """One full layer drawn on the host (numpy) + oracle metadata (not timed)."""
    from oracle import kvswap_oracle as O
    li = W.make_layer(wl.reduced(wl.name + "-layer", walk_steps=1), layer, meta_heads)
    meta = np.concatenate([O.project_keys(li.K[b:b + 1], li.proj, meta_heads, "f16" if wl.meta_dtype == W.F16 else "f32")
                           for b in range(wl.batch)])
    return li.K, li.V, li.q, li.proj, meta.astype(np.float32)


def oracle_baseline(times, wl, what):
    from oracle import omp_twin as T
    t_layer = statistics.mean(times)
    value = 1.0 / (t_layer * wl.layers)
    return {"value": value, "unit": UNIT, "cores": T.threads(), "kind": "oracle",
            "sample": f"{what}; {len(times)} timed passes of {t_layer:.2f} s each over one full layer "
                      f"({wl.batch} sequences x {wl.n_kv_heads} KV heads), scaled to L = {wl.layers} layers per step",
            "implementation": "oracle/kvswap_oracle_omp.cpp (C++/OpenMP twin of the numpy oracle, float64)",
            "host_cores_available": len(os.sched_getaffinity(0)), "cpu": cpu_model()}


def run_reference(args, wl):
    """The oracle's OpenMP twin, on the host cores, on one full layer of the same workload per step."""
    from oracle import omp_twin as T
    T.build()
    steps = args.steps if args.steps is not None else 5
    warmup = args.warmup if args.warmup is not None else 1
    meta_heads = 1 if args.meta == "joint" else wl.n_kv_heads
    K, V, q, proj, meta = host_layer_inputs(wl, 0, meta_heads)
    t_probe = oracle_layer_seconds(K, V, q, proj, meta, wl, args.scope)
    # keep the whole run within a few minutes whatever the driver asks for
    n_timed = int(max(1, min(steps, 120.0 // max(t_probe, 1e-3))))
    n_warm = int(max(0, min(warmup, 20.0 // max(t_probe, 1e-3))))
    for _ in range(n_warm):
        oracle_layer_seconds(K, V, q, proj, meta, wl, args.scope)
    times = [oracle_layer_seconds(K, V, q, proj, meta, wl, args.scope) for _ in range(n_timed)]
    base = oracle_baseline(times, wl, "each timed step = layer 0 of the workload drawn on the host")
    value = base["value"]
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(wl, args)},
        "keys_scored_per_sec": value * wl.batch * wl.n_ctx * wl.layers,
        "timed_passes": n_timed,
        "cpu_baseline": base,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def cpu_baseline(wl, dw, meta_heads, scope_name, rt):
    """The OpenMP twin on layer 0 of the resident workload (device tensors copied to the host, untimed)."""
    from oracle import omp_twin as T
    T.build()
    K, V = rt.to_host_f32(dw.K[0]), rt.to_host_f32(dw.V[0])
    q, meta = rt.to_host_f32(dw.q_walk[0, 0]), rt.to_host_f32(dw.meta[0])
    proj = dw.proj[0].cpu().numpy()
    times, spent = [], 0.0
    while spent < 10.0 and len(times) < 8:
        t = oracle_layer_seconds(K, V, q, proj, meta, wl, scope_name)
        times.append(t)
        spent += t
    return oracle_baseline(times[1:] or times, wl, "layer 0 of the resident workload")


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
MIN_CALLS = 2000          # launches of a call timed per figure, whatever --steps says


def graph_call_us(torch, fns, min_calls=None):
    """Average duration (us) of the calls `fns` (a list: one per layer, each reading another layer's
    buffers, so nothing is served from L2) issued back to back on one stream.  The calls are
    captured once into a CUDA graph and the graph is replayed, so the host is not in the loop;
    CUDA events bracket the replays.  Returns (us per call, calls timed)."""
    min_calls = MIN_CALLS if min_calls is None else min(min_calls, MIN_CALLS)
    side = torch.cuda.Stream()
    reps = max(1, -(-min(72, min_calls) // len(fns)))       # calls per graph: at least 72
    with torch.cuda.stream(side):
        for f in fns:
            f()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(reps):
                for f in fns:
                    f()
        per_graph = reps * len(fns)
        replays = max(3, -(-min_calls // per_graph))
        graph.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(replays):
            graph.replay()
        b.record()
        torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / (replays * per_graph), replays * per_graph


def host_call_us(torch, fns, min_calls=None):
    """The same calls issued from Python call by call (the host in the loop)."""
    min_calls = MIN_CALLS if min_calls is None else min(min_calls, MIN_CALLS)
    for f in fns:
        f()
    reps = max(1, -(-min_calls // len(fns)))
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(reps):
        for f in fns:
            f()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e3 / (reps * len(fns))


def workload_bytes(wl, meta_heads, S):
    esz = {W.F32: 4, W.BF16: 2, W.F16: 2}
    Mp = min(wl.top_k, wl.n_groups)
    decode = 2 * wl.batch * wl.n_kv_heads * Mp * wl.group_size * wl.head_dim * esz[wl.kv_dtype] + wl.batch * S * wl.top_k * 4
    select = (wl.batch * meta_heads * wl.n_ctx * wl.rank * esz[wl.meta_dtype] + 2 * wl.batch * S * wl.n_groups * 4
              + wl.batch * S * wl.top_k * 4)
    return decode, select


def call_rooflines(torch, kv, wl, dw, meta, shape, idx, nsel, out, ws, layers_used, peak, peak_kind, traffic):
    """`roofline` and `roofline_score_select` objects of one workload: each C-ABI call on its own, back
    to back over `layers_used` layers' buffers, in the default mode (every call waits for the kernel
    before it) and with KVSWAP_INPUTS_SETTLED (consecutive launches overlap prologue and tail)."""
    S = shape.n_scopes
    meta_heads = shape.meta_heads
    decode_bytes, select_bytes = workload_bytes(wl, meta_heads, S)
    q0 = dw.q_walk[0]
    Ls = list(range(layers_used))
    shape_settled = shape.with_flags(kv.KVSWAP_INPUTS_SETTLED)
    sel = lambda sh: [(lambda l=l: kv.kvswap_score_select(sh, q0[l], dw.proj[l], meta[l], idx[l], nsel[l], None, ws)) for l in Ls]
    dec = lambda sh: [(lambda l=l: kv.kvswap_sparse_decode(sh, q0[l], dw.K[l], dw.V[l], idx[l], nsel[l], out[l], None, ws)) for l in Ls]
    sel_wait_us, sel_calls = graph_call_us(torch, sel(shape))
    sel_settled_us, _ = graph_call_us(torch, sel(shape_settled))
    sel_host_us = host_call_us(torch, sel(shape))
    dec_wait_us, dec_calls = graph_call_us(torch, dec(shape))
    dec_settled_us, _ = graph_call_us(torch, dec(shape_settled))
    dec_host_us = host_call_us(torch, dec(shape))
    gbs = lambda nbytes, us: nbytes / us / 1e3
    timing = ("CUDA events around back-to-back calls, one per layer over distinct buffers (nothing from L2), replayed "
              "as a CUDA graph (no host in the loop); every call waits for the kernel before it")
    roof = {"bound": "hbm", "kernel": "kvswap_sparse_decode (gather split-K + combine)",
            "achieved": gbs(decode_bytes, dec_wait_us), "peak": peak, "unit": "GB/s",
            "frac": gbs(decode_bytes, dec_wait_us) / peak, "frac_waiting_for_previous_kernel": gbs(decode_bytes, dec_wait_us) / peak,
            "peak_kind": peak_kind, "traffic": traffic,
            "algorithmic_bytes_per_launch": decode_bytes, "avg_ms": dec_wait_us / 1e3, "launches_timed": dec_calls,
            "timing": timing,
            "avg_ms_inputs_settled": dec_settled_us / 1e3, "frac_inputs_settled": gbs(decode_bytes, dec_settled_us) / peak,
            "avg_ms_issued_from_python": dec_host_us / 1e3,
            "frac_of_nominal_8000": gbs(decode_bytes, dec_wait_us) / 8000.0}
    roof_sel = {"bound": "hbm", "kernel": "kvswap_score_select (scorer with the low-rank queries + top-k)",
                "achieved": gbs(select_bytes, sel_wait_us), "peak": peak, "unit": "GB/s",
                "frac": gbs(select_bytes, sel_wait_us) / peak, "algorithmic_bytes_per_launch": select_bytes,
                "avg_ms": sel_wait_us / 1e3, "launches_timed": sel_calls,
                "avg_ms_inputs_settled": sel_settled_us / 1e3,
                "frac_inputs_settled": gbs(select_bytes, sel_settled_us) / peak,
                "avg_ms_issued_from_python": sel_host_us / 1e3,
                "keys_scored_per_sec_k2k3": wl.batch * wl.n_ctx / (sel_wait_us * 1e-6)}
    return roof, roof_sel


def read_probe(torch, kv, dw, peak):
    """What a kernel that only reads reaches on this GPU: kvswap_read_probe over buffers of the sizes the
    predictor streams (one layer's joint metadata), the attention gathers and 1 GiB, rotating over the
    layers' buffers so that nothing comes from L2; and the cost of an empty launch."""
    sink = torch.zeros(1, dtype=torch.int32, device=dw.K[0].device)
    L = len(dw.K)
    res = {}
    meta_bytes = dw.meta[0].numel() * dw.meta[0].element_size()
    kv_bytes = dw.K[0].numel() * dw.K[0].element_size()
    sizes = [("metadata_of_one_layer", dw.meta, meta_bytes // 16 * 16), ("gathered_kv_of_one_layer", dw.K, min(kv_bytes, 134217728)),
             ("1GiB", dw.K, min(kv_bytes // 16 * 16, 1 << 30))]
    for name, bufs, nbytes in sizes:
        fns = [(lambda l=l: kv.kvswap_read_probe(bufs[l], nbytes, sink)) for l in range(L)]
        us, _ = graph_call_us(torch, fns, 400)
        res[name] = {"bytes": nbytes, "us": us, "gbs": nbytes / us / 1e3, "frac_of_peak": nbytes / us / 1e3 / peak}
    us0, _ = graph_call_us(torch, [lambda: kv.kvswap_read_probe(dw.K[0], 0, sink)], 2000)
    return res, us0


def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2511_11907_b200 import binding as kv
    from paper_2511_11907_b200 import build as kvbuild
    from paper_2511_11907_b200 import device_workload as DW
    from paper_2511_11907_b200 import runtime as rt
    from paper_2511_11907_b200 import shard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py (impl=ours) needs a CUDA device: the kvswap hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if not os.path.exists(kv.LIB_PATH):
        if rank == 0:
            kvbuild.build()
        if world > 1:
            dist.barrier()
    kv.load()

    steps = args.steps if args.steps is not None else 400
    warmup = max(3, args.warmup if args.warmup is not None else 20)
    meta_heads = 1 if args.meta == "joint" else wl.n_kv_heads
    scope = W.SCOPE_KV_HEAD if args.scope == "kv_head" else W.SCOPE_ALL_HEADS

    dw = DW.build(wl, meta_heads, scope, device=dev, rank_offset=shard.rank_seed_offset(rank))
    shape, L = dw.shape, wl.layers
    ws = rt.alloc_workspace(shape, dev)
    stream = torch.cuda.current_stream()

    # ---- prefill: metadata build, timed separately (not part of the decode step) ----------------
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    kv.kvswap_project_keys(shape, dw.K[0], dw.proj[0], dw.meta[0], 0, wl.n_ctx, ws)   # first-call set-up, untimed
    torch.cuda.synchronize()
    ev0.record()
    for l in range(L):
        kv.kvswap_project_keys(shape, dw.K[l], dw.proj[l], dw.meta[l], 0, wl.n_ctx, ws)
    ev1.record()
    torch.cuda.synchronize()
    prefill_ms = ev0.elapsed_time(ev1)

    # the schedule a model can run: the predictor one layer ahead of the attention
    layers = dw.layer_tables(max_lookahead=1)
    S, M = shape.n_scopes, wl.top_k
    idx = torch.empty((L, wl.batch, S, M), dtype=torch.int32, device=dev)
    nsel = torch.empty((L, wl.batch, S), dtype=torch.int32, device=dev)
    out = torch.empty((L, wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32, device=dev)
    n_walk = dw.q_walk.shape[0]

    def step(i, probe=None):
        kv.kvswap_decode_step(shape, layers, dw.q_walk[i % n_walk], out, None, idx, nsel, ws, probe)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    for i in range(warmup):
        step(i)

    # ---- timed region: K steps, inputs resident in HBM ----------------------------------------------
    prev_sel, overlaps = None, []
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    wall0 = time.time()
    t_start.record()
    for i in range(steps):
        step(warmup + i)
    t_stop.record()
    sync_all()
    wall1 = time.time()
    elapsed_ms = t_start.elapsed_time(t_stop)
    # a longer run of the same loop for the clock record when the driver's K is small
    clock_pad = 0
    while rank == 0 and time.time() - wall0 < 0.6 and clock_pad < 2000:
        step(clock_pad)
        clock_pad += 1
        if clock_pad % 50 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    wall1_pad = time.time()

    # ---- selection overlap between consecutive steps (Sec. 4.4.2), outside the timed region ----
    for i in range(min(8, n_walk)):
        step(i)
        torch.cuda.synchronize()
        cur = idx[0].clone()
        if prev_sel is not None:
            a, b = cur.reshape(-1, M), prev_sel.reshape(-1, M)
            hit = (a.unsqueeze(2) == b.unsqueeze(1)).any(dim=2) & (a >= 0)
            overlaps.append(float(hit.float().sum() / (a >= 0).float().sum()))
        prev_sel = cur

    # ---- end to end: host queries in, host outputs back, every step ---------------------------------
    q_host = torch.empty((n_walk,) + tuple(dw.q_walk.shape[1:]), dtype=dw.q_walk.dtype).pin_memory()
    q_host.copy_(dw.q_walk)
    out_host = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    q_dev = torch.empty_like(dw.q_walk[0])
    e2e_steps = steps

    def step_host(i):
        kv.kvswap_decode_step_host(shape, layers, q_host[i % n_walk], out_host, q_dev, out, idx, nsel, ws)
        stream.synchronize()                     # the step's result is needed before the next token

    for i in range(3):
        step_host(i)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    e0.record()
    for i in range(e2e_steps):
        step_host(i)
    e1.record()
    sync_all()
    e2e_ms = e0.elapsed_time(e1)
    clocks = sampler.stop(wall0, max(wall1, wall1_pad)) if sampler else None
    if clocks is not None and clock_pad:
        clocks["window"] = "timed region and the same step loop continued to 0.6 s"

    # ---- growing context (Sec. 4.4.1): every step first appends one token per layer to the rolling buffer
    # (a completed group is flushed into the compact cache), then decodes over the grown context.  The
    # store's last rows serve as the spare rows, so the walk ends at the full length N. ------------------------
    N, Hkv, d_, r_ = wl.n_ctx, wl.n_kv_heads, wl.head_dim, wl.rank
    grow_steps = max(1, min(64, steps, N - 1))
    cap = dict(kv_strides=(Hkv * N * d_, N * d_, d_), meta_strides=(meta_heads * N * r_, N * r_, r_))
    grow_shapes = [rt.shape_for(wl, meta_heads, scope, n_ctx=n, **cap) for n in range(N - grow_steps, N + 1)]
    kv_t = dw.K[0].dtype
    k_new = torch.randn((L, wl.batch, Hkv, d_), device=dev).to(kv_t)
    v_new = torch.randn((L, wl.batch, Hkv, d_), device=dev).to(kv_t)

    def grow(t):
        kv.kvswap_append_step(grow_shapes[t], layers, k_new, v_new)
        kv.kvswap_decode_step(grow_shapes[t + 1], layers, dw.q_walk[t % n_walk], out, None, idx, nsel, ws, None)

    for t in range(min(2, grow_steps)):
        grow(t)
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    g0.record()
    for t in range(grow_steps):
        grow(t)
    g1.record()
    sync_all()
    grow_ms = g0.elapsed_time(g1)
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record()
    for t in range(grow_steps):
        kv.kvswap_append_step(grow_shapes[t], layers, k_new, v_new)
    a1.record()
    sync_all()
    append_ms = a0.elapsed_time(a1)
    # the appended rows changed the metadata of the last groups: rebuild it for the legs below
    for l in range(L):
        kv.kvswap_project_keys(shape, dw.K[l], dw.proj[l], dw.meta[l], max(0, N - 2 * grow_steps - wl.group_size), N, ws)

    reuse = reuse_buffer_leg(torch, kv, rt, wl, dw, shape, scope, idx, nsel, out, ws, dev) if rank == 0 else None

    # ---- max over ranks ----------------------------------------------------------------------------
    elapsed_ms, e2e_ms, grow_ms, append_ms = shard.max_over_ranks([elapsed_ms, e2e_ms, grow_ms, append_ms], device=dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- each call on its own, the read-only probe, the other workloads (rank 0) --------------------
    peak, peak_kind = measured_peak()
    step(0)                                                  # selections of a whole step in place
    torch.cuda.synchronize()
    traffic = NCU_TRAFFIC.get((wl.config, args.meta, args.scope))
    roof, roof_sel = call_rooflines(torch, kv, wl, dw, dw.meta, shape, idx, nsel, out, ws, L, peak, peak_kind, traffic)
    probe, launch_floor_us = read_probe(torch, kv, dw, peak)
    roof["read_probe_gbs"] = {k: v["gbs"] for k, v in probe.items()}
    roof["read_probe"] = probe
    roof["launch_floor_us"] = launch_floor_us
    shape_soft = shape.with_flags(kv.KVSWAP_SCORE_SOFTMAX)
    q0 = dw.q_walk[0]
    soft_us, _ = graph_call_us(torch, [(lambda l=l: kv.kvswap_score_select(shape_soft, q0[l], dw.proj[l], dw.meta[l], idx[l],
                                                                          nsel[l], None, ws)) for l in range(L)], 400)
    _, select_bytes = workload_bytes(wl, meta_heads, S)
    fp8 = fp8_metadata_leg(torch, kv, rt, wl, dw, meta_heads, scope, idx, nsel, dev, peak) if wl.meta_dtype == W.F16 and wl.rank == 32 else None
    shapes = prefill_shapes_leg(torch, kv, rt, wl, dw, dev, peak) if wl.kv_dtype == W.BF16 and not args.no_secondary else None
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        cpu = cpu_baseline(wl, dw, meta_heads, args.scope, rt)
    esz = {W.F32: 4, W.BF16: 2, W.F16: 2}
    kv_resident_gb = round(dw.layers_resident * 2 * dw.K[0].numel() * esz[wl.kv_dtype] / 1e9, 1)
    secondary = None
    if world == 1 and not args.no_secondary and wl.config == 5 and args.meta == "joint" and args.layers is None:
        secondary = secondary_workloads(torch, kv, rt, DW, wl, dw, scope, idx, nsel, out, dev, peak, peak_kind)

    ms_per_step = elapsed_ms / steps
    value = shard.aggregate_throughput(1.0, steps, elapsed_ms, world)
    keys_per_step = wl.batch * wl.n_ctx * L
    q_bytes = q_host[0].numel() * q_host.element_size()
    out_bytes = out_host.numel() * 4
    decode_bytes, _ = workload_bytes(wl, meta_heads, S)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if wl.kv_dtype == W.BF16 else ("f16" if wl.kv_dtype == W.F16 else "f32"),
        "data": "synthetic",
        "config": {"workload": workload_name(wl, args), "parallelism": f"batch shards x{world}, no collective",
                   "global_batch": wl.batch * world, "layers_resident": dw.layers_resident,
                   "l2": "inputs larger than L2: every step streams all layers' metadata and gathers from "
                         f"{dw.layers_resident} distinct KV stores (>> 126 MB) before any buffer repeats",
                   "kv_resident_gb": kv_resident_gb},
        "keys_scored_per_sec": value * keys_per_step,
        "keys_scored_per_sec_k2k3": roof_sel["keys_scored_per_sec_k2k3"],
        "schedule": {"predictor_lookahead_layers": 1,
                     "order": "score(l+1), attention(l), [combine(l) + top-k(l+1)] on one stream; programmatic dependent launches",
                     "step_bytes_per_sec_gbs": (decode_bytes + select_bytes) * L / (ms_per_step * 1e-3) / 1e9},
        "growing_context": {"value": world * 1e3 * grow_steps / grow_ms, "unit": UNIT, "steps": grow_steps,
                            "n_ctx": [N - grow_steps, N], "ms_per_step": grow_ms / grow_steps,
                            "append_ms_per_step": append_ms / grow_steps,
                            "flushes": sum(1 for n in range(N - grow_steps, N) if (n + 1) % wl.group_size == 0)},
        "reuse_buffer": reuse,
        "e2e": {"value": world * 1e3 * e2e_steps / e2e_ms, "unit": UNIT, "h2d_bytes_per_step": q_bytes,
                "d2h_bytes_per_step": out_bytes, "steps": e2e_steps},
        "gpu_launches": (3 * L + 1) * steps,
        "roofline": roof,
        "roofline_score_select": roof_sel,
        "secondary": secondary,
        "predictor_softmax_variant": {"kernel": "kvswap_score_select with KVSWAP_SCORE_SOFTMAX", "avg_ms": soft_us / 1e3,
                                      "frac": select_bytes / soft_us / 1e3 / peak,
                                      "algorithmic_bytes_per_launch": select_bytes},
        "metadata_8bit": fp8,
        "prefill": {"project_keys_ms_all_layers": prefill_ms,
                    "keys_projected_per_sec": keys_per_step / prefill_ms * 1e3,
                    "read_gbs": L * wl.batch * wl.n_kv_heads * wl.n_ctx * wl.head_dim * esz[wl.kv_dtype] / prefill_ms / 1e6,
                    "other_shapes_one_layer": shapes},
        "selection_overlap_ratio": statistics.mean(overlaps) if overlaps else None,
        "clocks": clocks,
    }
    if cpu is not None:
        line["cpu_baseline"] = cpu
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def prefill_shapes_leg(torch, kv, rt, wl, dw, dev, peak):
    """kvswap_project_keys (K1) on one layer of the workload's size for the other head dimensions and ranks
    the tensor-core projection takes (bf16 K, joint adapter): with a workspace (tcgen05) and without one
    (the warp-level kernel), read bandwidth over the K bytes.  Random adapters; timing only."""
    res = {}
    B, Hkv, N = wl.batch, wl.n_kv_heads, wl.n_ctx
    for d in (128, 64):
        K = dw.K[0] if d == wl.head_dim else (torch.randn((B, Hkv, N, d), device=dev, dtype=torch.float32) * 0.5).to(torch.bfloat16)
        for r in (16, 32, 64):
            shape = kv.make_shape(batch=B, n_ctx=N, n_q_heads=wl.n_q_heads, n_kv_heads=Hkv, head_dim=d, rank=r,
                                  meta_heads=1, group_size=wl.group_size, top_k=wl.top_k, kv_dtype=W.BF16,
                                  meta_dtype=W.F16, q_dtype=W.BF16)
            proj = torch.randn((Hkv, d, r), device=dev, dtype=torch.float32) * 0.05
            meta = torch.empty((B, 1, N, r), device=dev, dtype=torch.float16)
            ws = rt.alloc_workspace(shape, dev)
            us = []
            for w in (ws, None):
                for _ in range(3):
                    kv.kvswap_project_keys(shape, K, proj, meta, 0, N, w)
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(10):
                    kv.kvswap_project_keys(shape, K, proj, meta, 0, N, w)
                b.record()
                torch.cuda.synchronize()
                us.append(a.elapsed_time(b) * 100.0)
            nbytes = B * Hkv * N * d * 2
            res[f"d{d}_r{r}"] = {"us": us[0], "read_gbs": nbytes / us[0] / 1e3, "frac": nbytes / us[0] / 1e3 / peak,
                                 "us_without_workspace": us[1]}
            del meta, ws, proj
        del K
    return res


def fp8_metadata_leg(torch, kv, rt, wl, dw, meta_heads, scope, idx, nsel, dev, peak):
    """The predictor over an 8-bit compact cache (KVSWAP_E4M3: half the bytes of the fp16 one): the
    metadata of every layer rebuilt in that format, kvswap_score_select timed like the fp16 calls, and
    how many of the fp16 predictor's groups it still selects (reported, not graded)."""
    L, S = wl.layers, 1 if scope == W.SCOPE_ALL_HEADS else wl.n_kv_heads
    wl8 = wl.reduced(wl.name + "-e4m3", meta_dtype=W.E4M3)
    shape8 = rt.shape_for(wl8, meta_heads, scope)
    ws8 = rt.alloc_workspace(shape8, dev)
    meta8 = [torch.empty((wl.batch, meta_heads, wl.n_ctx, wl.rank), dtype=torch.uint8, device=dev) for _ in range(L)]
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    kv.kvswap_project_keys(shape8, dw.K[0], dw.proj[0], meta8[0], 0, wl.n_ctx, ws8)
    torch.cuda.synchronize()
    a.record()
    for l in range(L):
        kv.kvswap_project_keys(shape8, dw.K[l], dw.proj[l], meta8[l], 0, wl.n_ctx, ws8)
    b.record()
    torch.cuda.synchronize()
    prefill_ms = a.elapsed_time(b)
    q0 = dw.q_walk[0]
    idx8, nsel8 = torch.empty_like(idx), torch.empty_like(nsel)
    fns = [(lambda l=l: kv.kvswap_score_select(shape8, q0[l], dw.proj[l], meta8[l], idx8[l], nsel8[l], None, ws8)) for l in range(L)]
    us, calls = graph_call_us(torch, fns)
    torch.cuda.synchronize()
    both = (idx8.unsqueeze(-1) == idx.unsqueeze(-2)).any(dim=-1) & (idx8 >= 0)
    agree = float(both.float().sum() / (idx8 >= 0).float().sum())
    nbytes = wl.batch * meta_heads * wl.n_ctx * wl.rank + 2 * wl.batch * S * wl.n_groups * 4 + wl.batch * S * wl.top_k * 4
    return {"format": "E4M3, one byte per entry, power-of-two exponent 0", "avg_ms": us / 1e3, "launches_timed": calls,
            "algorithmic_bytes_per_launch": nbytes, "achieved": nbytes / us / 1e3, "unit": "GB/s",
            "frac": nbytes / us / 1e3 / peak, "prefill_ms_all_layers": prefill_ms,
            "groups_shared_with_the_fp16_predictor": agree}


def secondary_workloads(torch, kv, rt, DW, wl5, dw5, scope, idx, nsel, out, dev, peak, peak_kind):
    """The per-call rooflines and a short step loop on config 5 with per-head metadata (the resident
    K/V stores, metadata rebuilt per head for a few layers) and on config 4 (as many layers resident
    as fit beside nothing else: the config-5 stores are released first)."""
    res = {}
    # ---- config 5, one adapter per KV head ----------------------------------------------------------------
    Lp = min(6, wl5.layers)
    wl_p = wl5.reduced(wl5.name + "-per-head", layers=Lp)
    shape_p = rt.shape_for(wl_p, wl_p.n_kv_heads, scope)
    ws_p = rt.alloc_workspace(shape_p, dev)
    meta_p = [torch.empty((wl_p.batch, wl_p.n_kv_heads, wl_p.n_ctx, wl_p.rank), dtype=dw5.meta[0].dtype, device=dev) for _ in range(Lp)]
    proj_p = []
    for l in range(Lp):
        gen = torch.Generator(device=dev)
        gen.manual_seed(W.layer_seed(wl_p, l) * 131 + 5)
        calib = torch.randn((wl_p.calib_rows, wl_p.n_kv_heads, wl_p.head_dim), generator=gen, device=dev)
        proj_p.append(DW.adapter_on_device(calib, wl_p.rank, wl_p.n_kv_heads))
        kv.kvswap_project_keys(shape_p, dw5.K[l], proj_p[l], meta_p[l], 0, wl_p.n_ctx, ws_p)
    view = DW.DeviceWorkload(wl=wl_p, shape=shape_p, K=dw5.K[:Lp], V=dw5.V[:Lp], proj=proj_p, meta=meta_p,
                             q_walk=dw5.q_walk[:, :Lp], layers_resident=Lp)
    res["config5_per_head"] = secondary_leg(torch, kv, wl_p, view, shape_p, idx, nsel, out, ws_p, peak, peak_kind,
                                            NCU_TRAFFIC.get((5, "per_head", "kv_head")), wl5.layers)
    del meta_p, view, ws_p
    # ---- config 4 -------------------------------------------------------------------------------------------
    wl4 = W.CONFIGS[4]
    L4 = min(8, wl4.layers)
    dw5.K.clear(); dw5.V.clear(); dw5.meta.clear()
    torch.cuda.empty_cache()
    wl4r = wl4.reduced(wl4.name + "-resident", layers=L4)
    dw4 = DW.build(wl4r, 1, scope, device=dev)
    shape4 = dw4.shape
    ws4 = rt.alloc_workspace(shape4, dev)
    for l in range(L4):
        kv.kvswap_project_keys(shape4, dw4.K[l], dw4.proj[l], dw4.meta[l], 0, wl4r.n_ctx, ws4)
    S4, M4 = shape4.n_scopes, wl4r.top_k
    idx4 = torch.empty((L4, wl4r.batch, S4, M4), dtype=torch.int32, device=dev)
    nsel4 = torch.empty((L4, wl4r.batch, S4), dtype=torch.int32, device=dev)
    out4 = torch.empty((L4, wl4r.batch, wl4r.n_q_heads, wl4r.head_dim), dtype=torch.float32, device=dev)
    res["config4_joint"] = secondary_leg(torch, kv, wl4r, dw4, shape4, idx4, nsel4, out4, ws4, peak, peak_kind, None,
                                         wl4.layers)
    return res


def secondary_leg(torch, kv, wl, dw, shape, idx, nsel, out, ws, peak, peak_kind, traffic, layers_full):
    L = wl.layers
    layers = dw.layer_tables(max_lookahead=1)
    idx_l, nsel_l, out_l = idx[:L], nsel[:L], out[:L]
    q = dw.q_walk[0]
    for _ in range(5):
        kv.kvswap_decode_step(shape, layers, q, out_l, None, idx_l, nsel_l, ws, None)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = 100
    torch.cuda.synchronize()
    a.record()
    for _ in range(n):
        kv.kvswap_decode_step(shape, layers, q, out_l, None, idx_l, nsel_l, ws, None)
    b.record()
    torch.cuda.synchronize()
    us_per_layer = a.elapsed_time(b) * 1e3 / (n * L)
    roof, roof_sel = call_rooflines(torch, kv, wl, dw, dw.meta, shape, idx_l, nsel_l, out_l, ws, L, peak, peak_kind, traffic)
    return {"workload": f"config{wl.config}: B={wl.batch} N={wl.n_ctx} Hq/Hkv={wl.n_q_heads}/{wl.n_kv_heads} G={wl.group_size} "
                        f"M={wl.top_k} meta_heads={shape.meta_heads}",
            "layers_resident": dw.layers_resident, "layers_in_config": layers_full,
            "step_us_per_layer": us_per_layer,
            "steps_per_sec_scaled_to_all_layers": 1e6 / (us_per_layer * layers_full),
            "roofline": roof, "roofline_score_select": roof_sel}


def reuse_buffer_leg(torch, kv, rt, wl, dw, shape, scope, idx, nsel, out, ws, dev):
    """Reuse buffer (Sec. 4.4.2) on layer 0: the random-walk queries select overlapping groups step after
    step; hits are served from 2M slots in HBM, misses fetched from a copy of the layer's K/V in pinned
    host memory (the slow tier).  Reported: reuse rate and the cost of each phase; then the same through
    kvswap_decode_step_tiered over the first layers of the model."""
    n_walk = dw.q_walk.shape[0]
    if n_walk < 4 or wl.top_k > 8192:
        return None
    L, S = wl.layers, shape.n_scopes
    Hkv, d_, N = wl.n_kv_heads, wl.head_dim, wl.n_ctx
    kv_t = dw.K[0].dtype
    G_, M_, NG_ = wl.group_size, wl.top_k, wl.n_ctx // wl.group_size
    C_ = min(32768, 2 * M_)
    try:
        K_slow, V_slow = dw.K[0].cpu().pin_memory(), dw.V[0].cpu().pin_memory()
    except RuntimeError as exc:
        return {"skipped": f"could not pin the slow tier: {exc}"[:120]}
    Rr = (C_ + 1) * G_
    K_r = torch.zeros((wl.batch, Hkv, Rr, d_), dtype=kv_t, device=dev)
    V_r = torch.zeros((wl.batch, Hkv, Rr, d_), dtype=kv_t, device=dev)
    tail_ = N % G_
    K_r[:, :, C_ * G_:C_ * G_ + tail_] = dw.K[0][:, :, NG_ * G_:]
    V_r[:, :, C_ * G_:C_ * G_ + tail_] = dw.V[0][:, :, NG_ * G_:]
    shape_r = kv.reuse_attention_shape(shape, C_)
    ws_r = rt.alloc_workspace(shape_r, dev)
    state = torch.empty(kv.kvswap_reuse_state_bytes(shape, C_, NG_) // 4, dtype=torch.int32, device=dev)
    kv.kvswap_reuse_init(shape, C_, NG_, state)
    slot_i = torch.empty((wl.batch, S, M_), dtype=torch.int32, device=dev)
    m_g, m_s = torch.empty_like(slot_i), torch.empty_like(slot_i)
    n_m = torch.empty((wl.batch, S), dtype=torch.int32, device=dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    rates, t_look, t_fill, t_att, fill_bytes = [], [], [], [], []
    for t in range(min(n_walk, 32)):
        qt = dw.q_walk[t][0]
        kv.kvswap_score_select(shape, qt, dw.proj[0], dw.meta[0], idx[0], nsel[0], None, ws)
        ev[0].record()
        kv.kvswap_reuse_lookup(shape, C_, NG_, idx[0], nsel[0], state, slot_i, m_g, m_s, n_m)
        ev[1].record()
        kv.kvswap_reuse_fill(shape, C_, K_slow, V_slow, K_r, V_r, m_g, m_s, n_m)
        ev[2].record()
        kv.kvswap_sparse_decode(shape_r, qt, K_r, V_r, slot_i, nsel[0], out[0], None, ws_r)
        ev[3].record()
        torch.cuda.synchronize()
        misses = int(n_m.sum().item())
        rates.append(1.0 - misses / (wl.batch * S * min(M_, NG_)))
        t_look.append(ev[0].elapsed_time(ev[1])); t_fill.append(ev[1].elapsed_time(ev[2]))
        t_att.append(ev[2].elapsed_time(ev[3]))
        fill_bytes.append(misses * 2 * G_ * d_ * esz_of(wl.kv_dtype) * (1 if scope == W.SCOPE_KV_HEAD else Hkv))
    warm = slice(1, None)
    reuse = {"layer": 0, "n_slots": C_, "slow_tier": "pinned host memory", "steps": len(rates),
             "reuse_rate_mean": statistics.mean(rates[warm]), "reuse_rate_min": min(rates[warm]),
             "paper_reuse_rate": "0.753-0.812 (its datasets, its models)",
             "lookup_us": 1e3 * statistics.mean(t_look[warm]), "fill_us": 1e3 * statistics.mean(t_fill[warm]),
             "fill_gbs_from_host": statistics.mean(fill_bytes[warm]) / statistics.mean(t_fill[warm]) / 1e6,
             "attention_from_slots_us": 1e3 * statistics.mean(t_att[warm])}
    del K_slow, V_slow, K_r, V_r
    Lt = min(L, 4)
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
    Ks, Vs = [pin(dw.K[l]) for l in range(Lt)], [pin(dw.V[l]) for l in range(Lt)]
    Kr = [torch.zeros((wl.batch, Hkv, Rr, d_), dtype=kv_t, device=dev) for _ in range(Lt)]
    Vr = [torch.zeros((wl.batch, Hkv, Rr, d_), dtype=kv_t, device=dev) for _ in range(Lt)]
    for l in range(Lt):
        Kr[l][:, :, C_ * G_:C_ * G_ + tail_] = dw.K[l][:, :, NG_ * G_:]
        Vr[l][:, :, C_ * G_:C_ * G_ + tail_] = dw.V[l][:, :, NG_ * G_:]
    states = [torch.empty_like(state) for _ in range(Lt)]
    for st_l in states:
        kv.kvswap_reuse_init(shape, C_, NG_, st_l)
    sl_t = torch.empty((Lt, wl.batch, S, M_), dtype=torch.int32, device=dev)
    mg_t, ms_t = torch.empty_like(sl_t), torch.empty_like(sl_t)
    nm_t = torch.empty((Lt, wl.batch, S), dtype=torch.int32, device=dev)
    tiers = kv.make_tiers(C_, NG_, Ks, Vs, Kr, Vr, states, sl_t, mg_t, ms_t, nm_t)
    layers_t = kv.make_layers(Kr, Vr, dw.meta[:Lt], dw.proj[:Lt])
    ws_t = torch.empty(kv.kvswap_tiered_workspace_bytes(shape, C_), dtype=torch.uint8, device=dev)
    kv.kvswap_workspace_init(ws_t)
    step_ms, step_rate = [], []
    for t in range(min(n_walk, 16)):
        ev[0].record()
        kv.kvswap_decode_step_tiered(shape, layers_t, tiers, dw.q_walk[t][:Lt], out[:Lt], None, idx[:Lt],
                                     nsel[:Lt], ws_t)
        ev[1].record()
        torch.cuda.synchronize()
        step_ms.append(ev[0].elapsed_time(ev[1]))
        step_rate.append(1.0 - int(nm_t.sum().item()) / (Lt * wl.batch * S * min(M_, NG_)))
    reuse["tiered_step"] = {"layers": Lt, "steps": len(step_ms), "ms_per_layer": statistics.mean(step_ms[warm]) / Lt,
                            "ms_per_layer_cold": step_ms[0] / Lt, "reuse_rate_mean": statistics.mean(step_rate[warm])}
    return reuse


def main():
    global MIN_CALLS
    args = parse_args()
    if args.min_calls is not None:
        MIN_CALLS = max(1, args.min_calls)
    wl = W.CONFIGS[args.config]
    if args.layers is not None:
        wl = wl.reduced(wl.name + f"-L{args.layers}", layers=args.layers)
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            run_reference(args, wl)
        return
    run_ours(args, wl)


if __name__ == "__main__":
    main()
