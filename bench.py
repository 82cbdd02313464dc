#!/usr/bin/env python
"""Benchmark of the KVSwap decode hot path (predictor + sparse decode attention) on B200.

A *step* is one decode step over all L layers of the workload through kvswap_decode_step: per
layer the predictor (low-rank scoring -> head sum -> group max -> top-k) and the sparse decode
attention (gather + split-K online-softmax attention + combine); the predictor's kernels run on
the library's internal stream ahead of the attention's, as the paper's runtime overlaps them.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 5] [--meta joint|per_head]
    python bench.py --impl reference ...      # the CPU oracle timed on the host cores

Prints ONE JSON line (rank 0).  `value` is decode steps/s with every input resident in HBM;
`e2e` is the same step driven through kvswap_decode_step_host with the step's queries in pinned
host memory and its outputs read back, both copies inside the timed region.  Beside them:
`roofline` (the attention call against the measured HBM peak), `roofline_score_select`,
`schedule.lookahead_1` (the predictor held one layer ahead), `growing_context` (a token appended
per layer before every step), `reuse_buffer` (hit rate and phase costs with the slow tier in
pinned host memory, and the tiered step), `prefill`, `cpu_baseline`.
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
# kernel, from the ncu capture summarised in profiles/decode_kernels_config5_one_layer.md (taken at
# full config-5 shapes on one layer; the traffic of a launch does not depend on the layer count).
# None for workloads that were not captured.  Key: (config, metadata layout, scope).
NCU_TRAFFIC = {(5, "joint", "kv_head"): 134455808 + 3698688}


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
# CPU oracle timing (cpu_baseline leg and the --impl reference arm)
# --------------------------------------------------------------------------------------------
def oracle_unit_time(K, V, q, proj, meta, wl, scope_name, heads=None):
    """Seconds the oracle needs for one (layer, sequence) unit: score_select then attend.
    K, V [1,H_kv,N,d]; q [1,H_q,d]; meta [1,H_m,N,r].  `heads` limits the unit to the first
    KV heads (per-head work is independent; the caller scales)."""
    from oracle import kvswap_oracle as O
    if heads is not None and heads < wl.n_kv_heads:
        rho = wl.rho
        K, V, q, proj = K[:, :heads], V[:, :heads], q[:, :heads * rho], proj[:heads]
        if meta.shape[1] != 1:
            meta = meta[:, :heads]
    t0 = time.perf_counter()
    idx, _ = O.score_select(q, proj, meta, wl.group_size, wl.top_k, scope_name)
    O.attend(q, K, V, idx, wl.group_size, scope_name)
    return time.perf_counter() - t0


def host_unit_inputs(wl, layer, meta_heads, seed_salt=0):
    """One sequence of one layer drawn on the host (numpy) + oracle metadata (not timed)."""
    from oracle import kvswap_oracle as O
    one = wl.reduced(wl.name + "-unit", batch=1, walk_steps=1)
    li = W.make_layer(one, layer, meta_heads)
    meta = O.project_keys(li.K, li.proj, meta_heads, "f16" if wl.meta_dtype == W.F16 else "f32")
    return li.K, li.V, li.q, li.proj, meta


def threads_used():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return 1


def run_reference(args, wl):
    """The oracle as it stands, on the host cores, on a bounded sample of the same workload."""
    steps = args.steps if args.steps is not None else 5
    warmup = args.warmup if args.warmup is not None else 1
    meta_heads = 1 if args.meta == "joint" else wl.n_kv_heads
    scope_name = args.scope
    K, V, q, proj, meta = host_unit_inputs(wl, 0, meta_heads)
    # size the per-step sample so that the whole run stays within a few minutes
    t_probe = oracle_unit_time(K, V, q, proj, meta, wl, scope_name, heads=1)
    budget = 150.0 / max(1, steps + warmup)
    heads = int(max(1, min(wl.n_kv_heads, budget // max(t_probe, 1e-3))))
    if scope_name == "all_heads":
        heads = wl.n_kv_heads
    for _ in range(warmup):
        oracle_unit_time(K, V, q, proj, meta, wl, scope_name, heads)
    times = [oracle_unit_time(K, V, q, proj, meta, wl, scope_name, heads) for _ in range(steps)]
    t_unit = statistics.mean(times) * (wl.n_kv_heads / heads)
    ms_per_step = t_unit * wl.layers * wl.batch * 1e3
    value = 1e3 / ms_per_step
    sample = (f"each timed step = oracle score_select+attend on 1 of {wl.layers} layers x 1 of {wl.batch} sequences "
              f"x {heads} of {wl.n_kv_heads} KV heads; scaled linearly to the full step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(wl, args)},
        "keys_scored_per_sec": value * wl.batch * wl.n_ctx * wl.layers,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads_used(), "kind": "oracle", "sample": sample,
                         "host_cores_available": len(os.sched_getaffinity(0))},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
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

    layers = dw.layer_tables()
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
    probes = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
               torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    probe_structs = [kv.make_probe(i % L, *probes[i]) for i in range(steps)]
    prev_sel, overlaps = None, []
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    wall0 = time.time()
    t_start.record()
    for i in range(steps):
        step(warmup + i, probe_structs[i])
    t_stop.record()
    sync_all()
    wall1 = time.time()
    elapsed_ms = t_start.elapsed_time(t_stop)
    select_ms = [p[0].elapsed_time(p[1]) for p in probes]
    decode_ms = [p[1].elapsed_time(p[2]) for p in probes]

    # ---- the same step with the predictor held to one layer ahead of the attention (what a model's
    # own layer-to-layer dependency allows); reported beside the headline, which uses the default --------
    layers_1 = dw.layer_tables(max_lookahead=1)
    n1 = max(1, min(steps, 100))
    for i in range(3):
        kv.kvswap_decode_step(shape, layers_1, dw.q_walk[i % n_walk], out, None, idx, nsel, ws, None)
    a1, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    a1.record()
    for i in range(n1):
        kv.kvswap_decode_step(shape, layers_1, dw.q_walk[i % n_walk], out, None, idx, nsel, ws, None)
    b1.record()
    sync_all()
    look1_ms = a1.elapsed_time(b1)

    # ---- each call on its own, back to back over all layers (every launch reads a different layer's
    # buffers, so nothing is served from L2): the average launch duration the roofline uses -----------
    def per_call_ms(fn):
        reps = max(1, min(steps, 200 // L + 1))
        for l in range(L):
            fn(l)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            for l in range(L):
                fn(l)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * L), reps * L

    q0 = dw.q_walk[0]
    # the selections are in place before these calls are enqueued: the launch configuration of the step
    # (KVSWAP_INPUTS_SETTLED, consecutive launches overlap their prologue and tail); the default mode,
    # which waits for the previous kernel first, is timed beside it
    shape_settled = shape.with_flags(kv.KVSWAP_INPUTS_SETTLED)
    dec_call_ms, dec_calls = per_call_ms(lambda l: kv.kvswap_sparse_decode(
        shape_settled, q0[l], dw.K[l], dw.V[l], idx[l], nsel[l], out[l], None, ws))
    sel_call_ms, sel_calls = per_call_ms(lambda l: kv.kvswap_score_select(
        shape_settled, q0[l], dw.proj[l], dw.meta[l], idx[l], nsel[l], None, ws))
    sel_wait_ms, _ = per_call_ms(lambda l: kv.kvswap_score_select(
        shape, q0[l], dw.proj[l], dw.meta[l], idx[l], nsel[l], None, ws))
    dec_wait_ms, _ = per_call_ms(lambda l: kv.kvswap_sparse_decode(
        shape, q0[l], dw.K[l], dw.V[l], idx[l], nsel[l], out[l], None, ws))
    # predictor variant: per-head softmax over the context before the head sum (general fp32 kernels)
    shape_soft = shape.with_flags(kv.KVSWAP_SCORE_SOFTMAX | kv.KVSWAP_INPUTS_SETTLED)
    soft_ms, _ = per_call_ms(lambda l: kv.kvswap_score_select(
        shape_soft, q0[l], dw.proj[l], dw.meta[l], idx[l], nsel[l], None, ws))

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
    clocks = sampler.stop(wall0, wall1) if sampler else None

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

    # ---- reuse buffer (Sec. 4.4.2) on layer 0: the random-walk queries select overlapping groups step
    # after step; hits are served from 2M slots in HBM, misses fetched from a copy of the layer's K/V in
    # pinned host memory (the slow tier).  Reported: reuse rate and the cost of each phase. ------------------
    reuse = None
    if rank == 0 and n_walk >= 4 and wl.top_k <= 8192:
        G_, M_, NG_ = wl.group_size, wl.top_k, wl.n_ctx // wl.group_size
        C_ = min(32768, 2 * M_)
        try:
            K_slow, V_slow = dw.K[0].cpu().pin_memory(), dw.V[0].cpu().pin_memory()
        except RuntimeError as exc:
            K_slow = None
            reuse = {"skipped": f"could not pin the slow tier: {exc}"[:120]}
        if K_slow is not None:
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
            # the same through kvswap_decode_step_tiered over the first layers of the model: lookup and miss
            # gather run on the predictor stream, ahead of the attention of the layers before
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
            del Ks, Vs, Kr, Vr

    # ---- max over ranks ----------------------------------------------------------------------------
    elapsed_ms, e2e_ms, look1_ms, grow_ms, append_ms = shard.max_over_ranks(
        [elapsed_ms, e2e_ms, look1_ms, grow_ms, append_ms], device=dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    esz = {W.F32: 4, W.BF16: 2, W.F16: 2}
    Mp = min(M, wl.n_groups)
    ms_per_step = elapsed_ms / steps
    value = shard.aggregate_throughput(1.0, steps, elapsed_ms, world)
    keys_per_step = wl.batch * wl.n_ctx * L
    decode_bytes = 2 * wl.batch * wl.n_kv_heads * Mp * wl.group_size * wl.head_dim * esz[wl.kv_dtype] + wl.batch * S * M * 4
    select_bytes = (wl.batch * meta_heads * wl.n_ctx * wl.rank * esz[wl.meta_dtype] + 2 * wl.batch * S * wl.n_groups * 4
                    + wl.batch * S * M * 4)
    peak, peak_kind = measured_peak()
    dec_ms, sel_ms = dec_call_ms, sel_call_ms
    dec_gbs, sel_gbs = decode_bytes / dec_ms / 1e6, select_bytes / sel_ms / 1e6
    traffic = NCU_TRAFFIC.get((wl.config, args.meta, args.scope))
    q_bytes = q_host[0].numel() * q_host.element_size()
    out_bytes = out_host.numel() * 4

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if wl.kv_dtype == W.BF16 else ("f16" if wl.kv_dtype == W.F16 else "f32"),
        "data": "synthetic",
        "config": {"workload": workload_name(wl, args), "parallelism": f"batch shards x{world}, no collective",
                   "global_batch": wl.batch * world, "layers_resident": dw.layers_resident,
                   "l2": "inputs larger than L2: every step streams all layers' metadata and gathers from "
                         f"{dw.layers_resident} distinct KV stores (>> 126 MB) before any buffer repeats",
                   "kv_resident_gb": round(dw.layers_resident * 2 * dw.K[0].numel() * esz[wl.kv_dtype] / 1e9, 1)},
        "keys_scored_per_sec": value * keys_per_step,
        "schedule": {"predictor_lookahead_layers": "unbounded",
                     "lookahead_1": {"value": world * 1e3 * n1 / look1_ms, "unit": UNIT, "steps": n1,
                                     "ms_per_step": look1_ms / n1}},
        "growing_context": {"value": world * 1e3 * grow_steps / grow_ms, "unit": UNIT, "steps": grow_steps,
                            "n_ctx": [N - grow_steps, N], "ms_per_step": grow_ms / grow_steps,
                            "append_ms_per_step": append_ms / grow_steps,
                            "flushes": sum(1 for n in range(N - grow_steps, N) if (n + 1) % wl.group_size == 0)},
        "reuse_buffer": reuse,
        "e2e": {"value": world * 1e3 * e2e_steps / e2e_ms, "unit": UNIT, "h2d_bytes_per_step": q_bytes,
                "d2h_bytes_per_step": out_bytes, "steps": e2e_steps},
        "gpu_launches": 5 * L * steps,
        "roofline": {"bound": "hbm", "kernel": "kvswap_sparse_decode (gather split-K + combine)",
                     "achieved": dec_gbs, "peak": peak, "unit": "GB/s", "frac": dec_gbs / peak, "peak_kind": peak_kind,
                     "traffic": traffic, "algorithmic_bytes_per_launch": decode_bytes, "avg_ms": dec_ms,
                     "launches_timed": dec_calls,
                     "timing": "CUDA events around back-to-back calls over all layers, inputs settled as in the step",
                     "avg_ms_waiting_for_previous_kernel": dec_wait_ms,
                     "frac_waiting_for_previous_kernel": decode_bytes / dec_wait_ms / 1e6 / peak,
                     "in_step_probe_ms": statistics.mean(decode_ms), "frac_of_nominal_8000": dec_gbs / 8000.0},
        "roofline_score_select": {"bound": "hbm", "kernel": "kvswap_score_select (lowrank_query + score_pool + topk)",
                                  "achieved": sel_gbs, "peak": peak, "unit": "GB/s", "frac": sel_gbs / peak,
                                  "algorithmic_bytes_per_launch": select_bytes, "avg_ms": sel_ms,
                                  "launches_timed": sel_calls,
                                  "avg_ms_waiting_for_previous_kernel": sel_wait_ms,
                                  "frac_waiting_for_previous_kernel": select_bytes / sel_wait_ms / 1e6 / peak,
                                  "in_step_probe_ms": statistics.mean(select_ms)},
        "predictor_softmax_variant": {"kernel": "kvswap_score_select with KVSWAP_SCORE_SOFTMAX", "avg_ms": soft_ms,
                                      "frac": select_bytes / soft_ms / 1e6 / peak,
                                      "algorithmic_bytes_per_launch": select_bytes},
        "prefill": {"project_keys_ms_all_layers": prefill_ms,
                    "keys_projected_per_sec": keys_per_step / prefill_ms * 1e3,
                    "read_gbs": L * wl.batch * wl.n_kv_heads * wl.n_ctx * wl.head_dim * esz[wl.kv_dtype] / prefill_ms / 1e6},
        "selection_overlap_ratio": statistics.mean(overlaps) if overlaps else None,
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(wl, dw, meta_heads, args.scope, rt)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def cpu_baseline(wl, dw, meta_heads, scope_name, rt):
    """The oracle on (layer, sequence) units of the resident workload until ~10 s are spent."""
    units, spent, t_units = 0, 0.0, []
    while spent < 10.0 and units < wl.layers * wl.batch:
        l, b = units % wl.layers, (units // wl.layers) % wl.batch
        K = rt.to_host_f32(dw.K[l][b:b + 1])
        V = rt.to_host_f32(dw.V[l][b:b + 1])
        q = rt.to_host_f32(dw.q_walk[0, l, b:b + 1])
        meta = rt.to_host_f32(dw.meta[l][b:b + 1])
        proj = dw.proj[l].cpu().numpy()
        t = oracle_unit_time(K, V, q, proj, meta, wl, scope_name)
        t_units.append(t)
        spent += t
        units += 1
    t_step = statistics.mean(t_units) * wl.layers * wl.batch
    return {"value": 1.0 / t_step, "unit": UNIT, "cores": threads_used(), "kind": "oracle",
            "sample": f"{units} (layer, sequence) units of the same workload ({spent:.1f} s of oracle time), "
                      f"scaled to L*B = {wl.layers * wl.batch} units per step",
            "host_cores_available": len(os.sched_getaffinity(0))}


def main():
    args = parse_args()
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
