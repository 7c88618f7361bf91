#!/usr/bin/env python
"""Benchmark of the AhaKV eviction step (score + select + compact) on B200.

A step is one fused ``ahakv_evict`` call over one layer of synthetic Q/K/V of the
named workload.  Prints ONE JSON line (rank 0).  ``--impl reference`` times the
CPU oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "context_tokens_evicted_per_sec_per_layer"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "long_32k"
SPEC_HBM_GBS = 8000.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--resident-layers", type=int, default=4,
                    help="distinct layers of input kept in HBM and cycled through")
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling small cases)")
    ap.add_argument("--capture", action="store_true",
                    help="profiler-friendly run: exactly --warmup and --steps calls of ahakv_evict, nothing else")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def algorithmic_work(w):
    """Bytes and FLOPs one eviction call must move / compute: K and V read once, Q_obs read, the kept
    K and V rows written once; 2*B*Hq*r*n*d FLOPs for the logits."""
    es = w.elem_size
    kv_read = 2 * w.batch * w.n_kv_heads * w.n_ctx * w.head_dim * es
    q_read = w.batch * w.n_q_heads * w.obs_window * w.head_dim * es
    kv_write = 2 * w.batch * w.n_kv_heads * w.n_keep * w.head_dim * es
    flops = 2 * w.batch * w.n_q_heads * w.obs_window * w.n_ctx * w.head_dim
    # the scoring kernel: K once and, with the value prior, V once (its value-norm warps), Q_obs, and the
    # raw score and nu vectors it writes (4 bytes per token and KV head each)
    per_token = 4 * w.batch * w.n_kv_heads * w.n_ctx
    score_bytes = kv_read // 2 + q_read + per_token + ((kv_read // 2 + per_token) if w.value_prior else 0)
    return dict(bytes=kv_read + q_read + kv_write, flops=flops, score_bytes=score_bytes)


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            pass

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), power_w_max=max(power),
                    samples=len(sm), reasons=sorted(reasons))


def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: what a multi-GPU number is divided by (no other data-path collective exists)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_step: int, world: int, ms_step: float) -> float:
    """Replicas only: every rank evicts its own layer, so the job's throughput is world x one replica's
    tokens over the slowest rank's time."""
    return world * tokens_per_step / (ms_step * 1e-3)


def cpu_oracle_sample(w, seconds_hint=15.0):
    """Times the oracle, as it stands, on a bounded sample of the workload: whole (sequence, KV head)
    units of layer 0, one per host thread per round.  Returns (tokens/s for a full layer, info)."""
    import torch
    from oracle import ahakv_oracle as orc
    from paper_2506_03762_b200 import synth
    orc.build()
    cores = len(os.sched_getaffinity(0))
    per_unit_macs = w.group * w.obs_window * w.n_ctx * w.head_dim
    units_total = w.batch * w.n_kv_heads
    # ~0.35 GMAC/s per core is what the plain loops reach; size the sample for about seconds_hint
    est_unit_s = per_unit_macs / 0.35e9
    rounds = max(1, min(4, int(seconds_hint / max(est_unit_s, 1e-3))))
    n_units = min(units_total, cores * rounds)
    Hkv_s = min(w.n_kv_heads, n_units)
    B_s = max(1, min(w.batch, n_units // Hkv_s))
    n_units = B_s * Hkv_s
    ws = w.scaled(batch=B_s, n_q_heads=Hkv_s * w.group, n_kv_heads=Hkv_s)
    q, k, v = synth.make_layer(ws, layer=0, device="cpu")
    code = {"f32": orc.F32, "f16": orc.F16, "bf16": orc.BF16}[w.dtype]
    p = orc.OracleParams(ws.batch, ws.n_q_heads, ws.n_kv_heads, ws.head_dim, ws.n_ctx, ws.obs_window,
                         ws.recent_window, ws.budget, dtype=code, n_total=ws.n_total,
                         pool_kernel=ws.pool_kernel, flags=orc.FLAG_VALUE_PRIOR if ws.value_prior else 0)
    qn, kn, vn = (synth.to_numpy(t) for t in (q, k, v))
    prev = None
    if w.n_total is not None:
        prev = synth.make_score_prev(ws, new_rows=ws.obs_window).double().numpy()
    t0 = time.perf_counter()
    orc.evict(p, qn, kn, vn, prev, nthreads=cores)
    dt = time.perf_counter() - t0
    tokens = n_units / w.n_kv_heads * w.n_ctx        # context tokens of whole sequences' worth of heads
    value = tokens / dt
    info = dict(value=value, unit=UNIT, cores=min(cores, n_units), kind="oracle",
                sample=f"{n_units} of {units_total} (sequence, KV head) units of one {w.name} layer "
                       f"in {dt:.2f} s, scaled to a full layer")
    return value, dt, info


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2506_03762_b200 import synth
    w = synth.WORKLOADS[args.workload]
    steps = max(1, min(args.steps, 3))
    warm = min(args.warmup, 1)
    for _ in range(warm):
        cpu_oracle_sample(w, seconds_hint=5.0)
    vals, times, info = [], [], None
    for _ in range(steps):
        v, dt, info = cpu_oracle_sample(w, seconds_hint=5.0)
        vals.append(v); times.append(dt)
    value = statistics.mean(vals)
    info["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": 1e3 * statistics.mean(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, args),
        "cpu_baseline": info,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "note": "the CPU oracle (double precision, one thread per unit) on a bounded sample per step",
    }))


def workload_config(w, args):
    return {"workload": w.name, "batch": w.batch, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
            "head_dim": w.head_dim, "n_ctx": w.n_ctx, "obs_window": w.obs_window,
            "recent_window": w.recent_window, "budget": w.budget, "layers_per_pass": w.n_layers,
            "resident_layers": args.resident_layers, "value_prior": w.value_prior,
            "scale_mode": "adaptive_row", "pool_kernel": w.pool_kernel,
            "l2": "each step's inputs (K+V of a layer) are larger than L2 and steps cycle through "
                  "distinct resident layers", "parallelism": "replicas only"}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2506_03762_b200 import binding as ab
    from paper_2506_03762_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; the eviction path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    ab.lib()

    w = synth.WORKLOADS[args.workload]
    if args.batch > 0:
        w = w.scaled(batch=args.batch)
    flags = ab.FLAG_VALUE_PRIOR if w.value_prior else 0
    p = ab.Params(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_ctx, w.obs_window, w.recent_window,
                  w.budget, dtype={"f32": ab.F32, "f16": ab.F16, "bf16": ab.BF16}[w.dtype],
                  n_total=w.n_total, pool_kernel=w.pool_kernel, flags=flags)
    L = max(1, min(args.resident_layers, max(w.n_layers, 1)))
    layers = [synth.make_layer(w, layer=l, device=dev, seed=synth.BASE_SEED + rank) for l in range(L)]
    prev = synth.make_score_prev(w, device=dev, new_rows=w.obs_window) if w.n_total is not None else None
    ws = ab.alloc_workspace(p, dev)
    k_out, v_out, s_out, idx = ab.alloc_outputs(p, dev)
    stream = torch.cuda.current_stream()

    def step(i):
        q, k, v = layers[i % L]
        ab.ahakv_evict(p, q, k, v, prev, k_out, v_out, s_out, idx, ws, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    n_warm = args.warmup if args.capture else max(args.warmup, 3)
    for i in range(n_warm):
        step(i)
    barrier()
    if args.capture:
        for i in range(args.steps):
            step(i)
        barrier()
        print(json.dumps({"capture": True, "workload": w.name, "batch": w.batch, "steps": args.steps,
                          "warmup": n_warm, "device_status": ab.ahakv_last_device_status(ws)}))
        return
    assert ab.ahakv_last_device_status(ws) == ab.OK, "device-side wait timed out during warm-up"

    # ---- timed region: exactly K steps, device-timed -------------------------------------------------
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ab.ahakv_launch_count()
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    launches = ab.ahakv_launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    status = ab.ahakv_last_device_status(ws)
    ms_total = max_over_ranks(ms_total, world, dev)
    ms_step = ms_total / args.steps
    tokens_per_step = w.batch * w.n_ctx
    value = whole_job_value(tokens_per_step, world, ms_step)

    # ---- per-stage device times over the same K steps (events inside the library) ----------------------
    ab.ahakv_profile_enable(True)
    for i in range(args.steps):
        step(i)
    calls, stage_ms = ab.ahakv_profile_read()
    ab.ahakv_profile_enable(False)
    stage_ms = {k_: v_ / max(calls, 1) for k_, v_ in stage_ms.items()}
    # a stage that launched nothing in this configuration (value norms and selection are fused into their
    # neighbours on the tensor-core path) still brackets a pair of events, a few microseconds: leave it out
    stage_ms = {k_: v_ for k_, v_ in stage_ms.items() if v_ > 0.004 or k_ in ("score", "compact")}

    # ---- end to end: pinned host inputs -> device, evict, outputs -> host, every step --------------------
    e2e = None
    if args.e2e_steps > 0:
        q0, k0, v0 = layers[0]
        hq, hk, hv = (torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for t in (q0, k0, v0))
        dq, dk, dv = (torch.empty_like(t) for t in (q0, k0, v0))
        houts = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in (k_out, v_out, s_out, idx)]

        def e2e_step():
            dq.copy_(hq, non_blocking=True); dk.copy_(hk, non_blocking=True); dv.copy_(hv, non_blocking=True)
            ab.ahakv_evict(p, dq, dk, dv, prev, k_out, v_out, s_out, idx, ws, stream=stream)
            for h, d_ in zip(houts, (k_out, v_out, s_out, idx)):
                h.copy_(d_, non_blocking=True)

        e2e_step()
        barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step()
        a1.record(stream)
        barrier()
        e2e_ms = a0.elapsed_time(a1) / args.e2e_steps
        e2e_ms = max_over_ranks(e2e_ms, world, dev)
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
        d2h = sum(t.numel() * t.element_size() for t in houts)
        e2e = {"value": whole_job_value(tokens_per_step, world, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": args.e2e_steps,
               "api": "ahakv_evict through the C ABI, pinned host buffers copied in and out every step"}
        del hq, hk, hv, dq, dk, dv, houts

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    work = algorithmic_work(w)
    t_roof_ms = 1e3 * max(work["flops"] / (pk["bf16_tflops_sustained"] * 1e12), work["bytes"] / (pk["hbm_gbs"] * 1e9))
    top = max(stage_ms, key=stage_ms.get)
    stage_bytes = {"score": work["score_bytes"],
                   "compact": 2 * 2 * w.batch * w.n_kv_heads * w.n_keep * w.head_dim * w.elem_size}
    dom = "score"
    achieved = stage_bytes[dom] / (stage_ms[dom] * 1e-3) / 1e9 if stage_ms[dom] > 0 else 0.0
    # DRAM bytes of one launch from the ncu capture summarised in profiles/score_tc_kernel_long32k_b2.txt:
    # 1108.4 MB at batch 2, scaled by the units a launch of this run processes (traffic grows with them).
    traffic = None
    if w.name == "long_32k" and w.value_prior:
        traffic = 1108.4e6 * w.batch / 2
    roofline = {"kernel": "score_tc_kernel (logits, SG-softmax, column sums, value norms)", "bound": "hbm",
                "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": achieved / pk["hbm_gbs"],
                "peak_source": f"{pk['source']} (sustained copy)", "traffic": traffic,
                "algorithmic_bytes_per_launch": stage_bytes[dom], "ms_per_launch": stage_ms[dom],
                "slowest_stage": top}
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": n_warm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic", "config": workload_config(w, args),
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "device_status": int(status),
        "roofline": roofline,
        "path_roofline": {"t_roof_ms": t_roof_ms, "frac": t_roof_ms / ms_step, "algorithmic_bytes": work["bytes"],
                          "flops": work["flops"], "frac_vs_spec_8TBs": 1e3 * work["bytes"] / (SPEC_HBM_GBS * 1e9) / ms_step,
                          "of": pk["source"]},
        "stage_ms": stage_ms,
        "stage_gbs": {s: stage_bytes[s] / (stage_ms[s] * 1e-3) / 1e9 for s in stage_bytes if stage_ms.get(s, 0) > 0},
        "tokens_per_step": tokens_per_step,
    }
    if world == 1 and not args.no_cpu_baseline:
        _, _, info = cpu_oracle_sample(w)
        out["cpu_baseline"] = info
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
