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
    ap.add_argument("--repeats", type=int, default=10,
                    help="the block of --steps calls is timed this many times; ms_per_step is the median block")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--resident-layers", type=int, default=4,
                    help="distinct layers of input kept in HBM and cycled through (at least; more when one "
                         "layer's K and V are small against L2)")
    ap.add_argument("--no-protocol", action="store_true",
                    help="decode_round only: skip the 256-step protocol (8 chained rounds, evict-every-step)")
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling small cases)")
    ap.add_argument("--widened", action="store_true",
                    help="time the entry points beyond the eviction step (variants, ragged batch, entropy) instead")
    ap.add_argument("--capture", action="store_true",
                    help="profiler-friendly run: exactly --warmup and --steps calls of ahakv_evict (for decode_round "
                         "also --steps generation steps of each kind), nothing else")
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


L2_BYTES = 126e6


def kernel_source_digest():
    """sha1 of the scoring kernel's sources: DRAM counters taken from an older kernel are not reported."""
    import hashlib
    h = hashlib.sha1()
    for name in ("score_tc.cu", "tc_common.cuh"):
        with open(os.path.join(ROOT, "paper_2506_03762_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_traffic(w):
    """DRAM bytes of one launch of the scoring kernel from the tracked ncu summary (profiles/*.json): counters of a
    small case (batch 2), scaled by the units a launch of this run processes -- traffic grows with them.  None when
    there is no summary for this workload or the kernel has changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", f"score_tc_kernel_{w.name}.json")
    if not os.path.exists(path):
        return None, None
    d = json.load(open(path))
    if d.get("kernel_source_sha1") != kernel_source_digest() or bool(d.get("value_prior")) != bool(w.value_prior):
        return None, os.path.relpath(path, ROOT) + " (stale: the kernel has changed since)"
    per_unit = (d["dram_bytes_read"] + d["dram_bytes_write"]) / float(d["units"])
    return per_unit * w.batch * w.n_kv_heads, os.path.relpath(path, ROOT)


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


def kv_bytes(w):
    return 2 * w.batch * w.n_kv_heads * w.n_ctx * w.head_dim * w.elem_size


def resident_copies(w, args):
    """Distinct seeded layers kept in HBM: enough that a step never finds its inputs in L2 (the copies between
    two uses of a layer amount to at least twice L2), within 48 GB."""
    need = int(-(-2 * L2_BYTES // kv_bytes(w))) + 1
    cap = max(1, int(48e9 // max(kv_bytes(w), 1)))
    return max(1, min(max(args.resident_layers, need), cap))


def workload_config(w, args, copies=None):
    copies = resident_copies(w, args) if copies is None else copies
    return {"workload": w.name, "batch": w.batch, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
            "head_dim": w.head_dim, "n_ctx": w.n_ctx, "obs_window": w.obs_window,
            "recent_window": w.recent_window, "budget": w.budget, "layers_per_pass": w.n_layers,
            "resident_layers": copies, "value_prior": w.value_prior,
            "scale_mode": "adaptive_row", "pool_kernel": w.pool_kernel,
            "l2": f"steps cycle through {copies} distinct seeded layers resident in HBM, "
                  f"{copies * kv_bytes(w) / 1e6:.0f} MB of K and V against {L2_BYTES / 1e6:.0f} MB of L2, so no step finds "
                  "its inputs in L2; warm_ms_per_step is the same call repeated on one layer",
            "parallelism": "replicas only"}


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
    L = resident_copies(w, args)
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
        if w.name == "decode_round":
            # the generation step's kernels on the same cache, held at budget + 1 rows: the three-call step and the
            # slot-cache step, --steps times each
            Bud, n1 = w.budget, w.budget + 1
            q, k, v = layers[0]
            kc, vc = k[:, :, :n1].contiguous(), v[:, :, :n1].contiguous()
            fc = torch.rand((w.batch, w.n_kv_heads, n1), device=dev)
            idx1 = torch.empty((w.batch, w.n_kv_heads, Bud), dtype=torch.int32, device=dev)
            pos = torch.arange(n1, dtype=torch.int32, device=dev).repeat(w.batch, w.n_kv_heads, 1).contiguous()
            pos[:, :, Bud] = -1
            free = torch.full((w.batch, w.n_kv_heads), Bud, dtype=torch.int32, device=dev)
            for t in range(args.steps):
                p1 = ab.Params(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, n1, 1, w.recent_window, Bud,
                               dtype={"f32": ab.F32, "f16": ab.F16, "bf16": ab.BF16}[w.dtype], n_total=n1 + t, flags=0)
                qt, kt, vt = synth.make_decode_step(w, t, device=dev)
                ab.ahakv_score_step(p1, qt, kc, fc, fc, stream=stream)
                ab.ahakv_select(p1, fc, idx1, stream=stream)
                ab.ahakv_compact_inplace(p1, kc, vc, fc, idx1, stream=stream)
                ab.ahakv_step_slots(p1, qt, kt, vt, kc, vc, fc, pos, free, stream=stream)
        barrier()
        print(json.dumps({"capture": True, "workload": w.name, "batch": w.batch, "steps": args.steps,
                          "warmup": n_warm, "device_status": ab.ahakv_last_device_status(ws)}))
        return
    assert ab.ahakv_last_device_status(ws) == ab.OK, "device-side wait timed out during warm-up"

    # ---- timed region: blocks of exactly K steps, each bracketed and device-timed; the median block counts ------
    sampler = ClockSampler(local) if rank == 0 else None
    blocks = []
    launches = 0
    for rep in range(max(1, args.repeats)):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = ab.ahakv_launch_count()
        barrier()
        e0.record(stream)
        for i in range(args.steps):
            step(rep * args.steps + i)
        e1.record(stream)
        barrier()
        launches = ab.ahakv_launch_count() - launches0
        blocks.append(max_over_ranks(e0.elapsed_time(e1), world, dev))
    clocks = sampler.stop() if sampler else None
    status = ab.ahakv_last_device_status(ws)
    ms_total = statistics.median(blocks)
    ms_step = ms_total / args.steps
    # the same call repeated on one resident layer (inputs that fit in L2 stay there)
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        step(0)
    barrier()
    w0.record(stream)
    for _ in range(args.steps):
        step(0)
    w1.record(stream)
    barrier()
    warm_ms_step = max_over_ranks(w0.elapsed_time(w1), world, dev) / args.steps
    tokens_per_step = w.batch * w.n_ctx
    value = whole_job_value(tokens_per_step, world, ms_step)
    # the same K steps captured once in a CUDA graph and replayed: what the call costs without the host's launch
    # overhead (it matters for the small workloads, whose kernels are shorter than the gaps between them)
    graph_ms_step = None
    if world == 1:
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        outer = stream
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                stream = torch.cuda.current_stream()
                for i in range(args.steps):
                    step(i)
        stream = outer
        torch.cuda.synchronize()
        reps = []
        for _ in range(3):
            w0.record(side)
            with torch.cuda.stream(side):
                graph.replay()
            w1.record(side)
            torch.cuda.synchronize()
            reps.append(w0.elapsed_time(w1) / args.steps)
        graph_ms_step = statistics.median(reps)
        del graph

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
    traffic, traffic_source = measured_traffic(w)
    roofline = {"kernel": "score_tc_kernel (logits, SG-softmax, column sums, value norms): the dominant kernel alone; "
                          "the whole step against its roofline is path_roofline",
                "bound": "hbm", "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / pk["hbm_gbs"], "peak_source": f"{pk['source']} (sustained copy)",
                "traffic": traffic, "traffic_source": traffic_source,
                "algorithmic_bytes_per_launch": stage_bytes[dom], "ms_per_launch": stage_ms[dom],
                "slowest_stage": top}
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": n_warm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic", "config": workload_config(w, args, L),
        "repeats": len(blocks), "ms_per_step_min": min(blocks) / args.steps,
        "ms_per_step_max": max(blocks) / args.steps, "block_ms_per_step": [b_ / args.steps for b_ in blocks],
        "warm_ms_per_step": warm_ms_step,
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "device_status": int(status),
        "roofline": roofline,
        "path_roofline": {"t_roof_ms": t_roof_ms, "frac": t_roof_ms / ms_step, "algorithmic_bytes": work["bytes"],
                          "flops": work["flops"], "frac_vs_spec_8TBs": 1e3 * work["bytes"] / (SPEC_HBM_GBS * 1e9) / ms_step,
                          "of": pk["source"]},
        "ms_per_step_replayed_from_a_cuda_graph": graph_ms_step,
        "stage_ms": stage_ms,
        "stage_gbs": {s: stage_bytes[s] / (stage_ms[s] * 1e-3) / 1e9 for s in stage_bytes if stage_ms.get(s, 0) > 0},
        "tokens_per_step": tokens_per_step,
    }
    if w.name == "decode_round" and world == 1 and not args.no_protocol:
        del layers
        torch.cuda.empty_cache()
        out["decode_protocol"] = decode_protocol(ab, synth, w, dev, stream)
    if world == 1 and not args.no_cpu_baseline:
        _, _, info = cpu_oracle_sample(w)
        out["cpu_baseline"] = info
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def decode_protocol(ab, synth, w, dev, stream):
    """The decode configuration as a protocol: an untimed prefill eviction of a 32768-token cache down to the budget,
    then 256 generation steps.  (a) One eviction round every 32 steps with the last 32 queries as observation
    window, timed per round (8 rounds), with and without the value prior.  (b) Algorithm 1 as printed: evict at
    every step (one-row score update, selection, compaction in place), 256 steps timed."""
    import torch
    B, Hq, Hkv, d, Bud, Br, r = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.budget, w.recent_window, w.obs_window
    dtc = {"f32": ab.F32, "f16": ab.F16, "bf16": ab.BF16}[w.dtype]
    n0 = 32768
    pre = w.scaled(n_ctx=n0, n_total=None, value_prior=True)
    pp = ab.Params(B, Hq, Hkv, d, n0, r, Br, Bud, dtype=dtc, flags=ab.FLAG_VALUE_PRIOR)
    q, k, v = synth.make_layer(pre, layer=0, device=dev)
    ws = ab.alloc_workspace(pp, dev)
    k0, v0, f0, idx0 = ab.alloc_outputs(pp, dev)
    ab.ahakv_evict(pp, q, k, v, None, k0, v0, f0, idx0, ws, stream=stream)
    torch.cuda.synchronize()
    del q, k, v, ws
    torch.cuda.empty_cache()
    new = [synth.make_decode_step(w, t, device=dev) for t in range(256)]

    def rounds(flags):
        n = Bud + r
        kc = torch.empty((B, Hkv, n, d), dtype=k0.dtype, device=dev)
        vc = torch.empty_like(kc)
        fc = torch.zeros((B, Hkv, n), device=dev)
        kc[:, :, :Bud], vc[:, :, :Bud], fc[:, :, :Bud] = k0, v0, f0
        ko, vo, fo, io = ab.alloc_outputs(ab.Params(B, Hq, Hkv, d, n, r, Br, Bud, dtype=dtc), dev)
        ms = []
        for rd in range(8):
            steps = new[rd * r:(rd + 1) * r]
            qr = torch.cat([x[0] for x in steps], 2).contiguous()
            kc[:, :, Bud:] = torch.cat([x[1] for x in steps], 2)
            vc[:, :, Bud:] = torch.cat([x[2] for x in steps], 2)
            fc[:, :, Bud:] = 0.0
            p = ab.Params(B, Hq, Hkv, d, n, r, Br, Bud, dtype=dtc, n_total=n0 + (rd + 1) * r, flags=flags)
            wsr = ab.alloc_workspace(p, dev)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            ab.ahakv_evict(p, qr, kc, vc, fc, ko, vo, fo, io, wsr, stream=stream)
            e1.record(stream)
            torch.cuda.synchronize()
            assert ab.ahakv_last_device_status(wsr) == ab.OK
            ms.append(e0.elapsed_time(e1))
            kc[:, :, :Bud], vc[:, :, :Bud], fc[:, :, :Bud] = ko, vo, fo
        return ms

    plain = rounds(0)
    prior = rounds(ab.FLAG_VALUE_PRIOR)

    # evict at every step: the cache holds budget + 1 rows when scored
    n = Bud + 1
    kc = torch.empty((B, Hkv, n, d), dtype=k0.dtype, device=dev)
    vc = torch.empty_like(kc)
    fc = torch.zeros((B, Hkv, n), device=dev)
    kc[:, :, :Bud], vc[:, :, :Bud], fc[:, :, :Bud] = k0, v0, f0
    idx = torch.empty((B, Hkv, Bud), dtype=torch.int32, device=dev)
    ps = [ab.Params(B, Hq, Hkv, d, n, 1, Br, Bud, dtype=dtc, n_total=n0 + t + 1, flags=0) for t in range(256)]
    zero = torch.zeros((B, Hkv), device=dev)

    def one(t):
        qt, kt, vt = new[t]
        kc[:, :, Bud] = kt[:, :, 0]
        vc[:, :, Bud] = vt[:, :, 0]
        fc[:, :, Bud] = zero
        ab.ahakv_score_step(ps[t], qt, kc, fc, fc, stream=stream)
        ab.ahakv_select(ps[t], fc, idx, stream=stream)
        ab.ahakv_compact_inplace(ps[t], kc, vc, fc, idx, stream=stream)

    for t in range(8):
        one(t)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for t in range(256):
        one(t)
    e1.record(stream)
    torch.cuda.synchronize()
    per_step_ms = e0.elapsed_time(e1) / 256
    # the same 256 steps captured once in a CUDA graph and replayed: what is left when the host's launch overhead
    # is taken away
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    saved = stream
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            stream = torch.cuda.current_stream()
            for t in range(256):
                one(t)
    stream = saved
    torch.cuda.synchronize()
    replay_ms = []
    for _ in range(3):
        e0.record(side)
        with torch.cuda.stream(side):
            graph.replay()
        e1.record(side)
        torch.cuda.synchronize()
        replay_ms.append(e0.elapsed_time(e1) / 256)
    # the same steps on a cache kept as slots: one launch a step, no row moves (ahakv_step_slots)
    kc[:, :, :Bud], vc[:, :, :Bud], fc[:, :, :Bud] = k0, v0, f0
    pos = torch.full((B, Hkv, n), -1, dtype=torch.int32, device=dev)
    pos[:, :, :Bud] = idx0.to(torch.int32)
    free = torch.full((B, Hkv), Bud, dtype=torch.int32, device=dev)
    ab.ahakv_step_slots(ps[0], new[0][0], new[0][1], new[0][2], kc, vc, fc, pos, free, stream=stream)
    torch.cuda.synchronize()
    slot_graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(slot_graph, stream=side):
            for t in range(1, 256):
                ab.ahakv_step_slots(ps[t], new[t][0], new[t][1], new[t][2], kc, vc, fc, pos, free,
                                    stream=torch.cuda.current_stream())
    torch.cuda.synchronize()
    e0.record(side)
    with torch.cuda.stream(side):
        slot_graph.replay()
    e1.record(side)
    torch.cuda.synchronize()
    slots_ms = e0.elapsed_time(e1) / 255
    assert bool(((free >= 0) & (free <= Bud)).all()) and int((pos >= 0).sum()) == B * Hkv * Bud
    tokens = B * (Bud + r)
    return {
        "prefill": f"untimed eviction of {B} x {n0} tokens to {Bud} rows per KV head (value prior on)",
        "rounds_ms": plain, "rounds_ms_median": statistics.median(plain), "rounds_ms_min": min(plain),
        "rounds_tokens_per_s_median": tokens / (statistics.median(plain) * 1e-3),
        "rounds_value_prior_on_ms": prior, "rounds_value_prior_on_ms_median": statistics.median(prior),
        "evict_every_step": {"steps": 256, "ms_per_step": per_step_ms,
                             "includes": "appending the new token's rows (three small torch copies), ahakv_score_step, "
                                         "ahakv_select, ahakv_compact_inplace",
                             "tokens_per_s": B * n / (per_step_ms * 1e-3),
                             "ms_per_step_replayed_from_a_cuda_graph": min(replay_ms),
                             "ms_per_step_on_a_slot_cache": slots_ms,
                             "slot_cache": "ahakv_step_slots, one launch a step, 255 steps replayed from a CUDA graph; "
                                           "the new rows are copied in by the kernel"},
        "note": "each round allocates its workspace outside the timed region; inputs of a round were written just "
                "before it, so they may still be in L2 (the cache of one round is 136 MB against 126 MB of L2)",
    }


def run_widened(args):
    """Device times (CUDA events, median of 9 after 3 warm-ups) of the entry points beyond the eviction step, on
    synthetic inputs of the long-context shape cut to what each call is for.  One JSON line."""
    import statistics
    import torch
    from paper_2506_03762_b200 import binding as ab, synth
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    stream = torch.cuda.current_stream()

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ms = []
        for _ in range(9):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream); fn(); e1.record(stream); torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        return statistics.median(ms)

    out = {"widened": True, "data": "synthetic", "timing": "CUDA events, median of 9 calls after 3"}
    base = synth.WORKLOADS["long_32k"]

    # accumulation over every causal row (Eq. 2-3) at 8192 tokens: 64 passes of 128 rows
    w = base.scaled(batch=1, n_ctx=8192)
    q, k, v = synth.make_layer(w, layer=0, device=dev)
    q_all = torch.randn((w.batch, w.n_q_heads, w.n_ctx, w.head_dim), device=dev).to(k.dtype)
    p = ab.Params(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_ctx, w.obs_window, w.recent_window, w.budget,
                  dtype=ab.F16, flags=ab.FLAG_VALUE_PRIOR)
    ws = ab.alloc_workspace(p, dev)
    score = torch.empty((w.batch, w.n_kv_heads, w.n_ctx), dtype=torch.float32, device=dev)
    ms = timed(lambda: ab.ahakv_score_full_causal(p, q_all, k, v, None, score, ws, stream=stream))
    flops = 2.0 * w.batch * w.n_q_heads * w.head_dim * w.n_ctx * (w.n_ctx + 1) / 2 * 2     # two products, causal half
    out["score_full_causal"] = {"shape": f"1 x {w.n_q_heads} heads x {w.n_ctx} tokens, all rows", "ms": ms,
                                "passes": w.n_ctx // w.obs_window, "tflops_of_the_unmasked_part": flops / ms * 1e-9}
    del q_all

    # observation rows at scattered positions (the same kernels as ahakv_score)
    w = base.scaled(batch=2)
    q, k, v = synth.make_layer(w, layer=0, device=dev)
    p = ab.Params(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_ctx, w.obs_window, w.recent_window, w.budget,
                  dtype=ab.F16, flags=ab.FLAG_VALUE_PRIOR)
    ws = ab.alloc_workspace(p, dev)
    score = torch.empty((w.batch, w.n_kv_heads, w.n_ctx), dtype=torch.float32, device=dev)
    rows = sorted(range(w.n_ctx - 1, w.n_ctx - 1 - 256 * w.obs_window, -256))
    ms_rows = timed(lambda: ab.ahakv_score_rows(p, rows, q, k, v, None, score, ws, stream=stream))
    ms_plain = timed(lambda: ab.ahakv_score(p, q, k, v, None, score, ws, stream=stream))
    out["score_rows"] = {"shape": f"2 x {w.n_kv_heads} heads x {w.n_ctx} tokens, {w.obs_window} rows 256 apart", "ms": ms_rows,
                         "ahakv_score_same_shape_ms": ms_plain}
    # entropy of the observation rows (Eq. 6)
    ent = torch.empty((w.batch, w.n_q_heads, w.obs_window), dtype=torch.float32, device=dev)
    ms = timed(lambda: ab.ahakv_row_entropy(p, q, k, ent, stream=stream))
    kbytes = k.numel() * k.element_size()
    out["row_entropy"] = {"shape": out["score_rows"]["shape"].split(",")[0] + f", {w.obs_window} rows", "ms": ms,
                          "gbs_of_k": kbytes / ms * 1e-6}

    # a ragged batch: eight sequences of 2K .. 32K tokens, budgets a quarter of each
    lens = [2048, 4096, 6144, 8192, 12288, 16384, 24576, 32768]
    w = base.scaled(batch=len(lens))
    q, k, v = synth.make_layer(w, layer=1, device=dev)
    p = ab.Params(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_ctx, w.obs_window, w.recent_window, w.n_ctx // 4,
                  dtype=ab.F16, flags=ab.FLAG_VALUE_PRIOR)
    ws = ab.alloc_workspace(p, dev)
    k_out, v_out, s_out, idx = ab.alloc_outputs(p, dev)
    seqs = [(n, n // 4, n) for n in lens]
    ms = timed(lambda: ab.ahakv_evict_ragged(p, seqs, q, k, v, None, k_out, v_out, s_out, idx, ws, stream=stream))
    assert ab.ahakv_last_device_status(ws) == ab.OK
    tokens = sum(lens)
    alg = sum(2 * n * w.n_kv_heads * w.head_dim * 2 for n in lens) + sum(4 * (n // 4) * w.n_kv_heads * w.head_dim * 2 for n in lens)
    out["evict_ragged"] = {"shape": f"{len(lens)} sequences of {lens[0]} .. {lens[-1]} tokens, {w.n_kv_heads} heads", "ms": ms,
                           "tokens_per_s": tokens / ms * 1e3, "gbs_algorithmic": alg / ms * 1e-6,
                           "launch_sets": len(lens)}
    print(json.dumps(out))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.widened:
        run_widened(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
