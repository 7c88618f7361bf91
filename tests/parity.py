"""Comparison rules between the CUDA path and the CPU oracle.

* scores: |gpu - ref| <= rtol * |ref| + atol with rtol = 1e-3 for 16-bit inputs and 1e-5 for
  float32, atol = rtol * 1e-3 * (r / n)  (r / n is the mean score, so atol sits six orders below it);
* kept indices: both sides hold exactly n_keep ascending indices containing the recent window; every
  index on which they differ must have an oracle score within rtol of the oracle's threshold (the
  B_s-th largest candidate score);
* compaction: given the GPU's own indices, K/V rows must be byte-identical to the oracle's gather.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import ahakv_oracle as orc
from paper_2506_03762_b200 import binding as ab
from paper_2506_03762_b200 import synth

RTOL = {ab.F32: 1e-5, ab.F16: 1e-3, ab.BF16: 1e-3}


def oracle_params(p: ab.Params, batch=None, n_q_heads=None, n_kv_heads=None) -> orc.OracleParams:
    return orc.OracleParams(
        p.batch if batch is None else batch, p.n_q_heads if n_q_heads is None else n_q_heads,
        p.n_kv_heads if n_kv_heads is None else n_kv_heads, p.head_dim, p.n_ctx, p.obs_window,
        p.recent_window, p.budget, dtype=p.dtype, n_total=p.n_total, scale_mode=p.scale_mode,
        scale=p.scale, pool_kernel=p.pool_kernel, flags=p.flags)


def unit_inputs(p: ab.Params, q, k, v, b: int, h: int, score_prev=None):
    """Dense host copies of one (sequence, KV head) unit as a B=1, Hkv=1, Hq=G problem."""
    G = p.n_q_heads // p.n_kv_heads
    qn = synth.to_numpy(q[b:b + 1, h * G:(h + 1) * G])
    kn = synth.to_numpy(k[b:b + 1, h:h + 1])
    vn = synth.to_numpy(v[b:b + 1, h:h + 1])
    sp = None if score_prev is None else score_prev[b:b + 1, h:h + 1].double().cpu().numpy()
    return oracle_params(p, batch=1, n_q_heads=G, n_kv_heads=1), qn, kn, vn, sp


def score_tolerance(p: ab.Params):
    rtol = RTOL[p.dtype]
    return rtol, rtol * 1e-3 * p.obs_window / p.n_ctx


def assert_scores_close(p: ab.Params, got: np.ndarray, ref: np.ndarray, what="score"):
    rtol, atol = score_tolerance(p)
    got = np.asarray(got, np.float64)
    err = np.abs(got - ref)
    bound = rtol * np.abs(ref) + atol
    worst = np.argmax(err - bound)
    assert (err <= bound).all(), (
        f"{what}: {int((err > bound).sum())} of {err.size} outside tolerance; worst at flat index {worst}: "
        f"gpu {got.flat[worst]!r} ref {ref.flat[worst]!r} rel {err.flat[worst] / max(abs(ref.flat[worst]), 1e-300):.3e}")
    return float((err / np.maximum(np.abs(ref), atol / rtol)).max())


def assert_kept_valid(p: ab.Params, got_idx: np.ndarray, ref_idx: np.ndarray, ref_score: np.ndarray):
    """got_idx, ref_idx [n_keep]; ref_score [n] (the oracle's refined score of the same unit)."""
    n, Br, Bud = p.n_ctx, p.recent_window, p.budget
    n_keep = min(n, Bud)
    assert got_idx.shape == (n_keep,) and (np.diff(got_idx) > 0).all(), "indices must be strictly ascending"
    assert got_idx.min() >= 0 and got_idx.max() < n
    if n <= Bud:
        assert np.array_equal(got_idx, np.arange(n))
        return 0
    assert np.array_equal(got_idx[Bud - Br:], np.arange(n - Br, n)), "recent window must be kept"
    diff = np.setxor1d(got_idx, ref_idx)
    if diff.size:
        Bs = Bud - Br
        tau = np.sort(ref_score[: n - Br])[::-1][Bs - 1]
        rtol, atol = score_tolerance(p)
        bad = diff[np.abs(ref_score[diff] - tau) > rtol * abs(tau) + atol]
        assert bad.size == 0, f"{bad.size} index disagreements outside the tolerance band, e.g. {bad[:8]}"
    return int(diff.size)


def run_evict(p: ab.Params, q, k, v, score_prev=None):
    """Fused ahakv_evict on device tensors; returns device outputs + the status word."""
    ws = ab.alloc_workspace(p, q.device)
    k_out, v_out, s_out, idx = ab.alloc_outputs(p, q.device)
    ab.ahakv_evict(p, q, k, v, score_prev, k_out, v_out, s_out, idx, ws)
    assert ab.ahakv_last_device_status(ws) == ab.OK
    return k_out, v_out, s_out, idx


def run_score(p: ab.Params, q, k, v, score_prev=None):
    ws = ab.alloc_workspace(p, q.device)
    score = torch.empty((p.batch, p.n_kv_heads, p.n_ctx), dtype=torch.float32, device=q.device)
    ab.ahakv_score(p, q, k, v, score_prev, score, ws)
    assert ab.ahakv_last_device_status(ws) == ab.OK
    return score


def oracle_units(p: ab.Params, q, k, v, units, score_prev=None, workers: int = 1):
    """The oracle's eviction of each listed (b, h) unit, `workers` units at a time (one host thread each; the
    oracle call releases the interpreter lock).  Yields (b, h, inputs, result) in the order given."""
    units = list(units)

    def one(bh):
        inp = unit_inputs(p, q, k, v, bh[0], bh[1], score_prev)
        return inp, orc.evict(*inp, nthreads=1)

    if workers <= 1:
        for bh in units:
            inp, ref = one(bh)
            yield bh[0], bh[1], inp, ref
        return
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=workers) as ex:
        for bh, (inp, ref) in zip(units, ex.map(one, units)):
            yield bh[0], bh[1], inp, ref


def check_units(p: ab.Params, q, k, v, units, score_prev=None, workers: int = 1):
    """Fused evict + separate score on the GPU, compared with the oracle on the listed (b, h) units."""
    score = run_score(p, q, k, v, score_prev)
    k_out, v_out, s_out, idx = run_evict(p, q, k, v, score_prev)
    stats = dict(max_rel=0.0, idx_diffs=0, units=0)
    for b, h, (op, qn, kn, vn, sp), ref in oracle_units(p, q, k, v, units, score_prev, workers):
        stats["max_rel"] = max(stats["max_rel"],
                               assert_scores_close(p, score[b, h].cpu().numpy(), ref["score"][0, 0]))
        gi = idx[b, h].cpu().numpy()
        stats["idx_diffs"] += assert_kept_valid(p, gi, ref["kept_idx"][0, 0], ref["score"][0, 0])
        # compaction of the GPU's own indices must be a byte copy
        ko, vo, so = orc.compact(op, kn, vn, gi.reshape(1, 1, -1), ref["score"])
        assert synth.to_numpy(k_out[b:b + 1, h:h + 1]).tobytes() == ko.tobytes(), "K_out is not a byte copy"
        assert synth.to_numpy(v_out[b:b + 1, h:h + 1]).tobytes() == vo.tobytes(), "V_out is not a byte copy"
        # carried score: the fused path's score rows equal the separate score call's rows, bit for bit
        assert torch.equal(s_out[b, h], score[b, h][idx[b, h].long()])
        assert_scores_close(p, s_out[b, h].cpu().numpy(), so[0, 0], "score_out")
        stats["units"] += 1
    stats["outputs"] = (score, k_out, v_out, s_out, idx)
    return stats


def assert_every_head_valid(p: ab.Params, idx, score_no_prior=None):
    """Properties that hold at any size, checked on the device for every (sequence, KV head) of a launch:
    kept indices strictly ascending, in range, exactly n_keep of them, recent window at the tail; and, for a
    score computed without the value prior and without a carried score, sum_j S_j = r (each of the r softmax
    rows carries mass 1; the mean over a group's query heads keeps it)."""
    n, Br, n_keep = p.n_ctx, p.recent_window, p.n_keep
    assert idx.shape == (p.batch, p.n_kv_heads, n_keep)
    i64 = idx.long()
    assert bool((i64[..., 1:] > i64[..., :-1]).all()), "kept indices must be strictly ascending in every head"
    assert int(i64.min()) >= 0 and int(i64.max()) < n
    if n > p.budget and Br > 0:
        want = torch.arange(n - Br, n, device=idx.device).expand(p.batch, p.n_kv_heads, Br)
        assert torch.equal(i64[..., n_keep - Br:], want), "recent window must close every head's kept list"
    if score_no_prior is not None:
        total = score_no_prior.double().sum(-1)
        assert bool((score_no_prior >= 0).all())
        assert torch.allclose(total, torch.full_like(total, float(p.obs_window)), rtol=2e-4), \
            f"softmax mass: min {float(total.min())} max {float(total.max())} want {p.obs_window}"


def all_units(p: ab.Params):
    return [(b, h) for b in range(p.batch) for h in range(p.n_kv_heads)]


def params_of(w: synth.Workload, **kw) -> ab.Params:
    flags = ab.FLAG_VALUE_PRIOR if w.value_prior else 0
    base = dict(dtype={"f32": ab.F32, "f16": ab.F16, "bf16": ab.BF16}[w.dtype], n_total=w.n_total,
                pool_kernel=w.pool_kernel, flags=flags)
    base.update(kw)
    return ab.Params(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_ctx, w.obs_window,
                     w.recent_window, w.budget, **base)
