"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import ahakv_oracle as orc
from paper_2506_03762_b200 import binding as ab
from paper_2506_03762_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu

DEV = "cuda"
TORCH_DT = {ab.F32: torch.float32, ab.F16: torch.float16, ab.BF16: torch.bfloat16}


def _rand_problem(B, Hq, Hkv, d, n, r, dtype, seed, spread=1.0):
    g = torch.Generator(device="cpu").manual_seed(seed)
    dt = TORCH_DT[dtype]
    q = (torch.randn((B, Hq, r, d), generator=g) * spread).to(dt).to(DEV)
    k = torch.randn((B, Hkv, n, d), generator=g).to(dt).to(DEV)
    v = (torch.randn((B, Hkv, n, d), generator=g) * (1 + torch.rand((B, Hkv, n, 1), generator=g))).to(dt).to(DEV)
    return q, k, v


# ---- the benchmark definition's configurations ---------------------------------------------------

def test_tiny_config_every_unit():
    w = synth.WORKLOADS["tiny"]
    p = parity.params_of(w)
    q, k, v = synth.make_layer(w, device=DEV)
    st = parity.check_units(p, q, k, v, parity.all_units(p))
    assert st["units"] == 4


def test_llama2_7b_4k_every_unit():
    w = synth.WORKLOADS["llama2_7b_4k"]
    p = parity.params_of(w)
    q, k, v = synth.make_layer(w, device=DEV)
    st = parity.check_units(p, q, k, v, parity.all_units(p))
    assert st["units"] == 32


def test_llama3_8b_gqa_16k_sampled_units():
    w = synth.WORKLOADS["llama3_8b_gqa_16k"]
    p = parity.params_of(w)
    q, k, v = synth.make_layer(w, device=DEV)
    parity.check_units(p, q, k, v, [(0, 0), (1, 3), (3, 7)])


def _spread_units(B, H, count, salt):
    """`count` distinct (sequence, head) pairs that touch every sequence and step through the heads."""
    return [((t * 3 + salt) % B, (t * 7 + 5 * salt + t // B) % H) for t in range(count)]


@pytest.mark.parametrize("layer,count", [(0, 32), (31, 32), (11, 16), (22, 16)])
def test_long_32k_full_size_sampled_units(layer, count):
    """The launch configuration the benchmark times (one layer of 8 x 32 heads x 32768 tokens).  The oracle
    recomputes sampled (sequence, head) units: thirty-two of the first and of the last layer, sixteen of two layers in
    between (about 1.5 s of double-precision loops each, one host thread a unit).  Every head of the same launch
    is held to the properties that need no oracle: kept indices ascending with the recent window at the tail,
    and, with the value prior off, softmax mass r."""
    import os
    w = synth.WORKLOADS["long_32k"]
    p = parity.params_of(w)
    units = _spread_units(w.batch, w.n_kv_heads, count, layer)
    assert len(set(units)) == count
    q, k, v = synth.make_layer(w, layer=layer, device=DEV)
    st = parity.check_units(p, q, k, v, units, workers=len(os.sched_getaffinity(0)))
    assert st["units"] == count
    idx = st["outputs"][4]
    raw = parity.run_score(parity.params_of(w, flags=0), q, k, v)
    parity.assert_every_head_valid(p, idx, raw)


def test_decode_round_with_carried_score():
    w = synth.WORKLOADS["decode_round"]
    p = parity.params_of(w)
    q, k, v = synth.make_layer(w, device=DEV)
    prev = synth.make_score_prev(w, device=DEV, new_rows=w.obs_window)
    parity.check_units(p, q, k, v, [(0, 0), (5, 2), (15, 7)], score_prev=prev)
    # the same shape with the value prior on (exercises the V stream at this size)
    p2 = parity.params_of(w, flags=ab.FLAG_VALUE_PRIOR)
    parity.check_units(p2, q, k, v, [(9, 4)], score_prev=prev)


def test_decode_rounds_chain_through_the_compacted_cache():
    """Two rounds: the second scores the first round's compacted cache plus new tokens, with the
    carried score_out as score_prev (zeros for the new rows)."""
    w = synth.WORKLOADS["decode_round"].scaled(batch=2)
    p = parity.params_of(w)
    q, k, v = synth.make_layer(w, device=DEV)
    prev = synth.make_score_prev(w, device=DEV, new_rows=w.obs_window)
    k1, v1, s1, _ = parity.run_evict(p, q, k, v, prev)
    new = [synth.make_decode_step(w, t, device=DEV) for t in range(w.obs_window)]
    q2 = torch.cat([x[0] for x in new], 2).contiguous()
    k2 = torch.cat([k1] + [x[1] for x in new], 2).contiguous()
    v2 = torch.cat([v1] + [x[2] for x in new], 2).contiguous()
    prev2 = torch.cat([s1, torch.zeros((w.batch, w.n_kv_heads, w.obs_window), device=DEV)], 2).contiguous()
    p2 = parity.params_of(w, n_total=w.n_total + w.obs_window)
    assert k2.shape[2] == p2.n_ctx
    parity.check_units(p2, q2, k2, v2, [(0, 0), (1, 5)], score_prev=prev2)


def test_per_step_generation_update_chains_to_the_batched_round():
    """Algorithm 1's generation phase one token at a time: F_t = SGsoftmax(A_t) + F_{t-1}, each step a call with
    one observation row, the grown cache and the carried score (0 for the new row).  After T steps the score
    must equal one call with T observation rows over the final cache, and the oracle's."""
    B, Hq, Hkv, d, n0, T, N0 = 2, 8, 2, 128, 1500, 8, 20000
    g = torch.Generator(device="cpu").manual_seed(77)
    k_all = torch.randn((B, Hkv, n0 + T, d), generator=g).to(torch.bfloat16).to(DEV)
    q_all = torch.randn((B, Hq, T, d), generator=g).to(torch.bfloat16).to(DEV)
    v_all = torch.randn((B, Hkv, n0 + T, d), generator=g).to(torch.bfloat16).to(DEV)    # not read: no value prior here
    f = (torch.rand((B, Hkv, n0), generator=g) * 0.01).to(DEV)
    f0 = f.clone()
    for t in range(T):
        n = n0 + t + 1
        p = ab.Params(B, Hq, Hkv, d, n, 1, 16, 512, dtype=ab.BF16, n_total=N0 + t + 1, flags=0)
        prev = torch.cat([f, torch.zeros((B, Hkv, 1), device=DEV)], 2).contiguous()
        f = parity.run_score(p, q_all[:, :, t:t + 1].contiguous(), k_all[:, :, :n].contiguous(),
                             v_all[:, :, :n].contiguous(), prev)
    n = n0 + T
    pT = ab.Params(B, Hq, Hkv, d, n, T, 16, 512, dtype=ab.BF16, n_total=N0 + T, flags=0)
    prevT = torch.cat([f0, torch.zeros((B, Hkv, T), device=DEV)], 2).contiguous()
    batched = parity.run_score(pT, q_all, k_all, v_all, prevT)
    parity.assert_scores_close(pT, f.cpu().numpy(), batched.cpu().numpy(), "chained vs batched")
    for b, h in [(0, 0), (1, 1)]:
        op, qn, kn, vn, sp = parity.unit_inputs(pT, q_all, k_all, v_all, b, h, prevT)
        ref = orc.evict(op, qn, kn, vn, sp)
        parity.assert_scores_close(pT, f[b, h].cpu().numpy(), ref["score"][0, 0], "chained vs oracle")


# ---- small shapes: tiles, ragged tails, degenerate cases ---------------------------------------------

EDGE_CASES = [
    # B, Hq, Hkv, d,   n,   r,  Br, Bud, dtype,  extra
    (1, 2, 2, 64, 300, 16, 16, 64, ab.F32, {}),
    (2, 4, 1, 128, 517, 24, 8, 100, ab.F16, {}),                           # G = 4, ragged tail, r % 16 != 0
    (1, 8, 1, 64, 700, 32, 32, 256, ab.BF16, {}),                          # G = 8
    (1, 1, 1, 128, 129, 1, 1, 128, ab.F16, {}),                            # n = Bud + 1, r = 1
    (1, 2, 2, 128, 96, 8, 4, 128, ab.F16, {}),                             # n <= Bud: keep everything
    (1, 2, 2, 128, 128, 8, 4, 128, ab.BF16, {}),                           # n == Bud
    (1, 2, 1, 64, 400, 37, 0, 50, ab.F16, {}),                             # B_r = 0
    (1, 2, 1, 64, 400, 20, 50, 50, ab.BF16, {}),                           # B_s = 0
    (1, 2, 2, 128, 1000, 48, 16, 200, ab.F16, dict(pool_kernel=1)),
    (1, 2, 2, 128, 1000, 48, 16, 200, ab.F16, dict(pool_kernel=31, flags=ab.FLAG_VALUE_PRIOR | ab.FLAG_POOL_ZERO_PAD)),
    (1, 2, 2, 128, 1000, 48, 16, 200, ab.BF16, dict(flags=0)),
    (1, 1, 1, 128, 2000, 200, 64, 400, ab.F16, {}),                        # r > 128: two row blocks
    (1, 1, 1, 64, 2000, 256, 64, 400, ab.F32, {}),                         # r at its maximum
    (1, 4, 2, 128, 1500, 64, 32, 300, ab.F16, dict(scale_mode=ab.SCALE_FIXED, scale=128 ** -0.5)),
    (1, 4, 2, 128, 1500, 64, 32, 300, ab.BF16, dict(scale_mode=ab.SCALE_ADAPTIVE_CALL, n_total=9000)),
    (1, 4, 2, 128, 1500, 64, 32, 300, ab.F16, dict(n_total=1501)),        # Eq. 12 barely inside its domain
    (3, 6, 2, 64, 260, 40, 10, 77, ab.F32, dict(n_total=100000)),         # G = 3: rows do not fill a block
    (1, 1, 1, 128, 64, 64, 8, 32, ab.F16, {}),                             # r == n: every row is causal
    (1, 1, 1, 64, 1, 1, 1, 1, ab.F32, {}),                                 # a single token
    (1, 2, 1, 64, 33500, 16, 32, 600, ab.F16, {}),                        # more scores per head than one CTA's registers hold
    (1, 2, 2, 128, 128 * 23 + 5, 40, 16, 300, ab.BF16, {}),                # odd run lengths, three row-block-sized heads
    (1, 2, 1, 64, 4097, 16, 32, 500, ab.F16, {}),                          # fused refine+select: 8 tokens a thread, barely
    (1, 1, 1, 64, 8192, 16, 32, 900, ab.BF16, {}),                         # ... 8 tokens a thread, exactly
    (1, 1, 1, 64, 8193, 16, 32, 900, ab.F16, {}),                          # ... 16 tokens a thread, barely
    # value norms staged in 40 to 48 KB of dynamic shared memory next to the kernel's static arrays
    (1, 1, 1, 64, 10133, 16, 32, 900, ab.F16, {}),
    (1, 2, 1, 64, 11000, 16, 32, 900, ab.BF16, {}),
    (1, 1, 1, 64, 12288, 16, 32, 900, ab.F16, {}),
    (1, 1, 1, 64, 12288, 16, 32, 900, ab.BF16, dict(n_total=40000)),
    # grouped query heads pooled by maximum instead of mean
    (1, 8, 2, 128, 1500, 32, 16, 300, ab.F16, dict(flags=ab.FLAG_VALUE_PRIOR | ab.FLAG_GROUP_MAX)),
    (2, 8, 2, 128, 700, 64, 16, 200, ab.BF16, dict(flags=ab.FLAG_GROUP_MAX)),
    (1, 6, 2, 64, 400, 20, 8, 100, ab.F32, dict(flags=ab.FLAG_VALUE_PRIOR | ab.FLAG_GROUP_MAX)),
    (1, 2, 2, 128, 600, 200, 16, 150, ab.F16, dict(flags=ab.FLAG_GROUP_MAX)),     # one head a group: same as the mean
    # query heads that do not fill the last row block of their KV head
    (1, 7, 1, 128, 1300, 32, 32, 300, ab.BF16, {}),                        # G = 7, r = 32: blocks of 4 + 3 heads
    (2, 14, 2, 128, 1300, 32, 32, 300, ab.F16, {}),
    (1, 5, 1, 64, 900, 48, 16, 200, ab.F16, {}),                           # G = 5, r = 48: blocks of 2 + 2 + 1 heads
    (1, 3, 1, 128, 700, 80, 16, 200, ab.BF16, {}),                         # one head a block, 80 of 128 rows live
]


@pytest.mark.parametrize("case", EDGE_CASES, ids=lambda c: f"B{c[0]}Hq{c[1]}Hkv{c[2]}d{c[3]}n{c[4]}r{c[5]}Br{c[6]}Bud{c[7]}t{c[8]}")
def test_edge_shapes(case):
    B, Hq, Hkv, d, n, r, Br, Bud, dtype, extra = case
    p = ab.Params(B, Hq, Hkv, d, n, r, Br, Bud, dtype=dtype, **extra)
    q, k, v = _rand_problem(B, Hq, Hkv, d, n, r, dtype, seed=n * 7 + r)
    parity.check_units(p, q, k, v, parity.all_units(p))


@pytest.mark.parametrize("Hq,r", [(7, 32), (5, 48), (28, 32)])
def test_uneven_head_groups_take_the_tensor_core_path(Hq, r):
    """Grouped queries whose heads do not fill the last 128-row block of their KV head (Qwen2-7B, the model of
    the paper's Appendix E, has 28 query heads on 4 KV heads) must not fall back to the FP32-pipe kernels: an
    eviction call is then three launches (scoring, refine+select, compact), not six."""
    Hkv = 1 if Hq < 28 else 4
    p = ab.Params(1, Hq, Hkv, 128, 2000, r, 32, 400, dtype=ab.BF16)
    q, k, v = _rand_problem(1, Hq, Hkv, 128, 2000, r, ab.BF16, seed=Hq * 100 + r)
    before = ab.ahakv_launch_count()
    parity.run_evict(p, q, k, v)
    assert ab.ahakv_launch_count() - before == 3
    parity.check_units(p, q, k, v, parity.all_units(p))


def test_peaked_attention_large_logits():
    """Queries 6x larger: logits reach the hundreds, single keys take almost all the mass."""
    B, Hq, Hkv, d, n, r = 1, 2, 2, 128, 900, 32
    # float32 inputs hold 1e-5 here too: their logits are formed, scaled and shifted in double
    for dtype, spread in ((ab.F16, 6.0), (ab.BF16, 6.0), (ab.F32, 6.0)):
        p = ab.Params(B, Hq, Hkv, d, n, r, 16, 100, dtype=dtype, n_total=50000)
        q, k, v = _rand_problem(B, Hq, Hkv, d, n, r, dtype, seed=5, spread=spread)
        parity.check_units(p, q, k, v, parity.all_units(p))


def test_strided_cache_layout():
    """K and V stored [B, n, Hkv, d] (token-major) and Q_obs stored [B, r, Hq, d]: same result as dense."""
    B, Hq, Hkv, d, n, r = 2, 4, 2, 128, 640, 32
    p = ab.Params(B, Hq, Hkv, d, n, r, 16, 128, dtype=ab.F16)
    q, k, v = _rand_problem(B, Hq, Hkv, d, n, r, ab.F16, seed=11)
    dense = parity.run_evict(p, q, k, v)
    qs = q.permute(0, 2, 1, 3).contiguous()      # storage [B, r, Hq, d]
    ks = k.permute(0, 2, 1, 3).contiguous()      # storage [B, n, Hkv, d]
    vs = v.permute(0, 2, 1, 3).contiguous()
    ps = ab.Params(B, Hq, Hkv, d, n, r, 16, 128, dtype=ab.F16,
                   q_stride=(r * Hq * d, d, Hq * d), k_stride=(n * Hkv * d, d, Hkv * d),
                   v_stride=(n * Hkv * d, d, Hkv * d))
    strided = parity.run_evict(ps, qs, ks, vs)
    for a, b in zip(dense, strided):
        assert torch.equal(a, b)


@pytest.mark.parametrize("name,over", [("llama2_7b_4k", {}), ("decode_round", dict(batch=8)),
                                       ("llama3_8b_gqa_16k", dict(batch=1, n_ctx=128 * 37 + 11))])
def test_runs_are_bitwise_reproducible(name, over):
    """Runs are handed to the CTAs in whatever order they come free; the result must not depend on it."""
    w = synth.WORKLOADS[name].scaled(**over)
    p = parity.params_of(w)
    q, k, v = synth.make_layer(w, device=DEV)
    prev = synth.make_score_prev(w, device=DEV, new_rows=w.obs_window) if w.n_total is not None else None
    first = parity.run_evict(p, q, k, v, prev)
    score = parity.run_score(p, q, k, v, prev)
    for _ in range(3):
        again = parity.run_evict(p, q, k, v, prev)
        for a, b in zip(first, again):
            assert torch.equal(a, b)
        assert torch.equal(parity.run_score(p, q, k, v, prev), score)


# ---- the separate entry points ----------------------------------------------------------------------------

@pytest.mark.parametrize("n,Br,Bud", [(5000, 64, 512), (32768, 128, 2048), (70000, 0, 4096), (1025, 1024, 1024), (300, 10, 299)])
def test_select_is_bit_exact_including_ties(n, Br, Bud):
    B, H = 2, 3
    g = torch.Generator(device="cpu").manual_seed(n)
    s = torch.rand((B, H, n), generator=g)
    s[0] = torch.round(s[0] * 50) / 50                     # heavy ties
    s[1, 0] = 0.25                                         # all equal: lowest indices win
    s[1, 1, ::3] *= -1                                     # negative scores order correctly too
    p = ab.Params(B, H, H, 128, n, 8, Br, Bud, dtype=ab.F16)
    ws = ab.alloc_workspace(p, DEV)
    idx = torch.empty((B, H, p.n_keep), dtype=torch.int32, device=DEV)
    ab.ahakv_select(p, s.to(DEV), idx, ws)
    ref = orc.select(parity.oracle_params(p), s.double().numpy())
    assert np.array_equal(idx.cpu().numpy(), ref)


@pytest.mark.parametrize("dtype,d", [(ab.F32, 64), (ab.F16, 128), (ab.BF16, 64), (ab.F32, 128)])
def test_compact_is_a_byte_copy(dtype, d):
    B, H, n, Bud = 2, 3, 777, 200
    p = ab.Params(B, H, H, d, n, 8, 16, Bud, dtype=dtype)
    g = torch.Generator(device="cpu").manual_seed(d)
    k = torch.randn((B, H, n, d), generator=g).to(TORCH_DT[dtype]).to(DEV)
    v = torch.randn((B, H, n, d), generator=g).to(TORCH_DT[dtype]).to(DEV)
    s = torch.rand((B, H, n), generator=g).to(DEV)
    idx = torch.stack([torch.randperm(n, generator=g)[:Bud].sort().values for _ in range(B * H)])
    idx = idx.view(B, H, Bud).to(torch.int32).to(DEV)
    k_out, v_out, s_out, _ = ab.alloc_outputs(p, DEV)
    ab.ahakv_compact(p, k, v, s, idx, k_out, v_out, s_out)
    ko, vo, so = orc.compact(parity.oracle_params(p), synth.to_numpy(k), synth.to_numpy(v),
                             idx.cpu().numpy(), s.double().cpu().numpy())
    assert synth.to_numpy(k_out).tobytes() == ko.tobytes()
    assert synth.to_numpy(v_out).tobytes() == vo.tobytes()
    assert np.array_equal(s_out.cpu().numpy().astype(np.float64), so)
    # without the score
    k2, v2, _, _ = ab.alloc_outputs(p, DEV)
    ab.ahakv_compact(p, k, v, None, idx, k2, v2, None)
    assert torch.equal(k2, k_out) and torch.equal(v2, v_out)


def test_score_mass_invariant_at_full_size():
    """Property that holds at any size: without the value prior, sum_j S_j = r for every KV head."""
    w = synth.WORKLOADS["llama3_8b_gqa_16k"]
    p = parity.params_of(w, flags=0)
    q, k, v = synth.make_layer(w, device=DEV)
    s = parity.run_score(p, q, k, v)
    total = s.double().sum(-1)
    assert torch.allclose(total, torch.full_like(total, float(w.obs_window)), rtol=2e-4)
    assert (s >= 0).all()


def test_wrong_device_arguments_leave_outputs_untouched():
    p = ab.Params(1, 2, 2, 128, 500, 16, 8, 64, dtype=ab.F16)
    q, k, v = _rand_problem(1, 2, 2, 128, 500, 16, ab.F16, seed=3)
    ws = ab.alloc_workspace(p, DEV)
    k_out, v_out, s_out, idx = ab.alloc_outputs(p, DEV)
    idx.fill_(-7)
    small = ws[: ws.numel() // 2]
    assert ab.ahakv_evict(p, q, k, v, None, k_out, v_out, s_out, idx, small, check=False) == ab.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert (idx == -7).all()
    assert ab.ahakv_launch_count() >= 0


def test_the_eviction_call_replays_from_a_cuda_graph():
    """ahakv_evict (two memsets, the cooperative scoring kernel, selection, compaction) captured once and replayed:
    the same kept indices, rows and scores as the eager call, and a clean device status."""
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    B, Hq, Hkv, d, n, r, Br, Bud = 2, 8, 4, 128, 3000, 32, 32, 512
    g = torch.Generator().manual_seed(99)
    q = torch.randn((B, Hq, r, d), generator=g).to(torch.float16).cuda()
    k = torch.randn((B, Hkv, n, d), generator=g).to(torch.float16).cuda()
    v = torch.randn((B, Hkv, n, d), generator=g).to(torch.float16).cuda()
    p = ab.Params(B, Hq, Hkv, d, n, r, Br, Bud, dtype=ab.F16)
    eager = parity.run_evict(p, q, k, v, None)
    ws = ab.alloc_workspace(p, "cuda")
    outs = ab.alloc_outputs(p, "cuda")
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            ab.ahakv_evict(p, q, k, v, None, *outs, ws, stream=torch.cuda.current_stream())
    torch.cuda.synchronize()
    for _ in range(2):
        for t in outs:
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert ab.ahakv_last_device_status(ws) == ab.OK
        for a, c in zip(eager, outs):
            assert torch.equal(a, c)
