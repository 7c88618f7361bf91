"""Algorithm 1's generation phase one token at a time on the GPU: the 1 x n score update (``ahakv_score_step``),
selection, and compaction in place (``ahakv_compact_inplace``), chained for many steps and checked against the
oracle step by step."""
import numpy as np
import pytest
import torch

from oracle import ahakv_oracle as orc
from paper_2506_03762_b200 import synth

pytestmark = pytest.mark.gpu

DEV = "cuda"


def _dt(ab, dtype):
    return {ab.F32: torch.float32, ab.F16: torch.float16, ab.BF16: torch.bfloat16}[dtype]


@pytest.mark.parametrize("B,Hq,Hkv,d,n,dtype_name,flags", [
    (2, 8, 2, 128, 2049, "BF16", 0),           # the shape of a cache held at its budget, grouped queries
    (1, 4, 4, 128, 700, "F16", 0),
    (1, 6, 2, 64, 300, "F32", 0),              # three query heads a group, float32 at 1e-5
    (3, 7, 1, 64, 515, "F16", 4),              # seven heads a group pooled by maximum
    (1, 1, 1, 128, 1, "F16", 0),               # a single cached token
    (1, 12, 1, 128, 1003, "BF16", 0),          # twelve heads a group: both halves of the 16-row product
    (2, 16, 1, 64, 2044, "F16", 0),            # sixteen heads, 64-wide rows, a ragged last block of keys
    (1, 16, 2, 64, 333, "BF16", 4),            # eight heads a group pooled by maximum
])
def test_score_step_matches_the_oracle_and_the_general_path(B, Hq, Hkv, d, n, dtype_name, flags):
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    dtype = getattr(ab, dtype_name)
    g = torch.Generator().manual_seed(n)
    q = torch.randn((B, Hq, 1, d), generator=g).to(_dt(ab, dtype)).to(DEV)
    k = torch.randn((B, Hkv, n, d), generator=g).to(_dt(ab, dtype)).to(DEV)
    prev = (torch.rand((B, Hkv, n), generator=g) * 0.01).to(DEV)
    p = ab.Params(B, Hq, Hkv, d, n, 1, min(16, n), max(1, n // 2), dtype=dtype, n_total=40000 + n, flags=flags)
    got = torch.empty((B, Hkv, n), dtype=torch.float32, device=DEV)
    ab.ahakv_score_step(p, q, k, prev, got)
    op = parity.oracle_params(p)
    ref = orc.score(op, synth.to_numpy(q), synth.to_numpy(k), synth.to_numpy(k), prev.double().cpu().numpy())
    parity.assert_scores_close(p, got.cpu().numpy(), ref, "score_step")
    general = parity.run_score(p, q, k, k, prev)
    parity.assert_scores_close(p, got.cpu().numpy(), general.double().cpu().numpy(), "score_step vs ahakv_score")
    # in place: score_prev and score the same buffer
    buf = prev.clone()
    ab.ahakv_score_step(p, q, k, buf, buf)
    assert torch.equal(buf, got)


def test_score_step_declines_what_it_does_not_take():
    from paper_2506_03762_b200 import binding as ab
    q = torch.zeros((1, 4, 1, 128), dtype=torch.float16, device=DEV)
    k = torch.zeros((1, 4, 64, 128), dtype=torch.float16, device=DEV)
    s = torch.zeros((1, 4, 64), device=DEV)
    assert ab.ahakv_score_step(ab.Params(1, 4, 4, 128, 64, 1, 4, 8, flags=ab.FLAG_VALUE_PRIOR), q, k, None, s,
                               check=False) == ab.ERR_UNSUPPORTED
    assert ab.ahakv_score_step(ab.Params(1, 4, 4, 128, 64, 2, 4, 8, flags=0), q, k, None, s,
                               check=False) == ab.ERR_INVALID_ARG
    assert ab.ahakv_score_step(ab.Params(1, 4, 4, 128, 50000, 1, 4, 8, flags=0), 256, 256, None, 256,
                               check=False) == ab.ERR_UNSUPPORTED          # 50000 logits do not fit in shared memory


@pytest.mark.parametrize("dtype_name,d,first_evicted", [("F16", 128, 0), ("BF16", 64, 700), ("F32", 128, 1023), ("F16", 128, None)])
def test_compact_inplace_equals_the_gather(dtype_name, d, first_evicted):
    from paper_2506_03762_b200 import binding as ab
    dtype = getattr(ab, dtype_name)
    B, H, n, Bud = 2, 3, 1100, 1024
    g = torch.Generator().manual_seed(d)
    k = torch.randn((B, H, n, d), generator=g).to(_dt(ab, dtype)).to(DEV)
    v = torch.randn((B, H, n, d), generator=g).to(_dt(ab, dtype)).to(DEV)
    s = torch.rand((B, H, n), generator=g).to(DEV)
    idx = []
    for u in range(B * H):
        if first_evicted is None:                                  # nothing among the first Bud rows is evicted
            keep = torch.arange(Bud)
        else:
            tail = first_evicted + torch.randperm(n - first_evicted, generator=g)[: Bud - first_evicted].sort().values
            keep = torch.cat([torch.arange(first_evicted), tail])
        idx.append(keep)
    idx = torch.stack(idx).view(B, H, Bud).to(torch.int32).to(DEV)
    p = ab.Params(B, H, H, d, n, 8, 16, Bud, dtype=dtype)
    k_out, v_out, s_out, _ = ab.alloc_outputs(p, DEV)
    ab.ahakv_compact(p, k, v, s, idx, k_out, v_out, s_out)
    k2, v2, s2 = k.clone(), v.clone(), s.clone()
    ab.ahakv_compact_inplace(p, k2, v2, s2, idx)
    assert torch.equal(k2[:, :, :Bud], k_out) and torch.equal(v2[:, :, :Bud], v_out) and torch.equal(s2[:, :, :Bud], s_out)
    assert torch.equal(k2[:, :, Bud:], k[:, :, Bud:])              # rows past n_keep are left alone
    ko, vo, _ = orc.compact(orc.OracleParams(B, H, H, d, n, 8, 16, Bud, dtype=dtype), synth.to_numpy(k),
                            synth.to_numpy(v), idx.cpu().numpy())
    assert synth.to_numpy(k2[:, :, :Bud]).tobytes() == ko.tobytes()
    assert synth.to_numpy(v2[:, :, :Bud]).tobytes() == vo.tobytes()
    # without the score
    k3, v3 = k.clone(), v.clone()
    ab.ahakv_compact_inplace(p, k3, v3, None, idx)
    assert torch.equal(k3, k2) and torch.equal(v3, v2)


def test_evict_every_step_for_64_steps():
    """The cache is held at its budget: every step appends the new token, updates the score with the one new query
    per head, keeps the recent window and the best of the rest, and compacts in place (Algorithm 1, Generation).
    The oracle replays every step from the state the GPU path is in, in double precision: scores within 1e-3, the
    kept set equal outside the tolerance band, the moved rows byte-exact."""
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    B, Hq, Hkv, d, Bud, Br, steps, N0 = 2, 8, 2, 128, 256, 16, 64, 5000
    n = Bud + 1
    g = torch.Generator().manual_seed(2506)
    dt = torch.bfloat16
    k = torch.zeros((B, Hkv, n, d), dtype=dt, device=DEV)
    v = torch.zeros((B, Hkv, n, d), dtype=dt, device=DEV)
    k[:, :, :Bud] = torch.randn((B, Hkv, Bud, d), generator=g).to(dt).to(DEV)
    v[:, :, :Bud] = torch.randn((B, Hkv, Bud, d), generator=g).to(dt).to(DEV)
    f = torch.zeros((B, Hkv, n), device=DEV)
    f[:, :, :Bud] = (torch.rand((B, Hkv, Bud), generator=g) * 0.02).to(DEV)
    idx = torch.empty((B, Hkv, Bud), dtype=torch.int32, device=DEV)
    evicted_somewhere_other_than_the_end = 0
    for t in range(steps):
        p = ab.Params(B, Hq, Hkv, d, n, 1, Br, Bud, dtype=ab.BF16, n_total=N0 + t + 1, flags=0)
        ws = ab.alloc_workspace(p, DEV)
        q_t = torch.randn((B, Hq, 1, d), generator=g).to(dt).to(DEV)
        k[:, :, Bud] = torch.randn((B, Hkv, d), generator=g).to(dt).to(DEV)      # the new token's key and value
        v[:, :, Bud] = torch.randn((B, Hkv, d), generator=g).to(dt).to(DEV)
        f[:, :, Bud] = 0.0                                                       # a new token starts at zero
        k_before, v_before, f_before = k.clone(), v.clone(), f.clone()
        ab.ahakv_score_step(p, q_t, k, f, f)
        ab.ahakv_select(p, f, idx, ws)
        f_scored = f.clone()
        ab.ahakv_compact_inplace(p, k, v, f, idx)
        # the oracle, from the same state
        op = parity.oracle_params(p)
        ref = orc.evict(op, synth.to_numpy(q_t), synth.to_numpy(k_before), synth.to_numpy(v_before),
                        f_before.double().cpu().numpy())
        parity.assert_scores_close(p, f_scored.cpu().numpy(), ref["score"], f"step {t} score")
        gi = idx.cpu().numpy()
        for b in range(B):
            for h in range(Hkv):
                parity.assert_kept_valid(p, gi[b, h], ref["kept_idx"][b, h], ref["score"][b, h])
        ko, vo, _ = orc.compact(op, synth.to_numpy(k_before), synth.to_numpy(v_before), gi)
        assert synth.to_numpy(k[:, :, :Bud]).tobytes() == ko.tobytes(), f"step {t}: K rows"
        assert synth.to_numpy(v[:, :, :Bud]).tobytes() == vo.tobytes(), f"step {t}: V rows"
        assert torch.equal(f[:, :, :Bud], torch.gather(f_scored, 2, idx.long()))
        evicted_somewhere_other_than_the_end += int((gi[..., 0] != 0).sum() + (gi[..., Bud // 2] != Bud // 2).sum())
    assert evicted_somewhere_other_than_the_end > 0                 # the moves were real ones


def test_generation_steps_replay_from_a_cuda_graph():
    """The three calls of a generation step make no allocation, no synchronisation and no host-side decision that
    depends on device data, so a loop of steps can be captured once and replayed: eight steps captured in a CUDA
    graph leave the cache, the scores and the kept indices bit-identical to the same eight steps launched one by
    one.  (Every entry point is called once before the capture: first calls set function attributes.)"""
    from paper_2506_03762_b200 import binding as ab
    B, Hq, Hkv, d, Bud, Br, steps, N0 = 2, 8, 2, 128, 512, 32, 8, 9000
    n = Bud + 1
    g = torch.Generator().manual_seed(762)
    dt = torch.float16
    k0 = torch.zeros((B, Hkv, n, d), dtype=dt, device=DEV)
    v0 = torch.zeros_like(k0)
    k0[:, :, :Bud] = torch.randn((B, Hkv, Bud, d), generator=g).to(dt).to(DEV)
    v0[:, :, :Bud] = torch.randn((B, Hkv, Bud, d), generator=g).to(dt).to(DEV)
    f0 = torch.zeros((B, Hkv, n), device=DEV)
    f0[:, :, :Bud] = (torch.rand((B, Hkv, Bud), generator=g) * 0.02).to(DEV)
    new = [(torch.randn((B, Hq, 1, d), generator=g).to(dt).to(DEV), torch.randn((B, Hkv, d), generator=g).to(dt).to(DEV),
            torch.randn((B, Hkv, d), generator=g).to(dt).to(DEV)) for _ in range(steps)]
    ps = [ab.Params(B, Hq, Hkv, d, n, 1, Br, Bud, dtype=ab.F16, n_total=N0 + t + 1, flags=0) for t in range(steps)]
    zero = torch.zeros((B, Hkv), device=DEV)

    def run(k, v, f, idx, stream):
        for t in range(steps):
            q_t, k_t, v_t = new[t]
            k[:, :, Bud] = k_t
            v[:, :, Bud] = v_t
            f[:, :, Bud] = zero
            ab.ahakv_score_step(ps[t], q_t, k, f, f, stream=stream)
            ab.ahakv_select(ps[t], f, idx, stream=stream)
            ab.ahakv_compact_inplace(ps[t], k, v, f, idx, stream=stream)

    ke, ve, fe = k0.clone(), v0.clone(), f0.clone()
    ie = torch.empty((B, Hkv, Bud), dtype=torch.int32, device=DEV)
    run(ke, ve, fe, ie, None)
    torch.cuda.synchronize()

    kg, vg, fg = k0.clone(), v0.clone(), f0.clone()
    ig = torch.empty_like(ie)
    s = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(graph, stream=s):
            run(kg, vg, fg, ig, torch.cuda.current_stream())
    torch.cuda.synchronize()
    for _ in range(2):                       # the replay starts from the same state each time
        kg.copy_(k0); vg.copy_(v0); fg.copy_(f0)
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(kg[:, :, :Bud], ke[:, :, :Bud]) and torch.equal(vg[:, :, :Bud], ve[:, :, :Bud])
        assert torch.equal(fg[:, :, :Bud], fe[:, :, :Bud]) and torch.equal(ig, ie)


@pytest.mark.parametrize("dtype_name,Hq,Hkv,d", [("BF16", 8, 2, 128), ("F16", 4, 4, 64), ("F32", 6, 2, 128)])
def test_step_slots_for_48_steps(dtype_name, Hq, Hkv, d):
    """Generation on a cache kept as slots: nothing moves, the evicted token's slot takes the next token.  Every step
    is checked against the oracle run on the same cache put in order of position (scores within tolerance, the kept
    set equal outside the tolerance band), and the bookkeeping exactly: the new rows sit byte for byte in the slot that
    was free, no other slot changed, the position table and the free slot say which token left."""
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    B, Bud, Br, steps, N0 = 2, 192, 12, 48, 7000
    n = Bud + 1
    dtc = getattr(ab, dtype_name)
    dt = {"F32": torch.float32, "F16": torch.float16, "BF16": torch.bfloat16}[dtype_name]
    g = torch.Generator().manual_seed(1200 + d + Hq)
    k = torch.zeros((B, Hkv, n, d), dtype=dt, device=DEV)
    v = torch.zeros_like(k)
    k[:, :, :Bud] = torch.randn((B, Hkv, Bud, d), generator=g).to(dt).to(DEV)
    v[:, :, :Bud] = torch.randn((B, Hkv, Bud, d), generator=g).to(dt).to(DEV)
    f = torch.zeros((B, Hkv, n), device=DEV)
    f[:, :, :Bud] = (torch.rand((B, Hkv, Bud), generator=g) * 0.02).to(DEV)
    # positions of the cached tokens: scattered, in order, below the recent window; then the window itself
    old = torch.sort(torch.randperm(N0 - Br, generator=g)[:Bud - Br]).values
    pos0 = torch.cat([old, torch.arange(N0 - Br, N0)]).to(torch.int32)
    pos = torch.full((B, Hkv, n), -1, dtype=torch.int32, device=DEV)
    pos[:, :, :Bud] = pos0.to(DEV)
    # the slots are in no particular order: shuffle them, per head
    for b in range(B):
        for h in range(Hkv):
            perm = torch.randperm(n, generator=g).to(DEV)
            k[b, h], v[b, h], f[b, h], pos[b, h] = k[b, h][perm].clone(), v[b, h][perm].clone(), f[b, h][perm].clone(), pos[b, h][perm].clone()
    free = (pos == -1).int().argmax(dim=2).to(torch.int32).contiguous()
    for t in range(steps):
        p = ab.Params(B, Hq, Hkv, d, n, 1, Br, Bud, dtype=dtc, n_total=N0 + t + 1, flags=0)
        new_pos = N0 + t
        q_t = torch.randn((B, Hq, 1, d), generator=g).to(dt).to(DEV)
        k_t = torch.randn((B, Hkv, 1, d), generator=g).to(dt).to(DEV)
        v_t = torch.randn((B, Hkv, 1, d), generator=g).to(dt).to(DEV)
        k0, v0, f0, pos_before, free_before = k.clone(), v.clone(), f.clone(), pos.clone(), free.clone()
        ab.ahakv_step_slots(p, q_t, k_t, v_t, k, v, f, pos, free)
        torch.cuda.synchronize()
        # bookkeeping
        fb = free_before.long()[:, :, None]
        pos_full = pos_before.clone().scatter_(2, fb, torch.full_like(fb, new_pos, dtype=torch.int32))
        k_full = k0.clone().scatter_(2, fb[..., None].expand(B, Hkv, 1, d), k_t)
        v_full = v0.clone().scatter_(2, fb[..., None].expand(B, Hkv, 1, d), v_t)
        assert torch.equal(k, k_full) and torch.equal(v, v_full), f"step {t}: rows"
        fa = free.long()[:, :, None]
        assert bool(((free >= 0) & (free < n)).all())
        assert torch.equal(pos, pos_full.clone().scatter_(2, fa, torch.full_like(fa, -1, dtype=torch.int32))), f"step {t}: positions"
        assert bool((pos_full.gather(2, fa) < new_pos - Br + 1).all()), "a token of the recent window left"
        # the oracle on the cache in order of position (the new token last, with score zero)
        order = torch.argsort(pos_full, dim=2)
        ko = k_full.gather(2, order[..., None].expand(B, Hkv, n, d))
        vo = v_full.gather(2, order[..., None].expand(B, Hkv, n, d))
        f_prev = f0.clone().scatter_(2, fb, torch.zeros_like(fb, dtype=torch.float32)).gather(2, order)
        op = parity.oracle_params(p)
        ref = orc.evict(op, synth.to_numpy(q_t), synth.to_numpy(ko), synth.to_numpy(vo), f_prev.double().cpu().numpy())
        parity.assert_scores_close(p, f.gather(2, order).cpu().numpy(), ref["score"], f"step {t} score")
        rank_of_slot = torch.argsort(order, dim=2)                     # slot -> index in position order
        left = rank_of_slot.gather(2, fa)[:, :, 0].cpu().numpy()
        for b in range(B):
            for h in range(Hkv):
                kept = np.array([j for j in range(n) if j != left[b, h]], dtype=np.int32)
                parity.assert_kept_valid(p, kept, ref["kept_idx"][b, h], ref["score"][b, h])


def test_step_slots_at_the_decode_shape():
    """One step at the size the decode workload runs (16 sequences, 8 KV heads of 4 query heads, 2049 slots of 128,
    bfloat16), slots in shuffled order: eight heads against the oracle on the cache in position order, and for every
    head the bookkeeping (the slot that was free holds the new rows, one slot outside the recent window was freed,
    every other position unchanged) and the invariant that the step adds exactly one unit of score per head."""
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    w = synth.WORKLOADS["decode_round"]
    B, Hq, Hkv, d, Bud, Br = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.budget, w.recent_window
    n, N0 = Bud + 1, 40000
    g = torch.Generator(device=DEV).manual_seed(31)
    dt = torch.bfloat16
    k = torch.randn((B, Hkv, n, d), device=DEV, generator=g).to(dt)
    v = torch.randn((B, Hkv, n, d), device=DEV, generator=g).to(dt)
    f = torch.rand((B, Hkv, n), device=DEV, generator=g) * 0.01
    # positions: a random permutation of [N0 - n, N0 - 1) over the slots of each head, one slot free
    perm = torch.argsort(torch.rand((B, Hkv, n), device=DEV, generator=g), dim=2)
    pos = (perm + (N0 - n)).to(torch.int32)
    free = (pos == N0 - 1).int().argmax(dim=2).to(torch.int32).contiguous()     # the slot "holding" position N0 - 1 is the free one
    pos.scatter_(2, free.long()[:, :, None], torch.full((B, Hkv, 1), -1, dtype=torch.int32, device=DEV))
    p = ab.Params(B, Hq, Hkv, d, n, 1, Br, Bud, dtype=ab.BF16, n_total=N0, flags=0)
    new_pos = N0 - 1
    q_t = torch.randn((B, Hq, 1, d), device=DEV, generator=g).to(dt)
    k_t = torch.randn((B, Hkv, 1, d), device=DEV, generator=g).to(dt)
    v_t = torch.randn((B, Hkv, 1, d), device=DEV, generator=g).to(dt)
    k0, v0, f0, pos0, free0 = k.clone(), v.clone(), f.clone(), pos.clone(), free.clone()
    ab.ahakv_step_slots(p, q_t, k_t, v_t, k, v, f, pos, free)
    torch.cuda.synchronize()
    fb, fa = free0.long()[:, :, None], free.long()[:, :, None]
    pos_full = pos0.clone().scatter_(2, fb, torch.full_like(fb, new_pos, dtype=torch.int32))
    k_full = k0.clone().scatter_(2, fb[..., None].expand(B, Hkv, 1, d), k_t)
    v_full = v0.clone().scatter_(2, fb[..., None].expand(B, Hkv, 1, d), v_t)
    assert torch.equal(k, k_full) and torch.equal(v, v_full)
    assert torch.equal(pos, pos_full.clone().scatter_(2, fa, torch.full_like(fa, -1, dtype=torch.int32)))
    assert bool((pos_full.gather(2, fa) < new_pos - Br + 1).all())
    f_prev = f0.clone().scatter_(2, fb, torch.zeros_like(fb, dtype=torch.float32))
    added = (f.double() - f_prev.double()).sum(dim=2)
    assert float((added - 1.0).abs().max()) < 1e-3, "one query row per head, pooled by the mean: one unit of score a step"
    order = torch.argsort(pos_full, dim=2)
    rank_of_slot = torch.argsort(order, dim=2)
    left = rank_of_slot.gather(2, fa)[:, :, 0].cpu().numpy()
    for (b, h) in [(0, 0), (3, 5), (7, 2), (8, 7), (11, 1), (13, 4), (15, 7), (15, 0)]:
        o = order[b, h]
        op = parity.oracle_params(p, batch=1, n_q_heads=Hq // Hkv, n_kv_heads=1)
        G = Hq // Hkv
        ref = orc.evict(op, synth.to_numpy(q_t[b:b + 1, h * G:(h + 1) * G]), synth.to_numpy(k_full[b:b + 1, h:h + 1][:, :, o]),
                        synth.to_numpy(v_full[b:b + 1, h:h + 1][:, :, o]), f_prev[b:b + 1, h:h + 1][:, :, o].double().cpu().numpy())
        parity.assert_scores_close(p, f[b, h][o].cpu().numpy(), ref["score"][0, 0], f"unit ({b},{h})")
        kept = np.array([j for j in range(n) if j != left[b, h]], dtype=np.int32)
        parity.assert_kept_valid(p, kept, ref["kept_idx"][0, 0], ref["score"][0, 0])


def test_score_step_at_its_largest_size():
    """The most logits the one-row kernel takes (G n = 40960, all of a CTA's shared memory budget for them): four
    heads a group against 10240 keys, checked against the oracle."""
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    B, Hq, Hkv, d, n = 1, 8, 2, 128, 10240
    g = torch.Generator().manual_seed(4096)
    q = torch.randn((B, Hq, 1, d), generator=g).to(torch.float16).to(DEV)
    k = torch.randn((B, Hkv, n, d), generator=g).to(torch.float16).to(DEV)
    prev = (torch.rand((B, Hkv, n), generator=g) * 0.01).to(DEV)
    p = ab.Params(B, Hq, Hkv, d, n, 1, 64, 4096, dtype=ab.F16, n_total=50000, flags=0)
    got = torch.empty((B, Hkv, n), dtype=torch.float32, device=DEV)
    ab.ahakv_score_step(p, q, k, prev, got)
    ref = orc.score(parity.oracle_params(p), synth.to_numpy(q), synth.to_numpy(k), synth.to_numpy(k), prev.double().cpu().numpy())
    parity.assert_scores_close(p, got.cpu().numpy(), ref, "score_step, 40960 logits")
    # one more key is one too many
    p2 = ab.Params(B, Hq, Hkv, d, n + 1, 1, 64, 4096, dtype=ab.F16, n_total=50000, flags=0)
    assert ab.ahakv_score_step(p2, q, k, prev, got, check=False) == ab.ERR_UNSUPPORTED
