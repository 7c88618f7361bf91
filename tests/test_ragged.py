"""A batch whose sequences differ in length, logical position and budget, through ``ahakv_evict_ragged``: every
sequence must get exactly what ``ahakv_evict`` gives it alone, and that must match the oracle.  And budgets per
(sequence, KV head) through ``ahakv_evict_head_budgets``."""
import numpy as np
import pytest
import torch

from oracle import ahakv_oracle as orc
from paper_2506_03762_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype_name,Hq,Hkv,d", [("F16", 8, 2, 128), ("BF16", 4, 4, 64), ("F32", 2, 2, 64)])
def test_ragged_batch_equals_one_call_per_sequence(dtype_name, Hq, Hkv, d):
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    dtype = getattr(ab, dtype_name)
    dt = {ab.F32: torch.float32, ab.F16: torch.float16, ab.BF16: torch.bfloat16}[dtype]
    r, Br = 16, 8
    seqs = [(900, 200, 900), (517, 150, 40000), (130, 256, 130), (1024, 256, 5000)]   # the third keeps everything
    B, n_max, bud_max = len(seqs), 1024, 256
    g = torch.Generator().manual_seed(d + Hq)
    q = torch.randn((B, Hq, r, d), generator=g).to(dt).cuda()
    k = torch.randn((B, Hkv, n_max, d), generator=g).to(dt).cuda()
    v = (torch.randn((B, Hkv, n_max, d), generator=g) * (1 + torch.rand((B, Hkv, n_max, 1), generator=g))).to(dt).cuda()
    prev = torch.zeros((B, Hkv * n_max)).cuda()
    for b, (n, _, _) in enumerate(seqs):                      # dense [Hkv, n_b] inside the sequence's slot
        prev[b, : Hkv * n] = (torch.rand((Hkv * n,), generator=g) * 0.01).cuda()
    p = ab.Params(B, Hq, Hkv, d, n_max, r, Br, bud_max, dtype=dtype)
    ws = ab.alloc_workspace(p, "cuda")
    k_out, v_out, s_out, idx = ab.alloc_outputs(p, "cuda")
    for t in (k_out, v_out, s_out, idx):
        t.zero_()
    ab.ahakv_evict_ragged(p, seqs, q, k, v, prev, k_out, v_out, s_out, idx, ws)
    assert ab.ahakv_last_device_status(ws) == ab.OK
    for b, (n, bud, nt) in enumerate(seqs):
        keep = min(n, bud)
        pb = ab.Params(1, Hq, Hkv, d, n, r, Br, bud, dtype=dtype, n_total=nt)
        qb, kb, vb = q[b:b + 1], k[b:b + 1, :, :n].contiguous(), v[b:b + 1, :, :n].contiguous()
        pvb = prev[b, : Hkv * n].view(1, Hkv, n).contiguous()
        alone = parity.run_evict(pb, qb, kb, vb, pvb)
        got_k = k_out[b].reshape(-1)[: Hkv * keep * d].view(1, Hkv, keep, d)
        got_v = v_out[b].reshape(-1)[: Hkv * keep * d].view(1, Hkv, keep, d)
        got_s = s_out[b].reshape(-1)[: Hkv * keep].view(1, Hkv, keep)
        got_i = idx[b].reshape(-1)[: Hkv * keep].view(1, Hkv, keep)
        for a, c in zip(alone, (got_k, got_v, got_s, got_i)):
            assert torch.equal(a, c), f"sequence {b}"
        ref = orc.evict(parity.oracle_params(pb), synth.to_numpy(qb), synth.to_numpy(kb), synth.to_numpy(vb),
                        pvb.double().cpu().numpy())
        for h in range(Hkv):
            parity.assert_kept_valid(pb, got_i[0, h].cpu().numpy(), ref["kept_idx"][0, h], ref["score"][0, h])
    # an invalid entry: nothing is queued, outputs stay as they are
    before = idx.clone()
    bad = list(seqs)
    bad[1] = (2000, 150, 40000)                               # longer than the allocation
    assert ab.ahakv_evict_ragged(p, bad, q, k, v, prev, k_out, v_out, s_out, idx, ws, check=False) == ab.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert torch.equal(idx, before)


@pytest.mark.parametrize("dtype_name,Hq,Hkv,d,n", [("F16", 8, 4, 128, 1500), ("BF16", 2, 2, 64, 33000), ("F32", 4, 2, 64, 600)])
def test_a_budget_per_head(dtype_name, Hq, Hkv, d, n):
    """Every (sequence, KV head) keeps its recent window and the best of the rest up to its own budget: what
    ``ahakv_evict`` gives that head when the whole batch has that budget, bit for bit, and what the oracle says;
    entries past a head's own count are -1 and the output rows there are not touched.  (33000 tokens take the separate selection
    kernel, the others the fused one.)"""
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    dtype = getattr(ab, dtype_name)
    dt = {ab.F32: torch.float32, ab.F16: torch.float16, ab.BF16: torch.bfloat16}[dtype]
    B, r, Br, Bud = 2, 16, 8, 256
    g = torch.Generator().manual_seed(n + d)
    q = torch.randn((B, Hq, r, d), generator=g).to(dt).cuda()
    k = torch.randn((B, Hkv, n, d), generator=g).to(dt).cuda()
    v = (torch.randn((B, Hkv, n, d), generator=g) * (1 + torch.rand((B, Hkv, n, 1), generator=g))).to(dt).cuda()
    budgets = torch.tensor([[256, 100, 8, 400], [37, 256, 1, 129]], dtype=torch.int32)[:, :Hkv].contiguous()
    effective = budgets.clamp(min=Br, max=Bud)                   # what the library holds them to
    # Eq. 12 takes its budget from the call, not from a head: with a fixed scale the per-head call and the calls with
    # one budget for all compute the same scores, and only the selection differs
    fixed = dict(scale_mode=ab.SCALE_FIXED, scale=float(ab.ahakv_lambda(n, Bud, d)))
    p = ab.Params(B, Hq, Hkv, d, n, r, Br, Bud, dtype=dtype, **fixed)
    ws = ab.alloc_workspace(p, "cuda")
    k_out, v_out, s_out, idx = ab.alloc_outputs(p, "cuda")
    k_out.fill_(7.0); v_out.fill_(7.0); s_out.fill_(-5.0); idx.fill_(-9)
    ab.ahakv_evict_head_budgets(p, budgets.cuda(), q, k, v, None, k_out, v_out, s_out, idx, ws)
    assert ab.ahakv_last_device_status(ws) == ab.OK
    G = Hq // Hkv
    uniform = {}                                                 # the whole batch evicted with one budget for all
    for bud in sorted(set(int(x) for x in effective.flatten())):
        uniform[bud] = parity.run_evict(ab.Params(B, Hq, Hkv, d, n, r, Br, bud, dtype=dtype, **fixed), q, k, v, None)
    for b in range(B):
        for h in range(Hkv):
            bud = int(effective[b, h])
            assert bool((idx[b, h, bud:] == -1).all())
            assert bool((k_out[b, h, bud:] == 7.0).all()) and bool((v_out[b, h, bud:] == 7.0).all())
            assert bool((s_out[b, h, bud:] == -5.0).all())
            for a, c in zip(uniform[bud], (k_out, v_out, s_out, idx)):
                assert torch.equal(a[b, h], c[b, h, :bud]), f"head ({b},{h}) with budget {bud}"
            p1 = ab.Params(1, G, 1, d, n, r, Br, bud, dtype=dtype, **fixed)
            q1 = q[b:b + 1, h * G:(h + 1) * G].contiguous()
            k1, v1 = k[b:b + 1, h:h + 1].contiguous(), v[b:b + 1, h:h + 1].contiguous()
            ref = orc.evict(parity.oracle_params(p1), synth.to_numpy(q1), synth.to_numpy(k1), synth.to_numpy(v1), None)
            parity.assert_kept_valid(p1, idx[b, h, :bud].cpu().numpy(), ref["kept_idx"][0, 0], ref["score"][0, 0])
    # without the array the call is refused, not guessed at
    assert ab.ahakv_evict_head_budgets(p, None, q, k, v, None, k_out, v_out, s_out, idx, ws, check=False) == ab.ERR_INVALID_ARG
