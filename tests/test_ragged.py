"""A batch whose sequences differ in length, logical position and budget, through ``ahakv_evict_ragged``: every
sequence must get exactly what ``ahakv_evict`` gives it alone, and that must match the oracle."""
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
