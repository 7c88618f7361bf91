"""Nothing is written outside what a call was given: the workspace and every output sit between guard bands filled
with a pattern, the eviction step runs on several shapes (tensor-core and FP32 paths, a ragged last tile, grouped
queries, a carried score), and the bands must come back untouched.  Stands in for a memory checker, which this
library's GPU tests cannot assume to have."""
import pytest
import torch

from paper_2506_03762_b200 import synth

pytestmark = pytest.mark.gpu

GUARD = 4096
PATTERN = 0xA5


def _guarded(nbytes, device):
    """A uint8 buffer of nbytes between two guard bands; returns (whole, interior view)."""
    nbytes = (nbytes + 255) // 256 * 256
    whole = torch.full((nbytes + 2 * GUARD,), PATTERN, dtype=torch.uint8, device=device)
    return whole, whole[GUARD:GUARD + nbytes]


def _intact(whole):
    return bool((whole[:GUARD] == PATTERN).all()) and bool((whole[-GUARD:] == PATTERN).all())


@pytest.mark.parametrize("B,Hq,Hkv,d,n,r,Br,Bud,dtype_name,carried", [
    (2, 8, 2, 128, 1500, 32, 16, 256, "F16", False),     # tensor-core path, ragged last tile, grouped queries
    (1, 4, 4, 64, 4096, 64, 64, 512, "BF16", True),      # a carried score, d = 64
    (1, 2, 2, 64, 300, 16, 8, 100, "F32", False),        # FP32 path
    (3, 6, 2, 128, 100, 8, 4, 40, "F16", False),         # fewer keys than a tile
    (1, 2, 1, 128, 200, 16, 8, 256, "BF16", False),      # nothing to evict: budget above the context
])
def test_the_eviction_step_stays_inside_its_buffers(B, Hq, Hkv, d, n, r, Br, Bud, dtype_name, carried):
    from paper_2506_03762_b200 import binding as ab
    dtype = getattr(ab, dtype_name)
    dt = {ab.F32: torch.float32, ab.F16: torch.float16, ab.BF16: torch.bfloat16}[dtype]
    es = torch.empty((), dtype=dt).element_size()
    g = torch.Generator().manual_seed(n)
    q = torch.randn((B, Hq, r, d), generator=g).to(dt).cuda()
    k = torch.randn((B, Hkv, n, d), generator=g).to(dt).cuda()
    v = torch.randn((B, Hkv, n, d), generator=g).to(dt).cuda()
    prev = (torch.rand((B, Hkv, n), generator=g) * 0.01).cuda() if carried else None
    p = ab.Params(B, Hq, Hkv, d, n, r, Br, Bud, dtype=dtype, n_total=(n + 1000 if carried else None),
                  flags=(0 if carried else ab.FLAG_VALUE_PRIOR))
    keep = min(n, Bud)
    ws_all, ws = _guarded(ab.ahakv_workspace_bytes(p), "cuda")
    ko_all, ko = _guarded(B * Hkv * keep * d * es, "cuda")
    vo_all, vo = _guarded(B * Hkv * keep * d * es, "cuda")
    so_all, so = _guarded(B * Hkv * keep * 4, "cuda")
    io_all, io = _guarded(B * Hkv * keep * 4, "cuda")
    inputs_before = [t.clone() for t in (q, k, v)]
    for _ in range(2):
        ab.ahakv_evict(p, q, k, v, prev, ko, vo, so, io, ws, ws_bytes=ab.ahakv_workspace_bytes(p))
    torch.cuda.synchronize()
    assert ab.ahakv_last_device_status(ws) == ab.OK
    for name, whole in (("workspace", ws_all), ("k_out", ko_all), ("v_out", vo_all), ("score_out", so_all), ("kept_idx", io_all)):
        assert _intact(whole), f"{name}: a guard band was written"
    for t, before in zip((q, k, v), inputs_before):
        assert torch.equal(t, before), "an input was written"
    idx = io[: B * Hkv * keep * 4].view(torch.int32).view(B, Hkv, keep)
    assert int(idx.min()) >= 0 and int(idx.max()) < n and bool((idx[..., 1:] > idx[..., :-1]).all())
    # the generation step's calls, on a cache of budget + 1 rows cut from the same tensors
    if n > Bud and dtype != ab.F32:
        n1 = Bud + 1
        p1 = ab.Params(B, Hq, Hkv, d, n1, 1, Br, Bud, dtype=dtype, n_total=5 * n, flags=0)
        kc_all, kc = _guarded(B * Hkv * n1 * d * es, "cuda")
        vc_all, vc = _guarded(B * Hkv * n1 * d * es, "cuda")
        fc_all, fc = _guarded(B * Hkv * n1 * 4, "cuda")
        ps_all, ps = _guarded(B * Hkv * n1 * 4, "cuda")
        fr_all, fr = _guarded(B * Hkv * 4, "cuda")
        kc[: B * Hkv * n1 * d * es].view(dt).view(B, Hkv, n1, d).copy_(k[:, :, :n1])
        vc[: B * Hkv * n1 * d * es].view(dt).view(B, Hkv, n1, d).copy_(v[:, :, :n1])
        fc[: B * Hkv * n1 * 4].view(torch.float32).zero_()
        pos = ps[: B * Hkv * n1 * 4].view(torch.int32).view(B, Hkv, n1)
        pos.copy_(torch.arange(4 * n, 4 * n + n1, dtype=torch.int32).cuda().expand(B, Hkv, n1))
        pos[:, :, Bud] = -1
        fr[: B * Hkv * 4].view(torch.int32).fill_(Bud)
        q_t = q[:, :, :1].contiguous()
        k_t, v_t = k[:, :, -1:].contiguous(), v[:, :, -1:].contiguous()
        ab.ahakv_step_slots(p1, q_t, k_t, v_t, kc, vc, fc, ps, fr)
        ab.ahakv_score_step(p1, q_t, kc, fc, fc)
        torch.cuda.synchronize()
        for name, whole in (("k", kc_all), ("v", vc_all), ("score", fc_all), ("pos", ps_all), ("free_slot", fr_all)):
            assert _intact(whole), f"generation step, {name}: a guard band was written"
