"""The accumulation variants the paper names next to Recent Accumulation:

* observation rows at positions other than the last r (Limitations section: "a constant number of accumulators"
  may be chosen otherwise, e.g. by a TopK rule) -- ``ahakv_score_rows``;
* accumulation over all rows (Section 4.1, Eq. 2-3; the "w/o RA" row of the ablation table; H2O's score with the
  plain softmax and no value prior) -- ``ahakv_score_full_causal``.

The oracle takes the rows' positions as an optional parameter; its default (the last r positions) is what every
other pin tests, and the first tests below tie the two together on the CPU.
"""
import numpy as np
import pytest
import torch

from oracle import ahakv_oracle as orc
from paper_2506_03762_b200 import synth


def _small(seed, B=1, Hq=2, Hkv=2, d=32, n=48):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, Hq, n, d)).astype(np.float32)
    k = rng.standard_normal((B, Hkv, n, d)).astype(np.float32)
    v = rng.standard_normal((B, Hkv, n, d)).astype(np.float32)
    return q, k, v


def test_oracle_default_positions_are_the_last_r():
    orc.build()
    q, k, v = _small(1)
    n, r = 48, 8
    qo = np.ascontiguousarray(q[:, :, n - r:])
    for nt in (n, n + 500):
        p0 = orc.OracleParams(1, 2, 2, 32, n, r, 4, 16, dtype=orc.F32, n_total=nt)
        p1 = orc.OracleParams(1, 2, 2, 32, n, r, 4, 16, dtype=orc.F32, n_total=nt, obs_pos=np.arange(nt - r, nt))
        assert np.array_equal(orc.score(p0, qo, k, v), orc.score(p1, qo, k, v))


def test_oracle_rows_in_passes_add_up_to_all_rows():
    """Eq. 2-3 over all n rows (obs_window = n, pinned elsewhere against closed forms) equals the sum of the scores of
    disjoint groups of rows given by position, whatever the grouping."""
    orc.build()
    q, k, v = _small(2)
    n = 48
    kw = dict(dtype=orc.F32, scale_mode=orc.SCALE_FIXED, scale=32 ** -0.5, flags=0)
    whole = orc.score(orc.OracleParams(1, 2, 2, 32, n, n, 4, 16, **kw), q, k, v)
    total = np.zeros_like(whole)
    for rows in (np.arange(0, 48, 3), np.arange(1, 48, 3), np.arange(2, 48, 3)):      # interleaved thirds
        p = orc.OracleParams(1, 2, 2, 32, n, len(rows), 4, 16, obs_pos=rows, **kw)
        total += orc.score(p, np.ascontiguousarray(q[:, :, rows]), k, v)
    assert np.allclose(total, whole, rtol=1e-12, atol=0)
    # a row placed at position j sees keys 0 .. j only: the single row at position 0 puts all its mass on key 0
    p = orc.OracleParams(1, 2, 2, 32, n, 1, 4, 16, obs_pos=[0], **kw)
    first = orc.score(p, np.ascontiguousarray(q[:, :, :1]), k, v)
    assert np.allclose(first[..., 0], 1.0) and np.all(first[..., 1:] == 0.0)


def test_oracle_rejects_positions_outside_the_cache_or_out_of_order():
    orc.build()
    q, k, v = _small(3)
    qo = np.ascontiguousarray(q[:, :, :3])
    for bad in ([5, 4, 6], [0, 1, 48], [-1, 0, 1], [3, 3, 4]):
        with pytest.raises(ValueError):
            orc.score(orc.OracleParams(1, 2, 2, 32, 48, 3, 4, 16, dtype=orc.F32, obs_pos=bad), qo, k, v)


# ---- GPU --------------------------------------------------------------------------------------------------------

def _gpu_case(B, Hq, Hkv, d, n, dtype, seed):
    from paper_2506_03762_b200 import binding as ab
    dt = {ab.F32: torch.float32, ab.F16: torch.float16, ab.BF16: torch.bfloat16}[dtype]
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((B, Hq, n, d), generator=g).to(dt).cuda()
    k = torch.randn((B, Hkv, n, d), generator=g).to(dt).cuda()
    v = (torch.randn((B, Hkv, n, d), generator=g) * (1 + torch.rand((B, Hkv, n, 1), generator=g))).to(dt).cuda()
    return q, k, v


@pytest.mark.gpu
@pytest.mark.parametrize("B,Hq,Hkv,d,n,r,dtype_name,tail", [
    (1, 2, 2, 128, 900, 40, "F16", 0),        # rows spread over the whole cache, the last one at the end
    (2, 8, 2, 128, 1300, 32, "BF16", 300),    # no row sees the last 300 keys: their tiles are skipped, V still squared
    (1, 2, 1, 64, 400, 24, "F32", 50),
    (1, 1, 1, 128, 2000, 200, "F16", 0),      # two row blocks
])
def test_score_rows_matches_the_oracle(B, Hq, Hkv, d, n, r, dtype_name, tail):
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    dtype = getattr(ab, dtype_name)
    q_all, k, v = _gpu_case(B, Hq, Hkv, d, n, dtype, seed=n + r)
    rng = np.random.default_rng(n)
    n_total = n + 777
    cache_rows = np.sort(rng.choice(n - tail, size=r, replace=False))
    if tail == 0:
        cache_rows[-1] = n - 1
    pos = (cache_rows + (n_total - n)).tolist()
    q = q_all[:, :, torch.as_tensor(cache_rows).cuda()].contiguous()
    p = ab.Params(B, Hq, Hkv, d, n, r, 16, 200, dtype=dtype, n_total=n_total)
    prev = (torch.rand((B, Hkv, n)) * 0.01).cuda()
    ws = ab.alloc_workspace(p, "cuda")
    score = torch.empty((B, Hkv, n), dtype=torch.float32, device="cuda")
    ab.ahakv_score_rows(p, pos, q, k, v, prev, score, ws)
    assert ab.ahakv_last_device_status(ws) == ab.OK
    op = parity.oracle_params(p)
    op.obs_pos = pos
    ref = orc.score(op, synth.to_numpy(q), synth.to_numpy(k), synth.to_numpy(v), prev.double().cpu().numpy())
    parity.assert_scores_close(p, score.cpu().numpy(), ref, "score_rows")
    # the default positions through the same entry point are ahakv_score, bit for bit
    last = list(range(n_total - r, n_total))
    q_last = q_all[:, :, n - r:].contiguous()
    a = torch.empty_like(score)
    b = torch.empty_like(score)
    ab.ahakv_score_rows(p, last, q_last, k, v, None, a, ws)
    ab.ahakv_score(p, q_last, k, v, None, b, ws)
    assert torch.equal(a, b)


@pytest.mark.gpu
@pytest.mark.parametrize("B,Hq,Hkv,d,n,R,dtype_name,plain", [
    (1, 2, 2, 128, 700, 128, "F16", True),     # H2O: plain softmax, no value prior; ragged last pass
    (2, 8, 2, 128, 1000, 64, "BF16", False),   # "w/o RA": Eq. 12 per row, value prior, grouped heads
    (1, 2, 2, 64, 300, 100, "F32", False),
])
def test_full_causal_accumulation_matches_the_oracle(B, Hq, Hkv, d, n, R, dtype_name, plain):
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    dtype = getattr(ab, dtype_name)
    q, k, v = _gpu_case(B, Hq, Hkv, d, n, dtype, seed=n)
    kw = dict(scale_mode=ab.SCALE_FIXED, scale=d ** -0.5, flags=0) if plain else {}
    p = ab.Params(B, Hq, Hkv, d, n, R, 16, 100, dtype=dtype, **kw)
    prev = None if plain else (torch.rand((B, Hkv, n)) * 0.01).cuda()
    ws = ab.alloc_workspace(p, "cuda")
    score = torch.empty((B, Hkv, n), dtype=torch.float32, device="cuda")
    ab.ahakv_score_full_causal(p, q, k, v, prev, score, ws)
    assert ab.ahakv_last_device_status(ws) == ab.OK
    op = parity.oracle_params(p)
    op.obs_window = n                                             # Eq. 2-3: every row accumulates
    ref = orc.score(op, synth.to_numpy(q), synth.to_numpy(k), synth.to_numpy(v),
                    None if prev is None else prev.double().cpu().numpy())
    # the tolerance of a score whose mean is 1 (n rows of mass 1 over n keys), not r / n
    pt = ab.Params(B, Hq, Hkv, d, n, n if n <= 256 // (Hq // Hkv) else R, 16, 100, dtype=dtype)
    rtol, _ = parity.score_tolerance(pt)
    got = score.double().cpu().numpy()
    assert (np.abs(got - ref) <= rtol * np.abs(ref) + rtol * 1e-3).all(), np.abs(got / ref - 1).max()
    if plain:                                                     # total mass n, and the early-token bias of Eq. 4
        assert np.allclose(got.sum(-1), n, rtol=2e-4)
        assert got[..., : n // 4].mean() > 3 * got[..., -n // 4:].mean()
    if Hq != Hkv:                                                 # pooling by maximum does not split into passes
        pg = ab.Params(B, Hq, Hkv, d, n, R, 16, 100, dtype=dtype, flags=ab.FLAG_GROUP_MAX)
        assert ab.ahakv_score_full_causal(pg, q, k, v, None, score, ws, check=False) == ab.ERR_UNSUPPORTED
