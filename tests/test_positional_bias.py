"""Positional bias of the kept set (Section 3.1, Eq. 4, and the retained-index plots of Appendix C, restated on
synthetic data): accumulating attention over ALL query rows with the plain softmax favours early tokens, because
token j collects mass from n - j rows; accumulating over the last r rows only (Eq. 5) does not.  The synthetic
layers place their heavy-hitter keys uniformly over the positions outside the recent window, so an unbiased
score keeps tokens uniformly and a biased one keeps the early ones.
"""
import numpy as np
import pytest
import torch

from oracle import ahakv_oracle as orc
from paper_2506_03762_b200 import synth


def _bin_shares(kept, n_cand, bins):
    """Share of the kept candidates (indices below n_cand) that falls into each of `bins` equal position bins."""
    kept = np.asarray(kept).reshape(-1)
    kept = kept[kept < n_cand]
    hist = np.histogram(kept, bins=bins, range=(0, n_cand))[0].astype(np.float64)
    return hist / hist.sum()


def test_oracle_recent_accumulation_keeps_positions_uniformly_full_accumulation_does_not():
    orc.build()
    w = synth.WORKLOADS["llama2_7b_4k"].scaled(n_q_heads=8, n_kv_heads=8, n_ctx=1024, head_dim=64, obs_window=32,
                                               recent_window=32, budget=160, dtype="f32", hitter_frac=0.04)
    q, k, v = synth.make_layer(w, device="cpu")
    qn, kn, vn = (synth.to_numpy(t) for t in (q, k, v))
    n_cand = w.n_ctx - w.recent_window
    # the method: last r rows, Eq. 12's scale, value prior
    p = orc.OracleParams(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_ctx, w.obs_window, w.recent_window,
                         w.budget, dtype=orc.F32, flags=orc.FLAG_VALUE_PRIOR)
    aha = _bin_shares(orc.evict(p, qn, kn, vn)["kept_idx"], n_cand, 4)
    # Eq. 2-3: every row accumulates (r = n), plain softmax.  The layer has queries for its last r rows only, so
    # the full query matrix is drawn here, from the same kind of stream.
    g = torch.Generator().manual_seed(synth.BASE_SEED + 99)
    q_full = torch.randn((w.batch, w.n_q_heads, w.n_ctx, w.head_dim), generator=g)
    q_full[:, :, w.n_ctx - w.obs_window:] = q
    ph = orc.OracleParams(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_ctx, w.n_ctx, w.recent_window,
                          w.budget, dtype=orc.F32, scale_mode=orc.SCALE_FIXED, scale=w.head_dim ** -0.5, flags=0)
    h2o = _bin_shares(orc.evict(ph, q_full.numpy(), kn, vn)["kept_idx"], n_cand, 4)
    assert np.abs(aha - 0.25).max() < 0.07, f"recent accumulation should keep positions evenly, got {aha}"
    assert h2o[0] > 0.5 and h2o[0] > 2.5 * h2o[3], f"full accumulation should favour early tokens, got {h2o}"
    assert h2o[0] > aha[0] + 0.2


@pytest.mark.gpu
def test_gpu_kept_positions_are_uniform_on_long_32k():
    """One full-size layer (8 x 32 heads x 32768 tokens): with the heavy hitters uniform over positions, the
    kept candidates of all 256 heads together spread evenly over eight position bins."""
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    w = synth.WORKLOADS["long_32k"]
    p = parity.params_of(w)
    q, k, v = synth.make_layer(w, layer=5, device="cuda")
    _, _, _, idx = parity.run_evict(p, q, k, v)
    shares = _bin_shares(idx.cpu().numpy(), w.n_ctx - w.recent_window, 8)
    assert np.abs(shares - 0.125).max() < 0.01, f"kept positions should be uniform, got {shares}"
    del ab


@pytest.mark.gpu
def test_gpu_full_accumulation_favours_early_tokens():
    """r = n with the plain softmax on the GPU path (the largest r a call takes, 256 rows of one head): the kept
    set leans to the early positions, and agrees with the oracle's."""
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    B, H, d, n, Br, Bud = 4, 8, 128, 256, 16, 64
    g = torch.Generator().manual_seed(31)
    q = torch.randn((B, H, n, d), generator=g).to(torch.float16).cuda()
    k = torch.randn((B, H, n, d), generator=g).to(torch.float16).cuda()
    v = torch.randn((B, H, n, d), generator=g).to(torch.float16).cuda()
    p = ab.Params(B, H, H, d, n, n, Br, Bud, dtype=ab.F16, scale_mode=ab.SCALE_FIXED, scale=d ** -0.5, flags=0)
    st = parity.check_units(p, q, k, v, parity.all_units(p))
    shares = _bin_shares(st["outputs"][4].cpu().numpy(), n - Br, 4)
    assert shares[0] > 0.45 and shares[0] > 2.0 * shares[3], f"got {shares}"
