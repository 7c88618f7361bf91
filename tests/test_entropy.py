"""Row entropy of the scaled softmax (Eq. 6) on the GPU against the oracle's, which is pinned in test_oracle_pins.py."""
import numpy as np
import pytest
import torch

from oracle import ahakv_oracle as orc
from paper_2506_03762_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,Hq,Hkv,d,n,r,dtype_name,extra", [
    (1, 2, 2, 64, 512, 32, "F32", {}),
    (2, 8, 2, 128, 1500, 32, "BF16", dict(n_total=9000)),
    (1, 4, 4, 128, 4096, 64, "F16", {}),
    (1, 1, 1, 128, 300, 200, "F16", dict(scale_mode=0, scale=128 ** -0.5)),     # plain softmax, rows deep in the mask
    (1, 2, 1, 64, 129, 1, "BF16", {}),
    (1, 2, 2, 64, 700, 256, "F16", {}),                                         # the most rows a call takes
])
def test_row_entropy_matches_the_oracle(B, Hq, Hkv, d, n, r, dtype_name, extra):
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    dtype = getattr(ab, dtype_name)
    dt = {ab.F32: torch.float32, ab.F16: torch.float16, ab.BF16: torch.bfloat16}[dtype]
    g = torch.Generator().manual_seed(n + r)
    q = torch.randn((B, Hq, r, d), generator=g).to(dt).cuda()
    k = torch.randn((B, Hkv, n, d), generator=g).to(dt).cuda()
    p = ab.Params(B, Hq, Hkv, d, n, r, 16, 100, dtype=dtype, **extra)
    H = ab.ahakv_row_entropy(p, q, k).cpu().numpy().astype(np.float64)
    again = ab.ahakv_row_entropy(p, q, k).cpu().numpy()
    assert np.array_equal(H.astype(np.float32), again)                          # fixed reduction order
    op = parity.oracle_params(p)
    qn, kn = synth.to_numpy(q), synth.to_numpy(k)
    ref = np.stack([np.stack([orc.row_entropy(op, qn, kn, b, h) for h in range(Hq)]) for b in range(B)])
    assert H.shape == ref.shape == (B, Hq, r)
    # entropies are a few nats; FP32 sums of up to 4096 terms, approximate exp2 and log2
    tol = 2e-5 if dtype == ab.F32 else 1e-4
    assert np.abs(H - ref).max() <= tol * max(1.0, np.abs(ref).max()), np.abs(H - ref).max()
    assert (H >= -1e-6).all() and (H <= np.log(n) + 1e-6).all()


def test_entropy_tracks_eq10_on_gaussian_data():
    """Eq. 10: E[H_i] = ln i - lambda^2 d / 2 for unit-variance Gaussian queries and keys (an approximation that
    holds for small lambda^2 d; checked loosely), and Eq. 12's lambda brings the mean entropy near ln(budget)."""
    from paper_2506_03762_b200 import binding as ab
    B, H, d, n, r, Bud = 4, 8, 128, 8192, 32, 2048
    g = torch.Generator().manual_seed(5)
    q = torch.randn((B, H, r, d), generator=g).to(torch.float16).cuda()
    k = torch.randn((B, H, n, d), generator=g).to(torch.float16).cuda()
    lam = 0.05
    p = ab.Params(B, H, H, d, n, r, 16, Bud, dtype=ab.F16, scale_mode=ab.SCALE_FIXED, scale=lam)
    Hm = float(ab.ahakv_row_entropy(p, q, k).double().mean())
    assert abs(Hm - (np.log(n) - lam * lam * d / 2)) < 0.05, Hm
    p12 = ab.Params(B, H, H, d, n, r, 16, Bud, dtype=ab.F16)                    # Eq. 12 per row
    H12 = float(ab.ahakv_row_entropy(p12, q, k).double().mean())
    assert abs(H12 - np.log(Bud)) < 0.35, (H12, np.log(Bud))
