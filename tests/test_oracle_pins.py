"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these re-type the oracle's own formula: each compares it with a library
routine on a special case, a closed form, an invariant, a hand-worked fixture
or brute force, chosen so that a dropped term, a wrong sign or index, or a
transposed operand fails at least one of them.
"""
import itertools
import math

import numpy as np
import pytest
import scipy.special
import torch

from tests.conftest import golden_path


def _rand(shape, seed, dtype=np.float32):
    return np.random.default_rng(seed).standard_normal(shape).astype(dtype)


def _params(oracle, B=1, Hq=1, Hkv=1, d=8, n=16, r=4, Br=2, Bud=8, **kw):
    kw.setdefault("dtype", oracle.F32)
    return oracle.OracleParams(B, Hq, Hkv, d, n, r, Br, Bud, **kw)


# ---- Eq. 1 / Eq. 9: softmax rows ---------------------------------------------------------------

def test_rows_sum_to_one_and_score_mass(oracle):
    """Each SG-softmax row has mass 1 (Eq. 1), so sum_j S_j = r before the value prior (Eq. 5)."""
    p = _params(oracle, B=2, Hq=4, Hkv=2, d=16, n=96, r=12, Br=8, Bud=32, flags=0)
    q, k, v = _rand((2, 4, 12, 16), 1), _rand((2, 2, 96, 16), 2), _rand((2, 2, 96, 16), 3)
    for b in range(2):
        for hq in range(4):
            a = oracle.attention(p, q, k, b, hq)
            assert np.allclose(a.sum(1), 1.0, atol=1e-12)
            assert (a >= 0).all()
            for i in range(12):                      # causal mask: row i sees columns <= n - r + i
                assert (a[i, 96 - 12 + i + 1:] == 0).all()
                assert a[i, 96 - 12 + i] > 0
    s = oracle.score(p, q, k, v)
    assert np.allclose(s.sum(-1), 12.0, atol=1e-10)


def test_fixed_scale_equals_library_attention(oracle):
    """lambda = 1/sqrt(d) is plain causal attention: torch's scaled_dot_product_attention applied to
    V = I returns the attention matrix itself (Eq. 1)."""
    n, d = 40, 16
    q, k = _rand((1, 1, n, d), 4), _rand((1, 1, n, d), 5)
    qt, kt = torch.from_numpy(q).double(), torch.from_numpy(k).double()
    A_lib = torch.nn.functional.scaled_dot_product_attention(
        qt, kt, torch.eye(n, dtype=torch.float64).view(1, 1, n, n), is_causal=True)[0, 0].numpy()
    # r = n: the whole causal matrix
    p = _params(oracle, d=d, n=n, r=n, Br=4, Bud=8, scale_mode=oracle.SCALE_FIXED, scale=1 / math.sqrt(d))
    assert np.allclose(oracle.attention(p, q, k, 0, 0), A_lib, atol=1e-12)
    # r < n: the last r rows of the same matrix (Recent Accumulation, Eq. 5)
    r = 7
    p = _params(oracle, d=d, n=n, r=r, Br=4, Bud=8, scale_mode=oracle.SCALE_FIXED, scale=1 / math.sqrt(d))
    q_obs = np.ascontiguousarray(q[:, :, n - r:, :])
    assert np.allclose(oracle.attention(p, q_obs, k, 0, 0), A_lib[n - r:], atol=1e-12)


def test_reduces_to_h2o_accumulated_attention(oracle):
    """Unit gain, no value prior, r = n: the H2O score S_j = sum_{i>=j} a_ij (Eq. 2-3); with r < n the
    SnapKV-style window score.  The library routine here is scipy's softmax over masked logits."""
    n, d = 64, 8
    q, k, v = _rand((1, 1, n, d), 6), _rand((1, 1, n, d), 7), _rand((1, 1, n, d), 8)
    logits = (q[0, 0].astype(np.float64) @ k[0, 0].astype(np.float64).T) / math.sqrt(d)
    logits[np.triu_indices(n, 1)] = -np.inf
    A = scipy.special.softmax(logits, axis=1)
    p = _params(oracle, d=d, n=n, r=n, Br=4, Bud=8, scale_mode=oracle.SCALE_FIXED, scale=1 / math.sqrt(d), flags=0)
    assert np.allclose(oracle.score(p, q, k, v)[0, 0], A.sum(0), atol=1e-12)
    r = 9
    p = _params(oracle, d=d, n=n, r=r, Br=4, Bud=8, scale_mode=oracle.SCALE_FIXED, scale=1 / math.sqrt(d), flags=0)
    s = oracle.score(p, np.ascontiguousarray(q[:, :, n - r:]), k, v)[0, 0]
    assert np.allclose(s, A[n - r:].sum(0), atol=1e-12)


def test_constant_keys_give_harmonic_sums(oracle):
    """Identical keys make every visible a_ij = 1/i, so the H2O score is the harmonic tail
    sum_{i=j..n} 1/i (the monotone bias of Eq. 4) and the recent-r score is flat outside the window."""
    n, d = 512, 4
    q, v = _rand((1, 1, n, d), 9), _rand((1, 1, n, d), 10)
    k = np.ones((1, 1, n, d), np.float32)
    p = _params(oracle, d=d, n=n, r=n, Br=4, Bud=8, flags=0, scale_mode=oracle.SCALE_FIXED, scale=0.5)
    s = oracle.score(p, q, k, v)[0, 0]
    want = np.array([sum(1.0 / i for i in range(j, n + 1)) for j in range(1, n + 1)])
    assert np.allclose(s, want, atol=1e-12)
    assert abs(s[0] - 6.8165) < 1e-4 and abs(s[255] - 0.6961) < 1e-4      # H_512, H_512 - H_255
    r = 32
    p = _params(oracle, d=d, n=n, r=r, Br=4, Bud=8, flags=0, scale_mode=oracle.SCALE_FIXED, scale=0.5)
    s = oracle.score(p, np.ascontiguousarray(q[:, :, n - r:]), k, v)[0, 0]
    flat = sum(1.0 / i for i in range(n - r + 1, n + 1))
    assert abs(flat - 0.06447) < 1e-5
    assert np.allclose(s[: n - r + 1], flat, atol=1e-13)
    # inside the window token j (1-based) is seen only by rows i >= j
    for j1 in range(n - r + 2, n + 1):
        assert math.isclose(s[j1 - 1], sum(1.0 / i for i in range(j1, n + 1)), rel_tol=1e-12)


def test_rational_closed_form_and_mask_boundary(oracle):
    """Keys k_j = (ln(j+1)/lambda, 0) and queries (1, 0) give e^{lambda q.k_j} = j+1, so
    a_ij = (j+1) / ((L+1)(L+2)/2) with L = n-r+i the last visible column: pins operand order, the sign
    of the exponent and the exact position of the causal boundary."""
    n, r, lam = 24, 5, 0.37
    k = np.zeros((1, 1, n, 2), np.float32)
    k[0, 0, :, 0] = np.log(np.arange(1, n + 1)) / lam
    k[0, 0, :, 1] = 3.0                                    # must not matter: q's second entry is 0
    q = np.zeros((1, 1, r, 2), np.float32)
    q[..., 0] = 1.0
    p = _params(oracle, d=2, n=n, r=r, Br=2, Bud=8, scale_mode=oracle.SCALE_FIXED, scale=lam)
    a = oracle.attention(p, q, k, 0, 0)
    for i in range(r):
        L = n - r + i
        want = np.zeros(n)
        want[: L + 1] = np.arange(1, L + 2) / ((L + 1) * (L + 2) / 2)
        assert np.allclose(a[i], want, rtol=1e-5, atol=0)     # float32 storage of ln(j+1)/lambda


# ---- Eq. 12: adaptive scale -----------------------------------------------------------------------

def test_eq12_lambda_values(oracle):
    for line in open(golden_path("eq12_lambda_values.txt")):
        if line.startswith("#") or not line.strip():
            continue
        i, k, d, lam, gain = line.split()
        got = oracle.eq12_lambda(int(i), int(k), int(d))
        assert math.isclose(got, float(lam), rel_tol=1e-14)
        assert math.isclose(got * math.sqrt(int(d)), float(gain), rel_tol=1e-14)
    assert math.isclose(oracle.eq12_lambda(100, 100, 64), 1 / 8)       # outside Eq. 12's domain
    assert math.isclose(oracle.eq12_lambda(50, 100, 64), 1 / 8)


@pytest.mark.parametrize("mode", ["row", "call", "fixed"])
def test_scale_mode_reaches_the_softmax(oracle, mode):
    """Recover lambda_i from ratios of attention weights on scalar keys and compare with Eq. 12 at the
    row's token count (its logical position + 1) or at n_total."""
    n, r, Bud, d, n_total = 40, 6, 10, 4, 1000
    k = np.zeros((1, 1, n, d), np.float32)
    k[0, 0, :, 0] = np.linspace(-1, 1, n, dtype=np.float32)
    q = np.zeros((1, 1, r, d), np.float32)
    q[..., 0] = 2.0
    sm = {"row": oracle.SCALE_ADAPTIVE_ROW, "call": oracle.SCALE_ADAPTIVE_CALL, "fixed": oracle.SCALE_FIXED}[mode]
    p = _params(oracle, d=d, n=n, r=r, Br=2, Bud=Bud, n_total=n_total, scale_mode=sm, scale=0.123)
    a = oracle.attention(p, q, k, 0, 0)
    kk = k[0, 0, :, 0].astype(np.float64)
    for i in range(r):
        lam_seen = math.log(a[i, 20] / a[i, 3]) / (2.0 * (kk[20] - kk[3]))
        tokens = {"row": n_total - r + i + 1, "call": n_total}.get(mode)
        want = 0.123 if mode == "fixed" else math.sqrt(2 * math.log(tokens / Bud) / d)
        assert math.isclose(lam_seen, want, rel_tol=1e-9)


def test_entropy_matches_eq10_and_eq12_target(oracle):
    """Eq. 10: E[H] = ln i - lambda^2 d / 2 for Gaussian logits (an approximation: loose tolerance);
    with Eq. 12's lambda the expected entropy is ln k, the entropy of k equal weights."""
    n, d, r, Bud = 4096, 64, 16, 1024
    q, k = _rand((1, 1, r, d), 11), _rand((1, 1, n, d), 12)
    q /= np.linalg.norm(q, axis=-1, keepdims=True) / math.sqrt(d)      # |q|^2 = d: logit variance = d
    # small gain: lambda^2 d = 1
    p = _params(oracle, d=d, n=n, r=r, Br=2, Bud=Bud, scale_mode=oracle.SCALE_FIXED, scale=1 / math.sqrt(d))
    H = oracle.row_entropy(p, q, k, 0, 0)
    assert abs(H.mean() - (math.log(n) - 0.5)) < 0.03
    # Eq. 12's gain
    p = _params(oracle, d=d, n=n, r=r, Br=2, Bud=Bud, scale_mode=oracle.SCALE_ADAPTIVE_CALL)
    H = oracle.row_entropy(p, q, k, 0, 0)
    assert abs(H.mean() - math.log(Bud)) < 0.08
    # entropy of a uniform row is ln(visible count)
    p = _params(oracle, d=d, n=n, r=r, Br=2, Bud=Bud, scale_mode=oracle.SCALE_FIXED, scale=0.0)
    H = oracle.row_entropy(p, q, k, 0, 0)
    assert np.allclose(H, np.log(np.arange(n - r + 1, n + 1)), atol=1e-9)


# ---- Eq. 13-15: value prior --------------------------------------------------------------------------

def _read_vectors(name):
    out = {}
    for line in open(golden_path(name)):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        out[key] = np.array([float(x) for x in vals])
    return out


def test_value_prior_worked_example(oracle):
    g = _read_vectors("value_prior_worked_example.txt")
    n = len(g["nu"])
    v = np.zeros((1, 1, n, 4), np.float32)
    v[0, 0, :, 2] = -np.sqrt(g["nu"])                      # sign and channel must not matter
    q, k = _rand((1, 1, 2, 4), 13), _rand((1, 1, n, 4), 14)
    for flags, key in ((oracle.FLAG_VALUE_PRIOR, "gamma_bar"),
                       (oracle.FLAG_VALUE_PRIOR | oracle.FLAG_POOL_ZERO_PAD, "gamma_bar_pad")):
        p = _params(oracle, d=4, n=n, r=2, Br=2, Bud=4, pool_kernel=3, flags=flags)
        s, raw = oracle.score(p, q, k, v, return_raw=True)
        assert np.allclose(s[0, 0], g[key] * raw[0, 0], rtol=1e-13)


def test_value_prior_invariants(oracle):
    n, d = 50, 8
    q, k, v = _rand((1, 1, 5, d), 15), _rand((1, 1, n, d), 16), _rand((1, 1, n, d), 17)
    p = _params(oracle, d=d, n=n, r=5, Br=2, Bud=8, pool_kernel=5)
    s, raw = oracle.score(p, q, k, v, return_raw=True)
    gbar = s[0, 0] / raw[0, 0]
    assert (gbar > 0).all() and gbar.max() == 1.0 and (gbar == 1.0).sum() == 1
    # width 1: gamma = nu, so gamma_bar = |V_j|^2 / max |V|^2
    p1 = _params(oracle, d=d, n=n, r=5, Br=2, Bud=8, pool_kernel=1)
    s1 = oracle.score(p1, q, k, v)
    nu = (v[0, 0].astype(np.float64) ** 2).sum(-1)
    assert np.allclose(s1[0, 0], raw[0, 0] * nu / nu.max(), rtol=1e-13)
    # equal value norms: the prior is the identity
    vc = np.zeros_like(v)
    vc[..., 3] = 1.5
    vc[0, 0, ::2, 3] = -1.5
    sc = oracle.score(p, q, k, vc)
    assert np.allclose(sc, raw, rtol=1e-13)
    # flag off: no prior
    p0 = _params(oracle, d=d, n=n, r=5, Br=2, Bud=8, flags=0)
    assert np.array_equal(oracle.score(p0, q, k, v), raw)
    # carried score is added after the refinement (Algorithm 1, generation: F_t = ... + F_{t-1})
    prev = np.random.default_rng(18).random((1, 1, n))
    assert np.allclose(oracle.score(p, q, k, v, score_prev=prev), s + prev, rtol=1e-14)


# ---- Algorithm 1: selection --------------------------------------------------------------------------

def test_selection_brute_force(oracle):
    """Over all subsets of the candidates, the chosen B_s maximise the summed score; the result has
    exactly B entries, ascending, and contains the recent window."""
    rng = np.random.default_rng(19)
    for trial in range(20):
        n, Br, Bud = 11, int(rng.integers(0, 4)), int(rng.integers(4, 8))
        Bs = Bud - Br
        s = rng.random((1, 1, n))
        p = _params(oracle, n=n, r=2, Br=Br, Bud=Bud)
        kept = oracle.select(p, s)[0, 0]
        assert len(kept) == Bud and (np.diff(kept) > 0).all()
        assert set(range(n - Br, n)) <= set(kept.tolist())
        chosen = [j for j in kept if j < n - Br]
        assert len(chosen) == Bs
        best = max(itertools.combinations(range(n - Br), Bs), key=lambda c: s[0, 0, list(c)].sum())
        assert set(chosen) == set(best)


def test_selection_against_argsort_ties_and_edges(oracle):
    rng = np.random.default_rng(20)
    B, H, n, Br, Bud = 2, 3, 300, 16, 64
    s = np.round(rng.random((B, H, n)) * 20) / 20            # many ties
    p = _params(oracle, B=B, Hq=H, Hkv=H, n=n, r=4, Br=Br, Bud=Bud)
    kept = oracle.select(p, s)
    for b in range(B):
        for h in range(H):
            cand = s[b, h, : n - Br]
            order = np.lexsort((np.arange(n - Br), -cand))    # score descending, then index ascending
            want = np.sort(np.concatenate([order[: Bud - Br], np.arange(n - Br, n)]))
            assert np.array_equal(kept[b, h], want)
    # B_r = 0, B_s = 0, and n <= budget (keep everything)
    p = _params(oracle, n=n, r=4, Br=0, Bud=10)
    assert np.array_equal(oracle.select(p, s[:1, :1])[0, 0], np.sort(np.lexsort((np.arange(n), -s[0, 0]))[:10]))
    p = _params(oracle, n=n, r=4, Br=10, Bud=10)
    assert np.array_equal(oracle.select(p, s[:1, :1])[0, 0], np.arange(n - 10, n))
    p = _params(oracle, n=n, r=4, Br=10, Bud=n + 5)
    assert np.array_equal(oracle.select(p, s[:1, :1])[0, 0], np.arange(n))
    p = _params(oracle, n=n, r=4, Br=10, Bud=n)
    assert np.array_equal(oracle.select(p, s[:1, :1])[0, 0], np.arange(n))


# ---- Algorithm 1: K <- K_S, V <- V_S -------------------------------------------------------------------

@pytest.mark.parametrize("dt", ["f32", "f16", "bf16"])
def test_compaction_is_a_byte_exact_gather(oracle, dt):
    rng = np.random.default_rng(21)
    B, H, n, d, Bud = 2, 2, 37, 8, 9
    npdt = {"f32": np.float32, "f16": np.float16, "bf16": np.uint16}[dt]
    code = {"f32": oracle.F32, "f16": oracle.F16, "bf16": oracle.BF16}[dt]
    if dt == "bf16":
        k, v = (rng.integers(0, 65536, (B, H, n, d)).astype(np.uint16) for _ in range(2))
    else:
        k, v = (rng.standard_normal((B, H, n, d)).astype(npdt) for _ in range(2))
    idx = np.sort(np.stack([rng.permutation(n)[:Bud] for _ in range(B * H)]).reshape(B, H, Bud), -1).astype(np.int32)
    s = rng.random((B, H, n))
    p = _params(oracle, B=B, Hq=H, Hkv=H, d=d, n=n, r=2, Br=2, Bud=Bud, dtype=code)
    ko, vo, so = oracle.compact(p, k, v, idx, s)
    assert ko.tobytes() == np.take_along_axis(k, idx[..., None], 2).tobytes()
    assert vo.tobytes() == np.take_along_axis(v, idx[..., None], 2).tobytes()
    assert np.array_equal(so, np.take_along_axis(s, idx, 2))


def test_half_and_bf16_widening_is_exact(oracle):
    """Every finite fp16 / bf16 bit pattern must reach the arithmetic unchanged: a single key row and a
    one-hot value row expose the widened element through |V_j|^2 with pool width 1."""
    bits = np.arange(0, 1 << 16, 97, dtype=np.uint16)
    for code, as_f64 in ((oracle.F16, lambda u: u.view(np.float16).astype(np.float64)),
                         (oracle.BF16, lambda u: (u.astype(np.uint32) << 16).view(np.float32).astype(np.float64))):
        with np.errstate(invalid="ignore"):
            vals = as_f64(bits)
        ok = np.isfinite(vals) & (np.abs(vals) < 1e15) & (np.abs(vals) > 1e-15)
        b = bits[ok]
        n = len(b)
        v = np.zeros((1, 1, n, 2), np.uint16)
        v[0, 0, :, 1] = b
        z = np.zeros((1, 1, n, 2), np.uint16)
        q = np.zeros((1, 1, 1, 2), np.uint16)
        if code == oracle.F16:
            v, z, q = v.view(np.float16), z.view(np.float16), q.view(np.float16)
        p = _params(oracle, d=2, n=n, r=1, Br=1, Bud=2, dtype=code, pool_kernel=1)
        s, raw = oracle.score(p, q, z, v, return_raw=True)
        nu = as_f64(b) ** 2
        assert np.allclose(s[0, 0] / raw[0, 0], nu / nu.max(), rtol=1e-14)


# ---- Algorithm 1, generation phase -----------------------------------------------------------------

def test_batched_round_equals_chained_single_steps(oracle):
    """F_t = SGsoftmax(A_t) + F_{t-1}: one call over the last r decode queries equals r one-row calls
    chained through score_prev, each seeing the cache as it was at its own step."""
    n, d, r, Bud, n_total = 60, 8, 5, 16, 500
    q, k, v = _rand((1, 2, r, d), 22), _rand((1, 1, n, d), 23), _rand((1, 1, n, d), 24)
    prev = np.random.default_rng(25).random((1, 1, n))
    prev[..., n - r:] = 0
    pb = _params(oracle, Hq=2, d=d, n=n, r=r, Br=4, Bud=Bud, n_total=n_total, flags=0)
    batched = oracle.score(pb, q, k, v, score_prev=prev)
    F = prev[..., : n - r].copy()
    for t in range(r):
        n_t = n - r + t + 1
        F = np.concatenate([F, np.zeros((1, 1, 1))], -1)
        ps = _params(oracle, Hq=2, d=d, n=n_t, r=1, Br=4, Bud=Bud, n_total=n_total - r + t + 1, flags=0)
        F = oracle.score(ps, np.ascontiguousarray(q[:, :, t:t + 1]), np.ascontiguousarray(k[:, :, :n_t]),
                         np.ascontiguousarray(v[:, :, :n_t]), score_prev=F)
    assert np.allclose(batched, F, rtol=1e-13)


# ---- grouped queries (the paper is silent: consistency only) ------------------------------------------

def test_gqa_is_the_mean_of_per_head_scores(oracle):
    B, Hq, Hkv, d, n, r = 2, 6, 2, 8, 48, 5
    q, k, v = _rand((B, Hq, r, d), 26), _rand((B, Hkv, n, d), 27), _rand((B, Hkv, n, d), 28)
    pg = _params(oracle, B=B, Hq=Hq, Hkv=Hkv, d=d, n=n, r=r, Br=4, Bud=16, flags=0)
    got = oracle.score(pg, q, k, v)
    # the same problem as MHA with each KV head repeated for its 3 query heads
    pm = _params(oracle, B=B, Hq=Hq, Hkv=Hq, d=d, n=n, r=r, Br=4, Bud=16, flags=0)
    per_head = oracle.score(pm, q, np.repeat(k, 3, 1), np.repeat(v, 3, 1))
    assert np.allclose(got, per_head.reshape(B, Hkv, 3, n).mean(2), rtol=1e-13)
    pmx = _params(oracle, B=B, Hq=Hq, Hkv=Hkv, d=d, n=n, r=r, Br=4, Bud=16, flags=oracle.FLAG_GROUP_MAX)
    assert np.allclose(oracle.score(pmx, q, k, v), per_head.reshape(B, Hkv, 3, n).max(2), rtol=1e-13)


# ---- whole step ------------------------------------------------------------------------------------------

def test_evict_composes_score_select_compact(oracle):
    B, Hq, Hkv, d, n, r = 1, 4, 2, 8, 80, 6
    q, k, v = _rand((B, Hq, r, d), 29), _rand((B, Hkv, n, d), 30), _rand((B, Hkv, n, d), 31)
    p = _params(oracle, B=B, Hq=Hq, Hkv=Hkv, d=d, n=n, r=r, Br=8, Bud=24)
    out = oracle.evict(p, q, k, v)
    s = oracle.score(p, q, k, v)
    idx = oracle.select(p, s)
    assert np.array_equal(out["score"], s) and np.array_equal(out["kept_idx"], idx)
    assert np.array_equal(out["k_out"], np.take_along_axis(k, idx[..., None], 2))
    assert np.array_equal(out["v_out"], np.take_along_axis(v, idx[..., None], 2))
    assert np.array_equal(out["score_out"], np.take_along_axis(s, idx, 2))
    # threads do not change the result
    assert np.array_equal(oracle.score(p, q, k, v, nthreads=1), oracle.score(p, q, k, v, nthreads=3))


def test_long_context_workload_matches_the_papers_memory_figure():
    from paper_2506_03762_b200.synth import WORKLOADS
    vals = dict(line.split() for line in open(golden_path("paper_section1_kv_bytes.txt"))
                if line.strip() and not line.startswith("#"))
    w = WORKLOADS["long_32k"]
    kv = 2 * w.n_layers * w.batch * w.n_kv_heads * w.n_ctx * w.head_dim * w.elem_size
    assert w.n_layers == int(vals["layers"]) and kv == int(vals["kv_bytes"]) == 128 * 2 ** 30
