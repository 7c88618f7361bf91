"""The seeded input generators: determinism, shapes, and the planted structure."""
import numpy as np
import torch

from paper_2506_03762_b200 import synth


def test_layers_are_reproducible_and_distinct():
    w = synth.WORKLOADS["llama2_7b_4k"].scaled(n_q_heads=4, n_kv_heads=4, n_ctx=1024)
    a = synth.make_layer(w, layer=3)
    b = synth.make_layer(w, layer=3)
    c = synth.make_layer(w, layer=4)
    for x, y, z in zip(a, b, c):
        assert torch.equal(x, y) and not torch.equal(x, z)
    q, k, v = a
    assert q.shape == (1, 4, 64, 128) and k.shape == v.shape == (1, 4, 1024, 128)
    assert q.dtype == k.dtype == v.dtype == torch.float16


def test_heavy_hitters_are_aligned_with_an_observation_query():
    w = synth.WORKLOADS["llama3_8b_gqa_16k"].scaled(batch=1, n_ctx=2048)
    q, k, v = synth.make_layer(w)
    G = w.group
    qn = torch.nn.functional.normalize(q.float(), dim=-1)          # [1,Hq,r,d]
    kn = torch.nn.functional.normalize(k.float(), dim=-1)          # [1,Hkv,n,d]
    qg = qn.view(1, w.n_kv_heads, G * w.obs_window, w.head_dim)
    cos = torch.einsum("bhsd,bhnd->bhsn", qg, kn).amax(2)          # best alignment per key
    n_hit = round(w.hitter_frac * w.n_ctx)
    top = cos.topk(n_hit, dim=-1)
    assert (top.values > 0.55).all() and (top.values < 0.65).all()
    assert (top.indices < w.n_ctx - w.recent_window).all()
    rest = cos.clone()
    rest.scatter_(-1, top.indices, 0.0)
    assert rest.max() < 0.55
    # outlier channels: 4 per KV head carry 8x the spread
    std = k.float().std(dim=2)[0]                                   # [Hkv,d]
    assert ((std > 4).sum(-1) == w.outlier_channels).all()


def test_tiny_has_a_sink_and_bf16_view_keeps_bits():
    w = synth.WORKLOADS["tiny"]
    q, k, v = synth.make_layer(w)
    assert k.dtype == torch.float32
    assert k[0, :, 0].abs().mean() > 2.5 * k[0, :, 1:].abs().mean()
    t = torch.randn(5, 3).to(torch.bfloat16)
    bits = synth.to_numpy(t)
    assert bits.dtype == np.uint16
    back = torch.from_numpy((bits.astype(np.uint32) << 16).view(np.float32))
    assert torch.equal(back, t.float())


def test_score_prev_zeroes_new_rows():
    w = synth.WORKLOADS["decode_round"].scaled(batch=1)
    s = synth.make_score_prev(w, new_rows=32)
    assert s.shape == (1, 8, 2080) and (s[..., -32:] == 0).all() and (s[..., :-32] >= 0).all()
