"""Seeded synthetic inputs for the eviction step: the only module that both the
CUDA path's callers and the oracle's callers take their inputs from.

It holds none of the method's arithmetic.  It only draws Q/K/V shaped like the
paper's LLaMA-class workloads (Section 5 uses LLaMA-2-7B, LLaMA-3-8B, Qwen2-7B;
Section 1's 128 GB example is LLaMA-2-7B at batch 8 x 32K tokens) and plants
the structure an eviction score has to find: an attention sink, heavy-hitter
keys aligned with an observation query, and outlier key channels.

Everything is a pure function of (workload, layer, seed); tensors come back on
the requested device in the workload's storage dtype, and those exact bits feed
both sides of every parity test.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

BASE_SEED = 20250603

TORCH_DTYPE = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_ctx: int
    dtype: str
    obs_window: int
    recent_window: int
    budget: int
    hitter_frac: float = 0.0        # share of tokens whose key is aligned to an observation query
    hitter_cos: float = 0.6
    sink_scale: float = 1.0         # token 0's key is multiplied by this
    outlier_channels: int = 0       # key channels per KV head multiplied by outlier_scale
    outlier_scale: float = 8.0
    n_layers: int = 1
    value_prior: bool = True
    pool_kernel: int = 7
    n_total: int | None = None      # None: prefill (n_total = n_ctx)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def n_keep(self) -> int:
        return min(self.n_ctx, self.budget)

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations of the benchmark definition.
WORKLOADS = {
    "tiny": Workload("tiny", 1, 4, 4, 64, 512, "f32", 32, 32, 128, sink_scale=4.0),
    "llama2_7b_4k": Workload("llama2_7b_4k", 1, 32, 32, 128, 4096, "f16", 64, 64, 512, hitter_frac=0.02),
    "llama3_8b_gqa_16k": Workload("llama3_8b_gqa_16k", 4, 32, 8, 128, 16384, "bf16", 64, 128, 1024,
                                  hitter_frac=0.01, outlier_channels=4),
    "long_32k": Workload("long_32k", 8, 32, 32, 128, 32768, "f16", 128, 128, 2048, hitter_frac=0.02,
                         n_layers=32),
    "decode_round": Workload("decode_round", 16, 32, 8, 128, 2080, "bf16", 32, 64, 2048,
                             value_prior=False, n_total=32768 + 32),
}


def _generator(device, seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) * 1000003 + int(stream))
    return g


def make_layer(w: Workload, layer: int = 0, device="cpu", seed: int = BASE_SEED):
    """Returns (q_obs [B,Hq,r,d], k [B,Hkv,n,d], v [B,Hkv,n,d]) for one layer."""
    dev = torch.device(device)
    dt = TORCH_DTYPE[w.dtype]
    g = _generator(dev, seed, 7919 * layer + 1)
    B, Hq, Hkv, d, n, r, G = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.n_ctx, w.obs_window, w.group
    q = torch.randn((B, Hq, r, d), generator=g, device=dev, dtype=torch.float32)
    k = torch.randn((B, Hkv, n, d), generator=g, device=dev, dtype=dt)
    v = torch.randn((B, Hkv, n, d), generator=g, device=dev, dtype=dt)

    if w.sink_scale != 1.0:
        k[:, :, 0, :] *= w.sink_scale

    if w.outlier_channels > 0:
        for h in range(Hkv):
            ch = torch.randperm(d, generator=g, device=dev)[: w.outlier_channels]
            k[:, h, :, ch] *= w.outlier_scale

    n_hit = int(round(w.hitter_frac * n))
    if n_hit > 0:
        n_cand = n - w.recent_window
        # positions without replacement, uniform over the tokens outside the recent window
        pos = torch.rand((B, Hkv, n_cand), generator=g, device=dev).topk(n_hit, dim=-1).indices
        # each hitter aligns with one (query head of the group, observation row)
        which_q = torch.randint(0, G, (B, Hkv, n_hit), generator=g, device=dev)
        which_i = torch.randint(0, r, (B, Hkv, n_hit), generator=g, device=dev)
        hq = torch.arange(Hkv, device=dev).view(1, Hkv, 1) * G + which_q
        bb = torch.arange(B, device=dev).view(B, 1, 1).expand_as(hq)
        u = q[bb, hq, which_i]                                   # [B,Hkv,n_hit,d]
        u = u / u.norm(dim=-1, keepdim=True)
        hh = torch.arange(Hkv, device=dev).view(1, Hkv, 1).expand_as(pos)
        rows = k[bb, hh, pos].float()
        z = rows - (rows * u).sum(-1, keepdim=True) * u          # part of the old key orthogonal to u
        z = z / z.norm(dim=-1, keepdim=True)
        s = (1.0 - w.hitter_cos ** 2) ** 0.5
        k[bb, hh, pos] = ((d ** 0.5) * (w.hitter_cos * u + s * z)).to(dt)

    return q.to(dt), k, v


def make_decode_step(w: Workload, step: int, device="cpu", seed: int = BASE_SEED):
    """One generation step's (q [B,Hq,1,d], k [B,Hkv,1,d], v [B,Hkv,1,d]) ~ N(0,1)."""
    dev = torch.device(device)
    dt = TORCH_DTYPE[w.dtype]
    g = _generator(dev, seed, 104729 + step)
    q = torch.randn((w.batch, w.n_q_heads, 1, w.head_dim), generator=g, device=dev, dtype=dt)
    k = torch.randn((w.batch, w.n_kv_heads, 1, w.head_dim), generator=g, device=dev, dtype=dt)
    v = torch.randn((w.batch, w.n_kv_heads, 1, w.head_dim), generator=g, device=dev, dtype=dt)
    return q, k, v


def make_score_prev(w: Workload, device="cpu", seed: int = BASE_SEED, new_rows: int = 0):
    """A carried score F_{t-1} [B,Hkv,n] >= 0 (float32) with zeros for the newest rows."""
    dev = torch.device(device)
    g = _generator(dev, seed, 15485863)
    s = torch.rand((w.batch, w.n_kv_heads, w.n_ctx), generator=g, device=dev, dtype=torch.float32)
    s = s * (w.obs_window / w.n_ctx)
    if new_rows > 0:
        s[..., w.n_ctx - new_rows:] = 0.0
    return s


def to_numpy(t: torch.Tensor):
    """Host numpy view of a tensor's exact bits (bfloat16 comes back as uint16)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view("uint16")
    return t.numpy()
