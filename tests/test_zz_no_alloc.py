"""ahakv_score_static: the scoring entry point for callers that cannot allocate device memory.

A serving process whose memory pool is closed after start-up, or an extension that is handed tensors
but no allocator, cannot give ``ahakv_score`` a workspace.  ``ahakv_score_static`` runs the same kernels
on a fixed scratch array that lives inside the library, so its result must equal ``ahakv_score``'s.
The array is shared by all calls and keeps the previous call's contents, hence two calls in a row.

This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2506_03762_b200 import binding as ab
from paper_2506_03762_b200 import synth
from tests import parity


def test_oversized_problem_is_rejected_before_any_launch():
    from paper_2506_03762_b200 import build
    build.build()
    w = synth.WORKLOADS["long_32k"]
    p = parity.params_of(w)
    assert ab.ahakv_workspace_bytes(p) > ab.ahakv_static_workspace_bytes() == 8 << 20
    before = ab.ahakv_launch_count()
    assert ab.ahakv_score_static(p, 256, 256, 256, None, 256, stream=0, check=False) == ab.ERR_WORKSPACE
    bad = parity.params_of(w.scaled(head_dim=96))
    assert ab.ahakv_score_static(bad, 256, 256, 256, None, 256, stream=0, check=False) == ab.ERR_INVALID_ARG
    assert ab.ahakv_launch_count() == before


@pytest.mark.gpu
@pytest.mark.parametrize("name,over", [
    ("tiny", {}),                                                       # float32, SIMT scoring
    ("llama2_7b_4k", dict(n_q_heads=8, n_kv_heads=8)),                  # float16, tensor-core scoring
    ("decode_round", dict(batch=4)),                                    # bfloat16, GQA, carried score
])
def test_static_scratch_matches_caller_workspace_twice_in_a_row(name, over):
    dev = "cuda"
    w = synth.WORKLOADS[name].scaled(**over)
    p = parity.params_of(w)
    assert ab.ahakv_workspace_bytes(p) <= ab.ahakv_static_workspace_bytes()
    rtol, atol = parity.score_tolerance(p)
    shape = (w.batch, w.n_kv_heads, w.n_ctx)
    for layer in (0, 1):                                # second call: the array still holds the first call's data
        q, k, v = synth.make_layer(w, layer=layer, device=dev)
        prev = synth.make_score_prev(w, device=dev, new_rows=w.obs_window) if w.n_total is not None else None
        want = parity.run_score(p, q, k, v, prev)                       # ahakv_score, caller's workspace
        got = torch.full(shape, float("nan"), dtype=torch.float32, device=dev)
        ab.ahakv_score_static(p, q, k, v, prev, got)
        assert ab.ahakv_static_last_device_status() == ab.OK        # synchronises the stream
        a, b = got.double().cpu().numpy(), want.double().cpu().numpy()
        assert np.isfinite(a).all()
        assert (np.abs(a - b) <= rtol * np.abs(b) + atol).all()
    # and against the oracle on one unit, so that "equal to ahakv_score" cannot hide a common mistake
    op, qn, kn, vn, sp = parity.unit_inputs(p, q, k, v, 0, 0, prev)
    from oracle import ahakv_oracle as orc
    ref = orc.evict(op, qn, kn, vn, sp)
    parity.assert_scores_close(p, got[0, 0].cpu().numpy(), ref["score"][0, 0], "static-scratch score")
