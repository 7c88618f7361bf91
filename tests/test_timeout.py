"""The failure path of the tensor-core scoring kernel: a bounded wait that runs out must be reported through the
status word, the call must return, and the next call on the same workspace must be as good as new.

No GPU is made to hang or fault for this: the library's test hook shortens the limit of the kernel's waits to a few
milliseconds and withholds one set of softmax statistics, so that the wait for them ends by its own limit."""
import pytest
import torch

from paper_2506_03762_b200 import synth

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_clean():
    from paper_2506_03762_b200 import binding as ab
    from tests import parity
    w = synth.WORKLOADS["llama2_7b_4k"].scaled(n_q_heads=8, n_kv_heads=8)
    p = parity.params_of(w)
    q, k, v = synth.make_layer(w, device="cuda")
    ws = ab.alloc_workspace(p, "cuda")
    outs = ab.alloc_outputs(p, "cuda")
    ab.ahakv_evict(p, q, k, v, None, *outs, ws)
    assert ab.ahakv_last_device_status(ws) == ab.OK
    clean = [t.clone() for t in outs]
    try:
        ab.ahakv_test_set_wait(20, True)
        for t in outs:
            t.zero_()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        assert ab.ahakv_evict(p, q, k, v, None, *outs, ws, check=False) == ab.OK      # the fault is on the device
        t1.record()
        assert ab.ahakv_last_device_status(ws) == ab.ERR_TIMEOUT                      # returns: the call ended by itself
        assert t0.elapsed_time(t1) < 2000.0                                           # a few wait limits, not a hang
    finally:
        ab.ahakv_test_set_wait(0, False)
    for t in outs:
        t.zero_()
    ab.ahakv_evict(p, q, k, v, None, *outs, ws)
    assert ab.ahakv_last_device_status(ws) == ab.OK
    for a, b in zip(outs, clean):
        assert torch.equal(a, b)
    # a short limit alone, with nothing withheld, changes nothing
    try:
        ab.ahakv_test_set_wait(50, False)
        ab.ahakv_evict(p, q, k, v, None, *outs, ws)
        assert ab.ahakv_last_device_status(ws) == ab.OK
    finally:
        ab.ahakv_test_set_wait(0, False)
    for a, b in zip(outs, clean):
        assert torch.equal(a, b)
