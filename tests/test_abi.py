"""The C ABI without a GPU: the library loads, exports what the header declares, and rejects bad
arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2506_03762_b200 import binding as ab
from tests.conftest import ROOT


@pytest.fixture(scope="module")
def lib():
    from paper_2506_03762_b200 import build
    build.build()
    return ab.lib()


def _good(**kw):
    base = dict(batch=1, n_q_heads=4, n_kv_heads=2, head_dim=128, n_ctx=1000, obs_window=32,
                recent_window=16, budget=128, dtype=ab.F16)
    base.update(kw)
    return ab.Params(**base)


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "ahakv.h")).read()
    declared = set(re.findall(r"\b(ahakv_[a-z_]+)\s*\(", header))
    assert {"ahakv_score", "ahakv_select", "ahakv_compact", "ahakv_evict", "ahakv_workspace_bytes"} <= declared
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in ahakv.h but not exported"
    assert declared <= set(ab.SIGNATURES), "the binding must cover every entry point"


def test_struct_mirror_matches_the_header_layout(lib):
    # int32 x5, int64, int32 x5, float, int32, uint32, 9 x int64
    assert ctypes.sizeof(ab.CParams) == 20 + 4 + 8 + 20 + 4 + 4 + 4 + 72 == 136
    assert ab.CParams.n_total.offset == 24 and ab.CParams.q_stride.offset == 64


def test_lambda_helper(lib):
    import math
    assert math.isclose(ab.ahakv_lambda(32768, 2048, 128), math.sqrt(2 * math.log(16) / 128), rel_tol=1e-15)
    assert math.isclose(ab.ahakv_lambda(100, 200, 64), 0.125)


def test_workspace_query(lib):
    assert ab.ahakv_workspace_bytes(_good()) > 0
    assert ab.ahakv_workspace_bytes(_good()) % 256 == 0
    big = ab.ahakv_workspace_bytes(_good(n_ctx=32768, obs_window=128, n_q_heads=32, n_kv_heads=32, batch=8))
    assert big > ab.ahakv_workspace_bytes(_good())
    assert big < 1 << 30


@pytest.mark.parametrize("bad", [
    dict(batch=0), dict(n_q_heads=3), dict(head_dim=96), dict(n_ctx=0), dict(n_total=10),
    dict(obs_window=0), dict(obs_window=2000), dict(obs_window=200), dict(recent_window=-1),
    dict(recent_window=129), dict(budget=0), dict(dtype=7), dict(scale_mode=3),
    dict(scale_mode=ab.SCALE_FIXED, scale=0.0), dict(pool_kernel=4), dict(pool_kernel=0),
    dict(flags=64), dict(k_stride=(1, 2, 3)), dict(k_stride=(128000, 128, 64)),
])
def test_bad_parameters_are_rejected_on_the_host(lib, bad):
    p = _good(**bad)
    assert ab.ahakv_workspace_bytes(p) == 0
    # pointers are never touched when the parameters are wrong
    assert ab.ahakv_score(p, 256, 256, 256, None, 256, 256, 1 << 40, stream=0, check=False) == ab.ERR_INVALID_ARG
    assert ab.ahakv_evict(p, 256, 256, 256, None, 256, 256, None, 256, 256, 1 << 40, stream=0,
                          check=False) == ab.ERR_INVALID_ARG


def test_bad_pointers_and_workspace_are_rejected_on_the_host(lib):
    p = _good()
    need = ab.ahakv_workspace_bytes(p)
    sc = lambda **kw: ab.ahakv_score(p, kw.get("q", 256), kw.get("k", 256), kw.get("v", 256), None,
                                     kw.get("score", 256), kw.get("ws", 256), kw.get("nbytes", need),
                                     stream=0, check=False)
    assert sc(q=None) == ab.ERR_INVALID_ARG
    assert sc(k=8) == ab.ERR_INVALID_ARG                  # not 16-byte aligned
    assert sc(v=None) == ab.ERR_INVALID_ARG               # value prior is on
    assert sc(score=None) == ab.ERR_INVALID_ARG
    assert sc(ws=None) == ab.ERR_WORKSPACE
    assert sc(ws=128) == ab.ERR_WORKSPACE                 # not 256-byte aligned
    assert sc(nbytes=need - 1) == ab.ERR_WORKSPACE
    assert ab.ahakv_select(p, None, 256, 256, need, stream=0, check=False) == ab.ERR_INVALID_ARG
    assert ab.ahakv_compact(p, 256, 256, 256, 256, 256, 256, None, stream=0, check=False) == ab.ERR_INVALID_ARG
    assert ab.ahakv_compact(p, 256, None, None, 256, 256, 256, None, stream=0, check=False) == ab.ERR_INVALID_ARG
    assert ab.ahakv_evict(p, 256, 256, 256, None, 256, 256, None, None, 256, need, stream=0,
                          check=False) == ab.ERR_INVALID_ARG
    assert ab.ahakv_workspace_bytes(_good(flags=ab.FLAG_GROUP_MAX)) > 0      # pooling by maximum is a legal request


def test_the_generation_step_entry_points_reject_bad_requests_on_the_host(lib):
    step = _good(n_ctx=257, obs_window=1, recent_window=16, budget=256, flags=0)
    slots = lambda p=step, **kw: ab.ahakv_step_slots(p, kw.get("q", 256), kw.get("k_t", 256), kw.get("v_t", 256),
                                                     kw.get("k", 256), kw.get("v", 256), kw.get("score", 256),
                                                     kw.get("pos", 256), kw.get("free", 256), stream=0, check=False)
    assert slots(q=None) == ab.ERR_INVALID_ARG
    assert slots(k_t=8) == ab.ERR_INVALID_ARG             # not 16-byte aligned
    assert slots(pos=None) == ab.ERR_INVALID_ARG
    assert slots(free=2) == ab.ERR_INVALID_ARG            # not 4-byte aligned
    # a slot cache holds budget + 1 rows and takes one query row
    assert slots(_good(n_ctx=300, obs_window=1, recent_window=16, budget=256, flags=0)) == ab.ERR_INVALID_ARG
    assert slots(_good(n_ctx=257, obs_window=2, recent_window=16, budget=256, flags=0)) == ab.ERR_INVALID_ARG
    # the generation phase has no value prior
    assert slots(_good(n_ctx=257, obs_window=1, recent_window=16, budget=256)) == ab.ERR_UNSUPPORTED
    assert ab.ahakv_score_step(_good(n_ctx=257, obs_window=2, recent_window=16, budget=256, flags=0), 256, 256, None,
                               256, stream=0, check=False) == ab.ERR_INVALID_ARG
    assert ab.ahakv_compact_inplace(step, 256, None, None, 256, stream=0, check=False) == ab.ERR_INVALID_ARG


def test_status_strings_and_errors(lib):
    assert ab.status_string(ab.OK) == "ok"
    assert "wait" in ab.status_string(ab.ERR_TIMEOUT)
    with pytest.raises(ab.AhakvError):
        ab.ahakv_score(_good(batch=0), 256, 256, 256, None, 256, 256, 1 << 40, stream=0)
    assert ab.ahakv_launch_count() == 0
