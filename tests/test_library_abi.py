"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its
host-side program compiler accepts the five workloads and rejects bad descriptions."""
import re
import os
import ctypes as C

import pytest

from paper_2609_22335_b200 import api, build
from vla_synth.configs import CONFIGS, CFG1, CFG4

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.load_library()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "vla.h")).read()
    declared = set(re.findall(r"\b(vla_[a-z_]+)\s*\(", header))
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


@pytest.mark.parametrize("name", list(CONFIGS))
def test_arena_size_for_every_workload(lib, name):
    m = CONFIGS[name]
    d = api.make_desc(m)
    o = api.vla_runtime_opts()
    o.n_streams, o.ring_depth, o.mode = m.n_streams, 2, 0
    nbytes = api.vla_required_arena_bytes(d, o)
    from vla_synth.gen import make_weights
    wbytes = make_weights(m).nbytes_bf16()
    assert nbytes > wbytes * 0.99 and nbytes < 40e9          # weights fit, far below 180 GB


def test_invalid_descriptions_are_rejected(lib):
    o = api.vla_runtime_opts()
    o.n_streams, o.ring_depth = 2, 2
    out = C.c_size_t(0)
    for field, value in (("patch", 7), ("hq", 3), ("head", 9), ("n_steps", 0), ("shuffle", 3), ("act_layers", 17)):
        d = api.make_desc(CFG4 if field == "act_layers" else CFG1)
        setattr(d, field, value)
        assert lib.vla_required_arena_bytes(C.byref(d), C.byref(o), C.byref(out)) == api.VLA_ERR_INVALID, field
    d = api.make_desc(CFG1)
    o.ring_depth = 1
    assert lib.vla_required_arena_bytes(C.byref(d), C.byref(o), C.byref(out)) == api.VLA_ERR_INVALID
    assert lib.vla_required_arena_bytes(None, C.byref(o), C.byref(out)) == api.VLA_ERR_INVALID


def test_null_context_calls_fail_cleanly(lib):
    assert lib.vla_poll_actions(None, 0, None, None) == api.VLA_ERR_INVALID
    assert lib.vla_destroy(None) == api.VLA_ERR_INVALID
    assert lib.vla_wait_idle(None, 1) == api.VLA_ERR_INVALID
