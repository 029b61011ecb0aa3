"""The allocation-free attention entry point against the ordinary one.

Some users of the library may not allocate GPU memory at all once they are running (a robot's
real-time control loop with a fixed memory budget, a plugin whose host owns every allocation).
`vla_op_attention_static` serves them: its scratch is a fixed array inside the library.  This test
calls it through the C ABI twice in a row -- the second call on a smaller problem, so anything the
first call left in the shared array would show -- and checks both results against
`vla_op_attention` with caller-provided scratch.  Collected last on purpose: a failure here must
not hide the other GPU tests from a run that stops at the first failure."""
import numpy as np
import pytest

from vla_synth.gen import round_to_bf16

pytestmark = pytest.mark.gpu


def _case(rng, tq, tkv, hq, hkv, hd):
    import torch
    mk = lambda *s, sc=1.0: torch.from_numpy(round_to_bf16((sc * rng.standard_normal(s)).astype(np.float32))).cuda().to(torch.bfloat16)
    return mk(tq, hq * hd, sc=1.5), mk(tkv, hkv * hd, sc=1.5), mk(tkv, hkv * hd)


def test_static_scratch_attention_matches_regular_entry_point_twice():
    import torch
    from paper_2609_22335_b200 import api
    rng = np.random.default_rng(42)
    for (tq, tkv, hq, hkv, hd, causal) in [(300, 300, 8, 4, 64, False), (50, 97, 4, 2, 128, False)]:
        q, k, v = _case(rng, tq, tkv, hq, hkv, hd)
        ref = api.op_attention(q, k, v, hq, hkv, hd, causal=causal)
        out = torch.empty_like(q)
        api.op_attention_static(q, k, v, out, hq, hkv, hd, causal=causal)
        torch.cuda.synchronize()
        a, b = out.float().cpu().numpy(), ref.float().cpu().numpy()
        assert np.isfinite(a).all()
        # same tolerance as the operator tests use against the oracle
        assert np.max(np.abs(a - b)) <= 2e-2 * max(1.0, float(np.abs(b).max()))
        assert np.linalg.norm(a - b) / np.linalg.norm(b) < 1e-2


def test_static_scratch_limit_is_enforced():
    import ctypes as C
    import torch
    from paper_2609_22335_b200 import api
    lib = api.load_library()
    cap = C.c_size_t(0)
    assert lib.vla_op_attention_static_capacity(C.byref(cap)) == api.VLA_OK and cap.value == 256 + (4 << 20)
    # 32 KV heads x 128 over 4096 keys needs 32 MiB of transposed V: refused, nothing runs
    t = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    rc = lib.vla_op_attention_static(t.data_ptr(), t.data_ptr(), t.data_ptr(), t.data_ptr(), 4096, 4096, 32, 32, 128, 0, None)
    assert rc == api.VLA_ERR_NOMEM
