"""Operator-level GPU parity: the GEMM and fused-attention tile bodies, called through the C ABI on
their own, against the CPU oracle's `linear`, activations and `attention` (fp64) on the same
bf16-representable inputs.  Shapes span several tiles, ragged tails and the degenerate cases."""
import numpy as np
import pytest

from oracle import vla_oracle as O
from vla_synth.gen import round_to_bf16

pytestmark = pytest.mark.gpu


def _bf16_tensor(x):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda().to(torch.bfloat16)


def _rand(rng, shape, scale=1.0):
    return round_to_bf16((scale * rng.standard_normal(shape)).astype(np.float32))


@pytest.mark.parametrize("m,n,k", [(1, 7, 8), (9, 128, 64), (51, 720, 1024), (80, 256, 192), (176, 960, 2560),
                                   (288, 300, 1000), (1024, 384, 768), (257, 129, 72)])
@pytest.mark.parametrize("act", [0, 1, 2])
def test_linear_matches_oracle(m, n, k, act):
    import torch
    from paper_2609_22335_b200 import api
    rng = np.random.default_rng(m * 1000 + n + k)
    a = _rand(rng, (m, k))
    w = _rand(rng, (n, k), 0.05)
    ref = O.linear(a.astype(np.float64), w.astype(np.float64))
    ref = [ref, O.gelu_tanh(ref), O.silu(ref)][act]
    got = api.op_linear(_bf16_tensor(a), _bf16_tensor(w), act=act)
    torch.cuda.synchronize()
    got = got.cpu().numpy().astype(np.float64)
    # fp32 accumulation of exact bf16 products; the activations use hardware approximations (~2^-11 relative)
    tol = 2e-3 * np.abs(ref).max() + 1e-5
    assert np.max(np.abs(got - ref)) <= tol, (np.max(np.abs(got - ref)), tol)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 1e-3


def test_linear_bf16_output_rounding():
    import torch
    from paper_2609_22335_b200 import api
    rng = np.random.default_rng(5)
    a, w = _rand(rng, (33, 128)), _rand(rng, (200, 128), 0.1)
    f32 = api.op_linear(_bf16_tensor(a), _bf16_tensor(w))
    b16 = api.op_linear(_bf16_tensor(a), _bf16_tensor(w), out_bf16=True)
    torch.cuda.synchronize()
    assert torch.equal(f32.to(torch.bfloat16), b16)            # same values, rounded to nearest even


@pytest.mark.parametrize("tq,tkv,hq,hkv,hd,causal", [
    (9, 80, 4, 4, 64, False), (50, 226, 15, 5, 64, False), (1024, 1024, 12, 12, 64, False), (17, 17, 16, 16, 64, False),
    (96, 96, 16, 8, 128, False), (300, 300, 8, 1, 256, False), (288, 288, 4, 4, 128, True), (130, 130, 2, 2, 32, True),
    (1, 1, 1, 1, 16, False), (256, 193, 3, 3, 80, False), (200, 200, 2, 2, 64, True),
    # few queries and grouped KV heads: query heads of one KV head are folded into one tile (2, 2, 5+1 and 2 per tile)
    (51, 867, 8, 1, 256, False), (9, 80, 4, 2, 64, False), (17, 40, 6, 1, 64, False), (30, 30, 4, 2, 32, True),
    (64, 100, 6, 3, 128, False)])
def test_attention_matches_oracle(tq, tkv, hq, hkv, hd, causal):
    import torch
    from paper_2609_22335_b200 import api
    rng = np.random.default_rng(tq * 7 + tkv + hd)
    q = _rand(rng, (tq, hq, hd), 1.5)          # logits of order 1..10 so the softmax is far from uniform
    k = _rand(rng, (tkv, hkv, hd), 1.5)
    v = _rand(rng, (tkv, hkv, hd))
    ref = O.attention(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), causal=causal)
    got = api.op_attention(_bf16_tensor(q.reshape(tq, -1)), _bf16_tensor(k.reshape(tkv, -1)),
                           _bf16_tensor(v.reshape(tkv, -1)), hq, hkv, hd, causal=causal)
    torch.cuda.synchronize()
    got = got.float().cpu().numpy().reshape(tq, hq, hd).astype(np.float64)
    # P is rounded to bf16 before P.V and the output is bf16: 2^-8 relative each
    assert np.max(np.abs(got - ref)) <= 2e-2 * max(1.0, np.abs(ref).max())
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 1e-2


def test_attention_special_cases_on_gpu():
    import torch
    from paper_2609_22335_b200 import api
    rng = np.random.default_rng(3)
    tq, tkv, h, hd = 5, 70, 2, 64
    q = _rand(rng, (tq, h * hd))
    v = _rand(rng, (tkv, h * hd))
    k0 = np.zeros((tkv, h * hd), np.float32)                    # equal logits -> mean of V rows
    out = api.op_attention(_bf16_tensor(q), _bf16_tensor(k0), _bf16_tensor(v), h, h, hd)
    torch.cuda.synchronize()
    assert np.allclose(out.float().cpu().numpy(), np.broadcast_to(v.mean(0), (tq, h * hd)), atol=2e-2)
    out1 = api.op_attention(_bf16_tensor(q), _bf16_tensor(k0[:1]), _bf16_tensor(v[:1]), h, h, hd)   # one key -> that V row
    torch.cuda.synchronize()
    assert np.array_equal(out1.float().cpu().numpy(), np.broadcast_to(v[0], (tq, h * hd)))


def test_op_argument_checks():
    import torch
    from paper_2609_22335_b200 import api
    lib = api.load_library()
    t = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    s = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    assert lib.vla_op_attention(t.data_ptr(), t.data_ptr(), t.data_ptr(), t.data_ptr(), 64, 64, 1, 1, 60, 0, s.data_ptr(), s.numel(), None) == api.VLA_ERR_INVALID
    assert lib.vla_op_attention(t.data_ptr(), t.data_ptr(), t.data_ptr(), t.data_ptr(), 64, 64, 1, 1, 64, 0, s.data_ptr(), 16, None) == api.VLA_ERR_NOMEM
    assert lib.vla_op_attention(t.data_ptr(), t.data_ptr(), t.data_ptr(), t.data_ptr(), 32, 64, 1, 1, 64, 1, s.data_ptr(), s.numel(), None) == api.VLA_ERR_INVALID
    assert lib.vla_op_linear(t.data_ptr(), t.data_ptr(), None, None, 64, 64, 64, 0, None) == api.VLA_ERR_INVALID
    assert lib.vla_op_linear(t.data_ptr(), t.data_ptr(), None, t.data_ptr(), 64, 64, 60, 0, None) == api.VLA_ERR_INVALID
