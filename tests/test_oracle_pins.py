"""Pins of the CPU oracle against things other than itself: brute-force loops,
closed forms, invariants and library routines (CPU only)."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import vla_oracle as O
from vla_synth.configs import CFG1, CFG2, CFG3, CFG4, CFG5, mini
from vla_synth.gen import make_weights, frame_inputs

F64 = np.float64
rng = np.random.default_rng(1234)


# ------------------------------------------------------------------ linear
def test_linear_bruteforce_and_library():
    x = rng.standard_normal((5, 7))
    w = rng.standard_normal((3, 7))
    y = O.linear(x, w)
    for i in range(5):
        for o in range(3):
            acc = 0.0
            for k in range(7):
                acc += x[i, k] * w[o, k]
            assert abs(y[i, o] - acc) < 1e-12
    yt = torch.nn.functional.linear(torch.from_numpy(x), torch.from_numpy(w)).numpy()
    assert np.allclose(y, yt, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ softmax / attention
def _attention_loops(q, k, v, causal):
    tq, hq, hd = q.shape
    tkv, hkv, _ = k.shape
    out = np.zeros_like(q)
    for h in range(hq):
        g = (h * hkv) // hq
        for i in range(tq):
            logits = []
            for j in range(tkv):
                if causal and j > i:
                    continue
                logits.append((j, sum(q[i, h, c] * k[j, g, c] for c in range(hd)) / math.sqrt(hd)))
            mx = max(l for _, l in logits)
            den = sum(math.exp(l - mx) for _, l in logits)
            for j, l in logits:
                p = math.exp(l - mx) / den
                for c in range(hd):
                    out[i, h, c] += p * v[j, g, c]
    return out


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("hq,hkv", [(4, 4), (6, 2), (4, 1)])
def test_attention_bruteforce(causal, hq, hkv):
    t = 6
    q = 3.0 * rng.standard_normal((t, hq, 8))      # logits of order 1..10 so softmax is far from uniform
    k = 3.0 * rng.standard_normal((t, hkv, 8))
    v = rng.standard_normal((t, hkv, 8))
    a = O.attention(q, k, v, causal=causal)
    b = _attention_loops(q, k, v, causal)
    assert np.allclose(a, b, rtol=1e-10, atol=1e-12)


def test_attention_cross_lengths_bruteforce():
    q = 2.0 * rng.standard_normal((3, 4, 8))
    k = 2.0 * rng.standard_normal((9, 2, 8))
    v = rng.standard_normal((9, 2, 8))
    assert np.allclose(O.attention(q, k, v), _attention_loops(q, k, v, False), rtol=1e-10, atol=1e-12)


def test_softmax_rows_sum_to_one_and_shift_invariant():
    s = 10.0 * rng.standard_normal((7, 13))
    p = O.softmax_rows(s)
    assert np.allclose(p.sum(-1), 1.0, atol=1e-12)
    assert np.allclose(p, O.softmax_rows(s + 1000.0), atol=1e-12)
    p32 = O.softmax_rows(s.astype(np.float32))
    assert np.allclose(p32.sum(-1), 1.0, atol=1e-6)


def test_attention_special_cases():
    t, h, hd = 5, 2, 4
    v = rng.standard_normal((t, h, hd))
    q = rng.standard_normal((3, h, hd))
    k_equal = np.zeros((t, h, hd))                 # all-equal logits -> mean of V rows
    assert np.allclose(O.attention(q, k_equal, v), np.broadcast_to(v.mean(0), (3, h, hd)), atol=1e-12)
    k1 = rng.standard_normal((1, h, hd))           # one key -> that V row
    assert np.allclose(O.attention(q, k1, v[:1]), np.broadcast_to(v[0], (3, h, hd)), atol=1e-12)


def test_attention_gqa_reduces_to_mha_and_matches_sdpa():
    t, hq, hkv, hd = 7, 6, 2, 8
    q = 2.0 * rng.standard_normal((t, hq, hd))
    k = 2.0 * rng.standard_normal((t, hkv, hd))
    v = rng.standard_normal((t, hkv, hd))
    rep = hq // hkv
    a = O.attention(q, k, v)
    b = O.attention(q, np.repeat(k, rep, axis=1), np.repeat(v, rep, axis=1))
    assert np.allclose(a, b, atol=1e-12)
    for causal in (False, True):
        ours = O.attention(q, np.repeat(k, rep, 1), np.repeat(v, rep, 1), causal=causal)
        tq = torch.from_numpy(q).permute(1, 0, 2)[None]
        tk = torch.from_numpy(np.repeat(k, rep, 1)).permute(1, 0, 2)[None]
        tv = torch.from_numpy(np.repeat(v, rep, 1)).permute(1, 0, 2)[None]
        ref = F.scaled_dot_product_attention(tq, tk, tv, is_causal=causal)[0].permute(1, 0, 2).numpy()
        assert np.allclose(ours, ref, rtol=1e-9, atol=1e-11)


def test_attention_causal_ignores_future_and_bidirectional_is_permutation_equivariant():
    t, h, hd = 6, 2, 4
    q = rng.standard_normal((t, h, hd)); k = rng.standard_normal((t, h, hd)); v = rng.standard_normal((t, h, hd))
    a = O.attention(q, k, v, causal=True)
    k2, v2 = k.copy(), v.copy()
    k2[4:] += 5.0; v2[4:] -= 3.0
    b = O.attention(q, k2, v2, causal=True)
    assert np.array_equal(a[:4], b[:4]) and not np.allclose(a[4:], b[4:])
    perm = rng.permutation(t)
    c = O.attention(q[perm], k[perm], v[perm])
    assert np.allclose(c, O.attention(q, k, v)[perm], atol=1e-12)


# ------------------------------------------------------------------ norms / activations
def test_rmsnorm():
    x = rng.standard_normal((4, 64)) * 3.0
    g = np.ones(64)
    y = O.rmsnorm(x, g)
    assert np.allclose((y * y).mean(-1), 1.0, atol=1e-5)
    assert np.allclose(O.rmsnorm(7.5 * x, g), y, atol=1e-6)
    g2 = rng.standard_normal(64)
    ref = F.rms_norm(torch.from_numpy(x), (64,), torch.from_numpy(g2), eps=1e-6).numpy()
    assert np.allclose(O.rmsnorm(x, g2), ref, rtol=1e-10, atol=1e-12)


def test_gelu_silu():
    x = np.linspace(-6, 6, 241)
    for f in (O.gelu_tanh, O.silu):
        assert np.allclose(f(x) - f(-x), x, atol=1e-12)      # f(x) - f(-x) = x
        assert f(np.zeros(1))[0] == 0.0
    assert np.allclose(O.gelu_tanh(x), F.gelu(torch.from_numpy(x), approximate="tanh").numpy(), atol=1e-12)
    assert np.allclose(O.silu(x), F.silu(torch.from_numpy(x)).numpy(), atol=1e-12)
    # the tanh form stays within 5e-4 of the erf form
    assert np.max(np.abs(O.gelu_tanh(x) - F.gelu(torch.from_numpy(x)).numpy())) < 5e-4


def test_gated_mlp_against_loops():
    d, hdim = 6, 5
    x = rng.standard_normal((3, d))
    w = {"p.wg": rng.standard_normal((hdim, d)), "p.wu": rng.standard_normal((hdim, d)),
         "p.wd": rng.standard_normal((d, hdim)), "p.w1": rng.standard_normal((hdim, d)),
         "p.w2": rng.standard_normal((d, hdim))}
    for kind in ("swiglu", "geglu", "gelu"):
        y = O.mlp(x, w, "p.", kind, F64)
        for i in range(3):
            hid = []
            for j in range(hdim):
                if kind == "gelu":
                    a = float(x[i] @ w["p.w1"][j])
                    hid.append(float(F.gelu(torch.tensor(a, dtype=torch.float64), approximate="tanh")))
                else:
                    g_ = float(x[i] @ w["p.wg"][j]); u_ = float(x[i] @ w["p.wu"][j])
                    tg = torch.tensor(g_, dtype=torch.float64)
                    a = float(F.silu(tg)) if kind == "swiglu" else float(F.gelu(tg, approximate="tanh"))
                    hid.append(a * u_)
            wd = w["p.w2"] if kind == "gelu" else w["p.wd"]
            for o in range(d):
                assert abs(y[i, o] - sum(hid[j] * wd[o, j] for j in range(hdim))) < 1e-10


# ------------------------------------------------------------------ RoPE
def test_rope_properties():
    t, h, hd = 5, 2, 16
    x = rng.standard_normal((t, h, hd))
    assert np.allclose(O.rope(x, np.zeros(t)), x)                                  # position 0 = identity
    y = O.rope(x, np.arange(t) + 3)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1))     # norm preserving
    q = rng.standard_normal((1, 1, hd)); k = rng.standard_normal((1, 1, hd))
    d1 = (O.rope(q, [7]) * O.rope(k, [4])).sum()
    d2 = (O.rope(q, [103]) * O.rope(k, [100])).sum()
    assert abs(d1 - d2) < 1e-9                                                     # depends on m - n only
    # pair (i, i+hd/2) rotates by pos * base^(-2i/hd)
    e = np.zeros((1, 1, hd)); e[0, 0, 3] = 1.0
    r = O.rope(e, [2.0])
    ang = 2.0 * 10000.0 ** (-2 * 3 / hd)
    assert abs(r[0, 0, 3] - math.cos(ang)) < 1e-12 and abs(r[0, 0, 3 + hd // 2] - math.sin(ang)) < 1e-12


# ------------------------------------------------------------------ patchify / shuffle / timestep
def test_patchify_matches_strided_conv():
    n, p, side, d = 2, 4, 16, 5
    img = rng.random((n, 3, side, side))
    wmat = rng.standard_normal((d, 3 * p * p))
    ours = O.linear(O.patchify(img, p), wmat)                                       # [n, T, d]
    conv = F.conv2d(torch.from_numpy(img), torch.from_numpy(wmat.reshape(d, 3, p, p)), stride=p)
    ref = conv.flatten(2).permute(0, 2, 1).numpy()
    assert np.allclose(ours, ref, atol=1e-12)


def test_pixel_shuffle_matches_unshuffle_up_to_documented_channel_order():
    grid, s, d = 8, 2, 3
    tok = rng.standard_normal((grid * grid, d))
    ours = O.pixel_shuffle_tokens(tok, grid, s)                                     # [(g/s)^2, (dy,dx,c)]
    t = torch.from_numpy(tok).reshape(grid, grid, d).permute(2, 0, 1)[None]         # [1,d,g,g]
    un = F.pixel_unshuffle(t, s)[0]                                                 # [(c,dy,dx), g/s, g/s]
    ref = un.reshape(d, s, s, grid // s, grid // s).permute(3, 4, 1, 2, 0).reshape((grid // s) ** 2, s * s * d)
    assert np.array_equal(ours, ref.numpy())
    # direct index check of one element
    Y, X, dy, dx, c = 1, 2, 1, 0, 2
    assert ours[Y * (grid // s) + X, (dy * s + dx) * d + c] == tok[(Y * s + dy) * grid + (X * s + dx), c]


def test_timestep_embedding():
    e0 = O.timestep_embedding(0.0, 32, F64)
    assert np.all(e0[:16] == 0.0) and np.all(e0[16:] == 1.0)
    e = O.timestep_embedding(437.0, 32, F64)
    assert abs((e * e).sum() - 16.0) < 1e-9
    assert abs(e[0] - math.sin(437.0)) < 1e-12                                       # w_0 = 1
    assert abs(e[16 + 8] - math.cos(437.0 * 10000 ** (-8 / 16))) < 1e-12


# ------------------------------------------------------------------ solvers
def test_euler_closed_form_linear_field():
    lam, b, n = -0.7, 0.3, 8
    x0 = rng.standard_normal((4, 3))
    xn = O.euler_solve(lambda x, t: lam * x + b, x0, n)
    g = (1 + lam / n) ** n
    assert np.allclose(xn, g * x0 + b * (g - 1) / lam, atol=1e-12)
    vconst = rng.standard_normal((4, 3))
    assert np.allclose(O.euler_solve(lambda x, t: vconst, x0, 5), x0 + vconst, atol=1e-12)
    big = O.euler_solve(lambda x, t: lam * x, x0, 20000)
    assert np.allclose(big, math.exp(lam) * x0, atol=1e-4)
    seen = []
    O.euler_solve(lambda x, t: (seen.append(t), x * 0)[1], x0, 4)
    assert seen == [0.0, 0.25, 0.5, 0.75]


def test_ddim_schedule_and_telescoping():
    ab = O.ddim_alpha_bar(100)
    assert np.all(np.diff(ab) < 0)

    def c(u):
        return math.cos((u + 0.008) / 1.008 * math.pi / 2) ** 2
    # while beta is unclipped the product telescopes to c((tau+1)/T)/c(0)
    for tau in (0, 10, 50, 90):
        assert abs(ab[tau] - c((tau + 1) / 100) / c(0.0)) < 1e-12
    assert abs(ab[0] - 0.99937) < 1e-5 and abs(ab[90] - 0.01954) < 1e-5
    assert O.ddim_timesteps(10) == [90, 80, 70, 60, 50, 40, 30, 20, 10, 0]
    xT = rng.standard_normal((3, 2))
    out = O.ddim_solve(lambda x, tau: np.zeros_like(x), xT, 10)
    assert np.allclose(out, xT / math.sqrt(ab[90]), rtol=1e-12)                      # eps = 0 telescopes
    xstar = rng.standard_normal((3, 2))

    def eps_for_target(x, tau):                                                      # makes the x0 estimate equal x*
        return (x - math.sqrt(ab[tau]) * xstar) / math.sqrt(1 - ab[tau])
    assert np.allclose(O.ddim_solve(eps_for_target, xT, 10), xstar, atol=1e-10)
    one = O.ddim_solve(lambda x, tau: 0.5 * x, xT, 1)                                # single step from tau = 0, prev alpha = 1
    assert np.allclose(one, (xT - math.sqrt(1 - ab[0]) * 0.5 * xT) / math.sqrt(ab[0]), atol=1e-12)


# ------------------------------------------------------------------ whole towers
TINY = {
    "A": CFG1,
    "B_nope": mini(CFG2, img=64, vis_layers=1, llm_layers=2, act_layers=2, horizon=6, n_steps=3, vocab=512),
    "C": mini(CFG3, img=56, vis_layers=1, vis_d=144, vis_heads=2, vis_mlp=256, llm_layers=1, d=256, hq=4, hkv=2,
              hd=64, mlp=512, act_layers=2, act_d=128, act_heads=4, act_mlp=256, vocab=512),
    "B_rope": mini(CFG4, n_cam=2, img=28, vis_layers=1, vis_d=144, vis_heads=2, vis_mlp=256, llm_layers=2, d=128,
                   hq=2, hkv=1, hd=64, mlp=256, act_layers=2, act_d=64, act_mlp=128, horizon=5, n_steps=3, vocab=512),
    "D": mini(CFG5, img=56, vis_layers=1, vis_d=128, vis_heads=2, vis_mlp=256, llm_layers=2, d=128, hq=2, hkv=2,
              hd=64, mlp=256, act_layers=2, act_d=64, act_heads=2, act_mlp=128, vocab=512),
}


def _zero_branch_outputs(w, prefixes=("act.",)):
    for name in w.names():
        leaf = name.split(".")[-1]
        if name.startswith(prefixes) and leaf in ("wo", "co", "w2", "wd"):
            w.override(name, np.zeros(w.shapes[name], np.float32))


@pytest.mark.parametrize("key", list(TINY))
def test_head_with_zeroed_branches_is_closed_form(key):
    m = TINY[key]
    w = make_weights(m, seed=3)
    _zero_branch_outputs(w)
    fr = frame_inputs(m, 0, 0, seed=3)
    vlm = O.vlm_forward(m, w, fr["image"], fr["text"], F64)
    x = fr["noise"].astype(F64)
    t_arg = 250.0
    v = O.head_velocity(m, w, vlm, fr["state"], x, t_arg, F64)
    # closed form: tokens -> final RMSNorm -> W_out, written out independently here
    e = np.concatenate([np.sin(t_arg * np.exp(-math.log(10000.0) * np.arange(m.act_d // 2) / (m.act_d // 2))),
                        np.cos(t_arg * np.exp(-math.log(10000.0) * np.arange(m.act_d // 2) / (m.act_d // 2)))])
    h1 = w["act.t1"].astype(F64) @ e
    c_t = w["act.t2"].astype(F64) @ (h1 / (1 + np.exp(-h1)))
    rows = []
    for i in range(m.horizon):
        tok = w["act.in"].astype(F64) @ x[i]
        if m.head in ("A", "B"):
            tok = tok + c_t
        if m.head_pos_table:
            tok = tok + w["act.pos"][m.act_first + i].astype(F64)
        n = tok / math.sqrt(float(np.mean(tok * tok)) + 1e-6)
        rows.append(w["act.out"].astype(F64) @ n)
    assert np.allclose(v, np.stack(rows), rtol=1e-9, atol=1e-12)


@pytest.mark.parametrize("key", list(TINY))
def test_zero_output_projection(key):
    m = TINY[key]
    w = make_weights(m, seed=4)
    w.override("act.out", np.zeros(w.shapes["act.out"], np.float32))
    fr = frame_inputs(m, 1, 2, seed=4)
    chunk = O.action_chunk(m, w, fr, F64)
    if m.solver == "euler":
        assert np.allclose(chunk, fr["noise"], atol=1e-12)                           # v = 0 -> chunk = noise
    else:
        ab = O.ddim_alpha_bar()
        assert np.allclose(chunk, fr["noise"].astype(F64) / math.sqrt(ab[O.ddim_timesteps(m.n_steps)[0]]), rtol=1e-9)


def test_vlm_with_zeroed_branches_is_normed_prefix():
    m = TINY["B_rope"]
    w = make_weights(m, seed=5)
    _zero_branch_outputs(w, prefixes=("llm.", "vis."))
    fr = frame_inputs(m, 0, 0, seed=5)
    out = O.vlm_forward(m, w, fr["image"], fr["text"], F64)
    pre = out["prefix"]
    assert np.allclose(out["hidden"], pre / np.sqrt((pre * pre).mean(-1, keepdims=True) + 1e-6), atol=1e-12)
    # text rows of the prefix are the embedding rows themselves
    assert np.array_equal(pre[m.n_img_tokens:], w["txt.emb"][fr["text"]].astype(F64))
    # image rows: patch embedding + position, normalised (no shuffle, connector applied)
    p0 = fr["image"][0, :, :m.patch, :m.patch].reshape(-1).astype(F64)               # first patch of camera 0, (c,py,px)
    tok = w["vis.patch.w"].astype(F64) @ p0 + w["vis.pos"][0].astype(F64)
    tok = tok / math.sqrt(float(np.mean(tok * tok)) + 1e-6)
    assert np.allclose(pre[0], w["conn.w"].astype(F64) @ tok, atol=1e-12)
    # layer-0 K is RoPE of W_k RMSNorm(prefix); position 0 is unrotated
    k0 = (w["llm.L0.wk"].astype(F64) @ out["hidden"][0]).reshape(m.hkv, m.hd)
    assert np.allclose(out["kv"][0][0][0], k0, atol=1e-12)


# ------------------------------------------------------------------ dependency rule (Section 2.1)
@pytest.mark.parametrize("key", ["A", "B_nope", "C", "D"])
def test_dependency_rule(key):
    m = TINY[key]
    w = make_weights(m, seed=6)
    frames = [[frame_inputs(m, r, n, seed=6) for n in range(3)] for r in range(2)]
    base = O.run_streams(m, w, frames, np.float32)
    # changing the image of frame n+1 leaves chunk n bit-unchanged and changes chunk n+1
    f2 = [[dict(f) for f in s] for s in frames]
    f2[0][2]["image"] = 1.0 - f2[0][2]["image"]
    alt = O.run_streams(m, w, f2, np.float32)
    assert np.array_equal(alt[0][1], base[0][1]) and np.array_equal(alt[0][0], base[0][0])
    assert not np.array_equal(alt[0][2], base[0][2])
    # the other stream is bit-unchanged
    for n in range(3):
        assert np.array_equal(alt[1][n], base[1][n])
    # identical inputs in two frames give identical chunks
    f3 = [[dict(f) for f in s] for s in frames]
    f3[1][1] = dict(f3[1][0])
    rep = O.run_streams(m, w, f3, np.float32)
    assert np.array_equal(rep[1][1], rep[1][0])


def test_fp32_and_fp64_oracles_agree_on_cfg1():
    w = make_weights(CFG1, seed=0)
    fr = frame_inputs(CFG1, 0, 0, seed=0)
    a = O.action_chunk(CFG1, w, fr, np.float32)
    b = O.action_chunk(CFG1, w, fr, F64)
    assert a.shape == (8, 7)
    assert np.linalg.norm(a - b) / np.linalg.norm(b) < 1e-5


# ------------------------------------------------------------------ shape table
def _matrix_params(m, prefixes):
    from vla_synth.configs import weight_shapes
    tot = 0
    for name, shp in weight_shapes(m).items():
        if name.startswith(prefixes) and len(shp) == 2 and name != "txt.emb":
            tot += shp[0] * shp[1]
    return tot


@pytest.mark.parametrize("m,prefix_len,act_tokens,vlm_mparams", [
    (CFG1, 80, 9, None), (CFG2, 176, 50, 255), (CFG3, 96, 17, 1210), (CFG4, 816, 51, 2396), (CFG5, 288, 17, 6783)])
def test_workload_shapes(m, prefix_len, act_tokens, vlm_mparams):
    assert m.prefix_len == prefix_len and m.act_tokens == act_tokens
    if vlm_mparams is not None:
        got = _matrix_params(m, ("vis.", "conn.", "llm.")) / 1e6
        if m.head == "C":       # the per-frame cross-attention K/V projections run in the VLM phase
            got += sum(2 * m.act_d * m.d for i in range(m.act_layers) if i % 2 == 1) / 1e6
        assert abs(got - vlm_mparams) / vlm_mparams < 0.02


# ------------------------------------------------------------------ asynchronous inference (Section 2.1)
def test_async_passes_are_the_head_on_one_vlm_output():
    m = TINY["A"]
    w = make_weights(m, seed=8)
    fr = frame_inputs(m, 0, 1, seed=8, passes=3)
    single = frame_inputs(m, 0, 1, seed=8)
    assert np.array_equal(fr["state"][0], single["state"]) and np.array_equal(fr["noise"][0], single["noise"])
    assert fr["noise"].shape == (3, m.horizon, m.act_dim) and not np.array_equal(fr["noise"][1], fr["noise"][2])
    out = O.action_chunks_async(m, w, fr, np.float32)
    assert out.shape == (3, m.horizon, m.act_dim)
    # pass p = the plain chunk of a frame with the same image/text and pass p's state and noise
    for p in range(3):
        one = dict(single, state=fr["state"][p], noise=fr["noise"][p])
        assert np.array_equal(out[p], O.action_chunk(m, w, one, np.float32))
    # passes do not see one another: another state for pass 1 changes pass 1 only
    fr2 = dict(fr, state=fr["state"].copy())
    fr2["state"][1] += 1.0
    out2 = O.action_chunks_async(m, w, fr2, np.float32)
    assert np.array_equal(out2[0], out[0]) and np.array_equal(out2[2], out[2]) and not np.array_equal(out2[1], out[1])
