"""Pins of the oracle's layer COMPOSITIONS: which norm feeds which projection, where RoPE is applied, what is
cached, how the four head kinds combine their own tokens with the VLM handoff.

Each oracle function is compared with a restatement written here from the readings of the workload
descriptions, in plain Python floats with explicit loops over tokens, heads and features.  The restatements
call nothing in ``oracle/`` and no array library routine beyond building the random inputs: a wrong norm, a
swapped concatenation, a missing RoPE offset, a transposed matrix or a dropped residual in the oracle fails one
of these pins.  Weights are drawn large enough that attention logits are of order 1..10 (far from uniform
softmax rows), every residual-branch output matrix is non-zero, and the norm gains differ from one another.
"""
import math

import numpy as np
import pytest

from oracle import vla_oracle as O
from vla_synth.configs import CFG1, CFG2, CFG3, CFG4, CFG5, mini, weight_shapes, is_gain

F64 = np.float64
EPS = 1e-6


# ------------------------------------------------------------------ scalar building blocks (lists of floats)
def matvec(W, x):
    """y[o] = sum_k W[o][k] x[k]   (matrices are stored [out][in])."""
    assert len(W[0]) == len(x)
    return [sum(W[o][k] * x[k] for k in range(len(x))) for o in range(len(W))]


def rms(x, g):
    ms = sum(v * v for v in x) / len(x)
    return [g[i] * x[i] / math.sqrt(ms + EPS) for i in range(len(x))]


def gelu(v):
    return 0.5 * v * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (v + 0.044715 * v ** 3)))


def silu(v):
    return v / (1.0 + math.exp(-v))


def add(a, b):
    return [a[i] + b[i] for i in range(len(a))]


def rotate(vec, pos):
    """Rotary embedding of one head vector: pairs (i, i + hd/2), angle pos * 10000^(-2i/hd)."""
    hd = len(vec)
    half = hd // 2
    out = [0.0] * hd
    for i in range(half):
        ang = pos * 10000.0 ** (-2.0 * i / hd)
        c, s = math.cos(ang), math.sin(ang)
        out[i] = vec[i] * c - vec[i + half] * s
        out[i + half] = vec[i + half] * c + vec[i] * s
    return out


def attend_one(q, keys, vals):
    """One query vector of one head over the visible keys: softmax(q.k / sqrt(hd)) weighted sum of values."""
    hd = len(q)
    logits = [sum(q[c] * k[c] for c in range(hd)) / math.sqrt(hd) for k in keys]
    mx = max(logits)
    e = [math.exp(l - mx) for l in logits]
    z = sum(e)
    return [sum(e[j] / z * vals[j][c] for j in range(len(keys))) for c in range(hd)]


def heads_of(vec, n_heads, hd):
    assert len(vec) == n_heads * hd
    return [vec[h * hd:(h + 1) * hd] for h in range(n_heads)]


def mha(q_rows, k_rows, v_rows, hq, hkv, hd, causal=False):
    """q_rows[t] = list of hq head vectors; k_rows/v_rows[t] = list of hkv head vectors.  Returns rows of hq*hd."""
    out = []
    for i, qh in enumerate(q_rows):
        row = []
        for h in range(hq):
            g = (h * hkv) // hq                     # query head h reads KV head floor(h * Hkv / Hq)
            vis = range(i + 1) if causal else range(len(k_rows))
            row += attend_one(qh[h], [k_rows[j][g] for j in vis], [v_rows[j][g] for j in vis])
        out.append(row)
    return out


def mlp_plain(x, W1, W2):
    return matvec(W2, [gelu(v) for v in matvec(W1, x)])


def mlp_gated(x, Wg, Wu, Wd, act):
    g, u = matvec(Wg, x), matvec(Wu, x)
    return matvec(Wd, [act(g[i]) * u[i] for i in range(len(g))])


def L(a):
    """numpy -> nested lists of Python floats."""
    return np.asarray(a, dtype=F64).tolist()


# ------------------------------------------------------------------ random tables with O(1) activations
def random_weights(m, rng, only=None):
    """name -> fp64 array; matrices ~ N(0, 2/sqrt(in)) so projections keep O(1..3) entries, gains in [0.5, 1.5]."""
    w = {}
    for name, shp in weight_shapes(m).items():
        if only and not name.startswith(only):
            continue
        if is_gain(name):
            w[name] = rng.uniform(0.5, 1.5, size=shp)
        elif len(shp) == 2 and name not in ("vis.pos", "llm.pos", "act.pos", "txt.emb"):
            w[name] = rng.standard_normal(shp) * (2.0 / math.sqrt(shp[1]))
        else:
            w[name] = rng.standard_normal(shp)
    return w


def close(a, b):
    a, b = np.asarray(a, dtype=F64), np.asarray(b, dtype=F64)
    assert a.shape == b.shape, (a.shape, b.shape)
    assert np.max(np.abs(a - b)) <= 1e-9 * max(1.0, float(np.max(np.abs(b)))), float(np.max(np.abs(a - b)))


# ------------------------------------------------------------------ vision encoder layer
def test_vision_encoder_layer_composition():
    rng = np.random.default_rng(101)
    T, d, heads, hd, mlp = 6, 12, 2, 8, 20                      # heads*hd != d: a transposed W_o would not even fit
    p = "vis.L0."
    w = {p + "n1": rng.uniform(0.5, 1.5, d), p + "n2": rng.uniform(0.5, 1.5, d),
         p + "wq": rng.standard_normal((heads * hd, d)), p + "wk": rng.standard_normal((heads * hd, d)),
         p + "wv": rng.standard_normal((heads * hd, d)) * 0.5, p + "wo": rng.standard_normal((d, heads * hd)) * 0.3,
         p + "w1": rng.standard_normal((mlp, d)) * 0.5, p + "w2": rng.standard_normal((d, mlp)) * 0.3}
    x = rng.standard_normal((T, d))
    got = O._encoder_layer(x.copy(), w, p, heads, hd, F64)

    W = {k: L(v) for k, v in w.items()}
    xs = L(x)
    h = [rms(r, W[p + "n1"]) for r in xs]
    q = [heads_of(matvec(W[p + "wq"], r), heads, hd) for r in h]
    k = [heads_of(matvec(W[p + "wk"], r), heads, hd) for r in h]
    v = [heads_of(matvec(W[p + "wv"], r), heads, hd) for r in h]
    a = mha(q, k, v, heads, heads, hd)                           # bidirectional, no positions inside the layer
    xs = [add(xs[t], matvec(W[p + "wo"], a[t])) for t in range(T)]
    h2 = [rms(r, W[p + "n2"]) for r in xs]                       # second norm reads the UPDATED stream
    want = [add(xs[t], mlp_plain(h2[t], W[p + "w1"], W[p + "w2"])) for t in range(T)]
    close(got, want)
    # the softmax rows really are far from uniform at this weight scale
    lg = [sum(q[0][0][c] * k[j][0][c] for c in range(hd)) / math.sqrt(hd) for j in range(T)]
    assert max(lg) - min(lg) > 1.0


def layer_norm(x, g, b):
    n = len(x)
    mu = sum(x) / n
    var = sum((v - mu) ** 2 for v in x) / n
    return [(x[i] - mu) / math.sqrt(var + 1e-6) * g[i] + b[i] for i in range(n)]


def test_layernorm_against_its_textbook_properties():
    rng = np.random.default_rng(7)
    x = rng.standard_normal((5, 16)) * 3.0 + 2.0
    ones, zeros = np.ones(16), np.zeros(16)
    y = O.layernorm(x, ones, zeros)
    assert np.allclose(y.mean(axis=-1), 0.0, atol=1e-12)
    assert np.allclose((y * y).mean(axis=-1), 1.0, atol=1e-6)             # unit variance up to the epsilon
    assert np.allclose(O.layernorm(x + 11.5, ones, zeros), y, atol=1e-9)  # a shift of the row changes nothing
    assert np.allclose(O.layernorm(4.0 * x, ones, zeros), y, atol=1e-6)   # nor does a positive scale
    g, b = rng.uniform(0.5, 1.5, 16), rng.standard_normal(16)
    close(O.layernorm(x, g, b), [layer_norm(r, L(g), L(b)) for r in L(x)])
    xc = x - x.mean(axis=-1, keepdims=True)                               # on a centred row it is RMSNorm plus the shift
    close(O.layernorm(xc, g, b), O.rmsnorm(xc, g) + b)


def test_vision_encoder_layer_with_layernorm_and_biases():
    rng = np.random.default_rng(202)
    T, d, heads, hd, mlp = 5, 12, 2, 8, 20
    p = "vis.L0."
    w = {p + "n1": rng.uniform(0.5, 1.5, d), p + "n2": rng.uniform(0.5, 1.5, d),
         p + "n1b": rng.standard_normal(d) * 0.5, p + "n2b": rng.standard_normal(d) * 0.5,
         p + "wq": rng.standard_normal((heads * hd, d)), p + "wk": rng.standard_normal((heads * hd, d)),
         p + "wv": rng.standard_normal((heads * hd, d)) * 0.5, p + "wo": rng.standard_normal((d, heads * hd)) * 0.3,
         p + "w1": rng.standard_normal((mlp, d)) * 0.5, p + "w2": rng.standard_normal((d, mlp)) * 0.3,
         p + "bq": rng.standard_normal(heads * hd), p + "bk": rng.standard_normal(heads * hd),
         p + "bv": rng.standard_normal(heads * hd), p + "bo": rng.standard_normal(d),
         p + "b1": rng.standard_normal(mlp), p + "b2": rng.standard_normal(d)}
    x = rng.standard_normal((T, d)) + 1.5                      # rows with a mean: RMSNorm in its place would differ
    got = O._encoder_layer_ln(x.copy(), w, p, heads, hd, F64)

    W = {k: L(v) for k, v in w.items()}
    xs = L(x)
    h = [layer_norm(r, W[p + "n1"], W[p + "n1b"]) for r in xs]
    q = [heads_of(add(matvec(W[p + "wq"], r), W[p + "bq"]), heads, hd) for r in h]
    k = [heads_of(add(matvec(W[p + "wk"], r), W[p + "bk"]), heads, hd) for r in h]
    v = [heads_of(add(matvec(W[p + "wv"], r), W[p + "bv"]), heads, hd) for r in h]
    a = mha(q, k, v, heads, heads, hd)
    xs = [add(add(xs[t], matvec(W[p + "wo"], a[t])), W[p + "bo"]) for t in range(T)]
    h2 = [layer_norm(r, W[p + "n2"], W[p + "n2b"]) for r in xs]
    want = []
    for t in range(T):
        mid = [gelu(u) for u in add(matvec(W[p + "w1"], h2[t]), W[p + "b1"])]      # bias BEFORE the activation
        want.append(add(add(xs[t], matvec(W[p + "w2"], mid)), W[p + "b2"]))
    close(got, want)
    # every bias and shift matters: zeroing any one of them changes the layer's output
    for name in ("n1b", "n2b", "bq", "bk", "bv", "bo", "b1", "b2"):
        w2 = dict(w)
        w2[p + name] = np.zeros_like(w[p + name])
        other = O._encoder_layer_ln(x.copy(), w2, p, heads, hd, F64)
        if name == "bk":
            # a key bias adds q.bk to EVERY logit of a query's row, which the softmax cancels: the output must not move
            assert np.allclose(other, got, atol=1e-9)
        else:
            assert np.max(np.abs(other - got)) > 1e-3, name


def test_vision_tokens_layernorm_variant_adds_patch_bias_and_final_shift():
    m = mini(CFG2, n_cam=1, img=28, patch=14, vis_layers=1, vis_d=12, vis_heads=2, vis_hd=8, vis_mlp=20, shuffle=1,
             vis_layernorm=1, d=12, n_text=2, vocab=8, llm_layers=1)
    rng = np.random.default_rng(5)
    w = random_weights(m, rng, only="vis.")
    if "conn.w" in weight_shapes(m):
        w["conn.w"] = rng.standard_normal(weight_shapes(m)["conn.w"]) * 0.3
    img = rng.standard_normal((1, 3, 28, 28))
    got = O.vision_tokens(m, w, img, F64)
    # restated: patch rows -> embedding + bias + positions -> one LN layer -> final LN -> connector (if any)
    pt = O.patchify(img, m.patch)[0]
    xs = [add(add(matvec(L(w["vis.patch.w"]), r), L(w["vis.patch.b"])), prow) for r, prow in zip(L(pt), L(w["vis.pos"]))]
    xs = O._encoder_layer_ln(np.array(xs), w, "vis.L0.", m.vis_heads, m.vis_hd, F64)     # pinned above
    xs = [layer_norm(r, L(w["vis.norm"]), L(w["vis.normb"])) for r in L(xs)]
    if "conn.w" in w:
        xs = [matvec(L(w["conn.w"]), r) for r in xs]
    close(got, xs)


# ------------------------------------------------------------------ LLM decoder layer
LLM_CASES = {
    # GQA + RoPE + causal + SwiGLU (the Llama-style prefix decoder)
    "gqa_rope_causal_swiglu": mini(CFG5, n_cam=1, img=28, patch=14, vis_layers=0, n_text=3, vocab=16, llm_layers=1, d=24,
                                   hq=4, hkv=2, hd=8, mlp=20, mlp_kind="swiglu", rope=True, causal=True),
    # MQA + RoPE + bidirectional + GeGLU
    "mqa_rope_bidir_geglu": mini(CFG4, n_cam=1, img=28, patch=14, vis_layers=0, n_text=3, vocab=16, llm_layers=1, d=24,
                                 hq=4, hkv=1, hd=8, mlp=20, mlp_kind="geglu", rope=True, causal=False),
    # MHA, learned positions (none inside the layer), bidirectional, plain GeLU MLP
    "mha_nope_bidir_gelu": mini(CFG1, n_text=3, vocab=16, llm_layers=1, d=24, hq=3, hkv=3, hd=8, mlp=20),
}


@pytest.mark.parametrize("key", list(LLM_CASES))
def test_llm_layer_composition(key):
    m = LLM_CASES[key]
    rng = np.random.default_rng(202)
    w = random_weights(m, rng, only="llm.L0.")
    S = 7
    x = rng.standard_normal((S, m.d))
    pos = np.arange(3, 3 + S)                                    # positions are an argument: a non-zero start shows they are used
    got_x, got_k, got_v = O.llm_layer(m, w, 0, x.copy(), pos, F64)

    p = "llm.L0."
    W = {k: L(v) for k, v in w.items()}
    xs = L(x)
    h = [rms(r, W[p + "n1"]) for r in xs]
    q = [heads_of(matvec(W[p + "wq"], r), m.hq, m.hd) for r in h]
    k = [heads_of(matvec(W[p + "wk"], r), m.hkv, m.hd) for r in h]
    v = [heads_of(matvec(W[p + "wv"], r), m.hkv, m.hd) for r in h]
    if m.rope:                                                   # q and k rotated, v not; the cache holds the rotated k
        q = [[rotate(q[t][hh], int(pos[t])) for hh in range(m.hq)] for t in range(S)]
        k = [[rotate(k[t][hh], int(pos[t])) for hh in range(m.hkv)] for t in range(S)]
    a = mha(q, k, v, m.hq, m.hkv, m.hd, causal=m.causal)
    xs = [add(xs[t], matvec(W[p + "wo"], a[t])) for t in range(S)]
    h2 = [rms(r, W[p + "n2"]) for r in xs]
    if m.mlp_kind == "gelu":
        br = [mlp_plain(r, W[p + "w1"], W[p + "w2"]) for r in h2]
    else:
        act = silu if m.mlp_kind == "swiglu" else gelu
        br = [mlp_gated(r, W[p + "wg"], W[p + "wu"], W[p + "wd"], act) for r in h2]
    want = [add(xs[t], br[t]) for t in range(S)]
    close(got_x, want)
    close(got_k, k)
    close(got_v, v)


def test_vlm_forward_chains_the_layers_and_caches_every_layers_kv():
    """vlm_forward = embed -> layer 0 -> layer 1 -> final norm, with kv[i] the K,V of layer i."""
    m = mini(CFG4, n_cam=1, img=28, patch=14, vis_layers=0, vis_d=12, connector=True, n_text=3, vocab=16, llm_layers=2,
             d=24, hq=4, hkv=1, hd=8, mlp=20)
    rng = np.random.default_rng(203)
    w = random_weights(m, rng)
    image = rng.uniform(0, 1, (1, 3, 28, 28))
    text = np.array([5, 0, 11])
    out = O.vlm_forward(m, w, image, text, F64)
    x = out["prefix"]
    assert x.shape == (m.prefix_len, m.d)
    pos = np.arange(m.prefix_len)
    for i in range(2):
        x, k, v = O.llm_layer(m, w, i, x, pos, F64)
        close(out["kv"][i][0], k)
        close(out["kv"][i][1], v)
    g = L(w["llm.norm"])
    close(out["hidden"], [rms(r, g) for r in L(x)])
    # prefix rows: image tokens (patch (c,py,px) . W_patch + pos, connector) then the text-embedding rows
    patch0 = [float(image[0, c, py, px]) for c in range(3) for py in range(14) for px in range(14)]
    tok = add(matvec(L(w["vis.patch.w"]), patch0), L(w["vis.pos"][0]))
    close(out["prefix"][0], matvec(L(w["conn.w"]), tok))
    close(out["prefix"][m.n_img_tokens + 1], w["txt.emb"][0])


# ------------------------------------------------------------------ action heads, end to end (one evaluation)
def time_condition(W, t_arg, da):
    half = da // 2
    om = [math.exp(-math.log(10000.0) * i / half) for i in range(half)]
    e = [math.sin(t_arg * o) for o in om] + [math.cos(t_arg * o) for o in om]
    return matvec(W["act.t2"], [silu(v) for v in matvec(W["act.t1"], e)])


def self_attention_rows(h, W, p, heads, hd):
    q = [heads_of(matvec(W[p + "wq"], r), heads, hd) for r in h]
    k = [heads_of(matvec(W[p + "wk"], r), heads, hd) for r in h]
    v = [heads_of(matvec(W[p + "wv"], r), heads, hd) for r in h]
    a = mha(q, k, v, heads, heads, hd)
    return [matvec(W[p + "wo"], r) for r in a]


def head_mlp(m, W, p, r):
    if m.act_mlp_kind == "gelu":
        return mlp_plain(r, W[p + "w1"], W[p + "w2"])
    return mlp_gated(r, W[p + "wg"], W[p + "wu"], W[p + "wd"], silu if m.act_mlp_kind == "swiglu" else gelu)


def restated_head(m, w, vlm, state, x, t_arg):
    """v (or eps) [H][A] for one evaluation of the head, all four kinds, from the readings of the workloads."""
    W = {k: L(v) for k, v in w.items() if k.startswith("act.")}
    da, H, S = m.act_d, m.horizon, m.prefix_len
    c_t = time_condition(W, t_arg, da)
    tok = [matvec(W["act.in"], L(x[i])) for i in range(H)]
    if m.head in ("A", "B"):                                     # time enters the action tokens additively
        tok = [add(r, c_t) for r in tok]
    if m.head in ("A", "C") or (m.head == "B" and m.state_dim > 0):
        tok = [matvec(W["act.state"], L(state))] + tok           # state token first, no time on it
    elif m.head == "D":
        cog = L(vlm["hidden"][S - 1])                            # last prefix position = cognition feature
        tok = [add(matvec(W["act.cond"], cog), c_t)] + tok       # condition token carries the time
    if not (m.head == "B" and m.rope):                           # learned positions unless the head uses RoPE
        tok = [add(tok[t], W["act.pos"][t]) for t in range(len(tok))]
    Ta = len(tok)
    z = tok
    for i in range(m.act_layers):
        p = f"act.L{i}."
        if m.head == "A":
            hd = da // m.act_heads
            br = self_attention_rows([rms(r, W[p + "n1"]) for r in z], W, p, m.act_heads, hd)
            z = [add(z[t], br[t]) for t in range(Ta)]
            h = [rms(r, W[p + "n2"]) for r in z]
            q = [heads_of(matvec(W[p + "cq"], r), m.hq, m.hd) for r in h]     # queries in the VLM's head geometry
            Kc, Vc = vlm["kv"][m.llm_layers - 1]                              # the LAST LLM layer's cache, attended as is
            a = mha(q, L(Kc), L(Vc), m.hq, m.hkv, m.hd)
            z = [add(z[t], matvec(W[p + "co"], a[t])) for t in range(Ta)]
            h = [rms(r, W[p + "n3"]) for r in z]
            z = [add(z[t], head_mlp(m, W, p, h[t])) for t in range(Ta)]
        elif m.head == "B":
            h = [rms(r, W[p + "n1"]) for r in z]
            q = [heads_of(matvec(W[p + "wq"], r), m.hq, m.hd) for r in h]
            k = [heads_of(matvec(W[p + "wk"], r), m.hkv, m.hd) for r in h]
            v = [heads_of(matvec(W[p + "wv"], r), m.hkv, m.hd) for r in h]
            if m.rope:                                                         # positions continue after the prefix
                q = [[rotate(q[t][hh], S + t) for hh in range(m.hq)] for t in range(Ta)]
                k = [[rotate(k[t][hh], S + t) for hh in range(m.hkv)] for t in range(Ta)]
            Kp, Vp = vlm["kv"][i]                                              # prefix cache of the SAME layer index
            first = Ta - H
            if getattr(m, "suffix_mask", 0):
                # blocked suffix mask: the leading state token sees the prefix and the state token(s) only; an action
                # token sees the prefix, the state token(s) and every action token
                a = []
                for t in range(Ta):
                    own = range(first) if t < first else range(Ta)
                    keys = L(Kp) + [k[j] for j in own]
                    vals = L(Vp) + [v[j] for j in own]
                    a += mha([q[t]], keys, vals, m.hq, m.hkv, m.hd)
            else:
                keys, vals = L(Kp) + k, L(Vp) + v                              # [prefix ; own], no mask
                a = mha(q, keys, vals, m.hq, m.hkv, m.hd)
            z = [add(z[t], matvec(W[p + "wo"], a[t])) for t in range(Ta)]
            h = [rms(r, W[p + "n2"]) for r in z]
            z = [add(z[t], head_mlp(m, W, p, h[t])) for t in range(Ta)]
        elif m.head == "C":
            hd = da // m.act_heads
            sc = [silu(v) for v in c_t]
            mod = matvec(W[p + "ada1"], sc)
            gam, bet = mod[:da], mod[da:]
            h = [[n[c] * (1.0 + gam[c]) + bet[c] for c in range(da)] for n in (rms(r, W[p + "n1"]) for r in z)]
            if i % 2 == 0:
                br = self_attention_rows(h, W, p, m.act_heads, hd)
            else:
                F = L(vlm["hidden"])                                           # final-norm VLM features, all S positions
                q = [heads_of(matvec(W[p + "cq"], r), m.act_heads, hd) for r in h]
                k = [heads_of(matvec(W[p + "ck"], f), m.act_heads, hd) for f in F]
                v = [heads_of(matvec(W[p + "cv"], f), m.act_heads, hd) for f in F]
                br = [matvec(W[p + "co"], r) for r in mha(q, k, v, m.act_heads, m.act_heads, hd)]
            z = [add(z[t], br[t]) for t in range(Ta)]
            mod = matvec(W[p + "ada2"], sc)
            gam, bet = mod[:da], mod[da:]
            h = [[n[c] * (1.0 + gam[c]) + bet[c] for c in range(da)] for n in (rms(r, W[p + "n2"]) for r in z)]
            z = [add(z[t], head_mlp(m, W, p, h[t])) for t in range(Ta)]
        else:                                                                  # D: plain pre-norm layers
            hd = da // m.act_heads
            br = self_attention_rows([rms(r, W[p + "n1"]) for r in z], W, p, m.act_heads, hd)
            z = [add(z[t], br[t]) for t in range(Ta)]
            h = [rms(r, W[p + "n2"]) for r in z]
            z = [add(z[t], head_mlp(m, W, p, h[t])) for t in range(Ta)]
    first = Ta - H
    return [matvec(W["act.out"], rms(z[first + i], W["act.norm"])) for i in range(H)]


_VLM = dict(n_cam=1, img=28, patch=14, vis_layers=0, n_text=3, vocab=16)        # prefix of 4 + 3 = 7 positions
HEAD_CASES = {
    "A": mini(CFG1, img=16, n_text=3, vocab=16, llm_layers=2, d=24, hq=2, hkv=2, hd=8, mlp=20, act_layers=2, act_d=12,
              act_heads=2, act_mlp=20, state_dim=5, horizon=4, act_dim=3),
    "B_nope": mini(CFG2, **_VLM, llm_layers=2, d=24, hq=4, hkv=2, hd=8, mlp=20, act_layers=2, act_d=12, act_mlp=20,
                   horizon=4, act_dim=3),
    "B_rope": mini(CFG4, **_VLM, llm_layers=2, d=24, hq=4, hkv=1, hd=8, mlp=20, act_layers=2, act_d=12, act_mlp=20,
                   state_dim=5, horizon=4, act_dim=3),
    "B_rope_blocked_suffix": mini(CFG4, **_VLM, llm_layers=2, d=24, hq=4, hkv=1, hd=8, mlp=20, act_layers=2, act_d=12, act_mlp=20,
                                  state_dim=5, horizon=4, act_dim=3, suffix_mask=1),
    "C": mini(CFG3, **_VLM, shuffle=1, llm_layers=1, d=24, hq=2, hkv=2, hd=8, mlp=20, act_layers=2, act_d=12, act_heads=2,
              act_mlp=20, state_dim=5, horizon=4, act_dim=3),
    "D": mini(CFG5, **_VLM, llm_layers=1, d=24, hq=2, hkv=2, hd=8, mlp=20, act_layers=2, act_d=12, act_heads=2, act_mlp=20,
              horizon=4, act_dim=3),
}


@pytest.mark.parametrize("key", list(HEAD_CASES))
def test_head_velocity_composition(key):
    m = HEAD_CASES[key]
    rng = np.random.default_rng(300 + len(key))
    w = random_weights(m, rng, only="act.")
    S = m.prefix_len
    # a hand-made VLM handoff (the head reads nothing else of the VLM): distinct K,V per LLM layer, distinct features
    vlm = {"kv": [(rng.standard_normal((S, m.hkv, m.hd)) * 1.5, rng.standard_normal((S, m.hkv, m.hd)))
                  for _ in range(m.llm_layers)],
           "hidden": rng.standard_normal((S, m.d))}
    state = rng.standard_normal(m.state_dim) if m.state_dim else None
    x = rng.standard_normal((m.horizon, m.act_dim))
    for t_arg in (0.0, 730.0):
        got = O.head_velocity(m, w, vlm, state, x, t_arg, F64)
        want = restated_head(m, w, vlm, state, x, t_arg)
        close(got, want)
    # the time argument matters for every head kind (it reaches C and D only through the layers / condition token)
    a = O.head_velocity(m, w, vlm, state, x, 0.0, F64)
    b = O.head_velocity(m, w, vlm, state, x, 730.0, F64)
    assert np.max(np.abs(a - b)) > 1e-3
    # and so does the handoff: another prefix cache / feature map changes the result
    vlm2 = {"kv": [(k + 0.5 * rng.standard_normal(k.shape), v) for k, v in vlm["kv"]],
            "hidden": vlm["hidden"] + 0.5 * rng.standard_normal(vlm["hidden"].shape)}
    c = O.head_velocity(m, w, vlm2, state, x, 0.0, F64)
    assert np.max(np.abs(a - c)) > 1e-3


def test_blocked_suffix_mask_changes_the_state_token_only_at_layer_one():
    """With one head layer the mask can only change what the state token computes; the action tokens' outputs
    (the only rows the head returns) then depend on it through nothing -- so a one-layer head is unchanged, a
    two-layer head is not."""
    rng = np.random.default_rng(77)
    for layers, same in ((1, True), (2, False)):
        base = mini(HEAD_CASES["B_rope"], act_layers=layers, llm_layers=max(layers, 2))
        w = random_weights(base, rng, only="act.")
        S = base.prefix_len
        vlm = {"kv": [(rng.standard_normal((S, base.hkv, base.hd)), rng.standard_normal((S, base.hkv, base.hd)))
                      for _ in range(base.llm_layers)], "hidden": rng.standard_normal((S, base.d))}
        state, x = rng.standard_normal(base.state_dim), rng.standard_normal((base.horizon, base.act_dim))
        a = O.head_velocity(base, w, vlm, state, x, 100.0, F64)
        b = O.head_velocity(mini(base, suffix_mask=1), w, vlm, state, x, 100.0, F64)
        assert (np.max(np.abs(a - b)) < 1e-12) == same


def test_action_chunk_is_solver_of_head_on_vlm_output():
    """action_chunk feeds frame n's own VLM output, state and noise to the solver (Euler: x += v/n, t_k = k/n,
    time argument 1000 t_k)."""
    m = HEAD_CASES["B_rope"]
    rng = np.random.default_rng(404)
    w = random_weights(mini(m, vis_d=m.d), rng)
    m2 = mini(m, vis_d=m.d, connector=False)
    fr = {"image": rng.uniform(0, 1, (1, 3, 28, 28)), "text": np.array([1, 2, 3]), "state": rng.standard_normal(5),
          "noise": rng.standard_normal((m.horizon, m.act_dim))}
    vlm = O.vlm_forward(m2, w, fr["image"], fr["text"], F64)
    x = [list(r) for r in L(fr["noise"])]
    for k in range(m2.n_steps):
        v = restated_head(m2, w, vlm, fr["state"], np.array(x), 1000.0 * k / m2.n_steps)
        x = [[x[i][j] + v[i][j] / m2.n_steps for j in range(m2.act_dim)] for i in range(m2.horizon)]
    close(O.action_chunk(m2, w, fr, F64), x)


def test_classifier_free_guidance_composition():
    """Head D with guidance: the unconditional branch is the head on a zero cognition feature (restated with loops),
    and the guided epsilon is e_u + s (e_c - e_u) fed to DDIM."""
    m = HEAD_CASES["D"]
    rng = np.random.default_rng(909)
    w = random_weights(m, rng, only="act.")
    S = m.prefix_len
    vlm = {"kv": [], "hidden": rng.standard_normal((S, m.d))}
    x = rng.standard_normal((m.horizon, m.act_dim))
    zero = {"kv": [], "hidden": vlm["hidden"].copy()}
    zero["hidden"][S - 1] = 0.0
    e_u = O.head_velocity(m, w, vlm, None, x, 40.0, F64, uncond=True)
    close(e_u, restated_head(m, w, zero, None, x, 40.0))
    e_c = O.head_velocity(m, w, vlm, None, x, 40.0, F64)
    assert np.max(np.abs(e_u - e_c)) > 1e-3
    # the guided chunk: DDIM driven by e_u + s (e_c - e_u), written out here with the restated head
    s_g = 2.5
    mg = mini(m, guidance=s_g, n_steps=2)
    noise = rng.standard_normal((m.horizon, m.act_dim))
    got = O.action_head(mg, w, vlm, None, noise, F64)
    ab = O.ddim_alpha_bar()
    xs = noise.copy()
    for tau in (50, 0):
        eu = np.array(restated_head(mg, w, zero, None, xs, float(tau)))
        ec = np.array(restated_head(mg, w, vlm, None, xs, float(tau)))
        eps = eu + s_g * (ec - eu)
        a_t, a_prev = ab[tau], (ab[tau - 50] if tau - 50 >= 0 else 1.0)
        x0 = (xs - math.sqrt(1 - a_t) * eps) / math.sqrt(a_t)
        xs = math.sqrt(a_prev) * x0 + math.sqrt(1 - a_prev) * eps
    close(got, xs)
    # s = 1 is the conditional head alone; s = 0 switches guidance off
    close(O.action_head(mini(m, guidance=1.0, n_steps=2), w, vlm, None, noise, F64),
          O.action_head(mini(m, guidance=0.0, n_steps=2), w, vlm, None, noise, F64))
