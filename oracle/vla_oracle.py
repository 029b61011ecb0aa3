"""CPU oracle of the two-phase VLA forward pass.  TEST INFRASTRUCTURE ONLY.

This is the plain definition of what the GPU path must compute, written out
with numpy and nothing else.  It shares no code with the CUDA library and is
never called by it: only the tests, the smoke check and the benchmark's CPU
baseline may import this module.

What it computes (paper Section 2.1, Figure 1): for every request stream r and
frame n, independently,

    chunk[r][n] = ActionHead( VLM(image[r][n], text[r][n]), state[r][n], noise[r][n] )

i.e. the action head of frame n consumes only frame n's VLM output (the
"sequential semantics" the paper's overlap of VLM(n+1) with ActionHead(n)
must preserve).  Co-scheduling changes when work runs, never what is computed,
so the oracle has no notion of tiles, queues or overlap.

The paper treats the models as black boxes; the layer formulas below are this
project's readings of the five workload descriptions (gathered in the design
notes).  Conventions: row-major, matrices stored [out, in], y = x @ W.T, no
biases, pre-norm residual blocks, RMSNorm everywhere.

Precision: ``dtype`` is the arithmetic type (float32 as the workload statement
asks, float64 for the self-checks).  Weights and pixels arrive already rounded
to bf16-representable values.

Pins (see tests/test_oracle_pins.py): every function here is checked against
something other than itself -- brute-force loops, closed forms, invariants or
a library routine.  The end-to-end chunk has no printed reference value in the
paper; it is pinned through those parts, the layer compositions (one vision
encoder layer, one LLM layer, every head kind end to end: explicit-loop
restatements in tests/test_oracle_layer_pins.py), the whole-tower closed forms
(zeroed residual branches) and the dependency rule.
"""
from __future__ import annotations

import math
import numpy as np

RMS_EPS = 1e-6
ROPE_BASE = 10000.0
DDIM_TRAIN_STEPS = 100


# --------------------------------------------------------------------------- primitives
def linear(x, w):
    """y = x @ W.T for W stored [out, in]."""
    return x @ w.T


def rmsnorm(x, g):
    """y_i = g_i * x_i / sqrt(mean_j x_j^2 + eps), over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + x.dtype.type(RMS_EPS)) * g


def layernorm(x, g, b):
    """y_i = g_i (x_i - mean) / sqrt(var + eps) + b_i over the last axis (biased variance)."""
    mu = np.mean(x, axis=-1, keepdims=True)
    xc = x - mu
    var = np.mean(xc * xc, axis=-1, keepdims=True)
    return xc / np.sqrt(var + x.dtype.type(RMS_EPS)) * g + b


def gelu_tanh(x):
    """0.5 x (1 + tanh( sqrt(2/pi) (x + 0.044715 x^3) ))."""
    c = x.dtype.type(math.sqrt(2.0 / math.pi))
    return x.dtype.type(0.5) * x * (1 + np.tanh(c * (x + x.dtype.type(0.044715) * x * x * x)))


def silu(x):
    """x / (1 + exp(-x))."""
    return x / (1 + np.exp(-x))


def mlp(x, w, prefix, kind, dtype):
    """Plain MLP  W2 GeLU(W1 x)  or gated MLP  Wd ( act(Wg x) * Wu x )."""
    if kind == "gelu":
        return linear(gelu_tanh(linear(x, w[prefix + "w1"].astype(dtype))), w[prefix + "w2"].astype(dtype))
    act = silu if kind == "swiglu" else gelu_tanh
    gate = act(linear(x, w[prefix + "wg"].astype(dtype)))
    up = linear(x, w[prefix + "wu"].astype(dtype))
    return linear(gate * up, w[prefix + "wd"].astype(dtype))


def softmax_rows(s):
    """Max-subtracted softmax over the last axis."""
    s = s - np.max(s, axis=-1, keepdims=True)
    e = np.exp(s)
    return e / np.sum(e, axis=-1, keepdims=True)


def attention(q, k, v, causal=False, visible=None):
    """softmax(Q K^T / sqrt(hd) + mask) V per head.

    q [Tq,Hq,hd]; k, v [Tkv,Hkv,hd]; query head h reads KV head floor(h*Hkv/Hq).
    causal: key j visible to query i iff j <= i (needs Tq == Tkv).
    visible: optional boolean [Tq,Tkv]; False entries are masked out (every row must keep one key).
    Returns [Tq,Hq,hd].
    """
    tq, hq, hd = q.shape
    tkv, hkv, _ = k.shape
    out = np.empty_like(q)
    scale = q.dtype.type(1.0 / math.sqrt(hd))
    for h in range(hq):
        g = (h * hkv) // hq
        s = (q[:, h, :] @ k[:, g, :].T) * scale
        if causal:
            assert tq == tkv
            s = np.where(np.tril(np.ones((tq, tkv), dtype=bool)), s, -np.inf)
        if visible is not None:
            s = np.where(visible, s, -np.inf)
        out[:, h, :] = softmax_rows(s) @ v[:, g, :]
    return out


def rope(x, positions):
    """Rotary embedding, rotate-half pairing (i, i+hd/2), angle = pos * base^(-2i/hd).

    x [T,H,hd]; positions [T].
    """
    t, h, hd = x.shape
    half = hd // 2
    inv = ROPE_BASE ** (-(np.arange(half, dtype=np.float64) * 2.0) / hd)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv[None, :]
    c = np.cos(ang).astype(x.dtype)[:, None, :]
    s = np.sin(ang).astype(x.dtype)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def patchify(image, patch):
    """[n_cam,3,H,W] -> [n_cam, (H/P)(W/P), 3 P P]; patch index row-major, inner order (c, py, px)."""
    n, c, hh, ww = image.shape
    gy, gx = hh // patch, ww // patch
    x = image.reshape(n, c, gy, patch, gx, patch)
    x = x.transpose(0, 2, 4, 1, 3, 5)          # n, gy, gx, c, py, px
    return x.reshape(n, gy * gx, c * patch * patch)


def pixel_shuffle_tokens(tok, grid, s):
    """[T=grid*grid, d] -> [(grid/s)^2, s*s*d]; sub-token order (dy, dx) row-major, then channel."""
    d = tok.shape[-1]
    g2 = grid // s
    x = tok.reshape(g2, s, g2, s, d)           # Y, dy, X, dx, d
    x = x.transpose(0, 2, 1, 3, 4)             # Y, X, dy, dx, d
    return x.reshape(g2 * g2, s * s * d)


def timestep_embedding(arg, width, dtype):
    """[sin(arg*w_i) ..., cos(arg*w_i) ...], w_i = exp(-ln(10000) i/(width/2)), i < width/2."""
    half = width // 2
    om = np.exp(-math.log(10000.0) * np.arange(half, dtype=np.float64) / half)
    a = float(arg) * om
    return np.concatenate([np.sin(a), np.cos(a)]).astype(dtype)


# --------------------------------------------------------------------------- VLM phase
def _encoder_layer_ln(x, w, p, heads, hd, dtype):
    """Vision encoder layer of the LayerNorm variant: LayerNorm with shift, and a bias on every linear layer."""
    W = lambda n: w[p + n].astype(dtype)  # noqa: E731
    t = x.shape[0]
    h = layernorm(x, W("n1"), W("n1b"))
    q = (linear(h, W("wq")) + W("bq")).reshape(t, heads, hd)
    k = (linear(h, W("wk")) + W("bk")).reshape(t, heads, hd)
    v = (linear(h, W("wv")) + W("bv")).reshape(t, heads, hd)
    a = attention(q, k, v).reshape(t, heads * hd)
    x = x + linear(a, W("wo")) + W("bo")
    h = layernorm(x, W("n2"), W("n2b"))
    return x + linear(gelu_tanh(linear(h, W("w1")) + W("b1")), W("w2")) + W("b2")


def _encoder_layer(x, w, p, heads, hd, dtype):
    h = rmsnorm(x, w[p + "n1"].astype(dtype))
    t = x.shape[0]
    q = linear(h, w[p + "wq"].astype(dtype)).reshape(t, heads, hd)
    k = linear(h, w[p + "wk"].astype(dtype)).reshape(t, heads, hd)
    v = linear(h, w[p + "wv"].astype(dtype)).reshape(t, heads, hd)
    a = attention(q, k, v).reshape(t, heads * hd)
    x = x + linear(a, w[p + "wo"].astype(dtype))
    h = rmsnorm(x, w[p + "n2"].astype(dtype))
    return x + mlp(h, w, p, "gelu", dtype)


def vision_tokens(m, w, image, dtype):
    """Cameras -> image tokens in the LLM width: patch embed (+pos) -> encoder -> final norm -> shuffle -> connector."""
    patches = patchify(image.astype(dtype), m.patch)
    ln = bool(getattr(m, "vis_layernorm", 0))
    outs = []
    for cam in range(m.n_cam):
        x = linear(patches[cam], w["vis.patch.w"].astype(dtype)) + w["vis.pos"].astype(dtype)
        if ln:
            x = x + w["vis.patch.b"].astype(dtype)
        for i in range(m.vis_layers):
            layer = _encoder_layer_ln if ln else _encoder_layer
            x = layer(x, w, f"vis.L{i}.", m.vis_heads, m.vis_hd, dtype)
        if m.vis_layers > 0:
            x = layernorm(x, w["vis.norm"].astype(dtype), w["vis.normb"].astype(dtype)) if ln else rmsnorm(x, w["vis.norm"].astype(dtype))
        if m.shuffle > 1:
            x = pixel_shuffle_tokens(x, m.grid, m.shuffle)
        if m.connector:
            x = linear(x, w["conn.w"].astype(dtype))
        outs.append(x)
    return np.concatenate(outs, axis=0)


def llm_layer(m, w, i, x, pos, dtype):
    """Decoder layer i of the prefix LLM on the stream x [S,d] at positions pos.

    Returns (x after the layer, K [S,Hkv,hd] as cached -- after RoPE where used --, V [S,Hkv,hd]).
    """
    s = x.shape[0]
    p = f"llm.L{i}."
    h = rmsnorm(x, w[p + "n1"].astype(dtype))
    q = linear(h, w[p + "wq"].astype(dtype)).reshape(s, m.hq, m.hd)
    k = linear(h, w[p + "wk"].astype(dtype)).reshape(s, m.hkv, m.hd)
    v = linear(h, w[p + "wv"].astype(dtype)).reshape(s, m.hkv, m.hd)
    if m.rope:
        q, k = rope(q, pos), rope(k, pos)
    a = attention(q, k, v, causal=m.causal).reshape(s, m.hq * m.hd)
    x = x + linear(a, w[p + "wo"].astype(dtype))
    h = rmsnorm(x, w[p + "n2"].astype(dtype))
    x = x + mlp(h, w, p, m.mlp_kind, dtype)
    return x, k, v


def vlm_forward(m, w, image, text, dtype=np.float32):
    """VLM phase of one frame.  Returns the handoff the action head consumes.

    keys: "kv" list over LLM layers of (K, V) [S,Hkv,hd] (K after RoPE where used),
    "hidden" final-RMSNorm hidden state [S,d], "prefix" the embedded prefix.
    """
    img_tok = vision_tokens(m, w, image, dtype)
    txt_tok = w["txt.emb"][np.asarray(text)].astype(dtype)
    x = np.concatenate([img_tok, txt_tok], axis=0)
    s = x.shape[0]
    assert s == m.prefix_len
    if not m.rope:
        x = x + w["llm.pos"].astype(dtype)
    prefix = x.copy()
    pos = np.arange(s)
    kv = []
    for i in range(m.llm_layers):
        x, k, v = llm_layer(m, w, i, x, pos, dtype)
        kv.append((k, v))
    hidden = rmsnorm(x, w["llm.norm"].astype(dtype))
    return {"kv": kv, "hidden": hidden, "prefix": prefix}


# --------------------------------------------------------------------------- action head
def time_condition(m, w, t_arg, dtype):
    """c_t = W_t2 SiLU(W_t1 e(t_arg))."""
    e = timestep_embedding(t_arg, m.act_d, dtype)
    return linear(silu(linear(e, w["act.t1"].astype(dtype))), w["act.t2"].astype(dtype))


def head_tokens(m, w, vlm, state, x, c_t, dtype, uncond=False):
    """Token sequence entering the head: [state or condition token ; W_a x_k[i]] plus positions / c_t.

    uncond (head D, classifier-free guidance): the condition token is built from a zero cognition feature."""
    tok = linear(x, w["act.in"].astype(dtype))                        # [H, d_a]
    if m.head in ("A", "B"):
        tok = tok + c_t                                               # time enters the action tokens
    first = None
    if m.has_state_token:
        first = linear(state.astype(dtype), w["act.state"].astype(dtype))
    elif m.head == "D":
        cog = vlm["hidden"][-1]                                       # last position = cognition feature
        if uncond:
            cog = np.zeros_like(cog)
        first = linear(cog, w["act.cond"].astype(dtype)) + c_t
    if first is not None:
        tok = np.concatenate([first[None, :], tok], axis=0)
    if m.head_pos_table:
        tok = tok + w["act.pos"].astype(dtype)
    return tok


def _self_attention_block(h, w, p, heads, dtype):
    t, da = h.shape
    hd = da // heads
    q = linear(h, w[p + "wq"].astype(dtype)).reshape(t, heads, hd)
    k = linear(h, w[p + "wk"].astype(dtype)).reshape(t, heads, hd)
    v = linear(h, w[p + "wv"].astype(dtype)).reshape(t, heads, hd)
    a = attention(q, k, v).reshape(t, da)
    return linear(a, w[p + "wo"].astype(dtype))


def head_velocity(m, w, vlm, state, x, t_arg, dtype=np.float32, uncond=False):
    """One evaluation of the head network: v (or eps) [H, A] at sample x and time argument t_arg."""
    c_t = time_condition(m, w, t_arg, dtype)
    z = head_tokens(m, w, vlm, state, x, c_t, dtype, uncond)
    ta = z.shape[0]
    s = m.prefix_len
    for i in range(m.act_layers):
        p = f"act.L{i}."
        if m.head == "A":
            z = z + _self_attention_block(rmsnorm(z, w[p + "n1"].astype(dtype)), w, p, m.act_heads, dtype)
            h = rmsnorm(z, w[p + "n2"].astype(dtype))
            q = linear(h, w[p + "cq"].astype(dtype)).reshape(ta, m.hq, m.hd)
            k, v = vlm["kv"][-1]                                      # last-layer K,V attended directly
            a = attention(q, k, v).reshape(ta, m.hq * m.hd)
            z = z + linear(a, w[p + "co"].astype(dtype))
            h = rmsnorm(z, w[p + "n3"].astype(dtype))
            z = z + mlp(h, w, p, m.act_mlp_kind, dtype)
        elif m.head == "B":
            h = rmsnorm(z, w[p + "n1"].astype(dtype))
            q = linear(h, w[p + "wq"].astype(dtype)).reshape(ta, m.hq, m.hd)
            k = linear(h, w[p + "wk"].astype(dtype)).reshape(ta, m.hkv, m.hd)
            v = linear(h, w[p + "wv"].astype(dtype)).reshape(ta, m.hkv, m.hd)
            if m.rope:
                pos = np.arange(s, s + ta)                            # positions continue after the prefix
                q, k = rope(q, pos), rope(k, pos)
            kp, vp = vlm["kv"][i]                                     # prefix K,V of the same layer index
            visible = None
            if getattr(m, "suffix_mask", 0):                          # blocked suffix mask: the leading state token(s)
                visible = np.ones((ta, s + ta), dtype=bool)           # see the prefix and themselves, not the actions
                visible[: m.act_first, s + m.act_first:] = False
            a = attention(q, np.concatenate([kp, k], 0), np.concatenate([vp, v], 0), visible=visible).reshape(ta, m.hq * m.hd)
            z = z + linear(a, w[p + "wo"].astype(dtype))
            h = rmsnorm(z, w[p + "n2"].astype(dtype))
            z = z + mlp(h, w, p, m.act_mlp_kind, dtype)
        elif m.head == "C":
            sc = silu(c_t)
            mod = linear(sc, w[p + "ada1"].astype(dtype))
            gamma, beta = mod[: m.act_d], mod[m.act_d:]
            h = rmsnorm(z, w[p + "n1"].astype(dtype)) * (1 + gamma) + beta
            if i % 2 == 0:
                z = z + _self_attention_block(h, w, p, m.act_heads, dtype)
            else:
                hd = m.act_d // m.act_heads
                f = vlm["hidden"]
                q = linear(h, w[p + "cq"].astype(dtype)).reshape(ta, m.act_heads, hd)
                k = linear(f, w[p + "ck"].astype(dtype)).reshape(s, m.act_heads, hd)
                v = linear(f, w[p + "cv"].astype(dtype)).reshape(s, m.act_heads, hd)
                a = attention(q, k, v).reshape(ta, m.act_d)
                z = z + linear(a, w[p + "co"].astype(dtype))
            mod = linear(sc, w[p + "ada2"].astype(dtype))
            gamma, beta = mod[: m.act_d], mod[m.act_d:]
            h = rmsnorm(z, w[p + "n2"].astype(dtype)) * (1 + gamma) + beta
            z = z + mlp(h, w, p, m.act_mlp_kind, dtype)
        elif m.head == "D":
            z = z + _self_attention_block(rmsnorm(z, w[p + "n1"].astype(dtype)), w, p, m.act_heads, dtype)
            h = rmsnorm(z, w[p + "n2"].astype(dtype))
            z = z + mlp(h, w, p, m.act_mlp_kind, dtype)
        else:
            raise ValueError(m.head)
    z = rmsnorm(z, w["act.norm"].astype(dtype))
    return linear(z[m.act_first:], w["act.out"].astype(dtype))


# --------------------------------------------------------------------------- solvers
def euler_solve(velocity, x0, n_steps):
    """Flow matching, explicit Euler: t_k = k/n, x_{k+1} = x_k + (1/n) v(x_k, t_k); returns x_n."""
    x = x0.copy()
    dt = x.dtype.type(1.0 / n_steps)
    for k in range(n_steps):
        x = x + dt * velocity(x, k / n_steps)
    return x


def ddim_alpha_bar(train_steps=DDIM_TRAIN_STEPS):
    """Cumulative product of (1 - beta_s) for the squared-cosine schedule with beta clipped at 0.999."""
    def c(u):
        return math.cos((u + 0.008) / 1.008 * math.pi / 2) ** 2
    ab, prod = [], 1.0
    for s_ in range(train_steps):
        beta = min(1.0 - c((s_ + 1) / train_steps) / c(s_ / train_steps), 0.999)
        prod *= 1.0 - beta
        ab.append(prod)
    return np.array(ab, dtype=np.float64)


def ddim_timesteps(n_steps, train_steps=DDIM_TRAIN_STEPS):
    """tau = (n-1) T/n, ..., T/n, 0."""
    stride = train_steps // n_steps
    return [i * stride for i in range(n_steps - 1, -1, -1)]


def ddim_solve(eps_fn, x_t, n_steps, train_steps=DDIM_TRAIN_STEPS):
    """Deterministic DDIM (eta = 0), eps-prediction, no clipping of the x0 estimate."""
    ab = ddim_alpha_bar(train_steps)
    stride = train_steps // n_steps
    x = x_t.copy()
    ty = x.dtype.type
    for tau in ddim_timesteps(n_steps, train_steps):
        a_t = ab[tau]
        a_prev = ab[tau - stride] if tau - stride >= 0 else 1.0
        eps = eps_fn(x, tau)
        x0 = (x - ty(math.sqrt(1.0 - a_t)) * eps) / ty(math.sqrt(a_t))
        x = ty(math.sqrt(a_prev)) * x0 + ty(math.sqrt(1.0 - a_prev)) * eps
    return x


# --------------------------------------------------------------------------- whole path
def action_head(m, w, vlm, state, noise, dtype=np.float32):
    """Denoising loop of one frame: noise [H,A] -> action chunk [H,A]."""
    x0 = noise.astype(dtype)
    if m.solver == "euler":
        return euler_solve(lambda x, t: head_velocity(m, w, vlm, state, x, 1000.0 * t, dtype), x0, m.n_steps)
    if m.solver == "ddim":
        s_g = float(getattr(m, "guidance", 0.0))
        if s_g != 0.0:                                                # classifier-free guidance (head D)
            def guided(x, tau):
                e_u = head_velocity(m, w, vlm, state, x, float(tau), dtype, uncond=True)
                e_c = head_velocity(m, w, vlm, state, x, float(tau), dtype)
                return e_u + dtype(s_g) * (e_c - e_u)
            return ddim_solve(guided, x0, m.n_steps)
        return ddim_solve(lambda x, tau: head_velocity(m, w, vlm, state, x, float(tau), dtype), x0, m.n_steps)
    raise ValueError(m.solver)


def action_chunk(m, w, frame, dtype=np.float32):
    """chunk = ActionHead(VLM(image, text), state, noise) for one frame's inputs."""
    vlm = vlm_forward(m, w, frame["image"], frame["text"], dtype)
    return action_head(m, w, vlm, frame["state"], frame["noise"], dtype)


def action_chunks_async(m, w, frame, dtype=np.float32):
    """Asynchronous inference (paper Section 2.1, decoupled update rates): one VLM pass, then the action head once per
    (state, noise) pair of the frame, every pass on that same VLM output.  frame["state"] [P, state_dim] or None,
    frame["noise"] [P, H, A]; returns [P, H, A]."""
    vlm = vlm_forward(m, w, frame["image"], frame["text"], dtype)
    out = []
    for p in range(frame["noise"].shape[0]):
        state = None if frame["state"] is None else frame["state"][p]
        out.append(action_head(m, w, vlm, state, frame["noise"][p], dtype))
    return np.stack(out)


def run_streams(m, w, frames, dtype=np.float32):
    """frames[r][n] -> chunks[r][n]; every (stream, frame) is computed from its own inputs alone."""
    return [[action_chunk(m, w, f, dtype) for f in stream] for stream in frames]
