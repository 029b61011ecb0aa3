"""Algorithmic work of one action chunk, from the model description alone.

FLOPs = 2*M*N*K per matrix product + 4*Tq*Tkv*Hq*hd per attention (full score
matrix, masked or not); bytes = every bf16 weight matrix once per pass in which
it is used (VLM once, head once per denoising step).  These are the numerators
of the roofline fractions the benchmark reports; nothing here runs on the hot path.
"""
from __future__ import annotations


def _enc_layer(t, d, heads, hd, mlp):
    p = 3 * d * heads * hd + heads * hd * d + 2 * d * mlp
    return p, 2 * t * p + 4 * t * t * heads * hd


def _dec_layer(t, d, hq, hkv, hd, mlp, gated, tkv=None):
    tkv = t if tkv is None else tkv
    p = d * hq * hd + 2 * d * hkv * hd + hq * hd * d + (3 if gated else 2) * d * mlp
    return p, 2 * t * p + 4 * t * tkv * hq * hd


def vlm_work(m):
    """(matrix parameters, FLOPs) of the VLM phase of one frame."""
    T, S = m.vis_tokens, m.prefix_len
    p = m.vis_d * m.patch_k
    f = m.n_cam * 2 * T * p
    for _ in range(m.vis_layers):
        pl, fl = _enc_layer(T, m.vis_d, m.vis_heads, m.vis_hd, m.vis_mlp)
        p += pl
        f += m.n_cam * fl
    if m.connector:
        pc = m.d * m.shuffle * m.shuffle * m.vis_d
        p += pc
        f += m.n_cam * 2 * m.img_tokens_per_cam * pc
    for _ in range(m.llm_layers):
        pl, fl = _dec_layer(S, m.d, m.hq, m.hkv, m.hd, m.mlp, m.gated)
        p += pl
        f += fl
    if m.head == "C":
        pk = sum(2 * m.act_d * m.d for i in range(m.act_layers) if i % 2 == 1)
        p += pk
        f += 2 * S * pk
    return p, f


def head_step_work(m):
    """(matrix parameters, FLOPs) of one evaluation of the action head."""
    ta, da, S = m.act_tokens, m.act_d, m.prefix_len
    p = da * m.act_dim + m.act_dim * da
    f = 2 * m.horizon * p
    mlp_p = (3 if m.act_gated else 2) * da * m.act_mlp
    for i in range(m.act_layers):
        if m.head == "B":
            pl = da * m.hq * m.hd + 2 * da * m.hkv * m.hd + m.hq * m.hd * da
            fl = 2 * ta * pl + 4 * ta * (S + ta) * m.hq * m.hd
        elif m.head == "C" and i % 2 == 1:
            pl = 2 * da * da
            fl = 2 * ta * pl + 4 * ta * S * da
        else:
            pl = 4 * da * da
            fl = 2 * ta * pl + 4 * ta * ta * da
        if m.head == "A":
            pc = 2 * da * m.hq * m.hd
            pl += pc
            fl += 2 * ta * pc + 4 * ta * S * m.hq * m.hd
        p += pl + mlp_p
        f += fl + 2 * ta * mlp_p
    return p, f


def chunk_work(m):
    """Algorithmic FLOPs and weight bytes (bf16, each matrix once per pass) of one action chunk."""
    pv, fv = vlm_work(m)
    ph, fh = head_step_work(m)
    return {
        "flops": fv + m.n_steps * fh,
        "vlm_flops": fv,
        "head_flops": m.n_steps * fh,
        "weight_bytes": 2 * (pv + m.n_steps * ph),
        "vlm_params": pv,
        "head_params": ph,
    }
