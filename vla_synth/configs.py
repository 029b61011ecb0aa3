"""Shape descriptors of the five two-phase VLA workloads and their weight tables.

This module holds shapes and names only: no arithmetic of the forward pass
lives here.  It serves the seeded generators (``vla_synth.gen``), the CPU oracle
and the GPU binding, which each turn a descriptor into their own structures.

A descriptor fixes one "VLM phase feeding an action head" model (paper Section
2.1, Figure 1): cameras -> patch tokens -> optional vision encoder ->
connector -> [image tokens ; text tokens] -> LLM prefill -> handoff -> action
head run inside a denoising loop -> action chunk.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict, replace
from collections import OrderedDict


@dataclass(frozen=True)
class ModelDesc:
    name: str
    # ---- cameras and patch embedding
    n_cam: int          # cameras per frame
    img: int            # square image side in pixels
    patch: int          # square patch side in pixels
    # ---- vision encoder (vis_layers == 0: patch embedding feeds the LLM directly)
    vis_layers: int
    vis_d: int
    vis_heads: int
    vis_hd: int
    vis_mlp: int
    shuffle: int        # s x s pixel-shuffle of the token grid before the connector (1 = none)
    connector: bool     # linear [d, s*s*vis_d]
    # ---- text
    n_text: int
    vocab: int
    # ---- LLM prefix decoder
    llm_layers: int
    d: int
    hq: int
    hkv: int
    hd: int
    mlp: int
    mlp_kind: str       # "gelu" | "swiglu" | "geglu"
    rope: bool
    causal: bool
    # ---- VLM -> head handoff
    handoff: str        # "kv_last" | "kv_all" | "features" | "cog"
    # ---- action head
    head: str           # "A" self+cross on cached KV | "B" joint-attention expert
                        # "C" DiT alternating self/cross with adaLN | "D" DiT with in-context condition token
    act_layers: int
    act_d: int
    act_heads: int      # heads of the head's own self-attention (A, C, D)
    act_mlp: int
    act_mlp_kind: str
    state_dim: int      # 0: no robot-state token
    horizon: int        # H, actions per chunk
    act_dim: int        # A, action dimension
    n_steps: int
    solver: str         # "euler" | "ddim"
    # ---- workload
    n_streams: int
    n_frames: int
    # ---- workload variants (defaults: the five stated workloads)
    vis_layernorm: int = 0  # vision encoder: 1 = LayerNorm (gain and shift) instead of RMSNorm, and a bias vector on every
                            # linear layer of the encoder (patch embedding, q, k, v, o, both MLP layers)
    guidance: float = 0.0   # head D: classifier-free guidance scale s (0 = off): eps = eps_u + s (eps_c - eps_u), the
                            # unconditional branch built from a zero cognition feature
    suffix_mask: int = 0    # head B: 1 = blocked suffix mask -- the leading state token attends the prefix and itself
                            # but not the action tokens (the action tokens still attend everything)

    # -------- derived sizes
    @property
    def grid(self) -> int:
        return self.img // self.patch

    @property
    def vis_tokens(self) -> int:            # tokens per camera inside the encoder
        return self.grid * self.grid

    @property
    def img_tokens_per_cam(self) -> int:    # tokens per camera entering the LLM
        return self.vis_tokens // (self.shuffle * self.shuffle)

    @property
    def patch_k(self) -> int:
        return 3 * self.patch * self.patch

    @property
    def n_img_tokens(self) -> int:
        return self.n_cam * self.img_tokens_per_cam

    @property
    def prefix_len(self) -> int:            # S
        return self.n_img_tokens + self.n_text

    @property
    def has_state_token(self) -> bool:
        return self.state_dim > 0

    @property
    def act_tokens(self) -> int:            # Ta
        extra = 1 if (self.has_state_token or self.head == "D") else 0
        return self.horizon + extra

    @property
    def act_first(self) -> int:             # index of the first action token
        return self.act_tokens - self.horizon

    @property
    def head_pos_table(self) -> bool:       # learned additive positions in the head
        return not (self.head == "B" and self.rope)

    @property
    def gated(self) -> bool:
        return self.mlp_kind in ("swiglu", "geglu")

    @property
    def act_gated(self) -> bool:
        return self.act_mlp_kind in ("swiglu", "geglu")

    def to_dict(self) -> dict:
        return asdict(self)

    def scaled(self, **kw) -> "ModelDesc":
        return replace(self, **kw)


CFG1 = ModelDesc(
    name="cfg1_tiny",
    n_cam=1, img=64, patch=8,
    vis_layers=0, vis_d=256, vis_heads=0, vis_hd=0, vis_mlp=0, shuffle=1, connector=False,
    n_text=16, vocab=1024,
    llm_layers=2, d=256, hq=4, hkv=4, hd=64, mlp=1024, mlp_kind="gelu", rope=False, causal=False,
    handoff="kv_last",
    head="A", act_layers=2, act_d=128, act_heads=4, act_mlp=512, act_mlp_kind="gelu",
    state_dim=32, horizon=8, act_dim=7, n_steps=4, solver="euler",
    n_streams=2, n_frames=8,
)

CFG2 = ModelDesc(
    name="cfg2_smolvla",
    n_cam=2, img=512, patch=16,
    vis_layers=12, vis_d=768, vis_heads=12, vis_hd=64, vis_mlp=3072, shuffle=4, connector=True,
    n_text=48, vocab=32000,
    llm_layers=16, d=960, hq=15, hkv=5, hd=64, mlp=2560, mlp_kind="swiglu", rope=False, causal=False,
    handoff="kv_all",
    head="B", act_layers=16, act_d=720, act_heads=0, act_mlp=2048, act_mlp_kind="swiglu",
    state_dim=0, horizon=50, act_dim=32, n_steps=10, solver="euler",
    n_streams=32, n_frames=16,
)

CFG3 = ModelDesc(
    name="cfg3_gr00t",
    n_cam=1, img=224, patch=14,
    vis_layers=27, vis_d=1152, vis_heads=16, vis_hd=72, vis_mlp=4304, shuffle=2, connector=True,
    n_text=32, vocab=32000,
    llm_layers=12, d=2048, hq=16, hkv=8, hd=128, mlp=8192, mlp_kind="swiglu", rope=False, causal=False,
    handoff="features",
    head="C", act_layers=16, act_d=1024, act_heads=16, act_mlp=4096, act_mlp_kind="gelu",
    state_dim=64, horizon=16, act_dim=32, n_steps=4, solver="euler",
    n_streams=8, n_frames=16,
)

CFG4 = ModelDesc(
    name="cfg4_pi0",
    n_cam=3, img=224, patch=14,
    vis_layers=27, vis_d=1152, vis_heads=16, vis_hd=72, vis_mlp=4304, shuffle=1, connector=True,
    n_text=48, vocab=32000,
    llm_layers=18, d=2048, hq=8, hkv=1, hd=256, mlp=16384, mlp_kind="geglu", rope=True, causal=False,
    handoff="kv_all",
    head="B", act_layers=18, act_d=1024, act_heads=0, act_mlp=4096, act_mlp_kind="geglu",
    state_dim=32, horizon=50, act_dim=32, n_steps=10, solver="euler",
    n_streams=4, n_frames=16,
)

CFG5 = ModelDesc(
    name="cfg5_cogact",
    n_cam=1, img=224, patch=14,
    vis_layers=24, vis_d=1024, vis_heads=16, vis_hd=64, vis_mlp=4096, shuffle=1, connector=True,
    n_text=32, vocab=32000,
    llm_layers=32, d=4096, hq=32, hkv=32, hd=128, mlp=11008, mlp_kind="swiglu", rope=True, causal=True,
    handoff="cog",
    head="D", act_layers=12, act_d=768, act_heads=12, act_mlp=3072, act_mlp_kind="gelu",
    state_dim=0, horizon=16, act_dim=7, n_steps=10, solver="ddim",
    n_streams=8, n_frames=8,
)

CONFIGS = OrderedDict((c.name, c) for c in (CFG1, CFG2, CFG3, CFG4, CFG5))


def get_config(key) -> ModelDesc:
    """Look a workload up by name ("cfg2_smolvla"), short name ("cfg2") or 1-based index."""
    if isinstance(key, ModelDesc):
        return key
    if isinstance(key, int):
        return list(CONFIGS.values())[key - 1]
    for name, c in CONFIGS.items():
        if name == key or name.split("_")[0] == key:
            return c
    raise KeyError(f"unknown config {key!r}")


def mini(desc: ModelDesc, **kw) -> ModelDesc:
    """A reduced copy of a workload (fewer layers / streams / frames) for quick parity cases."""
    return desc.scaled(name=desc.name + "_mini", **kw)


def weight_shapes(m: ModelDesc) -> "OrderedDict[str, tuple]":
    """Ordered table name -> shape of every weight tensor of a model.

    Matrices are stored ``[out, in]``; gains are vectors.  The order is the
    generation order, so it also keys the per-tensor random streams.
    """
    w: "OrderedDict[str, tuple]" = OrderedDict()
    dv = m.vis_d
    ln = bool(getattr(m, "vis_layernorm", 0))
    w["vis.patch.w"] = (dv, m.patch_k)
    if ln:
        w["vis.patch.b"] = (dv,)
    w["vis.pos"] = (m.vis_tokens, dv)
    hv = m.vis_heads * m.vis_hd
    for i in range(m.vis_layers):
        p = f"vis.L{i}."
        w[p + "n1"] = (dv,)
        w[p + "wq"] = (hv, dv)
        w[p + "wk"] = (hv, dv)
        w[p + "wv"] = (hv, dv)
        w[p + "wo"] = (dv, hv)
        w[p + "n2"] = (dv,)
        w[p + "w1"] = (m.vis_mlp, dv)
        w[p + "w2"] = (dv, m.vis_mlp)
        if ln:
            for leaf, n in (("n1b", dv), ("bq", hv), ("bk", hv), ("bv", hv), ("bo", dv), ("n2b", dv), ("b1", m.vis_mlp), ("b2", dv)):
                w[p + leaf] = (n,)
    if m.vis_layers > 0:
        w["vis.norm"] = (dv,)
        if ln:
            w["vis.normb"] = (dv,)
    if m.connector:
        w["conn.w"] = (m.d, m.shuffle * m.shuffle * dv)
    w["txt.emb"] = (m.vocab, m.d)
    if not m.rope:
        w["llm.pos"] = (m.prefix_len, m.d)
    for i in range(m.llm_layers):
        p = f"llm.L{i}."
        w[p + "n1"] = (m.d,)
        w[p + "wq"] = (m.hq * m.hd, m.d)
        w[p + "wk"] = (m.hkv * m.hd, m.d)
        w[p + "wv"] = (m.hkv * m.hd, m.d)
        w[p + "wo"] = (m.d, m.hq * m.hd)
        w[p + "n2"] = (m.d,)
        if m.gated:
            w[p + "wg"] = (m.mlp, m.d)
            w[p + "wu"] = (m.mlp, m.d)
            w[p + "wd"] = (m.d, m.mlp)
        else:
            w[p + "w1"] = (m.mlp, m.d)
            w[p + "w2"] = (m.d, m.mlp)
    w["llm.norm"] = (m.d,)

    da = m.act_d
    w["act.in"] = (da, m.act_dim)
    if m.has_state_token:
        w["act.state"] = (da, m.state_dim)
    if m.head == "D":
        w["act.cond"] = (da, m.d)
    if m.head_pos_table:
        w["act.pos"] = (m.act_tokens, da)
    w["act.t1"] = (da, da)
    w["act.t2"] = (da, da)
    for i in range(m.act_layers):
        p = f"act.L{i}."
        w[p + "n1"] = (da,)
        if m.head == "B":
            w[p + "wq"] = (m.hq * m.hd, da)
            w[p + "wk"] = (m.hkv * m.hd, da)
            w[p + "wv"] = (m.hkv * m.hd, da)
            w[p + "wo"] = (da, m.hq * m.hd)
        elif m.head == "C" and i % 2 == 1:
            w[p + "cq"] = (da, da)
            w[p + "ck"] = (da, m.d)
            w[p + "cv"] = (da, m.d)
            w[p + "co"] = (da, da)
        else:
            w[p + "wq"] = (da, da)
            w[p + "wk"] = (da, da)
            w[p + "wv"] = (da, da)
            w[p + "wo"] = (da, da)
        if m.head == "A":
            w[p + "n2"] = (da,)
            w[p + "cq"] = (m.hq * m.hd, da)
            w[p + "co"] = (da, m.hq * m.hd)
            w[p + "n3"] = (da,)
        else:
            w[p + "n2"] = (da,)
        if m.head == "C":
            w[p + "ada1"] = (2 * da, da)
            w[p + "ada2"] = (2 * da, da)
        if m.act_gated:
            w[p + "wg"] = (m.act_mlp, da)
            w[p + "wu"] = (m.act_mlp, da)
            w[p + "wd"] = (da, m.act_mlp)
        else:
            w[p + "w1"] = (m.act_mlp, da)
            w[p + "w2"] = (da, m.act_mlp)
    w["act.norm"] = (da,)
    w["act.out"] = (m.act_dim, da)
    return w


def is_vector(name: str) -> bool:
    """fp32 vectors of the weight table: norm gains, LayerNorm shifts and the biases of linear layers."""
    leaf = name.split(".")[-1]
    return is_gain(name) or leaf in ("n1b", "n2b", "normb", "bq", "bk", "bv", "bo", "b1", "b2", "b")


def is_gain(name: str) -> bool:
    """RMSNorm gain vectors (initialised to one, not drawn)."""
    leaf = name.split(".")[-1]
    return leaf in ("n1", "n2", "n3", "norm")
