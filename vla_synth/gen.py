"""Seeded synthetic weights and per-frame inputs for the VLA workloads.

Stand-ins for the pretrained checkpoints and the robot-camera frames the paper
traces (Section 4, "Workloads"): matrices, embeddings and position tables
~ N(0, 0.02); RMSNorm gains = 1; pixels ~ U[0,1]; text ids uniform over the
vocabulary; robot state and initial noise ~ N(0,1).  Every matrix and every
pixel is rounded once to the nearest bf16 value (ties to even), so both the
CPU oracle (which widens them) and the GPU path (which stores the 16-bit
pattern) start from identical numbers.

Random streams are counter-based (Philox) and keyed by (seed, tensor index)
or (seed, stream, frame, kind): any tensor can be regenerated on its own,
which lets the 7B-parameter workload be produced one tensor at a time.

No arithmetic of the model lives here.
"""
from __future__ import annotations

import numpy as np

from .configs import ModelDesc, weight_shapes, is_gain

WEIGHT_STD = 0.02
_KIND_IMAGE, _KIND_TEXT, _KIND_STATE, _KIND_NOISE = 1, 2, 3, 4


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of fp32 values to bf16, returned as fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)
    return out.reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The 16-bit patterns of fp32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(x.shape)


def _rng(seed: int, hi: int, lo: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 32) ^ hi, lo]))


class Weights:
    """Lazy, regenerable weight table: ``w[name]`` -> fp32 array of bf16-representable values."""

    def __init__(self, desc: ModelDesc, seed: int = 0, cache: bool = True):
        self.desc = desc
        self.seed = seed
        self.shapes = weight_shapes(desc)
        self._index = {n: i for i, n in enumerate(self.shapes)}
        self._cache = {} if cache else None
        self._override = {}

    def names(self):
        return list(self.shapes)

    def __contains__(self, name):
        return name in self.shapes

    def override(self, name: str, value: np.ndarray) -> None:
        """Replace one tensor (tests zero or perturb single matrices)."""
        assert tuple(value.shape) == tuple(self.shapes[name]), name
        self._override[name] = np.ascontiguousarray(value, dtype=np.float32)

    def __getitem__(self, name: str) -> np.ndarray:
        if name in self._override:
            return self._override[name]
        if self._cache is not None and name in self._cache:
            return self._cache[name]
        shape = self.shapes[name]
        if is_gain(name):
            t = np.ones(shape, dtype=np.float32)
        else:
            g = _rng(self.seed, 0x57, self._index[name])
            t = g.standard_normal(size=shape, dtype=np.float32)
            t *= np.float32(WEIGHT_STD)
            t = round_to_bf16(t)
        if self._cache is not None:
            self._cache[name] = t
        return t

    def nbytes_bf16(self) -> int:
        return sum(2 * int(np.prod(s)) for s in self.shapes.values())


def make_weights(desc: ModelDesc, seed: int = 0, cache: bool = True) -> Weights:
    return Weights(desc, seed, cache)


def frame_inputs(desc: ModelDesc, stream: int, frame: int, seed: int = 0, passes: int = 1) -> dict:
    """Inputs of one frame of one request stream.

    image [n_cam,3,H,W] fp32 (bf16-representable, U[0,1]); text int32 [n_text];
    state fp32 [state_dim] or None; noise fp32 [horizon, act_dim].  With ``passes`` > 1
    (several action-head passes per VLM pass) state is [passes, state_dim] and noise
    [passes, horizon, act_dim]; pass 0 holds the arrays of the single-pass frame.
    """
    if passes > 1:
        base = frame_inputs(desc, stream, frame, seed)
        states, noises = [base["state"]], [base["noise"]]
        lo = (stream << 24) | (frame << 4)
        for p in range(1, passes):
            if desc.state_dim > 0:
                states.append(_rng(seed, 0x1A + (p << 8), lo | _KIND_STATE).standard_normal(size=(desc.state_dim,), dtype=np.float32))
            noises.append(_rng(seed, 0x1A + (p << 8), lo | _KIND_NOISE).standard_normal(size=(desc.horizon, desc.act_dim), dtype=np.float32))
        base["state"] = np.stack(states) if desc.state_dim > 0 else None
        base["noise"] = np.stack(noises)
        return base
    lo = (stream << 24) | (frame << 4)
    g = _rng(seed, 0x1A, lo | _KIND_IMAGE)
    image = g.random(size=(desc.n_cam, 3, desc.img, desc.img), dtype=np.float32)
    image = round_to_bf16(image)
    g = _rng(seed, 0x1A, lo | _KIND_TEXT)
    text = g.integers(0, desc.vocab, size=(desc.n_text,), dtype=np.int64).astype(np.int32)
    state = None
    if desc.state_dim > 0:
        g = _rng(seed, 0x1A, lo | _KIND_STATE)
        state = g.standard_normal(size=(desc.state_dim,), dtype=np.float32)
    g = _rng(seed, 0x1A, lo | _KIND_NOISE)
    noise = g.standard_normal(size=(desc.horizon, desc.act_dim), dtype=np.float32)
    return {"image": image, "text": text, "state": state, "noise": noise}
