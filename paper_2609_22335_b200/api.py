"""ctypes binding of libvla_b200.so: the same entry points as include/vla.h.

Argument marshalling only -- every step of the forward pass runs inside the
CUDA library.  PyTorch supplies the device arena and the CUDA streams.  There
is no CPU fallback: importing this module without the built library, or
creating an engine without a CUDA device, raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvla_b200.so")

VLA_OK, VLA_ERR_INVALID, VLA_ERR_STATE, VLA_ERR_BUSY, VLA_ERR_NOT_READY, VLA_ERR_TIMEOUT, VLA_ERR_CUDA, VLA_ERR_NOMEM = range(8)
MODE_COSCHED, MODE_TWO_STREAM, MODE_SERIAL, MODE_MULTI_STREAM = 0, 1, 2, 3
MODES = {"cosched": MODE_COSCHED, "two_stream": MODE_TWO_STREAM, "serial": MODE_SERIAL, "multi_stream": MODE_MULTI_STREAM}
_MLP = {"gelu": 0, "swiglu": 1, "geglu": 2}
_HANDOFF = {"kv_last": 0, "kv_all": 1, "features": 2, "cog": 3}
_HEAD = {"A": 0, "B": 1, "C": 2, "D": 3}
_SOLVER = {"euler": 0, "ddim": 1}

EXPORTS = ["vla_required_arena_bytes", "vla_init", "vla_load_weights", "vla_submit_frame", "vla_submit_frame_device",
           "vla_poll_actions", "vla_hold_launches", "vla_wait_idle", "vla_get_trace", "vla_reset_trace", "vla_program_info", "vla_debug_fetch",
           "vla_get_counters", "vla_set_class_tags", "vla_get_class_tags", "vla_policy_probe", "vla_policy_probe_ex", "vla_debug_bump_dependency", "vla_debug_guards", "vla_last_error",
           "vla_destroy", "vla_op_status", "vla_debug_op_fault",
           "vla_op_attention_scratch_bytes", "vla_op_attention", "vla_op_linear",
           "vla_op_attention_static_capacity", "vla_op_attention_static"]


class vla_model_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_cam", "img", "patch", "vis_layers", "vis_d", "vis_heads", "vis_hd", "vis_mlp", "shuffle", "connector",
        "n_text", "vocab", "llm_layers", "d", "hq", "hkv", "hd", "mlp", "mlp_kind", "rope", "causal", "handoff",
        "head", "act_layers", "act_d", "act_heads", "act_mlp", "act_mlp_kind", "state_dim", "horizon", "act_dim",
        "n_steps", "solver")] + [("guidance", C.c_float), ("suffix_mask", C.c_int32), ("vis_layernorm", C.c_int32)]


class vla_runtime_opts(C.Structure):
    _fields_ = [("arena", C.c_void_p), ("arena_bytes", C.c_size_t), ("stream_a", C.c_void_p), ("stream_b", C.c_void_p),
                ("mode", C.c_int32), ("n_streams", C.c_int32), ("ring_depth", C.c_int32), ("policy", C.c_int32),
                ("wait_limit_ns", C.c_uint64), ("trace_capacity", C.c_uint32), ("workers_per_sm", C.c_int32),
                ("u_max", C.c_int32), ("head_passes", C.c_int32), ("reserved_", C.c_int32)]


class vla_tensor(C.Structure):
    _fields_ = [("name", C.c_char_p), ("host_ptr", C.c_void_p), ("dtype", C.c_int32), ("rank", C.c_int32),
                ("shape", C.c_int64 * 4)]


class vla_trace_rec(C.Structure):
    _fields_ = [("inst", C.c_uint32), ("node", C.c_uint32), ("tile", C.c_uint32), ("sm", C.c_uint16), ("worker", C.c_uint8),
                ("cls", C.c_uint8), ("frame", C.c_uint64), ("t_start", C.c_uint64), ("t_end", C.c_uint64)]


class vla_node_info(C.Structure):
    _fields_ = [("op", C.c_int32), ("cls", C.c_int32), ("n_tiles", C.c_int32), ("n_pred", C.c_int32), ("phase", C.c_int32),
                ("step", C.c_int32), ("succ_begin", C.c_int32), ("succ_count", C.c_int32), ("smem_bytes", C.c_int32), ("tmem_cols", C.c_int32),
                ("name", C.c_char * 48), ("flops", C.c_double), ("weight_bytes", C.c_double)]


TRACE_DTYPE = np.dtype([("inst", "<u4"), ("node", "<u4"), ("tile", "<u4"), ("sm", "<u2"), ("worker", "u1"), ("cls", "u1"),
                        ("frame", "<u8"), ("t_start", "<u8"), ("t_end", "<u8")])

_lib = None


def load_library() -> C.CDLL:
    """Loads the in-tree shared library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2609_22335_b200.build` (there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    P = C.POINTER
    lib.vla_required_arena_bytes.argtypes = [P(vla_model_desc), P(vla_runtime_opts), P(C.c_size_t)]
    lib.vla_init.argtypes = [P(vla_model_desc), P(vla_runtime_opts), P(C.c_void_p)]
    lib.vla_load_weights.argtypes = [C.c_void_p, P(vla_tensor), C.c_size_t, C.c_int32]
    for fn in (lib.vla_submit_frame, lib.vla_submit_frame_device):
        fn.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, P(C.c_uint64)]
    lib.vla_poll_actions.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, P(C.c_uint64)]
    lib.vla_wait_idle.argtypes = [C.c_void_p, C.c_uint32]
    lib.vla_hold_launches.argtypes = [C.c_void_p, C.c_int32]
    lib.vla_get_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, P(C.c_size_t)]
    lib.vla_reset_trace.argtypes = [C.c_void_p]
    lib.vla_program_info.argtypes = [C.c_void_p, P(vla_node_info), C.c_size_t, P(C.c_size_t), P(C.c_int32), C.c_size_t,
                                     P(C.c_size_t)]
    lib.vla_debug_fetch.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_char_p, C.c_void_p, C.c_size_t, P(C.c_size_t)]
    lib.vla_get_counters.argtypes = [C.c_void_p, P(C.c_uint64), P(C.c_uint64), P(C.c_uint64)]
    lib.vla_policy_probe.argtypes = [C.c_int32, P(C.c_int32), P(C.c_int32), P(C.c_int32), P(C.c_int32), P(C.c_int32),
                                     C.c_int32, C.c_int32, P(C.c_int32), P(C.c_int32)]
    lib.vla_policy_probe_ex.argtypes = [C.c_int32, P(C.c_int32), P(C.c_int32), P(C.c_int32), P(C.c_int32), P(C.c_int32),
                                        C.c_int32, C.c_int32, C.c_int32, P(C.c_int32), P(C.c_int32), P(C.c_int32), P(C.c_int32)]
    lib.vla_set_class_tags.argtypes = [C.c_void_p, P(C.c_int32)]
    lib.vla_get_class_tags.argtypes = [C.c_void_p, P(C.c_int32)]
    lib.vla_debug_guards.argtypes = [C.c_void_p, C.c_int32, P(C.c_size_t)]
    lib.vla_debug_bump_dependency.argtypes = [C.c_void_p] + [C.c_int32] * 4
    lib.vla_op_status.argtypes = [C.c_int32, C.c_void_p, C.c_void_p]
    lib.vla_debug_op_fault.argtypes = [C.c_int32, C.c_uint64]
    lib.vla_op_attention_scratch_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32, P(C.c_size_t)]
    lib.vla_op_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p] + [C.c_int32] * 6 + [C.c_void_p, C.c_size_t, C.c_void_p]
    lib.vla_op_linear.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p] + [C.c_int32] * 4 + [C.c_void_p]
    lib.vla_op_attention_static_capacity.argtypes = [P(C.c_size_t)]
    lib.vla_op_attention_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p] + [C.c_int32] * 6 + [C.c_void_p]
    lib.vla_last_error.argtypes = [C.c_void_p]
    lib.vla_last_error.restype = C.c_char_p
    lib.vla_destroy.argtypes = [C.c_void_p]
    for name in EXPORTS:
        if name != "vla_last_error":
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def make_desc(m) -> vla_model_desc:
    """vla_synth ModelDesc (or any object with the same fields) -> C struct."""
    d = vla_model_desc()
    for name, _ in vla_model_desc._fields_:
        v = getattr(m, name, 0)
        if name in ("mlp_kind", "act_mlp_kind"):
            v = _MLP[v]
        elif name == "handoff":
            v = _HANDOFF[v]
        elif name == "head":
            v = _HEAD[v]
        elif name == "solver":
            v = _SOLVER[v]
        setattr(d, name, float(v) if name == "guidance" else int(v))
    return d


class VlaError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"vla error {code}: {msg}")
        self.code = code


def vla_required_arena_bytes(desc: vla_model_desc, opts: vla_runtime_opts) -> int:
    out = C.c_size_t(0)
    rc = load_library().vla_required_arena_bytes(C.byref(desc), C.byref(opts), C.byref(out))
    if rc != VLA_OK:
        raise VlaError(rc, "invalid model description or options")
    return out.value


class Engine:
    """One library context plus the torch-owned arena and streams it runs on."""

    def __init__(self, model, mode="cosched", n_streams=None, ring_depth=2, policy=0, trace_capacity=0,
                 wait_limit_ns=0, workers_per_sm=0, u_max=0, head_passes=1, device="cuda:0"):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU fallback)")
        self.lib = load_library()
        self.torch = torch
        self.model = model
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.desc = make_desc(model)
        self.n_streams = int(n_streams if n_streams is not None else model.n_streams)
        self.ring_depth = ring_depth
        self.mode = MODES[mode] if isinstance(mode, str) else int(mode)
        self.opts = vla_runtime_opts()
        self.opts.mode = self.mode
        self.opts.n_streams = self.n_streams
        self.opts.ring_depth = ring_depth
        self.opts.policy = policy
        self.opts.wait_limit_ns = wait_limit_ns
        self.opts.trace_capacity = trace_capacity
        self.opts.workers_per_sm = workers_per_sm
        self.opts.u_max = u_max
        self.opts.head_passes = head_passes
        self.arena_bytes = vla_required_arena_bytes(self.desc, self.opts)
        self.arena = torch.empty(self.arena_bytes + 256, dtype=torch.uint8, device=self.device)
        base = self.arena.data_ptr()
        self.opts.arena = (base + 255) // 256 * 256
        self.opts.arena_bytes = self.arena_bytes
        self.stream_a = torch.cuda.Stream(device=self.device)
        self.stream_b = torch.cuda.Stream(device=self.device)
        self.opts.stream_a = self.stream_a.cuda_stream
        self.opts.stream_b = self.stream_b.cuda_stream
        self.ctx = C.c_void_p(None)
        rc = self.lib.vla_init(C.byref(self.desc), C.byref(self.opts), C.byref(self.ctx))
        if rc != VLA_OK:
            msg = self.last_error() if self.ctx else "vla_init failed"
            if self.ctx:
                self.lib.vla_destroy(self.ctx)
                self.ctx = C.c_void_p(None)
            raise VlaError(rc, msg)
        self.head_passes = max(1, int(head_passes))
        self.chunk_shape = (model.horizon, model.act_dim) if self.head_passes == 1 else (self.head_passes, model.horizon, model.act_dim)

    # ---- thin wrappers -------------------------------------------------------------
    def last_error(self) -> str:
        return (self.lib.vla_last_error(self.ctx) or b"").decode()

    def _check(self, rc):
        if rc != VLA_OK:
            raise VlaError(rc, self.last_error())

    def load_weights(self, weights, batch_bytes=1 << 30):
        """weights: mapping name -> fp32 ndarray of bf16-representable values (vla_synth.gen.Weights)."""
        from vla_synth.gen import bf16_bits
        from vla_synth.configs import is_vector
        names = list(weights.names())
        batch, keep, size = [], [], 0

        def flush(final):
            arr = (vla_tensor * len(batch))(*batch)
            self._check(self.lib.vla_load_weights(self.ctx, arr, len(batch), 1 if final else 0))
            batch.clear(); keep.clear()

        for i, name in enumerate(names):
            w = weights[name]
            fp32 = is_vector(name) or name in ("vis.pos", "llm.pos", "act.pos")
            a = np.ascontiguousarray(w, dtype=np.float32) if fp32 else bf16_bits(w)
            keep.append(a)
            t = vla_tensor()
            t.name = name.encode()
            t.host_ptr = a.ctypes.data
            t.dtype = 0 if fp32 else 1
            t.rank = a.ndim
            for k, s in enumerate(a.shape):
                t.shape[k] = s
            batch.append(t)
            size += a.nbytes
            if size >= batch_bytes and i + 1 < len(names):
                flush(False)
                size = 0
        flush(True)

    def submit(self, stream, frame) -> int:
        """frame: dict image/text/state/noise of host numpy arrays. Returns VLA_OK or VLA_ERR_BUSY; raises otherwise."""
        img = np.ascontiguousarray(frame["image"], dtype=np.float32)
        txt = np.ascontiguousarray(frame["text"], dtype=np.int32)
        st = None if frame.get("state") is None else np.ascontiguousarray(frame["state"], dtype=np.float32)
        nz = np.ascontiguousarray(frame["noise"], dtype=np.float32)
        rc = self.lib.vla_submit_frame(self.ctx, stream, img.ctypes.data, txt.ctypes.data,
                                       None if st is None else st.ctypes.data, nz.ctypes.data, None)
        if rc not in (VLA_OK, VLA_ERR_BUSY):
            self._check(rc)
        return rc

    def submit_ptrs(self, stream, image_ptr, text_ptr, state_ptr, noise_ptr, device=False) -> int:
        fn = self.lib.vla_submit_frame_device if device else self.lib.vla_submit_frame
        rc = fn(self.ctx, stream, image_ptr, text_ptr, state_ptr, noise_ptr, None)
        if rc not in (VLA_OK, VLA_ERR_BUSY):
            self._check(rc)
        return rc

    def poll(self, stream, out=None):
        """Returns (chunk ndarray, frame id) or None when nothing is ready."""
        if out is None:
            out = np.empty(self.chunk_shape, dtype=np.float32)
        fid = C.c_uint64(0)
        rc = self.lib.vla_poll_actions(self.ctx, stream, out.ctypes.data, C.byref(fid))
        if rc == VLA_ERR_NOT_READY:
            return None
        self._check(rc)
        return out, fid.value

    def hold_launches(self, on):
        """While on, submitted frames are queued but the persistent kernel is not launched (see vla_hold_launches)."""
        self._check(self.lib.vla_hold_launches(self.ctx, int(bool(on))))

    def wait_idle(self, timeout_ms=60000):
        self._check(self.lib.vla_wait_idle(self.ctx, timeout_ms))

    def run(self, frames, timeout_s=600.0):
        """frames[r][n] -> chunks[r][n]; submits as fast as the rings accept and polls in frame order."""
        import time
        R = len(frames)
        if not hasattr(self, "_frames_done"):
            self._frames_done = [0] * self.n_streams
        base = list(self._frames_done)
        nxt = [0] * R
        got = [[None] * len(frames[r]) for r in range(R)]
        remaining = sum(len(f) for f in frames)
        t0 = time.time()
        while remaining:
            progressed = False
            for r in range(R):
                while nxt[r] < len(frames[r]):
                    if self.submit(r, frames[r][nxt[r]]) == VLA_ERR_BUSY:
                        break
                    nxt[r] += 1
                    progressed = True
            for r in range(R):
                while True:
                    res = self.poll(r)
                    if res is None:
                        break
                    chunk, fid = res
                    got[r][fid - base[r]] = chunk
                    self._frames_done[r] += 1
                    remaining -= 1
                    progressed = True
            if not progressed:
                if time.time() - t0 > timeout_s:
                    raise TimeoutError("no progress")
                time.sleep(0.0002)
        return got

    def trace(self):
        n = C.c_size_t(0)
        self._check(self.lib.vla_get_trace(self.ctx, None, 0, C.byref(n)))
        cap = min(n.value, self.opts.trace_capacity)
        arr = np.zeros(cap, dtype=TRACE_DTYPE)
        if cap:
            self._check(self.lib.vla_get_trace(self.ctx, arr.ctypes.data, cap, C.byref(n)))
        return arr, n.value

    def reset_trace(self):
        self._check(self.lib.vla_reset_trace(self.ctx))

    def program_info(self):
        nn, ns = C.c_size_t(0), C.c_size_t(0)
        self._check(self.lib.vla_program_info(self.ctx, None, 0, C.byref(nn), None, 0, C.byref(ns)))
        nodes = (vla_node_info * nn.value)()
        succ = (C.c_int32 * max(ns.value, 1))()
        self._check(self.lib.vla_program_info(self.ctx, nodes, nn.value, C.byref(nn), succ, ns.value, C.byref(ns)))
        out = [dict(op=n.op, cls=n.cls, n_tiles=n.n_tiles, n_pred=n.n_pred, phase=n.phase, step=n.step,
                    smem_bytes=n.smem_bytes, tmem_cols=n.tmem_cols, flops=n.flops, weight_bytes=n.weight_bytes,
                    succ=[succ[n.succ_begin + i] for i in range(n.succ_count)], name=n.name.decode()) for n in nodes]
        return out

    def debug_fetch(self, stream, slot, name):
        n = C.c_size_t(0)
        self._check(self.lib.vla_debug_fetch(self.ctx, stream, slot, name.encode(), None, 0, C.byref(n)))
        out = np.empty(n.value, dtype=np.float32)
        self._check(self.lib.vla_debug_fetch(self.ctx, stream, slot, name.encode(), out.ctypes.data, n.value, C.byref(n)))
        return out

    def counters(self):
        a, b, c = C.c_uint64(0), C.c_uint64(0), C.c_uint64(0)
        self._check(self.lib.vla_get_counters(self.ctx, C.byref(a), C.byref(b), C.byref(c)))
        return dict(tiles=a.value, kernel_launches=b.value, persistent_launches=c.value)

    def class_tags(self):
        """The eight tile classes' (tau_TC, tau_ALU, tau_MEM) tags."""
        t = (C.c_int32 * 24)()
        self._check(self.lib.vla_get_class_tags(self.ctx, t))
        return [[t[3 * k + x] for x in range(3)] for k in range(8)]

    def set_class_tags(self, tags):
        """tags[8][3]; entries that are None keep their current value."""
        cur = self.class_tags()
        flat = [int((tags[k] or cur[k])[x]) for k in range(8) for x in range(3)]
        self._check(self.lib.vla_set_class_tags(self.ctx, (C.c_int32 * 24)(*flat)))

    def fill_guards(self):
        """Writes the guard pattern behind every buffer (see vla_debug_guards)."""
        self._check(self.lib.vla_debug_guards(self.ctx, 1, None))

    def overwritten_guards(self) -> int:
        """How many guards no longer hold the pattern (0 = no tile wrote outside its buffers)."""
        n = C.c_size_t(0)
        self._check(self.lib.vla_debug_guards(self.ctx, 0, C.byref(n)))
        return n.value

    def bump_dependency(self, stream, slot, node, delta):
        """Test hook: adds ``delta`` to one node's dependency counter (see vla_debug_bump_dependency)."""
        self._check(self.lib.vla_debug_bump_dependency(self.ctx, stream, slot, node, delta))

    def close(self):
        if self.ctx:
            self.lib.vla_destroy(self.ctx)
            self.ctx = C.c_void_p(None)
        self.arena = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


POLICIES = {"two_phase": 0, "class_order": 1, "round_robin": 2, "two_phase_g": 3, "two_phase_r": 4}
OP_LINEAR, OP_ATTENTION, OP_ATTENTION_STATIC = 0, 1, 2


def policy_probe(taus, pending, feasible, cta_count, u, rr_start=0, u_max=0, policy=0, grid=None, res=None):
    """Runs the device pick once on the GPU; returns (picked, phase, cta_count, u)."""
    lib = load_library()
    n = len(taus)
    flat = (C.c_int32 * (3 * n))(*[int(x) for t in taus for x in t])
    pend = (C.c_int32 * n)(*[int(bool(x)) for x in pending])
    feas = (C.c_int32 * n)(*[int(bool(x)) for x in feasible])
    cc = (C.c_int32 * n)(*[int(x) for x in cta_count])
    uu = (C.c_int32 * 3)(*[int(x) for x in u])
    picked, phase = C.c_int32(-1), C.c_int32(0)
    gg = None if grid is None else (C.c_int32 * n)(*[int(x) for x in grid])
    rs = None if res is None else (C.c_int32 * n)(*[int(x) for x in res])
    if policy == 0 and grid is None and res is None:
        rc = lib.vla_policy_probe(n, flat, pend, feas, cc, uu, rr_start, u_max, C.byref(picked), C.byref(phase))
    else:
        rc = lib.vla_policy_probe_ex(n, flat, pend, feas, cc, uu, rr_start, u_max, policy, gg, rs, C.byref(picked),
                                     C.byref(phase))
    if rc != VLA_OK:
        raise VlaError(rc, "policy probe failed")
    return picked.value, phase.value, list(cc), list(uu)


def _stream_ptr(stream):
    return None if stream is None else stream.cuda_stream


def op_attention_scratch_bytes(tkv, hkv, hd) -> int:
    out = C.c_size_t(0)
    rc = load_library().vla_op_attention_scratch_bytes(tkv, hkv, hd, C.byref(out))
    if rc != VLA_OK:
        raise VlaError(rc, "bad attention shape")
    return out.value


def op_attention(q, k, v, hq, hkv, hd, causal=False, scratch=None, stream=None):
    """q [tq, hq*hd], k/v [tkv, hkv*hd]: CUDA bf16 torch tensors.  Returns out [tq, hq*hd] bf16."""
    import torch
    tq, tkv = q.shape[0], k.shape[0]
    out = torch.empty_like(q)
    if scratch is None:
        scratch = torch.empty(op_attention_scratch_bytes(tkv, hkv, hd), dtype=torch.uint8, device=q.device)
    rc = load_library().vla_op_attention(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), tq, tkv, hq, hkv, hd,
                                         int(causal), scratch.data_ptr(), scratch.numel(), _stream_ptr(stream))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_op_attention failed")
    return out


def op_linear(a, w, act=0, out_bf16=False, stream=None):
    """a [m,k], w [n,k]: CUDA bf16 torch tensors.  Returns act(a w^T) as fp32 (or bf16) [m,n]."""
    import torch
    m, k = a.shape
    n = w.shape[0]
    out = torch.empty((m, n), dtype=torch.bfloat16 if out_bf16 else torch.float32, device=a.device)
    rc = load_library().vla_op_linear(a.data_ptr(), w.data_ptr(), None if out_bf16 else out.data_ptr(),
                                      out.data_ptr() if out_bf16 else None, m, n, k, act, _stream_ptr(stream))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_op_linear failed")
    return out


def op_attention_static(q, k, v, out, hq, hkv, hd, causal=False, stream=None):
    """Attention for callers that may not allocate: scratch lives in a fixed device array inside the library.

    Unlike ``op_attention`` this wrapper creates nothing either: the caller supplies ``out``.  Shapes whose
    scratch need exceeds the fixed array raise with VLA_ERR_NOMEM.  Calls share the array, so do not overlap them.
    """
    tq, tkv = q.shape[0], k.shape[0]
    rc = load_library().vla_op_attention_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), tq, tkv, hq, hkv, hd,
                                                int(causal), _stream_ptr(stream))
    if rc == VLA_ERR_NOMEM:
        raise VlaError(rc, "attention shape needs more scratch than the library's fixed array holds")
    if rc != VLA_OK:
        raise VlaError(rc, "vla_op_attention_static failed")
    return out


def op_status(op, scratch=None, stream=None) -> int:
    """Waits for ``stream`` and returns the operator's status word as a VLA_* code (VLA_OK or VLA_ERR_TIMEOUT)."""
    return load_library().vla_op_status(op, None if scratch is None else scratch.data_ptr(), _stream_ptr(stream))


def debug_op_fault(drop_operand_loads, wait_limit_ns=0):
    """Test hook: make the operators' bounded waits run out (see vla_debug_op_fault)."""
    rc = load_library().vla_debug_op_fault(int(bool(drop_operand_loads)), int(wait_limit_ns))
    if rc != VLA_OK:
        raise VlaError(rc, "vla_debug_op_fault failed")
