"""Times the stand-alone operators (the engine's GEMM and attention tile bodies as ordinary kernels).

    python -m paper_2609_22335_b200.opbench linear M N K [--act 0|1|2] [--f32] [--iters 20]
    python -m paper_2609_22335_b200.opbench attention TQ TKV HQ HKV HD [--causal] [--iters 20]

Prints one JSON line: microseconds per call (CUDA events around `iters` back-to-back calls after three
warm-up calls) and the achieved TFLOP/s (2 M N K, or 4 TQ TKV HQ HD).  Also the command to put under ncu
when a tile body is profiled on its own.
"""
from __future__ import annotations

import argparse
import json


def _time(fn, iters):
    import torch
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3


def main(argv=None):
    import torch
    from . import api
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("op", choices=["linear", "attention"])
    ap.add_argument("dims", type=int, nargs="+")
    ap.add_argument("--act", type=int, default=0)
    ap.add_argument("--f32", action="store_true", help="linear: fp32 output instead of bf16")
    ap.add_argument("--causal", action="store_true")
    ap.add_argument("--iters", type=int, default=20)
    a = ap.parse_args(argv)
    g = torch.Generator(device="cuda").manual_seed(0)
    rnd = lambda *s: torch.randn(*s, device="cuda", generator=g).to(torch.bfloat16)  # noqa: E731
    if a.op == "linear":
        m, n, k = a.dims
        x, w = rnd(m, k), (0.05 * torch.randn(n, k, device="cuda", generator=g)).to(torch.bfloat16)
        us = _time(lambda: api.op_linear(x, w, act=a.act, out_bf16=not a.f32), a.iters)
        status = api.op_status(api.OP_LINEAR)
        flops = 2.0 * m * n * k
        out = {"op": "linear", "m": m, "n": n, "k": k, "act": a.act, "out": "f32" if a.f32 else "bf16"}
    else:
        tq, tkv, hq, hkv, hd = a.dims
        q, kk, v = rnd(tq, hq * hd), rnd(tkv, hkv * hd), rnd(tkv, hkv * hd)
        scratch = torch.empty(api.op_attention_scratch_bytes(tkv, hkv, hd), dtype=torch.uint8, device="cuda")
        us = _time(lambda: api.op_attention(q, kk, v, hq, hkv, hd, causal=a.causal, scratch=scratch), a.iters)
        status = api.op_status(api.OP_ATTENTION, scratch)
        flops = 4.0 * tq * tkv * hq * hd
        out = {"op": "attention", "tq": tq, "tkv": tkv, "hq": hq, "hkv": hkv, "hd": hd, "causal": a.causal}
    out.update({"us_per_call": round(us, 2), "tflops": round(flops / us / 1e6, 1), "status": status})
    print(json.dumps(out))


if __name__ == "__main__":
    main()
