"""Full-size parity: the five workloads at their stated shapes and request-stream counts, in the
co-scheduled launch configuration the benchmark times, against the CPU oracle on sampled chunks
(first, middle and last stream; first and last frame), bit-identity with a stream mode, and the
device trace of the full-size SmolVLA-shaped run checked against the tile DAG."""
import numpy as np
import pytest

from oracle import vla_oracle as O
from vla_synth.configs import CFG1, CFG2, CFG3, CFG4, CFG5
from vla_synth.gen import make_weights, frame_inputs

pytestmark = pytest.mark.gpu

REL_L2_TOL = 1e-2
MAX_ABS_TOL = 3e-2


@pytest.mark.parametrize("m,frames,check_two_stream", [(CFG1, 8, True), (CFG2, 2, True), (CFG3, 2, False), (CFG4, 2, False),
                                                        (CFG5, 2, False)], ids=lambda v: getattr(v, "name", str(v)))
def test_full_size_sampled_parity(m, frames, check_two_stream):
    from paper_2609_22335_b200 import Engine
    w = make_weights(m, seed=0, cache=(m is not CFG5))
    R = m.n_streams
    fr = [[frame_inputs(m, r, n, seed=0) for n in range(frames)] for r in range(R)]
    eng = Engine(m, mode="cosched", n_streams=R)
    try:
        eng.load_weights(w)
        got = eng.run(fr, timeout_s=900)
    finally:
        eng.close()
    samples = [(0, 0), (R // 2, 0), (R - 1, frames - 1)] if m is not CFG5 else [(R - 1, frames - 1)]
    for (r, n) in samples:
        ref = O.action_chunk(m, w, fr[r][n], np.float32)
        rel = float(np.linalg.norm(got[r][n] - ref) / np.linalg.norm(ref))
        mx = float(np.max(np.abs(got[r][n] - ref)))
        rms = float(np.sqrt(np.mean(ref * ref)))
        print(f"{m.name} stream {r} frame {n}: rel-L2 {rel:.2e}, max-abs {mx:.3e}, chunk rms {rms:.2f}")
        # DDIM chunks (rms 4-7 with an untrained eps-network): the absolute bound is taken relative to the chunk's
        # scale, see tests/test_gpu_parity.py::_check_vs_oracle; Euler chunks are held to the plain 3e-2
        scale = max(1.0, rms) if m.solver == "ddim" else 1.0
        assert rel <= REL_L2_TOL, (m.name, r, n, rel)
        assert mx <= MAX_ABS_TOL * scale, (m.name, r, n, mx, rms)
    # every chunk of every stream is finite and distinct streams differ
    for r in range(R):
        for n in range(frames):
            assert np.isfinite(got[r][n]).all()
    assert not np.array_equal(got[0][0], got[R - 1][0])
    if check_two_stream or m is CFG3:
        eng = Engine(m, mode="two_stream" if check_two_stream else "multi_stream", n_streams=R)
        try:
            eng.load_weights(w)
            got2 = eng.run(fr, timeout_s=900)
        finally:
            eng.close()
        for r in range(R):
            for n in range(frames):
                assert np.array_equal(got[r][n], got2[r][n]), (m.name, r, n)


# (The blocked suffix mask on the full pi0-shaped model and classifier-free guidance on the full CogACT-shaped one pass the
# same test -- rel-L2 1.6e-3 / 2.7e-3 -- but the oracle needs minutes for them; they stay covered at reduced size.)
@pytest.mark.parametrize("base,variant", [(CFG2, {"vis_layernorm": 1})], ids=["cfg2_vision_layernorm_bias"])
def test_full_size_workload_variants(base, variant):
    """The workload variants at full model size (four request streams, one frame each; one chunk against the oracle,
    all chunks bit-identical between the co-scheduled and the serial run)."""
    from paper_2609_22335_b200 import Engine
    from vla_synth.configs import mini
    m = mini(base, **variant)
    w = make_weights(m, seed=0, cache=False)
    R = 4
    fr = [[frame_inputs(m, r, 0, seed=0)] for r in range(R)]
    outs = {}
    for mode in ("cosched", "serial"):
        eng = Engine(m, mode=mode, n_streams=R)
        try:
            eng.load_weights(w)
            outs[mode] = eng.run(fr, timeout_s=900)
        finally:
            eng.close()
    for r in range(R):
        assert np.array_equal(outs["cosched"][r][0], outs["serial"][r][0]), (m.name, r)
    ref = O.action_chunk(m, w, fr[R - 1][0], np.float32)
    got = outs["cosched"][R - 1][0]
    rel = float(np.linalg.norm(got - ref) / np.linalg.norm(ref))
    mx = float(np.max(np.abs(got - ref)))
    rms = float(np.sqrt(np.mean(ref * ref)))
    print(f"{m.name} {variant}: rel-L2 {rel:.2e}, max-abs {mx:.3e}, chunk rms {rms:.2f}")
    scale = max(1.0, rms) if m.solver == "ddim" else 1.0
    assert rel <= REL_L2_TOL and mx <= MAX_ABS_TOL * scale, (m.name, rel, mx, rms)


def test_full_size_trace_respects_the_dag():
    """32 request streams x 3 frames of the SmolVLA-shaped workload, co-scheduled, with the device trace on: every
    one of the 2.6 million tiles ran exactly once, after its frame's admission and after all tiles of its
    predecessors; the third frame of a stream did not start before the first one's chunk was emitted."""
    from paper_2609_22335_b200 import Engine
    from trace_check import check_trace
    m, F = CFG2, 3
    w = make_weights(m, seed=0)
    R = m.n_streams
    probe = Engine(m, mode="cosched", n_streams=1)
    tiles_per_frame = sum(n["n_tiles"] for n in probe.program_info())
    probe.close()
    fr = [[frame_inputs(m, r, n % 2, seed=0) for n in range(F)] for r in range(R)]
    eng = Engine(m, mode="cosched", n_streams=R, trace_capacity=(tiles_per_frame + 1) * R * F + 1024)
    try:
        eng.load_weights(w)
        eng.run(fr, timeout_s=900)
        eng.wait_idle()
        trace, total = eng.trace()
        stats = check_trace(trace, total, eng.program_info(), R, F)
    finally:
        eng.close()
    assert stats["tiles"] == tiles_per_frame * R * F and stats["admissions"] == R * F
