"""Failure paths and policy variants on the GPU.  Every failure is injected from the host (a dependency counter
raised by a host copy, operand loads switched off by a flag): a bounded device-side wait then runs out, the kernel
records the error and RETURNS, and the host sees a sticky VLA_ERR_TIMEOUT.  Nothing here faults or hangs the GPU."""
import random
import time

import numpy as np
import pytest

from oracle import vla_oracle as O
from vla_synth.configs import CFG1, CFG2, CFG4, mini
from vla_synth.gen import make_weights, frame_inputs, round_to_bf16

pytestmark = pytest.mark.gpu


def _cfg1_parity():
    from paper_2609_22335_b200 import Engine
    m = CFG1
    w = make_weights(m, seed=0)
    frames = [[frame_inputs(m, r, n, seed=0) for n in range(2)] for r in range(2)]
    eng = Engine(m, mode="cosched", n_streams=2)
    try:
        eng.load_weights(w)
        got = eng.run(frames)
    finally:
        eng.close()
    for r in range(2):
        for n in range(2):
            ref = O.action_chunk(m, w, frames[r][n], np.float32)
            assert np.linalg.norm(got[r][n] - ref) / np.linalg.norm(ref) <= 1e-2
            assert np.max(np.abs(got[r][n] - ref)) <= 3e-2


def test_stalled_frame_times_out_and_the_context_stays_usable():
    """A node whose dependency counter can never reach zero: the idle watchdog of the persistent kernel runs out,
    the kernel returns, poll/submit report the sticky timeout, destroy works, and a fresh context is healthy."""
    from paper_2609_22335_b200 import Engine, api
    m = CFG1
    w = make_weights(m, seed=0)
    eng = Engine(m, mode="cosched", n_streams=2, wait_limit_ns=2_000_000)       # 2 ms
    try:
        eng.load_weights(w)
        prog = eng.program_info()
        victim = next(i for i, n in enumerate(prog) if n["phase"] == 1 and n["n_pred"] > 0 and n["name"].endswith("L1.w2"))
        eng.bump_dependency(0, 0, victim, 1)                 # stream 0, ring slot 0: one predecessor tile too many
        fr = frame_inputs(m, 0, 0, seed=0)
        assert eng.submit(0, fr) == api.VLA_OK
        t0 = time.time()
        code = None
        while time.time() - t0 < 20:
            try:
                if eng.poll(0) is not None:
                    break
            except api.VlaError as e:
                code = e.code
                break
            time.sleep(0.001)
        assert code == api.VLA_ERR_TIMEOUT, code
        assert time.time() - t0 < 5.0                        # the watchdog fired after milliseconds, not the 20 s above
        assert "wait ran out" in eng.last_error()
        with pytest.raises(api.VlaError) as e:               # sticky: later calls keep reporting it
            eng.submit(1, fr)
        assert e.value.code == api.VLA_ERR_TIMEOUT
        with pytest.raises(api.VlaError) as e:
            eng.wait_idle(100)
        assert e.value.code == api.VLA_ERR_TIMEOUT
        import torch
        torch.cuda.synchronize()                             # the persistent kernel has returned: nothing is left running
    finally:
        eng.close()                                          # vla_destroy succeeds on the failed context
    _cfg1_parity()                                           # and the device is healthy for a fresh one


def test_operator_wait_runs_out_and_status_reports_it():
    """vla_op_linear / vla_op_attention with their operand loads switched off: the MMA issuer's bounded wait runs
    out, the kernels return, vla_op_status says VLA_ERR_TIMEOUT; switched back on, the same calls are correct."""
    import torch
    from paper_2609_22335_b200 import api
    rng = np.random.default_rng(1)
    a = torch.from_numpy(round_to_bf16(rng.standard_normal((40, 128)).astype(np.float32))).cuda().to(torch.bfloat16)
    w = torch.from_numpy(round_to_bf16(0.1 * rng.standard_normal((96, 128)).astype(np.float32))).cuda().to(torch.bfloat16)
    q = torch.from_numpy(round_to_bf16(rng.standard_normal((20, 128)).astype(np.float32))).cuda().to(torch.bfloat16)
    kv = torch.from_numpy(round_to_bf16(rng.standard_normal((70, 128)).astype(np.float32))).cuda().to(torch.bfloat16)
    scratch = torch.empty(api.op_attention_scratch_bytes(70, 2, 64), dtype=torch.uint8, device="cuda")
    out_s = torch.empty_like(q)
    assert api.op_status(api.OP_LINEAR) == api.VLA_OK
    api.debug_op_fault(True, wait_limit_ns=1_000_000)        # 1 ms
    try:
        api.op_linear(a, w)
        assert api.op_status(api.OP_LINEAR) == api.VLA_ERR_TIMEOUT
        api.op_attention(q, kv, kv, 2, 2, 64, scratch=scratch)
        assert api.op_status(api.OP_ATTENTION, scratch) == api.VLA_ERR_TIMEOUT
        api.op_attention_static(q, kv, kv, out_s, 2, 2, 64)
        assert api.op_status(api.OP_ATTENTION_STATIC) == api.VLA_ERR_TIMEOUT
    finally:
        api.debug_op_fault(False)
    good = api.op_linear(a, w)
    assert api.op_status(api.OP_LINEAR) == api.VLA_OK        # the word is cleared by the next call
    ref = a.float().cpu().numpy().astype(np.float64) @ w.float().cpu().numpy().astype(np.float64).T
    assert np.max(np.abs(good.cpu().numpy() - ref)) <= 2e-3 * np.abs(ref).max()
    o1 = api.op_attention(q, kv, kv, 2, 2, 64, scratch=scratch)
    assert api.op_status(api.OP_ATTENTION, scratch) == api.VLA_OK
    o2 = api.op_attention_static(q, kv, kv, out_s, 2, 2, 64)
    assert api.op_status(api.OP_ATTENTION_STATIC) == api.VLA_OK
    assert torch.equal(o1, o2)
    assert api.op_status(7) == api.VLA_ERR_INVALID
    assert api.op_status(api.OP_ATTENTION, None) == api.VLA_ERR_INVALID


def test_tiles_of_mixed_sizes_never_starve_for_room():
    """Head-dimension-256 attention tiles (36 of an SM's 55 shared-memory units) next to 16-18-unit GEMM tiles:
    a worker that waits for room is served before its SM's other workers get new tiles, so with a wait limit far
    below the default the run completes without a timeout, bit-identical to the serial mode."""
    from paper_2609_22335_b200 import Engine
    m = mini(CFG4, n_cam=2, img=112, vis_layers=1, llm_layers=2, act_layers=2, mlp=1024, n_steps=3, vocab=2048,
             n_streams=4, n_frames=4)
    w = make_weights(m, seed=0)
    frames = [[frame_inputs(m, r, n, seed=0) for n in range(m.n_frames)] for r in range(m.n_streams)]
    out = {}
    for mode, limit in (("serial", 0), ("cosched", 500_000_000)):
        eng = Engine(m, mode=mode, n_streams=m.n_streams, wait_limit_ns=limit)
        try:
            eng.load_weights(w)
            out[mode] = eng.run(frames)
        finally:
            eng.close()
    for r in range(m.n_streams):
        for n in range(m.n_frames):
            assert np.array_equal(out["cosched"][r][n], out["serial"][r][n])


def test_policy_probe_score_variants_match_the_oracle():
    """The -G and -R Phase-2 scores (Section 4) of the device pick, run on the GPU, against the oracle's exact ratios."""
    from oracle.admission_oracle import SMState, admission_decision
    from paper_2609_22335_b200 import policy_probe
    rnd = random.Random(12)
    for _ in range(40):
        n = rnd.randint(1, 6)
        taus = [tuple(rnd.randint(0, 15) for _ in range(3)) for _ in range(n)]
        st = SMState(n)
        st.cta_count = [rnd.randint(0, 3) for _ in range(n)]
        st.u = [sum(st.cta_count[k] * taus[k][x] for k in range(n)) for x in range(3)]
        pending = [rnd.random() < 0.8 for _ in range(n)]
        feas = [rnd.random() < 0.8 for _ in range(n)]
        rr = rnd.randint(0, n - 1)
        grid = [rnd.choice([1, 3, 30, 444, 100000]) for _ in range(n)]
        res = [rnd.choice([1, 12, 16, 18, 36]) for _ in range(n)]
        for policy, variant in ((3, "G"), (4, "R")):
            got = policy_probe(taus, pending, feas, st.cta_count, st.u, rr, u_max=45, policy=policy, grid=grid, res=res)
            so = st.copy()
            k, ph = admission_decision(so, taus, pending, feas, rr_start=rr, u_max=45, variant=variant, grid=grid, regs=res)
            assert got[0] == (-1 if k is None else k) and got[1] == ph, (variant, taus, st.cta_count, grid, res)


@pytest.mark.parametrize("policy", [1, 2, 3, 4])
def test_every_pick_policy_gives_the_same_chunks(policy):
    """The pick decides WHEN tiles run, never what they compute: class order, round robin, -G and -R all reproduce
    the chunks of the two-phase pick bit for bit, and their traces respect the DAG."""
    from paper_2609_22335_b200 import Engine
    from trace_check import check_trace
    m = mini(CFG2, img=128, vis_layers=2, llm_layers=3, act_layers=3, n_steps=3, vocab=2048, n_streams=3, n_frames=3)
    w = make_weights(m, seed=0)
    frames = [[frame_inputs(m, r, n, seed=0) for n in range(m.n_frames)] for r in range(m.n_streams)]
    out = {}
    for pol in (0, policy):
        eng = Engine(m, mode="cosched", n_streams=m.n_streams, policy=pol, trace_capacity=1 << 20)
        try:
            eng.load_weights(w)
            out[pol] = eng.run(frames)
            eng.wait_idle()
            trace, total = eng.trace()
            check_trace(trace, total, eng.program_info(), m.n_streams, m.n_frames)
        finally:
            eng.close()
    for r in range(m.n_streams):
        for n in range(m.n_frames):
            assert np.array_equal(out[0][r][n], out[policy][r][n])


def test_class_tags_round_trip_and_leave_the_chunks_unchanged():
    """vla_set_class_tags / vla_get_class_tags: tags steer the pick only -- the chunks stay bit-identical."""
    from paper_2609_22335_b200 import Engine, api
    m = CFG1
    w = make_weights(m, seed=0)
    frames = [[frame_inputs(m, r, n, seed=0) for n in range(2)] for r in range(2)]
    eng = Engine(m, mode="cosched", n_streams=2)
    try:
        eng.load_weights(w)
        hand = eng.class_tags()
        assert len(hand) == 8 and all(0 <= t <= 15 for row in hand for t in row)
        base = eng.run(frames)
        new = [[(3 * k + x) % 16 for x in range(3)] for k in range(8)]
        new[5] = None                                    # keep the current tags of class 5
        eng.set_class_tags(new)
        got = eng.class_tags()
        assert got[5] == hand[5] and all(got[k] == new[k] for k in range(8) if k != 5)
        again = eng.run(frames)
        for r in range(2):
            for n in range(2):
                assert np.array_equal(again[r][n], base[r][n])
        bad = (api.C.c_int32 * 24)(*([16] * 24))
        assert eng.lib.vla_set_class_tags(eng.ctx, bad) == api.VLA_ERR_INVALID
    finally:
        eng.close()
