"""Checker of a device trace against the tile program (shared by the GPU tests; plain numpy).

What it proves for a co-scheduled run (Section 2.1: overlap must preserve sequential semantics):
  * every tile of every (stream, frame) ran exactly once, in the ring slot frame % depth of its stream;
  * for every edge of the node DAG, every tile of the successor started after every tile of the predecessor ended;
  * no tile of a frame started before the frame was admitted into the persistent kernel;
  * write-after-read across frames: no tile of frame n + depth of a stream (same ring slot) started before
    the emit tile of frame n had ended.
"""
import numpy as np

ADMIT_NODE = 0xFFFFFFFF
OP_EMIT = 8


def check_trace(trace, total, program, n_streams, n_frames, depth=2, expect_admissions=True):
    assert total == len(trace), "trace ring overflowed"
    adm = trace[trace["node"] == ADMIT_NODE]
    t = trace[trace["node"] != ADMIT_NODE]
    n_nodes = len(program)
    n_tiles = np.array([n["n_tiles"] for n in program], dtype=np.int64)
    tiles_per_frame = int(n_tiles.sum())
    assert len(t) == tiles_per_frame * n_streams * n_frames, (len(t), tiles_per_frame, n_streams, n_frames)
    inst = t["inst"].astype(np.int64)
    frame = t["frame"].astype(np.int64)
    node = t["node"].astype(np.int64)
    tile = t["tile"].astype(np.int64)
    stream = inst // depth
    assert (inst % depth == frame % depth).all(), "a frame ran in the wrong ring slot"
    assert node.max() < n_nodes and (tile < n_tiles[node]).all()
    assert (t["t_end"] >= t["t_start"]).all()
    # ---- exactly once: (stream, frame, node, tile) keys are all distinct and complete
    fkey = stream * n_frames + frame                       # frames are numbered 0..n_frames-1 per stream
    assert frame.max() < n_frames and stream.max() < n_streams
    first_tile = np.concatenate([[0], np.cumsum(n_tiles)[:-1]])
    key = fkey * tiles_per_frame + first_tile[node] + tile
    uniq = np.unique(key)
    assert len(uniq) == len(key), "a tile ran twice"
    assert len(uniq) == tiles_per_frame * n_streams * n_frames and uniq[0] == 0 and uniq[-1] == len(key) - 1
    # ---- per (frame, node): first start and last end
    nkey = fkey * n_nodes + node
    start = np.full(n_streams * n_frames * n_nodes, np.iinfo(np.int64).max, dtype=np.int64)
    end = np.zeros(n_streams * n_frames * n_nodes, dtype=np.int64)
    np.minimum.at(start, nkey, t["t_start"].astype(np.int64))
    np.maximum.at(end, nkey, t["t_end"].astype(np.int64))
    start = start.reshape(n_streams * n_frames, n_nodes)
    end = end.reshape(n_streams * n_frames, n_nodes)
    for i, n in enumerate(program):
        for s in n["succ"]:
            bad = end[:, i] > start[:, s]
            assert not bad.any(), ("dependency violated", n["name"], program[s]["name"], int(np.flatnonzero(bad)[0]))
    first_start = start.min(axis=1)
    # ---- admission precedes every tile of the frame
    if expect_admissions:
        assert len(adm) == n_streams * n_frames, (len(adm), n_streams * n_frames)
        akey = (adm["inst"].astype(np.int64) // depth) * n_frames + adm["frame"].astype(np.int64)
        assert len(np.unique(akey)) == len(akey), "a frame was admitted twice"
        t_adm = np.zeros(n_streams * n_frames, dtype=np.int64)
        t_adm[akey] = adm["t_start"].astype(np.int64)
        assert (first_start >= t_adm).all(), "a tile started before its frame was admitted"
    # ---- ring-slot reuse: frame n + depth starts after frame n's emit tile ended
    emit = [i for i, n in enumerate(program) if n["op"] == OP_EMIT]
    assert len(emit) == 1
    emit_end = end[:, emit[0]].reshape(n_streams, n_frames)
    fs = first_start.reshape(n_streams, n_frames)
    if n_frames > depth:
        assert (fs[:, depth:] >= emit_end[:, :-depth]).all(), "a ring slot was reused before its chunk was emitted"
    # the emit tile is the last tile of its frame
    assert (emit_end == end.max(axis=1).reshape(n_streams, n_frames)).all()
    return {"tiles": int(len(t)), "admissions": int(len(adm))}
