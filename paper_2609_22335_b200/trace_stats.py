"""Statistics over the device trace of a run (one record per executed tile).

Host-side analysis only; nothing here runs on the hot path.  The figures follow the paper's
evaluation: the fraction of the overlap window in which an SM holds work of both phases at once
(Section 5.2, "Concurrent SM Utilization"), the size of the smaller side of concurrently running
node pairs (Section 5.3, grid-size disparity), plus what a software dispatcher can read off its
own trace: how busy the worker groups were, which tile classes the busy time went to, and the
rate each class achieved inside its tiles.

A trace is a numpy structured array with the fields of ``vla_trace_rec`` (``api.TRACE_DTYPE``):
inst, node, tile, sm, worker, cls, frame, t_start, t_end (ns).  Records whose node is
``ADMIT_NODE`` mark the admission of a frame and are not tiles.
"""
from __future__ import annotations

import numpy as np

ADMIT_NODE = 0xFFFFFFFF
N_KINDS = 4
CLASS_NAMES = ["vlm_gemm", "vlm_gated_gemm", "vlm_attention", "vlm_elementwise",
               "head_gemm", "head_gated_gemm", "head_attention", "head_elementwise"]


def tiles_only(trace):
    """The tile records of a trace (admission markers removed)."""
    return trace[trace["node"] != ADMIT_NODE]


def wall_ns(trace) -> int:
    t = tiles_only(trace)
    return int(t["t_end"].max() - t["t_start"].min()) if len(t) else 0


def busy_fraction(trace, n_workers: int | None = None) -> float:
    """Sum of tile durations / (worker groups x wall time).

    ``n_workers`` defaults to the distinct (sm, worker) pairs seen in the trace; pass
    SM count x worker groups per SM to count groups that never ran a tile."""
    t = tiles_only(trace)
    if len(t) == 0:
        return 0.0
    if n_workers is None:
        n_workers = len(np.unique(t["sm"].astype(np.int64) * 256 + t["worker"]))
    busy = float((t["t_end"] - t["t_start"]).sum())
    return busy / (n_workers * wall_ns(trace))


def class_shares(trace) -> dict:
    """Share of the busy time that went to each tile class (keys of CLASS_NAMES)."""
    t = tiles_only(trace)
    dur = (t["t_end"] - t["t_start"]).astype(np.float64)
    tot = dur.sum()
    out = {}
    for c, name in enumerate(CLASS_NAMES):
        s = dur[t["cls"] == c].sum()
        if s > 0:
            out[name] = float(s / tot)
    return out


def _union_length(starts, ends) -> int:
    """Total length of the union of intervals."""
    if len(starts) == 0:
        return 0
    order = np.argsort(starts, kind="stable")
    s, e = starts[order], ends[order]
    run_end = np.maximum.accumulate(e)
    # a new run starts where an interval begins after everything before it has ended
    new = np.empty(len(s), dtype=bool)
    new[0] = True
    new[1:] = s[1:] > run_end[:-1]
    run_start = s[new]
    idx = np.flatnonzero(new)
    run_stop = np.append(run_end[idx[1:] - 1], run_end[-1])
    return int((run_stop - run_start).sum())


def _both_length(s0, e0, s1, e1) -> int:
    """Time covered by at least one interval of set 0 AND at least one of set 1: |A| + |B| - |A u B|."""
    if len(s0) == 0 or len(s1) == 0:
        return 0
    return _union_length(s0, e0) + _union_length(s1, e1) - _union_length(np.concatenate([s0, s1]), np.concatenate([e0, e1]))


def overlap_window(trace):
    """[first instant both phases have started, last instant before either has finished] over the whole GPU."""
    t = tiles_only(trace)
    ph = t["cls"] // N_KINDS
    a, b = t[ph == 0], t[ph == 1]
    if len(a) == 0 or len(b) == 0:
        return None
    lo = max(int(a["t_start"].min()), int(b["t_start"].min()))
    hi = min(int(a["t_end"].max()), int(b["t_end"].max()))
    return (lo, hi) if hi > lo else None


def concurrency_fraction(trace, n_sms: int | None = None) -> dict:
    """Fraction of the overlap window in which an SM holds tiles of BOTH phases (Section 5.2).

    Returns the mean over SMs (SMs that never ran a tile count as zero when ``n_sms`` is given),
    the best and worst SM, and the window length."""
    win = overlap_window(trace)
    if win is None:
        return {"mean": 0.0, "min": 0.0, "max": 0.0, "window_ns": 0}
    lo, hi = win
    t = tiles_only(trace)
    s = np.clip(t["t_start"].astype(np.int64), lo, hi)
    e = np.clip(t["t_end"].astype(np.int64), lo, hi)
    keep = e > s
    t, s, e = t[keep], s[keep], e[keep]
    ph = t["cls"] // N_KINDS
    fr = []
    for sm in np.unique(t["sm"]):
        m = t["sm"] == sm
        m0, m1 = m & (ph == 0), m & (ph == 1)
        fr.append(_both_length(s[m0], e[m0], s[m1], e[m1]) / (hi - lo))
    n = max(n_sms or 0, len(fr))
    fr += [0.0] * (n - len(fr))
    return {"mean": float(np.mean(fr)), "min": float(np.min(fr)), "max": float(np.max(fr)), "window_ns": int(hi - lo)}


def per_class_rates(trace, program, n_workers: int) -> dict:
    """Rates achieved inside the tiles of each class.

    ``program`` is ``Engine.program_info()``: per node its tile count, algorithmic FLOPs and the weight
    bytes its tiles stream.  For class c: FLOPs (bytes) of its executed tiles / their summed duration =
    the rate of one worker group while it runs that class; times ``n_workers`` it is the rate the GPU
    would sustain if every worker group ran such tiles at the durations observed."""
    t = tiles_only(trace)
    nf = np.array([n.get("flops", 0.0) / max(n["n_tiles"], 1) for n in program], dtype=np.float64)
    nb = np.array([n.get("weight_bytes", 0.0) / max(n["n_tiles"], 1) for n in program], dtype=np.float64)
    dur = (t["t_end"] - t["t_start"]).astype(np.float64)
    out = {}
    for c, name in enumerate(CLASS_NAMES):
        m = t["cls"] == c
        if not m.any() or dur[m].sum() <= 0:
            continue
        secs = dur[m].sum() * 1e-9
        fl, by = nf[t["node"][m]].sum(), nb[t["node"][m]].sum()
        out[name] = {"tiles": int(m.sum()), "mean_tile_us": float(dur[m].mean() * 1e-3),
                     "tflops_all_workers": float(fl / secs * n_workers / 1e12),
                     "weight_gbs_all_workers": float(by / secs * n_workers / 1e9)}
    return out


def smaller_side_of_concurrent_pairs(trace, program) -> dict:
    """Grid-size disparity (Section 5.3): for every (VLM node, head node) pair of instances whose
    execution spans overlap in time, the tile count of the smaller node; bucketed 1 / 2-10 / 11+."""
    t = tiles_only(trace)
    if len(t) == 0:
        return {"pairs": 0}
    key = t["inst"].astype(np.int64) << 40 | t["frame"].astype(np.int64) % (1 << 19) << 21 | t["node"].astype(np.int64)
    order = np.argsort(key, kind="stable")
    k, s, e = key[order], t["t_start"][order].astype(np.int64), t["t_end"][order].astype(np.int64)
    first = np.flatnonzero(np.r_[True, k[1:] != k[:-1]])
    span_s = np.minimum.reduceat(s, first)
    span_e = np.maximum.reduceat(e, first)
    node = (k[first] & ((1 << 21) - 1)).astype(np.int64)
    ntiles = np.array([program[n]["n_tiles"] for n in node])
    phase = np.array([program[n]["phase"] for n in node])
    a = np.flatnonzero(phase == 0)
    b = np.flatnonzero(phase == 1)
    if len(a) == 0 or len(b) == 0:
        return {"pairs": 0}
    # for each head node instance, the VLM node instances alive during it (sorted sweep by start time)
    oa = a[np.argsort(span_s[a], kind="stable")]
    sa, ea, ta = span_s[oa], span_e[oa], ntiles[oa]
    small = []
    step = max(1, len(b) // 20000)          # sample when the trace is very large
    for j in b[::step]:
        hi = np.searchsorted(sa, span_e[j], side="left")
        alive = ea[:hi] > span_s[j]
        if alive.any():
            small.append(np.minimum(ta[:hi][alive], ntiles[j]))
    if not small:
        return {"pairs": 0}
    sm = np.concatenate(small)
    return {"pairs": int(len(sm)), "one_tile": float((sm == 1).mean()), "two_to_ten": float(((sm >= 2) & (sm <= 10)).mean()),
            "eleven_plus": float((sm >= 11).mean()), "median": float(np.median(sm))}


def gap_stats(trace) -> dict:
    """Idle time of the worker groups between two consecutive tiles, by the class of the tile that ended the gap.

    For every (sm, worker) the tiles are ordered by start time; gap = start of the next tile - end of this one.
    Returns per class: gaps, mean / median / 90th percentile in microseconds, and the class's share of all idle time
    between tiles (idle time before a worker's first and after its last tile is not counted)."""
    t = tiles_only(trace)
    if len(t) < 2:
        return {}
    key = t["sm"].astype(np.int64) * 256 + t["worker"]
    order = np.lexsort((t["t_start"], key))
    k, s, e, c = key[order], t["t_start"][order].astype(np.int64), t["t_end"][order].astype(np.int64), t["cls"][order]
    same = k[1:] == k[:-1]
    gap = (s[1:] - e[:-1])[same].astype(np.float64)
    nxt = c[1:][same]
    gap = np.maximum(gap, 0.0)
    if len(gap) == 0:
        return {}
    tot = gap.sum()
    out = {"all": {"gaps": int(len(gap)), "mean_us": float(gap.mean() * 1e-3), "median_us": float(np.median(gap) * 1e-3),
                   "p90_us": float(np.percentile(gap, 90) * 1e-3)}}
    for ci, name in enumerate(CLASS_NAMES):
        g = gap[nxt == ci]
        if len(g):
            out[name] = {"gaps": int(len(g)), "mean_us": float(g.mean() * 1e-3), "median_us": float(np.median(g) * 1e-3),
                         "p90_us": float(np.percentile(g, 90) * 1e-3), "share_of_idle": float(g.sum() / tot) if tot > 0 else 0.0}
    prv = c[:-1][same]
    for a_, an in ((0, "vlm"), (1, "head")):          # by the phases of the tile before and the tile after the gap
        for b_, bn in ((0, "vlm"), (1, "head")):
            g = gap[(prv // N_KINDS == a_) & (nxt // N_KINDS == b_)]
            if len(g):
                out[f"{an}->{bn}"] = {"gaps": int(len(g)), "mean_us": float(g.mean() * 1e-3), "median_us": float(np.median(g) * 1e-3),
                                      "share_of_idle": float(g.sum() / tot) if tot > 0 else 0.0}
    return out


def _node_instance_spans(t):
    """Per executed node instance (request-stream slot, frame, node): key, first start, last end, tiles seen."""
    key = t["inst"].astype(np.int64) << 40 | t["frame"].astype(np.int64) % (1 << 19) << 21 | t["node"].astype(np.int64)
    order = np.argsort(key, kind="stable")
    k, s, e = key[order], t["t_start"][order].astype(np.int64), t["t_end"][order].astype(np.int64)
    first = np.flatnonzero(np.r_[True, k[1:] != k[:-1]])
    return k[first], np.minimum.reduceat(s, first), np.maximum.reduceat(e, first), np.diff(np.r_[first, len(k)])


def backlog_stats(trace, program, n_workers: int) -> dict:
    """Was there work for the idle workers?  (Starvation against dispatch latency.)

    A tile is READY from the moment the last tile of the last predecessor node of its frame has ended (for a node
    without predecessors: from the frame's admission) and WAITS until it starts.  The backlog at time t is the number of
    ready tiles that have not started.  Reported: how long a tile waits once ready (by phase), the time-weighted mean
    backlog, and -- the figure that tells the two causes of idle workers apart -- the share of the worker-idle time
    (between a worker's tiles) during which the backlog was empty (nothing to run anywhere: the dependency chains are
    the limit) against non-empty (tiles were ready, but claim, hand-over and room had not caught up)."""
    t = tiles_only(trace)
    if len(t) == 0:
        return {}
    adm = trace[trace["node"] == ADMIT_NODE]
    key, span_s, span_e, seen = _node_instance_spans(t)
    node = (key & ((1 << 21) - 1)).astype(np.int64)
    inst_frame = key >> 21
    n_nodes = len(program)
    # ready time of every executed node instance: admission of its frame, then the ends of its predecessors
    ready = np.zeros(len(key), dtype=np.int64)
    if len(adm):
        akey = adm["inst"].astype(np.int64) << 19 | adm["frame"].astype(np.int64) % (1 << 19)
        ao = np.argsort(akey, kind="stable")
        pos = np.clip(np.searchsorted(akey[ao], inst_frame), 0, len(ao) - 1)
        hit = akey[ao][pos] == inst_frame
        ready = np.where(hit, adm["t_start"][ao][pos].astype(np.int64), span_s)     # (no marker: never earlier than its start)
    else:
        ready = span_s.copy()
    index = {int(k): i for i, k in enumerate(key)}
    preds = [[] for _ in range(n_nodes)]
    for u, n in enumerate(program):
        for v in n["succ"]:
            preds[v].append(u)
    for i in range(len(key)):
        base = int(inst_frame[i]) << 21
        for u in preds[int(node[i])]:
            j = index.get(base | u)
            if j is not None and span_e[j] > ready[i]:
                ready[i] = span_e[j]
    # per tile: the wait between ready and start
    tkey = t["inst"].astype(np.int64) << 40 | t["frame"].astype(np.int64) % (1 << 19) << 21 | t["node"].astype(np.int64)
    pos = np.searchsorted(key, tkey)
    t_ready = ready[pos]
    ts = t["t_start"].astype(np.int64)
    wait = np.maximum(ts - t_ready, 0).astype(np.float64)
    ph = t["cls"] // N_KINDS
    out = {"wait_ready_to_start_us": {nm: {"mean": float(wait[ph == q].mean() * 1e-3), "median": float(np.median(wait[ph == q]) * 1e-3),
                                             "p90": float(np.percentile(wait[ph == q], 90) * 1e-3)}
                                      for q, nm in ((0, "vlm"), (1, "head")) if (ph == q).any()}}
    # backlog(t): +1 per tile at its ready time, -1 at its start
    ev_t = np.concatenate([t_ready, ts])
    ev_d = np.concatenate([np.ones(len(ts), dtype=np.int64), -np.ones(len(ts), dtype=np.int64)])
    o = np.lexsort((ev_d, ev_t))          # at equal times the starts (-1) come first: never a phantom backlog
    ev_t, backlog = ev_t[o], np.cumsum(ev_d[o])
    dt = np.diff(ev_t).astype(np.float64)
    if dt.sum() > 0:
        out["mean_backlog_tiles"] = float((backlog[:-1] * dt).sum() / dt.sum())
    # idle intervals of the workers, split by whether tiles were ready meanwhile (sampled at 4 points per gap)
    wk = t["sm"].astype(np.int64) * 256 + t["worker"]
    order = np.lexsort((t["t_start"], wk))
    k2, s2, e2 = wk[order], ts[order], t["t_end"][order].astype(np.int64)
    same = k2[1:] == k2[:-1]
    g0, g1 = e2[:-1][same], s2[1:][same]
    keep = g1 > g0
    g0, g1 = g0[keep], g1[keep]
    if len(g0):
        length = (g1 - g0).astype(np.float64)
        empty = np.zeros(len(g0)); few = np.zeros(len(g0))
        for f in (0.125, 0.375, 0.625, 0.875):
            at = g0 + (length * f).astype(np.int64)
            b = backlog[np.clip(np.searchsorted(ev_t, at, side="right") - 1, 0, len(backlog) - 1)]
            empty += (b <= 0) * 0.25
            few += ((b > 0) & (b < n_workers // 8)) * 0.25
        tot = length.sum()
        out["idle_between_tiles"] = {"share_with_empty_backlog": float((empty * length).sum() / tot),
                                     "share_with_short_backlog": float((few * length).sum() / tot),
                                     "share_with_deep_backlog": float(((1.0 - empty - few) * length).sum() / tot),
                                     "short_backlog_means_fewer_than": int(n_workers // 8)}
    return out


def summary(trace, program=None, n_sms: int | None = None, workers_per_sm: int = 3) -> dict:
    """Everything the benchmark line reports from one traced pass."""
    n_workers = (n_sms * workers_per_sm) if n_sms else None
    out = {"tiles": int(len(tiles_only(trace))), "wall_ms": wall_ns(trace) * 1e-6,
           "sm_busy_frac": busy_fraction(trace, n_workers), "class_share_of_busy_time": class_shares(trace),
           "concurrency": concurrency_fraction(trace, n_sms), "gaps_between_tiles": gap_stats(trace)}
    if program is not None and n_workers:
        out["per_class"] = per_class_rates(trace, program, n_workers)
        out["smaller_side_of_concurrent_node_pairs"] = smaller_side_of_concurrent_pairs(trace, program)
        if all("succ" in n for n in program):
            out["backlog"] = backlog_stats(trace, program, n_workers)
    return out
