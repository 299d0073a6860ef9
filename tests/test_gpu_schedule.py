"""Replay of the recorded event order of the pipelined layer steps against the hazard rules of the
layer-scoped ring (Sec. 5.4 "Two-layer ping-pong buffering"; Sec. 5.3 for the urgent stream):

  read-after-write   the gather of layer step n is complete before the attention of n starts
  write-after-read   the attention of n is done before the gather of n + D (same slot) starts
  urgent stream      the missing pages of n are fetched after the prefetch of n is complete and before the
                     attention of n starts ("all transfers of the layer complete")

The timeline (dd_trace_*) holds, per call n, points of the compute stream and the start / end of the gather
that call n enqueued, which is gather n + min(D, L). The rules are checked for every n of a run that spans
several step boundaries, for ring depths 2..4, every gather engine, a selection stream, and miss correction.
Timing events that are ordered by a stream or an event wait carry non-decreasing time stamps, so the
comparisons need no slack."""
import numpy as np
import pytest
import torch

from paper_2607_26475_b200 import workloads as wl
from tests.test_gpu_pipeline import _inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dd():
    from paper_2607_26475_b200 import binding
    return binding


def check_schedule(tr: np.ndarray, ahead: int, corrected: bool, depth: int | None = None):
    """tr [n, 8] microseconds (see dd_trace_begin); row i is layer step i and carries the gather of layer step
    i + ahead, whose slot was last read by layer step i + ahead - depth. Returns the number of rule instances
    checked."""
    depth = ahead if depth is None else depth
    n = len(tr)
    checked = 0
    assert np.all(np.diff(tr[:, 0]) >= 0.0), "calls are ordered on the compute stream"
    assert np.all(np.diff(tr[:, :4], axis=1) >= 0.0), "points 0..3 of a call are ordered"
    assert np.all(tr[:, 5] >= tr[:, 4]), "a gather ends after it starts"
    for i in range(n):
        # write-after-read: the gather enqueued by call i (for i + ahead) reuses the slot of call i + ahead - depth
        r = i + ahead - depth
        if r >= 0:
            assert tr[r, 2] <= tr[i, 4], f"call {i}: gather of {i + ahead} started before attention {r} released the slot"
            checked += 1
        if i + ahead < n:
            # read-after-write: that gather is complete before attention i + ahead starts
            assert tr[i, 5] <= tr[i + ahead, 1], f"attention {i + ahead} started before its gather was complete"
            checked += 1
            if corrected:
                assert tr[i, 5] <= tr[i + ahead, 6], f"urgent fetch of {i + ahead} started before the prefetch was complete"
                checked += 1
        if corrected:
            assert tr[i, 6] <= tr[i, 7] <= tr[i, 1], f"call {i}: attention started before the missing pages arrived"
            checked += 1
    # gathers are issued in order on one stream
    assert np.all(np.diff(tr[:, 4]) >= 0.0)
    return checked


CASES = [
    dict(depth=2), dict(depth=3), dict(depth=4),
    dict(depth=2, mode="bulk"), dict(depth=3, mode="bulk"),
    dict(depth=2, mode="staged"), dict(depth=4, mode="staged"),
    dict(depth=2, side=True), dict(depth=3, side=True),
    dict(depth=2, correct=True), dict(depth=3, correct=True), dict(depth=2, correct=True, side=True),
    dict(depth=4, layers=2),                      # ring deeper than the model
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()))
def test_recorded_order_obeys_the_hazard_rules(dd, case):
    S = 4                                           # three step boundaries inside the trace
    L = case.get("layers", 4)
    depth = case["depth"]
    w = wl.small(wl.CONFIGS[2], n_layers=L, batch=2, ctx=16 * 160, budget=16 * 24)
    store, lms, ctx_len, npg, q_init, q_steps = _inputs(w, S)
    mode = {"loads": dd.DD_GATHER_LOADS, "bulk": dd.DD_GATHER_BULK, "staged": dd.DD_GATHER_STAGED}[case.get("mode", "loads")]
    kw = dict(stage_min_run_pages=2) if mode == dd.DD_GATHER_STAGED else {}
    c = dd.Context(n_layers=L, batch=w.batch, max_pages=w.n_pages, k_pages=w.k_pages, ring_depth=depth,
                   gather_mode=mode, miss_correction=case.get("correct", False),
                   select_stream=torch.cuda.Stream() if case.get("side") else None, **kw)
    c.bind([x.cuda() for x in lms], store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    qd = q_steps.cuda()
    outs = torch.zeros_like(qd)
    c.trace_begin(S * L)
    for t in range(S):
        for l in range(L):
            c.decode_layer_step(t, l, qd[t, l], outs[t, l])
    tr = c.trace_end()
    assert c.device_error() == (0, 0)
    c.close()
    assert tr.shape == (S * L, dd.DD_TRACE_FIELDS)
    n_checked = check_schedule(tr.astype(np.float64), ahead=min(depth, L), corrected=case.get("correct", False),
                               depth=depth)
    assert n_checked >= 2 * S * L - depth - min(depth, L)
