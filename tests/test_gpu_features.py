"""GPU parity of the calls beyond ingest / score: the node-level fold, checkpoint / resume of a
context, the deferred pipeline's ring protection, wide-fleet edge cases and the bounded wait.
Everything goes through the C ABI (ctypes binding) and is compared with the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import guard_oracle as go
from paper_2605_17879_b200 import synth
from parity_util import assert_bit_equal, compare_score, to_np
from test_gpu_parity import _rand_fleet

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2605_17879_b200 import build
    build.build_library()


def _compare_nodes(g, o, rpn, what):
    got = g.node_verdict()
    g.sync_status()
    ref = o.node_verdict(rpn)
    for key in ("node_flag", "node_tier", "node_stall"):
        assert_bit_equal(to_np(got[key]), ref[key], "%s %s" % (what, key))
    return ref


@pytest.mark.parametrize("R,M,rpn,W,cap,deferred", [
    (64, 4, 8, 20, 32, False),        # eight ranks per node, byte masks: the 64-bit fast path
    (64, 4, 8, 20, 32, True),
    (60, 3, 6, 10, 16, False),        # six ranks per node: the general path
    (48, 9, 4, 8, 12, False),         # 32-bit exceedance masks
    (4096, 8, 8, 12, 24, True),       # split cross-rank path, deferred
    (10, 2, 1, 4, 6, False),          # one rank per node: the fold is the identity
])
def test_node_verdict_matches_oracle(R, M, rpn, W, cap, deferred):
    from paper_2605_17879_b200 import guard
    T = 3 * W
    X, dirs = _rand_fleet(T, R, M, seed=7 * R + rpn)
    rng = np.random.default_rng(R + M)
    nodes = R // rpn
    for t in range(T):                                   # whole-node stalls on every metric
        for nd in rng.choice(nodes, 2, replace=False):
            if rng.random() < 0.5:
                for m in range(M):
                    X[t, nd * rpn:(nd + 1) * rpn, m] *= 2.0 if dirs[m] > 0 else 0.5
    g = guard.Guard(R, M, W, max(1, W // 2), dir=dirs, capacity=cap, topk=min(4, R), ranks_per_node=rpn, min_signals=min(2, M))
    g.set_deferred(deferred)
    o = go.Oracle(R, M, W, max(1, W // 2), min(4, R), dir=dirs, min_signals=min(2, M))
    Xd = torch.from_numpy(X).cuda()
    total_stalls = 0
    for t in range(0, T, W // 2):
        g.ingest(Xd[t:t + W // 2])
        o.ingest(X[t:t + W // 2])
        out = g.score()
        ref = o.score()
        nref = _compare_nodes(g, o, rpn, "t=%d" % t)
        compare_score(out, ref, "t=%d" % t)              # the evaluation itself is complete after sync_status
        total_stalls += int(nref["node_stall"].sum())
    assert total_stalls > 0
    if R > 3:
        assert nref["node_flag"][1 // rpn] == 1 and nref["node_flag"][(R // 2) // rpn] == 1   # the slow ranks' nodes
    # an ingest since the evaluation: no verdict
    g.ingest(Xd[:1])
    with pytest.raises(guard.GuardError) as ei:
        g.node_verdict()
    assert ei.value.code == -3
    g.close()
    if R % 7:
        g = guard.Guard(R, M, W, 1, dir=dirs, capacity=cap, ranks_per_node=7)
        g.ingest(Xd[:1])
        g.score()
        with pytest.raises(guard.GuardError) as ei:
            g.node_verdict()
        assert ei.value.code == -1
        g.close()


def test_node_verdict_on_the_streaming_configuration_prefix():
    """Streaming generator (whole-node stalls of all eight ranks), 32 768 ranks: the stall counts of the
    nodes the generator stalled, after 60 single-step ingests."""
    from paper_2605_17879_b200 import guard
    import dataclasses
    cfg = dataclasses.replace(synth.paper_configs()["streaming"], stall_p=2e-3)
    T = 60
    X = synth.fleet_block(cfg, 0, T, device="cuda")
    Xh = X.cpu().numpy()
    dirs = synth.fleet_dir(cfg.metrics)
    g = guard.Guard(cfg.ranks, cfg.metrics, cfg.W, cfg.k, dir=dirs, capacity=cfg.ring_capacity, topk=cfg.topk)
    o = go.Oracle(cfg.ranks, cfg.metrics, cfg.W, cfg.k, cfg.topk, dir=dirs)
    for t in range(T):
        g.ingest(X[t:t + 1])
        o.ingest(Xh[t:t + 1])
    out = g.score()
    ref = o.score()
    nref = _compare_nodes(g, o, 8, "streaming prefix")
    compare_score(out, ref, "streaming prefix")
    assert nref["node_stall"].sum() > 100 and nref["node_stall"].max() >= 1
    g.close()


@pytest.mark.parametrize("R,M,W,B,cap,cap2,deferred", [
    (48, 4, 10, 5, 16, 16, False),
    (48, 4, 10, 3, 16, 23, False),        # resumed into a ring of another capacity, ring wrapped
    (4096, 8, 12, 12, 24, 36, True),      # split cross-rank path + thread window path (hints are state)
    (130, 9, 12, 5, 16, 16, False),       # 32-bit exceedance masks
])
def test_state_export_import_resumes_bit_identically(R, M, W, B, cap, cap2, deferred):
    from paper_2605_17879_b200 import guard
    T = 6 * B + 3 * W
    T -= T % B
    X, dirs = _rand_fleet(T, R, M, seed=R + W)
    Xd = torch.from_numpy(X).cuda()
    kw = dict(dir=dirs, topk=min(6, R), n_consec=2, min_signals=min(2, M))
    o = go.Oracle(R, M, W, max(1, W // 2), min(6, R), dir=dirs, n_consec=2, min_signals=min(2, M))
    a = guard.Guard(R, M, W, max(1, W // 2), capacity=cap, **kw)
    a.set_deferred(deferred)
    cut = (T // B // 2) * B
    refs, outs_a = [], []
    for t in range(0, T, B):
        o.ingest(X[t:t + B])
        refs.append(o.score())
    state = None
    for i, t in enumerate(range(0, T, B)):
        if t == cut:
            state = a.state_export()
            assert state.numel() == a.state_bytes()
        a.ingest(Xd[t:t + B])
        out = a.score()
        a.sync_status()
        compare_score(out, refs[i], "uninterrupted t=%d" % t)
        outs_a.append({k: to_np(v).copy() for k, v in out.items()})
    fa, wa, ra = a.fallback_steps(), a.window_fallbacks(), a.sliding_rebuilds()
    a.close()
    b = guard.Guard(R, M, W, max(1, W // 2), capacity=cap2, **kw)
    b.set_deferred(deferred)
    b.state_import(state)
    assert b.steps_seen == cut
    for i, t in enumerate(range(0, T, B)):
        if t < cut:
            continue
        b.ingest(Xd[t:t + B])
        out = b.score()
        b.sync_status()
        compare_score(out, refs[i], "resumed t=%d" % t)
        for key, v in out.items():                       # and bit-identical to the run that never stopped
            assert np.array_equal(to_np(v).view(np.uint8), outs_a[i][key].view(np.uint8)), (key, t)
    # the resumed context took the same paths: its fallback counters continue the exported ones
    assert b.fallback_steps() == fa and b.window_fallbacks() == wa and b.sliding_rebuilds() == ra
    # rejects: another geometry, a buffer that is too small, garbage
    c = guard.Guard(R, M, W + 1, 1, capacity=cap2 + 1, dir=dirs)
    with pytest.raises(guard.GuardError) as ei:
        c.state_import(torch.zeros(c.state_bytes(), dtype=torch.uint8, device="cuda"))
    assert ei.value.code == -1
    with pytest.raises(guard.GuardError) as ei:
        b.state_import(state[:1024])
    assert ei.value.code == -2
    other = torch.zeros(max(c.state_bytes(), state.numel()), dtype=torch.uint8, device="cuda")
    other[:state.numel()] = state
    with pytest.raises(guard.GuardError) as ei:
        c.state_import(other)
    assert ei.value.code == -1
    b.close()
    c.close()


def test_state_export_before_any_step_and_before_any_evaluation():
    from paper_2605_17879_b200 import guard
    X, dirs = _rand_fleet(12, 20, 4, seed=4)
    Xd = torch.from_numpy(X).cuda()
    a = guard.Guard(20, 4, 6, 3, dir=dirs, capacity=8, topk=3)
    b = guard.Guard(20, 4, 6, 3, dir=dirs, capacity=8, topk=3)
    b.state_import(a.state_export())                     # empty state
    assert b.steps_seen == 0
    a.ingest(Xd[:4])
    b.state_import(a.state_export())                     # steps but no evaluation yet
    o = go.Oracle(20, 4, 6, 3, 3, dir=dirs)
    o.ingest(X[:4])
    b.ingest(Xd[4:9])
    o.ingest(X[4:9])
    out = b.score()
    b.sync_status()
    compare_score(out, o.score(), "resumed before the first evaluation")
    a.close()
    b.close()


def test_finite_values_whose_deviation_overflows_are_accepted_on_the_wide_paths():
    """Finite telemetry of opposite huge magnitude: x - median overflows to infinity, which is a
    legitimate deviation (the oracle accepts it), not a non-finite input."""
    from paper_2605_17879_b200 import guard
    for R, B in ((4096, 12), (20000, 9)):                # split path, cluster path
        X, dirs = _rand_fleet(2 * B, R, 8, seed=R)
        for m in (2, 7):                                 # one "larger is worse" and one "smaller is worse" metric
            X[..., m] = (X[..., m] / np.median(X[..., m])) * np.float32(1e38)
            for t in range(2 * B):                        # a rank is hit once per window: its median stays put
                X[t, (37 * t + 5) % 997:R:997, m] = np.float32(-3e38)
        assert np.isfinite(X).all()
        g = guard.Guard(R, 8, B, B // 2, dir=dirs, capacity=2 * B, topk=8)
        o = go.Oracle(R, 8, B, B // 2, 8, dir=dirs)
        Xd = torch.from_numpy(X).cuda()
        for t in range(0, 2 * B, B):
            smed = torch.empty((B, 8), dtype=torch.float32, device="cuda")
            smad = torch.empty((B, 8), dtype=torch.float32, device="cuda")
            g.ingest(Xd[t:t + B], smed, smad)
            ref_i = o.ingest(X[t:t + B])
            out = g.score()
            assert g.sync_status() == 0
            assert_bit_equal(to_np(smed), ref_i["step_med"], "step_med")
            assert_bit_equal(to_np(smad), ref_i["step_mad"], "step_mad")
            compare_score(out, o.score(), "R=%d t=%d" % (R, t))
        assert g.fallback_steps() == 0                   # served by the fast path itself
        g.close()


def test_deferred_ring_protection_with_several_ingests_between_evaluations():
    """Deferred mode on a ring of W + B steps: ingest, score, ingest, ingest.  The third ingest reuses
    slots the pending evaluation's window still reads; the library has to order it behind that
    evaluation by itself.  Every evaluation must match the oracle."""
    from paper_2605_17879_b200 import guard
    R, M, W, B = 4500, 8, 20, 10
    T = 12 * B
    X, dirs = _rand_fleet(T, R, M, seed=91)
    Xd = torch.from_numpy(X).cuda()
    for cap in (W + B, W + 2 * B, 2 * W + 4 * B):
        g = guard.Guard(R, M, W, 10, dir=dirs, capacity=cap, topk=8)
        g.set_deferred(True)
        o = go.Oracle(R, M, W, 10, 8, dir=dirs)
        bufs = [g.alloc_outputs() for _ in range(T // B)]
        refs = []
        for i, t in enumerate(range(0, T, B)):
            g.ingest(Xd[t:t + B])
            o.ingest(X[t:t + B])
            if i % 3 != 1:                               # evaluations after blocks 0, 2, 3, 5, 6, ...: one or two ingests apart
                g.score(bufs[len(refs)])
                refs.append(o.score())
        g.join()
        g.sync_status()
        for i, ref in enumerate(refs):
            compare_score(bufs[i], ref, "cap=%d eval %d" % (cap, i))
        g.close()
    # in-place producers are refused slots that deferred work still reads, whatever came in between
    g = guard.Guard(R, M, W, 10, dir=dirs, capacity=W + B, topk=8)
    g.set_deferred(True)
    g.ingest(Xd[:W])
    g.score()
    g.ingest(Xd[W:W + B])
    for _ in range(3):                                   # the evaluation may or may not have finished yet
        try:
            g.ring_reserve(B)
        except guard.GuardError as e:
            assert e.code == -3
    g.join()
    torch.cuda.synchronize()
    assert g.ring_reserve(B).shape[0] == B
    g.close()


def test_deferred_fleet_baseline_beside_a_bracketed_ingest():
    """40 000 ranks x 16 metrics: the cross-rank statistics of an ingest take the bracketed multi-kernel
    path with its one scratch; in deferred mode the fleet baseline of the pending evaluation runs
    beside the next ingest and must not share that scratch."""
    from paper_2605_17879_b200 import guard
    R, M, W, B = 40000, 16, 4, 4
    T = 5 * B
    X, dirs = _rand_fleet(T, R, M, seed=5)
    Xd = torch.from_numpy(X).cuda()
    g = guard.Guard(R, M, W, 2, dir=dirs, capacity=3 * B, topk=8)
    g.set_deferred(True)
    o = go.Oracle(R, M, W, 2, 8, dir=dirs)
    bufs = [g.alloc_outputs() for _ in range(T // B)]
    meds = []
    for i, t in enumerate(range(0, T, B)):
        smed = torch.empty((B, M), dtype=torch.float32, device="cuda")
        smad = torch.empty((B, M), dtype=torch.float32, device="cuda")
        g.ingest(Xd[t:t + B], smed, smad)
        g.score(bufs[i])
        meds.append((smed, smad))
    g.join()
    g.sync_status()
    for i, t in enumerate(range(0, T, B)):
        ref_i = o.ingest(X[t:t + B])
        assert_bit_equal(to_np(meds[i][0]), ref_i["step_med"], "step_med %d" % i)
        assert_bit_equal(to_np(meds[i][1]), ref_i["step_mad"], "step_mad %d" % i)
        compare_score(bufs[i], o.score(), "eval %d" % i)
    g.close()


def test_bounded_wait_runs_out_and_the_context_recovers():
    """The wait for a staged tile in the warp-per-series window kernel has a limit.  With the limit set
    to one clock cycle the wait runs out while the tile's copies are still in flight: the kernel must
    report GUARD_ERR_TIMEOUT through the status word, let the copies land and return; after
    guard_reset, with the default limit restored, the context works again and matches the oracle."""
    from paper_2605_17879_b200 import guard
    R, M, W = 256, 4, 64
    X, dirs = _rand_fleet(W, R, M, seed=13)
    Xd = torch.from_numpy(X).cuda()
    g = guard.Guard(R, M, W, W // 2, dir=dirs, topk=4)
    g.debug_set_wait_limit(1)
    g.ingest(Xd)
    g.score()                                            # first evaluation: warp-per-series kernel, staged tiles
    with pytest.raises(guard.GuardError) as ei:
        g.sync_status()
    assert ei.value.code == -5
    g.reset()
    g.debug_set_wait_limit(0)
    o = go.Oracle(R, M, W, W // 2, 4, dir=dirs)
    g.ingest(Xd)
    o.ingest(X)
    out = g.score()
    assert g.sync_status() == 0
    compare_score(out, o.score(), "after the reset")
    with pytest.raises(guard.GuardError):
        g.debug_set_wait_limit(-1)
    g.close()
