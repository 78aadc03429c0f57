"""Helpers shared by the GPU parity tests: run the CUDA library and the CPU oracle on the
same buffer and compare element by element.

Tolerances: every selection (medians, MADs, percentile cuts), count, mask, flag, tier and
top-k index must be bit-exact; reported robust-z scores are float32 on the GPU (one
multiply, one divide) and float64 in the oracle, compared within 1e-6 relative (absolute
1e-30 near zero)."""
import numpy as np
import torch

from oracle import guard_oracle as go

SCORE_RTOL = 1e-6
SCORE_ATOL = 1e-30

EXACT = ("wmed", "fleet_med", "fleet_mad", "counts", "mask", "flags", "tier", "topk_idx")


def bits(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a.view(np.uint32)
    return a


def assert_bit_equal(got, want, what):
    got, want = np.asarray(got), np.asarray(want)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    if not np.array_equal(bits(got), bits(want)):
        bad = np.nonzero(bits(got).ravel() != bits(want).ravel())[0]
        i = bad[0]
        raise AssertionError("%s: %d mismatches, first at %d: got %r want %r" %
                             (what, bad.size, i, got.ravel()[i], want.ravel()[i]))


def assert_scores_close(got, want, what):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, what
    inf = np.isinf(want)
    assert np.array_equal(np.isinf(got), inf), what
    assert np.array_equal(got[inf], want[inf]), what
    g, w = got[~inf], want[~inf]
    err = np.abs(g - w)
    ok = err <= SCORE_ATOL + SCORE_RTOL * np.abs(w)
    if not ok.all():
        i = np.nonzero(~ok)[0][0]
        raise AssertionError("%s: score mismatch got %r want %r" % (what, g[i], w[i]))


def to_np(t):
    return t.detach().cpu().numpy()


def compare_score(gout, oout, what=""):
    for key in EXACT:
        if gout.get(key) is not None:
            assert_bit_equal(to_np(gout[key]), oout[key], "%s %s" % (what, key))
    assert_scores_close(to_np(gout["scores"]), oout["scores"], what + " scores")
    if gout.get("topk_score") is not None and gout["topk_score"].numel():
        assert_scores_close(to_np(gout["topk_score"]), oout["topk_score"], what + " topk_score")


def run_both(X, W, k, K, dirs, blocks, capacity=None, score_every=1, in_place=False, max_fallback_steps=None, **kw):
    """Feeds X [T, R, M] (numpy float32) to both sides in the given block sizes and
    compares after every `score_every`-th block.  Returns the last oracle result."""
    from paper_2605_17879_b200 import guard
    T, R, M = X.shape
    g = guard.Guard(R, M, W, k, dir=dirs, capacity=capacity, topk=K, **kw)
    okw = {kk: v for kk, v in kw.items() if kk != "ranks_per_node"}
    o = go.Oracle(R, M, W, k, K, dir=dirs, **okw)
    Xd = torch.from_numpy(X).cuda()
    t = 0
    nb = 0
    last = None
    while t < T:
        B = blocks[nb % len(blocks)]
        B = min(B, T - t)
        smed = torch.empty((B, M), dtype=torch.float32, device="cuda")
        smad = torch.empty((B, M), dtype=torch.float32, device="cuda")
        if in_place:
            slot = g.ring_reserve(B)
            slot.copy_(Xd[t:t + B])
            g.ingest(slot, smed, smad)
        else:
            g.ingest(Xd[t:t + B].contiguous(), smed, smad)
        os_ = o.ingest(X[t:t + B])
        assert_bit_equal(to_np(smed), os_["step_med"], "step_med t=%d" % t)
        assert_bit_equal(to_np(smad), os_["step_mad"], "step_mad t=%d" % t)
        t += B
        nb += 1
        if nb % score_every == 0 or t >= T:
            gout = g.score()
            g.sync_status()
            last = o.score()
            compare_score(gout, last, "t=%d" % t)
    if max_fallback_steps is not None:
        # the fast cross-rank paths must have served the steps themselves, not the direct fallback
        assert g.fallback_steps() <= max_fallback_steps, g.fallback_steps()
    g.close()
    return last
