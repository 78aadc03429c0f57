"""Pins for the CPU oracle: it is checked against things other than itself.

Hand-worked fixtures, numpy's sort/median, a pure-Python brute force with which it
shares no code, the Gaussian closed form behind the 0.6745 constant, and the
behavioural invariants that Section 4.2 of the paper states in words (peer-relative,
multi-signal, sustained-not-transient, step time primary, response tiers) and
Section 5.4 (a node passes only if everything passes).
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import brute
from oracle import guard_oracle as go

GOLD = os.path.join(os.path.dirname(__file__), "golden")
F = np.float32


def _lines(name):
    with open(os.path.join(GOLD, name)) as f:
        for ln in f:
            ln = ln.strip()
            if ln and not ln.startswith("#"):
                yield ln


# ------------------------------------------------------------------ order statistics

def test_hand_worked_median_mad_modified_z():
    for ln in _lines("median_mad_cases.txt"):
        vals, med, mad, zs = [p.strip() for p in ln.split("|")]
        v = np.array(vals.split(), dtype=np.float32)
        m = go.median(v)
        d = go.mad(v, m)
        assert m == F(med), ln
        assert d == F(mad), ln
        for item in zs.split():
            i, z = item.split(":")
            got = 0.6745 * (float(v[int(i)]) - float(m)) / float(d)
            assert got == pytest.approx(float(z), rel=2e-4), ln


def test_thrp_constant():
    # 3.5 / 0.6745 = 5.18902891... ; the cut-off moved to the right-hand side
    assert float(go.thrp(3.5)) == pytest.approx(5.189028910, rel=1e-7)
    assert go.thrp(3.5) == F(3.5 / 0.6745)
    # with this constant a point at exactly 3.5 modified-z units is NOT an exceedance (strict >)
    o = go.Oracle(5, 1, 1, 1, 0, dir=[1], floor_rel=0.0)
    # ranks: 1,2,3,4,x ; med 3, MAD 1 => threshold at 3 + 5.18903
    for x, expect in ((8.18, 0), (8.19, 1)):
        o.reset()
        o.ingest(np.array([[[1], [2], [3], [4], [x]]], np.float32))
        assert o.score()["counts"][4, 0] == expect


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 8, 63, 64, 65, 200, 1001])
def test_median_mad_match_numpy(n):
    rng = np.random.default_rng(n)
    for trial in range(6):
        if trial % 3 == 0:
            v = rng.normal(1.0, 0.03, n).astype(np.float32)
        elif trial % 3 == 1:
            v = rng.integers(-3, 4, n).astype(np.float32)          # many duplicates, zeros
        else:
            v = (rng.standard_cauchy(n) * 1e3).astype(np.float32)   # wide range, both signs
        s = np.sort(v)
        ref = s[(n - 1) // 2] if n % 2 else F(0.5) * (s[n // 2 - 1] + s[n // 2])
        m = go.median(v)
        assert m == ref
        assert m == np.median(v)            # library median of float32 input
        dev = np.abs(v - m)
        sd = np.sort(dev)
        refd = sd[(n - 1) // 2] if n % 2 else F(0.5) * (sd[n // 2 - 1] + sd[n // 2])
        assert go.mad(v, m) == refd


def test_signed_zero_order():
    # total order: -0 sorts before +0, so the lower middle of {-0, +0} is -0
    v = np.array([0.0, -0.0, -0.0], np.float32)
    m = go.median(v)
    assert m == 0 and np.signbit(m)
    v = np.array([0.0, -0.0, 0.0], np.float32)
    m = go.median(v)
    assert m == 0 and not np.signbit(m)


def test_gaussian_closed_form_of_the_constant():
    # For N(mu, sigma) the MAD tends to Phi^-1(3/4) * sigma = 0.67449 sigma, which is why
    # 0.6745 * (x - median) / MAD reads in units of sigma.
    rng = np.random.default_rng(7)
    sigma = 0.03
    v = rng.normal(1.0, sigma, 16384).astype(np.float32)
    m = go.median(v)
    d = go.mad(v, m)
    assert abs(float(d) / sigma - 0.6745) < 0.02
    assert abs(float(m) - 1.0) < 4 * 1.2533 * sigma / math.sqrt(16384)


def test_scale_floors():
    assert go.scale(0.5, 10.0, 1e-4, 0.0) == F(0.5)
    assert go.scale(0.0, 10.0, 1e-4, 0.0) == F(1e-4) * F(10.0)
    assert go.scale(0.0, -10.0, 1e-4, 0.0) == F(1e-4) * F(10.0)
    assert go.scale(0.0, 10.0, 1e-4, 7.5) == F(7.5)
    assert go.scale(0.0, 0.0, 1e-4, 0.0) == 0


# ------------------------------------------------------------------ brute force, tiny fleets

def _tiny_params(M, rng):
    d = [int(x) for x in rng.choice([-1, 1], M)]
    d[0] = 1
    thr = [float(x) for x in rng.choice([1.0, 2.0, 3.5], M)]
    frel = [float(x) for x in rng.choice([0.0, 1e-4, 1e-2], M)]
    fab = [float(x) for x in rng.choice([0.0, 0.0, 0.05], M)]
    return d, thr, frel, fab


@pytest.mark.parametrize("seed", range(12))
def test_online_matches_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    R = int(rng.integers(2, 9))
    M = int(rng.integers(1, 5))
    W = int(rng.integers(1, 7))
    k = int(rng.integers(1, W + 1))
    K = int(rng.integers(0, R + 1))
    T = int(rng.integers(1, 15))
    d, thr, frel, fab = _tiny_params(M, rng)
    ms = int(rng.integers(1, 4))
    nc = int(rng.integers(1, 3))
    prim = int(rng.integers(0, M))
    kw = dict(primary=prim, min_signals=ms, n_consec=nc, tier_moderate=0.10, tier_severe=0.20)
    o = go.Oracle(R, M, W, k, K, dir=d, thr=thr, floor_rel=frel, floor_abs=fab, **kw)
    b = brute.Brute(R, M, W, k, K, d, thr, frel, fab, **kw)
    # quantised values give ties, duplicates and zero MADs; a slow rank gives flags
    X = np.round(rng.normal(1.0, 0.05, (T, R, M)) * 40) / 40
    X[:, 0, :] *= np.where(np.array(d) > 0, 1.5, 0.6)
    X = X.astype(np.float32)
    t = 0
    while t < T:
        nb = int(rng.integers(1, 4))
        blk = X[t:t + nb]
        so = o.ingest(blk)
        bm, bd = b.ingest(blk)
        assert np.array_equal(so["step_med"], bm)
        assert np.array_equal(so["step_mad"], bd)
        t += blk.shape[0]
        ro, rb = o.score(), b.score()
        for key in ("wmed", "fleet_med", "fleet_mad", "counts", "mask", "flags", "tier", "topk_idx"):
            assert np.array_equal(ro[key], rb[key]), (key, seed, t)
        # reported scores: 0.6745 * dir * (wmed - B) / scale in float64
        for r in range(R):
            for m in range(M):
                sc = brute.scale(ro["fleet_mad"][m], ro["fleet_med"][m], F(frel[m]), F(fab[m]))
                dev = d[m] * (float(ro["wmed"][r, m]) - float(ro["fleet_med"][m]))
                want = 0.0 if dev == 0 else (math.copysign(math.inf, dev) if sc == 0 else 0.6745 * dev / float(sc))
                assert ro["scores"][r, m] == pytest.approx(want, rel=1e-12)
        for i, r in enumerate(ro["topk_idx"]):
            assert ro["topk_score"][i] == ro["scores"][r, prim]


def test_k_of_w_counts_exhaustive_patterns():
    # rank 0 is far out in exactly the steps where the pattern has a 1; its count after
    # every step must be the number of ones among the last W steps (plain recount).
    W, T = 4, 7
    base = np.array([1.0, 0.99, 1.01, 1.02, 0.98], np.float32)
    for pattern in itertools.product([0, 1], repeat=T):
        o = go.Oracle(5, 1, W, 2, 0, dir=[1], min_signals=1)
        for t, bit in enumerate(pattern):
            row = base.copy()
            row[0] = 10.0 if bit else 1.0
            o.ingest(row.reshape(1, 5, 1))
            res = o.score()
            lo = max(0, t + 1 - W)
            assert res["counts"][0, 0] == sum(pattern[lo:t + 1])
            assert not res["counts"][1:, 0].any()


# ------------------------------------------------------------------ invariants (Section 4.2)

def _fleet(R=64, T=120, M=4, seed=0, sigma=0.02):
    rng = np.random.default_rng(seed)
    s = np.exp(sigma * rng.normal(size=(T, R)))
    X = np.empty((T, R, M))
    X[..., 0] = s
    X[..., 1] = 0.7 * s * np.exp(0.5 * sigma * rng.normal(size=(T, R)))
    X[..., 2] = 0.3 * s * np.exp(0.5 * sigma * rng.normal(size=(T, R)))
    X[..., 3] = 4096.0 / s
    return X[..., :M]


DIR4 = [1, 1, 1, -1]


def _run(X, W=50, k=30, K=8, block=50, **kw):
    T, R, M = X.shape
    o = go.Oracle(R, M, W, k, K, dir=DIR4[:M], **kw)
    outs = []
    for t in range(0, T, block):
        o.ingest(X[t:t + block].astype(np.float32))
        outs.append(o.score())
    return outs


def _slow(X, r, f):
    X = X.copy()
    X[:, r, 0] *= f
    X[:, r, 1] *= f
    X[:, r, 2] *= f
    X[:, r, 3] /= f
    return X


def test_constant_fleet_never_flags():
    X = np.full((60, 16, 4), 1.25)
    for res in _run(X):
        assert not res["flags"].any() and not res["mask"].any() and not res["tier"].any()
        assert not res["counts"].any()
        assert np.all(res["scores"] == 0)


def test_rank_permutation_invariance():
    X = _slow(_fleet(seed=3), 5, 1.2)
    perm = np.random.default_rng(1).permutation(X.shape[1])
    a = _run(X)
    b = _run(X[:, perm])
    inv = np.argsort(perm)   # rank r of X sits at position inv[r] of the permuted fleet
    for ra, rb in zip(a, b):
        for key in ("wmed", "counts", "mask", "flags", "tier", "scores"):
            assert np.array_equal(ra[key], rb[key][inv]), key
        for key in ("fleet_med", "fleet_mad"):
            assert np.array_equal(ra[key], rb[key])
        # distinct keys here, so the top-k list maps through the permutation
        assert np.array_equal(inv[ra["topk_idx"]], rb["topk_idx"])


def test_power_of_two_scaling_invariance():
    X = _slow(_fleet(seed=4), 9, 1.2).astype(np.float32)
    a = _run(X)
    b = _run(X * np.float32(2.0 ** 7))
    for ra, rb in zip(a, b):
        for key in ("counts", "mask", "flags", "tier", "topk_idx"):
            assert np.array_equal(ra[key], rb[key]), key
        assert np.array_equal(ra["scores"], rb["scores"])            # bit-identical
        assert np.array_equal(ra["wmed"] * np.float32(128), rb["wmed"])


def test_persistent_straggler_flagged_isolated_spike_not():
    X = _fleet(seed=5)
    X = _slow(X, 7, 1.2)
    for t in (10, 70):                       # isolated 3x spikes on otherwise healthy ranks
        X[t, 20, :3] *= 3.0
        X[t, 20, 3] /= 3.0
    outs = _run(X)
    for res in outs:
        assert res["flags"][7] == 1
        assert res["tier"][7] == 3 or res["tier"][7] == 2      # 1.2x sits at the 20 % boundary
        assert res["flags"][20] == 0
        assert res["flags"].sum() == 1
        assert res["topk_idx"][0] == 7
    # the spike is an exceedance of its own step (count 1) but moves no windowed median
    assert outs[0]["counts"][20, 0] == 1


def test_fleet_wide_shift_changes_no_exceedance():
    X = _slow(_fleet(seed=6, T=50), 3, 1.2).astype(np.float32)
    Y = X.copy()
    Y[17] *= np.float32(2.0)                 # the whole fleet is twice as slow in one step
    a = _run(X)[0]
    b = _run(Y)[0]
    assert np.array_equal(a["counts"], b["counts"])


def test_window_median_is_immune_to_one_spike():
    rng = np.random.default_rng(8)
    X = _fleet(seed=8, T=50).astype(np.float32)
    a = _run(X)[0]["wmed"]
    Y = X.copy()
    Y[23, 11, 0] *= np.float32(50.0)
    b = _run(Y)[0]["wmed"]
    col = np.sort(X[:, 11, 0])
    n = len(col)
    assert col[n // 2 - 2] <= b[11, 0] <= col[n // 2 + 1]
    other = np.ones(a.shape, bool)
    other[11, 0] = False
    assert np.array_equal(a[other], b[other])


@pytest.mark.parametrize("factor,flag,tier", [(1.03, 0, 0), (1.09, 1, 1), (1.15, 1, 2), (1.25, 1, 3)])
def test_response_tiers(factor, flag, tier):
    # sigma = 0.02: 1.09x is a clear per-step outlier but below the ~10 % tier, 1.15x is
    # the moderate tier, 1.25x the severe one, 1.03x is inside the noise.
    X = _slow(_fleet(R=256, T=50, seed=9), 100, factor)
    res = _run(X)[0]
    assert res["flags"][100] == flag
    assert res["tier"][100] == tier


def test_step_time_is_primary_and_multiple_signals_needed():
    X = _fleet(R=64, T=50, seed=10)
    only_support = X.copy()
    only_support[:, 4, 1] *= 1.3                 # compute phase alone, step time normal
    only_support[:, 4, 2] *= 1.3
    res = _run(only_support)[0]
    assert res["mask"][4] == 0b0110 and res["flags"][4] == 0 and res["tier"][4] == 1
    only_primary = X.copy()
    only_primary[:, 4, 0] *= 1.3                 # step time alone: one signal is not enough
    res = _run(only_primary)[0]
    assert res["mask"][4] == 0b0001 and res["flags"][4] == 0 and res["tier"][4] == 1
    res = _run(only_primary, min_signals=1)[0]
    assert res["flags"][4] == 1 and res["tier"][4] == 3


def test_consecutive_evaluations():
    X = _fleet(R=64, T=150, seed=11)
    X[50:, 9] = _slow(X, 9, 1.3)[50:, 9]         # slow from the second window on
    outs = _run(X, n_consec=2)
    assert [int(o["flags"][9]) for o in outs] == [0, 0, 1]
    outs = _run(X, n_consec=1)
    assert [int(o["flags"][9]) for o in outs] == [0, 1, 1]
    # an interruption restarts the run: slow, healthy, slow never gives two in a row
    Y = _fleet(R=64, T=200, seed=11)
    Y[:50, 9] = _slow(Y, 9, 1.3)[:50, 9]
    Y[100:150, 9] = _slow(Y, 9, 1.3)[100:150, 9]
    assert [int(o["flags"][9]) for o in _run(Y, n_consec=2)] == [0, 0, 0, 0]
    assert [int(o["flags"][9]) for o in _run(Y, n_consec=1)] == [1, 0, 1, 0]


def test_nonfinite_rejected():
    o = go.Oracle(4, 1, 2, 1, 0, dir=[1])
    bad = np.ones((1, 4, 1), np.float32)
    bad[0, 2, 0] = np.nan
    with pytest.raises(ValueError):
        o.ingest(bad)
    bad[0, 2, 0] = np.inf
    with pytest.raises(ValueError):
        o.ingest(bad)


# ------------------------------------------------------------------ node sweep (Sections 5.2-5.4)

def test_percentile_index_fixture():
    for ln in _lines("percentile_index_cases.txt"):
        ppm, G, j = (int(x) for x in ln.split())
        # distinct ascending values: the cut for a "smaller is worse" metric is the j-th smallest
        S = np.arange(1, G + 1, dtype=np.float32).reshape(G, 1, 1)
        res = go.sweep(S, G, 1, dir=[-1], pct_ppm=ppm)
        assert res["fleet_cut"][0] == F(j), ln
        res = go.sweep(S, G, 1, dir=[1], pct_ppm=ppm)
        assert res["fleet_cut"][0] == F(G - j + 1), ln


@pytest.mark.parametrize("seed", range(6))
def test_sweep_matches_brute_force(seed):
    rng = np.random.default_rng(200 + seed)
    nodes, gpn = int(rng.integers(1, 5)), int(rng.integers(1, 5))
    N, M = int(rng.integers(1, 8)), int(rng.integers(1, 5))
    G = nodes * gpn
    d = [int(x) for x in rng.choice([-1, 1], M)]
    thr = [float(x) for x in rng.choice([0.5, 1.0, 3.5], M)]
    frel = [float(x) for x in rng.choice([0.0, 1e-4], M)]
    fab = [float(x) for x in rng.choice([0.0, 0.02], M)]
    ppm = int(rng.choice([50_000, 250_000, 500_000]))
    S = np.round(rng.normal(1.0, 0.05, (G, N, M)) * 50) / 50
    S[0] *= 0.5
    S = S.astype(np.float32)
    a = go.sweep(S, nodes, gpn, dir=d, thr=thr, floor_rel=frel, floor_abs=fab, pct_ppm=ppm)
    b = brute.sweep(S, nodes, gpn, d, thr, frel, fab, ppm)
    for key in b:
        assert np.array_equal(a[key], b[key]), key


def test_sweep_degraded_gpu_fails_its_node_only():
    rng = np.random.default_rng(12)
    nodes, gpn, N, M = 32, 8, 20, 3
    S = (1.0 + 0.01 * rng.normal(size=(nodes * gpn, 1, M))) * np.exp(0.003 * rng.normal(size=(nodes * gpn, N, M)))
    S[8 * 5 + 3, :, 1] *= 0.8                     # one GPU of node 5 loses 20 % on one metric
    res = go.sweep(S.astype(np.float32), nodes, gpn, dir=[-1, -1, -1])
    assert res["fail_mask"][8 * 5 + 3] == 0b010
    assert res["gpu_pass"].sum() == nodes * gpn - 1
    assert list(np.nonzero(res["node_pass"] == 0)[0]) == [5]
    # quantised metric with zero MAD: the percentile tail keeps the modal GPUs passing
    clk = np.full((nodes * gpn, N, 1), 1965.0)
    clk[7] = 1800.0
    res = go.sweep(clk.astype(np.float32), nodes, gpn, dir=[-1], floor_abs=7.5)
    assert res["gpu_pass"].sum() == nodes * gpn - 1 and res["gpu_pass"][7] == 0


# ------------------------------------------------------------------ node-level verdicts (Section 4.2 / 7.1)

@pytest.mark.parametrize("seed", range(8))
def test_node_verdict_matches_brute_force(seed):
    rng = np.random.default_rng(500 + seed)
    rpn = int(rng.integers(1, 5))
    nodes = int(rng.integers(1, 5))
    R, M = rpn * nodes, int(rng.integers(1, 4))
    W = int(rng.integers(1, 7))
    k = int(rng.integers(1, W + 1))
    T = int(rng.integers(1, 14))
    d, thr, frel, fab = _tiny_params(M, rng)
    prim = int(rng.integers(0, M))
    kw = dict(primary=prim, min_signals=1, n_consec=1)
    o = go.Oracle(R, M, W, k, 0, dir=d, thr=thr, floor_rel=frel, floor_abs=fab, **kw)
    b = brute.Brute(R, M, W, k, 0, d, thr, frel, fab, **kw)
    X = np.round(rng.normal(1.0, 0.05, (T, R, M)) * 40) / 40
    X[:, 0, :] *= np.where(np.array(d) > 0, 1.5, 0.6)           # one slow rank: its node must be flagged
    stall = rng.random((T, nodes)) < 0.3                         # whole-node stalls on the primary metric
    for t in range(T):
        for nd in np.nonzero(stall[t])[0][: max(1, nodes // 2)]:
            X[t, nd * rpn:(nd + 1) * rpn, prim] *= 3.0 if d[prim] > 0 else 0.3
    X = X.astype(np.float32)
    for t in range(T):
        o.ingest(X[t:t + 1])
        b.ingest(X[t:t + 1])
        ro, rb = o.score(), b.score()
        assert np.array_equal(ro["flags"], rb["flags"])
        no, nb = o.node_verdict(rpn), brute.node_verdict(b, rpn)
        for key in ("node_flag", "node_tier", "node_stall"):
            assert np.array_equal(no[key], nb[key]), (key, seed, t)


def test_node_verdict_flags_the_node_of_a_slow_rank_and_counts_whole_node_stalls():
    X = _slow(_fleet(R=64, T=50, seed=21), 19, 1.3)              # rank 19 lives on node 2 (8 ranks per node)
    stalled = [3, 17, 40]
    for t in stalled:
        X[t, 40:48, :] *= np.array([2.0, 2.0, 2.0, 0.5], np.float32)   # node 5 stalls as a whole
    X[10, 8:15, 0] *= 2.0                                        # seven of node 1's eight ranks: not a whole-node stall
    o = go.Oracle(64, 4, 50, 30, 8, dir=DIR4)
    o.ingest(X)
    res = o.score()
    nv = o.node_verdict(8)
    assert nv["node_flag"].tolist() == [0, 0, 1, 0, 0, 0, 0, 0]
    assert nv["node_tier"][2] == res["tier"][19] == 3
    assert nv["node_stall"].tolist() == [0, 0, 0, 0, 0, len(stalled), 0, 0]
    # a stall is transient: node 5 is not flagged by three steps out of fifty
    assert nv["node_flag"][5] == 0
    # permuting the ranks inside every node changes no node verdict
    rng = np.random.default_rng(3)
    perm = np.concatenate([nd * 8 + rng.permutation(8) for nd in range(8)])
    o2 = go.Oracle(64, 4, 50, 30, 8, dir=DIR4)
    o2.ingest(X[:, perm])
    o2.score()
    nv2 = o2.node_verdict(8)
    for key in nv:
        assert np.array_equal(nv[key], nv2[key]), key
    # one rank per node: the fold is the identity
    o.ingest(X[:1])
    with pytest.raises(RuntimeError):
        o.node_verdict(8)                                        # an ingest since the evaluation: no verdict
    res = o.score()
    nv1 = o.node_verdict(1)
    assert np.array_equal(nv1["node_flag"], res["flags"]) and np.array_equal(nv1["node_tier"], res["tier"])
    with pytest.raises(ValueError):
        o.node_verdict(7)


# ------------------------------------------------------------------ triage repeat-offender rule (Section 6)

def test_triage_rule_three_entries_within_a_week():
    day = 86400
    # the paper's numbers: the third entry inside one week terminates
    assert go.triage([0, 2 * day, 5 * day]).tolist() == [0, 0, 1]
    assert go.triage([0, 2 * day, 7 * day]).tolist() == [0, 0, 1]            # exactly a week apart still counts
    assert go.triage([0, 2 * day, 7 * day + 1]).tolist() == [0, 0, 0]        # the first entry has aged out
    assert go.triage([0, 6 * day, 8 * day, 12 * day]).tolist() == [0, 0, 0, 1]   # a sliding week, not calendar weeks
    assert go.triage([5, 5, 5]).tolist() == [0, 0, 1]
    assert go.triage([]).tolist() == []
    assert go.triage([0, 1], limit=1).tolist() == [1, 1]
    with pytest.raises(ValueError):
        go.triage([10, 5])                                                   # times must not run backwards
    rng = np.random.default_rng(9)
    for _ in range(50):
        n = int(rng.integers(0, 12))
        times = np.sort(rng.integers(0, 20 * day, n)).tolist()
        period = int(rng.integers(0, 10 * day))
        limit = int(rng.integers(1, 5))
        assert go.triage(times, period, limit).tolist() == brute.triage(times, period, limit)
