"""Host-side checks that need no GPU: the library loads, exports every symbol the header
declares, sizes workspaces, rejects bad arguments before touching CUDA, and its key map
is order preserving."""
import ctypes as C
import math
import os
import re
import struct

import numpy as np
import pytest

from paper_2605_17879_b200 import build as gbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def glib():
    gbuild.build_library()
    from paper_2605_17879_b200 import guard
    return guard


def test_exports_every_declared_symbol(glib):
    hdr = open(os.path.join(ROOT, "include", "guard_b200.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(guard_[a-z_0-9]+)\s*\(", hdr))
    assert {"guard_create", "guard_ingest", "guard_score", "guard_sweep_qualify"} <= names
    lib = C.CDLL(glib.LIB_PATH)
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_workspace_bytes(glib):
    R, M, W, Cap, K = 1024, 8, 100, 200, 16
    n = glib.workspace_bytes(R, M, W, Cap, K)
    assert n >= Cap * R * M * 4 + Cap * R           # ring + byte-wide exceedance ring
    assert n < Cap * R * M * 4 * 1.2 + (1 << 20)
    assert n % 256 == 0
    assert glib.workspace_bytes(R, 9, W, Cap, K) >= Cap * R * 9 * 4 + Cap * R * 4   # 32-bit masks above 8 metrics
    for bad in [(0, M, W, Cap, K), (R, 0, W, Cap, K), (R, 33, W, Cap, K), (R, M, 0, Cap, K),
                (R, M, W, W - 1, K), (R, M, W, Cap, R + 1), (R, M, 65536, 65536, K), (4096, M, W, Cap, 1025)]:
        assert glib.workspace_bytes(*bad) == 0, bad
    L = glib.lib()
    assert L.guard_sweep_workspace_bytes(16384, 200, 6) >= 16384 * 6 * 4
    assert L.guard_sweep_workspace_bytes(0, 200, 6) == 0
    assert L.guard_sweep_workspace_bytes(8, 200, 33) == 0


def test_create_rejects_bad_arguments_on_the_host(glib):
    L = glib.lib()
    P = glib._Params(4, [1, 1, 1, -1], 3.5, 1e-4, 0.0)
    h = C.c_void_p()
    fake_ws = 256 * 1000       # never dereferenced: every call below fails before any CUDA work
    def create(R=8, M=4, W=4, k=2, cap=4, K=2, ws=fake_ws, nbytes=1 << 30, p=P):
        return L.guard_create(C.byref(h), R, M, W, k, C.byref(p.struct) if p else None, cap, K, ws, nbytes, None)
    assert create(R=0) == -1 and b"sizes" in L.guard_last_error(None)
    assert create(k=0) == -1 and create(k=5) == -1
    assert create(cap=3) == -1
    assert create(K=9) == -1
    assert create(p=None) == -1
    assert create(ws=None) == -2
    assert create(ws=fake_ws + 8) == -2          # misaligned
    assert create(nbytes=1024) == -2 and b"at least" in L.guard_last_error(None)
    bad = glib._Params(4, [1, 1, 0, -1], 3.5, 1e-4, 0.0)
    assert create(p=bad) == -1 and b"dir" in L.guard_last_error(None)
    bad = glib._Params(4, [1, 1, 1, -1], 3.5, 1e-4, 0.0, primary=4)
    assert create(p=bad) == -1
    bad = glib._Params(4, [1, 1, 1, -1], float("nan"), 1e-4, 0.0)
    assert create(p=bad) == -1
    bad = glib._Params(4, [1, 1, 1, -1], 3.5, 1e-4, 0.0, n_consec=0)
    assert create(p=bad) == -1
    assert h.value is None
    # NULL context is tolerated everywhere
    assert L.guard_ingest(None, None, 1, None, None, None) == -1
    assert L.guard_sync_status(None, None) == -1
    assert L.guard_set_deferred(None, 1) == -1
    assert L.guard_join(None, None) == -1
    L.guard_destroy(None)
    assert L.guard_steps_seen(None) == 0


def test_key_map_is_order_preserving_and_invertible(glib):
    rng = np.random.default_rng(0)
    bits = rng.integers(0, 1 << 32, 1 << 20, dtype=np.uint64).astype(np.uint32)
    vals = bits.view(np.float32)
    vals = vals[np.isfinite(vals)]
    edge = np.array([0.0, -0.0, np.finfo(np.float32).tiny, -np.finfo(np.float32).tiny, np.finfo(np.float32).max,
                     -np.finfo(np.float32).max, 1e-45, -1e-45, 1.0, -1.0, np.nextafter(np.float32(1), np.float32(2))],
                    np.float32)
    vals = np.concatenate([vals, edge])
    # the key map restated with numpy: flip all bits of negatives, the sign bit of the rest
    b = vals.view(np.uint32)
    keys = np.where(b >> 31 == 1, ~b, b | np.uint32(0x80000000)).astype(np.uint32)
    sample = rng.choice(len(vals), 2000, replace=False)
    for i in list(sample) + list(range(len(vals) - len(edge), len(vals))):
        k = glib.key_from_float(float(vals[i]))
        assert k == int(keys[i])
        back = glib.float_from_key(k)
        assert struct.pack("f", back) == struct.pack("f", float(vals[i]))
    order = np.argsort(keys, kind="stable")
    sv = vals[order]
    assert np.all(sv[:-1] <= sv[1:])                       # numeric order
    z = np.nonzero(sv == 0)[0]
    sb = np.signbit(sv[z])
    assert np.all(sb[:-1] >= sb[1:])                       # -0 before +0
    assert glib.key_from_float(-0.0) + 1 == glib.key_from_float(0.0)
    assert glib.key_from_float(-math.inf) < glib.key_from_float(-3e38) < glib.key_from_float(3e38) < glib.key_from_float(math.inf)


def test_triage_counter_matches_the_oracle_rule(glib):
    """Section 6's repeat-offender rule through the C ABI (host-only code) against the oracle's
    statement of it, node by node, on interleaved entries."""
    from oracle import guard_oracle as go
    rng = np.random.default_rng(17)
    day = 86400
    for limit, period in ((3, 7 * day), (1, 0), (4, 3 * day), (2, 10)):
        nodes = 6
        t = glib.Triage(nodes, limit, period)
        entries = sorted((int(rng.integers(0, 30 * day)), int(rng.integers(0, nodes))) for _ in range(80))
        entries += [(entries[-1][0], 2)] * 3                     # repeated entries at the same second
        per_node = {n: [] for n in range(nodes)}
        got = {n: [] for n in range(nodes)}
        for ts, n in entries:
            term, within = t.record(n, ts)
            per_node[n].append(ts)
            got[n].append(int(term))
            want_within = sum(1 for u in per_node[n] if ts - u <= period)
            assert within == min(want_within, limit)
        for n in range(nodes):
            assert got[n] == go.triage(per_node[n], period, limit).tolist(), (limit, period, n)
        with pytest.raises(glib.GuardError):
            t.record(nodes, 0)                                   # unknown node
        with pytest.raises(glib.GuardError):
            t.record(2, entries[-1][0] - 1)                      # time runs backwards for node 2
        t.close()
    # the paper's numbers
    t = glib.Triage(4)
    assert [t.record(1, d * day)[0] for d in (0, 2, 5)] == [False, False, True]
    assert [t.record(3, d * day)[0] for d in (0, 2, 8)] == [False, False, False]
    h = C.c_void_p()
    assert glib.lib().guard_triage_create(C.byref(h), 0, 3, 10) == -1
    assert glib.lib().guard_triage_create(C.byref(h), 4, 0, 10) == -1
    assert glib.lib().guard_triage_record(None, 0, 0, None) == -1
    glib.lib().guard_triage_destroy(None)
