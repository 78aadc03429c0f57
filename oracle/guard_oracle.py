"""ctypes wrapper around oracle/guard_oracle.c -- TEST INFRASTRUCTURE, not the product.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this.
It shares nothing with the CUDA library: it compiles its own C file with gcc and talks
to it through numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "guard_oracle.c")
_LIB = os.path.join(_HERE, "libguard_oracle.so")
_CFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c11", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", *_CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        fp, u8p, i8p = C.POINTER(C.c_float), C.POINTER(C.c_ubyte), C.POINTER(C.c_byte)
        L.oracle_median.restype = C.c_float
        L.oracle_median.argtypes = [fp, C.c_long]
        L.oracle_mad.restype = C.c_float
        L.oracle_mad.argtypes = [fp, C.c_long, C.c_float]
        L.oracle_scale.restype = C.c_float
        L.oracle_scale.argtypes = [C.c_float] * 4
        L.oracle_thrp.restype = C.c_float
        L.oracle_thrp.argtypes = [C.c_float]
        L.oracle_create.restype = C.c_void_p
        L.oracle_create.argtypes = [C.c_int] * 8 + [C.c_float, C.c_float, i8p, fp, fp, fp]
        L.oracle_destroy.argtypes = [C.c_void_p]
        L.oracle_reset.argtypes = [C.c_void_p]
        L.oracle_ingest.restype = C.c_int
        L.oracle_ingest.argtypes = [C.c_void_p, fp, C.c_int, fp, fp]
        L.oracle_score.restype = C.c_int
        L.oracle_score.argtypes = [C.c_void_p, fp, fp, fp, C.POINTER(C.c_double), C.POINTER(C.c_uint16),
                                   C.POINTER(C.c_uint32), u8p, u8p, C.POINTER(C.c_int32), C.POINTER(C.c_double)]
        L.oracle_node_verdict.restype = C.c_int
        L.oracle_node_verdict.argtypes = [C.c_void_p, C.c_int, u8p, u8p, C.POINTER(C.c_uint16)]
        L.oracle_triage.restype = C.c_int
        L.oracle_triage.argtypes = [C.POINTER(C.c_int64), C.c_int, C.c_int64, C.c_int, u8p]
        L.oracle_sweep.restype = C.c_int
        L.oracle_sweep.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_int, i8p, fp, fp, fp, C.c_int,
                                   fp, fp, fp, fp, C.POINTER(C.c_uint32), u8p, u8p]
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def _f32(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.float32))


def median(v) -> np.float32:
    v = _f32(v).ravel()
    return np.float32(lib().oracle_median(_p(v, C.c_float), v.size))


def mad(v, med) -> np.float32:
    v = _f32(v).ravel()
    return np.float32(lib().oracle_mad(_p(v, C.c_float), v.size, C.c_float(float(med))))


def scale(mad_, med, floor_rel, floor_abs) -> np.float32:
    return np.float32(lib().oracle_scale(float(mad_), float(med), float(floor_rel), float(floor_abs)))


def thrp(thr) -> np.float32:
    return np.float32(lib().oracle_thrp(float(thr)))


class Oracle:
    """Stateful online scorer: ingest blocks of steps, then score the current window."""

    def __init__(self, ranks: int, metrics: int, W: int, k: int, topk: int = 0, *, dir: Sequence[int],
                 thr: Sequence[float] | float = 3.5, floor_rel: Sequence[float] | float = 1e-4,
                 floor_abs: Sequence[float] | float = 0.0, primary: int = 0, min_signals: int = 2,
                 n_consec: int = 1, tier_moderate: float = 0.10, tier_severe: float = 0.20):
        self.R, self.M, self.W, self.k, self.topk = ranks, metrics, W, k, topk
        bc = lambda v: _f32(np.broadcast_to(np.asarray(v, dtype=np.float32), (metrics,)))
        self._dir = np.ascontiguousarray(np.asarray(dir, dtype=np.int8))
        assert self._dir.size == metrics
        self._thr, self._frel, self._fabs = bc(thr), bc(floor_rel), bc(floor_abs)
        self._h = lib().oracle_create(ranks, metrics, W, k, topk, primary, min_signals, n_consec,
                                      C.c_float(tier_moderate), C.c_float(tier_severe),
                                      _p(self._dir, C.c_byte), _p(self._thr, C.c_float),
                                      _p(self._frel, C.c_float), _p(self._fabs, C.c_float))
        if not self._h:
            raise ValueError("oracle_create rejected the arguments")

    def __del__(self):
        h = getattr(self, "_h", None)
        if h:
            lib().oracle_destroy(h)
            self._h = None

    def reset(self):
        lib().oracle_reset(self._h)

    def ingest(self, block) -> Dict[str, np.ndarray]:
        """block [B, R, M] float32 -> per-step cross-rank median and MAD, each [B, M]."""
        block = _f32(block)
        assert block.ndim == 3 and block.shape[1:] == (self.R, self.M), block.shape
        B = block.shape[0]
        med = np.empty((B, self.M), np.float32)
        mad_ = np.empty((B, self.M), np.float32)
        rc = lib().oracle_ingest(self._h, _p(block, C.c_float), B, _p(med, C.c_float), _p(mad_, C.c_float))
        if rc != 0:
            raise ValueError("oracle_ingest: non-finite input")
        return {"step_med": med, "step_mad": mad_}

    def score(self) -> Dict[str, np.ndarray]:
        R, M, K = self.R, self.M, self.topk
        out = {
            "wmed": np.empty((R, M), np.float32), "fleet_med": np.empty(M, np.float32),
            "fleet_mad": np.empty(M, np.float32), "scores": np.empty((R, M), np.float64),
            "counts": np.empty((R, M), np.uint16), "mask": np.empty(R, np.uint32),
            "flags": np.empty(R, np.uint8), "tier": np.empty(R, np.uint8),
            "topk_idx": np.empty(K, np.int32), "topk_score": np.empty(K, np.float64),
        }
        rc = lib().oracle_score(self._h, _p(out["wmed"], C.c_float), _p(out["fleet_med"], C.c_float),
                                _p(out["fleet_mad"], C.c_float), _p(out["scores"], C.c_double),
                                _p(out["counts"], C.c_uint16), _p(out["mask"], C.c_uint32),
                                _p(out["flags"], C.c_ubyte), _p(out["tier"], C.c_ubyte),
                                _p(out["topk_idx"], C.c_int32), _p(out["topk_score"], C.c_double))
        if rc != 0:
            raise RuntimeError("oracle_score: nothing ingested yet")
        return out

    def node_verdict(self, ranks_per_node: int = 8) -> Dict[str, np.ndarray]:
        """Node-level fold of the last evaluation (call right after score())."""
        if ranks_per_node < 1 or self.R % ranks_per_node:
            raise ValueError("ranks must be a multiple of ranks_per_node")
        N = self.R // ranks_per_node
        out = {"node_flag": np.empty(N, np.uint8), "node_tier": np.empty(N, np.uint8),
               "node_stall": np.empty(N, np.uint16)}
        rc = lib().oracle_node_verdict(self._h, ranks_per_node, _p(out["node_flag"], C.c_ubyte),
                                       _p(out["node_tier"], C.c_ubyte), _p(out["node_stall"], C.c_uint16))
        if rc != 0:
            raise RuntimeError("oracle_node_verdict: no evaluation of the current window (rc %d)" % rc)
        return out


def triage(times, period: int = 7 * 86400, limit: int = 3) -> np.ndarray:
    """Entry times (seconds, non-decreasing) of one node -> per entry 1 where the node is to be terminated."""
    t = np.ascontiguousarray(np.asarray(times, dtype=np.int64))
    out = np.zeros(t.size, np.uint8)
    rc = lib().oracle_triage(_p(t, C.c_int64), t.size, period, limit, _p(out, C.c_ubyte))
    if rc != 0:
        raise ValueError("oracle_triage rejected the input")
    return out


def sweep(S, nodes: int, gpus_per_node: int, *, dir: Sequence[int], thr=3.5, floor_rel=1e-4, floor_abs=0.0,
          pct_ppm: int = 50_000) -> Dict[str, np.ndarray]:
    """S [G, reps, M] float32 -> per-GPU medians, fleet statistics, fail masks, verdicts."""
    S = _f32(S)
    G = nodes * gpus_per_node
    assert S.ndim == 3 and S.shape[0] == G, S.shape
    reps, M = S.shape[1], S.shape[2]
    bc = lambda v: _f32(np.broadcast_to(np.asarray(v, dtype=np.float32), (M,)))
    d = np.ascontiguousarray(np.asarray(dir, dtype=np.int8))
    thr_, frel, fabs_ = bc(thr), bc(floor_rel), bc(floor_abs)
    out = {
        "gpu_med": np.empty((G, M), np.float32), "fleet_med": np.empty(M, np.float32),
        "fleet_mad": np.empty(M, np.float32), "fleet_cut": np.empty(M, np.float32),
        "fail_mask": np.empty(G, np.uint32), "gpu_pass": np.empty(G, np.uint8),
        "node_pass": np.empty(nodes, np.uint8),
    }
    rc = lib().oracle_sweep(_p(S, C.c_float), nodes, gpus_per_node, reps, M, _p(d, C.c_byte), _p(thr_, C.c_float),
                            _p(frel, C.c_float), _p(fabs_, C.c_float), pct_ppm, _p(out["gpu_med"], C.c_float),
                            _p(out["fleet_med"], C.c_float), _p(out["fleet_mad"], C.c_float),
                            _p(out["fleet_cut"], C.c_float), _p(out["fail_mask"], C.c_uint32),
                            _p(out["gpu_pass"], C.c_ubyte), _p(out["node_pass"], C.c_ubyte))
    if rc != 0:
        raise ValueError("oracle_sweep rejected the input")
    return out
