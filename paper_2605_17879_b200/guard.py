"""Thin ctypes binding of libguard_b200.so (the C ABI declared in include/guard_b200.h).

Argument marshalling only: every step of the scoring path runs in the library's CUDA
kernels.  PyTorch supplies device memory (the workspace and the output tensors) and the
current CUDA stream.  There is no CPU fallback: if the library has not been built the
import of this module's functions fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libguard_b200.so")

GUARD_OK = 0
ERR_NAMES = {0: "GUARD_OK", -1: "GUARD_ERR_ARG", -2: "GUARD_ERR_WORKSPACE", -3: "GUARD_ERR_NOT_READY",
             -4: "GUARD_ERR_NONFINITE", -5: "GUARD_ERR_TIMEOUT", -6: "GUARD_ERR_CUDA", -7: "GUARD_ERR_INTERNAL"}
MAX_METRICS, MAX_TOPK, MAX_WINDOW = 32, 1024, 65535


class GuardError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__("%s (%d): %s" % (ERR_NAMES.get(code, "?"), code, text))
        self.code = code


class _Thresholds(C.Structure):
    _fields_ = [("primary", C.c_int32), ("min_signals", C.c_int32), ("n_consec", C.c_int32),
                ("ranks_per_node", C.c_int32), ("tier_moderate", C.c_float), ("tier_severe", C.c_float),
                ("dir", C.POINTER(C.c_int8)), ("thr", C.POINTER(C.c_float)),
                ("floor_rel", C.POINTER(C.c_float)), ("floor_abs", C.POINTER(C.c_float))]


_lib = None


def lib():
    """The loaded shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libguard_b200.so is missing: build it with paper_2605_17879_b200.build.build_library() "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, fp = C.c_void_p, C.c_void_p  # device pointers travel as integers
        L.guard_workspace_bytes.restype = C.c_size_t
        L.guard_workspace_bytes.argtypes = [C.c_int] * 5
        L.guard_create.restype = C.c_int
        L.guard_create.argtypes = [C.POINTER(vp), C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(_Thresholds),
                                   C.c_int, C.c_int, vp, C.c_size_t, vp]
        L.guard_ring_reserve.restype = C.c_int
        L.guard_ring_reserve.argtypes = [vp, C.c_int, C.POINTER(vp)]
        L.guard_ingest.restype = C.c_int
        L.guard_ingest.argtypes = [vp, fp, C.c_int, fp, fp, vp]
        L.guard_score.restype = C.c_int
        L.guard_score.argtypes = [vp] + [fp] * 10 + [vp]
        L.guard_sweep_workspace_bytes.restype = C.c_size_t
        L.guard_sweep_workspace_bytes.argtypes = [C.c_int] * 3
        L.guard_sweep_qualify.restype = C.c_int
        L.guard_sweep_qualify.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(_Thresholds), C.c_int32,
                                          vp, C.c_size_t] + [fp] * 8 + [vp]
        L.guard_topk_static.restype = C.c_int
        L.guard_topk_static.argtypes = [fp, fp, fp, C.c_int, C.c_int, C.POINTER(_Thresholds), C.c_int, fp, fp, vp]
        L.guard_node_verdict.restype = C.c_int
        L.guard_node_verdict.argtypes = [vp, fp, fp, fp, vp]
        L.guard_state_bytes.restype = C.c_size_t
        L.guard_state_bytes.argtypes = [vp]
        L.guard_state_export.restype = C.c_int
        L.guard_state_export.argtypes = [vp, vp, C.c_size_t, vp]
        L.guard_state_import.restype = C.c_int
        L.guard_state_import.argtypes = [vp, vp, C.c_size_t, vp]
        L.guard_triage_create.restype = C.c_int
        L.guard_triage_create.argtypes = [C.POINTER(vp), C.c_int, C.c_int, C.c_int64]
        L.guard_triage_record.restype = C.c_int
        L.guard_triage_record.argtypes = [vp, C.c_int, C.c_int64, C.POINTER(C.c_int)]
        L.guard_triage_destroy.restype = None
        L.guard_triage_destroy.argtypes = [vp]
        L.guard_debug_set_wait_limit.restype = C.c_int
        L.guard_debug_set_wait_limit.argtypes = [vp, C.c_longlong]
        L.guard_sync_status.restype = C.c_int
        L.guard_sync_status.argtypes = [vp, vp]
        L.guard_reset.restype = C.c_int
        L.guard_reset.argtypes = [vp, vp]
        L.guard_steps_seen.restype = C.c_int64
        L.guard_steps_seen.argtypes = [vp]
        L.guard_kernel_launches.restype = C.c_int64
        L.guard_kernel_launches.argtypes = [vp]
        L.guard_fallback_steps.restype = C.c_int64
        L.guard_fallback_steps.argtypes = [vp, vp]
        L.guard_fallback_reasons.restype = C.c_int
        L.guard_fallback_reasons.argtypes = [vp, C.POINTER(C.c_uint32), vp]
        L.guard_window_fallbacks.restype = C.c_int
        L.guard_window_fallbacks.argtypes = [vp, C.POINTER(C.c_uint32), vp]
        L.guard_set_overlap.restype = C.c_int
        L.guard_set_overlap.argtypes = [vp, C.c_int]
        L.guard_set_sliding.restype = C.c_int
        L.guard_set_sliding.argtypes = [vp, C.c_int]
        L.guard_sliding_rebuilds.restype = C.c_int64
        L.guard_sliding_rebuilds.argtypes = [vp, vp]
        L.guard_set_row_hints.restype = C.c_int
        L.guard_set_row_hints.argtypes = [vp, C.c_int]
        L.guard_row_hints.restype = C.c_int
        L.guard_row_hints.argtypes = [vp, C.POINTER(C.c_uint32), vp]
        L.guard_set_deferred.restype = C.c_int
        L.guard_set_deferred.argtypes = [vp, C.c_int]
        L.guard_join.restype = C.c_int
        L.guard_join.argtypes = [vp, vp]
        L.guard_profile_enable.restype = C.c_int
        L.guard_profile_enable.argtypes = [vp, C.c_int]
        L.guard_profile_read.restype = C.c_int
        L.guard_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.guard_destroy.restype = None
        L.guard_destroy.argtypes = [vp]
        L.guard_last_error.restype = C.c_char_p
        L.guard_last_error.argtypes = [vp]
        L.guard_key_from_float.restype = C.c_uint32
        L.guard_key_from_float.argtypes = [C.c_float]
        L.guard_float_from_key.restype = C.c_float
        L.guard_float_from_key.argtypes = [C.c_uint32]
        _lib = L
    return _lib


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class _Here:
    """Stands in for torch.cuda.device(...) when the wanted device is already current."""

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        return False


_HERE_CTX = _Here()


def _ptr(t: Optional[torch.Tensor], dtype=None, numel: Optional[int] = None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError("expected dtype %s, got %s" % (dtype, t.dtype))
    if numel is not None and t.numel() < numel:
        raise ValueError("tensor too small: %d < %d elements" % (t.numel(), numel))
    return t.data_ptr()


class _Params:
    """Host-side arrays behind a guard_thresholds struct (kept alive with it)."""

    def __init__(self, metrics, dir, thr, floor_rel, floor_abs, primary=0, min_signals=2, n_consec=1,
                 ranks_per_node=8, tier_moderate=0.10, tier_severe=0.20):
        def bc(v, ctype):
            vals = list(v) if isinstance(v, (list, tuple)) or hasattr(v, "__len__") else [v] * metrics
            if len(vals) != metrics:
                raise ValueError("expected %d per-metric values, got %d" % (metrics, len(vals)))
            return (ctype * metrics)(*vals)
        self.dir = bc([int(d) for d in dir], C.c_int8)
        self.thr = bc(thr, C.c_float)
        self.floor_rel = bc(floor_rel, C.c_float)
        self.floor_abs = bc(floor_abs, C.c_float)
        self.struct = _Thresholds(primary, min_signals, n_consec, ranks_per_node, tier_moderate, tier_severe,
                                  self.dir, self.thr, self.floor_rel, self.floor_abs)


def workspace_bytes(ranks: int, metrics: int, W: int, capacity: int, topk: int) -> int:
    return int(lib().guard_workspace_bytes(ranks, metrics, W, capacity, topk))


_OUT_NAMES = ("wmed", "fleet_med", "fleet_mad", "scores", "counts", "mask", "flags", "tier", "topk_idx", "topk_score")


class Guard:
    """Online scorer: `ingest` blocks of steps, `score` the current window."""

    def __init__(self, ranks: int, metrics: int, W: int, k: int, *, dir: Sequence[int], thr=3.5, floor_rel=1e-4,
                 floor_abs=0.0, primary: int = 0, min_signals: int = 2, n_consec: int = 1, ranks_per_node: int = 8,
                 tier_moderate: float = 0.10, tier_severe: float = 0.20, capacity: Optional[int] = None, topk: int = 0,
                 device="cuda", workspace: Optional[torch.Tensor] = None):
        self.R, self.M, self.W, self.k, self.K = ranks, metrics, W, k, topk
        self.ranks_per_node = ranks_per_node
        self.C = capacity if capacity is not None else W
        self.device = torch.device(device)
        self._devidx = self.device.index if self.device.index is not None else torch.cuda.current_device()
        self._views = {}        # ring views handed out by ring_reserve, by (byte offset, steps)
        self._out_cache = None  # (dict, tensors, marshalled pointers) of the last score() outputs
        self._h = C.c_void_p()
        self._params = _Params(metrics, dir, thr, floor_rel, floor_abs, primary, min_signals, n_consec,
                               ranks_per_node, tier_moderate, tier_severe)
        need = workspace_bytes(ranks, metrics, W, self.C, topk)
        if need == 0:
            raise GuardError(-1, "invalid sizes (ranks=%d metrics=%d W=%d capacity=%d topk=%d)" % (ranks, metrics, W, self.C, topk))
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        self.workspace = workspace
        with self._dev():
            rc = lib().guard_create(C.byref(self._h), ranks, metrics, W, k, C.byref(self._params.struct), self.C, topk,
                                    _ptr(workspace, torch.uint8), workspace.numel(), _stream())
        if rc != GUARD_OK:
            raise GuardError(rc, lib().guard_last_error(None).decode())

    def close(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.guard_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _dev(self):
        """Context that makes the context's device current (nothing to do when it already is)."""
        return _HERE_CTX if torch.cuda.current_device() == self._devidx else torch.cuda.device(self.device)

    def _check(self, rc: int):
        if rc != GUARD_OK:
            raise GuardError(rc, lib().guard_last_error(self._h).decode())

    @property
    def steps_seen(self) -> int:
        return int(lib().guard_steps_seen(self._h))

    @property
    def kernel_launches(self) -> int:
        return int(lib().guard_kernel_launches(self._h))

    def fallback_steps(self) -> int:
        """Rows the fast cross-rank path handed to the direct selection (synchronises)."""
        with self._dev():
            n = int(lib().guard_fallback_steps(self._h, _stream()))
        if n < 0:
            self._check(n)
        return n

    def fallback_reasons(self):
        """Counts of the events that send rows to the direct selection (synchronises)."""
        out = (C.c_uint32 * 6)()
        with self._dev():
            self._check(lib().guard_fallback_reasons(self._h, out, _stream()))
        names = ("cta_list", "step_list", "deferred_list", "median_miss", "select", "mad_miss")
        return dict(zip(names, [int(v) for v in out]))

    def window_fallbacks(self):
        """Series the thread-per-series window kernel handed to its whole-warp fallback (synchronises)."""
        out = (C.c_uint32 * 6)()
        with self._dev():
            self._check(lib().guard_window_fallbacks(self._h, out, _stream()))
        names = ("total", "no_interval", "overflow", "below", "above", "no_convergence")
        return dict(zip(names, [int(v) for v in out]))

    def set_overlap(self, on: bool) -> None:
        """Window medians of an evaluation on an internal stream overlapping the preceding ingest."""
        self._check(lib().guard_set_overlap(self._h, 1 if on else 0))

    def set_sliding(self, on: bool) -> None:
        """Sliding update of the window medians for evaluations a few steps apart (default on)."""
        self._check(lib().guard_set_sliding(self._h, 1 if on else 0))

    def sliding_rebuilds(self) -> int:
        """Series the sliding evaluations rebuilt from their whole window (synchronises)."""
        with self._dev():
            n = int(lib().guard_sliding_rebuilds(self._h, _stream()))
        if n < 0:
            self._check(n)
        return n

    def set_row_hints(self, on: bool) -> None:
        """Single rows of wide fleets bracketed by the call site's previous result (default on)."""
        self._check(lib().guard_set_row_hints(self._h, 1 if on else 0))

    def row_hints(self):
        """Single rows seen and columns settled inside their brackets, per call site (synchronises)."""
        out = (C.c_uint32 * 6)()
        with self._dev():
            self._check(lib().guard_row_hints(self._h, out, _stream()))
        names = ("ingest_rows", "ingest_settled", "baseline_rows", "baseline_settled", "topk_hinted", "topk_full")
        return dict(zip(names, [int(v) for v in out]))

    def set_deferred(self, on: bool) -> None:
        """Deferred evaluations: score() does not make the current stream wait for its results; they
        are complete after the next score(), join(), sync_status() or reset()."""
        self._check(lib().guard_set_deferred(self._h, 1 if on else 0))

    def join(self) -> None:
        """Makes the current stream wait for the pending deferred evaluation, if any."""
        with self._dev():
            self._check(lib().guard_join(self._h, _stream()))

    def profile_enable(self, on=True) -> None:
        """0 / False: off; 1 / True: time the MAD sweep of every ingest; 2: the window kernel of every evaluation."""
        self._check(lib().guard_profile_enable(self._h, int(on)))

    def profile_read(self):
        """(total milliseconds, launches) of the profiled kernel since the last read."""
        ms, n = C.c_double(), C.c_int64()
        self._check(lib().guard_profile_read(self._h, C.byref(ms), C.byref(n)))
        return ms.value, n.value

    def ring_reserve(self, steps: int) -> torch.Tensor:
        """View [steps, ranks, metrics] of the ring slots the next `steps` steps occupy."""
        p = C.c_void_p()
        self._check(lib().guard_ring_reserve(self._h, steps, C.byref(p)))
        off = p.value - self.workspace.data_ptr()
        view = self._views.get((off, steps))
        if view is None:
            nbytes = steps * self.R * self.M * 4
            view = self.workspace[off:off + nbytes].view(torch.float32).view(steps, self.R, self.M)
            if len(self._views) < 4096:
                self._views[(off, steps)] = view
        return view

    def ingest(self, block: torch.Tensor, step_med: Optional[torch.Tensor] = None,
               step_mad: Optional[torch.Tensor] = None) -> None:
        if block.dim() != 3 or block.shape[1] != self.R or block.shape[2] != self.M:
            raise ValueError("block must be [B, %d, %d]" % (self.R, self.M))
        B = block.shape[0]
        with self._dev():
            self._check(lib().guard_ingest(self._h, _ptr(block, torch.float32), B,
                                           _ptr(step_med, torch.float32, B * self.M),
                                           _ptr(step_mad, torch.float32, B * self.M), _stream()))

    def alloc_outputs(self) -> Dict[str, torch.Tensor]:
        R, M, K, dev = self.R, self.M, self.K, self.device
        return {
            "wmed": torch.empty((R, M), dtype=torch.float32, device=dev),
            "fleet_med": torch.empty(M, dtype=torch.float32, device=dev),
            "fleet_mad": torch.empty(M, dtype=torch.float32, device=dev),
            "scores": torch.empty((R, M), dtype=torch.float32, device=dev),
            "counts": torch.empty((R, M), dtype=torch.uint16, device=dev),
            "mask": torch.empty(R, dtype=torch.uint32, device=dev),
            "flags": torch.empty(R, dtype=torch.uint8, device=dev),
            "tier": torch.empty(R, dtype=torch.uint8, device=dev),
            "topk_idx": torch.empty(K, dtype=torch.int32, device=dev),
            "topk_score": torch.empty(K, dtype=torch.float32, device=dev),
        }

    def score(self, out: Optional[Dict[str, Optional[torch.Tensor]]] = None) -> Dict[str, Optional[torch.Tensor]]:
        """One evaluation; `out` maps output names to tensors (missing / None entries are skipped)."""
        if out is None:
            out = self.alloc_outputs()
        g = out.get
        R, M, K = self.R, self.M, self.K
        # the same output tensors as last time (a monitor scores into the same buffers every step): reuse
        # the checked pointers
        cached = self._out_cache
        if cached is not None and cached[0] is out and all(
                g(n) is t and (t is None or t.data_ptr() == q) for (n, t), q in zip(cached[1], cached[2])):
            ptrs = cached[2]
        else:
            ptrs = (_ptr(g("wmed"), torch.float32, R * M), _ptr(g("fleet_med"), torch.float32, M),
                    _ptr(g("fleet_mad"), torch.float32, M), _ptr(g("scores"), torch.float32, R * M),
                    _ptr(g("counts"), torch.uint16, R * M), _ptr(g("mask"), torch.uint32, R),
                    _ptr(g("flags"), torch.uint8, R), _ptr(g("tier"), torch.uint8, R),
                    _ptr(g("topk_idx"), torch.int32, K) if K else None,
                    _ptr(g("topk_score"), torch.float32, K) if K else None)
            self._out_cache = (out, tuple((n, g(n)) for n in _OUT_NAMES), ptrs)
        with self._dev():
            self._check(lib().guard_score(self._h, *ptrs, _stream()))
        return out

    def node_verdict(self, out: Optional[Dict[str, Optional[torch.Tensor]]] = None) -> Dict[str, Optional[torch.Tensor]]:
        """Node-level fold of the evaluation just made (call right after score())."""
        N = self.R // self.ranks_per_node
        if out is None:
            out = {"node_flag": torch.empty(N, dtype=torch.uint8, device=self.device),
                   "node_tier": torch.empty(N, dtype=torch.uint8, device=self.device),
                   "node_stall": torch.empty(N, dtype=torch.uint16, device=self.device)}
        g = out.get
        with self._dev():
            self._check(lib().guard_node_verdict(self._h, _ptr(g("node_flag"), torch.uint8, N),
                                                 _ptr(g("node_tier"), torch.uint8, N),
                                                 _ptr(g("node_stall"), torch.uint16, N), _stream()))
        return out

    def state_bytes(self) -> int:
        return int(lib().guard_state_bytes(self._h))

    def state_export(self, state: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Copies the context's state into `state` (a uint8 CUDA tensor of state_bytes(), allocated if None)."""
        if state is None:
            state = torch.empty(self.state_bytes(), dtype=torch.uint8, device=self.device)
        with self._dev():
            self._check(lib().guard_state_export(self._h, _ptr(state, torch.uint8), state.numel(), _stream()))
        return state

    def state_import(self, state: torch.Tensor) -> None:
        """Loads a state written by state_export of a context of the same sizes (synchronises)."""
        with self._dev():
            self._check(lib().guard_state_import(self._h, _ptr(state, torch.uint8), state.numel(), _stream()))

    def debug_set_wait_limit(self, cycles: int) -> None:
        self._check(lib().guard_debug_set_wait_limit(self._h, int(cycles)))

    def sync_status(self) -> int:
        """Synchronises the current stream; raises GuardError on a sticky device error."""
        with self._dev():
            rc = lib().guard_sync_status(self._h, _stream())
        self._check(rc)
        return rc

    def reset(self) -> None:
        with self._dev():
            self._check(lib().guard_reset(self._h, _stream()))


def sweep_qualify(S: torch.Tensor, nodes: int, gpus_per_node: int, *, dir: Sequence[int], thr=3.5, floor_rel=1e-4,
                  floor_abs=0.0, pct_ppm: int = 50_000, workspace: Optional[torch.Tensor] = None,
                  out: Optional[Dict[str, Optional[torch.Tensor]]] = None) -> Dict[str, Optional[torch.Tensor]]:
    """Node-sweep qualification of S[gpu, rep, metric]; returns the output tensors plus 'status'."""
    if S.dim() != 3 or S.shape[0] != nodes * gpus_per_node:
        raise ValueError("S must be [nodes * gpus_per_node, reps, metrics]")
    G, reps, M = S.shape
    dev = S.device
    params = _Params(M, dir, thr, floor_rel, floor_abs)
    need = int(lib().guard_sweep_workspace_bytes(G, reps, M))
    if need == 0:
        raise GuardError(-1, "invalid sweep sizes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    if out is None:
        out = {
            "gpu_med": torch.empty((G, M), dtype=torch.float32, device=dev),
            "fleet_med": torch.empty(M, dtype=torch.float32, device=dev),
            "fleet_mad": torch.empty(M, dtype=torch.float32, device=dev),
            "fleet_cut": torch.empty(M, dtype=torch.float32, device=dev),
            "fail_mask": torch.empty(G, dtype=torch.uint32, device=dev),
            "gpu_pass": torch.empty(G, dtype=torch.uint8, device=dev),
            "node_pass": torch.empty(nodes, dtype=torch.uint8, device=dev),
            "status": torch.zeros(1, dtype=torch.uint32, device=dev),
        }
    g = out.get
    with torch.cuda.device(dev):
        rc = lib().guard_sweep_qualify(
            _ptr(S, torch.float32), nodes, gpus_per_node, reps, M, C.byref(params.struct), pct_ppm,
            _ptr(workspace, torch.uint8), workspace.numel(), _ptr(g("gpu_med"), torch.float32, G * M),
            _ptr(g("fleet_med"), torch.float32, M), _ptr(g("fleet_mad"), torch.float32, M),
            _ptr(g("fleet_cut"), torch.float32, M), _ptr(g("fail_mask"), torch.uint32, G),
            _ptr(g("gpu_pass"), torch.uint8, G), _ptr(g("node_pass"), torch.uint8, nodes),
            _ptr(g("status"), torch.uint32, 1), _stream())
    if rc != GUARD_OK:
        raise GuardError(rc, lib().guard_last_error(None).decode())
    return out


class Triage:
    """Repeat-offender bookkeeping of the triage workflow: record(node, time_s) -> True when the
    node has entered triage `limit` times within `period_s` seconds and is to be terminated."""

    def __init__(self, nodes: int, limit: int = 3, period_s: int = 7 * 86400):
        self._h = C.c_void_p()
        rc = lib().guard_triage_create(C.byref(self._h), nodes, limit, period_s)
        if rc != GUARD_OK:
            raise GuardError(rc, lib().guard_last_error(None).decode())

    def record(self, node: int, time_s: int):
        n = C.c_int(0)
        rc = lib().guard_triage_record(self._h, node, int(time_s), C.byref(n))
        if rc < 0:
            raise GuardError(rc, "bad node id, or a time before the node's previous entry")
        return bool(rc), n.value

    def close(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.guard_triage_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


TOPK_STATIC_MAX_K = 256


def topk_static(wmed: torch.Tensor, fleet_med: torch.Tensor, fleet_mad: torch.Tensor, topk: int, *,
                dir: Sequence[int], floor_rel=1e-4, floor_abs=0.0, primary: int = 0,
                out_idx: Optional[torch.Tensor] = None, out_score: Optional[torch.Tensor] = None) -> None:
    """Top-k of an evaluation through guard_topk_static: the library allocates nothing, the
    caller passes every input and output tensor (outputs may be None to skip them).  Meant
    for a sidecar that shares a GPU with a training job and must not call the device
    allocator; limited to topk <= TOPK_STATIC_MAX_K.  Calls on one device share a built-in
    scratch array, so keep them on one stream."""
    if wmed.dim() != 2:
        raise ValueError("wmed must be [ranks, metrics]")
    R, M = wmed.shape
    params = _Params(M, dir, 0.0, floor_rel, floor_abs, primary=primary)
    with torch.cuda.device(wmed.device):
        rc = lib().guard_topk_static(_ptr(wmed, torch.float32), _ptr(fleet_med, torch.float32, M),
                                     _ptr(fleet_mad, torch.float32, M), R, M, C.byref(params.struct), topk,
                                     _ptr(out_idx, torch.int32, topk), _ptr(out_score, torch.float32, topk), _stream())
    if rc != GUARD_OK:
        raise GuardError(rc, lib().guard_last_error(None).decode())


def key_from_float(x: float) -> int:
    return int(lib().guard_key_from_float(C.c_float(x)))


def float_from_key(k: int) -> float:
    return float(lib().guard_float_from_key(C.c_uint32(k)))
