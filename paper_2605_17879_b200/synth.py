"""Seeded synthetic fleet telemetry and node-sweep results.

The paper evaluates on production telemetry that is not public; these generators
stand in for it with the shapes and structure of the five workload configurations
(ranks x steps x metrics, log-normal step times, persistent stragglers, transient
spikes, fail-slow ramps, whole-node stalls, repeated per-GPU benchmark results).

Everything is drawn from one counter-based generator (splitmix64 of a counter built
from seed / stream / step / rank, Box-Muller for normals), written with torch integer
and float64 tensor ops so the same code runs on the CPU (small cases, tests) and on a
CUDA device (large cases, in chunks of steps).  This module holds none of the scoring
method's arithmetic: it only produces inputs, which are then handed, as the same
buffer, to both the CUDA library and the CPU oracle.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import torch

_MASK64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int -> the signed 64-bit value with the same low 64 bits."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 tensors (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _splitmix64(x: torch.Tensor) -> torch.Tensor:
    """The splitmix64 output function applied to counter tensor x (int64, wrapping)."""
    z = x + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def _splitmix64_int(x: int) -> int:
    z = (x + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


class _Streams:
    """Independent random streams indexed by an integer counter tensor."""

    def __init__(self, seed: int, domain: int):
        self.base = _splitmix64_int(_splitmix64_int(seed) ^ (domain * 0xD1B54A32D192ED03 & _MASK64))

    def _key(self, stream: int) -> int:
        return _s64(_splitmix64_int(self.base ^ (stream * 0x8CB92BA72F3D8DD7 & _MASK64)))

    def bits(self, stream: int, ctr: torch.Tensor) -> torch.Tensor:
        return _splitmix64(_splitmix64(ctr + self._key(stream)))

    def uniform(self, stream: int, ctr: torch.Tensor) -> torch.Tensor:
        """float64 uniform in (0, 1)."""
        h = _lsr(self.bits(stream, ctr), 12)
        return (h.to(torch.float64) + 0.5) * (1.0 / 4503599627370496.0)

    def normal(self, stream: int, ctr: torch.Tensor) -> torch.Tensor:
        """float64 standard normal by Box-Muller from two sub-streams."""
        u1 = self.uniform(2 * stream, ctr)
        u2 = self.uniform(2 * stream + 1, ctr)
        return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


# stream numbers (normal streams use 2s and 2s+1 internally, so keep them apart)
_S_BASE, _S_COMP, _S_COMM, _S_FWD, _S_BWD, _S_HOST = 0, 1, 2, 3, 4, 5
_S_T0, _S_T1, _S_T2, _S_T3 = 6, 7, 8, 9
_U_SPIKE, _U_SPIKE_MAG, _U_STALL = 40, 41, 42
_R_NODE, _R_PICK, _R_FACTOR, _R_START = 0, 1, 2, 3


@dataclasses.dataclass(frozen=True)
class FleetConfig:
    """One telemetry workload plus the detector parameters quoted with it."""

    name: str
    ranks: int
    steps: int
    metrics: int
    sigma: float
    seed: int
    W: int
    k: int
    topk: int
    block: int                        # steps per ingest call (score after each block)
    node_sigma: float = 0.0           # per-node (8-rank group) offset ~ N(0, node_sigma)
    n_persistent: int = 0             # ranks slowed for all steps
    persistent_lo: float = 1.2
    persistent_hi: float = 1.2
    spike_p: float = 0.0              # Bernoulli per (step, rank)
    spike_lo: float = 3.0
    spike_hi: float = 3.0
    n_ramp: int = 0                   # ranks with a linear fail-slow ramp
    ramp_to: float = 1.3
    ramp_len: int = 5000
    ramp_start_max: int = 0           # ramp start ~ U{0..ramp_start_max}
    heavy_tail: float = 0.0           # additive scale * Student-t(3) on ramp ranks
    stall_p: float = 0.0              # Bernoulli per (node, step): all ranks of node x stall_x
    stall_x: float = 2.0
    ranks_per_node: int = 8
    capacity: Optional[int] = None    # ring capacity in steps (default: max(W, block))

    @property
    def cells(self) -> int:
        return self.ranks * self.steps * self.metrics

    @property
    def ring_capacity(self) -> int:
        return self.capacity if self.capacity is not None else max(self.W, self.block)


# direction of "worse": +1 larger is worse (durations), -1 smaller is worse (throughput)
FLEET_DIR8 = (1, 1, 1, -1, 1, 1, 1, -1)


def fleet_dir(metrics: int) -> List[int]:
    if metrics <= 8:
        return list(FLEET_DIR8[:metrics])
    return list(FLEET_DIR8) + [1] * (metrics - 8)


def paper_configs() -> Dict[str, FleetConfig]:
    """The four telemetry configurations (tiny, medium, large, streaming)."""
    return {
        "tiny": FleetConfig("tiny", ranks=64, steps=1000, metrics=4, sigma=0.02, seed=0, W=50, k=30,
                            topk=8, block=50, n_persistent=2, persistent_lo=1.2, persistent_hi=1.2,
                            spike_p=0.001, spike_lo=3.0, spike_hi=3.0),
        "medium": FleetConfig("medium", ranks=1024, steps=10_000, metrics=8, sigma=0.03, seed=1, W=100,
                              k=60, topk=16, block=100, node_sigma=0.005, n_persistent=5,
                              persistent_lo=1.05, persistent_hi=1.5, spike_p=0.002, spike_lo=2.0,
                              spike_hi=5.0),
        "large": FleetConfig("large", ranks=16_384, steps=20_000, metrics=8, sigma=0.03, seed=2, W=200,
                             k=120, topk=64, block=200, node_sigma=0.005, n_ramp=16, ramp_to=1.3,
                             ramp_len=5000, ramp_start_max=14_999, heavy_tail=0.01),
        "streaming": FleetConfig("streaming", ranks=32_768, steps=50_000, metrics=8, sigma=0.03, seed=3,
                                 W=200, k=120, topk=64, block=1, node_sigma=0.005, n_ramp=33,
                                 ramp_to=1.3, ramp_len=5000, ramp_start_max=44_999, heavy_tail=0.01,
                                 stall_p=1e-4, stall_x=2.0, capacity=512),
    }


def _rank_tables(cfg: FleetConfig, device) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor, torch.Tensor]:
    """Per-rank tables drawn once from the seed: node offset, persistent factor,
    ramp flag and ramp start step."""
    st = _Streams(cfg.seed, domain=1)
    r = torch.arange(cfg.ranks, dtype=torch.int64, device=device)
    n_nodes = (cfg.ranks + cfg.ranks_per_node - 1) // cfg.ranks_per_node
    node = torch.arange(n_nodes, dtype=torch.int64, device=device)
    node_off = 1.0 + cfg.node_sigma * st.normal(_R_NODE, node)
    node_off_r = node_off[r // cfg.ranks_per_node]
    # pick the slowed ranks: those with the smallest hash
    pick = _lsr(st.bits(100 + _R_PICK, r), 1)
    order = torch.argsort(pick)
    factor = torch.ones(cfg.ranks, dtype=torch.float64, device=device)
    is_ramp = torch.zeros(cfg.ranks, dtype=torch.bool, device=device)
    start = torch.zeros(cfg.ranks, dtype=torch.int64, device=device)
    n_p = min(cfg.n_persistent, cfg.ranks)
    if n_p:
        chosen = order[:n_p]
        u = st.uniform(100 + _R_FACTOR, chosen)
        factor[chosen] = cfg.persistent_lo + (cfg.persistent_hi - cfg.persistent_lo) * u
    n_r = min(cfg.n_ramp, cfg.ranks - n_p)
    if n_r:
        chosen = order[n_p:n_p + n_r]
        is_ramp[chosen] = True
        u = st.uniform(100 + _R_START, chosen)
        start[chosen] = torch.clamp((u * (cfg.ramp_start_max + 1)).to(torch.int64), max=cfg.ramp_start_max)
    return node_off_r, factor, is_ramp, start


def fleet_truth(cfg: FleetConfig) -> Dict[str, List]:
    """Which ranks the generator degrades (for behavioural tests, not for parity)."""
    _, factor, is_ramp, start = _rank_tables(cfg, "cpu")
    pers = torch.nonzero(factor != 1.0).flatten().tolist()
    ramp = torch.nonzero(is_ramp).flatten().tolist()
    return {"persistent": pers, "persistent_factor": factor[pers].tolist() if pers else [],
            "ramp": ramp, "ramp_start": start[ramp].tolist() if ramp else []}


def fleet_block(cfg: FleetConfig, t0: int, t1: int, device="cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Telemetry for steps [t0, t1): float32 tensor [t1 - t0, ranks, metrics], metric innermost.

    Metric columns: 0 step time, 1 compute phase, 2 communication phase, 3 tokens/s and,
    with 8 metrics, 4 forward, 5 backward, 6 host/data wait, 7 TFLOP/s.  Extra columns
    beyond 8 (only used by tests) repeat the step time with independent noise.
    """
    R, M, sg = cfg.ranks, cfg.metrics, cfg.sigma
    st = _Streams(cfg.seed, domain=2)
    node_off, factor, is_ramp, start = _rank_tables(cfg, device)
    t = torch.arange(t0, t1, dtype=torch.int64, device=device)[:, None]
    r = torch.arange(R, dtype=torch.int64, device=device)[None, :]
    ctr = t * R + r                                                   # [B, R]
    s = torch.exp(sg * st.normal(_S_BASE, ctr)) * node_off[None, :] * factor[None, :]
    if cfg.n_ramp:
        frac = torch.clamp((t - start[None, :]).to(torch.float64) / float(cfg.ramp_len), 0.0, 1.0)
        ramp = 1.0 + (cfg.ramp_to - 1.0) * frac
        s = s * torch.where(is_ramp[None, :], ramp, torch.ones_like(ramp))
    if cfg.spike_p > 0.0:
        hit = st.uniform(_U_SPIKE, ctr) < cfg.spike_p
        mag = cfg.spike_lo + (cfg.spike_hi - cfg.spike_lo) * st.uniform(_U_SPIKE_MAG, ctr)
        s = s * torch.where(hit, mag, torch.ones_like(mag))
    if cfg.stall_p > 0.0:
        n_nodes = (R + cfg.ranks_per_node - 1) // cfg.ranks_per_node
        nctr = t * n_nodes + (r // cfg.ranks_per_node)
        stall = st.uniform(_U_STALL, nctr) < cfg.stall_p
        s = s * torch.where(stall, torch.full_like(s, cfg.stall_x), torch.ones_like(s))
    if cfg.heavy_tail > 0.0 and cfg.n_ramp:
        z = st.normal(_S_T0, ctr)
        chi = st.normal(_S_T1, ctr) ** 2 + st.normal(_S_T2, ctr) ** 2 + st.normal(_S_T3, ctr) ** 2
        t3 = z / torch.sqrt(chi / 3.0)
        s = s + torch.where(is_ramp[None, :], cfg.heavy_tail * t3, torch.zeros_like(t3))
        s = torch.clamp(s, min=0.05)
    if out is None:
        out = torch.empty((t1 - t0, R, M), dtype=torch.float32, device=device)
    half = 0.5 * sg
    cols = [s]
    if M > 1:
        m1 = 0.7 * s * torch.exp(half * st.normal(_S_COMP, ctr))
        cols.append(m1)
    if M > 2:
        cols.append(0.3 * s * torch.exp(half * st.normal(_S_COMM, ctr)))
    if M > 3:
        cols.append(4096.0 / s)
    if M > 4:
        cols.append(0.25 * s * torch.exp(half * st.normal(_S_FWD, ctr)))
    if M > 5:
        cols.append(0.45 * s * torch.exp(half * st.normal(_S_BWD, ctr)))
    if M > 6:
        cols.append(0.05 * torch.exp(sg * st.normal(_S_HOST, ctr)))
    if M > 7:
        cols.append(400.0 / m1)
    for m in range(8, M):
        cols.append(s * torch.exp(half * st.normal(10 + m, ctr)))
    for m in range(M):
        out[:, :, m] = cols[m].to(torch.float32)
    return out


def fleet_tensor(cfg: FleetConfig, device="cpu", chunk: int = 256, steps: Optional[int] = None,
                 out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """All steps (or the first `steps`) of a configuration, generated chunk by chunk."""
    T = cfg.steps if steps is None else steps
    if out is None:
        out = torch.empty((T, cfg.ranks, cfg.metrics), dtype=torch.float32, device=device)
    for t0 in range(0, T, chunk):
        t1 = min(T, t0 + chunk)
        fleet_block(cfg, t0, t1, device=out.device, out=out[t0:t1])
    return out


# ----------------------------------------------------------------------------- node sweep

@dataclasses.dataclass(frozen=True)
class SweepConfig:
    name: str = "sweep"
    nodes: int = 2048
    gpus_per_node: int = 8
    reps: int = 200
    metrics: int = 6
    seed: int = 4
    gpu_sigma: float = 0.01           # per-GPU spread of the normalised throughput metrics
    rep_sigma: float = 0.003          # per-repetition multiplicative noise
    degraded_frac: float = 0.01
    degrade_lo: float = 0.03
    degrade_hi: float = 0.25
    pct_ppm: int = 50_000             # 5 % tail

    @property
    def gpus(self) -> int:
        return self.nodes * self.gpus_per_node

    @property
    def cells(self) -> int:
        return self.gpus * self.reps * self.metrics


# GEMM, HBM, intra-node bus, inter-node bus (normalised, smaller is worse);
# temperature-throttle fraction (larger is worse); clock MHz (smaller is worse)
SWEEP_DIR6 = (-1, -1, -1, -1, 1, -1)
SWEEP_FLOOR_ABS6 = (0.0, 0.0, 0.0, 0.0, 1e-3, 7.5)


def sweep_dir(metrics: int) -> List[int]:
    return list(SWEEP_DIR6[:metrics]) + [-1] * max(0, metrics - 6)


def sweep_floor_abs(metrics: int) -> List[float]:
    return list(SWEEP_FLOOR_ABS6[:metrics]) + [0.0] * max(0, metrics - 6)


def sweep_tables(cfg: SweepConfig, device="cpu"):
    """Per-GPU tables: degraded flag, degraded metric, degradation amount."""
    st = _Streams(cfg.seed, domain=3)
    g = torch.arange(cfg.gpus, dtype=torch.int64, device=device)
    n_bad = int(round(cfg.degraded_frac * cfg.gpus))
    order = torch.argsort(_lsr(st.bits(200, g), 1))
    bad = torch.zeros(cfg.gpus, dtype=torch.bool, device=device)
    bad[order[:n_bad]] = True
    which = torch.clamp((st.uniform(201, g) * cfg.metrics).to(torch.int64), max=cfg.metrics - 1)
    amount = cfg.degrade_lo + (cfg.degrade_hi - cfg.degrade_lo) * st.uniform(202, g)
    return bad, which, amount


def sweep_tensor(cfg: SweepConfig, device="cpu") -> torch.Tensor:
    """Benchmark results S[gpu, rep, metric] float32 (gpu = node * gpus_per_node + local gpu)."""
    st = _Streams(cfg.seed, domain=4)
    G, N, M = cfg.gpus, cfg.reps, cfg.metrics
    g = torch.arange(G, dtype=torch.int64, device=device)
    bad, which, amount = sweep_tables(cfg, device)
    ctr = g[:, None] * N + torch.arange(N, dtype=torch.int64, device=device)[None, :]
    dirs = sweep_dir(M)
    out = torch.empty((G, N, M), dtype=torch.float32, device=device)
    for m in range(M):
        hit = (bad & (which == m))[:, None]
        if m == 4:      # fraction of time spent thermally throttled
            u = st.uniform(300 + m, g)
            base = torch.where(u < 0.97, torch.zeros_like(u), 0.02 * st.uniform(310 + m, g))
            col = base[:, None] * torch.exp(cfg.rep_sigma * st.normal(20 + m, ctr))
            col = torch.where(hit, col + amount[:, None], col)          # larger is worse
        elif m == 5:    # clock in MHz, quantised to 15 MHz steps
            u = st.uniform(300 + m, g)
            geo = torch.floor(torch.log(st.uniform(310 + m, g)) / math.log(0.5)) + 1.0
            base = torch.where(u < 0.90, torch.full_like(u, 1965.0), 1965.0 - 15.0 * geo)
            base = torch.where(hit[:, 0], base * (1.0 - amount), base)
            base = torch.round(base / 15.0) * 15.0
            col = base[:, None].expand(G, N)
        else:           # normalised throughput / bandwidth
            base = 1.0 + cfg.gpu_sigma * st.normal(30 + m, g)
            col = base[:, None] * torch.exp(cfg.rep_sigma * st.normal(20 + m, ctr))
            sgn = 1.0 + amount if dirs[m] > 0 else 1.0 - amount
            col = torch.where(hit, col * sgn[:, None], col)
        out[:, :, m] = col.to(torch.float32)
    return out
