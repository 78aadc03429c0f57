"""Brute-force checker for tiny inputs -- TEST INFRASTRUCTURE, not the product.

A second, independent statement of the scoring definitions in pure Python: every
order statistic is `sorted(...)[index]`, every count is a loop, every float32 step is
a numpy.float32 scalar operation.  It is far too slow for anything but tiny fleets;
its only job is to pin the C oracle (oracle/guard_oracle.c), with which it shares no
code.  The statistics are the readings described in that file's header (Section 4.2
and Sections 5.2-5.4 of the paper fix the rules in words only).
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence

import numpy as np

F = np.float32


def _order_key(x: F):
    # numeric order, -0 before +0
    return (float(x), 0 if math.copysign(1.0, float(x)) < 0 else 1)


def median(vals: Sequence[F]) -> F:
    s = sorted((F(v) for v in vals), key=_order_key)
    n = len(s)
    if n % 2 == 1:
        return s[(n - 1) // 2]
    return F(F(0.5) * F(s[n // 2 - 1] + s[n // 2]))


def mad(vals: Sequence[F], med: F) -> F:
    return median([F(abs(F(F(v) - F(med)))) for v in vals])


def scale(mad_: F, med: F, floor_rel: F, floor_abs: F) -> F:
    return max(F(mad_), F(F(floor_rel) * F(abs(F(med)))), F(floor_abs))


def thrp(thr: float) -> F:
    return F(float(F(thr)) / 0.6745)


def exceeds(x: F, med: F, sc: F, d: int, tp: F) -> bool:
    dev = F(F(x) - F(med))
    if d < 0:
        dev = F(-dev)
    return bool(dev > F(F(tp) * F(sc)))


class Brute:
    def __init__(self, R, M, W, k, topk, dir, thr, floor_rel, floor_abs, primary=0, min_signals=2,
                 n_consec=1, tier_moderate=0.10, tier_severe=0.20):
        self.R, self.M, self.W, self.k, self.topk = R, M, W, k, topk
        self.dir = [(-1 if d < 0 else 1) for d in dir]
        self.tp = [thrp(t) for t in thr]
        self.frel = [F(v) for v in floor_rel]
        self.fabs = [F(v) for v in floor_abs]
        self.primary, self.min_signals, self.n_consec = primary, min_signals, n_consec
        self.tm, self.ts = F(tier_moderate), F(tier_severe)
        self.steps: List[np.ndarray] = []       # every ingested step [R, M]
        self.exc: List[List[List[bool]]] = []   # exceedance of every ingested step
        self.consec = [0] * R

    def ingest(self, block: np.ndarray):
        meds, mads = [], []
        for row in np.asarray(block, dtype=np.float32):
            e = [[False] * self.M for _ in range(self.R)]
            rm, rd = [], []
            for m in range(self.M):
                col = [row[r, m] for r in range(self.R)]
                med = median(col)
                md = mad(col, med)
                sc = scale(md, med, self.frel[m], self.fabs[m])
                for r in range(self.R):
                    e[r][m] = exceeds(col[r], med, sc, self.dir[m], self.tp[m])
                rm.append(med)
                rd.append(md)
            self.steps.append(row.copy())
            self.exc.append(e)
            meds.append(rm)
            mads.append(rd)
        return np.array(meds, np.float32), np.array(mads, np.float32)

    def score(self) -> Dict[str, np.ndarray]:
        R, M = self.R, self.M
        n = min(self.W, len(self.steps))
        win = self.steps[-n:]
        wexc = self.exc[-n:]
        wmed = [[median([s[r, m] for s in win]) for m in range(M)] for r in range(R)]
        B = [median([wmed[r][m] for r in range(R)]) for m in range(M)]
        D = [mad([wmed[r][m] for r in range(R)], B[m]) for m in range(M)]
        Ds = [scale(D[m], B[m], self.frel[m], self.fabs[m]) for m in range(M)]
        counts = [[sum(1 for e in wexc if e[r][m]) for m in range(M)] for r in range(R)]
        masks, flags, tiers = [], [], []
        p = self.primary
        for r in range(R):
            mask = 0
            for m in range(M):
                if exceeds(wmed[r][m], B[m], Ds[m], self.dir[m], self.tp[m]) and counts[r][m] >= self.k:
                    mask |= 1 << m
            cand = bool((mask >> p) & 1) and bin(mask).count("1") >= min(self.min_signals, M)
            self.consec[r] = min(self.consec[r] + 1, 255) if cand else 0
            flag = cand and self.consec[r] >= self.n_consec
            devp = F(wmed[r][p] - B[p])
            if self.dir[p] < 0:
                devp = F(-devp)
            aB = F(abs(B[p]))
            if flag and devp >= F(self.ts * aB):
                t = 3
            elif flag and devp >= F(self.tm * aB):
                t = 2
            elif mask != 0:
                t = 1
            else:
                t = 0
            masks.append(mask)
            flags.append(int(flag))
            tiers.append(t)
        self.last = (list(flags), list(tiers), n)
        keyf = lambda r: _order_key(F(-wmed[r][p]) if self.dir[p] < 0 else wmed[r][p])
        order = sorted(range(R), key=lambda r: (tuple(-c for c in keyf(r)), r))
        return {
            "wmed": np.array(wmed, np.float32), "fleet_med": np.array(B, np.float32),
            "fleet_mad": np.array(D, np.float32), "counts": np.array(counts, np.uint16),
            "mask": np.array(masks, np.uint32), "flags": np.array(flags, np.uint8),
            "tier": np.array(tiers, np.uint8), "topk_idx": np.array(order[: self.topk], np.int32),
        }


def node_verdict(b: "Brute", rpn: int):
    """Node-level fold of the last Brute.score(): any rank flagged, highest tier, and the number of
    window steps in which all ranks of the node exceeded on the primary metric together."""
    flags, tiers, n = b.last
    wexc = b.exc[-n:]
    nf, nt, ns = [], [], []
    for nd in range(b.R // rpn):
        rs = range(nd * rpn, (nd + 1) * rpn)
        nf.append(int(any(flags[r] for r in rs)))
        nt.append(max(tiers[r] for r in rs))
        ns.append(sum(1 for e in wexc if all(e[r][b.primary] for r in rs)))
    return {"node_flag": np.array(nf, np.uint8), "node_tier": np.array(nt, np.uint8),
            "node_stall": np.array(ns, np.uint16)}


def triage(times, period, limit):
    """Per entry: does the node reach `limit` triage entries no more than `period` apart?"""
    out = []
    for i, t in enumerate(times):
        out.append(int(sum(1 for u in times[: i + 1] if t - u <= period) >= limit))
    return out


def sweep(S: np.ndarray, nodes: int, gpn: int, dir, thr, floor_rel, floor_abs, pct_ppm: int):
    S = np.asarray(S, dtype=np.float32)
    G, N, M = S.shape
    gmed = [[median([S[g, i, m] for i in range(N)]) for m in range(M)] for g in range(G)]
    j = -((-pct_ppm * G) // 1_000_000)
    j = min(max(j, 1), G)
    fail = [0] * G
    Fm, Fd, Fc = [], [], []
    for m in range(M):
        col = [gmed[g][m] for g in range(G)]
        med = median(col)
        md = mad(col, med)
        sc = scale(md, med, F(floor_rel[m]), F(floor_abs[m]))
        asc = sorted(col, key=_order_key)
        d = -1 if dir[m] < 0 else 1
        cut = asc[j - 1] if d < 0 else asc[G - j]
        for g in range(G):
            z = exceeds(col[g], med, sc, d, thrp(thr[m]))
            pf = (col[g] < cut) if d < 0 else (col[g] > cut)
            if z and pf:
                fail[g] |= 1 << m
        Fm.append(med)
        Fd.append(md)
        Fc.append(cut)
    gpass = [int(f == 0) for f in fail]
    npass = [int(all(gpass[nd * gpn + q] for q in range(gpn))) for nd in range(nodes)]
    return {"gpu_med": np.array(gmed, np.float32), "fleet_med": np.array(Fm, np.float32),
            "fleet_mad": np.array(Fd, np.float32), "fleet_cut": np.array(Fc, np.float32),
            "fail_mask": np.array(fail, np.uint32), "gpu_pass": np.array(gpass, np.uint8),
            "node_pass": np.array(npass, np.uint8)}
