"""The allocation-free top-k entry point against the regular evaluation.

guard_topk_static serves callers that cannot allocate device memory -- a telemetry sidecar
on a GPU whose memory the training job's allocator already owns, where cudaMalloc would
also stall the job by synchronising the device.  Its scratch is a fixed array inside the
library, shared by every call on the device, so the check runs it twice in a row on
different data: the second call must not be disturbed by what the first one left behind.
Every result must equal the CPU oracle's top-k of the same telemetry (indices bit for bit,
scores within the 1e-6 relative tolerance of the other tests) and guard_score's.  This file sorts last so that a stop-at-first-failure run has already
run every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _evaluation(R, M, K, seed):
    from paper_2605_17879_b200 import guard
    rng = np.random.default_rng(seed)
    dirs = [1, 1, -1, 1][:M]
    X = np.exp(0.03 * rng.normal(size=(12, R, M)))
    X[:, rng.integers(0, R, 5), 0] *= 1.3
    X = X.astype(np.float32)
    g = guard.Guard(R, M, 12, 6, dir=dirs, topk=K)
    g.ingest(torch.from_numpy(X).cuda())
    out = g.score()
    g.sync_status()
    g.close()
    from oracle import guard_oracle as go
    o = go.Oracle(R, M, 12, 6, K, dir=dirs)
    o.ingest(X)
    ref = o.score()
    out["oracle_topk_idx"], out["oracle_topk_score"] = ref["topk_idx"], ref["topk_score"]
    return out, dirs


def test_static_scratch_topk_matches_score_twice_in_a_row():
    from paper_2605_17879_b200 import guard
    R, M, K = 5000, 4, 48            # three top-k CTAs, so the candidate scratch and the ticket are used
    ref_a, dirs = _evaluation(R, M, K, seed=1)
    ref_b, _ = _evaluation(R, M, K, seed=2)
    assert not torch.equal(ref_a["topk_idx"], ref_b["topk_idx"])
    idx = torch.empty(K, dtype=torch.int32, device="cuda")
    sc = torch.empty(K, dtype=torch.float32, device="cuda")
    for ref in (ref_a, ref_b, ref_a):
        idx.fill_(-1)
        sc.fill_(float("nan"))
        torch.cuda.synchronize()
        before = torch.cuda.memory_stats()["allocation.all.allocated"]
        guard.topk_static(ref["wmed"], ref["fleet_med"], ref["fleet_mad"], K, dir=dirs, out_idx=idx, out_score=sc)
        torch.cuda.synchronize()
        # the call itself went nowhere near torch's device allocator either
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == before
        assert np.array_equal(idx.cpu().numpy(), ref["oracle_topk_idx"])
        got = sc.cpu().numpy().astype(np.float64)
        assert np.allclose(got, ref["oracle_topk_score"], rtol=1e-6, atol=1e-30)
        assert torch.equal(idx, ref["topk_idx"])
        assert np.allclose(got, ref["topk_score"].cpu().numpy().astype(np.float64), rtol=1e-6, atol=1e-30)


def test_static_scratch_limits_are_rejected():
    from paper_2605_17879_b200 import guard
    w = torch.ones((512, 2), device="cuda")
    f = torch.ones(2, device="cuda")
    idx = torch.empty(512, dtype=torch.int32, device="cuda")
    with pytest.raises(guard.GuardError) as ei:
        guard.topk_static(w, f, f, guard.TOPK_STATIC_MAX_K + 1, dir=[1, 1], out_idx=idx)
    assert ei.value.code == -1 and "scratch" in str(ei.value)
    with pytest.raises(guard.GuardError):
        guard.topk_static(w, f, f, 0, dir=[1, 1], out_idx=idx)
    with pytest.raises(guard.GuardError):
        guard.topk_static(w[:8].contiguous(), f, f, 9, dir=[1, 1], out_idx=idx)     # more than there are ranks
