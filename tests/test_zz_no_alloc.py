"""The allocation-free entry point against the regular one.

simjoin_run_noalloc exists for callers that must not allocate device memory while they
run (a pool-owned serving loop, a plugin under a framework that owns the GPU's memory):
its scratch is a fixed array inside the library instead of cudaMalloc'd buffers.  It runs
the same kernels, so its pair set must equal simjoin_run's exactly -- checked on two calls
in a row, the second smaller than the first so that stale scratch from the first call
would show.  This file sorts last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2006_12608_b200 import binding as B
from paper_2006_12608_b200 import build
from paper_2006_12608_b200 import workloads as W

pytestmark = pytest.mark.gpu


def keys(t, cnt):
    p = t[:cnt].cpu().numpy().astype(np.int64)
    return np.sort((p[:, 0] << 32) | p[:, 1])


def both_ways(ctx, dtype, P, Q, kind, thr, cap=1 << 18):
    dP, dQ = B.to_device(P), B.to_device(Q)
    n, d = P.shape
    m = Q.shape[0]
    ref = torch.full((cap, 2), -1, dtype=torch.int32, device="cuda:0")
    out = torch.full((cap, 2), -1, dtype=torch.int32, device="cuda:0")
    st_ref, c_ref = ctx.simjoin_run(dP, n, dQ, m, d, kind, thr, ref, cap)
    stream = torch.cuda.current_stream(0).cuda_stream
    st, c = B.simjoin_run_noalloc(0, stream, dtype, dP, n, dQ, m, d, kind, thr, out, cap)
    assert st_ref == B.SIMJOIN_OK and st == B.SIMJOIN_OK, (B.strerror(st_ref), B.strerror(st))
    assert c == c_ref and c > 0
    assert np.array_equal(keys(out, c), keys(ref, c_ref))
    assert torch.all(out[c:] == -1)


def test_noalloc_matches_simjoin_run_twice_in_a_row():
    build.build()
    assert torch.cuda.is_available()
    with B.Simjoin("bf16", 0) as ctx:
        # first call: cosine join (uses the norm scratch for both sides and the per-tile bounds)
        w = W.make_workload(2, n=5000, m=4200, planted=150)
        both_ways(ctx, "bf16", w.P, w.Q, "cos", w.threshold)
        # second call, smaller and another kind: norms of the first call are still in the array
        w5 = W.make_workload(5, n=1500, m=1300, centers=20)
        both_ways(ctx, "bf16", w5.P, w5.Q, "l2", w5.threshold)
    with B.Simjoin("i8", 0) as ctx:
        w3 = W.make_workload(3, n=2100, m=1900, planted=80)
        both_ways(ctx, "i8", w3.P, w3.Q, "ip", w3.threshold)
        P, Q = W.random_points("i8", 700, 64, 41), W.random_points("i8", 900, 64, 42)
        both_ways(ctx, "i8", P, Q, "l2", 21.0)


def test_noalloc_rejects_sizes_beyond_its_scratch():
    build.build()
    big = B.SIMJOIN_NOALLOC_MAX_ROWS + 1
    X = torch.zeros((big, 16), dtype=torch.int8, device="cuda:0")
    out = torch.zeros((8, 2), dtype=torch.int32, device="cuda:0")
    stream = torch.cuda.current_stream(0).cuda_stream
    st, c = B.simjoin_run_noalloc(0, stream, "i8", X, big, X, 16, 16, "ip", 1.0, out, 8)
    assert st == B.SIMJOIN_ERR_UNSUPPORTED and c == 0
    st, c = B.simjoin_run_noalloc(0, stream, "i8", X, 16, X, big, 16, "l2", 1.0, out, 8)
    assert st == B.SIMJOIN_ERR_UNSUPPORTED and c == 0
    st, c = B.simjoin_run_noalloc(0, stream, "i8", X, 16, X, 16, 16, "ip", 1.0, out, 8)   # still usable
    assert st == B.SIMJOIN_OK and c == 0
