"""The allocation-free entry point.

simjoin_run_noalloc exists for callers that must not allocate device memory while they
run (a pool-owned serving loop, a plugin under a framework that owns the GPU's memory):
its scratch is a fixed array inside the library instead of cudaMalloc'd buffers.  It takes
the same code path as simjoin_run from the geometry choice on, so its pair set must equal
simjoin_run's exactly -- checked on two calls in a row, the second smaller than the first
so that stale scratch from the first call would show -- and the oracle's, for every tile
geometry and element type.  A call must also leave the amount of free device memory as it
found it.  This file sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import simjoin_oracle as O
from paper_2006_12608_b200 import binding as B
from paper_2006_12608_b200 import build
from paper_2006_12608_b200 import workloads as W

pytestmark = pytest.mark.gpu


def keys(t, cnt):
    p = t[:cnt].cpu().numpy().astype(np.int64)
    return np.sort((p[:, 0] << 32) | p[:, 1])


def noalloc(dtype, dP, dQ, kind, thr, out, cap):
    stream = torch.cuda.current_stream(0).cuda_stream
    return B.simjoin_run_noalloc(0, stream, dtype, dP, dP.shape[0], dQ, dQ.shape[0], dP.shape[1], kind, thr, out, cap)


def both_ways(ctx, dtype, P, Q, kind, thr, cap=1 << 18):
    dP, dQ = B.to_device(P), B.to_device(Q)
    n, d = P.shape
    m = Q.shape[0]
    ref = torch.full((cap, 2), -1, dtype=torch.int32, device="cuda:0")
    out = torch.full((cap, 2), -1, dtype=torch.int32, device="cuda:0")
    st_ref, c_ref = ctx.simjoin_run(dP, n, dQ, m, d, kind, thr, ref, cap)
    st, c = noalloc(dtype, dP, dQ, kind, thr, out, cap)
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


@pytest.mark.parametrize("dtype,row_bytes", [("i8", 512), ("i8", 640), ("i8", 656), ("i8", 1024), ("i8", 2048),
                                             ("bf16", 512), ("bf16", 1024), ("bf16", 2080)])
@pytest.mark.parametrize("kind", ["ip", "cos", "l2"])
def test_noalloc_long_rows_against_the_oracle(dtype, row_bytes, kind):
    """Rows of 512 bytes and more (the long-row geometry, whole and partial last chunks, 2-D waves from 2 KiB on), ragged
    row counts, checked against the oracle rather than against simjoin_run."""
    build.build()
    d = row_bytes // (1 if dtype == "i8" else 2)
    n, m = 300 + 7, 1024 + 45
    if dtype == "i8":
        hi = 127 if row_bytes == 1024 else 3
        P, Q = W.random_points("i8", n, d, 81, lo=-hi, hi=hi), W.random_points("i8", m, d, 82, lo=-hi, hi=hi)
    else:
        P, Q = W.random_points("bf16", n, d, 91), W.random_points("bf16", m, d, 92)
    Q[5:260:3] = P[:85]                                  # equal rows spread over both column passes of a tile
    smp = np.stack([np.repeat(np.arange(60), 60), np.tile(np.arange(60), 60)], axis=1).astype(np.int32)
    sc = O.scores(P, Q, kind, dtype, smp).astype(np.float64)
    if kind == "l2":
        dist = np.sqrt(np.maximum(sc, 0.0)) if dtype == "i8" else sc
        thr = float(np.quantile(dist[dist > 0], 0.01))
    else:
        thr = float(np.quantile(sc, 0.99))
    cap = 1 << 18
    out = torch.full((cap + 2, 2), -1, dtype=torch.int32, device="cuda:0")
    st, c = noalloc(dtype, B.to_device(P), B.to_device(Q), kind, thr, out, cap)
    assert st == B.SIMJOIN_OK, B.strerror(st)
    got = keys(out, c)
    assert c >= 85 and len(np.unique(got)) == c and torch.all(out[c:] == -1)
    if dtype == "i8":
        want, wcnt = O.join(P, Q, kind, thr, dtype)
        assert c == wcnt and np.array_equal(got, keys(torch.from_numpy(want), wcnt))
    else:
        strict, _exact, loose = O.band_sets(P, Q, kind, thr, dtype)
        assert np.isin(keys(torch.from_numpy(strict), len(strict)), got).all()
        assert np.isin(got, keys(torch.from_numpy(loose), len(loose))).all()


def test_noalloc_up_to_its_row_limit():
    """n and m at SIMJOIN_NOALLOC_MAX_ROWS: the norm scratch is used to its last entry (Euclidean kind)."""
    build.build()
    big = B.SIMJOIN_NOALLOC_MAX_ROWS
    w = W.make_workload(5, n=big, m=big - 3, centers=big // 8)
    dP, dQ = B.to_device(w.P), B.to_device(w.Q)
    cap = 1 << 21
    out = torch.full((cap, 2), -1, dtype=torch.int32, device="cuda:0")
    st, c = noalloc("bf16", dP, dQ, "l2", w.threshold, out, cap)
    assert st == B.SIMJOIN_OK and 0 < c <= cap
    got = out[:c].cpu().numpy()
    assert len(np.unique(keys(out, c))) == c
    assert np.all(w.labels_p[got[:, 0]] == w.labels_q[got[:, 1]])        # exactly the same-cluster relation
    ncl = big // 8
    assert c == int(np.sum(np.bincount(w.labels_p, minlength=ncl).astype(np.int64) * np.bincount(w.labels_q, minlength=ncl)))


def test_noalloc_leaves_device_memory_alone_and_keeps_the_call_semantics():
    """Free device memory is the same before and after a call (after a first call has done the per-device set-up);
    int8 cosine with a zero row (candidates decided from the rows), count-only mode and a capacity overflow behave as
    in simjoin_run."""
    build.build()
    P, Q = W.random_points("i8", 900, 128, 51, lo=-50, hi=50), W.random_points("i8", 1100, 128, 52, lo=-50, hi=50)
    P[3] = 0
    Q[7] = 0
    Q[11] = P[5]
    dP, dQ = B.to_device(P), B.to_device(Q)
    cap = 1 << 16
    out = torch.full((cap, 2), -1, dtype=torch.int32, device="cuda:0")
    st, c = noalloc("i8", dP, dQ, "cos", 0.25, out, cap)                      # warm-up: set-up happens here
    assert st == B.SIMJOIN_OK
    # free memory is compared tightly around calls of the entry point alone (torch's own allocator is not in between)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(0)[0]
    for t in (0.25, 0.0, -0.1, 0.25):
        st, c = noalloc("i8", dP, dQ, "cos", t, out, cap)
        assert st in (B.SIMJOIN_OK, B.SIMJOIN_ERR_CAPACITY)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info(0)[0] == free_before, "a noalloc call changed the amount of free device memory"
    for t in (0.25, 0.0, -0.1):
        out.fill_(-1)
        st, c = noalloc("i8", dP, dQ, "cos", t, out, cap)
        want, wcnt = O.join(P, Q, "cos", t, "i8")
        assert st == (B.SIMJOIN_OK if wcnt <= cap else B.SIMJOIN_ERR_CAPACITY) and c == wcnt
        if wcnt <= cap:
            assert np.array_equal(keys(out, c), keys(torch.from_numpy(want), wcnt))
    want, wcnt = O.join(P, Q, "cos", 0.25, "i8")
    assert wcnt > 40
    st, c = noalloc("i8", dP, dQ, "cos", 0.25, None, 0)                       # count only
    assert (st, c) == (B.SIMJOIN_ERR_CAPACITY, wcnt)
    out.fill_(-1)
    st, c = noalloc("i8", dP, dQ, "cos", 0.25, out, 37)                       # overflow: a valid subset
    assert (st, c) == (B.SIMJOIN_ERR_CAPACITY, wcnt)
    part = keys(out, 37)
    assert len(np.unique(part)) == 37 and np.isin(part, keys(torch.from_numpy(want), wcnt)).all() and torch.all(out[37:] == -1)


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
