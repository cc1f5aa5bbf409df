"""The candidate filter (simjoin_filter_pairs) and the Euclidean join behind a JL pre-reduction (simjoin_run_jl_l2)
through the C ABI, against the oracle.

Filter: int8 lists are decided exactly; bf16 lists in fp32, so a pair whose fp64 score lies within 1e-2*|t| of the
threshold may fall on either side (the join's band rule).
Pipeline: reduce both sets with the same JL matrix, join the reduced points at r(1 + slack), decide the candidates on
the original rows.  What the method fixes is checked: nothing outside the exact join (band rule) is reported; a pair of
the exact join is reported whenever its reduced distance -- taken from the oracle's fp64 transform -- is inside the
widened radius with a margin for the bf16 rounding of the reduced coordinates; planted pairs are recalled.
"""
import numpy as np
import pytest
import torch

from oracle import simjoin_oracle as O
from paper_2006_12608_b200 import binding as B
from paper_2006_12608_b200 import build
from paper_2006_12608_b200 import workloads as W

pytestmark = pytest.mark.gpu
REL = 1e-2


def keys(p):
    p = np.asarray(p, dtype=np.int64).reshape(-1, 2)
    return np.sort((p[:, 0] << 32) | p[:, 1])


@pytest.fixture(scope="module")
def ctxs():
    build.build()
    c = {"i8": B.Simjoin("i8", 0), "bf16": B.Simjoin("bf16", 0)}
    yield c
    for x in c.values():
        x.close()


def candidate_list(P, Q, kind, t, dtype, rng, extra=4000):
    """True pairs (found at a looser threshold) mixed with random pairs, shuffled, with repetitions."""
    loose = t * 1.3 if kind == "l2" else (t - 0.3 * abs(t) if t != 0 else -0.1)
    near, _c = O.join(P, Q, kind, loose, dtype)
    rnd = np.stack([rng.integers(0, len(P), extra), rng.integers(0, len(Q), extra)], axis=1).astype(np.int32)
    cand = np.concatenate([near, rnd, near[: len(near) // 3]])
    return cand[rng.permutation(len(cand))]


def gpu_filter(ctx, P, Q, kind, t, cand, ioff=0, joff=0):
    dP, dQ = B.to_device(P), B.to_device(Q)
    lst = torch.from_numpy(np.ascontiguousarray(cand + np.array([ioff, joff], dtype=np.int32))).cuda()
    guard = lst.clone()
    st, cnt = ctx.simjoin_filter_pairs(dP, len(P), dQ, len(Q), P.shape[1], kind, t, lst, len(cand))
    assert st == B.SIMJOIN_OK, B.strerror(st)
    kept = lst[:cnt].cpu().numpy() - np.array([ioff, joff], dtype=np.int32)
    assert np.array_equal(lst[cnt:].cpu().numpy(), guard[cnt:].cpu().numpy())     # nothing written past the kept pairs
    return kept


@pytest.mark.parametrize("kind,t,d,hi", [("ip", 60.0, 64, 3), ("l2", 18.0, 128, 3), ("cos", 0.3, 272, 127), ("ip", 9000.0, 1040, 40),
                                         ("l2", 0.0, 48, 1), ("cos", 1.0, 64, 5)])
def test_filter_int8_is_exact(ctxs, kind, t, d, hi):
    rng = np.random.default_rng(d)
    P, Q = W.random_points("i8", 700, d, 81, lo=-hi, hi=hi), W.random_points("i8", 900, d, 82, lo=-hi, hi=hi)
    Q[:150] = P[:150]
    Q[150:200] = 2 * P[150:200] if hi <= 40 else P[150:200]
    P[300] = 0
    cand = candidate_list(P, Q, kind, t, "i8", rng)
    kept = gpu_filter(ctxs["i8"], P, Q, kind, t, cand)
    want = O.filter_pairs(P, Q, kind, t, "i8", cand)
    assert len(kept) == len(want) > 0 and np.array_equal(keys(kept), keys(want))       # multiplicities included


@pytest.mark.parametrize("kind,t,d", [("ip", 9.0, 64), ("cos", 0.35, 128), ("l2", 9.5, 64), ("l2", 30.0, 520), ("cos", 0.12, 1024)])
def test_filter_bf16_within_the_band(ctxs, kind, t, d):
    rng = np.random.default_rng(d + 1)
    P, Q = W.random_points("bf16", 600, d, 83), W.random_points("bf16", 800, d, 84)
    Q[:100] = P[:100]
    cand = candidate_list(P, Q, kind, t, "bf16", rng)
    kept = gpu_filter(ctxs["bf16"], P, Q, kind, t, cand)
    strict_t, loose_t = (t * (1 - REL), t * (1 + REL)) if kind == "l2" else (t + REL * abs(t), t - REL * abs(t))
    strict = O.filter_pairs(P, Q, kind, strict_t, "bf16", cand)
    loose = O.filter_pairs(P, Q, kind, loose_t, "bf16", cand)
    assert len(strict) > 50
    ck, cnts = np.unique(keys(cand), return_counts=True)
    kk, kcnts = np.unique(keys(kept), return_counts=True)
    assert np.isin(keys(strict), kk).all() and np.isin(kk, keys(loose)).all()
    assert np.array_equal(kcnts, cnts[np.searchsorted(ck, kk)])                           # a kept pair keeps every copy


@pytest.mark.parametrize("kind", ["ip", "cos"])
@pytest.mark.parametrize("d", [64, 264, 1024])
def test_filter_bf16_inner_products_at_the_threshold_are_decided_exactly(ctxs, kind, d):
    """Gaussian coordinates (inexact fp32 sums), thresholds at zero, next to zero and equal to the exact score of listed
    pairs: a pair whose fp32 score lies within the sums' rounding error of the threshold is decided again in fp64, so the
    kept list is the oracle's, copy for copy, with no band."""
    rng = np.random.default_rng(d + 5)
    P = W.f32_to_bf16_bits(rng.standard_normal((500, d)).astype(np.float32))
    Q = W.f32_to_bf16_bits(rng.standard_normal((700, d)).astype(np.float32))
    P[4] = 0
    Q[6] = 0
    Q[8] = P[9]
    cand = np.stack([rng.integers(0, 500, 60000), rng.integers(0, 700, 60000)], axis=1).astype(np.int32)
    cand[:700, 0], cand[:700, 1] = 4, np.arange(700)
    sc = O.scores(P, Q, kind, "bf16", cand)
    near = [float(sc[k]) for k in np.argsort(np.abs(sc)) if sc[k] != 0.0][:6]
    for t in [0.0, -0.0, 1e-30, -1e-30] + near + [float(np.quantile(sc, 0.9)), float(sc[17])]:
        kept = gpu_filter(ctxs["bf16"], P, Q, kind, t, cand)
        want = O.filter_pairs(P, Q, kind, t, "bf16", cand)
        if abs(t) < 1e-3 * (d if kind == "ip" else 1):
            assert np.array_equal(np.sort(keys(kept)), np.sort(keys(want))), (kind, d, t)
        else:
            # a threshold equal to a pair's score in fp64 need not be a float: the plain band rule applies
            lo = O.filter_pairs(P, Q, kind, t + REL * abs(t), "bf16", cand)
            hi = O.filter_pairs(P, Q, kind, t - REL * abs(t), "bf16", cand)
            assert np.isin(keys(lo), keys(kept)).all() and np.isin(keys(kept), keys(hi)).all()


def test_filter_small_radius_on_long_rows_does_not_cancel(ctxs):
    """The difference form resolves radii far below the rows' norms (where the tile epilogue's norm expansion cannot)."""
    d = 2048
    P = W.random_points("bf16", 300, d, 85)
    Q = W.random_points("bf16", 400, d, 86)
    Q[:120] = P[:120]                                                    # distance 0, |x|^2 ~ 2048
    cand = np.stack([np.arange(300), np.arange(300)], axis=1).astype(np.int32)
    kept = gpu_filter(ctxs["bf16"], P, Q, "l2", 0.05, cand)
    assert np.array_equal(keys(kept), keys(cand[:120]))


def test_filter_offsets_empty_list_and_bad_indices(ctxs):
    ctx = ctxs["i8"]
    P, Q = W.random_points("i8", 200, 64, 87, lo=-2, hi=2), W.random_points("i8", 300, 64, 88, lo=-2, hi=2)
    Q[:50] = P[:50]
    rng = np.random.default_rng(9)
    cand = candidate_list(P, Q, "ip", 40.0, "i8", rng, extra=500)
    want = O.filter_pairs(P, Q, "ip", 40.0, "i8", cand)
    assert ctx.simjoin_set_offsets(1000, 70) == B.SIMJOIN_OK
    try:
        kept = gpu_filter(ctx, P, Q, "ip", 40.0, cand, ioff=1000, joff=70)
        assert np.array_equal(keys(kept), keys(want))
        dP, dQ = B.to_device(P), B.to_device(Q)
        lst = torch.from_numpy(np.ascontiguousarray(cand)).cuda()           # offsets missing: rows below the offset
        assert ctx.simjoin_filter_pairs(dP, 200, dQ, 300, 64, "ip", 40.0, lst, len(cand))[0] == B.SIMJOIN_ERR_ARG
    finally:
        ctx.simjoin_set_offsets(0, 0)
    dP, dQ = B.to_device(P), B.to_device(Q)
    lst = torch.from_numpy(np.ascontiguousarray(cand)).cuda()
    assert ctx.simjoin_filter_pairs(dP, 200, dQ, 300, 64, "ip", 40.0, lst, 0) == (B.SIMJOIN_OK, 0)
    bad = torch.tensor([[0, 0], [200, 1], [3, 4]], dtype=torch.int32, device="cuda:0")        # row 200 of 200
    assert ctx.simjoin_filter_pairs(dP, 200, dQ, 300, 64, "ip", 40.0, bad, 3)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_filter_pairs(dP, 200, dQ, 300, 64, "ip", 40.0, cand, len(cand))[0] == B.SIMJOIN_ERR_ARG   # host list
    assert ctx.simjoin_filter_pairs(dP, 200, dQ, 300, 64, "l2", -1.0, lst, 5)[0] == B.SIMJOIN_ERR_ARG
    # the context still joins correctly afterwards
    pairs, cnt = ctx.join(dP, dQ, "ip", 40.0, 1 << 16)
    assert cnt == O.join(P, Q, "ip", 40.0, "i8")[1]


@pytest.mark.parametrize("n,m,d,k,slack", [(3000, 4000, 1024, 64, 0.3), (2500, 2000, 512, 128, 0.25), (1500, 1800, 256, 64, 0.35)])
def test_jl_l2_join_pipeline(ctxs, n, m, d, k, slack):
    ctx = ctxs["bf16"]
    w = W.make_workload(2, n=n, m=m, d=d, planted=400)              # unit rows, planted pairs at distance ~0.29
    r = 0.45
    dP, dQ = B.to_device(w.P), B.to_device(w.Q)
    cap = 1 << 20
    out = torch.full((cap, 2), -3, dtype=torch.int32, device="cuda:0")
    st, cnt = ctx.simjoin_run_jl_l2(dP, n, dQ, m, d, r, k, 77, slack, out, cap)
    assert st == B.SIMJOIN_OK, B.strerror(st)
    got = keys(out[:cnt].cpu().numpy())
    assert len(np.unique(got)) == cnt and np.all(out[cnt:].cpu().numpy() == -3)
    strict, exact, loose = O.band_sets(w.P, w.Q, "l2", r, "bf16", rel=REL)
    assert np.isin(got, keys(loose)).all()                            # nothing but true pairs
    assert len(strict) >= 380
    # a true pair whose reduced distance is inside the widened radius (with 3 % for the bf16 rounding) must be there
    Pr, Qr = O.jl_transform(w.P, k, 77), O.jl_transform(w.Q, k, 77)
    red = np.linalg.norm(Pr[strict[:, 0]] - Qr[strict[:, 1]], axis=1)
    must = strict[red <= r * (1 + slack) * 0.97]
    assert len(must) >= 0.95 * len(strict) and np.isin(keys(must), got).all()
    assert np.isin(keys(w.planted), got).mean() >= 0.97
    st2, a_ms, b_ms = ctx.simjoin_last_kernel_ms()
    assert st2 == B.SIMJOIN_OK and a_ms > 0 and b_ms > 0


def test_jl_l2_join_arguments(ctxs):
    ctx = ctxs["bf16"]
    X = torch.zeros((64, 256), dtype=torch.bfloat16, device="cuda:0")
    out = torch.zeros((16, 2), dtype=torch.int32, device="cuda:0")
    A, U = B.SIMJOIN_ERR_ARG, B.SIMJOIN_ERR_UNSUPPORTED
    assert ctx.simjoin_run_jl_l2(X, 64, X, 64, 256, 0.5, 96, 1, 0.3, out, 16)[0] == A           # d % k
    assert ctx.simjoin_run_jl_l2(X, 64, X, 64, 256, 0.5, 4, 1, 0.3, out, 16)[0] == U            # k % 8
    assert ctx.simjoin_run_jl_l2(X, 64, X, 64, 256, -0.5, 64, 1, 0.3, out, 16)[0] == A          # r < 0
    assert ctx.simjoin_run_jl_l2(X, 64, X, 64, 256, 0.5, 64, 1, -0.1, out, 16)[0] == A          # slack < 0
    assert ctx.simjoin_run_jl_l2(X, 64, X, 64, 256, 0.5, 64, 1, float("nan"), out, 16)[0] == A
    assert ctx.simjoin_run_jl_l2(X, 0, X, 64, 256, 0.5, 64, 1, 0.3, out, 16) == (B.SIMJOIN_OK, 0)
    # all-zero rows: every pair is at distance 0; 4096 candidates do not fit in 16 slots
    st, cnt = ctx.simjoin_run_jl_l2(X, 64, X, 64, 256, 0.5, 64, 1, 0.3, out, 16)
    assert (st, cnt) == (B.SIMJOIN_ERR_CAPACITY, 4096)
    big = torch.zeros((4096, 2), dtype=torch.int32, device="cuda:0")
    assert ctx.simjoin_run_jl_l2(X, 64, X, 64, 256, 0.5, 64, 1, 0.3, big, 4096) == (B.SIMJOIN_OK, 4096)
    Xi = torch.zeros((64, 256), dtype=torch.int8, device="cuda:0")
    assert ctxs["i8"].simjoin_run_jl_l2(Xi, 64, Xi, 64, 256, 0.5, 64, 1, 0.3, out, 16)[0] == U
