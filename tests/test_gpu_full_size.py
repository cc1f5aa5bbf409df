"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot enumerate 10^12 pairs in a test, so at full size the checks are:
  - every emitted pair is scored one by one by the oracle (no false positive, band rule for bf16),
  - no pair is emitted twice,
  - for a sample of P rows the oracle's whole row join equals the emitted pairs of those rows
    (no false negative), within the band rule for bf16,
  - every planted pair is found; the count matches what the generator's structure fixes.
"""
import numpy as np
import pytest
import torch

from oracle import simjoin_oracle as O
from paper_2006_12608_b200 import binding as B
from paper_2006_12608_b200 import build
from paper_2006_12608_b200 import workloads as W

pytestmark = pytest.mark.gpu
BAND_REL = 1e-2


def keys(p):
    p = np.asarray(p, dtype=np.int64).reshape(-1, 2)
    return (p[:, 0] << 32) | p[:, 1]


def run_full(w, capacity):
    build.build()
    with B.Simjoin(w.dtype, 0) as ctx:
        dP, dQ = B.to_device(w.P), B.to_device(w.Q)
        out = torch.empty((capacity, 2), dtype=torch.int32, device="cuda:0")
        st, cnt = ctx.simjoin_run(dP, w.n, dQ, w.m, w.d, w.kind, w.threshold, out, capacity)
        assert st == B.SIMJOIN_OK, B.strerror(st)
        pairs = out[:cnt].cpu().numpy()
    del dP, dQ, out
    torch.cuda.empty_cache()
    return pairs, cnt


def check_sampled_rows(w, pairs, rows, exact):
    """Oracle join of the sampled rows of P against all of Q vs the emitted pairs in those rows."""
    rows = np.sort(np.asarray(rows))
    sub = w.P[rows]
    got = pairs[np.isin(pairs[:, 0], rows)]
    gk = np.sort(keys(got))
    t = w.threshold
    if exact:
        want, _c = O.join(sub, w.Q, w.kind, t, w.dtype)
        want[:, 0] = rows[want[:, 0]]
        assert np.array_equal(gk, np.sort(keys(want)))
    else:
        strict, _e, loose = O.band_sets(sub, w.Q, w.kind, t, w.dtype, rel=BAND_REL)
        strict[:, 0] = rows[strict[:, 0]]
        loose[:, 0] = rows[loose[:, 0]]
        assert np.isin(keys(strict), gk).all() and np.isin(gk, keys(loose)).all()


def sample_rows(w, pairs, k=48, seed=3):
    rng = np.random.default_rng(seed)
    rows = set(rng.choice(w.n, size=k, replace=False).tolist())
    rows |= set(pairs[:: max(1, len(pairs) // 16), 0].tolist()[:16])      # rows known to have output
    rows |= {0, w.n - 1}
    return sorted(rows)


@pytest.mark.parametrize("cfg", [3, 4])
def test_full_size_int8(cfg):
    w = W.make_workload(cfg)
    pairs, cnt = run_full(w, capacity=4 * len(w.planted))
    k = keys(pairs)
    assert len(np.unique(k)) == cnt
    assert cnt == len(w.planted)                       # background pairs: < 1e-3 expected (closed-form tails)
    assert np.isin(keys(w.planted), k).all()
    sc = O.scores(w.P, w.Q, "ip", "i8", pairs)
    assert np.all(sc >= w.threshold)                   # every emitted pair verified one by one
    check_sampled_rows(w, pairs, sample_rows(w, pairs), exact=True)


def test_full_size_cfg2_cosine():
    w = W.make_workload(2)
    pairs, cnt = run_full(w, capacity=1 << 16)
    k = keys(pairs)
    assert len(np.unique(k)) == cnt == len(w.planted)
    assert np.isin(keys(w.planted), k).all()
    sc = O.scores(w.P, w.Q, "cos", "bf16", pairs)
    assert np.all(sc >= w.threshold * (1 - BAND_REL))
    check_sampled_rows(w, pairs, sample_rows(w, pairs), exact=False)


def test_full_size_cfg5_mixture_dense():
    w = W.make_workload(5)
    per_p = np.bincount(w.labels_p, minlength=1024).astype(np.int64)
    per_q = np.bincount(w.labels_q, minlength=1024).astype(np.int64)
    same_cluster = int(np.sum(per_p * per_q))
    pairs, cnt = run_full(w, capacity=int(same_cluster * 1.02))
    assert cnt == same_cluster                         # independent pin: the join is the same-cluster relation
    assert np.all(w.labels_p[pairs[:, 0]] == w.labels_q[pairs[:, 1]])
    k = keys(pairs)
    k.sort()
    assert np.all(k[1:] != k[:-1])                     # no duplicates
    sub = pairs[:: max(1, cnt // 20000)]
    d = O.scores(w.P, w.Q, "l2", "bf16", sub)
    assert np.all(d <= w.threshold * (1 + BAND_REL))
    check_sampled_rows(w, pairs, sample_rows(w, pairs, k=24), exact=False)


def test_full_size_cfg5_literal_sigma_is_empty():
    w = W.make_workload(5, sigma_reading="percoord")
    pairs, cnt = run_full(w, capacity=1 << 16)
    assert cnt == 0
