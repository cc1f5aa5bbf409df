"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot enumerate 10^12 pairs in a test, so at full size the checks are:
  - every emitted pair is scored one by one by the oracle (no false positive, band rule for bf16),
  - no pair is emitted twice,
  - for a sample of P rows the oracle's whole row join equals the emitted pairs of those rows
    (no false negative), within the band rule for bf16,
  - every planted pair is found; the count matches what the generator's structure fixes,
  - the WHOLE sorted pair set equals the one the oracle's plain double loop produced over all n x m pairs, compared
    through the digest tests/golden/make_full_size_digests.py stored (that oracle run takes up to an hour of host
    time per configuration, so it is not repeated here).
"""
import hashlib
import json
import os

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


def run_full(w, capacity, dense_epilogue=None):
    """One join at full size, in the launch configuration `bench.py` times.  dense_epilogue: SIMJOIN_OPT_DENSE_EPILOGUE
    (None: the default, under which a context picks the layout from a sample's pair count or from its previous join)."""
    build.build()
    with B.Simjoin(w.dtype, 0) as ctx:
        if dense_epilogue is not None:
            assert ctx.simjoin_set_option(B.SIMJOIN_OPT_DENSE_EPILOGUE, float(dense_epilogue)) == B.SIMJOIN_OK
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


def test_full_size_int8_cosine_on_the_config_4_points():
    """The cosine join of int8 points at full size: the config-4 points, t = threshold / d (unit-modulus rows)."""
    w = W.make_workload(4)
    assert np.all(np.abs(w.P[:64]) == 1)                # +-1 rows: cosine = <x,y> / d
    w.kind, w.threshold = "cos", w.threshold / w.d
    pairs, cnt = run_full(w, capacity=4 * len(w.planted))
    k = keys(pairs)
    assert len(np.unique(k)) == cnt == len(w.planted)
    assert np.isin(keys(w.planted), k).all()
    assert np.all(O.scores(w.P, w.Q, "cos", "i8", pairs) >= w.threshold)
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


@pytest.mark.parametrize("dense_epilogue", [0, 1])
def test_full_size_cfg5_mixture_dense(dense_epilogue):
    """Both layouts, each forced: 8 epilogue warps on the points themselves, and 16
    warps on the operands with the squared-L2 embedding appended (every later call of a dense join)."""
    w = W.make_workload(5)
    per_p = np.bincount(w.labels_p, minlength=1024).astype(np.int64)
    per_q = np.bincount(w.labels_q, minlength=1024).astype(np.int64)
    same_cluster = int(np.sum(per_p * per_q))
    pairs, cnt = run_full(w, capacity=int(same_cluster * 1.02), dense_epilogue=dense_epilogue)
    assert cnt == same_cluster                         # independent pin: the join is the same-cluster relation
    assert np.all(w.labels_p[pairs[:, 0]] == w.labels_q[pairs[:, 1]])
    k = keys(pairs)
    k.sort()
    assert np.all(k[1:] != k[:-1])                     # no duplicates
    sub = pairs[:: max(1, cnt // 20000)]
    d = O.scores(w.P, w.Q, "l2", "bf16", sub)
    assert np.all(d <= w.threshold * (1 + BAND_REL))
    check_sampled_rows(w, pairs, sample_rows(w, pairs, k=24), exact=False)


def stored_digests():
    with open(os.path.join(os.path.dirname(__file__), "golden", "full_size_digests.json")) as f:
        return json.load(f)


@pytest.mark.parametrize("cfg", [2, 3, 4, 5])
def test_full_size_whole_join_equals_the_oracles(cfg):
    """The complete result at full size against the oracle's complete result (stored as a digest of the sorted pair
    keys).  int8: the two sets are equal.  bf16: the result minus the oracle's 1 % band equals the oracle's strict set."""
    g = stored_digests().get(str(cfg))
    if g is None:
        pytest.skip("no stored oracle digest for this configuration (make_full_size_digests.py writes it)")
    w = W.make_workload(cfg)
    assert (w.n, w.m, w.d, w.kind, w.dtype, w.threshold) == (g["n"], g["m"], g["d"], g["kind"], g["dtype"], g["threshold"])
    assert hashlib.sha256(w.P.tobytes()).hexdigest() == g["inputs_sha256"]["P"]
    assert hashlib.sha256(w.Q.tobytes()).hexdigest() == g["inputs_sha256"]["Q"]
    want = g["count"] if w.dtype == "i8" else g["loose_count"]
    pairs, cnt = run_full(w, capacity=int(want * 1.02) + 1024)
    k = np.sort(keys(pairs))
    assert len(k) == cnt and np.all(k[1:] != k[:-1])
    if w.dtype == "i8":
        assert cnt == g["count"]
        assert hashlib.sha256(k.astype("<i8").tobytes()).hexdigest() == g["sorted_keys_sha256"]
    else:
        band = keys(np.asarray(g["band_pairs"], dtype=np.int64).reshape(-1, 2))
        k = k[~np.isin(k, band)]
        assert len(k) == g["strict_count"]
        assert hashlib.sha256(k.astype("<i8").tobytes()).hexdigest() == g["strict_sorted_keys_sha256"]


def test_full_size_cfg5_literal_sigma_is_empty():
    w = W.make_workload(5, sigma_reading="percoord")
    pairs, cnt = run_full(w, capacity=1 << 16)
    assert cnt == 0


@pytest.mark.parametrize("family", ["bits", "hyperplanes"])
def test_full_size_lsh_join_cfg4(family):
    """The LSH-bucketed join at the headline size (1 048 576 x 1 048 576, 8 tables of 7 bits), as `bench.py --lsh 8,7`
    (`--lsh-family hyperplanes`) times it, for both hash families (int8: hyperplane keys are exact integers' signs).  The result is the set {brute-force pairs whose keys agree in some table}: every emitted pair is scored
    by the oracle and its keys (the oracle's) agree in a table; nothing is emitted twice; every planted pair whose
    oracle keys agree in a table is present, and only those; sampled rows are joined whole by the oracle."""
    L, k, seed = 8, 7, 2006
    w = W.make_workload(4)
    build.build()
    cap = 4 * len(w.planted)
    with B.Simjoin("i8", 0) as ctx:
        dP, dQ = B.to_device(w.P), B.to_device(w.Q)
        out = torch.empty((cap, 2), dtype=torch.int32, device="cuda:0")
        st, cnt = ctx.simjoin_run_lsh(dP, w.n, dQ, w.m, w.d, w.threshold, L, k, seed, out, cap, family=family)
        assert st == B.SIMJOIN_OK, B.strerror(st)
        pairs = out[:cnt].cpu().numpy().astype(np.int64)
    del dP, dQ, out
    torch.cuda.empty_cache()
    gk = keys(pairs)
    assert len(np.unique(gk)) == cnt
    assert np.all(O.scores(w.P, w.Q, "ip", "i8", pairs.astype(np.int32)) >= w.threshold)
    kp, kq = O.lsh_keys(w.P, L, k, seed, family=family), O.lsh_keys(w.Q, L, k, seed, family=family)          # (L, rows)
    assert np.all((kp[:, pairs[:, 0]] == kq[:, pairs[:, 1]]).any(axis=0))      # every emitted pair collides in a table
    pl = w.planted
    collide = (kp[:, pl[:, 0]] == kq[:, pl[:, 1]]).any(axis=0)
    assert np.array_equal(np.isin(keys(pl), gk), collide)                      # planted pairs: present iff they collide
    # closed forms: bit sampling 1 - (1 - (120/128)^7)^8 = 0.9997; hyperplanes at angle acos(0.875): 1 - (1 - 0.839^7)^8 = 0.938
    assert collide.mean() > (0.999 if family == "bits" else 0.92)
    rows = sample_rows(w, pairs, k=24)
    sub_keys = kp[:, rows]
    want, _c = O.join(w.P[rows], w.Q, "ip", w.threshold, "i8")                 # brute force on the sampled rows ...
    keep = (sub_keys[:, want[:, 0]] == kq[:, want[:, 1]]).any(axis=0)          # ... restricted to colliding pairs
    want = want[keep].astype(np.int64)
    want[:, 0] = np.asarray(rows)[want[:, 0]]
    got = pairs[np.isin(pairs[:, 0], rows)]
    assert np.array_equal(np.sort(keys(got)), np.sort(keys(want)))


def test_full_size_jl_transform_sampled_rows():
    """The JL transform at the size `bench.py --jl 1048576,1024,64` times: sampled rows against the fp64 oracle, within
    the bound derived from the per-level bf16 rounding (see tests/test_gpu_jl.py)."""
    n, d, k, seed = 1 << 20, 1024, 64, 2006
    build.build()
    gen = torch.Generator(device="cuda").manual_seed(7)
    X = torch.randn((n, d), generator=gen, device="cuda:0", dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty((n, k), dtype=torch.bfloat16, device="cuda:0")
    with B.Simjoin("bf16", 0) as ctx:
        assert ctx.simjoin_jl_transform(X, n, d, k, seed, out) == B.SIMJOIN_OK
    rows = np.unique(np.concatenate([np.random.default_rng(5).choice(n, size=60, replace=False), [0, 127, 128, 255, 256, n - 1]]))
    rows_t = torch.from_numpy(rows).cuda()
    Xs = X[rows_t].view(torch.int16).cpu().numpy().view(np.uint16)
    got = out[rows_t].float().cpu().numpy().astype(np.float64)
    del X, out
    torch.cuda.empty_cache()
    want = O.jl_transform(np.ascontiguousarray(Xs), k, seed)
    sh = O.jl_shapes(d, k)
    xn = np.linalg.norm(W.bf16_bits_to_f32(Xs).astype(np.float64), axis=1)
    bound = 2.0 ** -9 * xn * (1.5 * sum(np.sqrt(c / ki) for _r, c, ki in sh) + 1.0)
    err = np.abs(got - want)
    assert np.all(err <= bound[:, None]), (err.max(), bound.min())
    assert np.sqrt((err ** 2).mean()) <= 4.0 * np.sqrt(len(sh)) * 2.0 ** -9 * np.sqrt((want ** 2).mean()) / np.sqrt(3.0)


def test_full_size_hamming_join():
    """Hamming join on 1 048 576 x 1 048 576 bit-packed points of 128 bits, r = 14: every emitted pair is checked by
    the oracle's bit count, every planted pair (8 flipped bits) is present, sampled rows are joined whole by the oracle.
    Random pairs are at distance ~64 +- 5.7, so nothing but the planted pairs is expected within 14."""
    n, d, r, k = 1 << 20, 128, 14, 50000
    P = W.random_bits(n, d, 31)
    Q = W.random_bits(n, d, 32, planted_from=P[:k], flips=8)
    build.build()
    cap = 4 * k
    with B.Simjoin("i8", 0) as ctx:
        dP, dQ = torch.from_numpy(P).cuda(), torch.from_numpy(Q).cuda()
        out = torch.empty((cap, 2), dtype=torch.int32, device="cuda:0")
        st, cnt = ctx.simjoin_run_hamming(dP, n, dQ, n, d, r, out, cap)
        assert st == B.SIMJOIN_OK, B.strerror(st)
        pairs = out[:cnt].cpu().numpy().astype(np.int64)
    del dP, dQ, out
    torch.cuda.empty_cache()
    gk = keys(pairs)
    assert len(np.unique(gk)) == cnt and cnt >= k
    x = np.unpackbits(P[pairs[:, 0]] ^ Q[pairs[:, 1]], axis=1).sum(axis=1)       # independent popcount of the emitted pairs
    assert np.all(x <= r)
    assert all(O.hamming(P[i], Q[j], d) <= r for i, j in pairs[:: max(1, cnt // 64)])
    planted = np.stack([np.arange(k), np.arange(k)], axis=1)
    assert np.isin(keys(planted), gk).all()
    rows = np.unique(np.concatenate([np.random.default_rng(9).choice(n, size=20, replace=False), [0, k - 1, k, n - 1]]))
    want, _c = O.join_hamming(P[rows], Q, d, r)
    want = want.astype(np.int64)
    want[:, 0] = rows[want[:, 0]]
    got = pairs[np.isin(pairs[:, 0], rows)]
    assert np.array_equal(np.sort(keys(got)), np.sort(keys(want)))
