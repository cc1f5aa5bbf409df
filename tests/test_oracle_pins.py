"""Pins for the CPU oracle: everything here checks the oracle against something
other than itself -- hand-worked joins (tests/golden), closed forms, an
independent bit-counting formulation, exact rational brute force, a BLAS
product, and the invariants the join's definition (Section 4) fixes.  No GPU."""
import glob
import itertools
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import simjoin_oracle as O
from paper_2006_12608_b200 import workloads as W


def as_set(pairs):
    return set(map(tuple, np.asarray(pairs).reshape(-1, 2).tolist()))


def to_arr(rows, dtype):
    a = np.asarray(rows, dtype=np.float64)
    if dtype == "i8":
        return a.astype(np.int8)
    bits = W.f32_to_bf16_bits(a.astype(np.float32))
    assert np.array_equal(W.bf16_bits_to_f32(bits).astype(np.float64), a), "fixture value not exact in bf16"
    return bits


# ------------------------------------------------------------------ hand-worked
GOLDEN = sorted(g for g in glob.glob(os.path.join(os.path.dirname(__file__), "golden", "*.json"))
                if not os.path.basename(g).startswith(("hamming", "lsh_", "full_size_")))


@pytest.mark.parametrize("path", GOLDEN, ids=[os.path.basename(p) for p in GOLDEN])
def test_hand_worked_cases(path):
    with open(path) as f:
        g = json.load(f)
    P, Q = to_arr(g["P"], g["dtype"]), to_arr(g["Q"], g["dtype"])
    allp = np.array(list(itertools.product(range(len(P)), range(len(Q)))), dtype=np.int32)
    sc = O.scores(P, Q, g["kind"], g["dtype"], allp).reshape(len(P), len(Q))
    np.testing.assert_allclose(sc, np.array(g["scores"], dtype=np.float64), rtol=1e-15, atol=0)
    for case in g["cases"]:
        pairs, cnt = O.join(P, Q, g["kind"], case["threshold"], g["dtype"])
        assert cnt == len(case["pairs"]), case
        assert pairs.tolist() == sorted(case["pairs"]), case      # sorted by (i, j)


def test_hamming_hand_worked_case():
    with open(os.path.join(os.path.dirname(__file__), "golden", "hamming_bits_d16.json")) as f:
        g = json.load(f)
    d = g["d"]
    P = np.packbits(np.array(g["P"], dtype=np.uint8), axis=1, bitorder="little")
    Q = np.packbits(np.array(g["Q"], dtype=np.uint8), axis=1, bitorder="little")
    for i in range(len(P)):
        for j in range(len(Q)):
            assert O.hamming(P[i], Q[j], d) == g["distances"][i][j]
    for case in g["cases"]:
        pairs, cnt = O.join_hamming(P, Q, d, case["r"])
        assert cnt == len(case["pairs"]) and pairs.tolist() == sorted(case["pairs"]), case


def test_hamming_oracle_against_embeddings_and_pm1_inner_product():
    # three independent routes to the same set: (a) the paper's f, g embedding with d' = 2d,
    # (b) <x+-, y+-> = d - 2*Hamming through the int8 inner-product oracle, (c) numpy on unpacked bits
    d = 128
    P = W.random_bits(60, d, 1)
    Q = W.random_bits(90, d, 2, planted_from=P[:12], flips=9)
    pu = np.unpackbits(P, axis=1, bitorder="little").astype(np.int64)
    qu = np.unpackbits(Q, axis=1, bitorder="little").astype(np.int64)
    f = np.stack([pu, 1 - pu], axis=2).reshape(len(P), -1)
    g = np.stack([1 - qu, qu], axis=2).reshape(len(Q), -1)
    H = f @ g.T
    assert np.array_equal(H, (pu[:, None, :] != qu[None, :, :]).sum(axis=2))
    for r in (0, 9, 40.5, 58, 64):
        pairs, cnt = O.join_hamming(P, Q, d, r)
        ii, jj = np.nonzero(H <= r)
        assert as_set(pairs) == set(zip(ii.tolist(), jj.tolist())) and cnt == len(ii)
        pm_p, pm_q = (2 * pu - 1).astype(np.int8), (2 * qu - 1).astype(np.int8)
        ip_pairs, _c = O.join(pm_p, pm_q, "ip", d - 2 * math.floor(r), "i8")
        assert as_set(ip_pairs) == as_set(pairs)
    assert all((i, i) in as_set(O.join_hamming(P, Q, d, 9)[0]) for i in range(12))      # planted at distance 9
    with pytest.raises(ValueError):
        O.join_hamming(P, Q, d, -1.0)


# ------------------------------------------------------------------ LSH-bucketed join
def _splitmix64(seed, idx):
    M = (1 << 64) - 1
    z = (seed + (idx + 1) * 0x9E3779B97F4A7C15) & M
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M
    return z ^ (z >> 31)


def _lsh_coords(seed, L, k, d):
    """Bit b of repetition l samples the first of splitmix64(seed, 64 l + b + 4096 a) mod d, a = 0, 1, ..., that no
    earlier bit of the repetition took (sampling without replacement)."""
    out = []
    for l in range(L):
        row = []
        for b in range(k):
            a = 0
            while True:
                c = _splitmix64(seed, l * 64 + b + 4096 * a) % d
                if b >= d or c not in row:
                    row.append(c)
                    break
                a += 1
        out.append(row)
    return np.array(out).reshape(L, k)


def test_lsh_coordinates_are_distinct_within_a_repetition():
    for seed, L, k, d in [(2006, 8, 7, 128), (1, 64, 12, 16), (7, 5, 12, 8)]:
        c = _lsh_coords(seed, L, k, d)
        assert all(O.lsh_coordinate(seed, l, b, d) == c[l, b] for l in range(L) for b in range(k))
        assert all(len(set(c[l, :min(k, d)])) == min(k, d) for l in range(L))
        assert all(c[l, 0] == _splitmix64(seed, l * 64) % d for l in range(L))     # the first bit is the plain sample
    # the plain samples of seed 2006 repeat a coordinate in repetitions 0 and 4 (6 and 5 distinct of 7)
    plain = [[_splitmix64(2006, l * 64 + b) % 128 for b in range(7)] for l in range(8)]
    assert [len(set(r)) for r in plain] == [6, 7, 7, 7, 5, 7, 7, 7]


def test_lsh_join_is_brute_force_restricted_to_colliding_pairs():
    # independent route: python-int splitmix64 for the sampled coordinates, numpy for keys and scores
    w = W.make_workload(4, n=700, m=600, planted=80)
    L, k, seed, d = 5, 4, 1234, w.d
    coords = _lsh_coords(seed, L, k, d)
    assert all(O.lsh_coordinate(seed, l, b, d) == coords[l, b] for l in range(L) for b in range(k))
    kp = ((w.P[:, coords] > 0).astype(np.uint32) << np.arange(k, dtype=np.uint32)).sum(axis=2).T      # (L, n)
    kq = ((w.Q[:, coords] > 0).astype(np.uint32) << np.arange(k, dtype=np.uint32)).sum(axis=2).T
    assert np.array_equal(kp, O.lsh_keys(w.P, L, k, seed)) and np.array_equal(kq, O.lsh_keys(w.Q, L, k, seed))
    collide = (kp[:, :, None] == kq[:, None, :]).any(axis=0)
    S = w.P.astype(np.int64) @ w.Q.astype(np.int64).T
    for t in (100.0, 40.0, 24.0):
        ii, jj = np.nonzero(collide & (S >= t))
        pairs, cnt = O.lsh_join(w.P, w.Q, t, L, k, seed)
        assert as_set(pairs) == set(zip(ii.tolist(), jj.tolist())) and cnt == len(ii)
        exact, _c = O.join(w.P, w.Q, "ip", t, "i8")
        assert as_set(pairs) <= as_set(exact)                       # precision is 1 by construction
    # mixed tables: 3 repetitions of k bits, then 2 of k - 1 bits (the low bits of the same samples)
    kmix = np.concatenate([kp[:3], kp[3:] & ((1 << (k - 1)) - 1)]), np.concatenate([kq[:3], kq[3:] & ((1 << (k - 1)) - 1)])
    assert np.array_equal(kmix[0], O.lsh_keys(w.P, 3, k, seed, L_low=2))
    cmix = (kmix[0][:, :, None] == kmix[1][:, None, :]).any(axis=0)
    ii, jj = np.nonzero(cmix & (S >= 40.0))
    pairs, cnt = O.lsh_join(w.P, w.Q, 40.0, 3, k, seed, L_low=2)
    assert as_set(pairs) == set(zip(ii.tolist(), jj.tolist())) and cnt == len(ii)
    # no hash bits: everything collides and the LSH join is the brute-force join
    all_pairs, _c = O.lsh_join(w.P, w.Q, 40.0, 3, 0, seed)
    assert as_set(all_pairs) == as_set(O.join(w.P, w.Q, "ip", 40.0, "i8")[0])


def test_lsh_hamming_join_is_the_hamming_join_restricted_to_equal_sampled_bits():
    # independent route: keys straight from the packed bits (the sampled bit is the hash), distances by XOR + popcount
    d, L, k, seed = 128, 4, 5, 321
    Pb = W.random_bits(500, d, 41)
    Qb = W.random_bits(600, d, 42, planted_from=Pb[:60], flips=6)
    coords = _lsh_coords(seed, L, k, d)
    bp = np.unpackbits(Pb, axis=1, bitorder="little")[:, :d]
    bq = np.unpackbits(Qb, axis=1, bitorder="little")[:, :d]
    kp = (bp[:, coords].astype(np.uint32) << np.arange(k, dtype=np.uint32)).sum(axis=2).T
    kq = (bq[:, coords].astype(np.uint32) << np.arange(k, dtype=np.uint32)).sum(axis=2).T
    collide = (kp[:, :, None] == kq[:, None, :]).any(axis=0)
    H = (bp[:, None, :] != bq[None, :, :]).sum(axis=2)
    for r in (6, 40.5, 55):
        ii, jj = np.nonzero(collide & (H <= r))
        pairs, cnt = O.lsh_join_hamming(Pb, Qb, d, r, L, k, seed)
        assert as_set(pairs) == set(zip(ii.tolist(), jj.tolist())) and cnt == len(ii)
        assert as_set(pairs) <= as_set(O.join_hamming(Pb, Qb, d, r)[0])


def test_lsh_sign_keys_for_bf16_rows_and_joins_of_any_kind():
    # keys re-derived in numpy from the decoded values; the restricted join equals the int8-specific oracle where both apply
    L, k, seed, d = 4, 6, 55, 96
    X = W.random_points("bf16", 300, d, 13)
    X[0, :5] = [0x0000, 0x8000, 0x3f80, 0xbf80, 0x0001]                      # +0, -0, 1, -1, smallest subnormal
    coords = _lsh_coords(seed, L, k, d)
    vals = W.bf16_bits_to_f32(X).astype(np.float64)
    want = ((vals[:, coords] > 0).astype(np.uint32) << np.arange(k, dtype=np.uint32)).sum(axis=2).T
    assert np.array_equal(want, O.lsh_keys(X, L, k, seed, dtype="bf16"))
    w = W.make_workload(4, n=400, m=500, planted=60)
    a, ca = O.lsh_join(w.P, w.Q, 40.0, 3, 4, 9, L_low=1)
    b, cb = O.lsh_join_kind(w.P, w.Q, "ip", 40.0, "i8", 3, 4, 9, L_low=1)
    assert ca == cb and as_set(a) == as_set(b)
    # an int8 Euclidean LSH join is a subset of the brute-force one, and everything at distance 0 with equal keys is in it
    c, cc = O.lsh_join_kind(w.P, w.P, "l2", 3.0, "i8", 2, 5, 9)
    assert {(i, i) for i in range(400)} <= as_set(c) <= as_set(O.join(w.P, w.P, "l2", 3.0, "i8")[0])


def test_lsh_sign_hash_collision_probability_is_one_minus_theta_over_pi():
    # unit Gaussian rows y = cos(theta) x + sin(theta) z: every sampled sign agrees with probability 1 - theta / pi
    rng = np.random.default_rng(4)
    n, d, theta = 3000, 256, 0.5
    x = rng.standard_normal((n, d)); z = rng.standard_normal((n, d))
    y = np.cos(theta) * x + np.sin(theta) * z
    X, Y = W.f32_to_bf16_bits(x.astype(np.float32)), W.f32_to_bf16_bits(y.astype(np.float32))
    kx, ky = O.lsh_keys(X, 8, 1, 3, dtype="bf16"), O.lsh_keys(Y, 8, 1, 3, dtype="bf16")     # 8 independent single-bit keys
    agree = (kx == ky).mean()
    assert abs(agree - (1 - theta / np.pi)) < 0.01, agree


def test_lsh_recall_matches_the_collision_probability():
    # planted pairs differ in h = 8 of d = 128 coordinates: a repetition of k distinct sampled coordinates collides
    # with probability C(d-h, k) / C(d, k), so the recall over L repetitions is about 1 - (1 - that)^L
    w = W.make_workload(4, n=4000, m=4000, planted=2000)
    L, k = 4, 8
    pairs, _c = O.lsh_join(w.P, w.Q, w.threshold, L, k, 99)
    found = np.isin(O.pairs_to_set(w.planted), O.pairs_to_set(pairs)).mean()
    p1 = math.comb(128 - 8, k) / math.comb(128, k)
    expect = 1 - (1 - p1) ** L
    assert abs(found - expect) < 0.04, (found, expect)
    with pytest.raises(ValueError):
        O.lsh_join(w.P, w.Q, 1.0, 0, 4, 1)
    with pytest.raises(ValueError):
        O.lsh_join(w.P, w.Q, 1.0, 1, 0, 1, L_low=1)          # k - 1 bits needs k >= 1


# ------------------------------------------------------------------ JL transform (Section 3)
def test_jl_level_sizes_chain_up_as_the_construction_requires():
    # d = r_1 c_1,  r_i k_i = r_{i+1} c_{i+1},  r_l k_l = k  (the size equations of the lemma's proof), zeta = 2
    for d, k in [(128, 64), (256, 32), (1024, 64), (4096, 8), (512, 128)]:
        sh = O.jl_shapes(d, k)
        assert len(sh) == int(np.log2(d // k))
        assert sh[0][0] * sh[0][1] == d and sh[0][1] == 2 * k
        for (r0, _c0, k0), (r1, c1, _k1) in zip(sh, sh[1:]):
            assert r0 * k0 == r1 * c1 and r1 * 2 == r0
        assert sh[-1][0] == 1 and sh[-1][2] == k
        for i, (r, c, ki) in enumerate(sh, start=1):
            assert ki == (i * k if i < len(sh) else k) and c == (2 * k if i == 1 else 2 * (i - 1) * k)
    assert O.jl_shapes(1024, 64) == [(8, 128, 64), (4, 128, 128), (2, 256, 192), (1, 384, 64)]   # worked by hand
    for d, k in [(96, 32), (64, 64), (100, 7)]:
        with pytest.raises(ValueError):
            O.jl_shapes(d, k)


def test_jl_transform_is_the_kronecker_product_chain():
    # M = (I_{r_l} (x) A_l) ... (I_{r_1} (x) A_1) written out with numpy.kron; signs re-derived in python ints
    d, k, seed = 256, 16, 77
    sh = O.jl_shapes(d, k)
    M = np.eye(d)
    for i, (r, c, ki) in enumerate(sh, start=1):
        A = np.array([[1.0 if _splitmix64(seed, (i << 40) + a * c + b) & 1 else -1.0 for b in range(c)] for a in range(ki)])
        assert np.array_equal(A.astype(np.int8), O.jl_sign_matrix(seed, i, ki, c))
        M = np.kron(np.eye(r), A / np.sqrt(ki)) @ M
    assert M.shape == (k, d)
    X = W.random_points("bf16", 9, d, 5)
    want = W.bf16_bits_to_f32(X).astype(np.float64) @ M.T
    got = O.jl_transform(X, k, seed)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    # one level (d = 2k): a plain random-sign projection
    X2 = W.random_points("bf16", 4, 32, 6)
    A1 = O.jl_sign_matrix(3, 1, 16, 32).astype(np.float64) / 4.0
    assert np.allclose(O.jl_transform(X2, 16, 3), W.bf16_bits_to_f32(X2).astype(np.float64) @ A1.T, rtol=1e-12, atol=1e-12)


def test_jl_transform_preserves_norms_in_expectation_and_concentrates():
    # E |Mx|^2 = |x|^2 for independent sign matrices scaled by 1/sqrt(k_i); the distortion of one draw is O(1/sqrt(k))
    d, k = 512, 64
    X = W.random_points("bf16", 6, d, 11)
    n2 = (W.bf16_bits_to_f32(X).astype(np.float64) ** 2).sum(axis=1)
    ratios = np.array([(O.jl_transform(X, k, seed) ** 2).sum(axis=1) / n2 for seed in range(60)])     # (60, 6)
    assert abs(ratios.mean() - 1.0) < 0.03, ratios.mean()
    assert np.abs(np.sqrt(ratios) - 1.0).max() < 0.45
    # linear: M(2x) = 2 Mx, M(x + y) = Mx + My (inputs chosen so that the sums are exact in bf16)
    ints = np.random.default_rng(1).integers(-8, 9, size=(2, d)).astype(np.float32)
    xb, yb, sb = (W.f32_to_bf16_bits(v[None, :]) for v in (ints[0], ints[1], ints[0] + ints[1]))
    tx, ty, ts = (O.jl_transform(v, k, 5) for v in (xb, yb, sb))
    assert np.allclose(tx + ty, ts, rtol=1e-12, atol=1e-9)
    # distances between points are preserved like norms (what a join after the reduction relies on)
    Y = W.random_points("bf16", 6, d, 12)
    dist = np.linalg.norm(W.bf16_bits_to_f32(X).astype(np.float64) - W.bf16_bits_to_f32(Y).astype(np.float64), axis=1)
    dred = np.mean([np.linalg.norm(O.jl_transform(X, k, s) - O.jl_transform(Y, k, s), axis=1) / dist for s in range(30)])
    assert abs(dred - 1.0) < 0.05, dred


# ------------------------------------------------- independent formulations
def _packbits_rows(X):
    return np.packbits(X > 0, axis=1)


_POP8 = np.array([bin(v).count("1") for v in range(256)], dtype=np.int32)


def hamming_matrix(P, Q):
    """Hamming distance of +-1 rows through XOR + popcount: no multiply, no sum of products."""
    bp, bq = _packbits_rows(P), _packbits_rows(Q)
    return _POP8[bp[:, None, :] ^ bq[None, :, :]].sum(axis=2)


def test_pm1_inner_product_is_d_minus_2_hamming_cfg1_full():
    # <x,y> = d - 2*Hamming(x,y) for +-1 vectors: the Hamming ip-distance of Section 4 in disguise.
    w = W.make_workload(1)
    pairs, cnt = O.join(w.P, w.Q, "ip", w.threshold, "i8")
    want = set()
    for i0 in range(0, w.n, 256):
        ham = hamming_matrix(w.P[i0:i0 + 256], w.Q)
        ii, jj = np.nonzero(w.d - 2 * ham >= w.threshold)
        want |= set(zip((ii + i0).tolist(), jj.tolist()))
    assert as_set(pairs) == want and cnt == len(want)
    assert as_set(w.planted) <= want
    # closed-form tail: background pairs pass with p = P[Bin(64,1/2) <= 12]; expectation ~0.96
    p_bg = sum(math.comb(64, k) for k in range(13)) / 2.0 ** 64
    assert abs(p_bg * 2048 * 2048 - 0.958) < 0.01
    assert 32 <= cnt <= 32 + 8


def test_binomial_tail_closed_form_pins_count():
    # iid +-1 rows, no planted pairs: count ~ Binomial(n*m, P[Bin(d,1/2) <= (d-t)/2])
    n = m = 1024
    d, t = 64, 16
    w = W.make_workload(1, n=n, m=m, planted=0, seed=5)
    _, cnt = O.join(w.P, w.Q, "ip", t, "i8")
    p = sum(math.comb(d, k) for k in range((d - t) // 2 + 1)) / 2.0 ** d
    mean, sd = n * m * p, math.sqrt(n * m * p * (1 - p))
    assert abs(cnt - mean) < 5 * sd, (cnt, mean, sd)


@pytest.mark.parametrize("cfg,kw", [(3, dict(n=700, m=900, planted=25)), (4, dict(n=1000, m=513, planted=40))])
def test_blas_product_gives_same_integer_set(cfg, kw):
    w = W.make_workload(cfg, **kw)
    S = w.P.astype(np.float64) @ w.Q.astype(np.float64).T          # exact: all values < 2^53
    ii, jj = np.nonzero(S >= w.threshold)
    pairs, cnt = O.join(w.P, w.Q, "ip", w.threshold, "i8")
    assert as_set(pairs) == set(zip(ii.tolist(), jj.tolist())) and cnt == len(ii)
    assert as_set(w.planted) <= as_set(pairs)
    assert cnt >= kw["planted"]


def test_blas_product_outside_band_bf16():
    w = W.make_workload(2, n=600, m=500, planted=30)
    Pf, Qf = W.bf16_bits_to_f32(w.P).astype(np.float64), W.bf16_bits_to_f32(w.Q).astype(np.float64)
    C = (Pf @ Qf.T) / np.outer(np.linalg.norm(Pf, axis=1), np.linalg.norm(Qf, axis=1))
    pairs, _ = O.join(w.P, w.Q, "cos", w.threshold, "bf16")
    got = np.zeros(C.shape, dtype=bool)
    got[pairs[:, 0], pairs[:, 1]] = True
    clear = np.abs(C - w.threshold) > 1e-9
    assert np.array_equal(got[clear], (C >= w.threshold)[clear])
    assert as_set(w.planted) <= as_set(pairs)


def test_mixture_join_is_same_cluster_relation():
    w = W.make_workload(5, n=1500, m=1300, centers=40)
    pairs, cnt = O.join(w.P, w.Q, "l2", w.threshold, "bf16")
    ii, jj = np.nonzero(w.labels_p[:, None] == w.labels_q[None, :])
    assert as_set(pairs) == set(zip(ii.tolist(), jj.tolist()))
    wl = W.make_workload(5, n=1500, m=1300, centers=40, sigma_reading="percoord")
    _, cnt_lit = O.join(wl.P, wl.Q, "l2", wl.threshold, "bf16")
    assert cnt_lit == 0


# ------------------------------------------------------ exact rational brute force
def frac_rows(X, dtype):
    if dtype == "i8":
        return [[Fraction(int(v)) for v in r] for r in X]
    return [[Fraction(float(v)) for v in r] for r in W.bf16_bits_to_f32(X)]


def frac_pass(x, y, kind, t):
    s = sum(a * b for a, b in zip(x, y))
    if kind == "ip":
        return s >= t, s - t
    if kind == "l2":
        dd = sum((a - b) ** 2 for a, b in zip(x, y))
        return dd <= t * t, dd - t * t
    nx, ny = sum(a * a for a in x), sum(b * b for b in y)
    if nx == 0 or ny == 0:
        return Fraction(0) >= t, Fraction(1)
    # s/(sqrt(nx) sqrt(ny)) >= t without square roots
    lhs, rhs = s * s, t * t * nx * ny
    if t >= 0:
        return (s >= 0 and lhs >= rhs), lhs - rhs
    return (s >= 0 or lhs <= rhs), lhs - rhs


@pytest.mark.parametrize("dtype,kind", [("i8", "ip"), ("i8", "l2"), ("bf16", "ip"), ("bf16", "cos"), ("bf16", "l2")])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_exact_rational_brute_force(dtype, kind, seed):
    n, m, d = 7, 9, 5
    P = W.random_points(dtype, n, d, seed)
    Q = W.random_points(dtype, m, d, seed + 100)
    if dtype == "bf16" and seed == 2:
        P[3] = 0                                            # a zero row (bits of +0.0)
    FP, FQ = frac_rows(P, dtype), frac_rows(Q, dtype)
    thresholds = {"ip": [-2.5, 0, 1, 3.25], "cos": [-0.5, 0.0, 0.3, 0.8], "l2": [0.0, 1.5, 3.0, 4.75]}[kind]
    for t in thresholds:
        ft = Fraction(t)
        want = set()
        for i, j in itertools.product(range(n), range(m)):
            ok, margin = frac_pass(FP[i], FQ[j], kind, ft)
            if dtype == "bf16" and kind != "ip" and margin != 0 and abs(margin) < Fraction(1, 10 ** 9):
                pytest.skip("near tie: fp64 rounding may decide")
            if ok:
                want.add((i, j))
        pairs, cnt = O.join(P, Q, kind, t, dtype)
        assert as_set(pairs) == want and cnt == len(want), (kind, dtype, t)


# ------------------------------------------------ the paper's f, g embeddings
def test_hamming_embedding_identity():
    # Section 4: f(x) = (x_0, 1-x_0, ...), g(y) = (1-y_0, y_0, ...) on {0,1}^d gives Hamming(x,y);
    # on binary vectors Hamming equals the squared Euclidean distance the oracle computes.
    rng = np.random.default_rng(3)
    X = rng.integers(0, 2, size=(6, 11), dtype=np.int8)
    Y = rng.integers(0, 2, size=(5, 11), dtype=np.int8)
    f = np.stack([X, 1 - X], axis=2).reshape(len(X), -1).astype(np.int64)
    g = np.stack([1 - Y, Y], axis=2).reshape(len(Y), -1).astype(np.int64)
    allp = np.array(list(itertools.product(range(6), range(5))), dtype=np.int32)
    got = O.scores(X, Y, "l2", "i8", allp).reshape(6, 5)
    assert np.array_equal(got, f @ g.T)
    assert np.array_equal(got, (X[:, None, :] != Y[None, :, :]).sum(axis=2))


def test_squared_l2_embedding_identity():
    # Section 4 (g is misprinted there): f(x) = (x_k^2, 1, -2 x_k)_k, g(y) = (1, y_k^2, y_k)_k.
    rng = np.random.default_rng(4)
    X = rng.integers(-9, 10, size=(6, 7), dtype=np.int8)
    Y = rng.integers(-9, 10, size=(5, 7), dtype=np.int8)
    x, y = X.astype(np.int64), Y.astype(np.int64)
    f = np.stack([x * x, np.ones_like(x), -2 * x], axis=2).reshape(len(X), -1)
    g = np.stack([np.ones_like(y), y * y, y], axis=2).reshape(len(Y), -1)
    allp = np.array(list(itertools.product(range(6), range(5))), dtype=np.int32)
    assert np.array_equal(O.scores(X, Y, "l2", "i8", allp).reshape(6, 5), f @ g.T)
    # and the norm expansion the GPU path uses: ||x||^2 + ||y||^2 - 2<x,y>
    ip = O.scores(X, Y, "ip", "i8", allp).reshape(6, 5)
    nx, ny = O.sq_norms(X, "i8"), O.sq_norms(Y, "i8")
    assert np.array_equal(nx[:, None] + ny[None, :] - 2 * ip, f @ g.T)
    assert np.array_equal(nx, (x * x).sum(axis=1))


def test_cosine_embedding_identity():
    X = W.random_points("bf16", 6, 9, 11)
    Y = W.random_points("bf16", 5, 9, 12)
    xf, yf = W.bf16_bits_to_f32(X).astype(np.float64), W.bf16_bits_to_f32(Y).astype(np.float64)
    f = xf / np.sqrt((xf * xf).sum(axis=1, keepdims=True))
    g = yf / np.sqrt((yf * yf).sum(axis=1, keepdims=True))
    allp = np.array(list(itertools.product(range(6), range(5))), dtype=np.int32)
    np.testing.assert_allclose(O.scores(X, Y, "cos", "bf16", allp).reshape(6, 5), f @ g.T, rtol=0, atol=1e-14)
    np.testing.assert_allclose(O.sq_norms(X, "bf16"), (xf * xf).sum(axis=1), rtol=1e-15)
    d2 = O.scores(X, Y, "l2", "bf16", allp).reshape(6, 5) ** 2
    np.testing.assert_allclose(d2, ((xf[:, None, :] - yf[None, :, :]) ** 2).sum(axis=2), rtol=1e-14)


# ------------------------------------------------------------------ invariants
CASES = [("i8", "ip", 3, 2.0), ("i8", "l2", None, 9.5), ("bf16", "ip", None, 1.0),
         ("bf16", "cos", None, 0.2), ("bf16", "l2", None, 3.5)]


@pytest.mark.parametrize("dtype,kind,_,t", CASES)
def test_invariants(dtype, kind, _, t):
    n, m, d = 90, 70, 16
    P, Q = W.random_points(dtype, n, d, 1), W.random_points(dtype, m, d, 2)
    base, cnt = O.join(P, Q, kind, t, dtype)
    S = as_set(base)
    assert 0 < cnt < n * m, "test threshold should split the pairs"
    # join(Q, P) is the transpose
    tr, _c = O.join(Q, P, kind, t, dtype)
    assert {(j, i) for (i, j) in as_set(tr)} == S
    # self join: symmetric and (for these kinds at these thresholds) reflexive where defined
    self_pairs, _c = O.join(P, P, kind, t, dtype)
    SS = as_set(self_pairs)
    assert {(j, i) for (i, j) in SS} == SS
    if kind in ("l2", "cos"):
        assert all((i, i) in SS for i in range(n))
    # monotone in the threshold
    t_more = t + 0.5 if kind == "l2" else t - 0.5
    more, _c = O.join(P, Q, kind, t_more, dtype)
    assert S <= as_set(more)
    # extreme thresholds: everything / nothing
    big = 1e30
    everything, c_all = O.join(P, Q, kind, big if kind == "l2" else -big, dtype)
    assert c_all == n * m and everything.tolist() == [[i, j] for i in range(n) for j in range(m)]
    if kind != "l2":
        assert O.join(P, Q, kind, big, dtype)[1] == 0
    # Theorem 1's block decomposition: the union over any row/column split is the whole join
    for r_cut, c_cut in [(1, 1), (37, 64), (89, 3)]:
        U = set()
        for (r0, r1) in [(0, r_cut), (r_cut, n)]:
            for (c0, c1) in [(0, c_cut), (c_cut, m)]:
                part, _c = O.join(P[r0:r1], Q[c0:c1], kind, t, dtype)
                U |= {(i + r0, j + c0) for (i, j) in as_set(part)}
        assert U == S
    # permuting the rows of P permutes i
    perm = np.random.default_rng(9).permutation(n)
    pp, _c = O.join(P[perm], Q, kind, t, dtype)
    assert {(int(perm[i]), j) for (i, j) in as_set(pp)} == S
    # appending zero columns changes no score
    Pz = np.concatenate([P, np.zeros((n, 5), dtype=P.dtype)], axis=1)
    Qz = np.concatenate([Q, np.zeros((m, 5), dtype=Q.dtype)], axis=1)
    assert as_set(O.join(Pz, Qz, kind, t, dtype)[0]) == S
    # capacity smaller than the result: count is still the total, prefix is the sorted prefix
    few, c_few = O.join(P, Q, kind, t, dtype, capacity=5)
    assert c_few == cnt and few.tolist() == base[:5].tolist()
    # thread count does not change the result
    one, c_one = O.join(P, Q, kind, t, dtype, threads=1)
    assert c_one == cnt and np.array_equal(one, base)


def test_band_sets_are_nested():
    w = W.make_workload(2, n=300, m=300, planted=20)
    s_strict, s_exact, s_loose = O.band_sets(w.P, w.Q, "cos", 0.1, "bf16")
    assert as_set(s_strict) <= as_set(s_exact) <= as_set(s_loose)
    assert len(s_strict) < len(s_loose)
    w5 = W.make_workload(5, n=300, m=300, centers=8)
    a, b, c = O.band_sets(w5.P, w5.Q, "l2", 0.07, "bf16")
    assert as_set(a) <= as_set(b) <= as_set(c) and len(a) < len(c)


def test_empty_and_rejected_inputs():
    P = np.zeros((0, 8), dtype=np.int8)
    Q = np.ones((4, 8), dtype=np.int8)
    assert O.join(P, Q, "ip", 0, "i8")[1] == 0
    assert O.join(Q, P, "ip", 0, "i8")[1] == 0
    with pytest.raises(ValueError):
        O.join(Q, Q, "l2", -1.0, "i8")
    with pytest.raises(ValueError):
        O.join(Q, Q, "ip", float("nan"), "i8")
    assert O.join(Q, Q, "cos", 0.5, "i8")[1] == 16              # equal rows: cosine 1


def test_planted_scores_match_the_recipes():
    w1 = W.make_workload(1)
    assert np.all(O.scores(w1.P, w1.Q, "ip", "i8", w1.planted) == 64 - 2 * 4)
    w4 = W.make_workload(4, n=3000, m=2000, planted=100)
    assert np.all(O.scores(w4.P, w4.Q, "ip", "i8", w4.planted) == 128 - 2 * 8)
    w3 = W.make_workload(3, n=3000, m=2000, planted=100)
    s3 = O.scores(w3.P, w3.Q, "ip", "i8", w3.planted)
    assert s3.min() > 4000 and abs(s3.mean() - 256 * 24) < 300     # E<x,x> = d*E[x^2] = 256*24
    w2 = W.make_workload(2, n=3000, m=2000, planted=100)
    c2 = O.scores(w2.P, w2.Q, "cos", "bf16", w2.planted)
    assert c2.min() > 0.93 and abs(c2.mean() - 1 / math.sqrt(1.09)) < 5e-3


# ------------------------------------------------------------------ int8 cosine
def _cos_passes_exactly(s: int, nx: int, ny: int, t: Fraction) -> bool:
    """s / sqrt(nx * ny) >= t over the reals, decided in integers and rationals (0 for a zero vector)."""
    if nx == 0 or ny == 0:
        return 0 >= t
    if s >= 0 and t < 0:
        return True
    if s < 0 and t >= 0:
        return False
    lhs, rhs = Fraction(s * s), t * t * nx * ny
    return lhs >= rhs if s >= 0 else lhs <= rhs


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_int8_cosine_against_exact_rational_decisions(seed):
    rng = np.random.default_rng(seed)
    P = rng.integers(-127, 128, size=(23, 24)).astype(np.int8)
    Q = rng.integers(-127, 128, size=(31, 24)).astype(np.int8)
    P[5] = 0
    Q[7] = 0
    Q[9] = P[3]                                           # cosine exactly 1
    Q[10] = -P[4]                                         # cosine exactly -1 (no -128 in range)
    allp = np.array(list(itertools.product(range(len(P)), range(len(Q)))), dtype=np.int32)
    sc = O.scores(P, Q, "cos", "i8", allp)
    assert sc[3 * len(Q) + 9] == 1.0 and sc[4 * len(Q) + 10] == -1.0 and np.all(sc[5 * len(Q):6 * len(Q)] == 0.0)
    Pi, Qi = P.astype(np.int64), Q.astype(np.int64)
    for t in (0.3, 0.05, 0.0, -0.2, 1.0, -1.0, float(np.sort(sc)[-20]) + 1e-7):
        if t not in (0.0, 1.0, -1.0):
            assert np.abs(sc - t).min() > 1e-9             # away from every score: the fp64 rounding cannot matter
        tq = Fraction(t)
        want = {(i, j) for i in range(len(P)) for j in range(len(Q))
                if _cos_passes_exactly(int(Pi[i] @ Qi[j]), int(Pi[i] @ Pi[i]), int(Qi[j] @ Qi[j]), tq)}
        got, cnt = O.join(P, Q, "cos", t, "i8")
        assert cnt == len(want) and as_set(got) == want, t


def test_int8_cosine_equals_the_bf16_cosine_of_the_same_integers():
    rng = np.random.default_rng(11)
    P = rng.integers(-127, 128, size=(40, 32)).astype(np.int8)
    Q = rng.integers(-127, 128, size=(50, 32)).astype(np.int8)
    Pb, Qb = to_arr(P, "bf16"), to_arr(Q, "bf16")           # integers up to 127 are exact in bfloat16
    allp = np.array(list(itertools.product(range(len(P)), range(len(Q)))), dtype=np.int32)
    si, sb = O.scores(P, Q, "cos", "i8", allp), O.scores(Pb, Qb, "cos", "bf16", allp)
    np.testing.assert_allclose(si, sb, rtol=5e-16, atol=0)  # sqrt of the exact product vs product of two square roots
    for t in (0.25, 0.0, -0.3):
        assert np.abs(si - t).min() > 1e-9
        a, ca = O.join(P, Q, "cos", t, "i8")
        b, cb = O.join(Pb, Qb, "cos", t, "bf16")
        assert ca == cb > 0 and np.array_equal(a, b)


def test_int8_cosine_is_scale_invariant():
    rng = np.random.default_rng(12)
    P = rng.integers(-42, 43, size=(30, 16)).astype(np.int8)
    Q = rng.integers(-63, 64, size=(35, 16)).astype(np.int8)
    allp = np.array(list(itertools.product(range(len(P)), range(len(Q)))), dtype=np.int32)
    sc = O.scores(P, Q, "cos", "i8", allp)
    t = 0.2
    assert np.abs(sc - t).min() > 1e-9
    base, _ = O.join(P, Q, "cos", t, "i8")
    assert len(base) > 0
    assert np.array_equal(O.join((3 * P).astype(np.int8), (2 * Q).astype(np.int8), "cos", t, "i8")[0], base)
    assert np.array_equal(O.join(Q, P, "cos", t, "i8")[0], np.array(sorted((j, i) for i, j in base.tolist()), dtype=np.int32))


def test_int8_cosine_of_parallel_rows_is_exactly_one_even_beyond_2_to_53():
    rng = np.random.default_rng(13)
    P = rng.integers(-63, 64, size=(6, 32768)).astype(np.int8)
    P[0] = 63                                               # |x|^2 = 1.3e8, |x|^2 |2x|^2 = 6.8e16 > 2^53
    P[1] = np.where(rng.random(32768) < 0.5, 63, -63)
    Q = (2 * P).astype(np.int8)
    Q[5] = -Q[5]
    diag = np.array([[i, i] for i in range(6)], dtype=np.int32)
    sc = O.scores(P, Q, "cos", "i8", diag)
    assert np.array_equal(sc, [1, 1, 1, 1, 1, -1])
    assert int(P[0].astype(np.int64) @ P[0]) * int(Q[0].astype(np.int64) @ Q[0]) > 2 ** 53
    got, cnt = O.join(P, Q, "cos", 1.0, "i8")
    assert got.tolist() == [[i, i] for i in range(5)]


# ------------------------------------------------------------------ the pair filter
@pytest.mark.parametrize("dtype,kind,t", [("i8", "ip", 30.0), ("i8", "l2", 14.5), ("i8", "cos", 0.2),
                                          ("bf16", "ip", 2.0), ("bf16", "cos", 0.25), ("bf16", "l2", 5.0)])
def test_filter_of_every_pair_is_the_join(dtype, kind, t):
    if dtype == "i8":
        P, Q = W.random_points("i8", 37, 24, 5, lo=-4, hi=4), W.random_points("i8", 41, 24, 6, lo=-4, hi=4)
    else:
        P, Q = W.random_points("bf16", 37, 24, 5), W.random_points("bf16", 41, 24, 6)
    allp = np.array(list(itertools.product(range(len(P)), range(len(Q)))), dtype=np.int32)
    want, cnt = O.join(P, Q, kind, t, dtype)
    assert 0 < cnt < len(allp)
    assert np.array_equal(O.filter_pairs(P, Q, kind, t, dtype, allp), want)
    rng = np.random.default_rng(3)
    some = allp[rng.permutation(len(allp))[:400]]
    kept = O.filter_pairs(P, Q, kind, t, dtype, some)
    assert as_set(kept) == as_set(want) & as_set(some)
    assert [tuple(p) for p in kept.tolist()] == [tuple(p) for p in some.tolist() if tuple(p) in as_set(want)]   # order kept


# ------------------------------------------------------------------ hyperplane (sign random projection) LSH family
def _hp_signs(seed, L, k, d):
    """(L, k, d) array of +-1: coordinate c of the hyperplane of repetition l, bit b -- Python integers."""
    return np.array([[[1 if _splitmix64(seed, (1 << 60) + ((l * 64 + b) << 20) + c) & 1 else -1 for c in range(d)]
                      for b in range(k)] for l in range(L)], dtype=np.int64)


def test_lsh_hyperplane_keys_golden(golden_dir):
    g = json.load(open(os.path.join(golden_dir, "lsh_hyperplane_d8.json")))
    X = np.array(g["points"], dtype=np.int8)
    keys = O.lsh_keys(X, g["L"], g["k"], g["seed"], L_low=g["L_low"], family="hyperplanes")
    assert keys.tolist() == g["keys"]
    planes = np.array(g["hyperplanes"])
    assert all(O.hp_sign(g["seed"], l, b, c) == planes[l, b, c] for l in range(3) for b in range(3) for c in range(8))
    # the same integer points as bf16 rows (exact in bf16) hash alike, and none of their projections is in doubt except 0
    Xb = W.f32_to_bf16_bits(X.astype(np.float32))
    kb, unsure = O.lsh_keys_unsure(Xb, g["L"], g["k"], g["seed"], L_low=g["L_low"])
    assert kb.tolist() == g["keys"]
    proj = g["projections"]
    for l in range(3):
        for i in range(len(X)):
            zero_bits = sum(1 << b for b, v in enumerate(proj[l][i]) if v == 0)
            assert unsure[l, i] == zero_bits


def test_lsh_hyperplane_keys_against_python_int_signs_and_numpy_products():
    seed, L, L_low, k, d = 77, 3, 2, 5, 48
    R = _hp_signs(seed, L + L_low, k, d)
    X = W.random_points("i8", 300, d, 5, lo=-128, hi=127)
    proj = np.einsum("lbc,ic->lib", R, X.astype(np.int64))                      # exact integers
    want = ((proj > 0).astype(np.uint32) << np.arange(k, dtype=np.uint32)).sum(axis=2).astype(np.uint32)
    want[L:] &= (1 << (k - 1)) - 1                                             # L_low tables: the same planes without the last
    assert np.array_equal(want, O.lsh_keys(X, L, k, seed, L_low=L_low, family="hyperplanes"))
    # bf16 rows: fp64 products of the widened values; bits agree wherever the projection is not in doubt
    Xb = W.random_points("bf16", 300, d, 6)
    projf = np.einsum("lbc,ic->lib", R.astype(np.float64), W.bf16_bits_to_f32(Xb).astype(np.float64))
    wantb = ((projf > 0).astype(np.uint32) << np.arange(k, dtype=np.uint32)).sum(axis=2).astype(np.uint32)
    wantb[L:] &= (1 << (k - 1)) - 1
    kb, unsure = O.lsh_keys_unsure(Xb, L, k, seed, L_low=L_low)
    assert np.array_equal(wantb & ~unsure, kb & ~unsure) and (unsure != 0).mean() < 0.01
    assert np.array_equal(kb, O.lsh_keys(Xb, L, k, seed, L_low=L_low, dtype="bf16", family="hyperplanes"))


def test_lsh_hyperplane_key_symmetries():
    seed, L, k, d = 5, 4, 6, 64
    X = W.random_points("i8", 200, d, 9, lo=-60, hi=60)
    keys = O.lsh_keys(X, L, k, seed, family="hyperplanes")
    assert np.array_equal(keys, O.lsh_keys((2 * X).astype(np.int8), L, k, seed, family="hyperplanes"))          # scale invariant
    R = _hp_signs(seed, L, k, d)
    nonzero = (np.einsum("lbc,ic->lib", R, X.astype(np.int64)) != 0).all(axis=2)       # (L, rows)
    flipped = O.lsh_keys((-X).astype(np.int8), L, k, seed, family="hyperplanes")
    assert np.array_equal(flipped[nonzero], (~keys & ((1 << k) - 1))[nonzero])           # -x lies on the other side of every plane
    assert not O.lsh_keys(np.zeros((3, d), np.int8), L, k, seed, family="hyperplanes").any()                   # sign(0) := bit 0
    # permuting the rows permutes the keys; a different seed gives different planes
    perm = np.random.default_rng(0).permutation(len(X))
    assert np.array_equal(keys[:, perm], O.lsh_keys(X[perm], L, k, seed, family="hyperplanes"))
    assert not np.array_equal(keys, O.lsh_keys(X, L, k, seed + 1, family="hyperplanes"))


def test_lsh_hyperplane_collision_law_holds_on_anisotropic_data_where_coordinate_signs_fail():
    """Pairs at a known angle theta collide on a hyperplane bit with probability 1 - theta / pi whatever the shape of
    the data; the sampled-coordinate sign only has that law for rotation-invariant data.  Data: 16 of 128 coordinates
    are five times larger than the rest and carry all of the difference between the two points of a pair, so the
    angle is set by coordinates that a sampled-coordinate hash rarely looks at."""
    rng = np.random.default_rng(21)
    d, npairs, big = 128, 400, 16
    scale = np.ones(d)
    scale[:big] = 5.0
    base = rng.standard_normal((npairs, d)) * scale
    other = base.copy()
    other[:, :big] += 0.8 * 5.0 * rng.standard_normal((npairs, big))
    X, Y = W.f32_to_bf16_bits(base.astype(np.float32)), W.f32_to_bf16_bits(other.astype(np.float32))
    xf, yf = W.bf16_bits_to_f32(X).astype(np.float64), W.bf16_bits_to_f32(Y).astype(np.float64)
    cos = (xf * yf).sum(axis=1) / np.sqrt((xf * xf).sum(axis=1) * (yf * yf).sum(axis=1))
    expect = float(np.mean(1.0 - np.arccos(np.clip(cos, -1, 1)) / np.pi))           # about 0.81
    L = 64
    kx, ky = (O.lsh_keys(Z, L, 1, 3, dtype="bf16", family="hyperplanes") for Z in (X, Y))      # 64 single-bit keys
    agree_hp = float((kx == ky).mean())
    assert abs(agree_hp - expect) < 0.01, (agree_hp, expect)                        # 25 600 bits: sigma = 0.0025
    bx, by = (O.lsh_keys(Z, L, 1, 3, dtype="bf16", family="bits") for Z in (X, Y))
    agree_bits = float((bx == by).mean())
    assert agree_bits > expect + 0.1, (agree_bits, expect)      # seven sampled coordinates in eight are equal in x and y


def test_lsh_hyperplane_join_is_the_join_restricted_to_colliding_pairs():
    w = W.make_workload(3, n=500, m=400, planted=60)
    L, k, seed = 4, 5, 11
    pairs, cnt = O.lsh_join_kind(w.P, w.Q, "ip", w.threshold, "i8", L, k, seed, family="hyperplanes")
    R = _hp_signs(seed, L, k, w.d)
    kp = ((np.einsum("lbc,ic->lib", R, w.P.astype(np.int64)) > 0) << np.arange(k)).sum(axis=2)
    kq = ((np.einsum("lbc,ic->lib", R, w.Q.astype(np.int64)) > 0) << np.arange(k)).sum(axis=2)
    full, _c = O.join(w.P, w.Q, "ip", w.threshold, "i8")
    keep = (kp[:, full[:, 0]] == kq[:, full[:, 1]]).any(axis=0)
    assert cnt == int(keep.sum()) and np.array_equal(pairs, full[keep]) and 0 < cnt
    everything, c0 = O.lsh_join_kind(w.P, w.Q, "ip", w.threshold, "i8", 1, 0, seed, family="hyperplanes")          # k = 0: one bucket
    assert c0 == len(full)
    # bf16: the strict / loose collision sets bracket the plain one
    wb = W.make_workload(2, n=400, m=300, planted=80)
    s, e, lo = O.lsh_band_sets(wb.P, wb.Q, "cos", wb.threshold, "bf16", 6, 4, 5, family="hyperplanes")
    ks, ke, kl = (O.pairs_to_set(z) for z in (s, e, lo))
    assert np.isin(ks, kl).all() and len(ke) > 0 and len(kl) >= len(ks)


def test_lsh_iid_bit_sampling_is_the_plain_concatenation_of_independent_samples():
    """family "bits_iid": bit b of repetition l reads coordinate splitmix64(seed, 64 l + b) mod d whether or not an earlier
    bit took it -- the paper's concatenation of k independent base hashes, whose collision probability for a pair at
    Hamming distance h is exactly (1 - h/d)^k."""
    seed, L, k, d = 2006, 8, 7, 128
    coords = np.array([[_splitmix64(seed, l * 64 + b) % d for b in range(k)] for l in range(L)])
    assert [len(set(r)) for r in coords.tolist()] == [6, 7, 7, 7, 5, 7, 7, 7]       # repetitions 0 and 4 repeat a coordinate
    X = W.random_points("i8", 500, d, 3, lo=-1, hi=1)
    want = ((X[:, coords] > 0).astype(np.uint32) << np.arange(k, dtype=np.uint32)).sum(axis=2).T
    got = O.lsh_keys(X, L, k, seed, family="bits_iid")
    assert np.array_equal(want, got)
    assert not np.array_equal(got, O.lsh_keys(X, L, k, seed))                        # the distinct-coordinate family differs there
    assert np.array_equal(O.lsh_keys(X, L, k, seed), O.lsh_keys(X, L, k, seed, family="bits"))      # and the default is unchanged
    # collision law on +-1 rows at Hamming distance h: 64 repetitions x 3000 pairs
    rng = np.random.default_rng(4)
    h, kk, reps = 16, 5, 64
    A = (rng.integers(0, 2, size=(3000, d), dtype=np.int8) * 2 - 1).astype(np.int8)
    Bm = A.copy()
    flip = np.argsort(rng.random((3000, d)), axis=1)[:, :h]
    Bm[np.repeat(np.arange(3000), h), flip.ravel()] *= -1
    ka, kb = O.lsh_keys(A, reps, kk, 9, family="bits_iid"), O.lsh_keys(Bm, reps, kk, 9, family="bits_iid")
    assert abs((ka == kb).mean() - (1 - h / d) ** kk) < 0.004                        # 0.5129; sigma = 0.0011
    kd, ke = O.lsh_keys(A, reps, kk, 9), O.lsh_keys(Bm, reps, kk, 9)
    hyper = math.comb(d - h, kk) / math.comb(d, kk)                                 # distinct coordinates: hypergeometric, 0.5090
    assert abs((kd == ke).mean() - hyper) < 0.004
    # the join of the family is the join restricted to its collisions
    w = W.make_workload(4, n=600, m=500, planted=100)
    pairs, cnt = O.lsh_join_kind(w.P, w.Q, "ip", 40.0, "i8", 3, 6, seed, family="bits_iid")
    full, _c = O.join(w.P, w.Q, "ip", 40.0, "i8")
    cp = np.array([[_splitmix64(seed, l * 64 + b) % w.d for b in range(6)] for l in range(3)])
    kp = ((w.P[:, cp] > 0).astype(np.uint32) << np.arange(6, dtype=np.uint32)).sum(axis=2).T
    kq = ((w.Q[:, cp] > 0).astype(np.uint32) << np.arange(6, dtype=np.uint32)).sum(axis=2).T
    keep = (kp[:, full[:, 0]] == kq[:, full[:, 1]]).any(axis=0)
    assert np.array_equal(pairs, full[keep]) and cnt == int(keep.sum()) > 0
