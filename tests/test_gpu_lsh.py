"""LSH-bucketed inner-product join (Section 4, second algorithm) through the C ABI: hashing, regrouping,
work list and bucketed tile join all on the device.  The result is a set fixed by (L, k, seed), so it is
compared with the oracle pair by pair; no pair may be reported twice."""
import numpy as np
import pytest
import torch

from oracle import simjoin_oracle as O
from paper_2006_12608_b200 import binding as B
from paper_2006_12608_b200 import build
from paper_2006_12608_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = B.Simjoin("i8", 0)
    yield c
    c.close()


def keys(p):
    p = np.asarray(p, dtype=np.int64).reshape(-1, 2)
    return np.sort((p[:, 0] << 32) | p[:, 1])


def gpu_lsh(ctx, P, Q, t, L, k, seed, cap=1 << 21, expect=B.SIMJOIN_OK, L_low=0):
    dP, dQ = torch.from_numpy(P).cuda(), torch.from_numpy(Q).cuda()
    out = torch.full((cap + 2, 2), -5, dtype=torch.int32, device="cuda:0")
    st, cnt = ctx.simjoin_run_lsh(dP, P.shape[0], dQ, Q.shape[0], P.shape[1], t, L, k, seed, out, cap, L_low=L_low)
    assert st == expect, B.strerror(st)
    host = out.cpu().numpy()
    assert np.all(host[min(cnt, cap):] == -5)
    return host[:min(cnt, cap)], cnt


def check(ctx, P, Q, t, L, k, seed, L_low=0):
    pairs, cnt = gpu_lsh(ctx, P, Q, t, L, k, seed, L_low=L_low)
    want, wcnt = O.lsh_join(P, Q, t, L, k, seed, L_low=L_low)
    got = keys(pairs)
    assert len(np.unique(got)) == len(got), "a pair was reported twice"
    assert cnt == wcnt and np.array_equal(got, keys(want)), (P.shape, Q.shape, t, L, k, cnt, wcnt)
    return cnt


@pytest.mark.parametrize("n,m,L,k", [(700, 600, 5, 4), (1, 1, 1, 0), (129, 257, 3, 1), (5000, 7000, 4, 3),
                                      (3000, 2500, 2, 12), (20000, 30000, 6, 5)])
def test_lsh_join_matches_oracle(ctx, n, m, L, k):
    w = W.make_workload(4, n=n, m=m, planted=min(n, m, 300))
    total = 0
    for t in (w.threshold, 40.0, 26.0 if n * m < 10**8 else 34.0):
        total += check(ctx, w.P, w.Q, t, L, k, 1234 + k)
    assert total > 0 or min(n, m) == 1


@pytest.mark.parametrize("L,L_low,k", [(3, 2, 4), (0, 4, 3), (2, 3, 1), (1, 1, 12)])
def test_lsh_mixed_tables(ctx, L, L_low, k):
    # the paper's remedy for a fractional number of base hashes: L tables of k bits, L_low of k - 1
    w = W.make_workload(4, n=4000, m=5000, planted=300)
    for t in (w.threshold, 36.0):
        assert check(ctx, w.P, w.Q, t, L, k, 77, L_low=L_low) > 0


def test_lsh_dense_output(ctx):
    # every colliding pair passes: blocks with more hits than the staging buffer holds take the direct
    # output path, which must drop the pairs of earlier tables too
    w = W.make_workload(4, n=900, m=1100, planted=50)
    assert check(ctx, w.P, w.Q, -1000.0, 4, 2, 31) > 400000
    assert check(ctx, w.P, w.Q, 4.0, 5, 3, 32) > 50000


def test_no_hash_bits_is_the_brute_force_join(ctx):
    w = W.make_workload(4, n=3000, m=4100, planted=200)
    pairs, cnt = gpu_lsh(ctx, w.P, w.Q, 30.0, 3, 0, 7)
    want, wcnt = O.join(w.P, w.Q, "ip", 30.0, "i8")
    assert cnt == wcnt and np.array_equal(keys(pairs), keys(want))


@pytest.mark.parametrize("d", [64, 256, 384, 1024])
def test_lsh_row_lengths(ctx, d):
    # 64: partial chunk; 256: two-chunk fast path; 384: three chunks; 1024: streamed P
    P = W.random_points("i8", 2100, d, 11, lo=-1, hi=1)
    Q = W.random_points("i8", 2600, d, 12, lo=-1, hi=1)
    Q[:100] = P[:100]
    check(ctx, P, Q, 0.25 * d, 4, 3, 99)


def test_lsh_wide_values_use_the_32_bit_epilogue(ctx):
    P = W.random_points("i8", 1500, 128, 21, lo=-127, hi=127)
    Q = W.random_points("i8", 1700, 128, 22, lo=-127, hi=127)
    Q[:64] = P[:64]
    assert check(ctx, P, Q, 150000.0, 4, 4, 5) >= 1


def test_lsh_recall_on_planted_pairs(ctx):
    # planted pairs differ in 8 of 128 coordinates; 8 repetitions of 6 bits miss one with probability ~1e-4
    w = W.make_workload(4, n=40000, m=40000, planted=4000)
    pairs, cnt = gpu_lsh(ctx, w.P, w.Q, w.threshold, 8, 6, 3)
    found = np.isin(keys(w.planted), keys(pairs)).mean()
    assert found > 0.995, found
    exact, _ = O.join(w.P, w.Q, "ip", w.threshold, "i8")
    assert np.isin(keys(pairs), keys(exact)).all()


def test_lsh_offsets_capacity_and_errors(ctx):
    w = W.make_workload(4, n=2000, m=2000, planted=300)
    dP, dQ = torch.from_numpy(w.P).cuda(), torch.from_numpy(w.Q).cuda()
    want, wcnt = O.lsh_join(w.P, w.Q, w.threshold, 4, 3, 17)
    assert wcnt > 50
    assert ctx.simjoin_set_offsets(1000, 50000) == B.SIMJOIN_OK
    try:
        pairs, cnt = gpu_lsh(ctx, w.P, w.Q, w.threshold, 4, 3, 17)
    finally:
        ctx.simjoin_set_offsets(0, 0)
    assert np.array_equal(keys(pairs), keys(want + np.array([1000, 50000])))
    # too small an output list: the count is still the full one, only `capacity` pairs are written
    pairs, cnt = gpu_lsh(ctx, w.P, w.Q, w.threshold, 4, 3, 17, cap=20, expect=B.SIMJOIN_ERR_CAPACITY)
    assert cnt == wcnt and np.isin(keys(pairs), keys(want)).all() and len(pairs) == 20
    out = torch.zeros((8, 2), dtype=torch.int32, device="cuda:0")
    args = (dP, 2000, dQ, 2000, 128, 100.0)
    assert ctx.simjoin_run_lsh(*args, 0, 3, 1, out, 8)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_run_lsh(*args, 65, 3, 1, out, 8)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_run_lsh(*args, 2, -1, 1, out, 8)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_run_lsh(*args, 2, 13, 1, out, 8)[0] == B.SIMJOIN_ERR_UNSUPPORTED
    assert ctx.simjoin_run_lsh(*args, 2, 0, 1, out, 8, L_low=1)[0] == B.SIMJOIN_ERR_ARG          # k - 1 bits needs k >= 1
    assert ctx.simjoin_run_lsh(*args, 60, 3, 1, out, 8, L_low=5)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_run_lsh(dP, 0, dQ, 2000, 128, 100.0, 2, 3, 1, out, 8) == (B.SIMJOIN_OK, 0)
    # the plain join still works on the same context afterwards
    got, cnt = ctx.join(dP, dQ, "ip", w.threshold, 1 << 16)
    assert cnt == O.join(w.P, w.Q, "ip", w.threshold, "i8")[1]


@pytest.mark.parametrize("n,m,d,L,k", [(700, 900, 128, 4, 3), (3000, 2600, 256, 6, 5), (1200, 800, 1024, 3, 2)])
def test_lsh_hamming_join_on_packed_bits(ctx, n, m, d, L, k):
    """simjoin_run_hamming_lsh: bits -> +-1 operand transform, then the LSH-bucketed join; the sampled bit is the hash."""
    Pb = W.random_bits(n, d, 51)
    Qb = W.random_bits(m, d, 52, planted_from=Pb[: min(n, m, 200)], flips=d // 16)
    dP, dQ = torch.from_numpy(Pb).cuda(), torch.from_numpy(Qb).cuda()
    for r in (d // 16, 0.43 * d):
        out = torch.full((1 << 20, 2), -5, dtype=torch.int32, device="cuda:0")
        st, cnt = ctx.simjoin_run_hamming_lsh(dP, n, dQ, m, d, r, L, k, 77, out, 1 << 20, L_low=1)
        assert st == B.SIMJOIN_OK, B.strerror(st)
        want, wcnt = O.lsh_join_hamming(Pb, Qb, d, r, L, k, 77, L_low=1)
        got = keys(out[:cnt].cpu().numpy())
        assert cnt == wcnt and len(np.unique(got)) == cnt and np.array_equal(got, keys(want)), (n, m, d, r, cnt, wcnt)
        assert cnt > 0
    assert ctx.simjoin_run_hamming_lsh(dP, n, dQ, m, d, -1.0, L, k, 1, out, 8)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_run_hamming_lsh(dP, n, dQ, m, d, 3.0, 0, k, 1, out, 8)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_run_hamming_lsh(dP, n, dQ, m, d + 64, 3.0, L, k, 1, out, 8)[0] == B.SIMJOIN_ERR_UNSUPPORTED


# ------------------------------------------------------------------ every kind and element type
@pytest.fixture(scope="module")
def ctx_bf16():
    build.build()
    c = B.Simjoin("bf16", 0)
    yield c
    c.close()


@pytest.mark.parametrize("d,L,k", [(128, 4, 3), (64, 3, 2), (256, 3, 4), (528, 2, 2)])
def test_lsh_int8_euclidean_join(ctx, d, L, k):
    """int8 rows, L2 kind: row norms and per-tile bounds are taken on the regrouped rows; exact pair set."""
    P = W.random_points("i8", 1500 + 9, d, 61, lo=-2, hi=2)
    Q = W.random_points("i8", 1900 + 5, d, 62, lo=-2, hi=2)
    Q[7:600:3] = P[:198]
    Q[8:600:3] = np.clip(P[200:398].astype(np.int16) + W.random_points("i8", 198, d, 63, lo=0, hi=1), -128, 127).astype(np.int8)
    for r in (0.0, (0.3 * d) ** 0.5, (2.2 * d) ** 0.5):
        dP, dQ = torch.from_numpy(P).cuda(), torch.from_numpy(Q).cuda()
        out = torch.full((1 << 21, 2), -5, dtype=torch.int32, device="cuda:0")
        st, cnt = ctx.simjoin_run_lsh(dP, len(P), dQ, len(Q), d, r, L, k, 19, out, 1 << 21, L_low=1, kind="l2")
        assert st == B.SIMJOIN_OK, B.strerror(st)
        want, wcnt = O.lsh_join_kind(P, Q, "l2", r, "i8", L, k, 19, L_low=1)
        got = keys(out[:cnt].cpu().numpy())
        assert cnt == wcnt and len(np.unique(got)) == cnt and np.array_equal(got, keys(want)), (d, r, cnt, wcnt)
        assert cnt >= 100


@pytest.mark.parametrize("d,L,k,hi", [(128, 4, 3, 2), (64, 3, 2, 127), (256, 3, 4, 127), (528, 2, 2, 40)])
def test_lsh_int8_cosine_join(ctx, d, L, k, hi):
    """int8 rows, cosine: the fp32 filter's candidates are decided exactly on the regrouped rows; exact pair set."""
    P = W.random_points("i8", 1500 + 9, d, 71, lo=-hi, hi=hi)
    Q = W.random_points("i8", 1900 + 5, d, 72, lo=-hi, hi=hi)
    Q[7:600:3] = P[:198]
    Q[8:600:3] = np.clip(P[200:398].astype(np.int16) + W.random_points("i8", 198, d, 73, lo=-1, hi=1), -127, 127).astype(np.int8)
    P[1400] = 0
    Q[1700] = 0
    for t in (1.0, 0.8, 0.0):
        dP, dQ = torch.from_numpy(P).cuda(), torch.from_numpy(Q).cuda()
        out = torch.full((1 << 22, 2), -5, dtype=torch.int32, device="cuda:0")
        st, cnt = ctx.simjoin_run_lsh(dP, len(P), dQ, len(Q), d, t, L, k, 23, out, 1 << 22, L_low=1, kind="cos")
        assert st == B.SIMJOIN_OK, B.strerror(st)
        want, wcnt = O.lsh_join_kind(P, Q, "cos", t, "i8", L, k, 23, L_low=1)
        got = out[:cnt].cpu().numpy()
        assert cnt == wcnt > 0 and np.array_equal(np.sort(keys(got)), np.sort(keys(want)))
        assert np.all(out[cnt:].cpu().numpy() == -5)


@pytest.mark.parametrize("kind", ["ip", "cos", "l2"])
@pytest.mark.parametrize("d,L,k", [(128, 4, 3), (64, 3, 5), (264, 3, 2)])
def test_lsh_bf16_sign_hash_join(ctx_bf16, kind, d, L, k):
    """bf16 rows, the sign of a sampled coordinate as the hash: within the threshold band of the oracle's sets
    restricted to colliding pairs; nothing twice."""
    w = W.make_workload(2, n=1800 + 11, m=2100 + 3, d=d, planted=300)
    t = {"ip": 0.85, "cos": 0.85, "l2": 0.55}[kind]
    dP, dQ = B.to_device(w.P), B.to_device(w.Q)
    out = torch.full((1 << 20, 2), -5, dtype=torch.int32, device="cuda:0")
    st, cnt = ctx_bf16.simjoin_run_lsh(dP, w.n, dQ, w.m, d, t, L, k, 23, out, 1 << 20, L_low=1, kind=kind)
    assert st == B.SIMJOIN_OK, B.strerror(st)
    got = keys(out[:cnt].cpu().numpy())
    assert len(np.unique(got)) == cnt
    strict, exact, loose = O.lsh_band_sets(w.P, w.Q, kind, t, "bf16", L, k, 23, L_low=1)
    assert np.isin(keys(strict), got).all() and np.isin(got, keys(loose)).all(), (kind, d, cnt, len(strict), len(loose))
    assert len(strict) >= 50                                            # planted pairs that collide
    # recall against the brute-force join: a planted pair at angle theta survives a k-bit table with (1 - theta/pi)^k
    full = O.join(w.P, w.Q, kind, t, "bf16")[0]
    assert len(exact) <= len(full) and len(exact) > 0.3 * len(full)


@pytest.mark.parametrize("kind", ["ip", "cos"])
@pytest.mark.parametrize("d,L,k", [(64, 3, 2), (128, 2, 1), (520, 2, 1)])
def test_lsh_bf16_thresholds_near_zero_are_decided_from_the_rows(ctx_bf16, kind, d, L, k):
    """The bucketed join of bf16 points at inner-product / cosine thresholds with an empty tolerance band (zero, next to
    zero, the exact score of a colliding pair): candidates are decided from the regrouped rows in fp64, so the result is
    the oracle's exact set restricted to colliding pairs, bit for bit (the sampled-sign keys are exact)."""
    rng = np.random.default_rng(d + L)
    n, m = 900, 1100
    P = W.f32_to_bf16_bits(rng.standard_normal((n, d)).astype(np.float32))
    Q = W.f32_to_bf16_bits(rng.standard_normal((m, d)).astype(np.float32))
    P[2] = 0
    Q[3] = 0
    dP, dQ = B.to_device(P), B.to_device(Q)
    cap = n * m + 8
    out = torch.full((cap, 2), -5, dtype=torch.int32, device="cuda:0")
    coll = O.lsh_join_kind(P, Q, kind, float("-inf"), "bf16", L, k, 29)[0]        # every colliding pair
    sc = O.scores(P, Q, kind, "bf16", coll)
    near = [float(sc[i]) for i in np.argsort(np.abs(sc)) if sc[i] != 0.0][:5]
    for t in [0.0, 1e-30, -1e-30] + near:
        st, cnt = ctx_bf16.simjoin_run_lsh(dP, n, dQ, m, d, t, L, k, 29, out, cap, kind=kind)
        assert st == B.SIMJOIN_OK, B.strerror(st)
        got = keys(out[:cnt].cpu().numpy())
        want = keys(O.lsh_join_kind(P, Q, kind, t, "bf16", L, k, 29)[0])
        assert len(np.unique(got)) == cnt
        assert np.array_equal(np.sort(got), np.sort(want)), (kind, d, t, cnt, len(want))


def test_lsh_more_key_bits_than_coordinates(ctx_bf16, ctx):
    """k > d: the first d bits take every coordinate once, the later ones sample as they come.  8-coordinate bf16
    rows (16 bytes) with 12 key bits, and 16-coordinate int8 rows with 12 of 16 coordinates taken."""
    rng = np.random.default_rng(8)
    Pb = W.f32_to_bf16_bits(rng.standard_normal((900, 8)).astype(np.float32))
    Qb = W.f32_to_bf16_bits(rng.standard_normal((1100, 8)).astype(np.float32))
    Qb[:300] = Pb[:300]
    out = torch.full((1 << 20, 2), -5, dtype=torch.int32, device="cuda:0")
    st, cnt = ctx_bf16.simjoin_run_lsh(B.to_device(Pb), 900, B.to_device(Qb), 1100, 8, 0.5, 3, 12, 7, out, 1 << 20, L_low=2, kind="l2")
    assert st == B.SIMJOIN_OK, B.strerror(st)
    got = keys(out[:cnt].cpu().numpy())
    strict, exact, loose = O.lsh_band_sets(Pb, Qb, "l2", 0.5, "bf16", 3, 12, 7, L_low=2)
    assert len(np.unique(got)) == cnt and np.isin(keys(strict), got).all() and np.isin(got, keys(loose)).all()
    assert len(strict) >= 300
    Pi = W.random_points("i8", 700, 16, 97, lo=-1, hi=1)
    Qi = W.random_points("i8", 800, 16, 98, lo=-1, hi=1)
    Qi[:200] = Pi[:200]
    assert check(ctx, Pi, Qi, 6.0, 4, 12, 3) >= 200



# ------------------------------------------------------------------ the random-hyperplane family (keys on the tensor cores)
def run_family(ctx, P, Q, kind, t, L, k, seed, L_low=0, cap=1 << 21, family="hyperplanes"):
    dP, dQ = B.to_device(P), B.to_device(Q)
    out = torch.full((cap + 2, 2), -5, dtype=torch.int32, device="cuda:0")
    st, cnt = ctx.simjoin_run_lsh(dP, P.shape[0], dQ, Q.shape[0], P.shape[1], t, L, k, seed, out, cap, L_low=L_low, kind=kind, family=family)
    assert st == B.SIMJOIN_OK, B.strerror(st)
    host = out.cpu().numpy()
    assert np.all(host[cnt:] == -5)
    got = keys(host[:cnt])
    assert len(np.unique(got)) == cnt, "a pair was reported twice"
    return got


@pytest.mark.parametrize("kind", ["ip", "cos", "l2"])
@pytest.mark.parametrize("n,m,d,L,L_low,k,hi", [(700, 600, 128, 5, 0, 4, 1), (129, 257, 64, 3, 2, 1, 3), (5000, 7000, 144, 4, 1, 6, 127),
                                               (3000, 2500, 16, 2, 0, 12, 5), (900, 1100, 640, 17, 0, 3, 3), (600, 500, 2064, 3, 1, 5, 127),
                                               (1500, 1800, 256, 33, 2, 2, 2)])
def test_hyperplane_lsh_join_int8_is_exact(ctx, kind, n, m, d, L, L_low, k, hi):
    """int8 projections are exact integers, so the keys -- and with them the result -- equal the oracle's bit for bit:
    one and several key words per record (L + L_low up to 35: three P tiles of hyperplanes), partial chunks, rows that
    stream both operands, values up to +-127 (projections up to 2^18)."""
    P, Q = W.random_points("i8", n, d, 201, lo=-hi, hi=hi), W.random_points("i8", m, d, 202, lo=-hi, hi=hi)
    kp = min(n, m, 200) // 2
    Q[:kp] = P[:kp]
    Q[kp:2 * kp:2] = -P[kp:2 * kp:2]                      # opposite points: every bit differs
    P[7] = 0                                              # projections of exactly zero hash to bit 0
    smp = np.stack([np.arange(kp), np.arange(kp)], axis=1).astype(np.int32)
    sc = O.scores(P, Q, kind, "i8", smp).astype(np.float64)
    t = {"ip": float(np.quantile(sc, 0.3)), "cos": 0.95, "l2": 0.5}[kind]
    got = run_family(ctx, P, Q, kind, t, L, k, 4242 + k, L_low=L_low)
    want, wcnt = O.lsh_join_kind(P, Q, kind, t, "i8", L, k, 4242 + k, L_low=L_low, family="hyperplanes")
    assert len(got) == wcnt and np.array_equal(got, keys(want)) and wcnt > 0


@pytest.mark.parametrize("kind", ["ip", "cos", "l2"])
@pytest.mark.parametrize("d,L,k", [(128, 4, 3), (64, 3, 5), (264, 3, 2), (1040, 2, 4)])
def test_hyperplane_lsh_join_bf16_within_the_band(ctx_bf16, kind, d, L, k):
    """bf16: the threshold band of the join, and a band on the hash as well -- a projection too close to zero for fp32
    accumulation to decide may put the point on either side, so the result lies between the strict and the loose
    collision sets of the oracle."""
    w = W.make_workload(2, n=1800 + 11, m=2100 + 3, d=d, planted=300)
    t = {"ip": 0.85, "cos": 0.85, "l2": 0.55}[kind]
    got = run_family(ctx_bf16, w.P, w.Q, kind, t, L, k, 23, L_low=1)
    strict, exact, loose = O.lsh_band_sets(w.P, w.Q, kind, t, "bf16", L, k, 23, L_low=1, family="hyperplanes")
    assert np.isin(keys(strict), got).all() and np.isin(got, keys(loose)).all(), (kind, d, len(got), len(strict), len(loose))
    assert len(strict) >= 50 and len(loose) - len(strict) <= max(3, len(loose) // 50)


def test_hyperplane_lsh_recall_on_anisotropic_data_beats_coordinate_signs(ctx_bf16):
    """16 of 128 coordinates are five times larger than the rest and carry the difference inside a near pair, as in the
    oracle's collision-law pin: sampled-coordinate signs see mostly the 112 small, equal coordinates, so near and
    far-but-equal-on-the-small-coordinates pairs collide alike; hyperplanes follow the angle."""
    rng = np.random.default_rng(5)
    n, d, big = 4000, 128, 16
    scale = np.ones(d, dtype=np.float32)
    scale[:big] = 5.0
    Pf = rng.standard_normal((n, d)).astype(np.float32) * scale
    Qf = rng.standard_normal((n, d)).astype(np.float32) * scale
    Qf[:400] = Pf[:400]
    Qf[:400, :big] += 0.25 * 5.0 * rng.standard_normal((400, big)).astype(np.float32)        # near pairs, cosine about 0.97
    P, Q = W.f32_to_bf16_bits(Pf), W.f32_to_bf16_bits(Qf)
    t = 0.93
    full = keys(O.join(P, Q, "cos", t, "bf16")[0])
    assert 380 <= len(full) <= 420
    L, k = 6, 8
    hp = run_family(ctx_bf16, P, Q, "cos", t, L, k, 9)
    recall_hp = np.isin(full, hp).mean()
    want = 1.0 - (1.0 - (1.0 - np.arccos(0.97) / np.pi) ** k) ** L
    assert abs(recall_hp - want) < 0.08, (recall_hp, want)


def test_hyperplane_lsh_argument_checks(ctx):
    X = B.to_device(W.random_points("i8", 64, 64, 1))
    out = torch.zeros((8, 2), dtype=torch.int32, device="cuda:0")
    assert ctx.simjoin_run_lsh(X, 64, X, 64, 64, 10.0, 2, 3, 1, out, 8, family=7)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_run_lsh(X, 64, X, 64, 64, 10.0, 2, 13, 1, out, 8, family="hyperplanes")[0] == B.SIMJOIN_ERR_UNSUPPORTED
    assert ctx.simjoin_run_lsh(X, 0, X, 64, 64, 10.0, 2, 3, 1, out, 8, family="hyperplanes") == (B.SIMJOIN_OK, 0)


@pytest.mark.parametrize("kind", ["ip", "l2"])
def test_iid_bit_sampling_family_matches_the_oracle(ctx, kind):
    """SIMJOIN_LSH_BITS_IID: the k bits of a repetition are independent samples.  With seed 2006 two of eight 7-bit repetitions
    repeat a coordinate (half the buckets there), which the distinct-coordinate family avoids; both are exact on int8 rows."""
    w = W.make_workload(4, n=5000, m=6000, planted=400)
    t = {"ip": 40.0, "l2": 9.5}[kind]
    got = run_family(ctx, w.P, w.Q, kind, t, 8, 7, 2006, L_low=1, family="bits_iid")
    want, wcnt = O.lsh_join_kind(w.P, w.Q, kind, t, "i8", 8, 7, 2006, L_low=1, family="bits_iid")
    assert len(got) == wcnt > 0 and np.array_equal(got, keys(want))
    if kind == "ip":      # enough pairs of middling score that the two families' collisions differ
        assert not np.array_equal(got, run_family(ctx, w.P, w.Q, kind, t, 8, 7, 2006, L_low=1, family="bits"))
