"""Randomised parity: a few hundred seeded cases over element type, kind, brute force / LSH, row length (all three tile
geometries, partial chunks), ragged row counts and value ranges, each compared with the oracle (int8: the exact pair set;
bf16: inside the threshold band); half of the cases also run the pair filter on a random candidate list.  Thresholds are
taken from a sample of the oracle's scores so that every case has hits; bf16 Euclidean radii go down to whatever the
sample's low tail gives, including radii far below the rows' norms (small point sets, where the sample meets the planted
equal rows), which the join decides from the rows in the difference form.  bf16 points are small integers (exact sums) or
Gaussian (inexact ones); a fifth of the inner-product and cosine cases take a threshold at or next to zero -- or equal to a
sampled pair's exact score -- where the band is empty and the join decides its candidates from the rows in fp64."""
import numpy as np
import pytest
import torch

from oracle import simjoin_oracle as O
from paper_2006_12608_b200 import binding as B
from paper_2006_12608_b200 import build
from paper_2006_12608_b200 import workloads as W

pytestmark = pytest.mark.gpu
ROW_BYTES = [16, 32, 48, 64, 96, 128, 128, 144, 256, 256, 272, 384, 400, 512, 528, 640, 1024, 1040, 2048, 2064, 4096]


def keys(p):
    p = np.asarray(p, dtype=np.int64).reshape(-1, 2)
    return np.sort((p[:, 0] << 32) | p[:, 1])


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_cases_match_the_oracle(seed):
    build.build()
    rng = np.random.default_rng(seed)
    ctxs = {"i8": B.Simjoin("i8", 0), "bf16": B.Simjoin("bf16", 0)}
    cap = 1 << 21
    out = torch.empty((cap + 2, 2), dtype=torch.int32, device="cuda:0")
    try:
        for case in range(130):
            dtype = "i8" if rng.random() < 0.5 else "bf16"
            kind = str(rng.choice(["ip", "cos", "l2"]))
            d = int(rng.choice(ROW_BYTES)) // (1 if dtype == "i8" else 2)
            n = int(rng.integers(1, 1200)) if rng.random() < 0.7 else int(rng.integers(1200, 40 * 256))
            m = int(rng.integers(1, 3000))
            if n * m * d > 2e9:
                n = max(1, int(2e9 / (m * d)))
            # thresholds at or next to zero (inner product, cosine): half of all pairs pass, and the tolerance band is empty
            near_zero = kind != "l2" and rng.random() < 0.2
            if near_zero:
                n, m = min(n, 1000), min(m, 2000)
            lsh = rng.random() < 0.35
            s1, s2 = int(rng.integers(1 << 30)), int(rng.integers(1 << 30))
            small_ints = False
            if dtype == "i8":
                hi = int(rng.choice([1, 2, 5, 127]))
                P, Q = W.random_points("i8", n, d, s1, lo=-hi, hi=hi), W.random_points("i8", m, d, s2, lo=-hi, hi=hi)
            elif rng.random() < 0.6:
                P, Q = W.random_points("bf16", n, d, s1), W.random_points("bf16", m, d, s2)
                small_ints = True
            else:   # Gaussian coordinates: sums that fp32 does not hold exactly
                g = np.random.default_rng(s1)
                P = W.f32_to_bf16_bits(g.standard_normal((n, d)).astype(np.float32) * float(rng.choice([1e-3, 1.0, 50.0])))
                Q = W.f32_to_bf16_bits(g.standard_normal((m, d)).astype(np.float32) * float(rng.choice([1e-3, 1.0, 50.0])))
            kpl = min(n, m, 64)
            Q[:kpl] = P[:kpl]                                   # equal rows: hits under every kind
            smp = np.stack([rng.integers(0, n, 2000), rng.integers(0, m, 2000)], axis=1).astype(np.int32)
            sc = O.scores(P, Q, kind, dtype, smp).astype(np.float64)
            if kind == "l2":
                dist = np.sqrt(np.maximum(sc, 0.0)) if dtype == "i8" else sc
                t = float(np.quantile(dist, 0.002))
                if dtype == "bf16" and small_ints and rng.random() < 0.25:
                    t = float(rng.choice([0.0, 1e-3, 0.05, 0.3]))   # radii far below the norms: equal and near-equal rows only
            else:
                t = float(np.quantile(sc, 0.998))
            if near_zero:
                nz = sc[sc != 0.0]
                t = float(rng.choice([0.0, -0.0, 1e-30, -1e-30, float(nz[np.argmin(np.abs(nz))]) if len(nz) else 0.0]))
            ctx = ctxs[dtype]
            if dtype == "i8":     # small joins: the device's choice of the epilogue width, or the 32-bit one unasked
                assert ctx.simjoin_set_option(B.SIMJOIN_OPT_SELECT_MIN_OPS, 0.0 if rng.random() < 0.7 else 2e11) == B.SIMJOIN_OK
            else:                 # 8 or 16 epilogue warps (where both exist), or by the previous call's density
                assert ctx.simjoin_set_option(B.SIMJOIN_OPT_DENSE_EPILOGUE, float(rng.integers(0, 3))) == B.SIMJOIN_OK
            dP, dQ = B.to_device(P), B.to_device(Q)
            out.fill_(-5)
            L = k = L_low = 0
            family = "bits"
            if lsh:
                L, k = int(rng.integers(1, 5)), int(rng.integers(0, 6))
                L_low = int(rng.integers(0, 2)) if k >= 1 else 0
                family = str(rng.choice(["bits", "bits", "hyperplanes", "hyperplanes", "bits_iid"]))
                st, cnt = ctx.simjoin_run_lsh(dP, n, dQ, m, d, t, L, k, s1, out, cap, L_low=L_low, kind=kind, family=family)
            else:
                st, cnt = ctx.simjoin_run(dP, n, dQ, m, d, kind, t, out, cap)
            what = dict(case=case, dtype=dtype, kind=kind, n=n, m=m, d=d, t=t, lsh=(L, k, L_low, family) if lsh else None, s1=s1, s2=s2)
            assert st == B.SIMJOIN_OK, (B.strerror(st), what)
            host = out.cpu().numpy()
            got = keys(host[:cnt])
            assert np.all(host[cnt:] == -5) and len(np.unique(got)) == cnt, what
            if dtype == "i8":
                want = O.lsh_join_kind(P, Q, kind, t, dtype, L, k, s1, L_low=L_low, family=family)[0] if lsh else O.join(P, Q, kind, t, dtype)[0]
                assert np.array_equal(got, keys(want)), what
            else:
                sets = O.lsh_band_sets(P, Q, kind, t, dtype, L, k, s1, L_low=L_low, family=family) if lsh else O.band_sets(P, Q, kind, t, dtype)
                assert np.isin(keys(sets[0]), got).all() and np.isin(got, keys(sets[2])).all(), what
            # the pair filter on a random candidate list of the same points (plus some reported pairs)
            if rng.random() < 0.5:
                nc = int(rng.integers(1, 2000))
                cand = np.stack([rng.integers(0, n, nc), rng.integers(0, m, nc)], axis=1).astype(np.int32)
                cand = np.concatenate([cand, host[:min(cnt, 300)]])
                lst = torch.from_numpy(np.ascontiguousarray(cand)).cuda()
                st2, kc = ctx.simjoin_filter_pairs(dP, n, dQ, m, d, kind, t, lst, len(cand))
                assert st2 == B.SIMJOIN_OK, (B.strerror(st2), what)
                kept = keys(lst[:kc].cpu().numpy())
                if dtype == "i8":
                    assert np.array_equal(kept, keys(O.filter_pairs(P, Q, kind, t, dtype, cand))), what
                else:
                    t_loose, t_strict = (t * 1.01, t * 0.99) if kind == "l2" else (t - 0.01 * abs(t), t + 0.01 * abs(t))
                    assert np.isin(keys(O.filter_pairs(P, Q, kind, t_strict, dtype, cand)), kept).all(), what
                    assert np.isin(kept, keys(O.filter_pairs(P, Q, kind, t_loose, dtype, cand))).all(), what
    finally:
        for c in ctxs.values():
            c.close()
