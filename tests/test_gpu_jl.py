"""JL transform (Section 3) through the C ABI: every level is one launch of the tile kernel with the level's
random-sign matrix resident and the points' blocks streamed.  Compared with the fp64 oracle element by element.

Tolerance.  The products are exact and accumulate in fp32; what differs from fp64 is that each level's output is
rounded to bf16 (relative error <= 2^-9 per element) before it feeds the next level.  A level maps an error
vector e to A_i e / sqrt(k_i), whose entries are at most |e|_1 / sqrt(k_i) <= 2^-9 |z|_2 sqrt(c_i / k_i), with z
the level's input block and |z|_2 <= 1.5 |x|_2 for every block met here (JL distortion).  Summed over the levels
and with the final rounding this bounds every output entry's error by
    2^-9 * |x|_2 * (1.5 * sum_i sqrt(c_i / k_i) + 1).
The root-mean-square error is far smaller (errors are independent), about sqrt(l) * 2^-9 * rms(y) / sqrt(3);
the test allows 4x that, which any structural mistake (a wrong sign, block or scale) exceeds by orders of magnitude.
"""
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
    c = B.Simjoin("bf16", 0)
    yield c
    c.close()


def gpu_jl(ctx, X, k, seed):
    n, d = X.shape
    dX = B.to_device(X)
    out = torch.full((n + 1, k), 7.0, dtype=torch.bfloat16, device="cuda:0")
    st = ctx.simjoin_jl_transform(dX, n, d, k, seed, out)
    assert st == B.SIMJOIN_OK, B.strerror(st)
    host = out.float().cpu().numpy().astype(np.float64)
    assert np.all(host[n:] == 7.0)                       # nothing written past the n rows
    return host[:n]


@pytest.mark.parametrize("n,d,k", [(1000, 128, 64), (777, 256, 32), (3000, 1024, 64), (513, 512, 128), (300, 2048, 8),
                                    (40000, 256, 64), (1, 64, 8), (260, 1024, 256)])
def test_jl_transform_matches_oracle(ctx, n, d, k):
    X = W.random_points("bf16", n, d, 40 + k, scale=1.0)
    got = gpu_jl(ctx, X, k, 99)
    want = O.jl_transform(X, k, 99)
    sh = O.jl_shapes(d, k)
    xn = np.linalg.norm(W.bf16_bits_to_f32(X).astype(np.float64), axis=1)
    bound = 2.0 ** -9 * xn * (1.5 * sum(np.sqrt(c / ki) for _r, c, ki in sh) + 1.0)
    err = np.abs(got - want)
    assert np.all(err <= bound[:, None]), (err.max(), bound.min())
    rms_err, rms_y = np.sqrt((err ** 2).mean()), np.sqrt((want ** 2).mean())
    assert rms_err <= 4.0 * np.sqrt(len(sh)) * 2.0 ** -9 * rms_y / np.sqrt(3.0), (rms_err, rms_y)


def test_one_level_on_small_integers_is_exact(ctx):
    # d = 2k, k = 64: every output is (a sum of 128 values in {-1, 0, 1}) / 8 -- exactly representable in bf16
    X = W.f32_to_bf16_bits(np.random.default_rng(3).integers(-1, 2, size=(900, 128)).astype(np.float32))
    assert np.array_equal(gpu_jl(ctx, X, 64, 5), O.jl_transform(X, 64, 5))


def test_jl_preserves_norms_and_distances_on_the_device(ctx):
    w = W.make_workload(2, n=4000, m=4000, planted=500)          # unit rows, planted near pairs
    d, k = w.d, 64
    P, Q = gpu_jl(ctx, w.P, k, 8), gpu_jl(ctx, w.Q, k, 8)       # the same M for both sets
    ratio = np.linalg.norm(P, axis=1)                            # |x| = 1
    assert abs(ratio.mean() - 1.0) < 0.03 and np.abs(ratio - 1.0).max() < 0.5
    Pf, Qf = W.bf16_bits_to_f32(w.P).astype(np.float64), W.bf16_bits_to_f32(w.Q).astype(np.float64)
    i, j = w.planted[:, 0], w.planted[:, 1]
    near = np.linalg.norm(P[i] - Q[j], axis=1) / np.linalg.norm(Pf[i] - Qf[j], axis=1)
    far = np.linalg.norm(P[i] - Q[j[::-1]], axis=1) / np.linalg.norm(Pf[i] - Qf[j[::-1]], axis=1)
    assert abs(near.mean() - 1.0) < 0.05 and abs(far.mean() - 1.0) < 0.05
    # the reduced points keep the near pairs joinable: an L2 join on them finds the planted pairs
    rnear = np.linalg.norm(Pf[i] - Qf[j], axis=1).max()
    dP, dQ = torch.from_numpy(P).cuda().to(torch.bfloat16), torch.from_numpy(Q).cuda().to(torch.bfloat16)
    pairs, cnt = ctx.join(dP, dQ, "l2", 1.5 * rnear, 1 << 20)
    got = pairs.cpu().numpy().astype(np.int64)
    keys = (got[:, 0] << 32) | got[:, 1]
    assert np.isin((i << 32) | j, keys).mean() > 0.99


def test_jl_argument_errors(ctx):
    X = torch.zeros((64, 256), dtype=torch.bfloat16, device="cuda:0")
    out = torch.zeros((64, 256), dtype=torch.bfloat16, device="cuda:0")
    assert ctx.simjoin_jl_transform(X, 64, 256, 96, 1, out) == B.SIMJOIN_ERR_ARG          # d % k
    assert ctx.simjoin_jl_transform(X, 64, 256, 256, 1, out) == B.SIMJOIN_ERR_ARG         # no level
    assert ctx.simjoin_jl_transform(X, 64, 192, 64, 1, out) == B.SIMJOIN_ERR_ARG          # d / k = 3
    assert ctx.simjoin_jl_transform(X, 64, 256, 4, 1, out) == B.SIMJOIN_ERR_UNSUPPORTED   # k % 8
    assert ctx.simjoin_jl_transform(X, -1, 256, 64, 1, out) == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_jl_transform(X.cpu().float().numpy(), 64, 256, 64, 1, out) == B.SIMJOIN_ERR_ARG   # host pointer
    assert ctx.simjoin_jl_transform(X, 0, 256, 64, 1, out) == B.SIMJOIN_OK
    with B.Simjoin("i8", 0) as ci:
        assert ci.simjoin_jl_transform(X, 64, 256, 64, 1, out) == B.SIMJOIN_ERR_UNSUPPORTED


def test_binding_conveniences(ctx):
    X = B.to_device(W.random_points("bf16", 500, 256, 3))
    Y = ctx.jl_transform(X, 32, 9)
    assert Y.shape == (500, 32) and Y.dtype == torch.bfloat16
    want = O.jl_transform(W.random_points("bf16", 500, 256, 3), 32, 9)
    assert np.abs(Y.float().cpu().numpy() - want).max() < 0.05 * np.abs(want).max()
    with pytest.raises(B.SimjoinError):
        ctx.jl_transform(X, 96, 9)
    w = W.make_workload(4, n=1500, m=1200, planted=100)
    with B.Simjoin("i8", 0) as ci:
        pairs, cnt = ci.join_lsh(B.to_device(w.P), B.to_device(w.Q), w.threshold, 4, 3, 5, 1 << 16)
        want_pairs, wcnt = O.lsh_join(w.P, w.Q, w.threshold, 4, 3, 5)
        got = pairs.cpu().numpy().astype(np.int64)
        assert cnt == wcnt and set(map(tuple, got)) == set(map(tuple, want_pairs.astype(np.int64)))
