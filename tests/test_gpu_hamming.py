"""Hamming join on bit-packed points (the first ip-distance of Section 4) through the C ABI:
bits -> +-1 int8 operand transform on the device, then the int8 inner-product join.  Exact."""
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


def gpu_hamming(ctx, P, Q, d, r, cap=1 << 21):
    dP, dQ = torch.from_numpy(P).cuda(), torch.from_numpy(Q).cuda()
    out = torch.full((cap + 2, 2), -5, dtype=torch.int32, device="cuda:0")
    st, cnt = ctx.simjoin_run_hamming(dP, P.shape[0], dQ, Q.shape[0], d, r, out, cap)
    assert st == B.SIMJOIN_OK, B.strerror(st)
    host = out.cpu().numpy()
    assert np.all(host[cnt:] == -5)
    return host[:cnt], cnt


@pytest.mark.parametrize("n,m,d", [(1, 1, 128), (129, 257, 128), (700, 1500, 256), (300, 4100, 384), (1030, 520, 1024)])
def test_hamming_join_is_exact(ctx, n, m, d):
    P = W.random_bits(n, d, 5)
    Q = W.random_bits(m, d, 6, planted_from=P[: min(n, m, 40)], flips=d // 16)
    for r in (0, d // 16, d // 16 + 0.99, 0.42 * d, d):
        pairs, cnt = gpu_hamming(ctx, P, Q, d, r)
        want, wcnt = O.join_hamming(P, Q, d, r)
        assert cnt == wcnt and np.array_equal(keys(pairs), keys(want)), (n, m, d, r)
    k = min(n, m, 40)
    planted = keys(np.stack([np.arange(k), np.arange(k)], axis=1))
    pairs, _ = gpu_hamming(ctx, P, Q, d, d // 16)
    assert np.isin(planted, keys(pairs)).all()


def test_hamming_argument_errors(ctx):
    P = torch.zeros((64, 16), dtype=torch.uint8, device="cuda:0")
    out = torch.zeros((8, 2), dtype=torch.int32, device="cuda:0")
    assert ctx.simjoin_run_hamming(P, 64, P, 64, 128, -1.0, out, 8)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_run_hamming(P, 64, P, 64, 128, float("nan"), out, 8)[0] == B.SIMJOIN_ERR_ARG
    assert ctx.simjoin_run_hamming(P, 64, P, 64, 64, 3.0, out, 8)[0] == B.SIMJOIN_ERR_UNSUPPORTED       # d % 128
    assert ctx.simjoin_run_hamming(P.cpu().numpy(), 64, P, 64, 128, 3.0, out, 8)[0] == B.SIMJOIN_ERR_ARG  # host pointer
    assert ctx.simjoin_run_hamming(P, 0, P, 64, 128, 3.0, out, 8) == (B.SIMJOIN_OK, 0)
    with B.Simjoin("bf16", 0) as cb:
        assert cb.simjoin_run_hamming(P, 64, P, 64, 128, 3.0, out, 8)[0] == B.SIMJOIN_ERR_UNSUPPORTED
    st, cnt = ctx.simjoin_run_hamming(P, 64, P, 64, 128, 0.0, out, 8)        # all rows identical: 64*64 pairs
    assert (st, cnt) == (B.SIMJOIN_ERR_CAPACITY, 64 * 64)
