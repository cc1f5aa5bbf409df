"""Parity of the CUDA join (through the C ABI) with the CPU oracle, element by element.

int8 joins must equal the oracle's sorted pair set bit for bit.  bf16 joins must lie
between the oracle's strict and loose band sets (scores within 1e-2*|t| of the
threshold may fall on either side); in-band disagreements are reported."""
import os

import numpy as np
import pytest
import torch

from oracle import simjoin_oracle as O
from paper_2006_12608_b200 import binding as B
from paper_2006_12608_b200 import build
from paper_2006_12608_b200 import workloads as W

pytestmark = pytest.mark.gpu
BAND_REL = 1e-2      # the band half-width relative to |threshold| (the stated tolerance)


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    B.load()


@pytest.fixture(scope="module")
def ctx_i8():
    """An int8 context that asks the device for the epilogue width on every join, however small, so that the small
    shapes below reach the max|x| pre-pass, the device-side choice and both epilogues (the default skips them on
    joins this small: test_small_int8_joins_skip_the_epilogue_choice)."""
    c = B.Simjoin("i8", 0)
    assert c.simjoin_set_option(B.SIMJOIN_OPT_SELECT_MIN_OPS, 0.0) == B.SIMJOIN_OK
    yield c
    c.close()


@pytest.fixture(scope="module")
def ctx_bf16():
    c = B.Simjoin("bf16", 0)
    yield c
    c.close()


def gpu_join(ctx, P, Q, kind, t, capacity=None):
    dP, dQ = B.to_device(P), B.to_device(Q)
    cap = 1 << 16 if capacity is None else capacity
    while True:
        out = torch.full((max(cap, 1) + 4, 2), -7, dtype=torch.int32, device="cuda:0")   # 4 canary rows
        st, cnt = ctx.simjoin_run(dP, P.shape[0], dQ, Q.shape[0], P.shape[1], kind, t, out if cap else None, cap)
        assert st in (B.SIMJOIN_OK, B.SIMJOIN_ERR_CAPACITY), B.strerror(st)
        assert (st == B.SIMJOIN_ERR_CAPACITY) == (cnt > cap)
        host = out.cpu().numpy()
        assert np.all(host[cap:] == -7), "wrote past capacity"
        wrote = min(cnt, cap)
        assert np.all(host[wrote:cap] == -7), "wrote more rows than min(count, capacity)"
        if capacity is not None or cnt <= cap:
            return host[:wrote], cnt
        cap = cnt


def keys(pairs):
    p = np.asarray(pairs, dtype=np.int64).reshape(-1, 2)
    return (p[:, 0] << 32) | p[:, 1]


def assert_exact(gpu_pairs, cnt, P, Q, kind, t, dtype="i8"):
    want, wcnt = O.join(P, Q, kind, t, dtype)
    assert cnt == wcnt
    g = np.sort(keys(gpu_pairs))
    assert len(np.unique(g)) == len(g), "duplicate pairs"
    assert np.array_equal(g, keys(want))            # oracle output is already sorted by (i, j)


def assert_band(gpu_pairs, cnt, P, Q, kind, t):
    s_strict, s_exact, s_loose = O.band_sets(P, Q, kind, t, "bf16", rel=BAND_REL)
    g = np.sort(keys(gpu_pairs))
    assert len(g) == cnt and len(np.unique(g)) == len(g), "duplicate pairs"
    assert np.isin(keys(s_strict), g).all(), "missing a pair that is clearly inside the threshold"
    assert np.isin(g, keys(s_loose)).all(), "emitted a pair that is clearly outside the threshold"
    disagreements = len(np.setxor1d(g, keys(s_exact)))
    in_band = len(s_loose) - len(s_strict)
    print(f"[band] kind={kind} t={t}: |GPU|={len(g)} |exact|={len(s_exact)} in-band={in_band} disagreements={disagreements}")
    return disagreements, in_band


# ------------------------------------------------------------------ configuration 1, full size
def test_cfg1_full_bit_exact(ctx_i8):
    w = W.make_workload(1)
    pairs, cnt = gpu_join(ctx_i8, w.P, w.Q, "ip", w.threshold)
    assert_exact(pairs, cnt, w.P, w.Q, "ip", w.threshold)
    assert np.isin(keys(w.planted), keys(pairs)).all()


# ------------------------------------------------------------------ shapes: ragged tails, K chunks
I8_SHAPES = [(1, 1, 16), (5, 3, 16), (128, 256, 128), (129, 257, 128), (300, 700, 64), (1000, 513, 144),
             (257, 1030, 256), (77, 300, 384), (200, 260, 512), (130, 520, 640), (140, 300, 1024), (64, 64, 8192)]


@pytest.mark.parametrize("n,m,d", I8_SHAPES)
def test_i8_ip_shapes(ctx_i8, n, m, d):
    P, Q = W.random_points("i8", n, d, 1), W.random_points("i8", m, d, 2)
    sd = (d * (28.0 / 7.0) ** 2) ** 0.5        # std of <x,y> for iid uniform{-3..3}: var(x)=4
    for t in (2.0 * sd, 0.5 * sd + 0.5):
        pairs, cnt = gpu_join(ctx_i8, P, Q, "ip", t)
        assert_exact(pairs, cnt, P, Q, "ip", t)


@pytest.mark.parametrize("n,m,d", [(5, 3, 16), (129, 257, 128), (300, 700, 64), (257, 1030, 256), (140, 300, 1024)])
def test_i8_l2_shapes(ctx_i8, n, m, d):
    P, Q = W.random_points("i8", n, d, 3), W.random_points("i8", m, d, 4)
    mean = (8.0 * d) ** 0.5                     # E|x-y|^2 = 2*var*d = 8d
    for r in (0.93 * mean, 0.8 * mean, float(int(mean))):
        pairs, cnt = gpu_join(ctx_i8, P, Q, "l2", r)
        assert_exact(pairs, cnt, P, Q, "l2", r)


BF_SHAPES = [(1, 1, 8), (5, 3, 8), (128, 256, 64), (129, 257, 64), (300, 700, 128), (513, 1000, 72),
             (257, 1030, 256), (140, 300, 512), (64, 64, 4096)]


@pytest.mark.parametrize("kind", ["ip", "cos", "l2"])
@pytest.mark.parametrize("n,m,d", BF_SHAPES)
def test_bf16_shapes(ctx_bf16, kind, n, m, d):
    P, Q = W.random_points("bf16", n, d, 5), W.random_points("bf16", m, d, 6)
    t = {"ip": 1.5 * d ** 0.5, "cos": 1.5 / d ** 0.5, "l2": (2 * d) ** 0.5 - 1.2}[kind]
    pairs, cnt = gpu_join(ctx_bf16, P, Q, kind, t)
    assert_band(pairs, cnt, P, Q, kind, t)


def test_bf16_negative_threshold_and_zero_rows(ctx_bf16):
    P, Q = W.random_points("bf16", 200, 32, 7), W.random_points("bf16", 300, 32, 8)
    P[17] = 0
    Q[5] = 0
    Q[299] = 0
    for t in (-0.2, 0.0, 0.25):
        pairs, cnt = gpu_join(ctx_bf16, P, Q, "cos", t)
        assert_band(pairs, cnt, P, Q, "cos", t) if t != 0.0 else None
        want, _c = O.join(P, Q, "cos", t, "bf16")
        zero_rows = {(i, j) for (i, j) in map(tuple, want.tolist()) if i == 17 or j in (5, 299)}
        got = set(map(tuple, pairs.tolist()))
        assert {(i, j) for (i, j) in got if i == 17 or j in (5, 299)} == zero_rows   # cosine with 0 counts as 0
    pairs, cnt = gpu_join(ctx_bf16, P, Q, "ip", -1.0)
    assert_band(pairs, cnt, P, Q, "ip", -1.0)


def test_bf16_inner_product_threshold_zero_counts_scores_of_either_zero(ctx_bf16):
    """t = 0: a pair whose score is exactly zero passes, whichever zero the accumulator holds (a zero row against a row
    of negative values sums products that are all -0)."""
    P = W.f32_to_bf16_bits(np.zeros((40, 64), dtype=np.float32))
    Q = W.f32_to_bf16_bits(-np.abs(np.random.default_rng(4).standard_normal((70, 64))).astype(np.float32) - 0.5)
    P[1::2] = W.f32_to_bf16_bits(np.ones((20, 64), dtype=np.float32))          # odd rows: score < 0 against every Q row
    for t in (0.0, -0.0):
        pairs, cnt = gpu_join(ctx_bf16, P, Q, "ip", t)
        want, wcnt = O.join(P, Q, "ip", t, "bf16")
        assert cnt == wcnt == 20 * 70
        assert set(map(tuple, pairs.tolist())) == set(map(tuple, want.tolist()))


def test_bf16_cosine_zero_vectors_and_scores_of_either_zero(ctx_bf16):
    """Cosine with a zero vector counts as 0: it passes t <= 0 and fails t > 0, also when the accumulator holds -0
    (a zero row against rows of negative values) and next to rows and columns that do pass."""
    rng = np.random.default_rng(6)
    P = W.random_points("bf16", 70, 64, 91)
    Q = W.f32_to_bf16_bits(-np.abs(rng.standard_normal((90, 64))).astype(np.float32) - 0.25)      # all negative
    P[::7] = 0
    Q[5] = 0
    Q[40:44] = 0
    Q[60] = P[3]
    for t in (0.0, -0.0, -0.3, 1e-3, 0.4, 1e-42):
        pairs, cnt = gpu_join(ctx_bf16, P, Q, "cos", t)
        want, wcnt = O.join(P, Q, "cos", t, "bf16")
        zero = lambda s: {(i, j) for (i, j) in s if i % 7 == 0 or j in (5, 40, 41, 42, 43)}
        got = set(map(tuple, pairs.tolist()))
        assert zero(got) == zero(set(map(tuple, want.tolist()))), t
        if t not in (0.0, -0.0, 1e-42):
            assert_band(pairs, cnt, P, Q, "cos", t)


def test_i8_packed_16_bit_epilogue_boundary(ctx_i8):
    """int8 scores that provably fit in 16 bits take a packed epilogue; check both sides of that
    decision and scores at the very ends of the 16-bit range."""
    d = 16
    for amp, narrow in ((45, True), (46, False), (127, False)):     # d*amp*amp = 32400 / 33856 / 258064
        P = W.random_points("i8", 300, d, 31, lo=-amp, hi=amp)
        Q = W.random_points("i8", 520, d, 32, lo=-amp, hi=amp)
        P[7] = amp
        Q[11] = amp                  # score +d*amp^2
        Q[12] = -amp                 # score -d*amp^2
        if amp == 127:
            P[8] = -128
            Q[13] = -128             # score d*128*128 = 262144
        top = d * amp * amp
        for kind, t in (("ip", top), ("ip", top - 1.5), ("ip", 0.6 * top), ("ip", -top), ("ip", -top + 0.5),
                        ("l2", 0.0), ("l2", 0.35 * (2 * top) ** 0.5), ("l2", 2.0 * (top ** 0.5) * 2)):
            pairs, cnt = gpu_join(ctx_i8, P, Q, kind, t)
            assert_exact(pairs, cnt, P, Q, kind, t)
        assert (d * amp * amp <= 32767) == narrow


def test_small_int8_joins_skip_the_epilogue_choice():
    """The default context takes the 32-bit epilogue unasked on small joins (two launches less) and the device's
    choice from SIMJOIN_OPT_SELECT_MIN_OPS operations on; the pair set is the oracle's either way, also when calls
    of both sorts alternate on one context (they share the two control blocks)."""
    P, Q = W.random_points("i8", 900, 64, 33, lo=-3, hi=3), W.random_points("i8", 1300, 64, 34, lo=-3, hi=3)
    with B.Simjoin("i8", 0) as ctx:
        assert ctx.simjoin_set_option(99, 1.0) == B.SIMJOIN_ERR_ARG
        assert ctx.simjoin_set_option(B.SIMJOIN_OPT_SELECT_MIN_OPS, -1.0) == B.SIMJOIN_ERR_ARG
        for min_ops in (None, 0.0, 1e18, 0.0, 2e11):
            if min_ops is not None:
                assert ctx.simjoin_set_option(B.SIMJOIN_OPT_SELECT_MIN_OPS, min_ops) == B.SIMJOIN_OK
            for kind, t in (("ip", 30.0), ("l2", 19.0), ("cos", 0.4)):
                pairs, cnt = gpu_join(ctx, P, Q, kind, t)
                assert_exact(pairs, cnt, P, Q, kind, t)
                assert cnt > 0


def test_staged_compaction_flush_paths(ctx_i8, ctx_bf16):
    """Several tiles per CTA with ~100 hits per 32x128 warp block: the per-warp staging buffer
    (256 pairs) fills and is flushed mid-kernel, not only at the end; a lower threshold then sends
    blocks with more hits than the buffer holds straight to global memory."""
    P, Q = W.random_points("i8", 2048, 64, 51), W.random_points("i8", 8192 + 37, 64, 52)
    sd = (64 * 16.0) ** 0.5
    for t in (2.0 * sd, 1.2 * sd, 0.2 * sd):
        pairs, cnt = gpu_join(ctx_i8, P, Q, "ip", t, capacity=1 << 23)
        assert_exact(pairs, cnt, P, Q, "ip", t)
    Pb, Qb = W.random_points("bf16", 1100, 32, 53), W.random_points("bf16", 4096 + 5, 32, 54)
    pairs, cnt = gpu_join(ctx_bf16, Pb, Qb, "l2", 6.5, capacity=1 << 22)
    assert_band(pairs, cnt, Pb, Qb, "l2", 6.5)


# ------------------------------------------------------------------ degenerate thresholds and sizes
def test_everything_and_nothing(ctx_i8, ctx_bf16):
    P, Q = W.random_points("i8", 200, 64, 9), W.random_points("i8", 300, 64, 10)
    pairs, cnt = gpu_join(ctx_i8, P, Q, "ip", -1e30)
    assert cnt == 200 * 300 and np.array_equal(np.sort(keys(pairs)), keys([[i, j] for i in range(200) for j in range(300)]))
    assert gpu_join(ctx_i8, P, Q, "ip", 1e30)[1] == 0
    assert gpu_join(ctx_i8, P, Q, "ip", float("inf"))[1] == 0
    assert gpu_join(ctx_i8, P, Q, "ip", float("-inf"))[1] == 200 * 300
    assert gpu_join(ctx_i8, P, Q, "l2", 1e9)[1] == 200 * 300
    pairs, cnt = gpu_join(ctx_i8, P, P, "l2", 0.0)                     # only identical rows
    assert_exact(pairs, cnt, P, P, "l2", 0.0)
    assert cnt >= 200
    Pb, Qb = W.random_points("bf16", 150, 64, 11), W.random_points("bf16", 260, 64, 12)
    assert gpu_join(ctx_bf16, Pb, Qb, "l2", 1e18)[1] == 150 * 260
    assert gpu_join(ctx_bf16, Pb, Qb, "cos", -1.5)[1] == 150 * 260
    assert gpu_join(ctx_bf16, Pb, Qb, "cos", 1.5)[1] == 0
    assert gpu_join(ctx_bf16, Pb, Qb, "ip", float("inf"))[1] == 0


def test_self_join_is_symmetric_with_diagonal(ctx_i8):
    w = W.make_workload(3, n=700, m=700, planted=0)
    pairs, cnt = gpu_join(ctx_i8, w.P, w.P, "ip", 3000.0)
    S = set(map(tuple, pairs.tolist()))
    assert {(j, i) for (i, j) in S} == S and all((i, i) in S for i in range(700))
    assert_exact(pairs, cnt, w.P, w.P, "ip", 3000.0)


def test_empty_inputs_count_only_and_capacity(ctx_i8):
    P, Q = W.random_points("i8", 300, 64, 13), W.random_points("i8", 500, 64, 14)
    dP, dQ = B.to_device(P), B.to_device(Q)
    out = torch.zeros((8, 2), dtype=torch.int32, device="cuda:0")
    assert ctx_i8.simjoin_run(dP, 0, dQ, 500, 64, "ip", 0.0, out, 8) == (B.SIMJOIN_OK, 0)
    assert ctx_i8.simjoin_run(dP, 300, dQ, 0, 64, "ip", 0.0, out, 8) == (B.SIMJOIN_OK, 0)
    want, wcnt = O.join(P, Q, "ip", 20.0, "i8")
    assert wcnt > 100
    st, cnt = ctx_i8.simjoin_run(dP, 300, dQ, 500, 64, "ip", 20.0, None, 0)       # count-only mode
    assert (st, cnt) == (B.SIMJOIN_ERR_CAPACITY, wcnt)
    part, cnt = gpu_join(ctx_i8, P, Q, "ip", 20.0, capacity=37)                   # overflow: valid subset
    assert cnt == wcnt and len(part) == 37
    k = keys(part)
    assert len(np.unique(k)) == 37 and np.isin(k, keys(want)).all()


def test_offsets_shift_emitted_indices(ctx_i8):
    P, Q = W.random_points("i8", 260, 64, 15), W.random_points("i8", 300, 64, 16)
    base, cnt = gpu_join(ctx_i8, P, Q, "ip", 18.0)
    assert ctx_i8.simjoin_set_offsets(1000, 70000) == B.SIMJOIN_OK
    try:
        shifted, cnt2 = gpu_join(ctx_i8, P, Q, "ip", 18.0)
    finally:
        assert ctx_i8.simjoin_set_offsets(0, 0) == B.SIMJOIN_OK
    assert cnt2 == cnt and np.array_equal(np.sort(keys(shifted - np.array([1000, 70000]))), np.sort(keys(base)))
    assert ctx_i8.simjoin_set_offsets(-1, 0) == B.SIMJOIN_ERR_ARG


@pytest.mark.parametrize("world", [2, 3, 8])
def test_row_block_shards_on_the_gpu_union_to_the_whole_join(ctx_i8, ctx_bf16, world):
    """Theorem 1's block decomposition through the CUDA path: the row blocks of `sharding.row_block`, joined one after
    another with simjoin_set_offsets(start, 0) -- what each rank of a sharded run does on its own GPU -- concatenate to
    the oracle's whole join (int8 exact, bf16 inside the band), ragged n."""
    from paper_2006_12608_b200 import sharding
    w = W.make_workload(4, n=3001, m=1700, planted=400)
    wb = W.make_workload(2, n=2003, m=1500, planted=300)
    for ctx, wl, exact in ((ctx_i8, w, True), (ctx_bf16, wb, False)):
        parts, total = [], 0
        try:
            for rank in range(world):
                start, rows = sharding.row_block(wl.n, world, rank)
                assert ctx.simjoin_set_offsets(start, 0) == B.SIMJOIN_OK
                pairs, cnt = gpu_join(ctx, wl.P[start:start + rows], wl.Q, wl.kind, wl.threshold)
                assert len(pairs) == cnt and (cnt == 0 or (pairs[:, 0].min() >= start and pairs[:, 0].max() < start + rows))
                parts.append(pairs)
                total += cnt
        finally:
            assert ctx.simjoin_set_offsets(0, 0) == B.SIMJOIN_OK
        allp = np.concatenate(parts)
        if exact:
            assert_exact(allp, total, wl.P, wl.Q, wl.kind, wl.threshold)
        else:
            assert_band(allp, total, wl.P, wl.Q, wl.kind, wl.threshold)
        assert np.isin(keys(wl.planted), keys(allp)).all()


def test_context_on_a_stream_of_its_own():
    """A context bound to a non-default stream: every launch, the selection words, the control-block hand-over between
    consecutive calls and the result the kernel stores to host memory follow that stream."""
    w = W.make_workload(3, n=2500, m=1900, planted=150)
    wb = W.make_workload(5, n=1200, m=1500, centers=15)
    dP, dQ, bP, bQ = B.to_device(w.P), B.to_device(w.Q), B.to_device(wb.P), B.to_device(wb.Q)
    out = torch.full((1 << 18, 2), -7, dtype=torch.int32, device="cuda:0")
    torch.cuda.synchronize()
    stream = torch.cuda.Stream(device=0)
    ci, cb = B.Simjoin("i8", 0, stream=stream.cuda_stream), B.Simjoin("bf16", 0, stream=stream.cuda_stream)
    try:
        assert ci.simjoin_set_option(B.SIMJOIN_OPT_SELECT_MIN_OPS, 0.0) == B.SIMJOIN_OK
        want, wcnt = O.join(w.P, w.Q, "ip", w.threshold, "i8")
        for _ in range(3):
            st, cnt = ci.simjoin_run(dP, w.n, dQ, w.m, w.d, "ip", w.threshold, out, 1 << 18)
            assert (st, cnt) == (B.SIMJOIN_OK, wcnt)
            stream.synchronize()
            assert np.array_equal(np.sort(keys(out[:cnt].cpu().numpy())), keys(want))
        for _ in range(3):                      # dense: the second and third call take the 16-warp layout
            st, cnt = cb.simjoin_run(bP, wb.n, bQ, wb.m, wb.d, "l2", wb.threshold, out, 1 << 18)
            assert st == B.SIMJOIN_OK
            assert_band(out[:cnt].cpu().numpy(), cnt, wb.P, wb.Q, "l2", wb.threshold)
    finally:
        ci.close()
        cb.close()


def test_bad_arguments_are_rejected_before_launch(ctx_i8, ctx_bf16):
    P = B.to_device(W.random_points("i8", 64, 64, 17))
    out = torch.zeros((8, 2), dtype=torch.int32, device="cuda:0")
    E = B.SIMJOIN_ERR_ARG
    assert ctx_i8.simjoin_run(None, 64, P, 64, 64, "ip", 0.0, out, 8)[0] == E
    assert ctx_i8.simjoin_run(P, -1, P, 64, 64, "ip", 0.0, out, 8)[0] == E
    assert ctx_i8.simjoin_run(P, 64, P, 64, 0, "ip", 0.0, out, 8)[0] == E
    assert ctx_i8.simjoin_run(P, 64, P, 64, 64, "ip", float("nan"), out, 8)[0] == E
    assert ctx_i8.simjoin_run(P, 64, P, 64, 64, "l2", -1.0, out, 8)[0] == E
    assert ctx_i8.simjoin_run(P, 64, P, 64, 64, "ip", 0.0, None, 8)[0] == E
    assert ctx_i8.simjoin_run(P.cpu().numpy(), 64, P, 64, 64, "ip", 0.0, out, 8)[0] == E     # host pointer
    assert ctx_i8.simjoin_run(P, 64, P, 64, 64, "ip", 0.0, out.cpu().numpy(), 8)[0] == E
    U = B.SIMJOIN_ERR_UNSUPPORTED
    assert ctx_i8.simjoin_run(P, 64, P, 64, 24, "ip", 0.0, out, 8)[0] == U                   # 24 B rows
    assert ctx_i8.simjoin_run(P.data_ptr() + 1, 32, P, 64, 64, "ip", 0.0, out, 8)[0] == U    # misaligned
    assert ctx_i8.simjoin_run(P, 1, P, 1, 16384, "ip", 0.0, out, 8)[0] == U                  # row too long
    assert ctx_i8.simjoin_last_kernel_ms()[0] in (B.SIMJOIN_OK, B.SIMJOIN_ERR_ARG)
    # the context is still usable afterwards
    assert ctx_i8.simjoin_run(P, 64, P, 64, 64, "ip", 1e9, out, 8) == (B.SIMJOIN_OK, 0)


def test_bounded_wait_gives_up_and_context_survives(ctx_i8):
    """A wait on a barrier nothing completes must expire (status ERR_TIMEOUT), not hang; the context
    keeps working afterwards.  Nothing is faulted: the wait simply runs out of its cycle budget."""
    assert ctx_i8.simjoin_selftest_wait_timeout() == B.SIMJOIN_ERR_TIMEOUT
    w = W.make_workload(1)
    pairs, cnt = gpu_join(ctx_i8, w.P, w.Q, "ip", w.threshold)
    assert_exact(pairs, cnt, w.P, w.Q, "ip", w.threshold)


def test_run_host_matches_device_path(ctx_i8):
    w = W.make_workload(4, n=3000, m=2500, planted=120)
    want, wcnt = O.join(w.P, w.Q, "ip", w.threshold, "i8")
    out = np.full((wcnt + 10, 2), -7, dtype=np.int32)
    st, cnt = ctx_i8.simjoin_run_host(w.P, w.n, w.Q, w.m, w.d, "ip", w.threshold, out, wcnt + 10)
    assert (st, cnt) == (B.SIMJOIN_OK, wcnt)
    assert np.array_equal(np.sort(keys(out[:cnt])), keys(want)) and np.all(out[cnt:] == -7)
    dP = B.to_device(w.P)
    assert ctx_i8.simjoin_run_host(dP, w.n, w.Q, w.m, w.d, "ip", w.threshold, out, 10)[0] == B.SIMJOIN_ERR_ARG


def test_run_host_uploads_a_large_q_in_slices(ctx_i8, ctx_bf16):
    """A Q above 64 MiB goes up in ~32 MiB slices that are joined one by one while the next ones are still being
    copied: the union of the slices' results, with their column offsets, must be the whole join; the capacity
    is shared by the slices and the count stays the full one when it runs out."""
    P, Q = W.random_points("i8", 200, 8192, 65), W.random_points("i8", 9000, 8192, 66)      # Q: 73.7 MB -> 3 slices of 4096 rows
    t = 2.2 * (8192 * 16.0) ** 0.5
    want, wcnt = O.join(P, Q, "ip", t, "i8")
    assert wcnt > 1000 and len(np.unique(want[:, 1] // 4096)) == 3                          # hits in every slice
    out = np.full((wcnt + 10, 2), -7, dtype=np.int32)
    assert ctx_i8.simjoin_set_offsets(7, 100) == B.SIMJOIN_OK
    try:
        st, cnt = ctx_i8.simjoin_run_host(P, 200, Q, 9000, 8192, "ip", t, out, wcnt + 10)
    finally:
        ctx_i8.simjoin_set_offsets(0, 0)
    assert (st, cnt) == (B.SIMJOIN_OK, wcnt)
    assert np.array_equal(np.sort(keys(out[:cnt])), keys(want + np.array([7, 100]))) and np.all(out[cnt:] == -7)
    small = np.full((wcnt // 2 + 4, 2), -7, dtype=np.int32)
    st, cnt = ctx_i8.simjoin_run_host(P, 200, Q, 9000, 8192, "ip", t, small, wcnt // 2)
    assert (st, cnt) == (B.SIMJOIN_ERR_CAPACITY, wcnt)
    assert np.isin(keys(small[:wcnt // 2]), keys(want)).all() and np.all(small[wcnt // 2:] == -7)
    assert len(np.unique(keys(small[:wcnt // 2]))) == wcnt // 2
    # a norm kind through the same path (row terms are recomputed per slice)
    Pb, Qb = W.random_points("bf16", 150, 4096, 67), W.random_points("bf16", 8500, 4096, 68)  # Q: 69.6 MB
    outb = np.full((1 << 20, 2), -7, dtype=np.int32)
    st, cnt = ctx_bf16.simjoin_run_host(Pb, 150, Qb, 8500, 4096, "cos", 0.03, outb, 1 << 20)
    assert st == B.SIMJOIN_OK and cnt > 1000
    assert_band(outb[:cnt], cnt, Pb, Qb, "cos", 0.03)


def test_run_host_uploads_a_mid_size_q_in_four_slices(ctx_i8):
    """A Q of 32 to 64 MiB (here 33 000 rows of 1 KiB) is joined in four slices of 8448 rows; hits in every slice, ragged last one."""
    P, Q = W.random_points("i8", 150, 1024, 85), W.random_points("i8", 33000, 1024, 86)
    Q[::1100] = P[:30]
    t = 3.3 * (1024 * 16.0) ** 0.5
    want, wcnt = O.join(P, Q, "ip", t, "i8")
    assert wcnt >= 30 and len(np.unique(want[:, 1] // 8448)) == 4
    out = np.full((wcnt + 10, 2), -7, dtype=np.int32)
    st, cnt = ctx_i8.simjoin_run_host(P, 150, Q, 33000, 1024, "ip", t, out, wcnt + 10)
    assert (st, cnt) == (B.SIMJOIN_OK, wcnt)
    assert np.array_equal(np.sort(keys(out[:cnt])), keys(want)) and np.all(out[cnt:] == -7)


def test_run_host_downloads_a_dense_result_slice_by_slice(ctx_i8):
    """Room for 2^23 pairs and more: Q is joined in eight slices and every slice's pairs travel to the host while the
    next slice is joined.  Result and overflow behaviour are those of the one-piece call."""
    P, Q = W.random_points("i8", 300, 64, 75, lo=-3, hi=3), W.random_points("i8", 40000 + 37, 64, 76, lo=-3, hi=3)
    t = 4.0
    want, wcnt = O.join(P, Q, "ip", t, "i8")
    assert wcnt > 3_000_000
    cap = 1 << 23
    out = np.full((cap + 4, 2), -7, dtype=np.int32)
    st, cnt = ctx_i8.simjoin_run_host(P, len(P), Q, len(Q), 64, "ip", t, out, cap)
    assert (st, cnt) == (B.SIMJOIN_OK, wcnt)
    assert np.array_equal(np.sort(keys(out[:cnt])), keys(want)) and np.all(out[cnt:] == -7)
    # more pairs than room: capacity is shared by the slices, the count stays the full one
    P2 = W.random_points("i8", 900, 64, 77, lo=-3, hi=3)
    want2, wcnt2 = O.join(P2, Q, "ip", t, "i8")
    assert wcnt2 > cap
    st, cnt = ctx_i8.simjoin_run_host(P2, len(P2), Q, len(Q), 64, "ip", t, out, cap)
    assert (st, cnt) == (B.SIMJOIN_ERR_CAPACITY, wcnt2)
    got = keys(out[:cap])
    assert len(np.unique(got)) == cap and np.isin(got, keys(want2)).all() and np.all(out[cap:] == -7)


def test_row_norms_prepass(ctx_i8, ctx_bf16):
    for rows, d in [(1, 16), (300, 64), (1000, 144), (513, 1024)]:
        X = W.random_points("i8", rows, d, 18, lo=-128, hi=127)
        out = torch.zeros(rows, dtype=torch.int32, device="cuda:0")
        assert ctx_i8.simjoin_row_norms(B.to_device(X), rows, d, out) == B.SIMJOIN_OK
        assert np.array_equal(out.cpu().numpy().astype(np.int64), O.sq_norms(X, "i8"))       # exact
    for rows, d in [(1, 8), (300, 64), (1000, 72), (513, 512)]:
        X = W.random_points("bf16", rows, d, 19, scale=3.0)
        out = torch.zeros(rows, dtype=torch.float32, device="cuda:0")
        assert ctx_bf16.simjoin_row_norms(B.to_device(X), rows, d, out) == B.SIMJOIN_OK
        np.testing.assert_allclose(out.cpu().numpy().astype(np.float64), O.sq_norms(X, "bf16"), rtol=2e-6)


# ------------------------------------------------------------------ scheduling: several waves + a split tail
def test_multiple_waves_and_split_tail(ctx_i8):
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n = 128 * (sms + 21) + 5           # one full wave, then a 22-block tail split over the CTAs
    w = W.make_workload(4, n=n, m=2048 + 77, planted=500)
    pairs, cnt = gpu_join(ctx_i8, w.P, w.Q, "ip", w.threshold)
    assert_exact(pairs, cnt, w.P, w.Q, "ip", w.threshold)
    assert np.isin(keys(w.planted), keys(pairs)).all()


@pytest.mark.parametrize("d", [384, 512, 640, 2048])
def test_many_tiles_per_cta_with_long_rows(ctx_i8, d):
    """3, 4, 5 and 16 K chunks per tile with a dozen tiles per CTA: consecutive tiles share ring stages
    here, which is the case where only one warp may issue MMAs."""
    P, Q = W.random_points("i8", 1024 + 19, d, 71), W.random_points("i8", 40 * 256 + 3, d, 72)
    t = 2.4 * (d * 16.0) ** 0.5
    pairs, cnt = gpu_join(ctx_i8, P, Q, "ip", t, capacity=1 << 20)
    assert_exact(pairs, cnt, P, Q, "ip", t)
    assert cnt > 1000


def test_several_q_panels(ctx_i8, ctx_bf16):
    """Long rows make the L2-sized Q panels short (16 tiles at 8 KiB rows), so m = 9000 spans three
    panels with a ragged last one; every panel has its own split partial wave."""
    P, Q = W.random_points("i8", 300, 8192, 61), W.random_points("i8", 9000, 8192, 62)
    t = 2.2 * (8192 * 16.0) ** 0.5
    pairs, cnt = gpu_join(ctx_i8, P, Q, "ip", t, capacity=1 << 20)
    assert_exact(pairs, cnt, P, Q, "ip", t)
    assert cnt > 1000
    Pb, Qb = W.random_points("bf16", 200, 4096, 63), W.random_points("bf16", 8500, 4096, 64)
    pairs, cnt = gpu_join(ctx_bf16, Pb, Qb, "cos", 0.03, capacity=1 << 20)
    assert_band(pairs, cnt, Pb, Qb, "cos", 0.03)
    assert cnt > 1000


# ------------------------------------------------------------------ the five configurations, reduced
def test_cfg2_reduced(ctx_bf16):
    w = W.make_workload(2, n=6000, m=5000, planted=200)
    pairs, cnt = gpu_join(ctx_bf16, w.P, w.Q, "cos", w.threshold)
    dis, _band = assert_band(pairs, cnt, w.P, w.Q, "cos", w.threshold)
    assert np.isin(keys(w.planted), keys(pairs)).all() and dis == 0


def test_cfg3_reduced(ctx_i8):
    w = W.make_workload(3, n=5000, m=4100, planted=300)
    pairs, cnt = gpu_join(ctx_i8, w.P, w.Q, "ip", w.threshold)
    assert_exact(pairs, cnt, w.P, w.Q, "ip", w.threshold)
    assert np.isin(keys(w.planted), keys(pairs)).all()


def test_cfg4_reduced(ctx_i8):
    w = W.make_workload(4, n=9000, m=7000, planted=900)
    pairs, cnt = gpu_join(ctx_i8, w.P, w.Q, "ip", w.threshold)
    assert_exact(pairs, cnt, w.P, w.Q, "ip", w.threshold)
    assert np.isin(keys(w.planted), keys(pairs)).all()


@pytest.mark.parametrize("reading", ["radial", "percoord"])
def test_cfg5_reduced(ctx_bf16, reading):
    w = W.make_workload(5, n=6000, m=5000, centers=50, sigma_reading=reading)
    pairs, cnt = gpu_join(ctx_bf16, w.P, w.Q, "l2", w.threshold, capacity=1 << 20)
    assert_band(pairs, cnt, w.P, w.Q, "l2", w.threshold)
    if reading == "radial":     # dense: exactly the same-cluster relation
        assert cnt == int(sum(np.sum(w.labels_p == c) * np.sum(w.labels_q == c) for c in range(50)))
        assert np.all(w.labels_p[pairs[:, 0]] == w.labels_q[pairs[:, 1]])
    else:
        assert cnt == 0


@pytest.mark.parametrize("d", [64, 1024, 2048])
@pytest.mark.parametrize("r", [0.05, 0.0, 2.0])
def test_bf16_l2_radius_far_below_the_norms(ctx_bf16, d, r):
    """N(0,1) rows (|x|^2 about d) with planted equal and near-equal rows, and radii whose square is far below what
    |x|^2 + |y|^2 - 2<x,y> resolves in fp32: the join must still be inside the band of the oracle's difference-form
    distances (equal rows at r = 0; rows one or two bf16 steps apart in a single coordinate, 0.016 to 0.031, at
    r = 0.05).  d = 64 at r = 2 stays on the norm-expansion path, the others are decided from the rows."""
    rng = np.random.default_rng(d)
    n, m = 700 + 13, 900 + 5
    Pf = rng.standard_normal((n, d)).astype(np.float32)
    Qf = rng.standard_normal((m, d)).astype(np.float32)
    P, Q = W.f32_to_bf16_bits(Pf), W.f32_to_bf16_bits(Qf)
    Q[3:603:3] = P[:200]                                   # equal rows
    # near-equal rows: one coordinate of value v moved by one or two bf16 steps (2^-8 |v| each: 0.004 .. 0.03 apart)
    for t, (i, j) in enumerate(zip(range(200, 400), range(4, 604, 3))):
        row = P[i].copy()
        c = int(np.argmax(W.bf16_bits_to_f32(row) * (1 if t % 2 else -1)))
        row[c] += 1 + (t % 3 == 0)
        Q[j] = row
    pairs, cnt = gpu_join(ctx_bf16, P, Q, "l2", r, capacity=1 << 20)
    assert_band(pairs, cnt, P, Q, "l2", r)
    assert cnt >= 200
    got = set(map(tuple, pairs.tolist()))
    assert all((i, 3 + 3 * i) in got for i in range(200)), "an equal pair is missing"


@pytest.mark.parametrize("kind", ["ip", "cos", "l2"])
@pytest.mark.parametrize("n,m,d", [(129, 257, 64), (700, 1300, 64), (513, 1000, 128), (300, 2100, 128), (140, 300, 72)])
def test_bf16_dense_epilogue_matches_the_oracle(kind, n, m, d):
    """The 16-epilogue-warp instantiations (rows of one or two whole chunks; Euclidean joins of rows up to 240 bytes through
    the operand transform), forced on: sparse and dense outputs, ragged tiles, hits in both 64-column halves of a block;
    other row lengths fall back to the regular kernel.  Then the default
    mode, where a context switches to them after a dense join and back after a sparse one: same sets."""
    P, Q = W.random_points("bf16", n, d, 15), W.random_points("bf16", m, d, 16)
    Q[1:m:7][:n] = P[:len(Q[1:m:7][:n])]
    sparse = {"ip": 1.5 * d ** 0.5, "cos": 1.5 / d ** 0.5, "l2": (2 * d) ** 0.5 - 1.2}[kind]
    dense = {"ip": -0.3 * d ** 0.5, "cos": -0.3 / d ** 0.5, "l2": (2 * d) ** 0.5 + 0.4}[kind]
    with B.Simjoin("bf16", 0) as ctx:
        assert ctx.simjoin_set_option(B.SIMJOIN_OPT_DENSE_EPILOGUE, 3.0) == B.SIMJOIN_ERR_ARG
        for mode in (1.0, 2.0):
            assert ctx.simjoin_set_option(B.SIMJOIN_OPT_DENSE_EPILOGUE, mode) == B.SIMJOIN_OK
            for t in (sparse, dense, dense, sparse, sparse):
                pairs, cnt = gpu_join(ctx, P, Q, kind, t, capacity=1 << 22)
                assert_band(pairs, cnt, P, Q, kind, t)
                assert cnt > 0
            if kind == "l2":
                # A Euclidean join in the 16-warp layout runs on transformed operands (the squared-L2 embedding appended
                # to copies of the rows) where those fit two chunks; a radius far below the norms must still select the
                # form that decides candidates from the original rows: only the planted equal rows are that close.
                for t in (0.01, 0.0):
                    pairs, cnt = gpu_join(ctx, P, Q, kind, t, capacity=1 << 22)
                    assert_band(pairs, cnt, P, Q, kind, t)
                    assert cnt == len(Q[1:m:7][:n])


@pytest.mark.parametrize("kind", ["ip", "cos"])
@pytest.mark.parametrize("d", [24, 64, 112])
def test_bf16_dense_sign_test_handles_zero_vectors_and_every_threshold(kind, d):
    """Dense inner-product and cosine joins of rows up to 240 bytes run as the sign of one inner product on transformed
    operands (the threshold, and for the cosine the norms, travel as appended coordinates).  Zero vectors on both sides
    (their cosine counts as 0: they pass iff t <= 0), equal and opposite rows, thresholds of both signs, zero, tiny, huge
    and infinite; the exact set outside the band, everything at +-inf."""
    n, m = 300, 700
    P, Q = W.random_points("bf16", n, d, 31), W.random_points("bf16", m, d, 32)
    P[5] = 0
    P[130] = 0
    Q[7] = 0
    Q[300:303] = 0
    Q[11:311:3] = P[:100]
    Q[12] = P[1] ^ np.uint16(0x8000)                     # the opposite row
    Q[13] = W.f32_to_bf16_bits(W.bf16_bits_to_f32(P[2]) * 2.0 ** -60)      # a tiny multiple: cosine 1, inner product ~0
    scale = d ** 0.5 if kind == "ip" else 1.0 / d ** 0.5
    with B.Simjoin("bf16", 0) as ctx:
        assert ctx.simjoin_set_option(B.SIMJOIN_OPT_DENSE_EPILOGUE, 1.0) == B.SIMJOIN_OK
        for t in (0.0, -0.0, 1e-30, -1e-30, 0.2 * scale, -0.2 * scale, 1.7 * scale, -2.5 * scale, 0.999 if kind == "cos" else 3.0 * d,
                  1.0 if kind == "cos" else 1e30, -1.0 if kind == "cos" else -1e30):
            pairs, cnt = gpu_join(ctx, P, Q, kind, t, capacity=n * m + 8)
            assert_band(pairs, cnt, P, Q, kind, t)
        pairs, cnt = gpu_join(ctx, P, Q, kind, float("inf"), capacity=n * m + 8)
        assert cnt == 0
        pairs, cnt = gpu_join(ctx, P, Q, kind, float("-inf"), capacity=n * m + 8)
        assert cnt == n * m
    with B.Simjoin("bf16", 0) as ctx:                        # the same on the points themselves (8-warp layout)
        assert ctx.simjoin_set_option(B.SIMJOIN_OPT_DENSE_EPILOGUE, 0.0) == B.SIMJOIN_OK
        pairs, cnt = gpu_join(ctx, P, Q, kind, float("-inf"), capacity=n * m + 8)
        assert cnt == n * m
        pairs, cnt = gpu_join(ctx, P, Q, kind, float("inf"), capacity=n * m + 8)
        assert cnt == 0
        for t in (0.0, 1e-30, -1e-30):
            pairs, cnt = gpu_join(ctx, P, Q, kind, t, capacity=n * m + 8)
            assert_band(pairs, cnt, P, Q, kind, t)


@pytest.mark.parametrize("kind", ["ip", "cos"])
@pytest.mark.parametrize("n,m,d", [(300, 700, 64), (513, 1000, 128), (200, 600, 72), (150, 700, 520)])
@pytest.mark.parametrize("dense", [0.0, 1.0])
def test_bf16_thresholds_near_zero_are_decided_from_the_rows(kind, n, m, d, dense):
    """An inner-product or cosine threshold at or near zero leaves no tolerance band (1e-2 |t|) for the fp32 accumulation
    error of the tile product.  There the tile test is a filter and every candidate is decided from its rows in fp64, in the
    oracle's order of operations: the result is the oracle's exact set, bit for bit -- Gaussian coordinates (inexact sums),
    zero vectors, opposite rows, short, two-chunk and long rows, both epilogue layouts asked for.  Thresholds whose band
    is wide enough keep the plain test (band rule)."""
    rng = np.random.default_rng(d + n)
    P = W.f32_to_bf16_bits(rng.standard_normal((n, d)).astype(np.float32))
    Q = W.f32_to_bf16_bits(rng.standard_normal((m, d)).astype(np.float32))
    P[3] = 0
    Q[5] = 0
    Q[9] = P[7] ^ np.uint16(0x8000)
    Q[11] = P[8]
    scale = float(d) if kind == "ip" else 1.0
    with B.Simjoin("bf16", 0) as ctx:
        assert ctx.simjoin_set_option(B.SIMJOIN_OPT_DENSE_EPILOGUE, dense) == B.SIMJOIN_OK
        for t in (0.0, -0.0, 1e-30, -1e-30, 1e-7 * scale, -1e-7 * scale, 3e-5 * scale, -2e-4 * scale):
            pairs, cnt = gpu_join(ctx, P, Q, kind, t, capacity=n * m + 8)
            assert_exact(pairs, cnt, P, Q, kind, t, dtype="bf16")
        for t in (0.05 * scale ** 0.5, -0.05 * scale ** 0.5, 0.2 * scale ** 0.5):
            pairs, cnt = gpu_join(ctx, P, Q, kind, t, capacity=n * m + 8)
            assert_band(pairs, cnt, P, Q, kind, t)
        if d == 64:
            # thresholds equal to the exact score of a pair whose score is nearly zero: that pair passes by equality, which
            # an fp32-accumulated score gets right only by chance
            cand = np.stack(np.meshgrid(np.arange(64), np.arange(m), indexing="ij"), axis=-1).reshape(-1, 2).astype(np.int32)
            sc = O.scores(P, Q, kind, "bf16", cand)
            order = np.argsort(np.abs(sc))
            picked = [k for k in order if sc[k] != 0.0][:12]
            for k in picked:
                t = float(sc[k])
                pairs, cnt = gpu_join(ctx, P, Q, kind, t, capacity=n * m + 8)
                assert_exact(pairs, cnt, P, Q, kind, t, dtype="bf16")
                assert tuple(cand[k]) in set(map(tuple, pairs.tolist()))


def test_first_large_join_of_a_context_samples_its_density():
    """A fresh context in the default mode counts a sample's pairs before a join of 1e12 operations or more and picks the
    layout from that: the dense mixture then runs on transformed operands at once, a sparse join of the same size does not;
    either way the result is the one the forced 8-warp layout gives."""
    w = W.make_workload(5, n=98304, m=98304, centers=1024)
    cap = 12_000_000
    per_p = np.bincount(w.labels_p, minlength=1024).astype(np.int64)
    per_q = np.bincount(w.labels_q, minlength=1024).astype(np.int64)
    for t in (w.threshold, 0.01):
        sets = []
        for mode in (2.0, 0.0):
            with B.Simjoin("bf16", 0) as ctx:
                assert ctx.simjoin_set_option(B.SIMJOIN_OPT_DENSE_EPILOGUE, mode) == B.SIMJOIN_OK
                pairs, cnt = gpu_join(ctx, w.P, w.Q, "l2", t, capacity=cap)
                sets.append(np.sort(keys(pairs)))
        assert np.array_equal(sets[0], sets[1])
        if t == w.threshold:
            assert len(sets[0]) == int(np.sum(per_p * per_q))


def test_debug_log_names_the_layout_the_sample_chose():
    """SIMJOIN_DEBUG=1: the sample's line, then the join's own line with the dense layout, on a context's very first call."""
    import subprocess
    import sys
    code = (
        "import torch\n"
        "from paper_2006_12608_b200 import binding as B, workloads as W\n"
        "w = W.make_workload(5, n=98304, m=98304, centers=1024)\n"
        "out = torch.empty((12_000_000, 2), dtype=torch.int32, device='cuda:0')\n"
        "with B.Simjoin('bf16', 0) as ctx:\n"
        "    st, cnt = ctx.simjoin_run(B.to_device(w.P), w.n, B.to_device(w.Q), w.m, w.d, 'l2', w.threshold, out, 12_000_000)\n"
        "    assert st == 0, st\n")
    env = dict(os.environ, SIMJOIN_DEBUG="1")
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, cwd=os.path.dirname(os.path.dirname(__file__)), timeout=600)
    assert r.returncode == 0, r.stderr
    lines = [ln for ln in r.stderr.splitlines() if ln.startswith("[simjoin] run")]
    assert len(lines) == 2
    assert "n=256 " in lines[0] and "capacity=0" in lines[0] and "8 epilogue warps" in lines[0]
    assert "n=98304 " in lines[1] and "16 epilogue warps on transformed operands" in lines[1]


def test_repeated_runs_give_the_same_set(ctx_bf16):
    w = W.make_workload(5, n=3000, m=3000, centers=30)
    a, ca = gpu_join(ctx_bf16, w.P, w.Q, "l2", w.threshold, capacity=1 << 19)
    b, cb = gpu_join(ctx_bf16, w.P, w.Q, "l2", w.threshold, capacity=1 << 19)
    assert ca == cb and np.array_equal(np.sort(keys(a)), np.sort(keys(b)))


# ------------------------------------------------------------------ long rows: 256 x 256 tiles, two epilogue passes
@pytest.mark.parametrize("kind", ["ip", "l2"])
@pytest.mark.parametrize("d,lo,hi", [(512, -3, 3), (656, -1, 1), (1024, -127, 127)])
def test_i8_long_row_geometry(ctx_i8, kind, d, lo, hi):
    """Rows of 512 bytes and more: whole chunks, a 16-byte last chunk (656), and values too wide for the packed
    epilogue (1024); ragged row counts, hits in both column passes of a tile."""
    P, Q = W.random_points("i8", 300 + 7, d, 81, lo=lo, hi=hi), W.random_points("i8", 1024 + 45, d, 82, lo=lo, hi=hi)
    Q[5:260:3] = P[:85]                                  # planted equal rows, spread over both passes and several tiles
    sd = (d * ((hi - lo + 1) ** 2 - 1) / 12.0)           # variance of one coordinate product sum, roughly
    if kind == "ip":
        t = 2.5 * (d * ((hi * (hi + 1)) / 3.0) ** 2) ** 0.5
    else:
        t = (2.0 * sd) ** 0.5 * 0.86                      # a little below the typical distance: the low tail passes
    pairs, cnt = gpu_join(ctx_i8, P, Q, kind, t, capacity=1 << 20)
    assert_exact(pairs, cnt, P, Q, kind, t)
    assert cnt >= 85


@pytest.mark.parametrize("kind", ["ip", "cos", "l2"])
@pytest.mark.parametrize("d", [256, 264, 1040])
def test_bf16_long_row_geometry(ctx_bf16, kind, d):
    """bf16 rows of 512, 528 (16-byte last chunk) and 2080 bytes (the last also takes the two-dimensional waves)."""
    P, Q = W.random_points("bf16", 260 + 3, d, 91), W.random_points("bf16", 800 + 31, d, 92)
    Q[3:200:2] = P[:99]
    t = {"ip": 3.0 * d ** 0.5, "cos": 0.12, "l2": (2.0 * d) ** 0.5 - 1.5}[kind]
    pairs, cnt = gpu_join(ctx_bf16, P, Q, kind, t, capacity=1 << 20)
    assert_band(pairs, cnt, P, Q, kind, t)
    assert cnt >= 99


def test_two_dimensional_waves_cover_every_tile_pair_once(ctx_i8):
    """2 KiB rows switch to waves of 37 x 4 tile pairs: 39 P tiles x 6 Q tiles need two waves in each direction,
    with partly empty ones at both edges."""
    P, Q = W.random_points("i8", 38 * 256 + 17, 2048, 95, lo=-1, hi=1), W.random_points("i8", 5 * 256 + 40, 2048, 96, lo=-1, hi=1)
    Q[::11] = P[:len(Q[::11])]
    t = 3.6 * (2048 * 4.0 / 9.0) ** 0.5
    pairs, cnt = gpu_join(ctx_i8, P, Q, "ip", t, capacity=1 << 20)
    assert_exact(pairs, cnt, P, Q, "ip", t)
    assert cnt >= len(Q[::11])


# ------------------------------------------------------------------ int8 cosine (exact, as every int8 kind)
def int8_cos_case(ctx_i8, P, Q, t, cap=1 << 20):
    pairs, cnt = gpu_join(ctx_i8, P, Q, "cos", t, cap)
    want, wcnt = O.join(P, Q, "cos", t, "i8")
    assert cnt == wcnt, (cnt, wcnt, t)
    got = np.asarray(pairs, dtype=np.int64).reshape(-1, 2)
    assert len(np.unique((got[:, 0] << 32) | got[:, 1])) == cnt
    assert set(map(tuple, got.tolist())) == set(map(tuple, want.tolist()))
    return cnt


@pytest.mark.parametrize("n,m,d,hi", [(300, 500, 64, 127), (1000, 777, 128, 3), (513, 1025, 48, 127), (700, 900, 272, 127),
                                      (600, 400, 640, 5), (300, 700, 1040, 127), (260, 300, 2064, 127)])
@pytest.mark.parametrize("t", [0.35, 0.0, -0.2])
def test_i8_cosine_matches_oracle(ctx_i8, n, m, d, hi, t):
    """Both epilogue widths (hi = 3, 5: scores fit 16 bits), every tile geometry, positive / zero / negative t."""
    P, Q = W.random_points("i8", n, d, 51, lo=-hi, hi=hi), W.random_points("i8", m, d, 52, lo=-hi, hi=hi)
    P[3] = 0
    Q[7] = 0
    Q[11] = P[5]                                              # cosine exactly 1
    if t > 0:
        allp = np.stack([np.repeat(np.arange(40), 50), np.tile(np.arange(50), 40)], axis=1).astype(np.int32)
        t = float(np.quantile(O.scores(P, Q, "cos", "i8", allp), 0.995))   # a threshold that has hits at every d
    assert int8_cos_case(ctx_i8, P, Q, t, cap=1 << 21) > 0


def test_i8_cosine_threshold_one_and_ties(ctx_i8):
    """Parallel rows score exactly 1 and pass t = 1; thresholds equal to attained scores are inclusive."""
    rng = np.random.default_rng(5)
    P = rng.integers(-60, 61, size=(400, 128)).astype(np.int8)
    Q = rng.integers(-60, 61, size=(600, 128)).astype(np.int8)
    Q[:100] = 2 * P[:100]
    Q[100:150] = -P[100:150]
    assert int8_cos_case(ctx_i8, P, Q, 1.0) == 100
    assert int8_cos_case(ctx_i8, P, Q, -1.0) == 400 * 600
    allp = np.stack([np.repeat(np.arange(400), 600), np.tile(np.arange(600), 400)], axis=1).astype(np.int32)
    sc = np.sort(O.scores(P, Q, "cos", "i8", allp))
    for t in (sc[-150], sc[-1000], np.nextafter(sc[-150], 2.0), np.nextafter(sc[-1000], -2.0)):
        int8_cos_case(ctx_i8, P, Q, float(t))


def test_i8_cosine_planted_pairs_at_scale(ctx_i8):
    w = W.make_workload(4, n=20000, m=30000, planted=300)          # +-1 rows: cosine = <x,y> / d
    t = w.threshold / w.d
    cnt = int8_cos_case(ctx_i8, w.P, w.Q, t)
    assert cnt >= 300 and cnt == O.join(w.P, w.Q, "ip", w.threshold, "i8")[1]


def test_repeated_calls_give_the_same_set(ctx_i8, ctx_bf16):
    """The output order is unspecified (atomics), the set is not: repeated calls on one context, other calls in
    between, return the same pairs -- also for bf16, where in-band pairs could fall on either side but the arithmetic
    of a given launch configuration is fixed."""
    w = W.make_workload(4, n=5000, m=7000, planted=300)
    wb = W.make_workload(2, n=4000, m=3000, planted=300)
    Pb, Qb = W.random_points("bf16", 2000, 64, 95), W.random_points("bf16", 2500, 64, 96)
    first = {}
    for rep in range(3):
        runs = {"i8": gpu_join(ctx_i8, w.P, w.Q, "ip", 40.0, 1 << 22)[0],
                "cos": gpu_join(ctx_bf16, wb.P, wb.Q, "cos", 0.2, 1 << 22)[0],
                "l2": gpu_join(ctx_bf16, Pb, Qb, "l2", 9.0, 1 << 22)[0]}
        for name, pairs in runs.items():
            k = np.sort(keys(pairs))
            assert len(k) > 1000
            if rep == 0:
                first[name] = k
            else:
                assert np.array_equal(first[name], k), name

