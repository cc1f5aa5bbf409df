"""The seeded input generators: determinism, shapes, value ranges, planted structure.
Nothing here evaluates a join score."""
import numpy as np
import pytest
import torch

from paper_2006_12608_b200 import workloads as W


def test_bf16_bit_conversion_matches_torch_cast():
    a = np.random.default_rng(0).standard_normal(10000).astype(np.float32) * 3
    a[:4] = [0.0, -0.0, 1.0, 65504.0]
    bits = W.f32_to_bf16_bits(a)
    t = torch.from_numpy(a).to(torch.bfloat16)
    assert np.array_equal(bits.view(np.int16), t.view(torch.int16).numpy())
    assert np.array_equal(W.bf16_bits_to_f32(bits), t.to(torch.float32).numpy())


@pytest.mark.parametrize("cfg,kw", [(1, {}), (2, dict(n=500, m=300, planted=20)), (3, dict(n=400, m=600, planted=30)),
                                    (4, dict(n=700, m=900, planted=50)), (5, dict(n=500, m=400, centers=16))])
def test_deterministic_and_well_formed(cfg, kw):
    a, b = W.make_workload(cfg, **kw), W.make_workload(cfg, **kw)
    assert np.array_equal(a.P, b.P) and np.array_equal(a.Q, b.Q) and np.array_equal(a.planted, b.planted)
    c = W.make_workload(cfg, seed=1, **kw)
    assert not np.array_equal(a.P, c.P)
    assert a.P.shape == (a.n, a.d) and a.Q.shape == (a.m, a.d)
    assert a.P.dtype == (np.int8 if a.dtype == "i8" else np.uint16)
    assert a.P.flags["C_CONTIGUOUS"] and a.Q.flags["C_CONTIGUOUS"]
    assert a.ops == 2 * a.n * a.m * a.d
    if len(a.planted):
        assert len(np.unique(a.planted[:, 0])) == len(a.planted) == len(np.unique(a.planted[:, 1]))


def test_planted_structure():
    w = W.make_workload(1)
    assert set(np.unique(w.P)) == {-1, 1} and set(np.unique(w.Q)) == {-1, 1}
    x, y = w.P[w.planted[:, 0]], w.Q[w.planted[:, 1]]
    assert np.all((x != y).sum(axis=1) == 4)
    w4 = W.make_workload(4, n=5000, m=4000, planted=300)
    assert np.all((w4.P[w4.planted[:, 0]] != w4.Q[w4.planted[:, 1]]).sum(axis=1) == 8)
    w3 = W.make_workload(3, n=5000, m=4000, planted=300)
    assert w3.P.min() == -8 and w3.P.max() == 8
    e = w3.Q[w3.planted[:, 1]].astype(int) - w3.P[w3.planted[:, 0]].astype(int)
    assert set(np.unique(e)) == {-1, 0, 1} and abs(w3.Q).max() == 9


def test_full_size_parameters_match_the_benchmark_table():
    c = W.CONFIGS
    assert (c[1]["n"], c[1]["d"], c[1]["threshold"], c[1]["planted"]) == (2048, 64, 40.0, 32)
    assert (c[2]["n"], c[2]["d"], c[2]["threshold"], c[2]["planted"]) == (65536, 128, 0.9, 1000)
    assert (c[3]["n"], c[3]["d"], c[3]["threshold"], c[3]["planted"]) == (262144, 256, 3000.0, 10000)
    assert (c[4]["n"], c[4]["d"], c[4]["threshold"], c[4]["planted"]) == (1048576, 128, 100.0, 100000)
    assert (c[5]["n"], c[5]["d"], c[5]["threshold"], c[5]["centers"]) == (524288, 64, 0.25, 1024)


# sha256 of the generated arrays (the bits every report's `inputs_sha256` names): guards the recipe against drift.
# Written from the generator itself; these are inputs, not results.
INPUT_SHA256 = {
    1: ("cc9e8c4d39b49eb4c8cf9f6e01a01ded4d4eedc5dc2df9230e9b522874e58c77",
        "0a4938c48a5f227fc5e45409c4087bee9ac569b0be4d7c6ba7daf800f06810e9"),
    2: ("42199fde961e89aa19e75611b773b392cb36065f437aa282f5e3a17643efcd93",
        "aec654e9d5d0adb86f0889852e8726f3f843342232ba2644f2b3d8ffbf716e5b"),
    3: ("615a900578b4d996839c4928cdcaaf400a55adedab8bba587e82da141721b549",
        "69ad8faef9a3425802989835650910d1406a9d2b52a407232d54c8252d1e4e32"),
    4: ("6b25980a41b34306e72f85aa50340e9b80c765df6112c6c81fb9165942c6d371",
        "823e1aca23c611d05517b00a278a3169fcdb7701fe3eb433d9fed01838d02b3d"),
    5: ("38545e49488b86ae623b11f7dde58b7cc309cbcfa8fa311a16564ebecf742e1d",
        "6092bca46ff31113246b175073696d709d362fb2aa4bd5055e7aa2bdac1e9537"),
}
SHA_SIZES = {1: {}, 2: {}, 3: dict(n=4096, m=4096, planted=64), 4: dict(n=4096, m=4096, planted=64), 5: dict(n=4096, m=4096)}


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_generated_inputs_have_the_recorded_hashes(cfg):
    import hashlib
    w = W.make_workload(cfg, **SHA_SIZES[cfg])
    assert (hashlib.sha256(w.P).hexdigest(), hashlib.sha256(w.Q).hexdigest()) == INPUT_SHA256[cfg]


def test_full_size_digest_file_is_well_formed_and_names_these_inputs():
    """The stored digests of the oracle's whole joins (tests/golden/full_size_digests.json): one entry per full-size
    configuration with the fields the GPU test reads, for the inputs this generator produces (configuration 2 is hashed
    at full size above; the GPU test regenerates and compares all four)."""
    import json
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "full_size_digests.json")) as f:
        g = json.load(f)
    assert sorted(g) == ["2", "3", "4", "5"]
    for cfg, e in g.items():
        c = W.CONFIGS[int(cfg)]
        assert (e["n"], e["m"], e["d"], e["threshold"]) == (c["n"], c["m"], c["d"], c["threshold"])
        assert len(e["inputs_sha256"]["P"]) == len(e["inputs_sha256"]["Q"]) == 64
        if e["dtype"] == "i8":
            assert e["count"] > 0 and len(e["sorted_keys_sha256"]) == 64
        else:
            assert e["strict_count"] <= e["exact_count"] <= e["loose_count"]
            assert len(e["band_pairs"]) == e["loose_count"] - e["strict_count"] and len(e["strict_sorted_keys_sha256"]) == 64
    assert (g["2"]["inputs_sha256"]["P"], g["2"]["inputs_sha256"]["Q"]) == INPUT_SHA256[2]
