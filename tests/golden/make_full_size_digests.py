"""Writes full_size_digests.json: the CPU oracle's WHOLE join of the full-size benchmark configurations, as digests.

For every configuration the script regenerates the seeded inputs, runs the oracle's plain double loop over all n x m
pairs (minutes to an hour of host time per configuration) and stores

  - the sha256 of the input arrays,
  - int8 configurations: the number of pairs and the sha256 of the sorted pair keys ((i << 32) | j as little-endian
    int64), i.e. of the exact result,
  - bf16 configurations: the same for the join at the threshold moved by 1 % towards fewer pairs (the strict set)
    and the list of pairs that only the threshold moved by 1 % towards more pairs admits (the band); a floating-point
    join G is right when G minus the band equals the strict set.

It calls the oracle and the shared input generator only; nothing here comes from the CUDA library.

    python tests/golden/make_full_size_digests.py [--configs 2 3 4 5] [--threads N]
"""
import argparse
import hashlib
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import simjoin_oracle as O                      # noqa: E402
from paper_2006_12608_b200 import workloads as W            # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "full_size_digests.json")
BAND_REL = 1e-2
CAPACITY = 300_000_000          # one pass of the oracle: room for the densest configuration (2.7e8 pairs, 2.4 GB)


def keys(pairs):
    p = np.asarray(pairs, dtype=np.int64).reshape(-1, 2)
    return (p[:, 0] << 32) | p[:, 1]


def digest(sorted_keys):
    return hashlib.sha256(np.ascontiguousarray(sorted_keys, dtype="<i8").tobytes()).hexdigest()


def one_config(cfg, threads):
    w = W.make_workload(cfg)
    entry = {"workload": w.name, "n": w.n, "m": w.m, "d": w.d, "kind": w.kind, "dtype": w.dtype, "threshold": w.threshold,
             "inputs_sha256": {"P": hashlib.sha256(w.P.tobytes()).hexdigest(), "Q": hashlib.sha256(w.Q.tobytes()).hexdigest()}}
    t0 = time.time()
    if w.dtype == "i8":
        pairs, count = O.join(w.P, w.Q, w.kind, w.threshold, w.dtype, capacity=CAPACITY, threads=threads)
        assert count <= CAPACITY
        entry["oracle_seconds"] = round(time.time() - t0, 1)
        k = np.sort(keys(pairs))
        assert len(k) == count and (len(k) < 2 or (np.diff(k) > 0).all())
        entry.update({"count": int(count), "sorted_keys_sha256": digest(k)})
    else:
        t = float(w.threshold)
        delta = BAND_REL * abs(t)
        strict_t, loose_t = (t - delta, t + delta) if w.kind == "l2" else (t + delta, t - delta)
        loose, count = O.join(w.P, w.Q, w.kind, loose_t, w.dtype, capacity=CAPACITY, threads=threads)
        assert count <= CAPACITY
        entry["oracle_seconds"] = round(time.time() - t0, 1)
        # split the loose set by the oracle's own scores (one pass over its pairs instead of two more joins)
        s = O.scores(w.P, w.Q, w.kind, w.dtype, loose)
        in_strict = s <= strict_t if w.kind == "l2" else s >= strict_t
        in_exact = s <= t if w.kind == "l2" else s >= t
        ks = np.sort(keys(loose[in_strict]))
        band = loose[~in_strict]
        band = band[np.argsort(keys(band))]
        assert len(band) <= 100000, "band too large to store as a list"
        entry.update({"band_rel": BAND_REL, "strict_count": int(len(ks)), "strict_sorted_keys_sha256": digest(ks),
                      "exact_count": int(in_exact.sum()), "loose_count": int(len(loose)), "band_pairs": band.tolist()})
    entry["oracle_threads"] = threads or O.max_threads()
    return entry


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", type=int, nargs="+", default=[2, 3, 4, 5])
    ap.add_argument("--threads", type=int, default=0)
    a = ap.parse_args()
    O.build()
    data = json.load(open(OUT)) if os.path.exists(OUT) else {}
    for cfg in a.configs:
        e = one_config(cfg, a.threads)
        data[str(cfg)] = e
        with open(OUT, "w") as f:
            json.dump(data, f, indent=1, sort_keys=True)
            f.write("\n")
        print(cfg, {k: v for k, v in e.items() if k != "band_pairs"}, "band", len(e.get("band_pairs", [])), flush=True)


if __name__ == "__main__":
    main()
