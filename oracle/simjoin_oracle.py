"""ctypes front end of the CPU oracle (``simjoin_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
benchmark's cpu_baseline / reference legs may import this module.  It imports
nothing from the CUDA package and the CUDA package imports nothing from here.

The C file is the oracle: the join's definition (Section 4 of the paper) as a
plain double loop in exact integer / fp64 arithmetic.  This module only builds
it with gcc on first use, marshals numpy arrays and derives the band sets used
to compare floating-point joins (a pure re-run of the same oracle at a shifted
threshold).
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from typing import Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "simjoin_oracle.c")
KIND = {"ip": 0, "cos": 1, "l2": 2}
_lib = None


def _cpu_tag() -> str:
    """Short tag of the host CPU so a library built with -march=native on one
    machine is never loaded on a different one."""
    try:
        with open("/proc/cpuinfo") as f:
            txt = f.read()
        lines = [l for l in txt.splitlines() if l.startswith(("model name", "flags"))][:2]
        return hashlib.sha1("\n".join(lines).encode()).hexdigest()[:10]
    except OSError:
        return "generic"


def lib_path() -> str:
    return os.path.join(_HERE, f"liboracle_simjoin_{_cpu_tag()}.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O3 -march=native -fopenmp); returns the .so path."""
    out = lib_path()
    if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
        return out
    tmp = out + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, out)
    return out


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c = ctypes
    vp, i64, i32, dbl = c.c_void_p, c.c_int64, c.c_int32, c.c_double
    for name in ("oracle_join_i8", "oracle_join_bf16"):
        fn = getattr(lib, name)
        fn.restype = i64
        fn.argtypes = [vp, i64, vp, i64, i32, i32, dbl, vp, i64, i32]
    lib.oracle_join_hamming_bits.restype = i64
    lib.oracle_join_hamming_bits.argtypes = [vp, i64, vp, i64, i32, dbl, vp, i64, i32]
    lib.oracle_hamming_bits.restype = i64
    lib.oracle_hamming_bits.argtypes = [vp, vp, i32]
    lib.oracle_lsh_join_i8.restype = i64
    lib.oracle_lsh_join_i8.argtypes = [vp, i64, vp, i64, i32, dbl, i32, i32, i32, c.c_uint64, vp, i64, i32]
    lib.oracle_lsh_keys_i8.restype = None
    lib.oracle_lsh_keys_i8.argtypes = [vp, i64, i32, i32, i32, i32, c.c_uint64, vp]
    lib.oracle_lsh_keys_bf16.restype = None
    lib.oracle_lsh_keys_bf16.argtypes = [vp, i64, i32, i32, i32, i32, c.c_uint64, vp]
    lib.oracle_lsh_hp_sign.restype = i32
    lib.oracle_lsh_hp_sign.argtypes = [c.c_uint64, i32, i32, i32]
    lib.oracle_lsh_keys_hp_i8.restype = None
    lib.oracle_lsh_keys_hp_i8.argtypes = [vp, i64, i32, i32, i32, i32, c.c_uint64, vp]
    lib.oracle_lsh_keys_hp_bf16.restype = None
    lib.oracle_lsh_keys_hp_bf16.argtypes = [vp, i64, i32, i32, i32, i32, c.c_uint64, dbl, vp, vp]
    lib.oracle_lsh_set_iid_sampling.restype = None
    lib.oracle_lsh_set_iid_sampling.argtypes = [i32]
    lib.oracle_lsh_coordinate.restype = i32
    lib.oracle_lsh_coordinate.argtypes = [c.c_uint64, i32, i32, i32]
    lib.oracle_jl_levels.restype = i32
    lib.oracle_jl_levels.argtypes = [i32, i32]
    lib.oracle_jl_shape.restype = i32
    lib.oracle_jl_shape.argtypes = [i32, i32, i32, c.POINTER(i32), c.POINTER(i32), c.POINTER(i32)]
    lib.oracle_jl_sign.restype = i32
    lib.oracle_jl_sign.argtypes = [c.c_uint64, i32, i64, i64, i32]
    lib.oracle_jl_transform_bf16.restype = i32
    lib.oracle_jl_transform_bf16.argtypes = [vp, i64, i32, i32, c.c_uint64, vp]
    lib.oracle_scores_i8.restype = i32
    lib.oracle_scores_i8.argtypes = [vp, vp, i32, i32, vp, i64, vp]
    lib.oracle_scores_cos_i8.restype = i32
    lib.oracle_scores_cos_i8.argtypes = [vp, vp, i32, vp, i64, vp]
    lib.oracle_scores_bf16.restype = i32
    lib.oracle_scores_bf16.argtypes = [vp, vp, i32, i32, vp, i64, vp]
    lib.oracle_sq_norms_bf16.restype = None
    lib.oracle_sq_norms_bf16.argtypes = [vp, i64, i32, vp]
    lib.oracle_sq_norms_i8.restype = None
    lib.oracle_sq_norms_i8.argtypes = [vp, i64, i32, vp]
    lib.oracle_max_threads.restype = i32
    lib.oracle_max_threads.argtypes = []
    _lib = lib
    return lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def _check(X: np.ndarray, dtype: str) -> np.ndarray:
    want = np.int8 if dtype == "i8" else np.uint16
    if X.dtype != want or X.ndim != 2:
        raise TypeError(f"expected 2-D {want.__name__} array for dtype {dtype}, got {X.dtype} ndim {X.ndim}")
    return np.ascontiguousarray(X)


def join(P: np.ndarray, Q: np.ndarray, kind: str, threshold: float, dtype: str,
         capacity: int | None = None, threads: int = 0) -> Tuple[np.ndarray, int]:
    """All (i, j) with score(P[i], Q[j]) >= threshold (ip, cos) or
    distance <= threshold (l2), sorted by (i, j).

    Returns (pairs[min(count, capacity), 2] int32, count).  With capacity=None
    the call is repeated with a larger buffer until everything fits.
    """
    lib = _load()
    P = _check(P, dtype)
    Q = _check(Q, dtype)
    n, d = P.shape
    m, d2 = Q.shape
    if d != d2:
        raise ValueError("P and Q must have the same number of columns")
    fn = lib.oracle_join_i8 if dtype == "i8" else lib.oracle_join_bf16
    cap = 1 << 16 if capacity is None else int(capacity)
    while True:
        out = np.empty((max(cap, 1), 2), dtype=np.int32)
        cnt = fn(P.ctypes.data, n, Q.ctypes.data, m, d, KIND[kind], float(threshold),
                 out.ctypes.data, cap, threads)
        if cnt < 0:
            raise ValueError("oracle rejected the arguments")
        if capacity is not None or cnt <= cap:
            return out[:min(cnt, cap)].copy(), int(cnt)
        cap = int(cnt)


def join_hamming(Pbits: np.ndarray, Qbits: np.ndarray, d: int, r: float, threads: int = 0):
    """All (i, j) with Hamming(P[i], Q[j]) <= r over bit-packed uint8 rows (d/8 bytes per row, bit k%8 of
    byte k/8 is coordinate k), sorted by (i, j).  Returns (pairs, count)."""
    lib = _load()
    if Pbits.dtype != np.uint8 or Qbits.dtype != np.uint8 or Pbits.ndim != 2 or Qbits.ndim != 2:
        raise TypeError("expected 2-D uint8 arrays of packed bits")
    if Pbits.shape[1] * 8 != d or Qbits.shape[1] * 8 != d:
        raise ValueError("rows must hold d/8 bytes")
    Pbits, Qbits = np.ascontiguousarray(Pbits), np.ascontiguousarray(Qbits)
    cap = 1 << 16
    while True:
        out = np.empty((cap, 2), dtype=np.int32)
        cnt = lib.oracle_join_hamming_bits(Pbits.ctypes.data, Pbits.shape[0], Qbits.ctypes.data, Qbits.shape[0], d,
                                           float(r), out.ctypes.data, cap, threads)
        if cnt < 0:
            raise ValueError("oracle rejected the arguments")
        if cnt <= cap:
            return out[:cnt].copy(), int(cnt)
        cap = int(cnt)


def hamming(x: np.ndarray, y: np.ndarray, d: int) -> int:
    """Hamming distance of two bit-packed rows."""
    x, y = np.ascontiguousarray(x, dtype=np.uint8), np.ascontiguousarray(y, dtype=np.uint8)
    return int(_load().oracle_hamming_bits(x.ctypes.data, y.ctypes.data, d))


def lsh_join(P: np.ndarray, Q: np.ndarray, threshold: float, L: int, k: int, seed: int, threads: int = 0, L_low: int = 0):
    """The LSH-bucketed inner-product join over int8 rows with bit-sampling hashes: all (i, j) of the
    brute-force join whose hashes agree in at least one repetition -- L repetitions of k bits followed by
    L_low repetitions of k - 1 bits.  Returns (pairs, count)."""
    lib = _load()
    P, Q = _check(P, "i8"), _check(Q, "i8")
    n, d = P.shape
    m = Q.shape[0]
    cap = 1 << 16
    while True:
        out = np.empty((cap, 2), dtype=np.int32)
        cnt = lib.oracle_lsh_join_i8(P.ctypes.data, n, Q.ctypes.data, m, d, float(threshold), L, L_low, k, seed,
                                     out.ctypes.data, cap, threads)
        if cnt < 0:
            raise ValueError("oracle rejected the arguments")
        if cnt <= cap:
            return out[:cnt].copy(), int(cnt)
        cap = int(cnt)


def lsh_join_hamming(Pbits: np.ndarray, Qbits: np.ndarray, d: int, r: float, L: int, k: int, seed: int, threads: int = 0,
                     L_low: int = 0):
    """The LSH-bucketed Hamming join on bit-packed rows: the points are widened to +-1 rows (x -> 2x - 1, the operand
    transform of the Hamming ip-distance), on which <x, y> = d - 2 Hamming(x, y) and the bit-sampling hash [x_c > 0] is
    the sampled bit itself; then lsh_join with threshold d - 2 floor(r).  Returns (pairs, count)."""
    def widen(b):
        bits = np.unpackbits(np.ascontiguousarray(b), axis=1, bitorder="little")[:, :d]
        return (2 * bits.astype(np.int8) - 1).astype(np.int8)
    return lsh_join(widen(Pbits), widen(Qbits), float(d) - 2.0 * np.floor(r), L, k, seed, threads=threads, L_low=L_low)


FAMILIES = ("bits", "hyperplanes", "bits_iid")


def hp_tolerance(d: int) -> float:
    """Relative size (to sum |x_c|) below which an fp32 accumulation of d exact products, in any order and with the
    tensor core's internal truncation, may decide the sign of a hyperplane projection differently from fp64."""
    return (d + 64) * 2.0 ** -23


def lsh_keys(X: np.ndarray, L: int, k: int, seed: int, L_low: int = 0, dtype: str = "i8", family: str = "bits") -> np.ndarray:
    """(L + L_low, rows) uint32 hash keys.  family "bits": bit b = [x_c > 0] at the sampled coordinate (int8 rows or
    bf16 bit patterns), the k coordinates of a repetition distinct; "bits_iid": the same with k independent samples
    (the paper's plain concatenation of base hashes); "hyperplanes": bit b = [<a, x> > 0] for a random-sign vector a."""
    lib = _load()
    X = _check(X, dtype)
    out = np.empty((L + L_low, X.shape[0]), dtype=np.uint32)
    if family in ("bits", "bits_iid"):
        fn = lib.oracle_lsh_keys_i8 if dtype == "i8" else lib.oracle_lsh_keys_bf16
        lib.oracle_lsh_set_iid_sampling(1 if family == "bits_iid" else 0)       # k independent samples, or k distinct ones
        try:
            fn(X.ctypes.data, X.shape[0], X.shape[1], L, L_low, k, seed, out.ctypes.data)
        finally:
            lib.oracle_lsh_set_iid_sampling(0)
    elif family == "hyperplanes":
        if dtype == "i8":
            lib.oracle_lsh_keys_hp_i8(X.ctypes.data, X.shape[0], X.shape[1], L, L_low, k, seed, out.ctypes.data)
        else:
            lib.oracle_lsh_keys_hp_bf16(X.ctypes.data, X.shape[0], X.shape[1], L, L_low, k, seed, 0.0, out.ctypes.data, None)
    else:
        raise ValueError(family)
    return out


def lsh_keys_unsure(X: np.ndarray, L: int, k: int, seed: int, L_low: int = 0, tol: float | None = None):
    """Hyperplane keys of bf16 rows and, per repetition and row, the mask of the bits whose projection is within
    tol * sum |x_c| of zero (default tol: hp_tolerance(d)): (keys, unsure), both (L + L_low, rows) uint32."""
    lib = _load()
    X = _check(X, "bf16")
    keys = np.empty((L + L_low, X.shape[0]), dtype=np.uint32)
    unsure = np.empty_like(keys)
    lib.oracle_lsh_keys_hp_bf16(X.ctypes.data, X.shape[0], X.shape[1], L, L_low, k, seed,
                                hp_tolerance(X.shape[1]) if tol is None else float(tol), keys.ctypes.data, unsure.ctypes.data)
    return keys, unsure


def hp_sign(seed: int, rep: int, bit: int, c: int) -> int:
    return int(_load().oracle_lsh_hp_sign(seed, rep, bit, c))


def lsh_restrict(pairs: np.ndarray, P: np.ndarray, Q: np.ndarray, dtype: str, L: int, k: int, seed: int, L_low: int = 0,
                 family: str = "bits", unsure: str | None = None) -> np.ndarray:
    """The pairs of a (brute-force) join whose hash keys agree in at least one repetition: what the LSH-bucketed join of
    any kind returns, since it runs the brute-force join inside the buckets of every repetition and takes the union.
    bf16 hyperplane keys depend on floating-point signs: unsure="strict" keeps a pair only if some repetition's keys
    agree with no bit of either point in doubt, unsure="loose" if some repetition's keys agree on every bit that is
    not in doubt -- any correct fp32 implementation returns a set between the two."""
    pairs = np.asarray(pairs).reshape(-1, 2)
    if len(pairs) == 0:
        return pairs
    if unsure is None or family != "hyperplanes" or dtype != "bf16":
        kp, kq = lsh_keys(P, L, k, seed, L_low, dtype, family), lsh_keys(Q, L, k, seed, L_low, dtype, family)
        keep = (kp[:, pairs[:, 0]] == kq[:, pairs[:, 1]]).any(axis=0)
        return pairs[keep]
    (kp, up), (kq, uq) = lsh_keys_unsure(P, L, k, seed, L_low), lsh_keys_unsure(Q, L, k, seed, L_low)
    diff = kp[:, pairs[:, 0]] ^ kq[:, pairs[:, 1]]
    free = up[:, pairs[:, 0]] | uq[:, pairs[:, 1]]
    if unsure == "strict":
        keep = ((diff == 0) & (free == 0)).any(axis=0)
    elif unsure == "loose":
        keep = ((diff & ~free) == 0).any(axis=0)
    else:
        raise ValueError(unsure)
    return pairs[keep]


def lsh_join_kind(P, Q, kind: str, threshold: float, dtype: str, L: int, k: int, seed: int, L_low: int = 0, threads: int = 0,
                  family: str = "bits"):
    """LSH-bucketed join of any kind, element type and hash family: the brute-force join restricted to colliding pairs."""
    pairs, _c = join(P, Q, kind, threshold, dtype, threads=threads)
    out = lsh_restrict(pairs, P, Q, dtype, L, k, seed, L_low, family)
    return out, len(out)


def lsh_band_sets(P, Q, kind: str, threshold: float, dtype: str, L: int, k: int, seed: int, L_low: int = 0, rel: float = 1e-2,
                  family: str = "bits"):
    """band_sets restricted to colliding pairs: a floating-point LSH join G is accepted when S_strict <= G <= S_loose
    (hyperplane keys of bf16 rows: the strict set also needs a collision with no bit in doubt, the loose set accepts
    one on the bits that are not in doubt)."""
    s_strict, s_exact, s_loose = band_sets(P, Q, kind, threshold, dtype, rel=rel)
    hp = family == "hyperplanes" and dtype == "bf16"
    return (lsh_restrict(s_strict, P, Q, dtype, L, k, seed, L_low, family, "strict" if hp else None),
            lsh_restrict(s_exact, P, Q, dtype, L, k, seed, L_low, family),
            lsh_restrict(s_loose, P, Q, dtype, L, k, seed, L_low, family, "loose" if hp else None))


def lsh_coordinate(seed: int, rep: int, bit: int, d: int) -> int:
    return int(_load().oracle_lsh_coordinate(seed, rep, bit, d))


def jl_shapes(d: int, k: int):
    """[(r_i, c_i, k_i)] for the levels i = 1..l of the JL construction with zeta = 2; raises if d/k is not 2^l, l >= 1."""
    lib = _load()
    levels = lib.oracle_jl_levels(d, k)
    if levels < 1:
        raise ValueError("d / k must be a power of two >= 2")
    out = []
    for i in range(1, levels + 1):
        r, c, ko = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        lib.oracle_jl_shape(d, k, i, ctypes.byref(r), ctypes.byref(c), ctypes.byref(ko))
        out.append((r.value, c.value, ko.value))
    return out


def jl_sign_matrix(seed: int, level: int, k_i: int, c_i: int) -> np.ndarray:
    """The +-1 entries of A_level (k_i x c_i), unscaled."""
    lib = _load()
    return np.array([[lib.oracle_jl_sign(seed, level, a, b, c_i) for b in range(c_i)] for a in range(k_i)], dtype=np.int8)


def jl_transform(X: np.ndarray, k: int, seed: int) -> np.ndarray:
    """M x for every row x of X (bf16 bit patterns, rows x d) -> (rows, k) float64."""
    lib = _load()
    X = _check(X, "bf16")
    rows, d = X.shape
    out = np.empty((rows, k), dtype=np.float64)
    if lib.oracle_jl_transform_bf16(X.ctypes.data, rows, d, k, seed, out.ctypes.data) != 0:
        raise ValueError("oracle rejected the arguments (d / k must be a power of two >= 2)")
    return out


def band_sets(P, Q, kind, threshold, dtype, rel: float = 1e-2, threads: int = 0):
    """(S_strict, S_exact, S_loose): the join at the threshold moved by rel*|t|
    towards fewer pairs, at the threshold itself, and moved towards more pairs.
    A floating-point join G is accepted when S_strict <= G <= S_loose."""
    t = float(threshold)
    delta = rel * abs(t)
    if kind == "l2":
        strict_t, loose_t = t - delta, t + delta
    else:
        strict_t, loose_t = t + delta, t - delta
    s_strict, _ = join(P, Q, kind, strict_t, dtype, threads=threads)
    s_exact, _ = join(P, Q, kind, t, dtype, threads=threads)
    s_loose, _ = join(P, Q, kind, loose_t, dtype, threads=threads)
    return s_strict, s_exact, s_loose


def scores(P, Q, kind: str, dtype: str, pairs: np.ndarray) -> np.ndarray:
    """Score of each listed (i, j): int64 inner product / squared distance and fp64 cosine for
    int8 rows, fp64 inner product / cosine / distance for bf16 rows."""
    lib = _load()
    P = _check(P, dtype)
    Q = _check(Q, dtype)
    pairs = np.ascontiguousarray(pairs, dtype=np.int32).reshape(-1, 2)
    d = P.shape[1]
    if len(pairs) and (pairs[:, 0].max() >= P.shape[0] or pairs[:, 1].max() >= Q.shape[0] or pairs.min() < 0):
        raise IndexError("pair index out of range")
    if dtype == "i8" and kind == "cos":
        out = np.empty(len(pairs), dtype=np.float64)
        rc = lib.oracle_scores_cos_i8(P.ctypes.data, Q.ctypes.data, d, pairs.ctypes.data, len(pairs), out.ctypes.data)
    elif dtype == "i8":
        out = np.empty(len(pairs), dtype=np.int64)
        rc = lib.oracle_scores_i8(P.ctypes.data, Q.ctypes.data, d, KIND[kind], pairs.ctypes.data, len(pairs), out.ctypes.data)
    else:
        out = np.empty(len(pairs), dtype=np.float64)
        rc = lib.oracle_scores_bf16(P.ctypes.data, Q.ctypes.data, d, KIND[kind], pairs.ctypes.data, len(pairs), out.ctypes.data)
    if rc != 0:
        raise ValueError("oracle rejected the arguments")
    return out


def filter_pairs(P, Q, kind: str, threshold: float, dtype: str, pairs: np.ndarray) -> np.ndarray:
    """The listed pairs that pass: Section 4's join predicate applied pair by pair (same decisions as `join`)."""
    pairs = np.ascontiguousarray(pairs, dtype=np.int32).reshape(-1, 2)
    sc = scores(P, Q, kind, dtype, pairs)
    if kind == "l2":
        keep = sc.astype(np.float64) <= (float(threshold) * float(threshold) if dtype == "i8" else float(threshold))
    else:
        keep = sc.astype(np.float64) >= float(threshold)
    return pairs[keep]


def sq_norms(X: np.ndarray, dtype: str) -> np.ndarray:
    """Row squared norms: exact int64 (int8 rows) or fp64 (bf16 rows)."""
    lib = _load()
    X = _check(X, dtype)
    if dtype == "i8":
        out = np.empty(X.shape[0], dtype=np.int64)
        lib.oracle_sq_norms_i8(X.ctypes.data, X.shape[0], X.shape[1], out.ctypes.data)
    else:
        out = np.empty(X.shape[0], dtype=np.float64)
        lib.oracle_sq_norms_bf16(X.ctypes.data, X.shape[0], X.shape[1], out.ctypes.data)
    return out


def pairs_to_set(pairs: np.ndarray) -> np.ndarray:
    """Encode (i, j) rows as sorted unique int64 keys i*2^32 + j (for set algebra)."""
    p = np.asarray(pairs, dtype=np.int64).reshape(-1, 2)
    return np.unique((p[:, 0] << 32) | p[:, 1])
