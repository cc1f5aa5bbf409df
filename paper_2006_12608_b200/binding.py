"""ctypes binding of ``libsimjoin.so`` -- argument marshalling only.

Every step of the join runs in the library's CUDA kernels; this module converts
torch tensors / numpy arrays to pointers and sizes and maps status codes to
exceptions.  Function names mirror the C ABI in ``include/simjoin.h``.  There
is no CPU fallback: if the library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsimjoin.so")

SIMJOIN_I8, SIMJOIN_BF16 = 0, 1
SIMJOIN_IP, SIMJOIN_COS, SIMJOIN_L2 = 0, 1, 2
(SIMJOIN_OK, SIMJOIN_ERR_ARG, SIMJOIN_ERR_UNSUPPORTED, SIMJOIN_ERR_CAPACITY, SIMJOIN_ERR_CUDA,
 SIMJOIN_ERR_TIMEOUT, SIMJOIN_ERR_ARCH) = range(7)
DTYPE = {"i8": SIMJOIN_I8, "bf16": SIMJOIN_BF16}
KIND = {"ip": SIMJOIN_IP, "cos": SIMJOIN_COS, "l2": SIMJOIN_L2}
SIMJOIN_LSH_BITS, SIMJOIN_LSH_HYPERPLANES, SIMJOIN_LSH_BITS_IID = 0, 1, 2
LSH_FAMILY = {"bits": SIMJOIN_LSH_BITS, "hyperplanes": SIMJOIN_LSH_HYPERPLANES, "bits_iid": SIMJOIN_LSH_BITS_IID}

EXPORTS = ("simjoin_create", "simjoin_run", "simjoin_run_host", "simjoin_run_hamming", "simjoin_run_lsh", "simjoin_run_hamming_lsh", "simjoin_jl_transform", "simjoin_filter_pairs", "simjoin_run_jl_l2", "simjoin_row_norms", "simjoin_set_offsets", "simjoin_set_option",
           "simjoin_last_kernel_ms", "simjoin_run_noalloc", "simjoin_selftest_wait_timeout", "simjoin_destroy",
           "simjoin_strerror")
SIMJOIN_NOALLOC_MAX_ROWS = 65536
SIMJOIN_OPT_SELECT_MIN_OPS, SIMJOIN_OPT_KERNEL_TIMING, SIMJOIN_OPT_DENSE_EPILOGUE = 0, 1, 2

_lib = None


class SimjoinError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {strerror(status)} (status {int(status)})")


def load() -> ctypes.CDLL:
    """Load the library (once).  Raises if it has not been built: no fallback exists."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2006_12608_b200.build` "
                          "(nvcc, sm_100a). There is no CPU fallback.")
    lib = ctypes.CDLL(LIB_PATH)
    c = ctypes
    vp, i64, i32, u64, dbl = c.c_void_p, c.c_int64, c.c_int32, c.c_uint64, c.c_double
    lib.simjoin_create.restype = c.c_int
    lib.simjoin_create.argtypes = [c.POINTER(vp), c.c_int, c.c_int, vp]
    for name in ("simjoin_run", "simjoin_run_host"):
        fn = getattr(lib, name)
        fn.restype = c.c_int
        fn.argtypes = [vp, vp, i64, vp, i64, i32, c.c_int, dbl, vp, u64, c.POINTER(u64)]
    lib.simjoin_run_hamming.restype = c.c_int
    lib.simjoin_run_hamming.argtypes = [vp, vp, i64, vp, i64, i32, dbl, vp, u64, c.POINTER(u64)]
    lib.simjoin_run_lsh.restype = c.c_int
    lib.simjoin_run_lsh.argtypes = [vp, vp, i64, vp, i64, i32, c.c_int, dbl, c.c_int, i32, i32, i32, u64, vp, u64, c.POINTER(u64)]
    lib.simjoin_run_hamming_lsh.restype = c.c_int
    lib.simjoin_run_hamming_lsh.argtypes = [vp, vp, i64, vp, i64, i32, dbl, i32, i32, i32, u64, vp, u64, c.POINTER(u64)]
    lib.simjoin_jl_transform.restype = c.c_int
    lib.simjoin_jl_transform.argtypes = [vp, vp, i64, i32, i32, u64, vp]
    lib.simjoin_filter_pairs.restype = c.c_int
    lib.simjoin_filter_pairs.argtypes = [vp, vp, i64, vp, i64, i32, c.c_int, dbl, vp, u64, c.POINTER(u64)]
    lib.simjoin_run_jl_l2.restype = c.c_int
    lib.simjoin_run_jl_l2.argtypes = [vp, vp, i64, vp, i64, i32, dbl, i32, u64, dbl, vp, u64, c.POINTER(u64)]
    lib.simjoin_run_noalloc.restype = c.c_int
    lib.simjoin_run_noalloc.argtypes = [c.c_int, vp, c.c_int, vp, i64, vp, i64, i32, c.c_int, dbl, vp, u64, c.POINTER(u64)]
    lib.simjoin_row_norms.restype = c.c_int
    lib.simjoin_row_norms.argtypes = [vp, vp, i64, i32, vp]
    lib.simjoin_set_offsets.restype = c.c_int
    lib.simjoin_set_offsets.argtypes = [vp, i64, i64]
    lib.simjoin_set_option.restype = c.c_int
    lib.simjoin_set_option.argtypes = [vp, c.c_int, dbl]
    lib.simjoin_last_kernel_ms.restype = c.c_int
    lib.simjoin_last_kernel_ms.argtypes = [vp, c.POINTER(c.c_float), c.POINTER(c.c_float)]
    lib.simjoin_selftest_wait_timeout.restype = c.c_int
    lib.simjoin_selftest_wait_timeout.argtypes = [vp]
    lib.simjoin_destroy.restype = c.c_int
    lib.simjoin_destroy.argtypes = [vp]
    lib.simjoin_strerror.restype = c.c_char_p
    lib.simjoin_strerror.argtypes = [c.c_int]
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().simjoin_strerror(int(status)).decode()


def _ptr(x) -> Tuple[Optional[int], object]:
    """(address, keep-alive) of a torch tensor, numpy array, raw int address or None."""
    if x is None:
        return None, None
    if isinstance(x, int):
        return x, None
    if hasattr(x, "data_ptr"):
        return x.data_ptr(), x
    if hasattr(x, "ctypes"):
        return x.ctypes.data, x
    raise TypeError(f"cannot take the address of {type(x)}")


def simjoin_run_noalloc(device, stream, dtype, P, n, Q, m, d, kind, threshold, out_pairs, capacity):
    """The allocation-free entry point (no context): returns (status, count) without raising.
    For callers that may not allocate device memory while they run; rows are limited to
    SIMJOIN_NOALLOC_MAX_ROWS and overlapping calls on one device race on the shared scratch."""
    cnt = ctypes.c_uint64(0)
    (pp, _a), (qp, _b), (op, _c) = _ptr(P), _ptr(Q), _ptr(out_pairs)
    st = load().simjoin_run_noalloc(int(device), ctypes.c_void_p(stream), DTYPE[dtype] if isinstance(dtype, str) else dtype,
                                    pp, n, qp, m, d, KIND[kind] if isinstance(kind, str) else kind, float(threshold),
                                    op, capacity, ctypes.byref(cnt))
    return st, cnt.value


class Simjoin:
    """One library context: a dtype, a CUDA device and a stream."""

    def __init__(self, dtype: str = "i8", device: int = 0, stream: Optional[int] = None):
        lib = load()
        if stream is None:
            import torch
            stream = torch.cuda.current_stream(device).cuda_stream
        self._h = ctypes.c_void_p()
        self.dtype = dtype
        self.device = device
        st = lib.simjoin_create(ctypes.byref(self._h), DTYPE[dtype], int(device), ctypes.c_void_p(stream))
        if st != SIMJOIN_OK:
            self._h = ctypes.c_void_p()
            raise SimjoinError(st, "simjoin_create")

    # -- the C ABI, one method per entry point; each returns (status, ...) without raising
    def simjoin_run(self, P, n, Q, m, d, kind, threshold, out_pairs, capacity):
        cnt = ctypes.c_uint64(0)
        (pp, _a), (qp, _b), (op, _c) = _ptr(P), _ptr(Q), _ptr(out_pairs)
        st = load().simjoin_run(self._h, pp, n, qp, m, d, KIND[kind] if isinstance(kind, str) else kind,
                                float(threshold), op, capacity, ctypes.byref(cnt))
        return st, cnt.value

    def simjoin_run_host(self, P, n, Q, m, d, kind, threshold, out_pairs, capacity):
        cnt = ctypes.c_uint64(0)
        (pp, _a), (qp, _b), (op, _c) = _ptr(P), _ptr(Q), _ptr(out_pairs)
        st = load().simjoin_run_host(self._h, pp, n, qp, m, d, KIND[kind] if isinstance(kind, str) else kind,
                                     float(threshold), op, capacity, ctypes.byref(cnt))
        return st, cnt.value

    def simjoin_run_hamming(self, P_bits, n, Q_bits, m, d, r, out_pairs, capacity):
        cnt = ctypes.c_uint64(0)
        (pp, _a), (qp, _b), (op, _c) = _ptr(P_bits), _ptr(Q_bits), _ptr(out_pairs)
        st = load().simjoin_run_hamming(self._h, pp, n, qp, m, d, float(r), op, capacity, ctypes.byref(cnt))
        return st, cnt.value

    def simjoin_run_lsh(self, P, n, Q, m, d, threshold, L, k, seed, out_pairs, capacity, L_low=0, kind="ip", family="bits"):
        cnt = ctypes.c_uint64(0)
        (pp, _a), (qp, _b), (op, _c) = _ptr(P), _ptr(Q), _ptr(out_pairs)
        st = load().simjoin_run_lsh(self._h, pp, n, qp, m, d, KIND[kind] if isinstance(kind, str) else kind, float(threshold),
                                    LSH_FAMILY[family] if isinstance(family, str) else int(family),
                                    int(L), int(L_low), int(k), int(seed), op, capacity, ctypes.byref(cnt))
        return st, cnt.value

    def simjoin_run_hamming_lsh(self, P_bits, n, Q_bits, m, d, r, L, k, seed, out_pairs, capacity, L_low=0):
        cnt = ctypes.c_uint64(0)
        (pp, _a), (qp, _b), (op, _c) = _ptr(P_bits), _ptr(Q_bits), _ptr(out_pairs)
        st = load().simjoin_run_hamming_lsh(self._h, pp, n, qp, m, d, float(r), int(L), int(L_low), int(k), int(seed), op,
                                            capacity, ctypes.byref(cnt))
        return st, cnt.value

    def simjoin_jl_transform(self, X, n, d, k, seed, out):
        (xp, _a), (op, _b) = _ptr(X), _ptr(out)
        return load().simjoin_jl_transform(self._h, xp, n, d, k, int(seed), op)

    def simjoin_filter_pairs(self, P, n, Q, m, d, kind, threshold, pairs, count_in):
        cnt = ctypes.c_uint64(0)
        (pp, _a), (qp, _b), (lp, _c) = _ptr(P), _ptr(Q), _ptr(pairs)
        st = load().simjoin_filter_pairs(self._h, pp, n, qp, m, d, KIND[kind] if isinstance(kind, str) else kind,
                                         float(threshold), lp, count_in, ctypes.byref(cnt))
        return st, cnt.value

    def simjoin_run_jl_l2(self, P, n, Q, m, d, r, k, seed, slack, out_pairs, capacity):
        cnt = ctypes.c_uint64(0)
        (pp, _a), (qp, _b), (op, _c) = _ptr(P), _ptr(Q), _ptr(out_pairs)
        st = load().simjoin_run_jl_l2(self._h, pp, n, qp, m, d, float(r), k, int(seed), float(slack), op, capacity,
                                      ctypes.byref(cnt))
        return st, cnt.value

    def simjoin_row_norms(self, X, rows, d, out):
        (xp, _a), (op, _b) = _ptr(X), _ptr(out)
        return load().simjoin_row_norms(self._h, xp, rows, d, op)

    def simjoin_set_offsets(self, row_offset_p: int, row_offset_q: int):
        return load().simjoin_set_offsets(self._h, row_offset_p, row_offset_q)

    def simjoin_set_option(self, option: int, value: float):
        return load().simjoin_set_option(self._h, int(option), float(value))

    def simjoin_selftest_wait_timeout(self):
        return load().simjoin_selftest_wait_timeout(self._h)

    def simjoin_last_kernel_ms(self):
        a, b = ctypes.c_float(0), ctypes.c_float(0)
        st = load().simjoin_last_kernel_ms(self._h, ctypes.byref(a), ctypes.byref(b))
        return st, a.value, b.value

    # -- conveniences over the same calls
    def join(self, P, Q, kind: str, threshold: float, capacity: int, out=None):
        """Join two device tensors (rows x d; int8, or bfloat16 / int16 bit patterns).
        Returns (pairs[min(count, capacity), 2] int32 device tensor, count).
        Raises SimjoinError on any status other than OK / ERR_CAPACITY."""
        import torch
        n, d = P.shape
        m = Q.shape[0]
        if out is None:
            out = torch.empty((max(int(capacity), 1), 2), dtype=torch.int32, device=P.device)
        st, cnt = self.simjoin_run(P, n, Q, m, d, kind, threshold, out if capacity else None, capacity)
        if st not in (SIMJOIN_OK, SIMJOIN_ERR_CAPACITY):
            raise SimjoinError(st, "simjoin_run")
        return out[:min(cnt, capacity)], cnt

    def join_lsh(self, P, Q, threshold: float, L: int, k: int, seed: int, capacity: int, L_low: int = 0, out=None, kind: str = "ip",
                 family: str = "bits"):
        """LSH-bucketed join of two device tensors (simjoin_run_lsh).
        Returns (pairs[min(count, capacity), 2] int32 device tensor, count)."""
        import torch
        n, d = P.shape
        m = Q.shape[0]
        if out is None:
            out = torch.empty((max(int(capacity), 1), 2), dtype=torch.int32, device=P.device)
        st, cnt = self.simjoin_run_lsh(P, n, Q, m, d, threshold, L, k, seed, out if capacity else None, capacity, L_low=L_low, kind=kind,
                                       family=family)
        if st not in (SIMJOIN_OK, SIMJOIN_ERR_CAPACITY):
            raise SimjoinError(st, "simjoin_run_lsh")
        return out[:min(cnt, capacity)], cnt

    def jl_transform(self, X, k: int, seed: int, out=None):
        """JL transform of a bf16 device tensor (rows x d) to (rows x k) bf16 (simjoin_jl_transform)."""
        import torch
        n, d = X.shape
        if out is None:
            out = torch.empty((n, k), dtype=torch.bfloat16, device=X.device)
        st = self.simjoin_jl_transform(X, n, d, k, seed, out)
        if st != SIMJOIN_OK:
            raise SimjoinError(st, "simjoin_jl_transform")
        return out

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            load().simjoin_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()


def to_device(X, device="cuda:0"):
    """numpy int8 / uint16(bf16 bits) array -> device tensor with the same bytes."""
    import numpy as np
    import torch
    if X.dtype == np.uint16:
        return torch.from_numpy(X.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(X).to(device)
