"""ctypes loader for the CPU oracle (``gv_oracle.cpp``) -- TEST INFRASTRUCTURE ONLY.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this module.
It holds no arithmetic of its own: it compiles the C++ file beside it with the flags its header
states and marshals numpy arrays to it. The record layout is restated here (the oracle and the
CUDA library share no header).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gv_oracle.cpp")
_LIB = os.path.join(_HERE, "libgv_oracle.so")

# dtype codes of the oracle's own enum
F32, BF16, F16, I32, I64 = 0, 1, 2, 3, 4
ELEM_SIZE = {F32: 4, BF16: 2, F16: 2, I32: 4, I64: 8}

# 64-byte record as a numpy structured dtype (little-endian, no padding)
RESULT_DTYPE = np.dtype(
    [
        ("n_mismatch", "<u8"),
        ("first_mismatch", "<u8"),
        ("n_nan_disagree", "<u8"),
        ("n_inf_disagree", "<u8"),
        ("hash", "<u8"),
        ("max_abs_diff_int", "<u8"),
        ("max_abs_err", "<f4"),
        ("max_rel_err", "<f4"),
        ("reserved", "<u8"),
    ]
)
assert RESULT_DTYPE.itemsize == 64

NO_INDEX = 0xFFFFFFFFFFFFFFFF

PROFILE_BUCKETS = 66
PROFILE_LIST = 8
PROFILE_DTYPE = np.dtype(
    [
        ("ulp_hist", "<u8", (PROFILE_BUCKETS,)),
        ("n_mismatch", "<u8"),
        ("worst_index", "<u8"),
        ("worst_c_raw", "<u8"),
        ("worst_r_raw", "<u8"),
        ("n_first", "<u8"),
        ("first_index", "<u8", (PROFILE_LIST,)),
        ("first_c_raw", "<u8", (PROFILE_LIST,)),
        ("first_r_raw", "<u8", (PROFILE_LIST,)),
    ]
)
assert PROFILE_DTYPE.itemsize == 8 * (66 + 5 + 24)


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object beside its source (a second or two with g++)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = [
        "g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
        "-o", _LIB + ".tmp", _SRC,
    ]
    subprocess.run(cmd, check=True)
    os.replace(_LIB + ".tmp", _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.gvo_splitmix64.restype = ctypes.c_uint64
        L.gvo_splitmix64.argtypes = [ctypes.c_uint64]
        L.gvo_hash.restype = ctypes.c_uint64
        L.gvo_hash.argtypes = [ctypes.c_void_p, ctypes.c_uint64]
        L.gvo_hash2.restype = ctypes.c_uint64
        L.gvo_hash2.argtypes = [ctypes.c_void_p, ctypes.c_uint64]
        L.gvo_widen_bits.restype = ctypes.c_uint32
        L.gvo_widen_bits.argtypes = [ctypes.c_int, ctypes.c_uint32]
        L.gvo_verify.restype = ctypes.c_int
        L.gvo_verify.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int,
            ctypes.c_double, ctypes.c_double, ctypes.c_int, ctypes.c_void_p,
        ]
        L.gvo_verify_ragged.restype = ctypes.c_int
        L.gvo_verify_ragged.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.c_double, ctypes.c_int,
            ctypes.c_void_p,
        ]
        L.gvo_profile_pair.restype = ctypes.c_int
        L.gvo_profile_pair.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int, ctypes.c_double,
                                       ctypes.c_double, ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p]
        L.gvo_exec_summary.restype = ctypes.c_int
        L.gvo_exec_summary.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_void_p]
        L.gvo_speedup.restype = ctypes.c_int
        L.gvo_speedup.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.gvo_mem_efficiency.restype = ctypes.c_int
        L.gvo_mem_efficiency.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_double,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.gvo_accuracy_matrix.restype = ctypes.c_int
        L.gvo_accuracy_matrix.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.gvo_group.restype = ctypes.c_int
        L.gvo_group.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _lib = L
    return _lib


def _as_bytes_array(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    return a


def splitmix64(x: int) -> int:
    return int(lib().gvo_splitmix64(ctypes.c_uint64(x & NO_INDEX)))


def hash_bytes(a) -> int:
    """Content hash of a numpy array's byte image (or of a bytes object)."""
    if isinstance(a, (bytes, bytearray)):
        a = np.frombuffer(bytes(a), dtype=np.uint8)
    a = _as_bytes_array(a)
    return int(lib().gvo_hash(a.ctypes.data_as(ctypes.c_void_p), ctypes.c_uint64(a.nbytes)))


def hash2_bytes(a) -> int:
    """Second hash lane (word index multiplied by the odd constant before the xor)."""
    if isinstance(a, (bytes, bytearray)):
        a = np.frombuffer(bytes(a), dtype=np.uint8)
    a = _as_bytes_array(a)
    return int(lib().gvo_hash2(a.ctypes.data if a.size else None, a.nbytes))


def widen_bits(dtype: int, raw: int) -> int:
    return int(lib().gvo_widen_bits(dtype, raw))


def verify(ref: np.ndarray, cand: np.ndarray, dtype: int, atol: float = 0.0, rtol: float = 0.0,
           equal_nan: bool = False) -> np.ndarray:
    """One candidate against one reference; returns a 0-d structured record.

    ``ref`` / ``cand`` are numpy arrays whose bytes are the tensors (16-bit float types are
    passed as uint16 bit patterns); the element count is nbytes / element size.
    """
    ref = _as_bytes_array(ref)
    cand = _as_bytes_array(cand)
    assert ref.nbytes == cand.nbytes, "reference and candidate differ in size"
    n = ref.nbytes // ELEM_SIZE[dtype]
    out = np.zeros((), dtype=RESULT_DTYPE)
    rc = lib().gvo_verify(ref.ctypes.data_as(ctypes.c_void_p), cand.ctypes.data_as(ctypes.c_void_p),
                          ctypes.c_uint64(n), dtype, float(atol), float(rtol), int(bool(equal_nan)),
                          out.ctypes.data_as(ctypes.c_void_p))
    if rc != 0:
        raise ValueError(f"oracle rejected dtype {dtype}")
    return out


def verify_batch(ref: np.ndarray, cands, dtype: int, atol: float = 0.0, rtol: float = 0.0,
                 equal_nan: bool = False) -> np.ndarray:
    """N candidates against one reference: a plain loop over ``verify``."""
    out = np.zeros(len(cands), dtype=RESULT_DTYPE)
    for j, c in enumerate(cands):
        out[j] = verify(ref, c, dtype, atol, rtol, equal_nan)
    return out


def verify_ragged(ref_buf: np.ndarray, ref_off: np.ndarray, cand_buf: np.ndarray,
                  cand_off: np.ndarray, dtypes: np.ndarray, N: int, atol: float, rtol: float,
                  equal_nan: bool = False, n_elems: np.ndarray | None = None) -> np.ndarray:
    """Ragged batch (byte offsets; results tensor-major, shape [T*N]). ``n_elems`` (int64 [T])
    gives the element counts; without it they are read off consecutive ``ref_off`` entries."""
    ref_buf = _as_bytes_array(ref_buf)
    cand_buf = _as_bytes_array(cand_buf)
    ref_off = np.ascontiguousarray(ref_off, dtype=np.int64)
    cand_off = np.ascontiguousarray(cand_off, dtype=np.int64)
    dtypes = np.ascontiguousarray(dtypes, dtype=np.uint8)
    T = len(dtypes)
    assert ref_off.shape == (T + 1,) and cand_off.shape == (T * N,)
    ne_ptr = None
    if n_elems is not None:
        n_elems = np.ascontiguousarray(n_elems, dtype=np.int64)
        assert n_elems.shape == (T,)
        ne_ptr = n_elems.ctypes.data_as(ctypes.c_void_p)
    out = np.zeros(T * N, dtype=RESULT_DTYPE)
    rc = lib().gvo_verify_ragged(
        ref_buf.ctypes.data_as(ctypes.c_void_p), ref_off.ctypes.data_as(ctypes.c_void_p),
        cand_buf.ctypes.data_as(ctypes.c_void_p), cand_off.ctypes.data_as(ctypes.c_void_p),
        dtypes.ctypes.data_as(ctypes.c_void_p), ne_ptr, ctypes.c_int64(T), ctypes.c_int32(N),
        float(atol), float(rtol), int(bool(equal_nan)), out.ctypes.data_as(ctypes.c_void_p))
    if rc != 0:
        raise ValueError("oracle rejected a dtype code in the ragged batch")
    return out


def group(records: np.ndarray):
    """Duplicate groups of N result records -> (group_id[N] int32, group_count[N] int32, n_groups)."""
    rec = np.ascontiguousarray(records, dtype=RESULT_DTYPE)
    n = rec.shape[0]
    gid = np.zeros(max(n, 1), dtype=np.int32)
    cnt = np.zeros(max(n, 1), dtype=np.int32)
    ng = np.zeros(1, dtype=np.int32)
    rc = lib().gvo_group(rec.ctypes.data, n, gid.ctypes.data, cnt.ctypes.data, ng.ctypes.data)
    if rc:
        raise RuntimeError(f"gvo_group failed with {rc}")
    return gid[:n], cnt[:n], int(ng[0])


def profile(ref: np.ndarray, cand: np.ndarray, dtype: int, atol: float = 0.0, rtol: float = 0.0,
            equal_nan: bool = False, row_len: int = 0):
    """Error profile of one candidate -> (PROFILE_DTYPE scalar, per-row mismatch counts or None)."""
    r, c = _as_bytes_array(ref), _as_bytes_array(cand)
    assert r.nbytes == c.nbytes and r.nbytes % ELEM_SIZE[dtype] == 0
    n = r.nbytes // ELEM_SIZE[dtype]
    out = np.zeros(1, dtype=PROFILE_DTYPE)
    rows = np.zeros(max(1, (n + row_len - 1) // row_len), dtype=np.uint32) if row_len else None
    rc = lib().gvo_profile_pair(r.ctypes.data, c.ctypes.data, n, dtype, atol, rtol, int(equal_nan), row_len,
                                out.ctypes.data, rows.ctypes.data if rows is not None else None)
    if rc:
        raise RuntimeError(f"gvo_profile_pair failed with {rc}")
    if rows is not None:
        rows = rows[:(n + row_len - 1) // row_len]
    return out[0], rows


def exec_summary(records: np.ndarray, T: int, N: int, kmax: int):
    """(pass[N] uint8, n_pass, pass_at_k[kmax] float64) for T x N tensor-major records."""
    rec = np.ascontiguousarray(records, dtype=RESULT_DTYPE)
    assert rec.shape[0] == T * N
    ok = np.zeros(max(N, 1), dtype=np.uint8)
    c = np.zeros(1, dtype=np.int32)
    pk = np.zeros(max(kmax, 1), dtype=np.float64)
    rc = lib().gvo_exec_summary(rec.ctypes.data, T, N, kmax, ok.ctypes.data, c.ctypes.data, pk.ctypes.data)
    if rc:
        raise RuntimeError(f"gvo_exec_summary failed with {rc}")
    return ok[:N], int(c[0]), pk[:kmax]


def speedup(ref_lat: np.ndarray, gen_lat: np.ndarray):
    """(median_ref[T], median_gen[T], ratio[T] float32, speedup float64) for T x S latency samples."""
    a = np.ascontiguousarray(ref_lat, dtype=np.float32)
    b = np.ascontiguousarray(gen_lat, dtype=np.float32)
    T = a.shape[0]
    assert a.ndim == 2 and b.ndim == 2 and b.shape[0] == T
    mr, mg, ra = (np.zeros(max(T, 1), dtype=np.float32) for _ in range(3))
    sp = np.zeros(1, dtype=np.float64)
    rc = lib().gvo_speedup(a.ctypes.data, b.ctypes.data, T, a.shape[1], b.shape[1], mr.ctypes.data, mg.ctypes.data,
                           ra.ctypes.data, sp.ctypes.data)
    if rc:
        raise RuntimeError(f"gvo_speedup failed with {rc}")
    return mr[:T], mg[:T], ra[:T], float(sp[0])


def mem_efficiency(lat: np.ndarray, nbytes: np.ndarray, peak: float):
    """(median[T] float32, bandwidth[T], efficiency[T] float64, mean efficiency) for T x S latency samples,
    the bytes each unit test has to move and the peak bandwidth in bytes per latency unit."""
    a = np.ascontiguousarray(lat, dtype=np.float32)
    b = np.ascontiguousarray(nbytes, dtype=np.uint64)
    T = a.shape[0]
    assert a.ndim == 2 and b.shape == (T,)
    med = np.zeros(max(T, 1), dtype=np.float32)
    bw, eff = (np.zeros(max(T, 1), dtype=np.float64) for _ in range(2))
    mean = np.zeros(1, dtype=np.float64)
    rc = lib().gvo_mem_efficiency(a.ctypes.data, b.ctypes.data, T, a.shape[1], float(peak), med.ctypes.data,
                                  bw.ctypes.data, eff.ctypes.data, mean.ctypes.data)
    if rc:
        raise ValueError(f"gvo_mem_efficiency rejected its arguments ({rc})")
    return med[:T], bw[:T], eff[:T], float(mean[0])


def accuracy_matrix(status: np.ndarray, kmax: int):
    """(n_call[K], n_exec[K] int32, call_acc[kmax], exec_acc[kmax] float64) for a K x R uint8 status matrix
    (bit 0: the run compiled and ran, bit 1: it satisfied all unit tests)."""
    s = np.ascontiguousarray(status, dtype=np.uint8)
    assert s.ndim == 2
    K, R = s.shape
    nc, ne = (np.zeros(max(K, 1), dtype=np.int32) for _ in range(2))
    ca, ea = (np.zeros(max(kmax, 1), dtype=np.float64) for _ in range(2))
    rc = lib().gvo_accuracy_matrix(s.ctypes.data, K, R, kmax, nc.ctypes.data, ne.ctypes.data, ca.ctypes.data,
                                   ea.ctypes.data)
    if rc:
        raise ValueError(f"gvo_accuracy_matrix rejected its arguments ({rc})")
    return nc[:K], ne[:K], ca[:kmax], ea[:kmax]
