"""Thin Python binding of the C ABI in ``include/gv.h`` (argument marshalling only).

Every function here has the name and meaning of the C entry point it wraps; all computation runs
in the CUDA kernels of ``libgv.so``. PyTorch only supplies device memory (``data_ptr()``) and the
current stream. There is no CPU fallback: if the library is missing, importing this module fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

GV_F32, GV_BF16, GV_F16, GV_I32, GV_I64 = 0, 1, 2, 3, 4
GV_OK = 0
GV_ERR_INVALID_ARG, GV_ERR_UNSUPPORTED, GV_ERR_MISALIGNED, GV_ERR_WORKSPACE = 1, 2, 3, 4
GV_ERR_CUDA, GV_ERR_DEVICE_TIMEOUT, GV_ERR_BAD_TABLE = 5, 6, 7
GV_NO_INDEX = 0xFFFFFFFFFFFFFFFF

DTYPE_OF = {torch.float32: GV_F32, torch.bfloat16: GV_BF16, torch.float16: GV_F16,
            torch.int32: GV_I32, torch.int64: GV_I64}

#: gv_result as a numpy structured dtype (64 bytes)
RESULT_DTYPE = np.dtype([
    ("n_mismatch", "<u8"), ("first_mismatch", "<u8"), ("n_nan_disagree", "<u8"), ("n_inf_disagree", "<u8"),
    ("hash", "<u8"), ("max_abs_diff_int", "<u8"), ("max_abs_err", "<f4"), ("max_rel_err", "<f4"),
    ("reserved", "<u8")])
assert RESULT_DTYPE.itemsize == 64

#: gv_profile as a numpy structured dtype (760 bytes)
GV_PROFILE_BUCKETS, GV_PROFILE_LIST = 66, 8
PROFILE_DTYPE = np.dtype([
    ("ulp_hist", "<u8", (GV_PROFILE_BUCKETS,)), ("n_mismatch", "<u8"), ("worst_index", "<u8"),
    ("worst_c_raw", "<u8"), ("worst_r_raw", "<u8"), ("n_first", "<u8"),
    ("first_index", "<u8", (GV_PROFILE_LIST,)), ("first_c_raw", "<u8", (GV_PROFILE_LIST,)),
    ("first_r_raw", "<u8", (GV_PROFILE_LIST,))])
assert PROFILE_DTYPE.itemsize == 760


class gv_tol(ctypes.Structure):
    _fields_ = [("atol", ctypes.c_double), ("rtol", ctypes.c_double),
                ("equal_nan", ctypes.c_int32), ("reserved", ctypes.c_int32)]


EXPORTS = ["gv_verify_batch", "gv_verify_ragged", "gv_verify_ragged_noalloc", "gv_hash", "gv_hash2", "gv_group_candidates",
           "gv_group_workspace_bytes", "gv_error_profile", "gv_profile_workspace_bytes", "gv_exec_summary", "gv_speedup",
           "gv_mem_efficiency", "gv_accuracy_matrix", "gv_selftest_wait_expiry", "gv_selftest_read_sum", "gv_verify_batch_host", "gv_host_staging_bytes",
           "gv_workspace_bytes", "gv_check", "gv_status_string", "gv_last_cuda_error", "gv_version"]


def _load() -> ctypes.CDLL:
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2507_23194_b200.build` "
            "(or __graft_entry__.build()). There is no fallback implementation.")
    L = ctypes.CDLL(path)
    vp, i32, i64, u64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_size_t
    L.gv_verify_batch.restype = ctypes.c_int
    L.gv_verify_batch.argtypes = [vp, vp, i32, u64, ctypes.c_int, ctypes.POINTER(gv_tol), vp, vp, vp, sz, vp]
    L.gv_verify_ragged.restype = ctypes.c_int
    L.gv_verify_ragged.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, ctypes.POINTER(gv_tol), vp, vp, sz, vp]
    L.gv_verify_ragged_noalloc.restype = ctypes.c_int
    L.gv_verify_ragged_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, i64, i32, ctypes.POINTER(gv_tol), vp, vp, vp]
    L.gv_hash.restype = ctypes.c_int
    L.gv_hash.argtypes = [vp, u64, vp, vp]
    L.gv_hash2.restype = ctypes.c_int
    L.gv_hash2.argtypes = [vp, u64, vp, vp]
    L.gv_group_candidates.restype = ctypes.c_int
    L.gv_group_candidates.argtypes = [vp, i64, vp, vp, vp, vp, sz, vp]
    L.gv_group_workspace_bytes.restype = sz
    L.gv_group_workspace_bytes.argtypes = [i64]
    L.gv_error_profile.restype = ctypes.c_int
    L.gv_error_profile.argtypes = [vp, vp, u64, ctypes.c_int, ctypes.POINTER(gv_tol), u64, vp, vp, vp, sz, vp]
    L.gv_exec_summary.restype = ctypes.c_int
    L.gv_exec_summary.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp]
    L.gv_speedup.restype = ctypes.c_int
    L.gv_speedup.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, vp, vp]
    L.gv_mem_efficiency.restype = ctypes.c_int
    L.gv_mem_efficiency.argtypes = [vp, vp, i64, i32, ctypes.c_double, vp, vp, vp, vp, vp]
    L.gv_accuracy_matrix.restype = ctypes.c_int
    L.gv_accuracy_matrix.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp, vp]
    L.gv_selftest_wait_expiry.restype = ctypes.c_int
    L.gv_selftest_wait_expiry.argtypes = [vp, sz, vp]
    L.gv_selftest_read_sum.restype = ctypes.c_int
    L.gv_selftest_read_sum.argtypes = [vp, u64, vp, vp]
    L.gv_profile_workspace_bytes.restype = sz
    L.gv_profile_workspace_bytes.argtypes = []
    L.gv_verify_batch_host.restype = ctypes.c_int
    L.gv_verify_batch_host.argtypes = [vp, vp, i32, u64, ctypes.c_int, ctypes.POINTER(gv_tol), vp, vp, vp, sz, vp]
    L.gv_host_staging_bytes.restype = sz
    L.gv_host_staging_bytes.argtypes = [u64, ctypes.c_int, i32]
    L.gv_workspace_bytes.restype = sz
    L.gv_workspace_bytes.argtypes = [i64, i32]
    L.gv_check.restype = ctypes.c_int
    L.gv_check.argtypes = [vp, vp]
    L.gv_status_string.restype = ctypes.c_char_p
    L.gv_status_string.argtypes = [ctypes.c_int]
    L.gv_last_cuda_error.restype = ctypes.c_char_p
    L.gv_last_cuda_error.argtypes = []
    L.gv_version.restype = ctypes.c_uint32
    L.gv_version.argtypes = []
    return L


lib = _load()


class GvError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        msg = lib.gv_status_string(status).decode()
        if status == GV_ERR_CUDA:
            msg += ": " + lib.gv_last_cuda_error().decode()
        super().__init__(f"gv status {status}: {msg}")


def _raise(status: int) -> None:
    if status != GV_OK:
        raise GvError(status)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> ctypes.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _tol(atol: float, rtol: float, equal_nan: bool) -> gv_tol:
    return gv_tol(float(atol), float(rtol), int(bool(equal_nan)), 0)


def gv_workspace_bytes(T: int = 0, N: int = 0) -> int:
    return int(lib.gv_workspace_bytes(T, N))


def gv_version() -> int:
    return int(lib.gv_version())


def results_to_numpy(results: torch.Tensor) -> np.ndarray:
    """Device (or host) uint8 record buffer -> structured numpy array of gv_result records."""
    return results.cpu().numpy().view(RESULT_DTYPE).reshape(-1)


def gv_verify_batch(ref: torch.Tensor, cands: Sequence[torch.Tensor], atol: float = 0.0, rtol: float = 0.0,
                    equal_nan: bool = False, results: Optional[torch.Tensor] = None,
                    ref_hash: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                    stream: Optional[torch.cuda.Stream] = None, cand_ptrs=None) -> torch.Tensor:
    """Enqueue one dense verification; returns the device tensor of N 64-byte records (uint8 [N, 64]).

    Buffers not supplied are allocated here with torch (the C library itself allocates nothing).
    ``cand_ptrs`` may carry a prebuilt ``(ctypes.c_void_p * N)`` array to skip marshalling.
    """
    dt = DTYPE_OF[ref.dtype]
    N = len(cands)
    dev = ref.device
    if results is None:
        results = torch.empty((max(N, 1), 64), dtype=torch.uint8, device=dev)
    if workspace is None:
        workspace = torch.empty(gv_workspace_bytes(0, N), dtype=torch.uint8, device=dev)
    if cand_ptrs is None:
        cand_ptrs = (ctypes.c_void_p * max(N, 1))(*[c.data_ptr() for c in cands])
    t = _tol(atol, rtol, equal_nan)
    rc = lib.gv_verify_batch(ref.data_ptr(), ctypes.cast(cand_ptrs, ctypes.c_void_p), N, ref.numel(), dt,
                             ctypes.byref(t), results.data_ptr(),
                             ref_hash.data_ptr() if ref_hash is not None else None,
                             workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _raise(rc)
    return results[:N]


def gv_verify_ragged(ref_buf: torch.Tensor, ref_off: torch.Tensor, cand_buf: torch.Tensor, cand_off: torch.Tensor,
                     dtypes: torch.Tensor, N: int, atol: float, rtol: float, equal_nan: bool = False,
                     n_elems: Optional[torch.Tensor] = None, results: Optional[torch.Tensor] = None,
                     workspace: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Enqueue one ragged verification; returns the device tensor of T*N records (uint8 [T*N, 64])."""
    T = dtypes.numel()
    dev = ref_buf.device
    if results is None:
        results = torch.empty((max(T * N, 1), 64), dtype=torch.uint8, device=dev)
    if workspace is None:
        workspace = torch.empty(gv_workspace_bytes(T, N), dtype=torch.uint8, device=dev)
    t = _tol(atol, rtol, equal_nan)
    rc = lib.gv_verify_ragged(ref_buf.data_ptr(), ref_off.data_ptr(), cand_buf.data_ptr(), cand_off.data_ptr(),
                              dtypes.data_ptr(), n_elems.data_ptr() if n_elems is not None else None, T, N,
                              ctypes.byref(t), results.data_ptr(), workspace.data_ptr(), workspace.numel(),
                              _stream_ptr(stream))
    _raise(rc)
    return results[:T * N]


GV_NOALLOC_MAX_TENSORS = 65536


def gv_verify_ragged_noalloc(ref_buf: torch.Tensor, ref_off: torch.Tensor, cand_buf: torch.Tensor,
                             cand_off: torch.Tensor, dtypes: torch.Tensor, N: int, atol: float, rtol: float,
                             equal_nan: bool, results: torch.Tensor, n_elems: Optional[torch.Tensor] = None,
                             status_out: Optional[torch.Tensor] = None,
                             stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Ragged verification for callers that cannot provide a workspace: the library's own fixed scratch
    array is used and nothing is allocated, so ``results`` (uint8 [T*N, 64]) must be passed in, and
    ``status_out`` (one int32 on the device) too if the status bits are wanted. At most
    ``GV_NOALLOC_MAX_TENSORS`` tensors per call; calls that overlap on the GPU race on the shared
    scratch. Returns ``results``."""
    T = dtypes.numel()
    t = _tol(atol, rtol, equal_nan)
    rc = lib.gv_verify_ragged_noalloc(ref_buf.data_ptr(), ref_off.data_ptr(), cand_buf.data_ptr(),
                                      cand_off.data_ptr(), dtypes.data_ptr(),
                                      n_elems.data_ptr() if n_elems is not None else None, T, N, ctypes.byref(t),
                                      results.data_ptr(), status_out.data_ptr() if status_out is not None else None,
                                      _stream_ptr(stream))
    _raise(rc)
    return results[:T * N]


def gv_hash(buf: torch.Tensor, out: Optional[torch.Tensor] = None,
            stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Enqueue the content hash of ``buf``'s bytes; returns a device int64 tensor holding the u64 hash."""
    if out is None:
        out = torch.empty(1, dtype=torch.int64, device=buf.device)
    rc = lib.gv_hash(buf.data_ptr(), buf.numel() * buf.element_size(), out.data_ptr(), _stream_ptr(stream))
    _raise(rc)
    return out


def gv_exec_summary(results: torch.Tensor, T: int, N: int, kmax: int, stream: Optional[torch.cuda.Stream] = None):
    """Enqueue the pass/fail summary of T x N tensor-major records; returns device tensors
    (pass uint8[N], n_pass int32[1], pass_at_k float64[kmax])."""
    dev = results.device
    ok = torch.empty(max(N, 1), dtype=torch.uint8, device=dev)
    c = torch.empty(1, dtype=torch.int32, device=dev)
    pk = torch.empty(max(kmax, 1), dtype=torch.float64, device=dev)
    _raise(lib.gv_exec_summary(results.data_ptr(), T, N, kmax, ok.data_ptr(), c.data_ptr(), pk.data_ptr(),
                               _stream_ptr(stream)))
    return ok[:N], c, pk[:kmax]


def gv_speedup(ref_lat: torch.Tensor, gen_lat: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
    """Enqueue medians, ratios and the speedup for float32 latency samples of shape (T, S_ref) and
    (T, S_gen); returns device tensors (median_ref[T], median_gen[T], ratio[T], speedup float64[1])."""
    T = ref_lat.shape[0]
    dev = ref_lat.device
    mr, mg, ra = (torch.empty(max(T, 1), dtype=torch.float32, device=dev) for _ in range(3))
    sp = torch.empty(1, dtype=torch.float64, device=dev)
    _raise(lib.gv_speedup(ref_lat.data_ptr(), gen_lat.data_ptr(), T, ref_lat.shape[1], gen_lat.shape[1], mr.data_ptr(),
                          mg.data_ptr(), ra.data_ptr(), sp.data_ptr(), _stream_ptr(stream)))
    return mr[:T], mg[:T], ra[:T], sp


def gv_mem_efficiency(lat: torch.Tensor, nbytes: torch.Tensor, peak: float, stream: Optional[torch.cuda.Stream] = None):
    """Enqueue the memory efficiency for float32 latency samples of shape (T, S) and the int64/uint64 bytes each
    unit test has to move; returns device tensors (median[T] float32, bandwidth[T], efficiency[T], mean[1] float64)."""
    T = lat.shape[0]
    dev = lat.device
    med = torch.empty(max(T, 1), dtype=torch.float32, device=dev)
    bw, eff = (torch.empty(max(T, 1), dtype=torch.float64, device=dev) for _ in range(2))
    mean = torch.empty(1, dtype=torch.float64, device=dev)
    _raise(lib.gv_mem_efficiency(lat.data_ptr(), nbytes.data_ptr(), T, lat.shape[1], float(peak), med.data_ptr(),
                                 bw.data_ptr(), eff.data_ptr(), mean.data_ptr(), _stream_ptr(stream)))
    return med[:T], bw[:T], eff[:T], mean


def gv_accuracy_matrix(status: torch.Tensor, kmax: int, stream: Optional[torch.cuda.Stream] = None):
    """Enqueue call / execution accuracy of a (K, R) uint8 status matrix; returns device tensors
    (n_call[K], n_exec[K] int32, call_acc[kmax], exec_acc[kmax] float64)."""
    K, R = status.shape
    dev = status.device
    nc, ne = (torch.empty(max(K, 1), dtype=torch.int32, device=dev) for _ in range(2))
    ca, ea = (torch.empty(max(kmax, 1), dtype=torch.float64, device=dev) for _ in range(2))
    _raise(lib.gv_accuracy_matrix(status.data_ptr(), K, R, kmax, nc.data_ptr(), ne.data_ptr(), ca.data_ptr(),
                                  ea.data_ptr(), _stream_ptr(stream)))
    return nc[:K], ne[:K], ca[:kmax], ea[:kmax]


def gv_selftest_wait_expiry(workspace: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Enqueue the diagnostic kernel whose bounded wait expires; gv_check(workspace) then reports the timeout."""
    _raise(lib.gv_selftest_wait_expiry(workspace.data_ptr(), workspace.numel(), _stream_ptr(stream)))


def gv_selftest_read_sum(buf: torch.Tensor, out: Optional[torch.Tensor] = None,
                         stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Enqueue the read-only bandwidth probe (sum of the buffer's 32-bit words mod 2^64) -> device int64[1]."""
    if out is None:
        out = torch.empty(1, dtype=torch.int64, device=buf.device)
    _raise(lib.gv_selftest_read_sum(buf.data_ptr(), buf.numel() * buf.element_size(), out.data_ptr(), _stream_ptr(stream)))
    return out


def gv_hash2(buf: torch.Tensor, out: Optional[torch.Tensor] = None,
             stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Enqueue the second hash lane of ``buf``'s bytes; returns a device int64 tensor holding the u64."""
    if out is None:
        out = torch.empty(1, dtype=torch.int64, device=buf.device)
    _raise(lib.gv_hash2(buf.data_ptr(), buf.numel() * buf.element_size(), out.data_ptr(), _stream_ptr(stream)))
    return out


def gv_profile_workspace_bytes() -> int:
    return int(lib.gv_profile_workspace_bytes())


def gv_error_profile(ref: torch.Tensor, cand: torch.Tensor, atol: float = 0.0, rtol: float = 0.0,
                     equal_nan: bool = False, row_len: int = 0, out: Optional[torch.Tensor] = None,
                     rows: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None):
    """Enqueue the error profile of one candidate; returns (device uint8[760] holding a gv_profile,
    device int32 per-row mismatch counts or None). Read the profile with ``profile_to_numpy``."""
    dt = DTYPE_OF[ref.dtype]
    n = ref.numel()
    dev = ref.device
    if out is None:
        out = torch.empty(PROFILE_DTYPE.itemsize, dtype=torch.uint8, device=dev)
    if row_len and rows is None:
        rows = torch.empty(max(1, (n + row_len - 1) // row_len), dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = torch.empty(gv_profile_workspace_bytes(), dtype=torch.uint8, device=dev)
    t = _tol(atol, rtol, equal_nan)
    rc = lib.gv_error_profile(ref.data_ptr(), cand.data_ptr(), n, dt, ctypes.byref(t), row_len, out.data_ptr(),
                              rows.data_ptr() if rows is not None else None, workspace.data_ptr(), workspace.numel(),
                              _stream_ptr(stream))
    _raise(rc)
    return out, (rows[:(n + row_len - 1) // row_len] if rows is not None else None)


def profile_to_numpy(out: torch.Tensor) -> np.ndarray:
    return out.cpu().numpy().view(PROFILE_DTYPE)[0]


def gv_group_workspace_bytes(N: int) -> int:
    return int(lib.gv_group_workspace_bytes(N))


def gv_group_candidates(results: torch.Tensor, group_id: Optional[torch.Tensor] = None,
                        group_count: Optional[torch.Tensor] = None, n_groups: Optional[torch.Tensor] = None,
                        workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Enqueue the grouping of the N records in ``results`` (device uint8 tensor of shape (N, 64));
    returns device tensors (group_id int32[N], group_count int32[N], n_groups int32[1])."""
    N = results.shape[0]
    dev = results.device
    if group_id is None:
        group_id = torch.empty(max(N, 1), dtype=torch.int32, device=dev)
    if group_count is None:
        group_count = torch.empty(max(N, 1), dtype=torch.int32, device=dev)
    if n_groups is None:
        n_groups = torch.empty(1, dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = torch.empty(gv_group_workspace_bytes(N), dtype=torch.uint8, device=dev)
    rc = lib.gv_group_candidates(results.data_ptr(), N, group_id.data_ptr(), group_count.data_ptr(), n_groups.data_ptr(),
                                 workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _raise(rc)
    return group_id[:N], group_count[:N], n_groups


def gv_check(workspace: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> int:
    return int(lib.gv_check(workspace.data_ptr(), _stream_ptr(stream)))


def gv_host_staging_bytes(n_elems: int, dt: int, slab: int) -> int:
    return int(lib.gv_host_staging_bytes(n_elems, dt, slab))


def gv_verify_batch_host(ref: torch.Tensor, cands: Sequence[torch.Tensor], atol: float, rtol: float,
                         equal_nan: bool, staging: torch.Tensor, results: Optional[np.ndarray] = None,
                         want_ref_hash: bool = True, stream: Optional[torch.cuda.Stream] = None):
    """Host tensors in, host records out (synchronous). ``staging`` is a device uint8 buffer."""
    dt = DTYPE_OF[ref.dtype]
    N = len(cands)
    if results is None:
        results = np.zeros(max(N, 1), dtype=RESULT_DTYPE)
    ref_hash = np.zeros(1, dtype=np.uint64)
    ptrs = (ctypes.c_void_p * max(N, 1))(*[c.data_ptr() for c in cands])
    t = _tol(atol, rtol, equal_nan)
    rc = lib.gv_verify_batch_host(ref.data_ptr(), ctypes.cast(ptrs, ctypes.c_void_p), N, ref.numel(), dt,
                                  ctypes.byref(t), results.ctypes.data_as(ctypes.c_void_p),
                                  ref_hash.ctypes.data_as(ctypes.c_void_p) if want_ref_hash else None,
                                  staging.data_ptr(), staging.numel(), _stream_ptr(stream))
    _raise(rc)
    return results[:N], int(ref_hash[0])
