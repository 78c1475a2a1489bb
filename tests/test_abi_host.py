"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, and rejects bad arguments before touching the device (nothing is launched here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def gvlib():
    from paper_2507_23194_b200 import build as B
    B.build()
    from paper_2507_23194_b200 import gv
    return gv


def test_header_symbols_are_exported(gvlib):
    hdr = open(os.path.join(ROOT, "include", "gv.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(gv_[a-z0-9_]+)\s*\(", hdr))
    assert {"gv_verify_batch", "gv_verify_ragged", "gv_hash"} <= declared
    for name in declared:
        assert hasattr(gvlib.lib, name), f"{name} is declared in gv.h but not exported"
    assert declared == set(gvlib.EXPORTS), "binding and header disagree on the entry points"


def test_version_and_strings(gvlib):
    assert gvlib.gv_version() >= 0x000100
    assert gvlib.lib.gv_status_string(0) == b"ok"
    for s in range(1, 8):
        assert len(gvlib.lib.gv_status_string(s)) > 0
    assert gvlib.gv_workspace_bytes(0, 8) >= 256
    assert gvlib.gv_workspace_bytes(10000, 4) >= 256 + 8 * 10001
    assert gvlib.lib.gv_host_staging_bytes(1000, 1, 0) == 0


def test_result_layout(gvlib):
    assert gvlib.RESULT_DTYPE.itemsize == 64
    assert gvlib.RESULT_DTYPE.fields["hash"][1] == 32
    assert gvlib.RESULT_DTYPE.fields["max_abs_err"][1] == 48
    assert gvlib.RESULT_DTYPE.fields["max_rel_err"][1] == 52


def _call_batch(gv, ref=0x1000, cands=(0x2000,), N=1, n=16, dt=0, atol=1e-3, rtol=1e-3, results=0x3000,
                ref_hash=None, ws=0x4000, ws_bytes=4096, tol_null=False):
    ptrs = (ctypes.c_void_p * max(1, len(cands)))(*cands)
    t = gv.gv_tol(atol, rtol, 0, 0)
    return gv.lib.gv_verify_batch(ref, ctypes.cast(ptrs, ctypes.c_void_p), N, n, dt,
                                  None if tol_null else ctypes.byref(t), results, ref_hash, ws, ws_bytes, None)


def test_dense_argument_errors_return_before_any_launch(gvlib):
    gv = gvlib
    assert _call_batch(gv, dt=5) == gv.GV_ERR_UNSUPPORTED
    assert _call_batch(gv, dt=-1) == gv.GV_ERR_UNSUPPORTED
    assert _call_batch(gv, N=-1) == gv.GV_ERR_INVALID_ARG
    assert _call_batch(gv, ref=None) == gv.GV_ERR_INVALID_ARG
    assert _call_batch(gv, results=None) == gv.GV_ERR_INVALID_ARG
    assert _call_batch(gv, cands=(None,)) == gv.GV_ERR_INVALID_ARG
    assert _call_batch(gv, atol=float("nan")) == gv.GV_ERR_INVALID_ARG
    assert _call_batch(gv, rtol=-1.0) == gv.GV_ERR_INVALID_ARG
    assert _call_batch(gv, atol=float("inf")) == gv.GV_ERR_INVALID_ARG
    assert _call_batch(gv, atol=3.5e38) == gv.GV_ERR_INVALID_ARG          # not a finite binary32 value
    assert _call_batch(gv, rtol=1e300) == gv.GV_ERR_INVALID_ARG
    assert _call_batch(gv, tol_null=True) == gv.GV_ERR_INVALID_ARG
    assert _call_batch(gv, ws=None) == gv.GV_ERR_WORKSPACE
    assert _call_batch(gv, ws_bytes=8) == gv.GV_ERR_WORKSPACE
    assert _call_batch(gv, ws=0x4004) == gv.GV_ERR_WORKSPACE
    assert _call_batch(gv, ref=0x1002) == gv.GV_ERR_MISALIGNED            # fp32 needs 4-byte alignment
    assert _call_batch(gv, cands=(0x2001,), dt=1) == gv.GV_ERR_MISALIGNED   # bf16 needs 2-byte alignment
    assert _call_batch(gv, results=0x3004) == gv.GV_ERR_MISALIGNED
    assert _call_batch(gv, n=1 << 62) == gv.GV_ERR_INVALID_ARG
    # integer dtypes ignore tolerances, so a null tol is fine for them -- but then the call would
    # launch, which needs a device; only check that validation does not reject it for the tolerance
    assert _call_batch(gv, dt=3, tol_null=True, ws=None) == gv.GV_ERR_WORKSPACE


def test_ragged_and_hash_argument_errors(gvlib):
    gv = gvlib
    t = gv.gv_tol(1e-3, 1e-3, 0, 0)
    f = gv.lib.gv_verify_ragged
    ok_args = [0x1000, 0x2000, 0x3000, 0x4000, 0x5000, None, 4, 2, ctypes.byref(t), 0x6000, 0x7000, 1 << 20, None]

    def call(**kw):
        a = list(ok_args)
        names = ["ref_base", "ref_off", "cand_base", "cand_off", "dtypes", "n_elems", "T", "N", "tol", "results",
                 "ws", "ws_bytes", "stream"]
        for k, v in kw.items():
            a[names.index(k)] = v
        return f(*a)

    assert call(T=-1) == gv.GV_ERR_INVALID_ARG
    assert call(N=-1) == gv.GV_ERR_INVALID_ARG
    assert call(ref_off=None) == gv.GV_ERR_INVALID_ARG
    assert call(dtypes=None) == gv.GV_ERR_INVALID_ARG
    assert call(cand_off=None) == gv.GV_ERR_INVALID_ARG
    assert call(tol=None) == gv.GV_ERR_INVALID_ARG
    assert call(ws_bytes=16) == gv.GV_ERR_WORKSPACE
    assert call(ws=None) == gv.GV_ERR_WORKSPACE
    assert call(ref_off=0x2004) == gv.GV_ERR_MISALIGNED
    assert gv.lib.gv_hash(0x1000, 16, None, None) == gv.GV_ERR_INVALID_ARG
    assert gv.lib.gv_hash(None, 16, 0x1000, None) == gv.GV_ERR_INVALID_ARG
    assert gv.lib.gv_hash(0x1000, 16, 0x1004, None) == gv.GV_ERR_MISALIGNED
    assert gv.lib.gv_check(None, None) == gv.GV_ERR_INVALID_ARG


def test_group_argument_errors_return_before_any_launch(gvlib):
    gv = gvlib
    call = lambda res=0x1000, N=4, gid=0x2000, cnt=0x3000, ng=0x4000, ws=0x5000, wsb=4096: gv.lib.gv_group_candidates(
        res, N, gid, cnt, ng, ws, wsb, None)
    assert call(N=-1) == gv.GV_ERR_INVALID_ARG
    assert call(res=None) == gv.GV_ERR_INVALID_ARG
    assert call(gid=None) == gv.GV_ERR_INVALID_ARG
    assert call(res=0x1008) == gv.GV_ERR_MISALIGNED
    assert call(gid=0x2002) == gv.GV_ERR_MISALIGNED
    assert call(ws=None) == gv.GV_ERR_WORKSPACE
    assert call(ws=0x5004) == gv.GV_ERR_WORKSPACE
    assert call(wsb=128) == gv.GV_ERR_WORKSPACE
    assert call(N=5000, wsb=4096) == gv.GV_ERR_WORKSPACE            # beyond one CTA the table lives in the workspace
    assert call(N=(1 << 28) + 1, wsb=1 << 40) == gv.GV_ERR_UNSUPPORTED
    assert b"GV_GROUP_MAX" in gv.lib.gv_last_cuda_error()
    assert gv.gv_group_workspace_bytes(0) == 256
    assert gv.gv_group_workspace_bytes(2048) == 256
    assert gv.gv_group_workspace_bytes(2049) == 256 + 8192 * 8
    assert gv.gv_group_workspace_bytes(-1) == 0


def test_profile_argument_errors_return_before_any_launch(gvlib):
    gv = gvlib
    wsb = gv.gv_profile_workspace_bytes()
    assert wsb > 256
    t = gv.gv_tol(1e-3, 1e-3, 0, 0)

    def call(ref=0x1000, cand=0x2000, n=16, dt=0, tol=t, row_len=0, out=0x3000, rows=None, ws=0x4000, wsb=wsb):
        return gv.lib.gv_error_profile(ref, cand, n, dt, ctypes.byref(tol) if tol is not None else None, row_len, out,
                                       rows, ws, wsb, None)
    assert call(dt=7) == gv.GV_ERR_UNSUPPORTED
    assert call(out=None) == gv.GV_ERR_INVALID_ARG
    assert call(ref=None) == gv.GV_ERR_INVALID_ARG
    assert call(row_len=8) == gv.GV_ERR_INVALID_ARG                  # row counts asked for, no buffer given
    assert call(tol=None) == gv.GV_ERR_INVALID_ARG
    assert call(tol=gv.gv_tol(-1.0, 0.0, 0, 0)) == gv.GV_ERR_INVALID_ARG
    assert call(ref=0x1002) == gv.GV_ERR_MISALIGNED
    assert call(out=0x3004) == gv.GV_ERR_MISALIGNED
    assert call(ws=None) == gv.GV_ERR_WORKSPACE
    assert call(wsb=1024) == gv.GV_ERR_WORKSPACE
    assert gv.PROFILE_DTYPE.itemsize == 760


def test_stats_argument_errors_return_before_any_launch(gvlib):
    gv = gvlib
    es = lambda res=0x1000, T=2, N=4, kmax=4, ok=0x2000, c=0x3000, pk=0x4000: gv.lib.gv_exec_summary(res, T, N, kmax, ok, c, pk, None)
    assert es(T=-1) == gv.GV_ERR_INVALID_ARG
    assert es(kmax=5) == gv.GV_ERR_INVALID_ARG                       # more draws than candidates
    assert es(N=100000, kmax=70000) == gv.GV_ERR_INVALID_ARG         # beyond GV_PASSK_MAX
    assert es(c=None) == gv.GV_ERR_INVALID_ARG
    assert es(res=None) == gv.GV_ERR_INVALID_ARG
    assert es(pk=0x4004) == gv.GV_ERR_MISALIGNED
    sp = lambda a=0x1000, b=0x2000, T=3, sr=5, sg=5, mr=0x3000, mg=0x4000, ra=0x5000, out=0x6000: gv.lib.gv_speedup(
        a, b, T, sr, sg, mr, mg, ra, out, None)
    assert sp(sr=0) == gv.GV_ERR_INVALID_ARG
    assert sp(sg=4097) == gv.GV_ERR_INVALID_ARG
    assert sp(out=None) == gv.GV_ERR_INVALID_ARG
    assert sp(a=None) == gv.GV_ERR_INVALID_ARG
    assert sp(a=0x1002) == gv.GV_ERR_MISALIGNED
    assert sp(out=0x6004) == gv.GV_ERR_MISALIGNED


def test_new_aggregates_and_host_entry_argument_errors(gvlib):
    gv = gvlib
    me = lambda lat=0x1000, nb=0x2000, T=3, S=5, peak=1e9, med=0x3000, bw=0x4000, eff=0x5000, mean=0x6000: (
        gv.lib.gv_mem_efficiency(lat, nb, T, S, peak, med, bw, eff, mean, None))
    assert me(S=0) == gv.GV_ERR_INVALID_ARG
    assert me(S=4097) == gv.GV_ERR_INVALID_ARG
    assert me(peak=0.0) == gv.GV_ERR_INVALID_ARG
    assert me(peak=float("inf")) == gv.GV_ERR_INVALID_ARG
    assert me(peak=float("nan")) == gv.GV_ERR_INVALID_ARG
    assert me(mean=None) == gv.GV_ERR_INVALID_ARG
    assert me(nb=None) == gv.GV_ERR_INVALID_ARG
    assert me(nb=0x2004) == gv.GV_ERR_MISALIGNED
    assert me(bw=0x4004) == gv.GV_ERR_MISALIGNED
    am = lambda st=0x1000, K=4, R=10, kmax=10, nc=0x2000, ne=0x3000, ca=0x4000, ea=0x5000: gv.lib.gv_accuracy_matrix(
        st, K, R, kmax, nc, ne, ca, ea, None)
    assert am(K=-1) == gv.GV_ERR_INVALID_ARG
    assert am(kmax=11) == gv.GV_ERR_INVALID_ARG                      # more draws than runs
    assert am(R=1025, kmax=1) == gv.GV_ERR_INVALID_ARG               # beyond GV_RUNS_MAX
    assert am(st=None) == gv.GV_ERR_INVALID_ARG
    assert am(ca=None) == gv.GV_ERR_INVALID_ARG
    assert am(nc=0x2002) == gv.GV_ERR_MISALIGNED
    assert am(ea=0x5004) == gv.GV_ERR_MISALIGNED
    assert gv.lib.gv_selftest_wait_expiry(None, 256, None) == gv.GV_ERR_WORKSPACE
    assert gv.lib.gv_selftest_wait_expiry(0x1000, 16, None) == gv.GV_ERR_WORKSPACE
    # the host-buffer entry point checks the tolerances before it enqueues its first copy
    ptrs = (ctypes.c_void_p * 1)(0x2000)
    bad = gv.gv_tol(float("nan"), 0.0, 0, 0)
    rc = gv.lib.gv_verify_batch_host(0x1000, ctypes.cast(ptrs, ctypes.c_void_p), 1, 16, 0, ctypes.byref(bad), 0x3000, None,
                                     0x10000, 1 << 20, None)
    assert rc == gv.GV_ERR_INVALID_ARG
    rc = gv.lib.gv_verify_batch_host(0x1000, ctypes.cast(ptrs, ctypes.c_void_p), 1, 16, 0, None, 0x3000, None, 0x10000,
                                     1 << 20, None)
    assert rc == gv.GV_ERR_INVALID_ARG
    # ragged: more than 2^31 - 1 tensors is an argument error
    t = gv.gv_tol(1e-3, 1e-3, 0, 0)
    assert gv.lib.gv_verify_ragged(0x1000, 0x2000, 0x3000, 0x4000, 0x5000, None, 1 << 31, 2, ctypes.byref(t), 0x6000, 0x7000,
                                   1 << 40, None) == gv.GV_ERR_INVALID_ARG


def test_tile_index_arithmetic_exhaustively():
    """The decomposition every verify kernel relies on, restated on the host and checked for every size up to
    four CTA tiles and a bit, at every alignment of the tail: a tensor of nbytes bytes is covered exactly once by
    the full 512-byte warp-tiles [0, nbytes // 512) (fast loop, 32 lanes x 16 bytes) plus the tail tile whose
    lanes hold the remaining full vectors and at most one partial vector; the words the hash sums are exactly
    ceil(nbytes / 8); tile t belongs to warp t mod W of the grid; a ragged warp's contiguous stretch split is a
    partition of the global tile sequence."""
    tile, vec = 512, 16
    for esz in (2, 4, 8):
        for n in range(0, (4 * 8 * tile + 17 * esz) // esz + 1):
            nbytes = n * esz
            full_tiles, all_tiles = nbytes // tile, (nbytes + tile - 1) // tile
            covered = full_tiles * tile
            words = full_tiles * (tile // 8)
            for t in range(full_tiles, all_tiles):                  # at most one
                for lane in range(32):
                    voff = t * tile + lane * vec
                    rem = max(0, nbytes - voff)
                    nvalid = vec // esz if rem >= vec else rem // esz
                    covered += nvalid * esz
                    words += 0 if nvalid == 0 else (2 if nvalid * esz > 8 else 1)
            assert all_tiles - full_tiles in (0, 1)
            assert covered == nbytes and words == (nbytes + 7) // 8, (esz, n)
    for total in list(range(0, 70)) + [1000, 4097]:
        for W in (1, 2, 7, 16, 2368):
            per, extra = divmod(total, W)
            spans, pos = [], 0
            for gw in range(W):
                begin = gw * per + min(gw, extra)
                end = begin + per + (1 if gw < extra else 0)
                assert begin == pos
                pos = end
                spans.append((begin, end))
            assert pos == total
            assert sorted(t for gw in range(W) for t in range(gw, total, W)) == list(range(total))   # dense: t mod W
