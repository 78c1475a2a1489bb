"""The entry point for callers that cannot allocate device memory (gv_verify_ragged_noalloc), called
through the C ABI and compared record by record, byte for byte (the tolerance every parity test here
uses: zero), with the ordinary gv_verify_ragged on the same inputs -- twice in a row, with different
batches, because the library's fixed scratch array keeps the previous call's contents. The file is
named to be collected last and passes alone in a fresh process as well as after the other tests."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_2507_23194_b200 import gv, workloads as W  # noqa: E402

DEV = "cuda:0"


def _both(wl):
    count = wl.T * wl.N
    ws = torch.empty(gv.gv_workspace_bytes(wl.T, wl.N), dtype=torch.uint8, device=DEV)
    want = gv.gv_verify_ragged(wl.ref_buf, wl.ref_off, wl.cand_buf, wl.cand_off, wl.dtypes, wl.N, wl.atol, wl.rtol,
                               wl.equal_nan, n_elems=wl.n_elems_t, workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    # outputs are the caller's: the records and (optionally) one status word, allocated here by the test
    res = torch.full((count, 64), 0xAB, dtype=torch.uint8, device=DEV)
    status = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    got = gv.gv_verify_ragged_noalloc(wl.ref_buf, wl.ref_off, wl.cand_buf, wl.cand_off, wl.dtypes, wl.N, wl.atol,
                                      wl.rtol, wl.equal_nan, results=res, n_elems=wl.n_elems_t, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return gv.results_to_numpy(got), gv.results_to_numpy(want)


def test_noalloc_matches_workspace_entry_point_on_two_calls_in_a_row(oracle):
    # first call: a large batch that fills much of the scratch table ...
    big = W.config5(DEV, T=700, max_log2=14.0, seed=11)
    got, want = _both(big)
    assert got.tobytes() == want.tobytes()
    # ... second call right after it: a smaller, different batch (stale table entries must not matter)
    small = W.config5(DEV, T=90, max_log2=12.0, seed=12, align=0)
    got, want = _both(small)
    assert got.tobytes() == want.tobytes()
    for i, f in enumerate(small.facts):
        assert int(got[i]["n_mismatch"]) == f["n_mismatch"]
    # the small batch against the CPU oracle as well (not only one CUDA entry point against the other)
    ref = oracle.verify_ragged(small.ref_buf.cpu().numpy(), small.ref_off.cpu().numpy(), small.cand_buf.cpu().numpy(),
                               small.cand_off.cpu().numpy(), small.dtypes.cpu().numpy(), small.N, small.atol, small.rtol,
                               small.equal_nan, n_elems=small.n_elems_t.cpu().numpy())
    assert got.tobytes() == ref.tobytes()
    # and once more with the first batch
    got, want = _both(big)
    assert got.tobytes() == want.tobytes()


def test_noalloc_rejects_batches_beyond_its_limit_and_reports_bad_tables():
    wl = W.config5(DEV, T=8, max_log2=8.0, seed=13)
    res = torch.zeros((8 * wl.N, 64), dtype=torch.uint8, device=DEV)
    t = gv.gv_tol(1e-3, 1e-3, 0, 0)
    import ctypes
    too_many = gv.GV_NOALLOC_MAX_TENSORS + 1
    rc = gv.lib.gv_verify_ragged_noalloc(wl.ref_buf.data_ptr(), wl.ref_off.data_ptr(), wl.cand_buf.data_ptr(),
                                         wl.cand_off.data_ptr(), wl.dtypes.data_ptr(), None, too_many, wl.N,
                                         ctypes.byref(t), res.data_ptr(), None, None)
    assert rc == gv.GV_ERR_WORKSPACE
    assert b"GV_NOALLOC_MAX_TENSORS" in gv.lib.gv_last_cuda_error()
    # a corrupted offsets table is flagged in the caller's status word, records stay zero records
    bad = wl.ref_off.clone()
    bad[3] = bad[3] + 1                                   # not a multiple of the element size
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    gv.gv_verify_ragged_noalloc(wl.ref_buf, bad, wl.cand_buf, wl.cand_off, wl.dtypes, wl.N, wl.atol, wl.rtol,
                                wl.equal_nan, results=res, n_elems=wl.n_elems_t, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) & 2
