"""GPU parity for the grouping of duplicate candidates: group ids, group sizes and the number of
groups from the CUDA library, through its C ABI, against the CPU oracle (exact: integers)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_2507_23194_b200 import gv, workloads as W  # noqa: E402

DEV = "cuda:0"


def run_group(rec: np.ndarray):
    n = rec.shape[0]
    raw = np.ascontiguousarray(rec).view(np.uint8).reshape(n, 64) if n else np.zeros((0, 64), dtype=np.uint8)
    res = torch.from_numpy(raw.copy()).to(DEV)
    ws = torch.empty(gv.gv_group_workspace_bytes(n), dtype=torch.uint8, device=DEV)
    gid, cnt, ng = gv.gv_group_candidates(res, workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    return gid.cpu().numpy(), cnt.cpu().numpy(), int(ng.cpu()[0])


def random_records(rng, n, pool):
    base = rng.integers(0, 256, size=(pool, 64), dtype=np.uint8)
    return base[rng.integers(0, pool, size=n)].copy().view(gv.RESULT_DTYPE).reshape(-1)


@pytest.mark.parametrize("n,pool", [(0, 1), (1, 1), (2, 1), (7, 3), (255, 40), (256, 256), (2048, 100), (2048, 5000),
                                    (2049, 300), (5000, 5000), (20000, 700)])
def test_group_random_records_against_oracle(oracle, n, pool):
    rng = np.random.default_rng(n * 31 + pool)
    rec = random_records(rng, n, pool)
    gid, cnt, ng = run_group(rec)
    w_gid, w_cnt, w_ng = oracle.group(rec)
    assert np.array_equal(gid, w_gid)
    assert np.array_equal(cnt, w_cnt)
    assert ng == w_ng


@pytest.mark.parametrize("n", [300, 4000])
def test_group_records_that_differ_in_one_field_only(oracle, n):
    # same content hash everywhere; each of the other fields in turn tells candidates apart
    rec = np.zeros(n, dtype=gv.RESULT_DTYPE)
    rec["hash"] = 0xDEADBEEFCAFEF00D
    rec["first_mismatch"] = gv.GV_NO_INDEX
    names = ["n_mismatch", "first_mismatch", "n_nan_disagree", "n_inf_disagree", "max_abs_diff_int"]
    for j in range(n):
        f = names[j % 5]
        rec[f][j] = (j // 5) % 7
    rec["max_abs_err"][::3] = 0.5
    rec["max_rel_err"][::4] = -0.0           # the sign bit alone separates records
    gid, cnt, ng = run_group(rec)
    w_gid, w_cnt, w_ng = oracle.group(rec)
    assert np.array_equal(gid, w_gid) and np.array_equal(cnt, w_cnt) and ng == w_ng


def test_group_large_n_properties():
    # a million records: too many for the quadratic oracle; checked against a dictionary of byte strings
    rng = np.random.default_rng(5)
    n = 1 << 20
    rec = random_records(rng, n, 50000)
    gid, cnt, ng = run_group(rec)
    raw = rec.view(np.uint8).reshape(n, 64)
    _, first, inverse, counts = np.unique(raw, axis=0, return_index=True, return_inverse=True, return_counts=True)
    assert np.array_equal(gid, first[inverse.reshape(-1)].astype(np.int32))
    assert ng == len(first)
    want_cnt = np.zeros(n, dtype=np.int32)
    want_cnt[first] = counts
    assert np.array_equal(cnt, want_cnt)


def test_group_after_verify_of_reduced_config2(oracle):
    # the real use: records written by a verify call; exact copies of the reference share one record
    wl = W.config2(DEV, n=(1 << 16) + 8, n_cands=48)
    n_c = len(wl.cands)
    ws = torch.empty(gv.gv_workspace_bytes(0, n_c), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_batch(wl.ref, wl.cands, wl.atol, wl.rtol, wl.equal_nan, workspace=ws)
    gws = torch.empty(gv.gv_group_workspace_bytes(n_c), dtype=torch.uint8, device=DEV)
    gid, cnt, ng = gv.gv_group_candidates(res, workspace=gws)       # same stream, ordered after the verify
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK and gv.gv_check(gws) == gv.GV_OK
    rec = gv.results_to_numpy(res)
    w_gid, w_cnt, w_ng = oracle.group(rec)
    assert np.array_equal(gid.cpu().numpy(), w_gid)
    assert np.array_equal(cnt.cpu().numpy(), w_cnt)
    assert int(ng.cpu()[0]) == w_ng
    copies = [j for j, f in enumerate(wl.facts) if f["class"] == "copy"]
    assert len(copies) > 1 and all(int(gid[j]) == copies[0] for j in copies)
    assert int(cnt[copies[0]]) == len(copies)


def test_group_twice_on_one_workspace_is_repeatable():
    rng = np.random.default_rng(11)
    for n in (1000, 3000):
        rec = random_records(rng, n, 50)
        raw = torch.from_numpy(rec.view(np.uint8).reshape(n, 64).copy()).to(DEV)
        ws = torch.empty(gv.gv_group_workspace_bytes(n), dtype=torch.uint8, device=DEV)
        a = gv.gv_group_candidates(raw, workspace=ws)
        a = [t.clone() for t in a]
        b = gv.gv_group_candidates(raw, workspace=ws)
        torch.cuda.synchronize()
        for x, y in zip(a, b):
            assert torch.equal(x, y)
