"""GPU parity at the benchmark's full sizes, through the same call bench.py times.

Every record of every candidate is checked against what the workload recipe fixes by construction
(mismatch counts, first index, NaN/Inf counts, exact copies = zero record + reference hash), and a
sample of candidates (several per recipe class) is checked byte for byte against the CPU oracle,
which computes those records one by one on the host."""
import ctypes
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_2507_23194_b200 import gv, workloads as W  # noqa: E402

DEV = "cuda:0"


def host_bytes(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.uint8).cpu().numpy()


def run_dense(wl):
    n_c = len(wl.cands)
    res = torch.empty((n_c, 64), dtype=torch.uint8, device=DEV)
    ws = torch.empty(gv.gv_workspace_bytes(0, n_c), dtype=torch.uint8, device=DEV)
    rh = torch.zeros(1, dtype=torch.int64, device=DEV)
    ptrs = (ctypes.c_void_p * n_c)(*[c.data_ptr() for c in wl.cands])
    gv.gv_verify_batch(wl.ref, wl.cands, wl.atol, wl.rtol, wl.equal_nan, results=res, ref_hash=rh, workspace=ws,
                       cand_ptrs=ptrs)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    return gv.results_to_numpy(res), int(rh.cpu().numpy().view(np.uint64)[0])


def check_facts(wl, got, ref_hash):
    zero = np.zeros((), dtype=gv.RESULT_DTYPE)
    zero["first_mismatch"] = gv.GV_NO_INDEX
    zero["hash"] = ref_hash
    for j, f in enumerate(wl.facts):
        if "n_mismatch" in f:
            assert int(got[j]["n_mismatch"]) == f["n_mismatch"], (wl.name, j, f["class"])
            want_first = gv.GV_NO_INDEX if f["first"] is None else f["first"]
            assert int(got[j]["first_mismatch"]) == want_first, (wl.name, j, f["class"])
        if "n_nan" in f:
            assert int(got[j]["n_nan_disagree"]) == f["n_nan"], (wl.name, j)
            assert int(got[j]["n_inf_disagree"]) == f["n_inf"], (wl.name, j)
        if f.get("hash_equals_ref"):
            assert got[j].tobytes() == zero.tobytes(), (wl.name, j, "exact copy must give the zero record")
        assert int(got[j]["reserved"]) == 0


def oracle_sample(oracle, wl, got, sample):
    ref = host_bytes(wl.ref)

    def one(j):
        return j, oracle.verify(ref, host_bytes(wl.cands[j]), wl.dtype, wl.atol, wl.rtol, wl.equal_nan)

    with ThreadPoolExecutor(max_workers=8) as ex:
        for j, want in ex.map(one, sample):
            assert got[j].tobytes() == want.tobytes(), (
                f"{wl.name}: candidate {j} ({wl.facts[j]['class']})\n gpu    {got[j]}\n oracle {want}")


def pick(wl, per_class):
    seen, out = {}, []
    for j, f in enumerate(wl.facts):
        key = f["class"] + str(f.get("sigma", "")) + str(f.get("frac", ""))
        if seen.get(key, 0) < per_class:
            seen[key] = seen.get(key, 0) + 1
            out.append(j)
    return out


def test_config2_full(oracle):
    wl = W.config2(DEV)
    assert wl.n == 4096 * 4096 and len(wl.cands) == 256
    got, rh = run_dense(wl)
    assert rh == oracle.hash_bytes(host_bytes(wl.ref))
    check_facts(wl, got, rh)
    oracle_sample(oracle, wl, got, pick(wl, 6))


def test_config3_full(oracle):
    wl = W.config3(DEV)
    assert wl.n == 8 * 32 * 4096 * 128 and len(wl.cands) == 32
    got, rh = run_dense(wl)
    assert rh == oracle.hash_bytes(host_bytes(wl.ref))
    check_facts(wl, got, rh)
    oracle_sample(oracle, wl, got, pick(wl, 2))
    del wl
    torch.cuda.empty_cache()


@pytest.mark.parametrize("wide", [False, True])
def test_config4_full(oracle, wide):
    wl = W.config4(DEV, wide=wide)
    assert wl.n == 65536 * 1024 and len(wl.cands) == 64
    got, rh = run_dense(wl)
    assert rh == oracle.hash_bytes(host_bytes(wl.ref))
    check_facts(wl, got, rh)
    for j, f in enumerate(wl.facts):                      # float fields stay zero in exact mode
        assert got[j]["max_abs_err"] == 0 and got[j]["max_rel_err"] == 0
        assert int(got[j]["n_nan_disagree"]) == 0 and int(got[j]["n_inf_disagree"]) == 0
    oracle_sample(oracle, wl, got, pick(wl, 1))
    del wl
    torch.cuda.empty_cache()


def test_config5_full(oracle):
    wl = W.config5(DEV)
    assert wl.T == 10000 and wl.N == 4
    res = torch.empty((wl.T * wl.N, 64), dtype=torch.uint8, device=DEV)
    ws = torch.empty(gv.gv_workspace_bytes(wl.T, wl.N), dtype=torch.uint8, device=DEV)
    gv.gv_verify_ragged(wl.ref_buf, wl.ref_off, wl.cand_buf, wl.cand_off, wl.dtypes, wl.N, wl.atol, wl.rtol,
                        wl.equal_nan, n_elems=wl.n_elems_t, results=res, workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    got = gv.results_to_numpy(res)
    for i, f in enumerate(wl.facts):                      # by construction, every record
        assert int(got[i]["n_mismatch"]) == f["n_mismatch"], (i, f["class"])
        assert int(got[i]["first_mismatch"]) == (gv.GV_NO_INDEX if f["first"] is None else f["first"]), (i, f["class"])
        assert int(got[i]["n_nan_disagree"]) == 0 and int(got[i]["n_inf_disagree"]) == 0
    # oracle on a sample of tensors: every 9th, plus the 16 largest and the 16 smallest
    order = np.argsort(np.array(wl.n_elems))
    sample = sorted(set(range(0, wl.T, 9)) | set(order[:16].tolist()) | set(order[-16:].tolist()))
    ref_buf, cand_buf = wl.ref_buf.cpu().numpy(), wl.cand_buf.cpu().numpy()
    ref_off, cand_off = wl.ref_off.cpu().numpy(), wl.cand_off.cpu().numpy()
    dtypes, n_el = wl.dtypes.cpu().numpy(), wl.n_elems_t.cpu().numpy()

    def part(ts):
        ts = np.array(ts)
        ro = np.concatenate([ref_off[ts], [0]])            # last entry unused: counts are passed explicitly
        co = np.concatenate([cand_off[t * wl.N:(t + 1) * wl.N] for t in ts])
        return ts, oracle.verify_ragged(ref_buf, ro, cand_buf, co, dtypes[ts], wl.N, wl.atol, wl.rtol, wl.equal_nan,
                                        n_elems=n_el[ts])

    chunks = [sample[i::8] for i in range(8)]
    with ThreadPoolExecutor(max_workers=8) as ex:
        for ts, want in ex.map(part, [c for c in chunks if c]):
            for a, t in enumerate(ts):
                g = got[t * wl.N:(t + 1) * wl.N]
                w = want[a * wl.N:(a + 1) * wl.N]
                assert g.tobytes() == w.tobytes(), f"tensor {t} (n={wl.n_elems[t]}, dtype {dtypes[t]})\n{g}\n{w}"
