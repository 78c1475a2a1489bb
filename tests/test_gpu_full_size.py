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


def test_tensor_beyond_32_gib_uses_64_bit_word_indices(oracle):
    """Maximum sizes: a 40 GiB int32 tensor (word indices of the hash pass 2^32, element indices pass
    2^33). The oracle would need minutes for it, so the checks are properties that hold at any size:
    an exact copy gives the zero record with the reference's hash; the reference hash equals what the
    separate gv_hash kernel computes; a candidate changed in three known places differs from the copy
    by exactly those three terms of the hash (recomputed here with Python integers), with the counts,
    first index and exact maximum difference known by construction."""
    free, _ = torch.cuda.mem_get_info()
    n = 10 * (1 << 30)
    need = 3 * n * 4 + (4 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of free device memory")
    g = torch.Generator(device=DEV).manual_seed(99)
    ref = torch.empty(n, dtype=torch.int32, device=DEV)
    step = 1 << 28
    for s in range(0, n, step):                               # fill in slices (bounded temporaries)
        ref[s:s + step] = torch.randint(-(1 << 30), 1 << 30, (min(step, n - s),), generator=g, device=DEV,
                                        dtype=torch.int32)
    copy = ref.clone()
    mod = ref.clone()
    places = [5, (1 << 33) + 11, n - 1]
    deltas = [7, -3, 1 << 20]
    old = [int(ref[p]) for p in places]
    for p, d in zip(places, deltas):
        mod[p] += d
    res = torch.empty((2, 64), dtype=torch.uint8, device=DEV)
    ws = torch.empty(gv.gv_workspace_bytes(0, 2), dtype=torch.uint8, device=DEV)
    rh = torch.zeros(1, dtype=torch.int64, device=DEV)
    gv.gv_verify_batch(ref, [copy, mod], results=res, ref_hash=rh, workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    got = gv.results_to_numpy(res)
    ref_hash = int(rh.cpu().numpy().view(np.uint64)[0])
    assert ref_hash == int(gv.gv_hash(ref).cpu().numpy().view(np.uint64)[0])
    zero = np.zeros((), dtype=gv.RESULT_DTYPE)
    zero["first_mismatch"] = gv.GV_NO_INDEX
    zero["hash"] = ref_hash
    assert got[0].tobytes() == zero.tobytes()
    assert int(got[1]["n_mismatch"]) == 3 and int(got[1]["first_mismatch"]) == 5
    assert int(got[1]["max_abs_diff_int"]) == 1 << 20
    # hash delta in closed form: only the three touched 64-bit words change
    M64 = (1 << 64) - 1
    want = ref_hash
    for p in places:
        k = p // 2
        w_old = int.from_bytes(host_bytes(ref[2 * k:2 * k + 2]).tobytes(), "little")
        w_new = int.from_bytes(host_bytes(mod[2 * k:2 * k + 2]).tobytes(), "little")
        want = (want - oracle.splitmix64(k ^ w_old) + oracle.splitmix64(k ^ w_new)) & M64
    assert int(got[1]["hash"]) == want
    assert old == [int(ref[p]) for p in places]
    del ref, copy, mod
    torch.cuda.empty_cache()
