"""GPU parity at the benchmark's full sizes, through the same call bench.py times.

Every record of every candidate is checked against what the workload recipe fixes by construction
(mismatch counts, first index, NaN/Inf counts, exact copies = zero record + reference hash), and
every record of every candidate (every tensor of the ragged batch) is checked byte for byte against
the CPU oracle, which computes those records one by one on the host (one candidate per host thread)."""
import ctypes
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_2507_23194_b200 import gv, workloads as W  # noqa: E402

DEV = "cuda:0"
THREADS = max(1, min(32, len(os.sched_getaffinity(0))))      # host threads for the oracle (it releases the GIL)


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

    with ThreadPoolExecutor(max_workers=THREADS) as ex:
        for j, want in ex.map(one, sample):
            assert got[j].tobytes() == want.tobytes(), (
                f"{wl.name}: candidate {j} ({wl.facts[j]['class']})\n gpu    {got[j]}\n oracle {want}")


def test_config2_full(oracle):
    wl = W.config2(DEV)
    assert wl.n == 4096 * 4096 and len(wl.cands) == 256
    got, rh = run_dense(wl)
    assert rh == oracle.hash_bytes(host_bytes(wl.ref))
    check_facts(wl, got, rh)
    oracle_sample(oracle, wl, got, range(len(wl.cands)))


def test_config3_full(oracle):
    wl = W.config3(DEV)
    assert wl.n == 8 * 32 * 4096 * 128 and len(wl.cands) == 32
    got, rh = run_dense(wl)
    assert rh == oracle.hash_bytes(host_bytes(wl.ref))
    check_facts(wl, got, rh)
    oracle_sample(oracle, wl, got, range(len(wl.cands)))
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
    oracle_sample(oracle, wl, got, range(len(wl.cands)))
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
    # the oracle on every tensor, split among the host threads largest first so that the parts are balanced
    order = np.argsort(-np.array(wl.n_elems))
    sample = order.tolist()
    ref_buf, cand_buf = wl.ref_buf.cpu().numpy(), wl.cand_buf.cpu().numpy()
    ref_off, cand_off = wl.ref_off.cpu().numpy(), wl.cand_off.cpu().numpy()
    dtypes, n_el = wl.dtypes.cpu().numpy(), wl.n_elems_t.cpu().numpy()

    def part(ts):
        ts = np.array(ts)
        ro = np.concatenate([ref_off[ts], [0]])            # last entry unused: counts are passed explicitly
        co = np.concatenate([cand_off[t * wl.N:(t + 1) * wl.N] for t in ts])
        return ts, oracle.verify_ragged(ref_buf, ro, cand_buf, co, dtypes[ts], wl.N, wl.atol, wl.rtol, wl.equal_nan,
                                        n_elems=n_el[ts])

    chunks = [sample[i::4 * THREADS] for i in range(4 * THREADS)]
    with ThreadPoolExecutor(max_workers=THREADS) as ex:
        for ts, want in ex.map(part, [c for c in chunks if c]):
            for a, t in enumerate(ts):
                g = got[t * wl.N:(t + 1) * wl.N]
                w = want[a * wl.N:(a + 1) * wl.N]
                assert g.tobytes() == w.tobytes(), f"tensor {t} (n={wl.n_elems[t]}, dtype {dtypes[t]})\n{g}\n{w}"


def _patterned_hash(oracle, n_words: int, word: int) -> int:
    """Hash of a buffer whose every 64-bit word equals `word`: sum over k < n_words of splitmix64(k xor word).
    For a block of 2^22 word indices starting at a multiple k0 of 2^22, (k0 + j) xor word = j xor (k0 xor word),
    so the block's terms are the oracle's hash of a 32 MiB host buffer filled with the word (k0 xor word): the
    34 GiB tensor's hash comes from the CPU oracle block by block without ever holding it on the host. One
    block is also recomputed with numpy uint64 arithmetic straight from the formula."""
    block = 1 << 22
    M64 = (1 << 64) - 1

    def part(k0):
        m = min(block, n_words - k0)
        return oracle.hash_bytes(np.full(m, (k0 ^ word) & M64, dtype=np.uint64))

    with ThreadPoolExecutor(max_workers=THREADS) as ex:
        total = sum(ex.map(part, range(0, n_words, block))) & M64
    k0 = 5 * block
    if k0 + block <= n_words:
        g, c1, c2 = np.uint64(0x9E3779B97F4A7C15), np.uint64(0xBF58476D1CE4E5B9), np.uint64(0x94D049BB133111EB)
        with np.errstate(over="ignore"):
            z = (np.arange(k0, k0 + block, dtype=np.uint64) ^ np.uint64(word)) + g
            z = (z ^ (z >> np.uint64(30))) * c1
            z = (z ^ (z >> np.uint64(27))) * c2
            z = z ^ (z >> np.uint64(31))
            assert int(z.sum(dtype=np.uint64)) == part(k0)
    return total


def _big_case(oracle, torch_dtype, word_elems, places, bump):
    """A 34+ GiB tensor whose every 64-bit word holds the same pattern (so its hash has a closed form that
    numpy evaluates from the definition), an exact copy, and a candidate changed at three known places."""
    esz = torch.empty(0, dtype=torch_dtype).element_size()
    per_word = 8 // esz
    n_words = (34 << 30) // 8 + 3                            # 34 GiB and a ragged tail: word indices pass 2^32
    n = n_words * per_word
    free, _ = torch.cuda.mem_get_info()
    need = 3 * n * esz + (4 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of free device memory")
    pat = torch.tensor(word_elems, dtype=torch_dtype, device=DEV)
    word = int.from_bytes(host_bytes(pat).tobytes(), "little")
    ref = pat.repeat(n_words)
    assert ref.numel() == n
    copy = ref.clone()
    mod = ref.clone()
    for p in places(n):
        mod[p] = bump(mod[p])
    res = torch.empty((2, 64), dtype=torch.uint8, device=DEV)
    ws = torch.empty(gv.gv_workspace_bytes(0, 2), dtype=torch.uint8, device=DEV)
    rh = torch.zeros(1, dtype=torch.int64, device=DEV)
    gv.gv_verify_batch(ref, [copy, mod], 1e-3, 1e-3, False, results=res, ref_hash=rh, workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    got = gv.results_to_numpy(res)
    want_hash = _patterned_hash(oracle, n_words, word)       # pinned outside CUDA
    assert int(rh.cpu().numpy().view(np.uint64)[0]) == want_hash, "reference hash of the dense kernel"
    assert int(gv.gv_hash(ref).cpu().numpy().view(np.uint64)[0]) == want_hash, "gv_hash"
    zero = np.zeros((), dtype=gv.RESULT_DTYPE)
    zero["first_mismatch"] = gv.GV_NO_INDEX
    zero["hash"] = want_hash
    assert got[0].tobytes() == zero.tobytes()
    # the changed candidate: only the touched words' terms differ, recomputed with Python integers
    M64 = (1 << 64) - 1
    want = want_hash
    for k in sorted({p // per_word for p in places(n)}):
        w_new = int.from_bytes(host_bytes(mod[k * per_word:(k + 1) * per_word]).tobytes(), "little")
        want = (want - oracle.splitmix64(k ^ word) + oracle.splitmix64(k ^ w_new)) & M64
    assert int(got[1]["hash"]) == want
    ps = sorted(places(n))
    assert int(got[1]["n_mismatch"]) == len(ps) and int(got[1]["first_mismatch"]) == ps[0]
    out = got[1].copy()
    del ref, copy, mod
    torch.cuda.empty_cache()
    return out


def test_int32_tensor_beyond_32_gib_uses_64_bit_word_indices(oracle):
    """Maximum sizes: a 34 GiB int32 tensor (word indices of the hash pass 2^32, element indices pass 2^33).
    The absolute hash is pinned by the closed form of a patterned buffer evaluated with numpy; counts, first
    index and the exact maximum difference of the changed candidate are known by construction."""
    got = _big_case(oracle, torch.int32, [0x1234567, -77], lambda n: [5, (1 << 33) + 11, n - 1], lambda v: v + (1 << 20))
    assert int(got["max_abs_diff_int"]) == 1 << 20 and got["max_abs_err"] == 0


def test_bf16_tensor_beyond_32_gib_uses_64_bit_word_indices(oracle):
    """The same for a float dtype (the float instances of the kernel with 64-bit word indices): 34 GiB of bf16,
    three elements raised by 0.5 (far outside the tolerance)."""
    got = _big_case(oracle, torch.bfloat16, [1.0, -2.0, 0.5, 3.0], lambda n: [3, (1 << 34) + 6, n - 2], lambda v: v + 0.5)
    assert got["max_abs_err"] == np.float32(0.5) and int(got["max_abs_diff_int"]) == 0
    assert got["max_rel_err"] == np.float32(1.0)            # 0.5 -> 1.0 at two of the places; 3.0 -> 3.5 at the third


def test_ragged_tensor_beyond_32_gib(oracle):
    """Maximum sizes, ragged path: one 34 GiB int32 tensor (it takes the unstreamed path with 64-bit word
    indices) next to a small one, one candidate each. The giant's hash is pinned by the patterned-buffer closed
    form evaluated by the oracle block by block; the changed places are known by construction; the small
    tensor's records are compared with the oracle directly."""
    n_words = (34 << 30) // 8 + 1
    n_big = n_words * 2
    n_small = 1000
    free, _ = torch.cuda.mem_get_info()
    need = 2 * (n_big + n_small) * 4 + (6 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of free device memory")
    pat = torch.tensor([0x0BADF00D, -12345], dtype=torch.int32, device=DEV)
    word = int.from_bytes(host_bytes(pat).tobytes(), "little")
    g = torch.Generator(device=DEV).manual_seed(7)
    small = torch.randint(-100, 100, (n_small,), generator=g, device=DEV, dtype=torch.int32)
    ref = torch.cat([pat.repeat(n_words), small])
    cand = ref.clone()
    places = [1, (1 << 33) + 2, n_big - 1]
    for p in places:
        cand[p] += 5
    cand[n_big + 17] -= 1
    ref_off = torch.tensor([0, n_big * 4, (n_big + n_small) * 4], dtype=torch.int64, device=DEV)
    cand_off = torch.tensor([0, n_big * 4], dtype=torch.int64, device=DEV)
    dtypes = torch.full((2,), 3, dtype=torch.uint8, device=DEV)
    ws = torch.empty(gv.gv_workspace_bytes(2, 1), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_ragged(ref.view(torch.uint8), ref_off, cand.view(torch.uint8), cand_off, dtypes, 1, 0.0, 0.0, False,
                              workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    got = gv.results_to_numpy(res)
    M64 = (1 << 64) - 1
    want = _patterned_hash(oracle, n_words, word)
    for k in sorted({p // 2 for p in places}):
        w_new = int.from_bytes(host_bytes(cand[2 * k:2 * k + 2]).tobytes(), "little")
        want = (want - oracle.splitmix64(k ^ word) + oracle.splitmix64(k ^ w_new)) & M64
    assert int(got[0]["hash"]) == want
    assert int(got[0]["n_mismatch"]) == 3 and int(got[0]["first_mismatch"]) == 1 and int(got[0]["max_abs_diff_int"]) == 5
    w_small = oracle.verify(host_bytes(small), host_bytes(cand[n_big:]), oracle.I32)
    assert got[1].tobytes() == w_small.tobytes()
    del ref, cand
    torch.cuda.empty_cache()
