"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle, record by record
and byte by byte (tolerance 0: every field of every record must be identical). Sizes here are ones
the oracle finishes in seconds; they span several tiles, ragged tails, unaligned bases, more than one
candidate chunk and more than one launch. Full-size workloads are in test_gpu_full_size.py."""
import ctypes

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():          # collected everywhere, run only where a GPU exists
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_2507_23194_b200 import gv, workloads as W  # noqa: E402

DEV = "cuda:0"
TDT = {0: torch.float32, 1: torch.bfloat16, 2: torch.float16, 3: torch.int32, 4: torch.int64}
ESZ = {0: 4, 1: 2, 2: 2, 3: 4, 4: 8}


def host_bytes(t: torch.Tensor) -> np.ndarray:
    """Raw bytes of a tensor as a numpy uint8 array (what the oracle consumes)."""
    return t.detach().contiguous().view(torch.uint8).cpu().numpy()


def oracle_batch(oracle, wl_ref, cands, code, atol, rtol, equal_nan):
    r = host_bytes(wl_ref)
    return oracle.verify_batch(r, [host_bytes(c) for c in cands], code, atol, rtol, equal_nan)


def assert_records_equal(got: np.ndarray, want: np.ndarray, tag=""):
    assert got.shape == want.shape, tag
    if got.tobytes() != want.tobytes():
        for j in range(len(got)):
            if got[j].tobytes() != want[j].tobytes():
                raise AssertionError(f"{tag}: record {j} differs\n gpu    {got[j]}\n oracle {want[j]}")


def run_dense(ref, cands, atol, rtol, equal_nan, want_ref_hash=True):
    rh = torch.zeros(1, dtype=torch.int64, device=DEV) if want_ref_hash else None
    ws = torch.empty(gv.gv_workspace_bytes(0, len(cands)), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_batch(ref, cands, atol, rtol, equal_nan, ref_hash=rh, workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    out = gv.results_to_numpy(res)
    return out, (int(rh.cpu().numpy().view(np.uint64)[0]) if want_ref_hash else None)


# ------------------------------------------------------------------------------------------------
# gv_hash
# ------------------------------------------------------------------------------------------------
def test_hash_all_small_sizes_and_offsets(oracle):
    g = torch.Generator(device="cpu").manual_seed(11)
    data = torch.randint(0, 256, (5000,), generator=g, dtype=torch.uint8)
    dev = data.to(DEV)
    sizes = list(range(0, 80)) + [255, 256, 257, 1023, 1024, 4095, 4096, 4097, 4113, 4999]
    for off in (0, 1, 3, 8, 16):
        for nb in sizes:
            if off + nb > 5000:
                continue
            got = int(gv.gv_hash(dev[off:off + nb]).cpu().numpy().view(np.uint64)[0])
            assert got == oracle.hash_bytes(data[off:off + nb].numpy()), (off, nb)


def test_hash_large_and_config1_tensors(oracle):
    wl = W.config1(DEV)
    for c in [wl.ref] + wl.cands:
        got = int(gv.gv_hash(c).cpu().numpy().view(np.uint64)[0])
        assert got == oracle.hash_bytes(host_bytes(c))
    z = torch.zeros(1 << 20, dtype=torch.float32, device=DEV)
    assert int(gv.gv_hash(z).cpu().numpy().view(np.uint64)[0]) == 0x8C6F9C0F16C4607B
    big = torch.randint(-2 ** 31, 2 ** 31 - 1, (50_000_001,), dtype=torch.int32, device=DEV)
    assert int(gv.gv_hash(big).cpu().numpy().view(np.uint64)[0]) == oracle.hash_bytes(host_bytes(big))


# ------------------------------------------------------------------------------------------------
# dense: config 1 in full (the tiny correctness case), by-construction facts and oracle parity
# ------------------------------------------------------------------------------------------------
def test_config1_full(oracle):
    wl = W.config1(DEV)
    got, rh = run_dense(wl.ref, wl.cands, wl.atol, wl.rtol, wl.equal_nan)
    want = oracle_batch(oracle, wl.ref, wl.cands, oracle.F32, wl.atol, wl.rtol, wl.equal_nan)
    assert_records_equal(got, want, "config1")
    assert rh == oracle.hash_bytes(host_bytes(wl.ref))
    # by construction (independent of either implementation)
    for j, f in enumerate(wl.facts):
        if "n_mismatch" in f:
            assert int(got[j]["n_mismatch"]) == f["n_mismatch"]
            assert int(got[j]["first_mismatch"]) == (gv.GV_NO_INDEX if f["first"] is None else f["first"])
        assert int(got[j]["n_nan_disagree"]) == f["n_nan"] and int(got[j]["n_inf_disagree"]) == f["n_inf"]
    assert got[4].tobytes() == got[2].tobytes()
    assert got[5]["max_rel_err"] == np.float32(2.0) and got[6]["max_rel_err"] == np.float32(1.0)
    assert int(got[0]["hash"]) == rh and int(got[6]["hash"]) == 0x8C6F9C0F16C4607B
    # invariance to candidate order: permuting the pointer list permutes the records
    perm = [3, 0, 7, 5, 1, 6, 2, 4]
    got_p, _ = run_dense(wl.ref, [wl.cands[i] for i in perm], wl.atol, wl.rtol, wl.equal_nan)
    for pos, src in enumerate(perm):
        assert got_p[pos].tobytes() == got[src].tobytes()


# ------------------------------------------------------------------------------------------------
# dense: sizes x dtypes x alignments, random data with injected specials
# ------------------------------------------------------------------------------------------------
def make_pair(code, n, seed, n_cands, specials=True):
    g = torch.Generator(device="cpu").manual_seed(seed)
    if code in (3, 4):
        lo, hi = (-(1 << 31), (1 << 31) - 1) if code == 3 else (-(1 << 62), (1 << 62))
        r = torch.randint(lo, hi, (n,), generator=g, dtype=TDT[code])
        cands = []
        for j in range(n_cands):
            c = r.clone()
            if n and j % 3 != 0:
                k = max(1, n // (50 * (j + 1)))
                pos = torch.randint(0, n, (k,), generator=g)
                c[pos] = torch.randint(lo, hi, (k,), generator=g, dtype=TDT[code])
            cands.append(c)
        if code == 4 and n >= 4 and n_cands >= 2:
            r[0], cands[1][0] = -(1 << 63), (1 << 63) - 1      # extreme difference, exact in u64
        return r, cands
    r = torch.randn(n, generator=g, dtype=torch.float32)
    if specials and n >= 64:
        pos = torch.randint(0, n, (12,), generator=g)
        r[pos[0:2]] = float("nan")
        r[pos[2:4]] = float("inf")
        r[pos[4:6]] = float("-inf")
        r[pos[6:9]] = 0.0
        r[pos[9:12]] = -0.0
    r = r.to(TDT[code])
    cands = []
    for j in range(n_cands):
        kind = j % 6
        rf = r.float()
        if kind == 0:
            c = r.clone()
        elif kind == 1:
            c = (rf * (1 + 1e-3 * torch.randn(n, generator=g))).to(TDT[code])
        elif kind == 2:
            c = (rf + 0.05 * torch.randn(n, generator=g)).to(TDT[code])
        elif kind == 3:
            c = r.clone()
            if n:
                pos = torch.randint(0, n, (max(1, n // 100),), generator=g)
                vals = torch.tensor([float("nan"), float("inf"), float("-inf"), 0.0, 1e30, -1e30])
                c[pos] = vals[torch.randint(0, 6, (pos.numel(),), generator=g)].to(TDT[code])
        elif kind == 4:
            c = torch.zeros_like(r)
        else:
            c = (-rf).to(TDT[code])
        cands.append(c)
    return r, cands


SIZES = [0, 1, 2, 3, 7, 8, 9, 15, 16, 17, 255, 1023, 1024, 1025, 2047, 2048, 2049, 4096, 4100, 8191, 8192, 8193,
         12289, 20000, 65536 + 5]


@pytest.mark.parametrize("code", [0, 1, 2, 3, 4])
def test_dense_size_sweep(oracle, code):
    for i, n in enumerate(SIZES):
        r, cands = make_pair(code, n, 100 + i, n_cands=7)
        rd, cd = r.to(DEV), [c.to(DEV) for c in cands]
        for atol, rtol, en in [(1e-2, 1e-2, False), (0.0, 0.0, True)]:
            got, rh = run_dense(rd, cd, atol, rtol, en)
            want = oracle.verify_batch(host_bytes(r), [host_bytes(c) for c in cands], code, atol, rtol, en)
            assert_records_equal(got, want, f"dtype {code} n {n} tol {atol}")
            assert rh == oracle.hash_bytes(host_bytes(r))


@pytest.mark.parametrize("code", [0, 1, 2, 3, 4])
def test_dense_unaligned_bases(oracle, code):
    # reference and candidates start at element offsets 0..3 inside larger buffers (not 16-byte aligned)
    n = 9000
    for shift_r, shift_c in [(1, 0), (0, 1), (1, 1), (3, 2), (2, 3)]:
        r, cands = make_pair(code, n + 8, 7 + shift_r, n_cands=5)
        rd = r.to(DEV)[shift_r:shift_r + n]
        cd = [c.to(DEV)[(shift_c + j) % 4:(shift_c + j) % 4 + n] for j, c in enumerate(cands)]
        got, rh = run_dense(rd, cd, 1e-2, 1e-2, True)
        want = oracle.verify_batch(host_bytes(rd), [host_bytes(c) for c in cd], code, 1e-2, 1e-2, True)
        assert_records_equal(got, want, f"dtype {code} shifts {shift_r},{shift_c}")
        assert rh == oracle.hash_bytes(host_bytes(rd))


@pytest.mark.parametrize("code,n_cands", [(1, 17), (0, 33), (3, 40), (2, 300)])
def test_dense_many_candidates(oracle, code, n_cands):
    # more than one chunk of candidates; 300 > the per-launch pointer limit
    n = 30000 if n_cands < 100 else 5000
    r, cands = make_pair(code, n, 42, n_cands)
    got, _ = run_dense(r.to(DEV), [c.to(DEV) for c in cands], 1e-2, 1e-2, False)
    want = oracle.verify_batch(host_bytes(r), [host_bytes(c) for c in cands], code, 1e-2, 1e-2, False)
    assert_records_equal(got, want, f"dtype {code} N {n_cands}")


@pytest.mark.parametrize("code", [1, 2])
def test_all_16bit_patterns_against_interesting_references(oracle, code):
    raw_c = torch.arange(1 << 16, dtype=torch.int32).to(torch.int16).view(TDT[code])
    refs = ([0x0000, 0x8000, 0x0001, 0x0080, 0x3F80, 0xBF80, 0x7F7F, 0xFF7F, 0x7F80, 0xFF80, 0x7FC0, 0x3F7F, 0x4049]
            if code == 1 else
            [0x0000, 0x8000, 0x0001, 0x03FF, 0x0400, 0x3C00, 0xBC00, 0x7BFF, 0xFBFF, 0x7C00, 0xFC00, 0x7E00, 0x4248])
    cd = raw_c.to(DEV)
    for rb in refs:
        r = torch.full((1 << 16,), rb, dtype=torch.int32).to(torch.int16).view(TDT[code])
        for atol, rtol, en in [(1e-2, 1e-2, False), (0.0, 0.0, True), (1e30, 1e30, False)]:
            got, _ = run_dense(r.to(DEV), [cd], atol, rtol, en)
            want = oracle.verify_batch(host_bytes(r), [host_bytes(raw_c)], code, atol, rtol, en)
            assert_records_equal(got, want, f"dtype {code} ref {rb:#x} tol {atol}")


def test_fp32_canaries_and_extremes(oracle):
    # the golden truth-table rows as one batch, each row its own 1-element call, plus a tensor of
    # extreme values crossed with itself
    bits = np.array([0x00000000, 0x80000000, 0x00000001, 0x80000001, 0x007FFFFF, 0x00800000, 0x00800001,
                     0x3F800000, 0xBF800000, 0x7F7FFFFF, 0xFF7FFFFF, 0x7F800000, 0xFF800000, 0x7FC00000,
                     0xFFC00001, 0x3F7FFFFF, 0x3F800001, 0x7F61B1E6, 0xFF61B1E6, 0xBF38FA9F, 0xBF38F97E,
                     0x3F640C03, 0x3F68E32C, 0x3A78DE92, 0x3F8A0F08], dtype=np.uint32)
    c = torch.from_numpy(np.repeat(bits, len(bits)).view(np.float32).copy())
    r = torch.from_numpy(np.tile(bits, len(bits)).view(np.float32).copy())
    for atol, rtol, en in [(0.0, 0.0, False), (1e-5, 1e-5, False), (1e-2, 1e-2, True), (0.0, 2.0, False),
                           (1e30, 1e30, True)]:
        got, _ = run_dense(r.to(DEV), [c.to(DEV)], atol, rtol, en)
        want = oracle.verify_batch(host_bytes(r), [host_bytes(c)], oracle.F32, atol, rtol, en)
        assert_records_equal(got, want, f"extremes tol {atol},{rtol}")
        # element by element too, so compensating errors cannot hide in the aggregate
        if (atol, rtol) in [(1e-5, 1e-5), (0.0, 2.0)]:
            cd, rd = c.to(DEV), r.to(DEV)
            singles = [cd[i:i + 1].clone() for i in range(0, len(c), 7)]
            for i, s in zip(range(0, len(c), 7), singles):
                g1, _ = run_dense(rd[i:i + 1].clone(), [s], atol, rtol, en, want_ref_hash=False)
                w1 = oracle.verify(host_bytes(r[i:i + 1]), host_bytes(c[i:i + 1]), oracle.F32, atol, rtol, en)
                assert g1[0].tobytes() == w1.tobytes(), (i, g1[0], w1)


def test_dense_empty_inputs(oracle):
    r = torch.zeros(0, dtype=torch.float32, device=DEV)
    got, rh = run_dense(r, [r.clone(), r.clone()], 1e-3, 1e-3, False)
    for rec in got:
        assert int(rec["n_mismatch"]) == 0 and int(rec["first_mismatch"]) == gv.GV_NO_INDEX
        assert int(rec["hash"]) == 0 and rec["max_abs_err"] == 0 and rec["max_rel_err"] == 0
    assert rh == 0
    r = torch.randn(1000, device=DEV)
    got, rh = run_dense(r, [], 1e-3, 1e-3, False)
    assert len(got) == 0 and rh == oracle.hash_bytes(host_bytes(r))


def test_results_independent_of_schedule(oracle):
    # the same data verified as one batch, as single-candidate calls and in another order
    r, cands = make_pair(1, 70001, 5, 9)
    rd, cd = r.to(DEV), [c.to(DEV) for c in cands]
    a, _ = run_dense(rd, cd, 1e-2, 1e-2, True)
    for j in range(9):
        b, _ = run_dense(rd, [cd[j]], 1e-2, 1e-2, True)
        assert a[j].tobytes() == b[0].tobytes()
    c, _ = run_dense(rd, cd[::-1], 1e-2, 1e-2, True)
    assert c[::-1].tobytes() == a.tobytes()


# ------------------------------------------------------------------------------------------------
# differing vectors at every density: from none to all 32 lanes of a warp-tile, several tiles per warp
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("code,equal_nan,n_cands", [(1, True, 16), (0, False, 16), (2, True, 16), (3, False, 16),
                                                    (1, False, 37), (0, True, 37), (3, False, 21)])
def test_differing_lane_densities(oracle, code, equal_nan, n_cands):
    """Candidate j differs from the reference in a fraction (j mod 16)/15 of its 16-byte vectors, so the
    kernel meets visits with anything from 0 to 32 differing lanes. The tensors are large enough for
    the sampling pass to classify the candidates; with 37 or 21 of them both loops run (queued and
    in-place compares), one chunk straddles the classes, the last chunks hold 4 and 1 candidates,
    queues wrap around and are drained at chunk ends. The differing vectors mix noise inside the
    tolerance, plain mismatches and, for float dtypes, NaN/Inf; the reference itself holds a few NaNs."""
    g = torch.Generator().manual_seed(4242 + code)
    n = (6 * (1 << 20) + 1000 if ESZ[code] == 2 else 3 * (1 << 20) + 1000) // (1 if n_cands == 16 else 2)
    epv = 16 // ESZ[code]
    nv = n // epv
    if code == 3:
        r = torch.randint(-(1 << 20), 1 << 20, (n,), generator=g, dtype=torch.int32)
    else:
        r = torch.randn(n, generator=g).to(TDT[code])
        r[torch.randint(0, n, (64,), generator=g)] = float("nan")
    cands = []
    for j in range(n_cands):
        pick = torch.rand(nv, generator=g) < (((j * 7) % 16) / 15.0)
        elem = pick.repeat_interleave(epv)
        elem = torch.cat([elem, torch.zeros(n - nv * epv, dtype=torch.bool)])
        elem &= torch.rand(n, generator=g) < 0.6                      # not every element of a picked vector
        c = r.clone()
        if code == 3:
            c[elem] += torch.randint(1, 5, (int(elem.sum()),), generator=g, dtype=torch.int32)
        else:
            kind = torch.rand(n, generator=g)
            rf = r.float()
            small = (rf * (1 + 2e-3 * torch.randn(n, generator=g))).to(TDT[code])
            big = (rf + 1.0).to(TDT[code])
            c = torch.where(elem & (kind < 0.9), small, c)
            c = torch.where(elem & (kind >= 0.9) & (kind < 0.995), big, c)
            c = torch.where(elem & (kind >= 0.995) & (kind < 0.998), torch.full_like(c, float("inf")), c)
            c = torch.where(elem & (kind >= 0.998), torch.full_like(c, float("nan")), c)
        cands.append(c)
    got, rh = run_dense(r.to(DEV), [c.to(DEV) for c in cands], 1e-2, 1e-2, equal_nan)
    want = oracle_batch(oracle, r, cands, code, 1e-2, 1e-2, equal_nan)
    assert_records_equal(got, want, f"densities dtype {code}")
    assert rh == oracle.hash_bytes(host_bytes(r))


# ------------------------------------------------------------------------------------------------
# reduced versions of the dense workload recipes
# ------------------------------------------------------------------------------------------------
def test_reduced_configs_2_3_4(oracle):
    for wl in (W.config2(DEV, n=(1 << 18) + 24, n_cands=40), W.config3(DEV, n=(1 << 18) + 8, n_cands=10),
               W.config4(DEV, n=1 << 18, n_cands=12), W.config4(DEV, n=(1 << 17) + 2, n_cands=12, wide=True)):
        got, rh = run_dense(wl.ref, wl.cands, wl.atol, wl.rtol, wl.equal_nan)
        want = oracle_batch(oracle, wl.ref, wl.cands, wl.dtype, wl.atol, wl.rtol, wl.equal_nan)
        assert_records_equal(got, want, wl.name)
        for j, f in enumerate(wl.facts):
            if "n_mismatch" in f:
                assert int(got[j]["n_mismatch"]) == f["n_mismatch"], (wl.name, j)
            if f.get("hash_equals_ref"):
                assert int(got[j]["hash"]) == rh


# ------------------------------------------------------------------------------------------------
# ragged
# ------------------------------------------------------------------------------------------------
def run_ragged(wl, with_counts=True):
    ws = torch.empty(gv.gv_workspace_bytes(wl.T, wl.N), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_ragged(wl.ref_buf, wl.ref_off, wl.cand_buf, wl.cand_off, wl.dtypes, wl.N, wl.atol, wl.rtol,
                              wl.equal_nan, n_elems=wl.n_elems_t if with_counts else None, workspace=ws)
    torch.cuda.synchronize()
    return gv.results_to_numpy(res), gv.gv_check(ws)


def oracle_ragged(oracle, wl):
    return oracle.verify_ragged(wl.ref_buf.cpu().numpy(), wl.ref_off.cpu().numpy(), wl.cand_buf.cpu().numpy(),
                                wl.cand_off.cpu().numpy(), wl.dtypes.cpu().numpy(), wl.N, wl.atol, wl.rtol,
                                wl.equal_nan, n_elems=wl.n_elems_t.cpu().numpy())


@pytest.mark.parametrize("align", [16, 0])
def test_ragged_reduced_config5(oracle, align):
    wl = W.config5(DEV, T=300, max_log2=16.0, align=align)
    got, status = run_ragged(wl)
    assert status == gv.GV_OK
    want = oracle_ragged(oracle, wl)
    assert_records_equal(got, want, f"ragged align {align}")
    for i, f in enumerate(wl.facts):
        assert int(got[i]["n_mismatch"]) == f["n_mismatch"]
        assert int(got[i]["first_mismatch"]) == (gv.GV_NO_INDEX if f["first"] is None else f["first"])


def test_ragged_counts_from_offsets_and_bad_table(oracle):
    # tightly packed int32 tensors: element counts read off consecutive offsets
    g = torch.Generator(device="cpu").manual_seed(3)
    sizes = [0, 1, 5, 4096, 4097, 10000, 3]
    offs = np.concatenate([[0], np.cumsum([4 * s for s in sizes])]).astype(np.int64)
    total = int(offs[-1])
    ref = torch.randint(-100, 100, (total // 4,), generator=g, dtype=torch.int32)
    N = 3
    cand = torch.cat([ref.clone() for _ in range(N)])
    cand[5] += 1
    cand_off = np.array([[offs[t] + j * total for j in range(N)] for t in range(len(sizes))], dtype=np.int64).reshape(-1)
    dtypes = torch.full((len(sizes),), 3, dtype=torch.uint8)
    ws = torch.empty(gv.gv_workspace_bytes(len(sizes), N), dtype=torch.uint8, device=DEV)
    args = (ref.view(torch.uint8).to(DEV), torch.from_numpy(offs).to(DEV), cand.view(torch.uint8).to(DEV),
            torch.from_numpy(cand_off).to(DEV), dtypes.to(DEV), N, 0.0, 0.0, False)
    res = gv.gv_verify_ragged(*args, workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    want = oracle.verify_ragged(host_bytes(ref), offs, host_bytes(cand), cand_off, dtypes.numpy(), N, 0.0, 0.0, False)
    assert_records_equal(gv.results_to_numpy(res), want, "ragged tight int32")
    # a decreasing offset is flagged, not followed
    bad = offs.copy()
    bad[3] = bad[2] - 8
    res = gv.gv_verify_ragged(args[0], torch.from_numpy(bad).to(DEV), *args[2:], workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_ERR_BAD_TABLE


# ------------------------------------------------------------------------------------------------
# host-buffer entry point
# ------------------------------------------------------------------------------------------------
def test_verify_batch_host(oracle):
    r, cands = make_pair(1, 50003, 9, 11)
    rp, cp = r.pin_memory(), [c.pin_memory() for c in cands]
    for slab in (1, 4, 64):
        staging = torch.empty(gv.gv_host_staging_bytes(r.numel(), 1, slab), dtype=torch.uint8, device=DEV)
        got, rh = gv.gv_verify_batch_host(rp, cp, 1e-2, 1e-2, True, staging)
        want = oracle.verify_batch(host_bytes(r), [host_bytes(c) for c in cands], 1, 1e-2, 1e-2, True)
        assert_records_equal(got, want, f"host entry slab {slab}")
        assert rh == oracle.hash_bytes(host_bytes(r))


# ------------------------------------------------------------------------------------------------
# randomised sweep: dtype x size x alignment x candidate count x tolerances x value patterns
# ------------------------------------------------------------------------------------------------
def _rand_values(rng, code, n):
    """Reference values with a seeded mixture of scales and special values."""
    if code in (3, 4):
        info = np.iinfo(np.int32 if code == 3 else np.int64)
        kind = rng.integers(0, 3)
        if kind == 0:
            a = rng.integers(-100, 100, n)
        elif kind == 1:
            a = rng.integers(info.min, info.max, n, dtype=np.int64, endpoint=False)
        else:
            a = rng.choice(np.array([0, 1, -1, info.min, info.max]), n)
        return torch.from_numpy(a.astype(np.int32 if code == 3 else np.int64))
    scale = float(10.0 ** rng.integers(-8, 6))
    a = (rng.standard_normal(n) * scale).astype(np.float32)
    if n and rng.random() < 0.7:
        k = max(1, n // 50)
        pos = rng.integers(0, n, k)
        a[pos] = rng.choice(np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 1e-40, -1e-45, 3e38, 65504.0, 1.0],
                                     dtype=np.float32), k)
    return torch.from_numpy(a).to(TDT[code])


def _rand_candidate(rng, code, r):
    n = r.numel()
    kind = rng.integers(0, 7)
    if code in (3, 4):
        c = r.clone()
        if kind >= 2 and n:
            k = max(1, int(n * float(rng.choice([1e-3, 0.05, 1.0]))))
            pos = torch.from_numpy(rng.integers(0, n, k))
            c[pos] = _rand_values(rng, code, k)
        return c
    rf = r.float()
    if kind == 0 or n == 0:
        return r.clone()
    if kind == 1:
        return (rf * (1 + float(10.0 ** rng.integers(-7, -1)) * torch.from_numpy(rng.standard_normal(n).astype(np.float32)))).to(TDT[code])
    if kind == 2:
        return (rf + float(10.0 ** rng.integers(-9, 2)) * torch.from_numpy(rng.standard_normal(n).astype(np.float32))).to(TDT[code])
    if kind == 3:
        return torch.zeros_like(r)
    if kind == 4:
        return _rand_values(rng, code, n)
    c = r.clone()
    k = max(1, n // int(rng.choice([3, 30, 300])))
    pos = torch.from_numpy(rng.integers(0, n, k))
    c[pos] = _rand_values(rng, code, k)
    return c


@pytest.mark.parametrize("seed", range(12))
def test_randomised_sweep(oracle, seed):
    rng = np.random.default_rng(1000 + seed)
    for _ in range(30):
        code = int(rng.integers(0, 5))
        n = int(rng.choice([0, 1, 5, 33, 127, 128, 129, 1000, 4099, 8192 + 3, 40000, 100003]))
        n_cands = int(rng.choice([1, 2, 5, 16, 17, 31]))
        shift_r = int(rng.integers(0, 3)) if rng.random() < 0.3 else 0
        r_full = _rand_values(rng, code, n + 4)
        r = r_full[shift_r:shift_r + n]
        cands = []
        for j in range(n_cands):
            c_full = torch.zeros(n + 4, dtype=TDT[code])
            sh = int(rng.integers(0, 3)) if rng.random() < 0.2 else 0
            c_full[sh:sh + n] = _rand_candidate(rng, code, r)
            cands.append((c_full, sh))
        atol = float(rng.choice([0.0, 1e-8, 1e-3, 1.0, 1e30]))
        rtol = float(rng.choice([0.0, 1e-6, 1e-2, 0.5, 2.0]))
        en = bool(rng.integers(0, 2))
        rd_full = r_full.to(DEV)
        rd = rd_full[shift_r:shift_r + n]
        cd_full = [c.to(DEV) for c, _ in cands]
        cd = [cf[sh:sh + n] for cf, (_, sh) in zip(cd_full, cands)]
        got, rh = run_dense(rd, cd, atol, rtol, en)
        want = oracle.verify_batch(host_bytes(r), [host_bytes(c[sh:sh + n]) for c, sh in cands], code, atol, rtol, en)
        assert_records_equal(got, want, f"seed {seed} dtype {code} n {n} N {n_cands} tol {atol},{rtol},{en}")
        assert rh == oracle.hash_bytes(host_bytes(r))


@pytest.mark.parametrize("seed", range(16))
def test_randomised_ragged(oracle, seed):
    # random tensors of all five dtypes (including empty ones), random candidate counts, tight or
    # padded packing, special values; element counts passed explicitly
    rng = np.random.default_rng(2000 + seed)
    T = int(rng.choice([1, 7, 60, 150]))
    N = int(rng.choice([1, 3, 4, 17]))
    align = int(rng.choice([0, 16]))
    codes = rng.integers(0, 5, T)
    sizes = [int(rng.choice([0, 1, 3, 31, 64, 65, 127, 128, 129, 1000, 5000, 20011])) for _ in range(T)]
    ref_chunks, cand_chunks, ref_off, cand_off = [], [], [], []
    rc = cc = 0

    def place(cur, esz):
        a = align if align else esz
        return (cur + a - 1) // a * a

    for t in range(T):
        code, n = int(codes[t]), sizes[t]
        esz = ESZ[code]
        r = _rand_values(rng, code, n)
        start = place(rc, esz)
        ref_chunks.append((start, r))
        ref_off.append(start)
        rc = start + n * esz
        for j in range(N):
            c = _rand_candidate(rng, code, r)
            start = place(cc, esz)
            cand_chunks.append((start, c))
            cand_off.append(start)
            cc = start + n * esz
    ref_off.append(rc)
    ref_buf = torch.zeros(max(rc, 1), dtype=torch.uint8)
    cand_buf = torch.zeros(max(cc, 1), dtype=torch.uint8)
    for start, x in ref_chunks:
        if x.numel():
            ref_buf[start:start + x.numel() * x.element_size()] = x.contiguous().view(torch.uint8)
    for start, x in cand_chunks:
        if x.numel():
            cand_buf[start:start + x.numel() * x.element_size()] = x.contiguous().view(torch.uint8)
    ref_off_t = torch.tensor(ref_off, dtype=torch.int64)
    cand_off_t = torch.tensor(cand_off, dtype=torch.int64)
    dtypes_t = torch.tensor(codes, dtype=torch.uint8)
    n_el = torch.tensor(sizes, dtype=torch.int64)
    atol = float(rng.choice([0.0, 1e-3, 1.0]))
    rtol = float(rng.choice([0.0, 1e-2, 0.5]))
    en = bool(rng.integers(0, 2))
    ws = torch.empty(gv.gv_workspace_bytes(T, N), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_ragged(ref_buf.to(DEV), ref_off_t.to(DEV), cand_buf.to(DEV), cand_off_t.to(DEV),
                              dtypes_t.to(DEV), N, atol, rtol, en, n_elems=n_el.to(DEV), workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    want = oracle.verify_ragged(ref_buf.numpy(), ref_off_t.numpy(), cand_buf.numpy(), cand_off_t.numpy(),
                                dtypes_t.numpy(), N, atol, rtol, en, n_elems=n_el.numpy())
    assert_records_equal(gv.results_to_numpy(res), want, f"ragged seed {seed} T {T} N {N} align {align}")


def test_ragged_differing_lane_densities(oracle):
    """A few large tensors of every dtype, five candidates each with a differing-vector fraction of
    0, 1/4, 1/2, 3/4 and 1: warps stream many tiles of one tensor, their queues of differing vectors
    fill, wrap around and are drained when the warp leaves the tensor."""
    g = torch.Generator().manual_seed(777)
    N, T = 5, 10
    sizes = [(1 << 20) + 77, (1 << 19) + 5, 3 * (1 << 18), (1 << 20) - 3, (1 << 18) + 1, 40000, (1 << 19), 999999,
             (1 << 17) + 9, 1 << 20]
    codes = [0, 1, 2, 3, 4, 1, 0, 2, 3, 1]
    refs, cands = [], []
    for t in range(T):
        code, n = codes[t], sizes[t]
        if code >= 3:
            r = torch.randint(-(1 << 20), 1 << 20, (n,), generator=g, dtype=TDT[code])
        else:
            r = torch.randn(n, generator=g).to(TDT[code])
            r[torch.randint(0, n, (16,), generator=g)] = float("nan")
        refs.append(r)
        epv = 16 // ESZ[code]
        for j in range(N):
            pick = (torch.rand(n // epv + 1, generator=g) < j / 4.0).repeat_interleave(epv)[:n]
            pick &= torch.rand(n, generator=g) < 0.5
            if code >= 3:
                c = torch.where(pick, r + 3, r)
            else:
                kind = torch.rand(n, generator=g)
                c = torch.where(pick & (kind < 0.9), (r.float() * (1 + 2e-3 * torch.randn(n, generator=g))).to(TDT[code]), r)
                c = torch.where(pick & (kind >= 0.9) & (kind < 0.997), (r.float() - 2.0).to(TDT[code]), c)
                c = torch.where(pick & (kind >= 0.997), torch.full_like(c, float("-inf")), c)
            cands.append(c)
    ref_off, cand_off, rc, cc = [], [], 0, 0
    for t in range(T):
        nb = sizes[t] * ESZ[codes[t]]
        rc = (rc + 15) // 16 * 16
        ref_off.append(rc)
        rc += nb
        for j in range(N):
            cc = (cc + 15) // 16 * 16
            cand_off.append(cc)
            cc += nb
    ref_off.append(rc)
    ref_buf = torch.zeros(rc, dtype=torch.uint8)
    cand_buf = torch.zeros(cc, dtype=torch.uint8)
    for t in range(T):
        nb = sizes[t] * ESZ[codes[t]]
        ref_buf[ref_off[t]:ref_off[t] + nb] = refs[t].view(torch.uint8)
        for j in range(N):
            o = cand_off[t * N + j]
            cand_buf[o:o + nb] = cands[t * N + j].view(torch.uint8)
    ref_off_t, cand_off_t = torch.tensor(ref_off), torch.tensor(cand_off)
    dtypes_t, n_el = torch.tensor(codes, dtype=torch.uint8), torch.tensor(sizes)
    for en in (False, True):
        ws = torch.empty(gv.gv_workspace_bytes(T, N), dtype=torch.uint8, device=DEV)
        res = gv.gv_verify_ragged(ref_buf.to(DEV), ref_off_t.to(DEV), cand_buf.to(DEV), cand_off_t.to(DEV),
                                  dtypes_t.to(DEV), N, 1e-2, 1e-2, en, n_elems=n_el.to(DEV), workspace=ws)
        torch.cuda.synchronize()
        assert gv.gv_check(ws) == gv.GV_OK
        want = oracle.verify_ragged(ref_buf.numpy(), ref_off_t.numpy(), cand_buf.numpy(), cand_off_t.numpy(),
                                    dtypes_t.numpy(), N, 1e-2, 1e-2, en, n_elems=n_el.numpy())
        assert_records_equal(gv.results_to_numpy(res), want, f"ragged densities equal_nan {en}")


@pytest.mark.parametrize("code", [1, 0])
def test_candidates_that_fool_the_sampling_pass(oracle, code):
    """The sampling pass that picks a loop per candidate looks at 64 evenly spread 512-byte tiles. Here
    candidates differ from the reference exactly in those tiles and nowhere else (flagged as differing
    everywhere, in fact almost identical), everywhere but in those tiles (the opposite), in the first
    or second half only, plus plain copies and fully noisy ones, in an order that mixes the classes:
    the records must not depend on which loop a candidate was given."""
    g = torch.Generator().manual_seed(31 + code)
    per_tile = 512 // ESZ[code]
    tiles = 16384
    n = tiles * per_tile
    r = torch.randn(n, generator=g).to(TDT[code])
    noisy = (r.float() * (1 + 3e-2 * torch.randn(n, generator=g)) + 1e-3).to(TDT[code])
    tile_of = torch.arange(n) // per_tile
    sampled = (tile_of % (tiles // 64)) == 0
    first_half = tile_of < tiles // 2
    cands = [r.clone(), torch.where(sampled, noisy, r), torch.where(sampled, r, noisy), noisy.clone(),
             torch.where(first_half, noisy, r), torch.where(first_half, r, noisy), r.clone(), noisy.clone(),
             torch.where(sampled, noisy, r), noisy.clone(), torch.where(sampled, r, noisy)]
    got, rh = run_dense(r.to(DEV), [c.to(DEV) for c in cands], 1e-2, 1e-2, False)
    want = oracle_batch(oracle, r, cands, code, 1e-2, 1e-2, False)
    assert_records_equal(got, want, f"sampling dtype {code}")
    assert rh == oracle.hash_bytes(host_bytes(r))
    assert got[1].tobytes() == got[8].tobytes() and got[3].tobytes() == got[7].tobytes() == got[9].tobytes()


def test_many_classified_candidates_over_two_launches(oracle):
    """300 candidates of 256 KB each: more than one launch of 256 (the classification bytes of the second
    launch follow those of the first in the workspace), enough bytes for the sampling pass to run, and
    a second launch of 44 = 16 + 16 + 12 candidates. Every third candidate differs everywhere."""
    g = torch.Generator().manual_seed(2024)
    n = 128 * 1024
    r = torch.randn(n, generator=g).to(torch.bfloat16)
    noisy = [(r.float() * (1 + 2e-2 * torch.randn(n, generator=g))).to(torch.bfloat16) for _ in range(5)]
    cands = []
    for j in range(300):
        if j % 3 == 0:
            c = noisy[j % 5].clone()
            c[j] = float(j)                                   # make every record distinct
        else:
            c = r.clone()
            if j % 3 == 1:
                c[(j * 37) % n] = 100.0
        cands.append(c)
    got, rh = run_dense(r.to(DEV), [c.to(DEV) for c in cands], 1e-2, 1e-2, True)
    want = oracle_batch(oracle, r, cands, 1, 1e-2, 1e-2, True)
    assert_records_equal(got, want, "300 classified candidates")
    assert rh == oracle.hash_bytes(host_bytes(r))


@pytest.mark.parametrize("seed", range(6))
def test_randomised_large_batches(oracle, seed):
    """Random dtype, candidate count (1 ... 40), differing-vector density per candidate (0 ... 1),
    tolerances and equal_nan at 64-160 MB of candidates per call: the sizes at which the sampling pass
    runs and every chunk shape and loop of the dense kernel occurs."""
    for case in range(4):
        rng = np.random.default_rng(7000 + seed * 10 + case)
        g = torch.Generator().manual_seed(7000 + seed * 10 + case)
        code = int(rng.integers(0, 5))
        N = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 12, 16, 17, 20, 31, 33, 40]))
        n = (int(rng.integers(64, 160)) << 20) // (N * ESZ[code]) + int(rng.integers(0, 64))
        if code >= 3:
            r = torch.randint(-(1 << 20), 1 << 20, (n,), generator=g, dtype=TDT[code])
        else:
            r = (torch.randn(n, generator=g) * float(10.0 ** rng.integers(-3, 3))).to(TDT[code])
            if rng.random() < 0.5:
                r[torch.randint(0, n, (8,), generator=g)] = float("nan")
        epv = 16 // ESZ[code]
        cands = []
        for j in range(N):
            p = float(rng.choice([0.0, 0.0, 0.001, 0.05, 0.3, 0.6, 0.9, 1.0]))
            if p == 0.0:
                cands.append(r.clone())
                continue
            pick = (torch.rand(n // epv + 1, generator=g) < p).repeat_interleave(epv)[:n]
            if code >= 3:
                cands.append(torch.where(pick, r + int(rng.integers(1, 9)), r))
                continue
            kind = int(rng.integers(0, 3))
            if kind == 1:
                alt = (r.float() + 1.0).to(TDT[code])
            else:
                alt = (r.float() * (1 + 1e-2 * torch.randn(n, generator=g))).to(TDT[code])
            if kind == 2:
                alt[torch.randint(0, n, (64,), generator=g)] = float("inf")
                alt[torch.randint(0, n, (64,), generator=g)] = float("nan")
            cands.append(torch.where(pick, alt, r))
        atol = float(rng.choice([0.0, 1e-3, 1e-2]))
        rtol = float(rng.choice([0.0, 1e-2, 0.1]))
        en = bool(rng.integers(0, 2))
        got, rh = run_dense(r.to(DEV), [c.to(DEV) for c in cands], atol, rtol, en)
        want = oracle_batch(oracle, r, cands, code, atol, rtol, en)
        assert_records_equal(got, want, f"large seed {seed} case {case} dtype {code} N {N} n {n}")
        assert rh == oracle.hash_bytes(host_bytes(r))
        torch.cuda.empty_cache()


def test_hash2_sizes_and_offsets(oracle):
    # the second hash lane against the oracle: every small size, unaligned bases, a large buffer
    rng = np.random.default_rng(21)
    data = torch.from_numpy(rng.integers(0, 256, size=(1 << 22) + 100, dtype=np.uint8))
    dd = data.to(DEV)
    for off in (0, 1, 3, 8, 16):
        for nbytes in list(range(0, 50)) + [255, 256, 257, 4095, 4096, 4097, 65536 + 5]:
            h = gv.gv_hash2(dd[off:off + nbytes])
            assert int(h.cpu().numpy().view(np.uint64)[0]) == oracle.hash2_bytes(data[off:off + nbytes].numpy()), (off, nbytes)
    h = gv.gv_hash2(dd[:1 << 22])
    assert int(h.cpu().numpy().view(np.uint64)[0]) == oracle.hash2_bytes(data[:1 << 22].numpy())
    z, o = torch.zeros(2, dtype=torch.int64, device=DEV), torch.ones(2, dtype=torch.int64, device=DEV)
    assert int(gv.gv_hash(z).cpu()[0]) == int(gv.gv_hash(o).cpu()[0])          # the first lane's collision pair
    assert int(gv.gv_hash2(z).cpu()[0]) != int(gv.gv_hash2(o).cpu()[0])


def _tie_candidates(r: torch.Tensor):
    """Candidates whose relative errors tie, or nearly tie, with the running maximum in every element."""
    f = r.float()
    return [torch.zeros_like(r),                                  # |d| / |r| = 1 everywhere
            -r,                                                   # 2 everywhere
            (f * 3).to(r.dtype),                                  # 2 up to the rounding of 3r and of c - r
            (f * 1.5).to(r.dtype),                                # 0.5 up to rounding
            (f * (1 + 2.0 ** -7)).to(r.dtype),                    # a few quantised quotients
            torch.where(torch.arange(r.numel()) % 5 == 0, (f * 3).to(r.dtype), r),
            (f * (1 + 0.009 * torch.cos(torch.arange(r.numel()) * 0.37))).to(r.dtype)]   # inside rtol = 1e-2 everywhere


@pytest.mark.gpu
@pytest.mark.parametrize("code", [0, 1, 2])
def test_relative_maximum_under_ties(oracle, code):
    """The filter in front of the exact relative error lets an element through only when its quotient
    exceeds the running maximum. Here nearly every element ties with that maximum or misses it by one
    rounding, on the queueing path (small call) and the in-place path (a call large enough for the
    sampling pass, every vector differing)."""
    for n, scale in [(70001, 1.0), ((1 << 24) + 37 if code == 0 else (1 << 25) + 37, 0.05)]:
        g = torch.Generator().manual_seed(900 + code)
        r = (torch.randn(n, generator=g) * scale).to(TDT[code])
        cands = _tie_candidates(r)
        # (atol far below rtol selects the kernel whose in-place loop also settles vectors by the running
        # maximum of the relative error)
        for atol, rtol in [(1e-2, 1e-2), (0.0, 0.0), (1e-6, 1e-2)]:
            got, _ = run_dense(r.to(DEV), [c.to(DEV) for c in cands], atol, rtol, False)
            want = oracle.verify_batch(host_bytes(r), [host_bytes(c) for c in cands], code, atol, rtol, False)
            assert_records_equal(got, want, f"ties dtype {code} n {n} tol {atol}")


@pytest.mark.gpu
@pytest.mark.parametrize("code", [0, 1])
def test_relative_maximum_with_tiny_references(oracle, code):
    """Reference magnitudes from 2^-20 down to the subnormals (the relative-error filter trusts its
    multiply-add only above 2^-50 and must hand smaller elements to the exact path), mixed with ordinary
    values so that a running maximum exists, candidates tying with it."""
    rng = np.random.default_rng(77 + code)
    n = 40003
    expo = rng.integers(-149 if code == 0 else -133, -20, n)
    mant = 1.0 + rng.integers(0, 1 << 7, n) / 128.0
    vals = np.ldexp(mant, expo) * rng.choice([-1.0, 1.0], n)
    ordinary = rng.random(n) < 0.3
    vals[ordinary] = rng.standard_normal(int(ordinary.sum()))
    vals[rng.integers(0, n, 50)] = 0.0
    r = torch.from_numpy(vals.astype(np.float32)).to(TDT[code])
    cands = _tie_candidates(r)
    for atol, rtol in [(0.0, 0.0), (1e-30, 1e-3), (1e-2, 1e-2)]:
        got, _ = run_dense(r.to(DEV), [c.to(DEV) for c in cands], atol, rtol, False)
        want = oracle.verify_batch(host_bytes(r), [host_bytes(c) for c in cands], code, atol, rtol, False)
        assert_records_equal(got, want, f"tiny references dtype {code} tol {atol}")
    # the ragged kernel runs the same filter from its own loops: the same data as one ragged tensor
    nb = n * ESZ[code]
    stride = (nb + 15) // 16 * 16
    N = len(cands)
    cand_buf = torch.zeros(stride * N, dtype=torch.uint8)
    for j, c in enumerate(cands):
        cand_buf[j * stride:j * stride + nb] = c.view(torch.uint8)
    ref_buf = r.view(torch.uint8).clone()
    ref_off, cand_off = torch.tensor([0, nb]), torch.tensor([j * stride for j in range(N)])
    dtypes_t, n_el = torch.tensor([code], dtype=torch.uint8), torch.tensor([n])
    for atol, rtol in [(0.0, 0.0), (1e-2, 1e-2)]:
        ws = torch.empty(gv.gv_workspace_bytes(1, N), dtype=torch.uint8, device=DEV)
        res = gv.gv_verify_ragged(ref_buf.to(DEV), ref_off.to(DEV), cand_buf.to(DEV), cand_off.to(DEV), dtypes_t.to(DEV),
                                  N, atol, rtol, False, n_elems=n_el.to(DEV), workspace=ws)
        torch.cuda.synchronize()
        assert gv.gv_check(ws) == gv.GV_OK
        want = oracle.verify_ragged(ref_buf.numpy(), ref_off.numpy(), cand_buf.numpy(), cand_off.numpy(), dtypes_t.numpy(),
                                    N, atol, rtol, False, n_elems=n_el.numpy())
        assert_records_equal(gv.results_to_numpy(res), want, f"ragged tiny references dtype {code} tol {atol}")


@pytest.mark.gpu
@pytest.mark.parametrize("code", [0, 1, 2])
def test_relative_tolerance_regime(oracle, code):
    """Tolerances that are relative in effect (atol far below rtol |r|): the fast path may then declare a
    vector close because no quotient |d| / |r| exceeds a running maximum that is itself below rtol. Noise
    inside, across and exactly at the edge of rtol, the margin around rtol (1 - 2^-22) bracketed, a single
    far-off element that switches the shortcut off, zeros and tiny elements in the reference."""
    g = torch.Generator().manual_seed(4100 + code)
    # large enough that every warp sees many tiles of each candidate (the shortcut works on a per-CTA running
    # maximum), small enough that the whole call stays on the queueing path (below the sampling pass)
    n = 6000004 // ESZ[code] + 1
    r = torch.randn(n, generator=g)
    r[torch.randint(0, n, (40,), generator=g)] = 0.0
    r[torch.randint(0, n, (40,), generator=g)] = 2.0 ** -60 if code != 2 else 2.0 ** -20
    r = r.to(TDT[code])
    rf = r.double()
    u = torch.rand(n, generator=g, dtype=torch.float64) * 2 - 1
    sign = torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0).double()
    for rtol in [2.0 ** -7, 1e-2, 1.6e-2]:
        cands = [(rf * (1 + u * rtol * 0.9)).to(TDT[code]),
                 (rf * (1 + u * rtol * 1.1)).to(TDT[code]),
                 (rf * (1 + sign * rtol)).to(TDT[code]),
                 (rf * (1 + sign * rtol * (1 - 2.0 ** -22))).to(TDT[code]),
                 (rf * (1 + sign * rtol * (1 - 2.0 ** -21))).to(TDT[code]),
                 (rf * (1 + sign * rtol * (1 - 2.0 ** -23))).to(TDT[code])]
        far = (rf * (1 + u * rtol * 0.5)).to(TDT[code])
        far[n // 2] = far[n // 2] * 3 + 1
        cands.append(far)
        nz = r.clone()
        nz[r == 0] = 2.0 ** -24
        cands.append(nz)
        withnan = cands[0].clone()
        withnan[torch.randint(0, n, (9,), generator=g)] = float("nan")
        withnan[torch.randint(0, n, (9,), generator=g)] = float("inf")
        cands.append(withnan)
        for atol in [0.0, 1e-8, 1e-5]:
            got, _ = run_dense(r.to(DEV), [c.to(DEV) for c in cands], atol, rtol, False)
            want = oracle.verify_batch(host_bytes(r), [host_bytes(c) for c in cands], code, atol, rtol, False)
            assert_records_equal(got, want, f"relative regime dtype {code} rtol {rtol} atol {atol}")
        # the same through the ragged kernel: one tensor, all candidates
        nb = n * ESZ[code]
        stride = (nb + 15) // 16 * 16
        N = len(cands)
        cand_buf = torch.zeros(stride * N, dtype=torch.uint8)
        for j, c in enumerate(cands):
            cand_buf[j * stride:j * stride + nb] = c.view(torch.uint8)
        ref_buf = r.view(torch.uint8).clone()
        ref_off, cand_off = torch.tensor([0, nb]), torch.tensor([j * stride for j in range(N)])
        dtypes_t, n_el = torch.tensor([code], dtype=torch.uint8), torch.tensor([n])
        ws = torch.empty(gv.gv_workspace_bytes(1, N), dtype=torch.uint8, device=DEV)
        res = gv.gv_verify_ragged(ref_buf.to(DEV), ref_off.to(DEV), cand_buf.to(DEV), cand_off.to(DEV), dtypes_t.to(DEV),
                                  N, 1e-8, rtol, True, n_elems=n_el.to(DEV), workspace=ws)
        torch.cuda.synchronize()
        assert gv.gv_check(ws) == gv.GV_OK
        want = oracle.verify_ragged(ref_buf.numpy(), ref_off.numpy(), cand_buf.numpy(), cand_off.numpy(), dtypes_t.numpy(),
                                    N, 1e-8, rtol, True, n_elems=n_el.numpy())
        assert_records_equal(gv.results_to_numpy(res), want, f"ragged relative regime dtype {code} rtol {rtol}")


@pytest.mark.gpu
def test_relative_tolerance_edge_band(oracle):
    """fp32 elements whose quotient |d| / |r| is rtol exactly (close: |d| = tol) or one step of 2^-23 above
    it (not close), with atol = 0: the running maximum first settles at rtol through the ties, and the
    elements one step above must still be counted -- a shortcut that trusted a maximum slightly above rtol
    would call them close."""
    rng = np.random.default_rng(5)
    n = (1 << 22) + 3                                 # ~27 tiles per warp, so the per-CTA maximum settles
    rtol = 0.25
    sign = rng.choice([-1.0, 1.0], n)
    r = (sign * 2.0 ** 20).astype(np.float32)
    step = rng.choice([0, 0, 0, 1, 2], n).astype(np.float64)
    c = (sign * (2.0 ** 20 * 1.25 + step * 2.0 ** -3)).astype(np.float32)
    assert np.all(np.abs(c.astype(np.float64) - r) == 2.0 ** 18 + step * 2.0 ** -3)
    rt, ct = torch.from_numpy(r), torch.from_numpy(c)
    got, _ = run_dense(rt.to(DEV), [ct.to(DEV), ct.to(DEV).flip(0).flip(0)], 0.0, rtol, False)
    want = oracle.verify_batch(host_bytes(rt), [host_bytes(ct)] * 2, oracle.F32, 0.0, rtol, False)
    assert int(want[0]["n_mismatch"]) == int((step > 0).sum())          # by construction
    assert_records_equal(got, want, "edge band")


@pytest.mark.gpu
@pytest.mark.parametrize("code", [0, 1, 2, 3, 4])
def test_single_candidate_tile_pairs(oracle, code):
    """One candidate per call at sizes where the warps of the grid get two to five 512-byte tiles each, an
    odd or an even number and not the same for every warp: the loop for a single candidate takes its
    tiles two at a time and finishes with a single one."""
    g = torch.Generator().manual_seed(600 + code)
    warps = 148 * 2 * 8
    # (the last size is past 64 MB, where the sampling pass runs: the candidate that differs everywhere is then
    # flagged and takes the in-place form of the loop)
    for tiles in [2 * warps, 2 * warps + 1, 3 * warps + 777, 4 * warps - 1, 5 * warps + 5, (64 << 20) // 512 + warps + 1]:
        n = tiles * 512 // ESZ[code] + 3
        if code >= 3:
            r = torch.randint(-(1 << 20), 1 << 20, (n,), generator=g, dtype=TDT[code])
            c = torch.where(torch.rand(n, generator=g) < 1e-3, r + 7, r)
            d = torch.where(torch.rand(n, generator=g) < 0.7, r - 1, r)
        else:
            r = torch.randn(n, generator=g).to(TDT[code])
            r[torch.randint(0, n, (5,), generator=g)] = float("nan")
            c = torch.where(torch.rand(n, generator=g) < 1e-3, (r.float() + 1).to(TDT[code]), r)
            d = (r.float() * (1 + 3e-3 * torch.randn(n, generator=g))).to(TDT[code])
        for cand in (r.clone(), c, d):
            if tiles > 6 * warps and cand is c:
                continue
            got, rh = run_dense(r.to(DEV), [cand.to(DEV)], 1e-2, 1e-2, code == 1)
            want = oracle.verify_batch(host_bytes(r), [host_bytes(cand)], code, 1e-2, 1e-2, code == 1)
            assert_records_equal(got, want, f"single candidate dtype {code} tiles {tiles}")
            assert rh == oracle.hash_bytes(host_bytes(r))


@pytest.mark.gpu
def test_ragged_single_candidate_streams(oracle):
    """One candidate per tensor, tensors of hundreds to thousands of tiles of every dtype: the ragged kernel's
    loop for any candidate count takes a single candidate's tiles two at a time (and an odd one last)."""
    g = torch.Generator().manual_seed(888)
    sizes = [(1 << 20) + 77, (1 << 19) + 5, 999999, 3 * (1 << 18), 40000, (1 << 20) - 3, 128 * 7 + 1]
    codes = [0, 1, 2, 3, 4, 1, 0]
    T = len(sizes)
    refs, cands = [], []
    for t in range(T):
        code, n = codes[t], sizes[t]
        if code >= 3:
            r = torch.randint(-(1 << 20), 1 << 20, (n,), generator=g, dtype=TDT[code])
            c = torch.where(torch.rand(n, generator=g) < 0.01, r + 3, r)
        else:
            r = torch.randn(n, generator=g).to(TDT[code])
            r[torch.randint(0, n, (7,), generator=g)] = float("nan")
            c = torch.where(torch.rand(n, generator=g) < (0.01 if t % 2 else 1.0),
                            (r.float() * (1 + 2e-3 * torch.randn(n, generator=g))).to(TDT[code]), r)
        refs.append(r)
        cands.append(c)
    ref_off, cand_off, rc = [], [], 0
    for t in range(T):
        rc = (rc + 15) // 16 * 16
        ref_off.append(rc)
        cand_off.append(rc)
        rc += sizes[t] * ESZ[codes[t]]
    ref_off.append(rc)
    ref_buf = torch.zeros(rc, dtype=torch.uint8)
    cand_buf = torch.zeros(rc, dtype=torch.uint8)
    for t in range(T):
        nb = sizes[t] * ESZ[codes[t]]
        ref_buf[ref_off[t]:ref_off[t] + nb] = refs[t].view(torch.uint8)
        cand_buf[cand_off[t]:cand_off[t] + nb] = cands[t].view(torch.uint8)
    ro, co = torch.tensor(ref_off), torch.tensor(cand_off)
    dt, ne = torch.tensor(codes, dtype=torch.uint8), torch.tensor(sizes)
    for en in (False, True):
        ws = torch.empty(gv.gv_workspace_bytes(T, 1), dtype=torch.uint8, device=DEV)
        res = gv.gv_verify_ragged(ref_buf.to(DEV), ro.to(DEV), cand_buf.to(DEV), co.to(DEV), dt.to(DEV), 1, 1e-2, 1e-2, en,
                                  n_elems=ne.to(DEV), workspace=ws)
        torch.cuda.synchronize()
        assert gv.gv_check(ws) == gv.GV_OK
        want = oracle.verify_ragged(ref_buf.numpy(), ro.numpy(), cand_buf.numpy(), co.numpy(), dt.numpy(), 1, 1e-2, 1e-2, en,
                                    n_elems=ne.numpy())
        assert_records_equal(gv.results_to_numpy(res), want, f"ragged single candidate equal_nan {en}")
