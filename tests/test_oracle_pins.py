"""Pins for the CPU oracle: every check here compares the oracle with something fixed outside it
(published SplitMix64 outputs, a hand-derived truth table, exact integer / rational arithmetic in
Python, torch.isclose and numpy on the host, by-construction counts of the workload recipes).
None of these tests touches the CUDA library."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
M64 = (1 << 64) - 1
GAMMA = 0x9E3779B97F4A7C15


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line


def f32(bits):
    return np.array([bits], dtype=np.uint32).view(np.float32)


# --------------------------------------------------------------------------------------------
# hash
# --------------------------------------------------------------------------------------------
def test_splitmix64_published_vector(oracle):
    # output i of the generator seeded with 0 is mix(i * gamma)
    for row in _rows("splitmix64_published.txt"):
        i, hx = row.split()
        assert oracle.splitmix64((int(i) * GAMMA) & M64) == int(hx, 16)


def test_hash_is_sum_of_published_outputs(oracle):
    # words W_k = (k * gamma) xor k make k xor W_k = k * gamma, so the hash of these 24 bytes is the
    # wrapping sum of the three published outputs. A big-endian read, a missing index xor, or a
    # xor with the byte (not word) index would all fail here.
    words = [((k * GAMMA) & M64) ^ k for k in range(3)]
    buf = b"".join(w.to_bytes(8, "little") for w in words)
    want = sum(int(r.split()[1], 16) for r in _rows("splitmix64_published.txt")) & M64
    assert oracle.hash_bytes(buf) == want
    # and each prefix: 8 bytes -> first output alone; 16 bytes -> first two
    outs = [int(r.split()[1], 16) for r in _rows("splitmix64_published.txt")]
    assert oracle.hash_bytes(buf[:8]) == outs[0]
    assert oracle.hash_bytes(buf[:16]) == (outs[0] + outs[1]) & M64


def _py_splitmix64(x):
    z = (x + GAMMA) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def _py_hash(b: bytes) -> int:
    """Brute force with Python big integers (independent of C integer semantics)."""
    b = b + b"\0" * (-len(b) % 8)
    h = 0
    for k in range(len(b) // 8):
        h = (h + _py_splitmix64(k ^ int.from_bytes(b[8 * k:8 * k + 8], "little"))) & M64
    return h


def test_hash_brute_force_all_small_lengths(oracle):
    rng = np.random.default_rng(7)
    data = rng.integers(0, 256, size=4200, dtype=np.uint8).tobytes()
    for nbytes in list(range(0, 70)) + [255, 256, 257, 4095, 4096, 4097, 4113]:
        assert oracle.hash_bytes(data[:nbytes]) == _py_hash(data[:nbytes]), nbytes


def test_hash_special_cases(oracle):
    assert oracle.hash_bytes(b"") == 0                                   # empty
    assert oracle.hash_bytes(b"\0" * 8) == 0xE220A8397B1DCDAF            # = published output 0
    # zero padding of a partial last word: 5 bytes hash like the same 5 bytes followed by 3 zeros
    assert oracle.hash_bytes(b"\1\2\3\4\5") == oracle.hash_bytes(b"\1\2\3\4\5\0\0\0")
    # ... and the length is not mixed in, but the word index is: moving a word changes the hash
    a = (1).to_bytes(8, "little") + (2).to_bytes(8, "little")
    b = (2).to_bytes(8, "little") + (1).to_bytes(8, "little")
    assert oracle.hash_bytes(a) != oracle.hash_bytes(b)
    # documented weakness of index-xor-word: int64 [0, 0] and [1, 1] collide (k xor W_k = {0,1} both)
    z = np.array([0, 0], dtype=np.int64)
    o = np.array([1, 1], dtype=np.int64)
    assert oracle.hash_bytes(z) == oracle.hash_bytes(o) == (_py_splitmix64(0) + _py_splitmix64(1)) & M64
    # raw bits, not values: +0.0 and -0.0 hash differently
    assert oracle.hash_bytes(np.array([0.0], np.float32)) != oracle.hash_bytes(np.array([-0.0], np.float32))


def test_hash_four_mib_of_zeros_closed_form(oracle):
    # all-zero buffer: hash = sum_{k < 2^19} mix(k); evaluated here with numpy uint64 wrap-around
    k = np.arange(1 << 19, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = k + np.uint64(GAMMA)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
        want = int(np.add.reduce(z))
    assert oracle.hash_bytes(np.zeros(1 << 20, dtype=np.float32)) == want


def test_hash_partition_invariance(oracle):
    # the sum may be split over any partition of the word indices (what a tiled kernel relies on):
    # hash(buf) = sum over tiles of sum_k mix((k0 + k) xor W); checked via the Python brute force
    rng = np.random.default_rng(3)
    data = rng.integers(0, 256, size=8 * 100, dtype=np.uint8).tobytes()
    total = 0
    for k in range(100):
        total = (total + _py_splitmix64(k ^ int.from_bytes(data[8 * k:8 * k + 8], "little"))) & M64
    assert oracle.hash_bytes(data) == total


# --------------------------------------------------------------------------------------------
# widening
# --------------------------------------------------------------------------------------------
def test_widening_matches_numpy_and_torch_for_all_16bit_patterns(oracle):
    raw = np.arange(1 << 16, dtype=np.uint16)
    want_h = raw.view(np.float16).astype(np.float32).view(np.uint32)
    want_b = torch.from_numpy(raw.view(np.int16)).view(torch.bfloat16).float().numpy().view(np.uint32)
    for x in range(1 << 16):
        got_h = oracle.widen_bits(oracle.F16, x)
        got_b = oracle.widen_bits(oracle.BF16, x)
        if np.isnan(np.array([want_h[x]], np.uint32).view(np.float32))[0]:
            # NaN: class and sign must agree (payload conventions differ between libraries)
            assert (got_h & 0x7F800000) == 0x7F800000 and (got_h & 0x007FFFFF) != 0
        else:
            assert got_h == int(want_h[x]), hex(x)
        assert got_b == int(want_b[x]), hex(x)


# --------------------------------------------------------------------------------------------
# per-element rule
# --------------------------------------------------------------------------------------------
def test_truth_table(oracle):
    n_rows = 0
    for row in _rows("isclose_truth_table.txt"):
        lhs, rhs = row.split("|")
        cb, rb, atol, rtol, en = lhs.split()
        mm, nn, ni, ab, rl = rhs.split()
        c, r = f32(int(cb, 16)), f32(int(rb, 16))
        res = oracle.verify(r, c, oracle.F32, float(atol), float(rtol), bool(int(en)))
        assert int(res["n_mismatch"]) == int(mm), row
        assert int(res["first_mismatch"]) == (0 if int(mm) else oracle.NO_INDEX), row
        assert int(res["n_nan_disagree"]) == int(nn), row
        assert int(res["n_inf_disagree"]) == int(ni), row
        if ab != "*":
            assert int(res["max_abs_err"].view(np.uint32)) == int(ab, 16), row
        if rl != "*":
            assert int(res["max_rel_err"].view(np.uint32)) == int(rl, 16), row
        assert int(res["max_abs_diff_int"]) == 0 and int(res["reserved"]) == 0
        n_rows += 1
    assert n_rows >= 20
    # constants used in the table
    assert int(np.float32(3e38).view(np.uint32)) == 0x7F61B1E6
    assert int(np.float32(1e-5).view(np.uint32)) == 0x3727C5AC
    assert int(np.float32(1e-2).view(np.uint32)) == 0x3C23D70A


def _exact_tol_bits(atol, rtol, r_bits):
    """fl(atol_f + fl(rtol_f * |r|)) by exact rational arithmetic, rounding with numpy's
    float64->float32 conversion (products/sums of binary32 are exact in Fractions)."""
    def rne32(q: Fraction) -> np.float32:
        # correctly rounded binary32 of a rational: float(q) is correctly rounded to binary64, and
        # for the magnitudes used here (one product / one sum of binary32 values) a second rounding
        # to binary32 is innocuous (53 >= 2*24 + 2)
        return np.float32(float(q))
    a = Fraction(float(np.float32(atol)))
    t = Fraction(float(np.float32(rtol)))
    r = abs(Fraction(float(f32(r_bits)[0])))
    prod = rne32(t * r)
    return int(rne32(a + Fraction(float(prod))).view(np.uint32))


def test_two_roundings_not_fma():
    # the canary rows rest on this: the two-step tolerance is 0x37908000, the fused one is 1 ulp less
    assert _exact_tol_bits(1e-5, 1e-5, 0xBF38FA9F) == 0x37908000
    a = Fraction(float(np.float32(1e-5)))
    r = abs(Fraction(float(f32(0xBF38FA9F)[0])))
    fused = np.float32(float(a + a * r))
    assert int(fused.view(np.uint32)) == 0x37907FFF


def test_division_not_reciprocal(oracle):
    # |d| = 0x3A78DE92, |r| = 0x3F8A0F08: IEEE quotient 0x3A66BCBB; multiply by reciprocal gives ...BA.
    ad, r = f32(0x3A78DE92), f32(0x3F8A0F08)
    q = np.float32(float(Fraction(float(ad[0])) / Fraction(float(r[0]))))
    assert int(q.view(np.uint32)) == 0x3A66BCBB
    # build an element whose |d| is exactly ad: c = r + ad is not exact in general, so use r = |r|
    # and the pair (c, r) = (ad, 0)?  -> r == 0 is excluded from max_rel; instead scan for exact pairs
    rng = np.random.default_rng(11)
    rr = rng.standard_normal(20000).astype(np.float32)
    cc = (rr + rng.standard_normal(20000).astype(np.float32) * np.float32(1e-3)).astype(np.float32)
    res = oracle.verify(rr, cc, oracle.F32, 1.0, 1.0, False)
    d = np.abs((cc - rr).astype(np.float32))
    want = max(np.float32(float(Fraction(float(x)) / Fraction(float(abs(y))))) for x, y in zip(d, rr) if y != 0)
    assert res["max_rel_err"] == want
    # and a reciprocal-multiply would not reproduce it on this data (the pin has teeth)
    recip = np.max(d * (np.float32(1.0) / np.abs(rr)))
    exact_all = np.array([np.float32(float(Fraction(float(x)) / Fraction(float(abs(y))))) for x, y in zip(d, rr)])
    assert np.any(exact_all != d * (np.float32(1.0) / np.abs(rr)))
    del recip


SPECIALS32 = np.array([0x00000000, 0x80000000, 0x00000001, 0x80000001, 0x007FFFFF, 0x00800000, 0x3F800000,
                       0xBF800000, 0x7F7FFFFF, 0xFF7FFFFF, 0x7F800000, 0xFF800000, 0x7FC00000, 0xFFC00001,
                       0x3F7FFFFF, 0x3F800001, 0x40000000, 0x3DCCCCCD], dtype=np.uint32).view(np.float32)


def _host_reference_float(c32, r32, atol, rtol, equal_nan):
    """Independent host evaluation with library routines on widened fp32 data."""
    a32, t32 = float(np.float32(atol)), float(np.float32(rtol))
    ct, rt = torch.from_numpy(c32.copy()), torch.from_numpy(r32.copy())
    close = torch.isclose(ct, rt, rtol=t32, atol=a32, equal_nan=equal_nan).numpy()
    mism = ~close
    nan_dis = np.isnan(c32) != np.isnan(r32)
    cls = lambda x: np.where(np.isposinf(x), 1, np.where(np.isneginf(x), -1, 0))
    inf_dis = cls(c32) != cls(r32)
    fin = np.isfinite(c32) & np.isfinite(r32)
    with np.errstate(all="ignore"):
        d = np.abs((c32 - r32).astype(np.float32))
        max_abs = np.float32(d[fin].max()) if fin.any() else np.float32(0)
        sel = fin & (r32 != 0)
        rel = (d[sel].astype(np.float64) / np.abs(r32[sel]).astype(np.float64)).astype(np.float32)
        max_rel = np.float32(rel.max()) if sel.any() else np.float32(0)
    first = int(np.argmax(mism)) if mism.any() else 0xFFFFFFFFFFFFFFFF
    return int(mism.sum()), first, int(nan_dis.sum()), int(inf_dis.sum()), max_abs, max_rel


def _check_against_host(oracle, res, c32, r32, atol, rtol, equal_nan, tag):
    mm, first, nn, ni, ma, mr = _host_reference_float(c32, r32, atol, rtol, equal_nan)
    assert int(res["n_mismatch"]) == mm, tag
    assert int(res["first_mismatch"]) == first, tag
    assert int(res["n_nan_disagree"]) == nn, tag
    assert int(res["n_inf_disagree"]) == ni, tag
    assert res["max_abs_err"].view(np.uint32) == ma.view(np.uint32), tag
    assert res["max_rel_err"].view(np.uint32) == mr.view(np.uint32), tag


@pytest.mark.parametrize("equal_nan", [False, True])
def test_fp32_specials_cross_product_vs_torch_isclose(oracle, equal_nan):
    # torch.isclose computes |c - r| <= atol + rtol*|r| in fp32 with the same two roundings
    c = np.repeat(SPECIALS32, len(SPECIALS32))
    r = np.tile(SPECIALS32, len(SPECIALS32))
    for atol, rtol in [(0.0, 0.0), (1e-5, 1e-5), (1.0, 0.5), (1e30, 1e30)]:
        res = oracle.verify(r, c, oracle.F32, atol, rtol, equal_nan)
        _check_against_host(oracle, res, c, r, atol, rtol, equal_nan, (atol, rtol))
    # element by element as well (catches compensating errors in the aggregate)
    for i in range(len(c)):
        res = oracle.verify(r[i:i + 1], c[i:i + 1], oracle.F32, 1e-5, 1e-5, equal_nan)
        _check_against_host(oracle, res, c[i:i + 1], r[i:i + 1], 1e-5, 1e-5, equal_nan, i)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_fp32_random_vs_torch_isclose(oracle, seed):
    rng = np.random.default_rng(seed)
    n = 50000
    r = rng.standard_normal(n).astype(np.float32)
    c = r + rng.standard_normal(n).astype(np.float32) * np.float32(10.0 ** rng.integers(-7, 0))
    idx = rng.integers(0, n, 40)
    c[idx[:10]] = np.nan
    c[idx[10:20]] = np.inf
    r[idx[20:25]] = np.nan
    r[idx[25:30]] = -np.inf
    r[idx[30:35]] = 0.0
    c[idx[35:40]] = r[idx[35:40]]
    for atol, rtol in [(1e-5, 1e-5), (1e-3, 0.0), (0.0, 1e-2)]:
        for en in (False, True):
            res = oracle.verify(r, c, oracle.F32, atol, rtol, en)
            _check_against_host(oracle, res, c, r, atol, rtol, en, (seed, atol, rtol, en))


@pytest.mark.parametrize("code,tdt", [(1, torch.bfloat16), (2, torch.float16)])
def test_all_16bit_candidates_against_interesting_references(oracle, code, tdt):
    # every 16-bit pattern as candidate against a set of interesting reference values:
    # 65536 x 24 pairs per dtype, checked against torch.isclose on the widened values
    raw_c = np.arange(1 << 16, dtype=np.uint16)
    c32 = torch.from_numpy(raw_c.view(np.int16)).view(tdt).float().numpy()
    if code == 1:
        refs = [0x0000, 0x8000, 0x0001, 0x0080, 0x3F80, 0xBF80, 0x7F7F, 0xFF7F, 0x7F80, 0xFF80, 0x7FC0, 0x3F7F,
                0x4000, 0x3DCD, 0x0100, 0x4049]
    else:
        refs = [0x0000, 0x8000, 0x0001, 0x03FF, 0x0400, 0x3C00, 0xBC00, 0x7BFF, 0xFBFF, 0x7C00, 0xFC00, 0x7E00,
                0x3BFF, 0x4000, 0x2E66, 0x4248]
    for rb in refs:
        raw_r = np.full(1 << 16, rb, dtype=np.uint16)
        r32 = torch.from_numpy(raw_r.view(np.int16)).view(tdt).float().numpy()
        for atol, rtol, en in [(1e-2, 1e-2, False), (0.0, 0.0, True)]:
            res = oracle.verify(raw_r, raw_c, code, atol, rtol, en)
            _check_against_host(oracle, res, c32, r32, atol, rtol, en, (hex(rb), atol))
            assert int(res["hash"]) == oracle.hash_bytes(raw_c)


# --------------------------------------------------------------------------------------------
# integers
# --------------------------------------------------------------------------------------------
def test_integer_exact_mode(oracle):
    lo, hi = -(1 << 63), (1 << 63) - 1
    r = np.array([0, 5, lo, hi, -1, 7], dtype=np.int64)
    c = np.array([0, 9, hi, lo, -1, 6], dtype=np.int64)
    res = oracle.verify(r, c, oracle.I64, 123.0, 456.0, True)     # tolerances are ignored
    assert int(res["n_mismatch"]) == 4 and int(res["first_mismatch"]) == 1
    assert int(res["max_abs_diff_int"]) == (1 << 64) - 1            # hi - lo, exact in u64
    assert res["max_abs_err"] == 0 and res["max_rel_err"] == 0
    assert int(res["n_nan_disagree"]) == 0 and int(res["n_inf_disagree"]) == 0
    r32 = np.array([-(1 << 31), (1 << 31) - 1, 3], dtype=np.int32)
    c32 = np.array([(1 << 31) - 1, (1 << 31) - 1, 1], dtype=np.int32)
    res = oracle.verify(r32, c32, oracle.I32)
    assert int(res["n_mismatch"]) == 2 and int(res["first_mismatch"]) == 0
    assert int(res["max_abs_diff_int"]) == (1 << 32) - 1
    rng = np.random.default_rng(5)
    a = rng.integers(-1000, 1000, 5000).astype(np.int32)
    b = a.copy()
    pos = rng.choice(5000, 37, replace=False)
    b[pos] += rng.integers(1, 50, 37).astype(np.int32)
    res = oracle.verify(a, b, oracle.I32)
    assert int(res["n_mismatch"]) == 37 and int(res["first_mismatch"]) == int(pos.min())
    assert int(res["max_abs_diff_int"]) == int(np.abs(b.astype(np.int64) - a).max())
    assert int(res["hash"]) == _py_hash(b.tobytes())


# --------------------------------------------------------------------------------------------
# invariants and by-construction counts on the workload recipes (reduced sizes)
# --------------------------------------------------------------------------------------------
def _np(t: torch.Tensor) -> np.ndarray:
    if t.dtype in (torch.bfloat16, torch.float16):
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def _check_facts(oracle, wl, res):
    ref_hash = oracle.hash_bytes(_np(wl.ref))
    zero = np.zeros((), dtype=oracle.RESULT_DTYPE)
    zero["first_mismatch"] = oracle.NO_INDEX
    for j, (f, r) in enumerate(zip(wl.facts, res)):
        if "n_mismatch" in f:
            assert int(r["n_mismatch"]) == f["n_mismatch"], (j, f["class"])
            want_first = oracle.NO_INDEX if f["first"] is None else f["first"]
            assert int(r["first_mismatch"]) == want_first, (j, f["class"])
        if "n_nan" in f:
            assert int(r["n_nan_disagree"]) == f["n_nan"], (j, f["class"])
            assert int(r["n_inf_disagree"]) == f["n_inf"], (j, f["class"])
        if f.get("hash_equals_ref"):
            z = zero.copy()
            z["hash"] = ref_hash
            assert r.tobytes() == z.tobytes(), (j, f["class"])       # identical copy: all-zero stats
        if "same_as" in f:
            assert r.tobytes() == res[f["same_as"]].tobytes()


def test_config1_by_construction(oracle):
    from paper_2507_23194_b200 import workloads as W
    wl = W.config1("cpu")
    r = wl.ref.numpy()
    res = oracle.verify_batch(r, [_np(c) for c in wl.cands], oracle.F32, wl.atol, wl.rtol, wl.equal_nan)
    _check_facts(oracle, wl, res)
    ref_hash = oracle.hash_bytes(r)
    # 1: noise inside tolerance: bounded relative error, different bytes
    assert 0 < res[1]["max_rel_err"] < 1.1e-6 and int(res[1]["hash"]) != ref_hash
    # 2: r + 1 at 1000 places: max_abs is the numpy float32 expression over the injected positions
    p = wl.facts[2]["positions"].numpy()
    want = np.max(np.abs(((r[p] + np.float32(1.0)).astype(np.float32) - r[p]).astype(np.float32)))
    assert res[2]["max_abs_err"] == want and abs(float(want) - 1.0) < 1e-6
    # 3: NaN/Inf elements do not enter the maxima
    assert res[3]["max_abs_err"] == 0 and res[3]["max_rel_err"] == 0
    # 5: negated: |d| = 2|r| exactly, so max_rel is exactly 2 and max_abs exactly 2 max|r|
    a32, t32 = np.float32(wl.atol), np.float32(wl.rtol)
    tol = (a32 + (t32 * np.abs(r)).astype(np.float32)).astype(np.float32)
    assert res[5]["max_rel_err"] == np.float32(2.0)
    assert res[5]["max_abs_err"] == np.float32(2.0) * np.abs(r).max()
    assert int(res[5]["n_mismatch"]) == int(np.sum(~((2 * np.abs(r) <= tol) | (r == 0))))
    # 6: zeros: |d| = |r|, max_rel exactly 1, hash of 4 MiB of zero bytes
    assert res[6]["max_rel_err"] == np.float32(1.0) and res[6]["max_abs_err"] == np.abs(r).max()
    assert int(res[6]["n_mismatch"]) == int(np.sum(~(np.abs(r) <= tol)))
    assert int(res[6]["hash"]) == 0x8C6F9C0F16C4607B
    # 7: one ulp: hash differs from the reference's in exactly one term
    p7 = wl.facts[7]["position"]
    k = p7 // 2
    w_old = int.from_bytes(r[2 * k:2 * k + 2].tobytes(), "little")
    w_new = int.from_bytes(wl.cands[7].numpy()[2 * k:2 * k + 2].tobytes(), "little")
    assert int(res[7]["hash"]) == (ref_hash - _py_splitmix64(k ^ w_old) + _py_splitmix64(k ^ w_new)) & M64
    ulp = np.abs(wl.cands[7].numpy()[p7] - r[p7])
    assert res[7]["max_abs_err"] == ulp
    assert res[7]["max_rel_err"] == np.float32(np.float64(ulp) / np.float64(abs(r[p7])))
    # permuting the candidate list permutes the results
    perm = [3, 0, 7, 5, 1, 6, 2, 4]
    res_p = oracle.verify_batch(r, [_np(wl.cands[i]) for i in perm], oracle.F32, wl.atol, wl.rtol, wl.equal_nan)
    for out_pos, src in enumerate(perm):
        assert res_p[out_pos].tobytes() == res[src].tobytes()


def test_config2_3_4_reduced_by_construction(oracle):
    from paper_2507_23194_b200 import workloads as W
    wl = W.config2("cpu", n=1 << 16, n_cands=40)
    assert sorted(set(f["class"] for f in wl.facts)) == ["copy", "errors", "nan_inf", "noise"]
    res = oracle.verify_batch(_np(wl.ref), [_np(c) for c in wl.cands], oracle.BF16, wl.atol, wl.rtol, wl.equal_nan)
    _check_facts(oracle, wl, res)
    # secondary cross-check of a noisy and an error candidate against torch.isclose on widened data
    for j, f in enumerate(wl.facts):
        if f["class"] in ("noise", "errors", "nan_inf"):
            _check_against_host(oracle, res[j], wl.cands[j].float().numpy(), wl.ref.float().numpy(),
                                wl.atol, wl.rtol, wl.equal_nan, (j, f["class"]))
    wl = W.config3("cpu", n=1 << 16, n_cands=10)
    res = oracle.verify_batch(_np(wl.ref), [_np(c) for c in wl.cands], oracle.F16, wl.atol, wl.rtol, wl.equal_nan)
    _check_facts(oracle, wl, res)
    for j in range(10):
        _check_against_host(oracle, res[j], wl.cands[j].float().numpy(), wl.ref.float().numpy(),
                            wl.atol, wl.rtol, wl.equal_nan, j)
    for wide in (False, True):
        wl = W.config4("cpu", n=1 << 16, n_cands=8, wide=wide)
        res = oracle.verify_batch(_np(wl.ref), [_np(c) for c in wl.cands], wl.dtype)
        _check_facts(oracle, wl, res)
        for j, f in enumerate(wl.facts):
            assert int(res[j]["max_abs_diff_int"]) == int((wl.cands[j].long() - wl.ref.long()).abs().max())


@pytest.mark.parametrize("align", [16, 0])
def test_config5_reduced_by_construction(oracle, align):
    from paper_2507_23194_b200 import workloads as W
    wl = W.config5("cpu", T=120, max_log2=12.0, align=align)
    res = oracle.verify_ragged(wl.ref_buf.numpy(), wl.ref_off.numpy(), wl.cand_buf.numpy(), wl.cand_off.numpy(),
                               wl.dtypes.numpy(), wl.N, wl.atol, wl.rtol, wl.equal_nan, n_elems=wl.n_elems_t.numpy())
    assert len(res) == wl.T * wl.N
    esz = {0: 4, 1: 2, 2: 2, 3: 4}
    for t in range(wl.T):
        code = int(wl.dtypes[t])
        nb = wl.n_elems[t] * esz[code]
        o = int(wl.ref_off[t])
        ref_hash = oracle.hash_bytes(wl.ref_buf.numpy()[o:o + nb])
        for j in range(wl.N):
            f, r = wl.facts[t * wl.N + j], res[t * wl.N + j]
            assert int(r["n_mismatch"]) == f["n_mismatch"], (t, j, f["class"])
            assert int(r["first_mismatch"]) == (oracle.NO_INDEX if f["first"] is None else f["first"])
            if f.get("hash_equals_ref"):
                assert int(r["hash"]) == ref_hash
    # Counts read off consecutive offsets (no n_elems table): repack the same tensors back to back, the
    # 4-byte types first and the 2-byte types after them, so that no tensor needs padding before it and the
    # layout is tight whatever the recipe drew. Records are per tensor, so they must equal the ones above.
    order = sorted(range(wl.T), key=lambda t: -esz[int(wl.dtypes[t])])
    rb, cb, ro, co = bytearray(), bytearray(), [], []
    ref_np, cand_np = wl.ref_buf.numpy(), wl.cand_buf.numpy()
    for t in order:
        nb = wl.n_elems[t] * esz[int(wl.dtypes[t])]
        ro.append(len(rb))
        rb += ref_np[int(wl.ref_off[t]):int(wl.ref_off[t]) + nb].tobytes()
        for j in range(wl.N):
            o = int(wl.cand_off[t * wl.N + j])
            co.append(len(cb))
            cb += cand_np[o:o + nb].tobytes()
    ro.append(len(rb))
    dts = np.array([int(wl.dtypes[t]) for t in order], dtype=np.uint8)
    tight = all(ro[i + 1] - ro[i] == wl.n_elems[t] * esz[int(wl.dtypes[t])] for i, t in enumerate(order))
    assert tight
    res2 = oracle.verify_ragged(np.frombuffer(bytes(rb), dtype=np.uint8), np.array(ro, dtype=np.int64),
                                np.frombuffer(bytes(cb), dtype=np.uint8), np.array(co, dtype=np.int64), dts, wl.N,
                                wl.atol, wl.rtol, wl.equal_nan)
    want = np.concatenate([res[t * wl.N:(t + 1) * wl.N] for t in order])
    assert res2.tobytes() == want.tobytes()


# --------------------------------------------------------------------------------------------
# grouping of duplicate candidates
# --------------------------------------------------------------------------------------------
def _records(rows):
    """rows: tuples (n_mismatch, first, n_nan, n_inf, hash, maxint, maxabs, maxrel)."""
    from oracle import gv_oracle as O
    rec = np.zeros(len(rows), dtype=O.RESULT_DTYPE)
    for j, r in enumerate(rows):
        (rec[j]["n_mismatch"], rec[j]["first_mismatch"], rec[j]["n_nan_disagree"], rec[j]["n_inf_disagree"],
         rec[j]["hash"], rec[j]["max_abs_diff_int"], rec[j]["max_abs_err"], rec[j]["max_rel_err"]) = r
    return rec


def test_group_hand_worked_example(oracle):
    # seven candidates: A B A C B A D  ->  groups {0,2,5} {1,4} {3} {6}
    A = (0, M64, 0, 0, 0x1111, 0, 0.0, 0.0)
    B = (3, 17, 0, 0, 0x2222, 0, 0.5, 0.25)
    C = (3, 17, 0, 0, 0x2222, 0, 0.5, 0.125)        # same hash and counts as B, one statistic differs
    D = (0, M64, 0, 0, 0x1112, 0, 0.0, 0.0)         # differs from A in one bit of the hash
    gid, cnt, ng = oracle.group(_records([A, B, A, C, B, A, D]))
    assert gid.tolist() == [0, 1, 0, 3, 1, 0, 6]
    assert cnt.tolist() == [3, 2, 0, 1, 0, 0, 1]
    assert ng == 4


def test_group_degenerate_cases(oracle):
    gid, cnt, ng = oracle.group(_records([]))
    assert gid.size == 0 and cnt.size == 0 and ng == 0
    one = (1, 2, 3, 4, 5, 6, 7.0, 8.0)
    gid, cnt, ng = oracle.group(_records([one] * 9))
    assert gid.tolist() == [0] * 9 and cnt.tolist() == [9] + [0] * 8 and ng == 1
    distinct = [(0, M64, 0, 0, h, 0, 0.0, 0.0) for h in range(12)]
    gid, cnt, ng = oracle.group(_records(distinct))
    assert gid.tolist() == list(range(12)) and cnt.tolist() == [1] * 12 and ng == 12
    # -0.0 and +0.0 in a float field are different bytes, hence different records
    gid, _, ng = oracle.group(_records([(0, M64, 0, 0, 9, 0, 0.0, 0.0), (0, M64, 0, 0, 9, 0, -0.0, 0.0)]))
    assert gid.tolist() == [0, 1] and ng == 2


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_group_against_python_dict(oracle, seed):
    # independent restatement: first index of each distinct byte string, via a dict
    rng = np.random.default_rng(seed)
    from oracle import gv_oracle as O
    pool = rng.integers(0, 256, size=(40, 64), dtype=np.uint8)
    pick = rng.integers(0, 40, size=500)
    rec = pool[pick].copy().view(O.RESULT_DTYPE).reshape(-1)
    gid, cnt, ng = oracle.group(rec)
    first = {}
    want = []
    for j in range(500):
        want.append(first.setdefault(rec[j].tobytes(), j))
    assert gid.tolist() == want
    assert ng == len(first)
    for j in range(500):
        assert cnt[j] == (want.count(j) if want[j] == j else 0)
    # relabelling invariance: reversing the order maps each group onto the same member set
    gid_r, _, ng_r = oracle.group(rec[::-1].copy())
    assert ng_r == ng
    groups = {frozenset(np.nonzero(gid == g)[0].tolist()) for g in set(gid.tolist())}
    groups_r = {frozenset((499 - np.nonzero(gid_r == g)[0]).tolist()) for g in set(gid_r.tolist())}
    assert groups == groups_r


# --------------------------------------------------------------------------------------------
# error profile of one candidate (ulp histogram, worst element, first mismatches, per-row counts)
# --------------------------------------------------------------------------------------------
def test_profile_hand_worked_example(oracle):
    # element:        0     1      2      3      4           5
    r = np.array([1.0, 2.0, -0.0, np.nan, 3.0, -1.0], dtype=np.float32)
    c = np.array([1.0, 2.5, 0.0, 1.0, 3.0000002, 1.0], dtype=np.float32)
    # distances: 0; 0x40200000-0x40000000 = 2^21 -> bucket 22; -0/+0 coincide -> 0; NaN -> bucket 65;
    # next float after 3.0 -> 1 -> bucket 1; -1.0 to +1.0 = 2 * 0x3F800000 = 2^31 - 2^24 -> bucket 31
    p, rows = oracle.profile(r, c, oracle.F32, 1e-3, 1e-3, False, row_len=4)
    want = np.zeros(66, dtype=np.uint64)
    want[0], want[22], want[65], want[1], want[31] = 2, 1, 1, 1, 1
    assert p["ulp_hist"].tolist() == want.tolist()
    assert int(p["n_mismatch"]) == 3                       # 2.5 vs 2, 1 vs NaN, 1 vs -1
    assert int(p["worst_index"]) == 3                      # the NaN pair ranks above every finite error
    assert int(p["worst_c_raw"]) == 0x3F800000 and int(p["worst_r_raw"]) == 0x7FC00000
    assert int(p["n_first"]) == 3 and p["first_index"].tolist()[:3] == [1, 3, 5]
    assert p["first_index"].tolist()[3:] == [oracle.NO_INDEX] * 5
    assert p["first_c_raw"].tolist()[:3] == [0x40200000, 0x3F800000, 0x3F800000]
    assert p["first_r_raw"].tolist()[:3] == [0x40000000, 0x7FC00000, 0xBF800000]
    assert rows.tolist() == [2, 1]
    # with equal_nan nothing changes here (only one side is NaN); without the NaN pair the worst is 1 vs -1
    p2, _ = oracle.profile(r[[0, 1, 2, 4, 5]], c[[0, 1, 2, 4, 5]], oracle.F32, 1e-3, 1e-3, True)
    assert int(p2["worst_index"]) == 4 and int(p2["n_mismatch"]) == 2


def test_profile_ulp_distance_counts_representable_steps(oracle):
    # k steps of nextafter away from x are at distance k, in every dtype's own spacing
    x = np.float32(0.7)
    for k in (1, 2, 3, 4, 7, 8, 1000, 1 << 20):
        y = x
        if k <= 1000:
            for _ in range(k):
                y = np.nextafter(y, np.float32(np.inf))
        else:
            y = (np.array([x]).view(np.uint32) + np.uint32(k)).view(np.float32)[0]
        p, _ = oracle.profile(np.array([x]), np.array([y]), oracle.F32)
        assert int(p["ulp_hist"][1 + int(np.floor(np.log2(k)))]) == 1
    # across zero: smallest negative to smallest positive subnormal is two steps
    p, _ = oracle.profile(np.array([0x80000001], dtype=np.uint32), np.array([0x00000001], dtype=np.uint32), oracle.F32)
    assert int(p["ulp_hist"][2]) == 1
    # 16-bit dtypes: same-sign patterns a < b are b - a steps apart; +Inf is one step above the largest finite
    for code in (oracle.BF16, oracle.F16):
        inf = 0x7F80 if code == oracle.BF16 else 0x7C00
        a = np.array([0x3C00, 0x0001, inf - 1, 0x8005], dtype=np.uint16)
        b = np.array([0x3C07, 0x0009, inf, 0x0003], dtype=np.uint16)      # 7, 8, 1 and 5 + 3 = 8 steps
        p, _ = oracle.profile(a, b, code)
        assert int(p["ulp_hist"][3]) == 1 and int(p["ulp_hist"][4]) == 2 and int(p["ulp_hist"][1]) == 1


@pytest.mark.parametrize("code,tdt", [(0, torch.float32), (1, torch.bfloat16), (2, torch.float16)])
def test_profile_against_torch_and_numpy(oracle, code, tdt):
    g = torch.Generator().manual_seed(77 + code)
    n = 5000
    r = torch.randn(n, generator=g).to(tdt)
    c = (r.float() * (1 + 2e-2 * torch.randn(n, generator=g))).to(tdt)
    c[::97] = r[::97] + 1.0
    atol = rtol = 1e-2
    p, rows = oracle.profile(r.view(torch.uint8).numpy(), c.view(torch.uint8).numpy(), code, atol, rtol, False, row_len=128)
    close = torch.isclose(c.float(), r.float(), rtol=rtol, atol=atol)
    bad = (~close).numpy()
    assert int(p["n_mismatch"]) == int(bad.sum())
    idx = np.nonzero(bad)[0]
    assert p["first_index"].tolist() == idx[:8].tolist()
    ad = (c.float() - r.float()).abs().numpy()
    ad_bad = np.where(bad, ad, -1.0)
    assert int(p["worst_index"]) == int(np.argmax(ad_bad))          # argmax returns the first of equal maxima
    pad = np.zeros((n + 127) // 128 * 128, dtype=bool)
    pad[:n] = bad
    assert rows.tolist() == pad.reshape(-1, 128).sum(axis=1).tolist()
    assert int(p["ulp_hist"].sum()) == n and int(p["ulp_hist"][65]) == 0
    # the histogram restated with integer views (no NaN here)
    bits = (r.view(torch.int16 if code else torch.int32).numpy().astype(np.int64),
            c.view(torch.int16 if code else torch.int32).numpy().astype(np.int64))
    width = 16 if code else 32
    def order(b):
        u = b & ((1 << width) - 1)
        return np.where(u >> (width - 1), -(u & ((1 << (width - 1)) - 1)), u)
    dist = np.abs(order(bits[1]) - order(bits[0]))
    want = np.bincount(np.where(dist == 0, 0, 1 + np.floor(np.log2(np.maximum(dist, 1))).astype(np.int64)), minlength=66)
    assert p["ulp_hist"].tolist() == want.tolist()
    # consistency with the verifier's record
    rec = oracle.verify(r.view(torch.uint8).numpy(), c.view(torch.uint8).numpy(), code, atol, rtol, False)
    assert int(rec["n_mismatch"]) == int(p["n_mismatch"]) and int(rec["first_mismatch"]) == int(p["first_index"][0])


def test_profile_integers_and_degenerate_cases(oracle):
    i64 = np.iinfo(np.int64)
    r = np.array([0, 5, i64.min, -3, 7, 7], dtype=np.int64)
    c = np.array([0, 6, i64.max, 1, 7, 9], dtype=np.int64)
    p, rows = oracle.profile(r, c, oracle.I64, row_len=2)
    want = np.zeros(66, dtype=np.uint64)
    want[0], want[1], want[64], want[3], want[2] = 2, 1, 1, 1, 1        # 0; 1; 2^64-1; 4; 2
    assert p["ulp_hist"].tolist() == want.tolist()
    assert int(p["n_mismatch"]) == 4 and int(p["worst_index"]) == 2
    assert int(p["worst_c_raw"]) == i64.max and int(p["worst_r_raw"]) == 1 << 63
    assert p["first_index"].tolist()[:4] == [1, 2, 3, 5] and int(p["n_first"]) == 4
    assert rows.tolist() == [1, 2, 1]
    r32 = np.array([-1, 2], dtype=np.int32)
    p, _ = oracle.profile(r32, r32 + 1, oracle.I32)
    assert int(p["ulp_hist"][1]) == 2 and int(p["first_r_raw"][0]) == 0xFFFFFFFF       # raw bits, zero-extended
    # empty and identical inputs
    p, rows = oracle.profile(np.zeros(0, dtype=np.float32), np.zeros(0, dtype=np.float32), oracle.F32, row_len=4)
    assert int(p["ulp_hist"].sum()) == 0 and int(p["worst_index"]) == oracle.NO_INDEX and rows.size == 0
    x = np.linspace(-1, 1, 100, dtype=np.float32)
    p, _ = oracle.profile(x, x.copy(), oracle.F32)
    assert int(p["ulp_hist"][0]) == 100 and int(p["n_mismatch"]) == 0 and int(p["n_first"]) == 0
    # more than eight mismatches: the list keeps the first eight, the count goes on
    p, _ = oracle.profile(np.zeros(20, dtype=np.int32), np.ones(20, dtype=np.int32), oracle.I32)
    assert int(p["n_mismatch"]) == 20 and p["first_index"].tolist() == list(range(8))


# --------------------------------------------------------------------------------------------
# pass/fail summary, pass@k and speedup
# --------------------------------------------------------------------------------------------
def test_exec_summary_and_pass_at_k_exact(oracle):
    from math import comb
    rng = np.random.default_rng(8)
    for T, N in [(1, 1), (3, 5), (6, 20), (2, 64), (0, 4)]:
        rec = np.zeros(T * N, dtype=oracle.RESULT_DTYPE)
        fail = rng.random((T, N)) < 0.15
        rec["n_mismatch"] = np.where(fail, rng.integers(1, 100, (T, N)), 0).reshape(-1)
        ok, c, pk = oracle.exec_summary(rec, T, N, N)
        want_ok = (~fail).all(axis=0) if T else np.ones(N, dtype=bool)
        assert ok.astype(bool).tolist() == want_ok.tolist() and c == int(want_ok.sum())
        for k in range(1, N + 1):
            exact = 1 - Fraction(comb(N - c, k), comb(N, k))           # the estimator in exact rationals
            assert abs(pk[k - 1] - float(exact)) <= 1e-14, (T, N, k)
        if c:
            assert pk[0] == 1.0 - (N - c) / N                           # k = 1 is the plain pass fraction, one rounding each
        assert all(pk[k - 1] == 1.0 for k in range(N - c + 1, N + 1))   # more draws than failures: certain
        assert np.all(np.diff(pk) >= 0)
    # nobody passes / everybody passes
    rec = np.zeros(12, dtype=oracle.RESULT_DTYPE)
    rec["n_mismatch"][:4] = 1                                            # test 0 fails for all four candidates
    ok, c, pk = oracle.exec_summary(rec, 3, 4, 4)
    assert ok.tolist() == [0, 0, 0, 0] and c == 0 and pk.tolist() == [0.0] * 4
    ok, c, pk = oracle.exec_summary(np.zeros(12, dtype=oracle.RESULT_DTYPE), 3, 4, 2)
    assert ok.tolist() == [1] * 4 and c == 4 and pk.tolist() == [1.0, 1.0]


def test_speedup_hand_worked_and_numpy(oracle):
    ref = np.array([[3.0, 1.0, 2.0], [8.0, 8.0, 2.0]], dtype=np.float32)          # medians 2, 8
    gen = np.array([[1.0, 4.0, 1.0, 2.0], [4.0, 1.0, 16.0, 4.0]], dtype=np.float32)  # medians (1+2)/2 = 1.5, 4
    mr, mg, ra, sp = oracle.speedup(ref, gen)
    assert mr.tolist() == [2.0, 8.0] and mg.tolist() == [1.5, 4.0]
    assert ra.tolist() == [np.float32(2.0) / np.float32(1.5), 2.0]
    assert sp == (float(np.float32(2.0) / np.float32(1.5)) + 2.0) / 2
    rng = np.random.default_rng(2)
    for T, sr, sg in [(1, 1, 1), (7, 5, 8), (40, 16, 9), (3, 2, 2)]:
        ref = rng.lognormal(0, 0.3, (T, sr)).astype(np.float32)
        gen = rng.lognormal(-0.2, 0.3, (T, sg)).astype(np.float32)
        ref[0, :] = ref[0, 0]                                          # ties
        mr, mg, ra, sp = oracle.speedup(ref, gen)
        sref, sgen = np.sort(ref, axis=1), np.sort(gen, axis=1)
        wr = sref[:, sr // 2] if sr & 1 else ((sref[:, sr // 2 - 1] + sref[:, sr // 2]) * np.float32(0.5))
        wg = sgen[:, sg // 2] if sg & 1 else ((sgen[:, sg // 2 - 1] + sgen[:, sg // 2]) * np.float32(0.5))
        assert mr.tolist() == wr.tolist() and mg.tolist() == wg.tolist()
        assert ra.tolist() == (wr / wg).tolist()
        assert abs(sp - float(np.mean((wr / wg).astype(np.float64)))) <= 1e-12
    assert oracle.speedup(np.zeros((0, 3), dtype=np.float32), np.zeros((0, 2), dtype=np.float32))[3] == 0.0


def test_speedup_median_is_sort_then_middle_and_zero_is_positive(oracle):
    # both zeros in a row: whichever lands in the middle, the median is +0 (bit pattern 0)
    ref = np.array([[-0.0, 0.0, -0.0, 0.0, 5.0], [0.0, -0.0, -0.0, 1.0, 1.0]], dtype=np.float32)
    gen = np.array([[1.0, 1.0], [2.0, 2.0]], dtype=np.float32)
    mr, mg, ra, _ = oracle.speedup(ref, gen)
    assert mr.view(np.uint32).tolist() == [0, 0] and mg.tolist() == [1.0, 2.0] and ra.view(np.uint32).tolist() == [0, 0]
    ref = np.array([[0.0, -0.0, -0.0, 0.0]], dtype=np.float32)             # even count: (+0) + (+0)
    assert oracle.speedup(ref, gen[:1])[0].view(np.uint32).tolist() == [0]
    # the middle of a sorted row, by hand: 9 distinct values in scrambled order
    ref = np.array([[7, 1, 9, 3, 5, 2, 8, 4, 6]], dtype=np.float32)
    gen = np.array([[7, 1, 9, 3, 5, 2, 8, 4]], dtype=np.float32)          # sorted 1 2 3 4 5 7 8 9 -> (4 + 5) / 2
    mr, mg, ra, sp = oracle.speedup(ref, gen)
    assert mr.tolist() == [5.0] and mg.tolist() == [4.5] and ra.tolist() == [np.float32(5.0) / np.float32(4.5)]


# --------------------------------------------------------------------------------------------
# memory efficiency from latency samples; call / execution accuracy over (kernel x run) matrices
# --------------------------------------------------------------------------------------------
def test_mem_efficiency_hand_worked_and_exact(oracle):
    # two unit tests, latencies in ms, peak 8e9 bytes per ms (8 TB/s)
    lat = np.array([[0.5, 0.25, 1.0], [2.0, 4.0, 8.0]], dtype=np.float32)      # medians 0.5 and 4
    nbytes = np.array([2_000_000_000, 8_000_000_000], dtype=np.uint64)          # 4e9 B/ms and 2e9 B/ms
    med, bw, eff, mean = oracle.mem_efficiency(lat, nbytes, 8e9)
    assert med.tolist() == [0.5, 4.0] and bw.tolist() == [4e9, 2e9] and eff.tolist() == [0.5, 0.25] and mean == 0.375
    # the case study's argument (Appendix A): a kernel that reads and writes the data twice moves twice the
    # bytes a test has to move; at the same device bandwidth it takes twice as long and is half as efficient
    lat1 = np.array([[1.0, 1.0, 1.0]], dtype=np.float32)
    one = oracle.mem_efficiency(lat1, np.array([1 << 30], dtype=np.uint64), float(1 << 30))
    two = oracle.mem_efficiency(lat1 * 2, np.array([1 << 30], dtype=np.uint64), float(1 << 30))
    assert one[2].tolist() == [1.0] and two[2].tolist() == [0.5]
    # random data against exact rationals (each result is one or two correctly rounded binary64 divisions)
    rng = np.random.default_rng(12)
    for T, S in [(1, 1), (9, 4), (30, 7)]:
        lat = rng.lognormal(0, 0.5, (T, S)).astype(np.float32)
        nbytes = rng.integers(1, 1 << 40, T).astype(np.uint64)
        peak = 6.5e9
        med, bw, eff, mean = oracle.mem_efficiency(lat, nbytes, peak)
        srt = np.sort(lat, axis=1)
        want_med = srt[:, S // 2] if S & 1 else (srt[:, S // 2 - 1] + srt[:, S // 2]) * np.float32(0.5)
        assert med.tolist() == want_med.tolist()
        for t in range(T):
            exact_bw = Fraction(int(nbytes[t])) / Fraction(float(want_med[t]))
            assert bw[t] == float(exact_bw)                                      # float(Fraction) rounds correctly
            assert eff[t] == float(Fraction(bw[t]) / Fraction(peak))
        assert abs(mean - float(sum(Fraction(e) for e in eff) / T)) <= 1e-15
    assert oracle.mem_efficiency(np.zeros((0, 2), dtype=np.float32), np.zeros(0, dtype=np.uint64), 1.0)[3] == 0.0
    with pytest.raises(ValueError):
        oracle.mem_efficiency(lat1, np.array([1], dtype=np.uint64), 0.0)


def test_accuracy_printed_fractions_of_the_paper(oracle):
    # one run per kernel: the accuracy is correct / total, total = kernels in the benchmark
    for row in _rows("paper_accuracy_tables.txt"):
        correct, total, printed = row.split()
        correct, total = int(correct), int(total)
        status = np.zeros((total, 1), dtype=np.uint8)
        status[:correct, 0] = 3
        status[correct:correct + (total - correct) // 2, 0] = 1          # compiled, failed a test: counts for call only
        nc, ne, ca, ea = oracle.accuracy_matrix(status, 1)
        assert round(100 * ea[0], 2) == float(printed), row
        assert int(ne.sum()) == correct and ca[0] == (correct + (total - correct) // 2) / total


def test_accuracy_pass_at_k_endpoints_of_the_paper_and_exact_rationals(oracle):
    from math import comb
    rng = np.random.default_rng(13)
    for row in _rows("paper_pass_at_k_endpoints.txt"):
        K, R, with_good, good_total, p1, pR = row.split()
        K, R, with_good = int(K), int(R), int(with_good)
        # spread the good runs over `with_good` kernels (at least one each), any way
        counts = np.zeros(K, dtype=np.int64)
        counts[:with_good] = 1
        if good_total != "*":
            left = int(good_total) - with_good
            while left:
                q = int(rng.integers(0, with_good))
                if counts[q] < R:
                    counts[q] += 1
                    left -= 1
        counts = rng.permutation(counts)
        status = np.zeros((K, R), dtype=np.uint8)
        for q in range(K):
            status[q, rng.permutation(R)[:counts[q]]] = 3
        nc, ne, ca, ea = oracle.accuracy_matrix(status, R)
        assert ne.tolist() == counts.tolist() and nc.tolist() == counts.tolist()
        assert round(100 * ea[R - 1], 2) == float(pR), row
        if p1 != "*":
            assert round(100 * ea[0], 2) == float(p1), row
        for k in range(1, R + 1):                                            # every k against exact rationals
            exact = sum(1 - Fraction(comb(R - int(c), k), comb(R, k)) for c in counts) / K
            assert abs(ea[k - 1] - float(exact)) <= 1e-13
        assert np.all(np.diff(ea) >= -1e-15)
    # bit 1 without bit 0 does not count; bit 0 alone counts for call accuracy only
    status = np.array([[2, 2, 2], [1, 1, 0], [3, 0, 2]], dtype=np.uint8)
    nc, ne, ca, ea = oracle.accuracy_matrix(status, 3)
    assert nc.tolist() == [0, 2, 1] and ne.tolist() == [0, 0, 1]
    assert ca[0] == (0 + 2 / 3 + (1.0 - 2 / 3)) / 3 and ca[2] == 2 / 3 and ea[2] == 1 / 3
    # agreement with the per-kernel summary: one kernel's row gives that function's pass@k
    rec = np.zeros(5, dtype=oracle.RESULT_DTYPE)
    rec["n_mismatch"][[1, 4]] = 7
    ok, c, pk = oracle.exec_summary(rec, 1, 5, 5)
    _, ne, _, ea = oracle.accuracy_matrix((ok * 2 + 1).reshape(1, 5), 5)
    assert ne.tolist() == [c] and ea.tolist() == pk.tolist()
    assert oracle.accuracy_matrix(np.zeros((0, 4), dtype=np.uint8), 2)[2].tolist() == [0.0, 0.0]


# --------------------------------------------------------------------------------------------
# second hash lane (word index multiplied by the odd gamma before the xor)
# --------------------------------------------------------------------------------------------
def test_hash2_zero_words_are_the_published_generator_outputs(oracle):
    # word k of an all-zero buffer contributes splitmix64(k * gamma): output k of the generator seeded with 0
    outs = [int(row.split()[1], 16) for row in _rows("splitmix64_published.txt")]
    for n in range(1, len(outs) + 1):
        assert oracle.hash2_bytes(b"\0" * (8 * n)) == sum(outs[:n]) & M64


def test_hash2_brute_force_and_collision_pair(oracle):
    rng = np.random.default_rng(9)
    data = rng.integers(0, 256, size=4200, dtype=np.uint8).tobytes()
    for nbytes in list(range(0, 40)) + [255, 256, 257, 4096, 4099]:
        b = data[:nbytes] + b"\0" * (-nbytes % 8)
        want = 0
        for k in range(len(b) // 8):
            want = (want + _py_splitmix64(((k * GAMMA) & M64) ^ int.from_bytes(b[8 * k:8 * k + 8], "little"))) & M64
        assert oracle.hash2_bytes(data[:nbytes]) == want, nbytes
    # the pair that collides in the first lane is told apart by the second
    z = np.array([0, 0], dtype=np.int64)
    o = np.array([1, 1], dtype=np.int64)
    assert oracle.hash_bytes(z) == oracle.hash_bytes(o)
    assert oracle.hash2_bytes(z) != oracle.hash2_bytes(o)
    assert oracle.hash2_bytes(b"") == 0
