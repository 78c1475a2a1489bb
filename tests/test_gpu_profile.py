"""GPU parity for the error profile of one candidate (ulp histogram, worst element, first
mismatches, per-row counts): the CUDA library through its C ABI against the CPU oracle, byte for
byte (all outputs are integers or bit patterns)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_2507_23194_b200 import gv  # noqa: E402

DEV = "cuda:0"
TDT = {0: torch.float32, 1: torch.bfloat16, 2: torch.float16, 3: torch.int32, 4: torch.int64}


def hb(t):
    return t.detach().contiguous().view(torch.uint8).cpu().numpy()


def check(oracle, r, c, code, atol, rtol, en, row_len, rd=None, cd=None):
    rd = r.to(DEV) if rd is None else rd
    cd = c.to(DEV) if cd is None else cd
    out, rows = gv.gv_error_profile(rd, cd, atol, rtol, en, row_len)
    torch.cuda.synchronize()
    got = gv.profile_to_numpy(out)
    want, want_rows = oracle.profile(hb(r), hb(c), code, atol, rtol, en, row_len)
    assert got.tobytes() == want.tobytes(), f"dtype {code} n {r.numel()} row_len {row_len}\n gpu    {got}\n oracle {want}"
    if row_len:
        assert rows.cpu().numpy().view(np.uint32).tolist() == want_rows.tolist()


def make(code, n, g, kind):
    if code >= 3:
        r = torch.randint(-(1 << 20), 1 << 20, (n,), generator=g, dtype=TDT[code])
        c = r.clone()
        if kind != "copy" and n:
            k = max(1, n // (3 if kind == "many" else 500))
            pos = torch.randint(0, n, (k,), generator=g)
            c[pos] += torch.randint(-5, 6, (k,), generator=g, dtype=TDT[code])
        return r, c
    r = (torch.randn(n, generator=g) * 3).to(TDT[code])
    if n:
        sp = torch.randint(0, n, (max(1, n // 200),), generator=g)
        vals = torch.tensor([0.0, -0.0, float("inf"), float("-inf"), float("nan"), 1e-40, 65504.0, -1.0])
        r[sp] = vals[torch.randint(0, 8, (sp.numel(),), generator=g)].to(TDT[code])
    if kind == "copy":
        return r, r.clone()
    c = (r.float() * (1 + (3e-2 if kind == "many" else 1e-3) * torch.randn(n, generator=g))).to(TDT[code])
    if n:
        sp = torch.randint(0, n, (max(1, n // (50 if kind == "many" else 5000)),), generator=g)
        c[sp] = (torch.randn(sp.numel(), generator=g) * 10).to(TDT[code])
        sp = torch.randint(0, n, (max(1, n // 3000),), generator=g)
        c[sp] = float("nan")
    return r, c


@pytest.mark.parametrize("code", [0, 1, 2, 3, 4])
def test_profile_size_sweep(oracle, code):
    g = torch.Generator().manual_seed(500 + code)
    for n in (0, 1, 7, 64, 257, 4099, 70001, (1 << 20) + 13):
        for kind in ("copy", "few", "many"):
            r, c = make(code, n, g, kind)
            en = bool((n + len(kind)) & 1)
            row_len = [0, 1, 5, 128, 1000, 1 << 16][(n + len(kind)) % 6]
            check(oracle, r, c, code, 1e-2, 1e-2, en, row_len)


@pytest.mark.parametrize("code", [1, 0, 4])
def test_profile_unaligned_bases(oracle, code):
    g = torch.Generator().manual_seed(900 + code)
    n = 50003
    r, c = make(code, n + 8, g, "many")
    rd, cd = r.to(DEV), c.to(DEV)
    for sr, sc in ((1, 0), (0, 3), (1, 1), (2, 5)):
        check(oracle, r[sr:sr + n], c[sc:sc + n], code, 1e-3, 1e-2, False, 77, rd=rd[sr:sr + n], cd=cd[sc:sc + n])


def test_profile_extremes_and_ties(oracle):
    # every mismatch has the same error: the worst is the first of them; a NaN pair further on takes over
    r = torch.zeros(100000, dtype=torch.float32)
    c = r.clone()
    c[[70000, 123, 99999, 5000]] = 2.0
    check(oracle, r, c, 0, 1e-3, 1e-3, False, 4096)
    c[80000] = float("nan")
    check(oracle, r, c, 0, 1e-3, 1e-3, True, 4096)
    # all elements mismatch (the list keeps the first eight; every row counter is full)
    check(oracle, torch.zeros(300000, dtype=torch.bfloat16), torch.ones(300000, dtype=torch.bfloat16), 1, 0.0, 0.0, False, 1000)
    # int64 extremes: distance 2^64 - 1 falls into the top bucket
    i64 = torch.iinfo(torch.int64)
    r = torch.tensor([i64.min, 0, 5, i64.max] * 1000, dtype=torch.int64)
    c = torch.tensor([i64.max, 0, 6, i64.min] * 1000, dtype=torch.int64)
    check(oracle, r, c, 4, 0.0, 0.0, False, 3)
    # all 16-bit patterns against two references
    for code in (1, 2):
        pats = torch.arange(65536, dtype=torch.int32).to(torch.int16).view(TDT[code])
        for ref_bits in (0x3C00, 0x8001):
            rr = torch.full((65536,), ref_bits, dtype=torch.int32).to(torch.int16).view(TDT[code])
            check(oracle, rr, pats, code, 1e-2, 1e-2, False, 256)
            check(oracle, rr, pats, code, 1e-2, 1e-2, True, 0)


def test_profile_count_matches_verify_record(oracle):
    g = torch.Generator().manual_seed(3)
    r, c = make(1, 1 << 18, g, "many")
    rd, cd = r.to(DEV), c.to(DEV)
    res = gv.gv_verify_batch(rd, [cd], 1e-2, 1e-2, False)
    out, _ = gv.gv_error_profile(rd, cd, 1e-2, 1e-2, False)
    torch.cuda.synchronize()
    rec, prof = gv.results_to_numpy(res)[0], gv.profile_to_numpy(out)
    assert int(rec["n_mismatch"]) == int(prof["n_mismatch"]) and int(rec["first_mismatch"]) == int(prof["first_index"][0])
    assert int(prof["ulp_hist"].sum()) == 1 << 18
