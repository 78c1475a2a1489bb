"""Seeded synthetic workloads for the batched output verifier.

These stand in for the unit-test output tensors of the paper's benchmarks (Section 3: 184
TritonBench-revised kernels and 30 ROCm kernels, at most a handful of unit tests each), which
are not available here and whose shapes and tolerances the paper does not print. Five recipes:
a tiny fp32 correctness case, a dense bf16 GEMM-output batch, attention-output-shaped fp16
tensors, int32/int64 top-k index outputs, and a ragged batch of many small mixed-dtype tensors.

This module serves both the CUDA tests/benchmark and the CPU oracle's tests. It contains no part
of the verifier's arithmetic: it only draws random tensors, perturbs them, and records what it
did ("facts": how many elements it touched and where), so that some expected counts are known by
construction and not from either implementation.

Every candidate is a distinct allocation: "exact copies" are real copies, never aliases.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import torch

# dtype codes of the public C enum (gv_dtype)
GV_F32, GV_BF16, GV_F16, GV_I32, GV_I64 = 0, 1, 2, 3, 4
TORCH_DTYPE = {GV_F32: torch.float32, GV_BF16: torch.bfloat16, GV_F16: torch.float16,
               GV_I32: torch.int32, GV_I64: torch.int64}
ELEM_SIZE = {GV_F32: 4, GV_BF16: 2, GV_F16: 2, GV_I32: 4, GV_I64: 8}


@dataclass
class DenseWorkload:
    name: str
    dtype: int                      # gv_dtype code
    ref: torch.Tensor               # 1-D, contiguous
    cands: List[torch.Tensor]       # N tensors, same shape/dtype as ref, distinct storage
    atol: float
    rtol: float
    equal_nan: bool
    # per candidate: {"class": str, and, where known by construction, "n_mismatch", "first",
    # "n_nan", "n_inf", "same_as" (index of a byte-identical candidate)}
    facts: List[Dict] = field(default_factory=list)

    @property
    def n(self) -> int:
        return self.ref.numel()

    @property
    def cand_bytes(self) -> int:
        return len(self.cands) * self.n * ELEM_SIZE[self.dtype]


@dataclass
class RaggedWorkload:
    name: str
    T: int
    N: int
    ref_buf: torch.Tensor           # uint8, all reference tensors packed
    cand_buf: torch.Tensor          # uint8, all candidates packed
    ref_off: torch.Tensor           # int64 [T+1] byte offsets into ref_buf: starts, then the end of the last tensor
    cand_off: torch.Tensor          # int64 [T*N] byte offsets into cand_buf, tensor-major
    dtypes: torch.Tensor            # uint8 [T] gv_dtype codes
    n_elems: List[int]              # element count per tensor (host list)
    n_elems_t: torch.Tensor         # the same as int64 [T] on the device
    atol: float
    rtol: float
    equal_nan: bool
    facts: List[Dict] = field(default_factory=list)   # T*N entries, tensor-major

    @property
    def cand_bytes(self) -> int:
        return int(sum(n * ELEM_SIZE[int(d)] for n, d in zip(self.n_elems, self.dtypes.tolist()))) * self.N


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _distinct_positions(n: int, k: int, g: torch.Generator, device, allowed: Optional[torch.Tensor] = None,
                        even_only: bool = False) -> torch.Tensor:
    """k distinct seeded positions in [0, n) (int64, sorted), optionally restricted to a mask of
    allowed positions or to even positions i with i + 1 < n."""
    k = int(k)
    if k <= 0:
        return torch.empty(0, dtype=torch.int64, device=device)
    got = torch.empty(0, dtype=torch.int64, device=device)
    rounds = 0
    while got.numel() < k:
        rounds += 1
        if rounds > 64:
            raise RuntimeError("could not draw enough distinct positions")
        want = (k - got.numel()) * 2 + 16
        p = torch.randint(0, n, (want,), generator=g, device=device, dtype=torch.int64)
        if even_only:
            p = p & ~1
            p = p[p + 1 < n]
        if allowed is not None:
            p = p[allowed[p]]
        got = torch.unique(torch.cat([got, p]))
        if got.numel() > k:
            keep = torch.randperm(got.numel(), generator=g, device=device)[:k]
            got = got[keep]
    return torch.sort(got).values


def _fact(cls: str, **kw) -> Dict:
    d = {"class": cls}
    d.update(kw)
    return d


# ----------------------------------------------------------------------------------------------
# config 1: tiny fp32 correctness case
# ----------------------------------------------------------------------------------------------
def config1(device="cpu", n: int = 1 << 20, seed: int = 0) -> DenseWorkload:
    g = _gen(seed, device)
    r = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    cands, facts = [], []

    # 0: exact copy
    cands.append(r.clone())
    facts.append(_fact("copy", n_mismatch=0, first=None, n_nan=0, n_inf=0, hash_equals_ref=True))

    # 1: relative noise of at most 1e-6*|r| -- inside atol = rtol = 1e-5
    u = torch.rand(n, generator=g, device=device, dtype=torch.float32) * 2.0 - 1.0
    cands.append(r + u * 1e-6 * r.abs())
    facts.append(_fact("noise_within_tol", n_mismatch=0, first=None, n_nan=0, n_inf=0))

    # 2: 1000 elements (scaled down for short tensors) replaced by r + 1.0
    k2 = min(1000, max(1, n // 8))
    p2 = _distinct_positions(n, k2, g, device)
    c2 = r.clone()
    c2[p2] = r[p2] + 1.0
    cands.append(c2)
    facts.append(_fact("plus_one", n_mismatch=k2, first=int(p2[0]), n_nan=0, n_inf=0, positions=p2.cpu()))

    # 3: 17 NaNs and 5 +Inf at distinct positions
    k_nan, k_inf = (17, 5) if n >= 64 else (2, 1)
    p3 = _distinct_positions(n, k_nan + k_inf, g, device)
    perm = torch.randperm(k_nan + k_inf, generator=g, device=device)
    p_nan, p_inf = p3[perm[:k_nan]], p3[perm[k_nan:]]
    c3 = r.clone()
    c3[p_nan] = float("nan")
    c3[p_inf] = float("inf")
    cands.append(c3)
    facts.append(_fact("nan_inf", n_mismatch=k_nan + k_inf, first=int(p3[0]), n_nan=k_nan, n_inf=k_inf))

    # 4: byte-identical to #2, separate buffer, different list position
    cands.append(c2.clone())
    facts.append(_fact("plus_one", n_mismatch=k2, first=int(p2[0]), n_nan=0, n_inf=0, same_as=2))

    # 5: every element negated
    cands.append(-r)
    facts.append(_fact("negated", n_nan=0, n_inf=0))

    # 6: all zeros
    cands.append(torch.zeros_like(r))
    facts.append(_fact("zeros", n_nan=0, n_inf=0))

    # 7: copy with one element moved by one ulp (bit pattern + 1: away from zero)
    p7 = int(torch.randint(0, n, (1,), generator=g, device=device))
    c7 = r.clone()
    bits = c7.view(torch.int32)
    bits[p7] += 1
    cands.append(c7)
    facts.append(_fact("one_ulp", n_mismatch=0, first=None, n_nan=0, n_inf=0, position=p7))

    return DenseWorkload("cfg1_fp32_tiny", GV_F32, r, cands, 1e-5, 1e-5, False, facts)


# ----------------------------------------------------------------------------------------------
# config 2: dense bf16 batch (GEMM-output shaped), 256 candidates
# ----------------------------------------------------------------------------------------------
def _bf16_ulp(rf: torch.Tensor) -> torch.Tensor:
    """Spacing of bfloat16 at |r| as fp32: 2^(floor(log2|r|) - 7); 2^-133 at zero."""
    e = (rf.view(torch.int32) >> 23) & 0xFF                  # biased exponent
    e = torch.clamp(e, min=1)                                 # zero/subnormal: smallest normal binade
    return torch.ldexp(torch.ones_like(rf), (e - 127 - 7).to(torch.int32))


def config2(device="cpu", n: int = 4096 * 4096, n_cands: int = 256, seed: int = 1) -> DenseWorkload:
    g = _gen(seed, device)
    r = torch.randn(n, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    rf = r.float()

    n_copy = n_cands // 2
    n_noise = n_cands // 4
    n_err = int(round(n_cands * 0.15))
    n_nan = n_cands - n_copy - n_noise - n_err
    classes = ["copy"] * n_copy + ["noise"] * n_noise + ["errors"] * n_err + ["nan_inf"] * n_nan
    order = torch.randperm(n_cands, generator=g, device=device).tolist()
    classes = [classes[i] for i in order]

    safe = rf.abs() <= 3.0          # positions where an error of >= 0.1 is certainly out of tolerance
    cands, facts = [], []
    for cls in classes:
        if cls == "copy":
            cands.append(r.clone())
            facts.append(_fact(cls, n_mismatch=0, first=None, n_nan=0, n_inf=0, hash_equals_ref=True))
        elif cls == "noise":
            gn = torch.randn(n, generator=g, device=device, dtype=torch.float32)
            c = (rf + gn * 0.25 * _bf16_ulp(rf)).to(torch.bfloat16)
            del gn
            cands.append(c)
            facts.append(_fact(cls, n_mismatch=0, first=None, n_nan=0, n_inf=0))
        elif cls == "errors":
            k = int(torch.randint(1, 10001, (1,), generator=g, device=device))
            k = min(k, max(1, n // 16))
            p = _distinct_positions(n, k, g, device, allowed=safe)
            mag = torch.rand(k, generator=g, device=device) * 9.9 + 0.1
            sgn = torch.randint(0, 2, (k,), generator=g, device=device).float() * 2.0 - 1.0
            c = r.clone()
            c[p] = (rf[p] + sgn * mag).to(torch.bfloat16)
            cands.append(c)
            facts.append(_fact(cls, n_mismatch=k, first=int(p[0]), n_nan=0, n_inf=0))
        else:
            m = max(3, int(round(1e-6 * n)))
            p = _distinct_positions(n, m, g, device)
            kind = torch.randint(0, 3, (m,), generator=g, device=device)
            vals = torch.tensor([float("nan"), float("inf"), float("-inf")], device=device)[kind]
            c = r.clone()
            c[p] = vals.to(torch.bfloat16)
            cands.append(c)
            facts.append(_fact(cls, n_mismatch=m, first=int(p[0]), n_nan=int((kind == 0).sum()),
                               n_inf=int((kind != 0).sum())))
    return DenseWorkload("cfg2_bf16_dense", GV_BF16, r, cands, 1.6e-2, 1.6e-2, True, facts)


# ----------------------------------------------------------------------------------------------
# config 3: attention-output-shaped fp16, 32 candidates with relative noise
# ----------------------------------------------------------------------------------------------
def config3(device="cpu", n: int = 8 * 32 * 4096 * 128, n_cands: int = 32, seed: int = 2) -> DenseWorkload:
    g = _gen(seed, device)
    r = (torch.randn(n, generator=g, device=device, dtype=torch.float32) * 0.05).clamp_(-4.0, 4.0).to(torch.float16)
    sigmas = [0.0, 1e-4, 1e-3, 5e-3, 2e-2]
    cands, facts = [], []
    for j in range(n_cands):
        s = sigmas[j % len(sigmas)]
        if s == 0.0:
            cands.append(r.clone())
            facts.append(_fact("copy", n_mismatch=0, first=None, n_nan=0, n_inf=0, hash_equals_ref=True, sigma=s))
        else:
            eps = torch.randn(n, generator=g, device=device, dtype=torch.float32) * s
            c = (r.float() * (1.0 + eps)).to(torch.float16)
            del eps
            cands.append(c)
            facts.append(_fact("rel_noise", n_nan=0, n_inf=0, sigma=s))
    return DenseWorkload("cfg3_fp16_attention", GV_F16, r, cands, 1e-2, 1e-2, False, facts)


# ----------------------------------------------------------------------------------------------
# config 4: int32 top-k indices (and the same data widened to int64), exact mode
# ----------------------------------------------------------------------------------------------
def config4(device="cpu", n: int = 65536 * 1024, n_cands: int = 64, seed: int = 3, wide: bool = False) -> DenseWorkload:
    g = _gen(seed, device)
    r = torch.randint(0, 50257, (n,), generator=g, device=device, dtype=torch.int32)
    fracs = [1e-7, 1e-5, 1e-3]
    cands, facts = [], []
    out_dtype = torch.int64 if wide else torch.int32
    for j in range(n_cands):
        if j % 2 == 0:
            cands.append(r.to(out_dtype).clone())
            facts.append(_fact("copy", n_mismatch=0, first=None, n_nan=0, n_inf=0, hash_equals_ref=True))
            continue
        p = fracs[(j // 2) % 3]
        k = max(1, int(p * n / 2))
        pos = _distinct_positions(n, k, g, device, even_only=True)
        pos = pos[r[pos] != r[pos + 1]]          # a swap of equal neighbours changes nothing
        c = r.clone()
        c[pos] = r[pos + 1]
        c[pos + 1] = r[pos]
        cands.append(c.to(out_dtype))
        facts.append(_fact("swaps", n_mismatch=2 * int(pos.numel()),
                           first=(int(pos[0]) if pos.numel() else None), n_nan=0, n_inf=0, frac=p))
    ref = r.to(out_dtype)
    name = "cfg4_int64_topk" if wide else "cfg4_int32_topk"
    return DenseWorkload(name, GV_I64 if wide else GV_I32, ref, cands, 0.0, 0.0, False, facts)


# ----------------------------------------------------------------------------------------------
# config 5: ragged batch of many small test tensors, mixed dtypes, 4 candidates each
# ----------------------------------------------------------------------------------------------
def config5(device="cpu", T: int = 10000, max_log2: float = 20.0, seed: int = 4, align: int = 16) -> RaggedWorkload:
    """``align`` = 16 pads every tensor start to 16 bytes (the benchmark layout); ``align`` = 0
    packs tightly, each tensor starting on a multiple of its own element size only."""
    g = _gen(seed, device)
    N = 4
    u = torch.rand(T, generator=g, device=device, dtype=torch.float64)
    n_elems = torch.floor(torch.pow(2.0, max_log2 * u)).to(torch.int64).clamp_(min=1).tolist()
    codes = torch.tensor([GV_F32, GV_BF16, GV_F16, GV_I32], device=device)[
        torch.randint(0, 4, (T,), generator=g, device=device)].to(torch.uint8)
    codes_l = codes.tolist()

    def place(cursor: int, esz: int) -> int:
        a = align if align else esz
        return (cursor + a - 1) // a * a

    # layout pass
    ref_start, cand_off = [], []
    rc = cc = 0
    for t in range(T):
        esz = ELEM_SIZE[codes_l[t]]
        nb = n_elems[t] * esz
        rc = place(rc, esz)
        ref_start.append(rc)
        rc += nb
        for _ in range(N):
            cc = place(cc, esz)
            cand_off.append(cc)
            cc += nb
    ref_total, cand_total = rc, cc
    ref_buf = torch.zeros(max(ref_total, 1), dtype=torch.uint8, device=device)
    cand_buf = torch.zeros(max(cand_total, 1), dtype=torch.uint8, device=device)

    facts: List[Dict] = []
    for t in range(T):
        code = codes_l[t]
        n = n_elems[t]
        esz = ELEM_SIZE[code]
        td = TORCH_DTYPE[code]
        if code == GV_I32:
            r = torch.randint(-(1 << 20), (1 << 20) + 1, (n,), generator=g, device=device, dtype=torch.int32)
            noise = r.clone()
            one = r.clone()
            p1 = int(torch.randint(0, n, (1,), generator=g, device=device))
            one[p1] += 1
            k = math.ceil(0.01 * n)
            pk = _distinct_positions(n, k, g, device)
            many = r.clone()
            many[pk] += 1
        else:
            r = torch.randn(n, generator=g, device=device, dtype=torch.float32).to(td)
            uu = torch.rand(n, generator=g, device=device, dtype=torch.float32) * 2.0 - 1.0
            noise = (r.float() * (1.0 + 1e-4 * uu)).to(td)
            p1 = int(torch.randint(0, n, (1,), generator=g, device=device))
            one = r.clone()
            one[p1] = (r[p1].float() + 1.0).to(td)
            k = math.ceil(0.01 * n)
            pk = _distinct_positions(n, k, g, device)
            many = r.clone()
            many[pk] = (r[pk].float() + 1.0).to(td)
        nb = n * esz
        ref_buf[ref_start[t]:ref_start[t] + nb] = r.view(torch.uint8)
        for j, c in enumerate((r.clone(), noise, one, many)):
            o = cand_off[t * N + j]
            cand_buf[o:o + nb] = c.view(torch.uint8)
        facts.append(_fact("copy", n_mismatch=0, first=None, n_nan=0, n_inf=0, hash_equals_ref=True))
        facts.append(_fact("noise_within_tol", n_mismatch=0, first=None, n_nan=0, n_inf=0))
        facts.append(_fact("one_error", n_mismatch=1, first=p1, n_nan=0, n_inf=0))
        facts.append(_fact("one_percent", n_mismatch=k, first=int(pk[0]), n_nan=0, n_inf=0))

    # offsets table: T+1 entries; entry t is the start of tensor t, entry T the end of the last
    # tensor's payload. With padding between tensors the element counts cannot be read off
    # consecutive offsets, so they travel separately (n_elems).
    ref_off = torch.tensor(ref_start + [ref_start[-1] + n_elems[-1] * ELEM_SIZE[codes_l[-1]] if T else 0],
                           dtype=torch.int64, device=device)
    return RaggedWorkload(
        name=("cfg5_ragged_mixed" if align else "cfg5_ragged_mixed_tight"), T=T, N=N, ref_buf=ref_buf,
        cand_buf=cand_buf, ref_off=ref_off,
        cand_off=torch.tensor(cand_off, dtype=torch.int64, device=device), dtypes=codes,
        n_elems=n_elems, n_elems_t=torch.tensor(n_elems, dtype=torch.int64, device=device), atol=1e-3, rtol=1e-3, equal_nan=False, facts=facts)
