"""GPU checks of the boundary's promises outside the plain parity cases: nothing is written outside the
caller's records, inconsistent ragged tables are flagged without being followed (huge counts included), a
bounded device-side wait that expires is reported and leaves the device usable, and the second hash lane's
main loop agrees with the oracle on buffers large enough to reach it."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_2507_23194_b200 import gv, workloads as W  # noqa: E402

DEV = "cuda:0"


def host_bytes(t):
    return t.detach().contiguous().view(torch.uint8).cpu().numpy()


def test_hash2_main_loop_on_large_buffers(oracle):
    # the four-vector loop of the hash kernel runs only when a thread owns four vectors: 64 MiB and more
    rng = np.random.default_rng(31)
    data = torch.from_numpy(rng.integers(0, 256, size=(96 << 20) + 64, dtype=np.uint8))
    dd = data.to(DEV)
    for off, nbytes in [(0, 64 << 20), (0, (64 << 20) + 7), (16, (96 << 20) - 5), (0, (96 << 20) + 16), (3, 80 << 20)]:
        h2 = gv.gv_hash2(dd[off:off + nbytes])
        h1 = gv.gv_hash(dd[off:off + nbytes])
        part = data[off:off + nbytes].numpy()
        assert int(h2.cpu().numpy().view(np.uint64)[0]) == oracle.hash2_bytes(part), (off, nbytes)
        assert int(h1.cpu().numpy().view(np.uint64)[0]) == oracle.hash_bytes(part), (off, nbytes)


def test_records_have_guards_on_both_sides(oracle):
    # dense: N records inside a larger buffer of sentinel bytes; ragged: the same with T * N records
    wl = W.config1(DEV, n=(1 << 15) + 11)
    N = len(wl.cands)
    buf = torch.full((N + 8, 64), 0x5A, dtype=torch.uint8, device=DEV)
    ws = torch.empty(gv.gv_workspace_bytes(0, N), dtype=torch.uint8, device=DEV)
    rh_buf = torch.full((3,), 0x5A5A5A5A5A5A5A5A, dtype=torch.int64, device=DEV)
    gv.gv_verify_batch(wl.ref, wl.cands, wl.atol, wl.rtol, wl.equal_nan, results=buf[4:4 + N], ref_hash=rh_buf[1:2],
                       workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    out = buf.cpu().numpy()
    assert (out[:4] == 0x5A).all() and (out[4 + N:] == 0x5A).all()
    assert rh_buf.cpu().tolist()[0] == 0x5A5A5A5A5A5A5A5A and rh_buf.cpu().tolist()[2] == 0x5A5A5A5A5A5A5A5A
    want = oracle.verify_batch(host_bytes(wl.ref), [host_bytes(c) for c in wl.cands], oracle.F32, wl.atol, wl.rtol,
                               wl.equal_nan)
    assert out[4:4 + N].tobytes() == want.tobytes()
    rw = W.config5(DEV, T=50, max_log2=13.0, seed=21)
    cnt = rw.T * rw.N
    buf = torch.full((cnt + 8, 64), 0x5A, dtype=torch.uint8, device=DEV)
    ws = torch.empty(gv.gv_workspace_bytes(rw.T, rw.N), dtype=torch.uint8, device=DEV)
    gv.gv_verify_ragged(rw.ref_buf, rw.ref_off, rw.cand_buf, rw.cand_off, rw.dtypes, rw.N, rw.atol, rw.rtol, rw.equal_nan,
                        n_elems=rw.n_elems_t, results=buf[4:4 + cnt], workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    out = buf.cpu().numpy()
    assert (out[:4] == 0x5A).all() and (out[4 + cnt:] == 0x5A).all()
    want = oracle.verify_ragged(rw.ref_buf.cpu().numpy(), rw.ref_off.cpu().numpy(), rw.cand_buf.cpu().numpy(),
                                rw.cand_off.cpu().numpy(), rw.dtypes.cpu().numpy(), rw.N, rw.atol, rw.rtol, rw.equal_nan,
                                n_elems=rw.n_elems_t.cpu().numpy())
    assert out[4:4 + cnt].tobytes() == want.tobytes()


@pytest.mark.parametrize("huge", [1 << 62, (1 << 61) + 1, (1 << 40) + 1, -5])      # each beyond the limit for every element size
def test_huge_or_negative_counts_are_flagged_not_followed(oracle, huge):
    # one table entry claims an absurd element count: the tensor's records stay zero records, the status word
    # says so, every other tensor is verified as usual, and nothing outside the buffers is touched
    rw = W.config5(DEV, T=24, max_log2=11.0, seed=22)
    ne = rw.n_elems_t.clone()
    victim = 7
    ne[victim] = huge
    ws = torch.empty(gv.gv_workspace_bytes(rw.T, rw.N), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_ragged(rw.ref_buf, rw.ref_off, rw.cand_buf, rw.cand_off, rw.dtypes, rw.N, rw.atol, rw.rtol,
                              rw.equal_nan, n_elems=ne, workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_ERR_BAD_TABLE
    got = gv.results_to_numpy(res)
    want = oracle.verify_ragged(rw.ref_buf.cpu().numpy(), rw.ref_off.cpu().numpy(), rw.cand_buf.cpu().numpy(),
                                rw.cand_off.cpu().numpy(), rw.dtypes.cpu().numpy(), rw.N, rw.atol, rw.rtol, rw.equal_nan,
                                n_elems=rw.n_elems_t.cpu().numpy())
    zero = np.zeros((), dtype=gv.RESULT_DTYPE)
    zero["first_mismatch"] = gv.GV_NO_INDEX
    for t in range(rw.T):
        for j in range(rw.N):
            i = t * rw.N + j
            assert got[i].tobytes() == (zero if t == victim else want[i]).tobytes(), (t, j)
    # the same table through the entry point with the library's own scratch
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    res2 = torch.zeros((rw.T * rw.N, 64), dtype=torch.uint8, device=DEV)
    gv.gv_verify_ragged_noalloc(rw.ref_buf, rw.ref_off, rw.cand_buf, rw.cand_off, rw.dtypes, rw.N, rw.atol, rw.rtol,
                                rw.equal_nan, results=res2, n_elems=ne, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 2 and gv.results_to_numpy(res2).tobytes() == got.tobytes()


def test_offsets_spanning_an_absurd_size_are_flagged(oracle):
    # counts read off consecutive offsets: a span of 2^62 bytes is a bad entry, not a tensor. (It is the LAST
    # tensor's span: an offsets table cannot make an inner span huge without also moving the next tensor's
    # start out of the buffer, which the library has no means to detect -- buffer sizes are not arguments.)
    T, N = 2, 2
    ref = torch.arange(64, dtype=torch.int32, device=DEV)
    offs = torch.tensor([0, 64, (1 << 62) + 64], dtype=torch.int64, device=DEV)
    cand = torch.cat([ref, ref]).contiguous()
    cand_off = torch.tensor([0, 256, 64, 320], dtype=torch.int64, device=DEV)
    dtypes = torch.full((T,), 3, dtype=torch.uint8, device=DEV)
    ws = torch.empty(gv.gv_workspace_bytes(T, N), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_ragged(ref.view(torch.uint8), offs, cand.view(torch.uint8), cand_off, dtypes, N, 0.0, 0.0, False,
                              workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_ERR_BAD_TABLE
    got = gv.results_to_numpy(res)
    assert int(got[0]["hash"]) == oracle.hash_bytes(host_bytes(ref[:16])) and int(got[0]["n_mismatch"]) == 0
    assert int(got[1]["hash"]) == int(got[0]["hash"])
    assert int(got[2]["hash"]) == 0 and int(got[3]["hash"]) == 0            # the flagged tensor: zero records


def test_bounded_wait_that_expires_is_reported_and_the_device_stays_usable(oracle):
    ws = torch.zeros(gv.gv_workspace_bytes(0, 4), dtype=torch.uint8, device=DEV)
    gv.gv_selftest_wait_expiry(ws)
    assert gv.gv_check(ws) == gv.GV_ERR_DEVICE_TIMEOUT                        # gv_check synchronises: the kernel returned
    assert gv.lib.gv_status_string(gv.GV_ERR_DEVICE_TIMEOUT) == b"device-side wait timed out"
    # an ordinary call on the same workspace right after it is clean and correct
    wl = W.config1(DEV, n=(1 << 14) + 3)
    res = gv.gv_verify_batch(wl.ref, wl.cands[:4], wl.atol, wl.rtol, wl.equal_nan, workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    want = oracle.verify_batch(host_bytes(wl.ref), [host_bytes(c) for c in wl.cands[:4]], oracle.F32, wl.atol, wl.rtol,
                               wl.equal_nan)
    assert gv.results_to_numpy(res).tobytes() == want.tobytes()


def test_read_sum_probe_sums_the_words():
    rng = np.random.default_rng(32)
    for n_words in (0, 4, 4 * 257, (1 << 22) + 4 * 3, 40 << 20):
        a = rng.integers(0, 1 << 32, size=n_words, dtype=np.uint64).astype(np.uint32)
        d = torch.from_numpy(a.view(np.int32)).to(DEV)
        out = gv.gv_selftest_read_sum(d)
        assert int(out.cpu().numpy().view(np.uint64)[0]) == int(a.sum(dtype=np.uint64))


@pytest.mark.parametrize("equal_nan", [False, True])
def test_ragged_four_candidates_with_nan_and_inf_in_the_references(oracle, equal_nan):
    """The four-candidate instance of the ragged kernel on references that hold NaNs and infinities: candidate
    vectors identical to such a reference vector must still go through the rule (NaN is not close to NaN
    unless equal_nan), vectors identical to one holding an infinity may, and both must give the oracle's
    records. Large tensors (many streamed tiles per warp), all three float dtypes, plus an integer one."""
    g = torch.Generator().manual_seed(4242)
    tdt = {0: torch.float32, 1: torch.bfloat16, 2: torch.float16, 3: torch.int32}
    esz = {0: 4, 1: 2, 2: 2, 3: 4}
    codes = [0, 1, 2, 3, 2, 0]
    sizes = [(1 << 19) + 13, (1 << 20) + 8, 777777, 1 << 18, 4096, 33]
    N = 4
    refs, cands = [], []
    for code, n in zip(codes, sizes):
        if code == 3:
            r = torch.randint(-1000, 1000, (n,), generator=g, dtype=torch.int32)
        else:
            r = torch.randn(n, generator=g).to(tdt[code])
            where = torch.randint(0, n, (40,), generator=g)
            r[where[:15]] = float("nan")
            r[where[15:28]] = float("inf")
            r[where[28:]] = float("-inf")
        refs.append(r)
        cands.append(r.clone())                                          # identical, NaNs and infinities included
        c = r.clone()
        idx = torch.randint(0, n, (max(1, n // 100),), generator=g)
        c[idx] = (c[idx].float() + 1.0).to(tdt[code]) if code != 3 else c[idx] + 1
        cands.append(c)                                                  # about 1 % changed
        if code == 3:
            cands.append(r + 1)
        else:
            cands.append((r.float() * 1.0001).to(tdt[code]))             # differs (almost) everywhere, within tolerance
        c = r.clone()
        if code != 3:
            c[torch.isnan(r)] = 0.0                                      # NaN on one side only
            c[torch.isinf(r)] = -c[torch.isinf(r)]                       # the other infinity
        cands.append(c)
    ref_off, cand_off, rc, cc = [], [], 0, 0
    for t, (code, n) in enumerate(zip(codes, sizes)):
        rc = (rc + 15) // 16 * 16
        ref_off.append(rc)
        rc += n * esz[code]
        for j in range(N):
            cc = (cc + 15) // 16 * 16
            cand_off.append(cc)
            cc += n * esz[code]
    ref_off.append(rc)
    ref_buf = torch.zeros(rc, dtype=torch.uint8)
    cand_buf = torch.zeros(cc, dtype=torch.uint8)
    for t, (code, n) in enumerate(zip(codes, sizes)):
        nb = n * esz[code]
        ref_buf[ref_off[t]:ref_off[t] + nb] = refs[t].view(torch.uint8)
        for j in range(N):
            o = cand_off[t * N + j]
            cand_buf[o:o + nb] = cands[t * N + j].view(torch.uint8)
    ro, co = torch.tensor(ref_off), torch.tensor(cand_off)
    dts, ne = torch.tensor(codes, dtype=torch.uint8), torch.tensor(sizes)
    ws = torch.empty(gv.gv_workspace_bytes(len(codes), N), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_ragged(ref_buf.to(DEV), ro.to(DEV), cand_buf.to(DEV), co.to(DEV), dts.to(DEV), N, 1e-2, 1e-2,
                              equal_nan, n_elems=ne.to(DEV), workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    want = oracle.verify_ragged(ref_buf.numpy(), ro.numpy(), cand_buf.numpy(), co.numpy(), dts.numpy(), N, 1e-2, 1e-2,
                                equal_nan, n_elems=ne.numpy())
    got = gv.results_to_numpy(res)
    for i in range(len(got)):
        assert got[i].tobytes() == want[i].tobytes(), (i, got[i], want[i])
    n_nan = int(torch.isnan(refs[0]).sum())
    assert int(got[0]["n_mismatch"]) == (0 if equal_nan else n_nan)      # fp32 tensor, exact copy: only its NaNs can mismatch


@pytest.mark.parametrize("order", ["ascending", "descending", "small_last"])
def test_ragged_records_do_not_depend_on_the_order_of_the_tensors(oracle, order):
    """The ragged kernel hands out work in chunks of the tensor sequence; with the tensors sorted by size a
    chunk holds hundreds of tiny tensors or a slice of one large tensor. Same tensors, tables permuted on the
    host (the data stay where they are): every tensor's records must equal the oracle's for the original order."""
    wl = W.config5(DEV, T=2500, max_log2=17.0, seed=31)
    N = wl.N
    ne = wl.n_elems
    if order == "ascending":
        perm = sorted(range(wl.T), key=lambda t: ne[t])
    elif order == "descending":
        perm = sorted(range(wl.T), key=lambda t: -ne[t])
    else:
        perm = [t for t in range(wl.T) if ne[t] >= 2048] + [t for t in range(wl.T) if ne[t] < 2048]
    idx = torch.tensor(perm, device=DEV)
    ro = torch.cat([wl.ref_off[idx], wl.ref_off[-1:]])
    co = wl.cand_off.view(wl.T, N)[idx].contiguous().view(-1)
    ws = torch.empty(gv.gv_workspace_bytes(wl.T, N), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_ragged(wl.ref_buf, ro, wl.cand_buf, co, wl.dtypes[idx].contiguous(), N, wl.atol, wl.rtol,
                              wl.equal_nan, n_elems=wl.n_elems_t[idx].contiguous(), workspace=ws)
    torch.cuda.synchronize()
    assert gv.gv_check(ws) == gv.GV_OK
    got = gv.results_to_numpy(res).reshape(wl.T, N)
    want = oracle.verify_ragged(wl.ref_buf.cpu().numpy(), wl.ref_off.cpu().numpy(), wl.cand_buf.cpu().numpy(),
                                wl.cand_off.cpu().numpy(), wl.dtypes.cpu().numpy(), N, wl.atol, wl.rtol, wl.equal_nan,
                                n_elems=wl.n_elems_t.cpu().numpy()).reshape(wl.T, N)
    for pos, t in enumerate(perm):
        assert got[pos].tobytes() == want[t].tobytes(), (order, pos, t, ne[t])
