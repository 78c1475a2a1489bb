"""GPU parity for the aggregates (pass/fail summary with pass@k, speedup from latency samples): the
CUDA library through its C ABI against the CPU oracle, bit for bit (both sides evaluate the same
sequence of IEEE operations)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from paper_2507_23194_b200 import gv, workloads as W  # noqa: E402

DEV = "cuda:0"


@pytest.mark.parametrize("T,N,p_fail", [(0, 3, 0.0), (1, 1, 0.0), (1, 1, 1.0), (3, 5, 0.2), (6, 64, 0.05), (2, 300, 0.3),
                                        (40, 1000, 0.01), (1, 4096, 0.5)])
def test_exec_summary_against_oracle(oracle, T, N, p_fail):
    rng = np.random.default_rng(T * 1000 + N)
    rec = np.zeros(T * N, dtype=gv.RESULT_DTYPE)
    if T:
        rec["n_mismatch"] = np.where(rng.random(T * N) < p_fail, rng.integers(1, 1 << 40, T * N), 0)
        rec["hash"] = rng.integers(0, 1 << 62, T * N)
    res = torch.from_numpy(rec.view(np.uint8).reshape(-1, 64).copy() if T * N else np.zeros((0, 64), dtype=np.uint8)).to(DEV)
    ok, c, pk = gv.gv_exec_summary(res, T, N, N)
    torch.cuda.synchronize()
    w_ok, w_c, w_pk = oracle.exec_summary(rec, T, N, N)
    assert ok.cpu().numpy().tolist() == w_ok.tolist()
    assert int(c.cpu()[0]) == w_c
    assert pk.cpu().numpy().tobytes() == w_pk.tobytes()            # binary64, bit for bit


def test_exec_summary_of_a_ragged_verify(oracle):
    wl = W.config5(DEV, T=60, max_log2=12.0)
    ws = torch.empty(gv.gv_workspace_bytes(wl.T, wl.N), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_ragged(wl.ref_buf, wl.ref_off, wl.cand_buf, wl.cand_off, wl.dtypes, wl.N, wl.atol, wl.rtol,
                              wl.equal_nan, n_elems=wl.n_elems_t, workspace=ws)
    ok, c, pk = gv.gv_exec_summary(res, wl.T, wl.N, wl.N)
    torch.cuda.synchronize()
    w_ok, w_c, w_pk = oracle.exec_summary(gv.results_to_numpy(res), wl.T, wl.N, wl.N)
    assert ok.cpu().numpy().tolist() == w_ok.tolist() == [1, 1, 0, 0]     # copy and in-tolerance noise pass
    assert int(c.cpu()[0]) == w_c == 2 and pk.cpu().numpy().tobytes() == w_pk.tobytes()


@pytest.mark.parametrize("T,sr,sg", [(0, 3, 3), (1, 1, 1), (5, 2, 3), (33, 7, 8), (200, 100, 31), (4, 4096, 4095), (3000, 9, 9)])
def test_speedup_against_oracle(oracle, T, sr, sg):
    rng = np.random.default_rng(T + sr * 7 + sg)
    ref = rng.lognormal(0.0, 0.4, (T, sr)).astype(np.float32)
    gen = rng.lognormal(-0.3, 0.4, (T, sg)).astype(np.float32)
    if T:
        ref[0, :] = ref[0, 0]                                       # a row of ties
        gen[-1, ::2] = gen[-1, 0]
    mr, mg, ra, sp = gv.gv_speedup(torch.from_numpy(ref).to(DEV), torch.from_numpy(gen).to(DEV))
    torch.cuda.synchronize()
    w_mr, w_mg, w_ra, w_sp = oracle.speedup(ref, gen)
    assert mr.cpu().numpy().tobytes() == w_mr.tobytes()
    assert mg.cpu().numpy().tobytes() == w_mg.tobytes()
    assert ra.cpu().numpy().tobytes() == w_ra.tobytes()
    assert np.float64(sp.cpu()[0]).tobytes() == np.float64(w_sp).tobytes()


def test_speedup_zero_medians_are_positive_zero(oracle):
    ref = np.array([[-0.0, 0.0, -0.0, 0.0, 5.0], [0.0, -0.0, -0.0, 1.0, 1.0], [0.0, -0.0, -0.0, 0.0, 0.0]], dtype=np.float32)
    gen = np.array([[1.0, 1.0], [2.0, 2.0], [4.0, 4.0]], dtype=np.float32)
    for _ in range(5):                                                 # which thread writes last may vary: repeat
        mr, mg, ra, sp = gv.gv_speedup(torch.from_numpy(ref).to(DEV), torch.from_numpy(gen).to(DEV))
        torch.cuda.synchronize()
        w_mr, w_mg, w_ra, w_sp = oracle.speedup(ref, gen)
        assert mr.cpu().numpy().tobytes() == w_mr.tobytes() and mr.cpu().numpy().view(np.uint32).tolist() == [0, 0, 0]
        assert ra.cpu().numpy().tobytes() == w_ra.tobytes()


@pytest.mark.parametrize("T,S", [(0, 3), (1, 1), (5, 2), (33, 7), (200, 100), (4, 4096), (3000, 9)])
def test_mem_efficiency_against_oracle(oracle, T, S):
    rng = np.random.default_rng(T * 31 + S)
    lat = rng.lognormal(-1.0, 0.5, (T, S)).astype(np.float32)
    nbytes = rng.integers(1, 1 << 42, T).astype(np.uint64)
    if T:
        lat[0, :] = lat[0, 0]
    peak = 6.5424e9
    med, bw, eff, mean = gv.gv_mem_efficiency(torch.from_numpy(lat).to(DEV),
                                              torch.from_numpy(nbytes.view(np.int64)).to(DEV), peak)
    torch.cuda.synchronize()
    w_med, w_bw, w_eff, w_mean = oracle.mem_efficiency(lat, nbytes, peak)
    assert med.cpu().numpy().tobytes() == w_med.tobytes()
    assert bw.cpu().numpy().tobytes() == w_bw.tobytes() and eff.cpu().numpy().tobytes() == w_eff.tobytes()
    assert np.float64(mean.cpu()[0]).tobytes() == np.float64(w_mean).tobytes()


@pytest.mark.parametrize("K,R,p_call,p_exec", [(0, 4, 0.5, 0.5), (1, 1, 1.0, 1.0), (1, 1, 0.0, 0.0), (184, 10, 0.55, 0.6),
                                               (30, 10, 0.44, 0.8), (1000, 64, 0.3, 0.3), (7, 1024, 0.01, 0.5), (50000, 3, 0.5, 0.5)])
def test_accuracy_matrix_against_oracle(oracle, K, R, p_call, p_exec):
    rng = np.random.default_rng(K * 7 + R)
    call = rng.random((K, R)) < p_call
    ex = rng.random((K, R)) < p_exec                                     # bit 1 may be set without bit 0: must not count
    status = (call.astype(np.uint8) | (ex.astype(np.uint8) << 1)) | (rng.integers(0, 2, (K, R)).astype(np.uint8) << 4)
    nc, ne, ca, ea = gv.gv_accuracy_matrix(torch.from_numpy(status).to(DEV), R)
    torch.cuda.synchronize()
    w_nc, w_ne, w_ca, w_ea = oracle.accuracy_matrix(status, R)
    assert nc.cpu().numpy().tolist() == w_nc.tolist() and ne.cpu().numpy().tolist() == w_ne.tolist()
    assert ca.cpu().numpy().tobytes() == w_ca.tobytes() and ea.cpu().numpy().tobytes() == w_ea.tobytes()


def test_accuracy_from_verifier_records_end_to_end(oracle):
    # records of a ragged verify -> pass flags (gv_exec_summary) -> one row of the status matrix -> accuracies
    wl = W.config5(DEV, T=30, max_log2=11.0, seed=5)
    ws = torch.empty(gv.gv_workspace_bytes(wl.T, wl.N), dtype=torch.uint8, device=DEV)
    res = gv.gv_verify_ragged(wl.ref_buf, wl.ref_off, wl.cand_buf, wl.cand_off, wl.dtypes, wl.N, wl.atol, wl.rtol,
                              wl.equal_nan, n_elems=wl.n_elems_t, workspace=ws)
    ok, c, pk = gv.gv_exec_summary(res, wl.T, wl.N, wl.N)
    status = (ok * 2 + 1).reshape(1, wl.N).contiguous()                  # every run compiled; bit 1 = passed all tests
    nc, ne, ca, ea = gv.gv_accuracy_matrix(status, wl.N)
    torch.cuda.synchronize()
    assert ne.cpu().tolist() == [int(c.cpu()[0])] and nc.cpu().tolist() == [wl.N]
    assert ea.cpu().numpy().tobytes() == pk.cpu().numpy().tobytes()       # one kernel: its pass@k
    assert ca.cpu().numpy().tolist() == [1.0] * wl.N
