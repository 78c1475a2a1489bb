#!/usr/bin/env python
"""Benchmark of the batched output verifier: GB/s of candidate outputs verified.

One "step" is one pass of the whole hot path (result init, sampling pass and the fused verify kernel;
ragged: init, table pre-pass, verify kernel) over one batch of synthetic candidates. The headline
workload is the dense bf16 one (a 4096x4096 reference, 256 candidates, 8 GiB of candidate data per
step, far larger than L2, so no cache flush is needed between steps).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3|cfg4|cfg4w|cfg5|cfg1]
    python bench.py --impl reference ...     # the CPU oracle on a bounded sample, for context

The default single-GPU run also reports, after the headline's K timed steps, every seeded workload of the
recipe (`per_config`: cfg1, cfg2, cfg3, cfg4, cfg4w, cfg5, each timed for about half a second of kernel
time, with its own clock record and a sample of records compared with the CPU oracle), the headline
workload split by candidate class (`per_class`), and a read-only bandwidth probe beside the copy peak.
`--no-extras` (and any run with N > 1 or a non-default workload) prints the headline only.

With N > 1 (launched by torch.distributed.run) every rank verifies its own full batch on its own
GPU (weak scaling, no data-path collective: candidates are independent); timing is the maximum over
ranks. Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "GB/s of candidate outputs verified (fraction of B200 HBM peak)"
FALLBACK_HBM_GBS = 6650.0
ALL_WORKLOADS = ["cfg1", "cfg2", "cfg3", "cfg4", "cfg4w", "cfg5"]

# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum) from the
# ncu captures summarised under profiles/. The captures ran on a reduced number of candidates /
# tensors of the same shapes; the figures here are scaled to the full launch in proportion to the
# units processed (traffic is proportional to them: every candidate byte is read once, the reference
# once per chunk of 16 candidates).
def _scaled(measured, ref_bytes, cap_cands, full_cands, cap_chunks=None, full_chunks=None):
    """Capture on cap_cands candidates -> full launch: the candidate part scales with the number of
    candidates, the reference part with the number of chunks the kernel forms (16 candidates each
    unless the chunk table cuts at the class boundary, which the profile summary states)."""
    chunks = lambda n: (n + 15) // 16
    cap_chunks = chunks(cap_cands) if cap_chunks is None else cap_chunks
    full_chunks = chunks(full_cands) if full_chunks is None else full_chunks
    per_cand = (measured - cap_chunks * ref_bytes) / cap_cands
    return per_cand * full_cands + full_chunks * ref_bytes


NCU_TRAFFIC_BYTES = {
    "cfg2": _scaled(2.181e9 + 3.8e6, 33554432, 64, 256, cap_chunks=1, full_chunks=1),   # profiles/dense_kernel_bf16_cfg2.md (reference stays in L2)
    "cfg3": _scaled(5.100e9 + 5.1e6, 268435456, 16, 32, cap_chunks=3, full_chunks=2),   # profiles/dense_kernel_f16_cfg3.md
    "cfg4": _scaled(4.563e9 + 4.1e6, 268435456, 16, 64),      # profiles/dense_kernel_i32_cfg4.md
    "cfg4w": _scaled(4.832e9 + 3.8e6, 536870912, 8, 64, cap_chunks=1, full_chunks=4),   # profiles/dense_kernel_i64_cfg4w.md
    "cfg5": (2.300e9 + 45.4e6) * 10000 / 2000,                # profiles/ragged_kernel_cfg5.md (2000 of 10000 tensors)
}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 100):
        self.gpu_index = gpu_index
        self.period_ms = period_ms
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", str(self.period_ms),
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
                pw.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def build_workload(name: str, device, cands: int = 0, tensors: int = 0):
    """``cands`` / ``tensors`` shrink the batch (fewer candidates, fewer ragged tensors) for small
    profiling captures; 0 keeps the full recipe."""
    from paper_2507_23194_b200 import workloads as W
    kw = {"n_cands": cands} if cands else {}
    if name == "cfg1":
        return W.config1(device)
    if name == "cfg2":
        return W.config2(device, **kw)
    if name == "cfg3":
        return W.config3(device, **kw)
    if name == "cfg4":
        return W.config4(device, **kw)
    if name == "cfg4w":
        return W.config4(device, wide=True, **kw)
    if name == "cfg5":
        return W.config5(device, **({"T": tensors} if tensors else {}))
    raise SystemExit(f"unknown workload {name}")


def host_bytes(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.uint8).cpu().numpy()


def host_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def time_oracle_sample(wl, budget_s: float = 15.0, threads: int = 1):
    """The oracle, as it stands, on as many whole candidates of the workload as fit the time budget (at
    least one per thread): one thread (the oracle is single-threaded), or one candidate per host thread.
    Returns (GB/s, description)."""
    from oracle import gv_oracle as O
    O.build()
    from paper_2507_23194_b200 import workloads as W
    if isinstance(wl, W.RaggedWorkload):
        # a prefix of the tensors, all four candidates each, split among the threads
        take = max(threads, wl.T // 64 * threads)
        take = min(take, wl.T)
        rb, cb = wl.ref_buf.cpu().numpy(), wl.cand_buf.cpu().numpy()
        ro_all, co_all = wl.ref_off.cpu().numpy(), wl.cand_off.cpu().numpy()
        dt_all, ne_all = wl.dtypes.cpu().numpy(), wl.n_elems_t.cpu().numpy()

        def part(i):
            ts = np.arange(i, take, threads)
            ro = np.concatenate([ro_all[ts], [0]])
            co = np.concatenate([co_all[t * wl.N:(t + 1) * wl.N] for t in ts])
            O.verify_ragged(rb, ro, cb, co, dt_all[ts], wl.N, wl.atol, wl.rtol, wl.equal_nan, n_elems=ne_all[ts])

        t0 = time.perf_counter()
        if threads == 1:
            part(0)
        else:
            with ThreadPoolExecutor(max_workers=threads) as ex:
                list(ex.map(part, range(threads)))
        dt_s = time.perf_counter() - t0
        nbytes = int(sum(int(n) * W.ELEM_SIZE[int(d)] for n, d in zip(ne_all[:take], dt_all[:take]))) * wl.N
        return nbytes / dt_s / 1e9, f"first {take} of {wl.T} tensors x {wl.N} candidates, {threads} thread(s)"
    ref = host_bytes(wl.ref)
    per = wl.n * W.ELEM_SIZE[wl.dtype]
    if threads == 1:
        done, spent = 0, 0.0
        for j in range(len(wl.cands)):
            c = host_bytes(wl.cands[j])
            t0 = time.perf_counter()
            O.verify(ref, c, wl.dtype, wl.atol, wl.rtol, wl.equal_nan)
            spent += time.perf_counter() - t0
            done += 1
            if spent > budget_s:
                break
        return done * per / spent / 1e9, f"first {done} of {len(wl.cands)} candidates, all {wl.n} elements each, 1 thread"
    # one candidate per thread, rounds of `threads` candidates until the budget is spent
    done, spent = 0, 0.0
    while done < len(wl.cands) and spent < budget_s:
        batch = [host_bytes(wl.cands[j]) for j in range(done, min(done + threads, len(wl.cands)))]
        t0 = time.perf_counter()
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda c: O.verify(ref, c, wl.dtype, wl.atol, wl.rtol, wl.equal_nan), batch))
        spent += time.perf_counter() - t0
        done += len(batch)
    return done * per / spent / 1e9, (f"first {done} of {len(wl.cands)} candidates, one per thread on {threads} threads "
                                      f"(sched_getaffinity)")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    device = "cuda:0" if torch.cuda.is_available() else "cpu"
    wl = build_workload(args.workload, device, args.cands, args.tensors)
    vals, sample = [], ""
    per_step_budget = max(2.0, min(15.0, 120.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        v, sample = time_oracle_sample(wl, per_step_budget)
        if i >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": None, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": dtype_name(wl), "data": "synthetic",
        "config": {"workload": wl.name, "note": "CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def dtype_name(wl) -> str:
    from paper_2507_23194_b200 import workloads as W
    if isinstance(wl, W.RaggedWorkload):
        return "mixed(f32,bf16,f16,i32)"
    return {0: "f32", 1: "bf16 widened to f32", 2: "f16 widened to f32", 3: "i32", 4: "i64"}[wl.dtype]


class Runner:
    """One workload bound to its output buffers: `step()` enqueues one whole verification."""

    def __init__(self, wl, device):
        from paper_2507_23194_b200 import gv, workloads as W
        self.gv, self.wl, self.device = gv, wl, device
        self.ragged = isinstance(wl, W.RaggedWorkload)
        if self.ragged:
            self.n_records = wl.T * wl.N
            self.res = torch.empty((self.n_records, 64), dtype=torch.uint8, device=device)
            self.ws = torch.empty(gv.gv_workspace_bytes(wl.T, wl.N), dtype=torch.uint8, device=device)
            self.launches_per_step = 3                                   # init, table pre-pass, verify
            self.ref_bytes = wl.cand_bytes // wl.N
            self.n_cands = wl.N
        else:
            self.n_cands = self.n_records = len(wl.cands)
            self.res = torch.empty((self.n_cands, 64), dtype=torch.uint8, device=device)
            self.ws = torch.empty(gv.gv_workspace_bytes(0, self.n_cands), dtype=torch.uint8, device=device)
            self.rh = torch.zeros(1, dtype=torch.int64, device=device)
            self.ptrs = (ctypes.c_void_p * max(1, self.n_cands))(*[c.data_ptr() for c in wl.cands])
            self.ref_bytes = wl.n * W.ELEM_SIZE[wl.dtype]
            full_tiles = self.ref_bytes // 512
            per_launch = [min(256, self.n_cands - j0) for j0 in range(0, self.n_cands, 256)]
            classify = sum(1 for m in per_launch if full_tiles >= 64 and full_tiles * 512 * m >= (64 << 20))
            self.launches_per_step = 1 + len(per_launch) + classify      # init + verify (+ sampling pass) per 256 candidates
        self.cand_bytes = wl.cand_bytes
        self.algo_bytes = self.cand_bytes + self.ref_bytes + 64 * self.n_records

    def step(self):
        wl, gv = self.wl, self.gv
        if self.ragged:
            gv.gv_verify_ragged(wl.ref_buf, wl.ref_off, wl.cand_buf, wl.cand_off, wl.dtypes, wl.N, wl.atol, wl.rtol,
                                wl.equal_nan, n_elems=wl.n_elems_t, results=self.res, workspace=self.ws)
        else:
            gv.gv_verify_batch(wl.ref, wl.cands, wl.atol, wl.rtol, wl.equal_nan, results=self.res, ref_hash=self.rh,
                               workspace=self.ws, cand_ptrs=self.ptrs)

    def check(self):
        if self.gv.gv_check(self.ws) != self.gv.GV_OK:
            raise SystemExit("device status word reports an error")

    def records(self) -> np.ndarray:
        return self.gv.results_to_numpy(self.res)

    def oracle_sample_equal(self, max_bytes: float = 1.5e9):
        """Records of a bounded sample (one candidate per recipe class while the byte budget lasts; a spread of
        ragged tensors) recomputed by the CPU oracle, one candidate per host thread -> (equal?, description)."""
        from oracle import gv_oracle as O
        O.build()
        wl, got = self.wl, self.records()
        threads = min(8, host_threads())
        if self.ragged:
            step = max(1, wl.T // 400)
            ts = np.arange(0, wl.T, step)
            rb, cb = wl.ref_buf.cpu().numpy(), wl.cand_buf.cpu().numpy()
            ro, co = wl.ref_off.cpu().numpy(), wl.cand_off.cpu().numpy()
            dt, ne = wl.dtypes.cpu().numpy(), wl.n_elems_t.cpu().numpy()

            def part(i):
                tt = ts[i::threads]
                if len(tt) == 0:
                    return True
                want = O.verify_ragged(rb, np.concatenate([ro[tt], [0]]), cb,
                                       np.concatenate([co[t * wl.N:(t + 1) * wl.N] for t in tt]), dt[tt], wl.N,
                                       wl.atol, wl.rtol, wl.equal_nan, n_elems=ne[tt])
                mine = np.concatenate([got[t * wl.N:(t + 1) * wl.N] for t in tt])
                return mine.tobytes() == want.tobytes()

            with ThreadPoolExecutor(max_workers=threads) as ex:
                ok = all(ex.map(part, range(threads)))
            return ok, f"every {step}th tensor ({len(ts)} of {wl.T}), all {wl.N} candidates each"
        per = self.ref_bytes
        seen, sample = set(), []
        for j, f in enumerate(wl.facts):
            key = f["class"] + str(f.get("sigma", "")) + str(f.get("frac", ""))
            if key not in seen and (len(sample) + 1) * per <= max(max_bytes, per):
                seen.add(key)
                sample.append(j)
        ref = host_bytes(wl.ref)

        def one(j):
            want = O.verify(ref, host_bytes(wl.cands[j]), wl.dtype, wl.atol, wl.rtol, wl.equal_nan)
            return got[j].tobytes() == want.tobytes()

        with ThreadPoolExecutor(max_workers=threads) as ex:
            ok = all(ex.map(one, sample))
        return ok, f"candidates {sample} (one per recipe class within {max_bytes / 1e9:.1f} GB), whole tensors"


def timed_steps(step, n_steps: int, stream):
    """Enqueue n_steps steps with a CUDA event after each (on the launch stream); returns per-step ms."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps + 1)]
    ev[0].record(stream)
    for i in range(n_steps):
        step()
        ev[i + 1].record(stream)
    torch.cuda.synchronize()
    return [ev[i].elapsed_time(ev[i + 1]) for i in range(n_steps)], ev[0].elapsed_time(ev[-1])


def measure_config(runner: Runner, stream, gpu_index: int, peak: float, target_s: float = 0.5, check_oracle: bool = True):
    """About `target_s` seconds of kernel time (20..400 steps) of one workload, with its own clock record."""
    for _ in range(3):
        runner.step()
    probe, _ = timed_steps(runner.step, 3, stream)
    est = max(1e-3, statistics.median(probe))
    n_steps = int(min(400, max(20, round(target_s * 1e3 / est))))
    sampler = ClockSampler(gpu_index, period_ms=50)
    sampler.start()
    time.sleep(0.2)
    step_ms, total_ms = timed_steps(runner.step, n_steps, stream)
    clocks = sampler.stop()
    runner.check()
    gbs = lambda ms: runner.cand_bytes / (ms * 1e-3) / 1e9
    med = statistics.median(step_ms)
    out = {
        "workload": runner.wl.name, "dtype": dtype_name(runner.wl), "candidates": runner.n_cands,
        "candidate_bytes_per_step": runner.cand_bytes, "steps": n_steps,
        "ms_per_step": total_ms / n_steps, "ms_per_step_median": med,
        "GB/s": gbs(total_ms / n_steps), "GB/s_first_20_steps": gbs(sum(step_ms[:20]) / min(20, n_steps)),
        "GB/s_median_step": gbs(med),
        "frac_of_measured_hbm": gbs(total_ms / n_steps) / peak,
        "roofline_frac": runner.algo_bytes / (total_ms / n_steps * 1e-3) / 1e9 / peak,
        "algorithmic_bytes_per_step": runner.algo_bytes,
        "l2": "inputs larger than L2" if runner.cand_bytes > (1 << 28) else "fits L2: not a bandwidth number",
        "clocks": clocks,
    }
    if runner.ragged:
        out["tensors_per_s"] = runner.wl.T / (total_ms / n_steps * 1e-3)
        out["tensors"] = runner.wl.T
    if check_oracle:
        ok, what = runner.oracle_sample_equal()
        out["records_equal_oracle"] = bool(ok)
        out["oracle_sample"] = what
    return out


def read_only_peak(device, stream, gv, nbytes: int = 8 << 30):
    """The read-only sum-reduction probe on a buffer much larger than L2: GB/s, median of 20 launches."""
    buf = torch.empty(nbytes // 8, dtype=torch.int64, device=device)
    buf.random_()
    out = torch.empty(1, dtype=torch.int64, device=device)
    for _ in range(3):
        gv.gv_selftest_read_sum(buf, out)
    ms, total = timed_steps(lambda: gv.gv_selftest_read_sum(buf, out), 20, stream)
    del buf
    return {"GB/s": nbytes / (statistics.median(ms) * 1e-3) / 1e9, "GB/s_mean": nbytes / (total / 20 * 1e-3) / 1e9,
            "bytes": nbytes, "kernel": "read_sum_kernel (128-bit streaming loads, integer adds)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--cands", type=int, default=0, help="fewer candidates than the recipe (profiling captures)")
    ap.add_argument("--tensors", type=int, default=0, help="fewer ragged tensors than the recipe (profiling captures)")
    ap.add_argument("--only-class", default="", help="keep only candidates of this recipe class (dense workloads)")
    ap.add_argument("--as-int32", action="store_true",
                    help="verify the same bytes in exact integer mode (tensors viewed as int32)")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "candidates"],
                    help="N > 1: every rank verifies its own full batch (default), or the candidate list of ONE "
                         "batch is split among the ranks (strong scaling; records gathered on every rank)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="headline only: no per-config / per-class blocks, no read-only probe, no follow-on stages")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    if args.impl == "reference":
        run_reference(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the verifier")
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device(device))

    from paper_2507_23194_b200 import gv, replicas as R, workloads as W
    small_case = bool(args.cands or args.tensors or args.only_class or args.as_int32)
    extras = (not args.no_extras) and world == 1 and args.workload == "cfg2" and not small_case
    wl = build_workload(args.workload, device, args.cands, args.tensors)
    ragged = isinstance(wl, W.RaggedWorkload)
    if args.only_class and not ragged:
        # a recipe class ("noise"), or a class with its parameter as the recipe records it ("rel_noise0.005", "swaps1e-05")
        keep = [j for j, f in enumerate(wl.facts)
                if args.only_class in (f["class"], f["class"] + str(f.get("sigma", "")) + str(f.get("frac", "")))]
        if not keep:
            raise SystemExit(f"no candidate of class {args.only_class!r} in {wl.name}")
        wl.cands = [wl.cands[j] for j in keep]
        wl.facts = [wl.facts[j] for j in keep]
        wl.name += ":" + args.only_class
    sharded = args.shard == "candidates" and world > 1 and not ragged
    shard_counts = None
    if sharded:
        # one batch, candidates split among the ranks; every rank holds the (seeded, identical) reference
        shard_counts, mine = R.shard_plan(len(wl.cands), world, rank)
        wl.cands = [wl.cands[j] for j in mine]
        wl.facts = [wl.facts[j] for j in mine]
        wl.name += f":shard{rank}of{world}"
        torch.cuda.empty_cache()
    if args.as_int32 and not ragged:
        wl.ref = wl.ref.view(torch.int32)
        wl.cands = [c.view(torch.int32) for c in wl.cands]
        wl.dtype = W.GV_I32
        wl.name += ":as_int32"

    stream = torch.cuda.current_stream()
    runner = Runner(wl, device)
    n_cands, cand_bytes, ref_bytes = runner.n_cands, runner.cand_bytes, runner.ref_bytes

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- the headline: W warm-up steps, then exactly K timed steps between barriers ----
    for _ in range(args.warmup):
        runner.step()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    ev[0].record(stream)
    for i in range(args.steps):
        runner.step()
        ev[i + 1].record(stream)
    barrier()
    total_ms = ev[0].elapsed_time(ev[-1])
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    clocks = sampler.stop() if rank == 0 else None
    runner.check()
    if dist is not None:
        total_ms = R.max_over_ranks(total_ms, device)
    ms_per_step = total_ms / args.steps
    job_bytes = world * cand_bytes
    if sharded:
        t = torch.tensor([cand_bytes], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        job_bytes = float(t.item())                       # the one batch, all shards
        all_records = R.gather_records(runner.res, shard_counts)
        if all_records.shape[0] != sum(shard_counts):
            raise SystemExit("gathered records do not cover the batch")
    value = job_bytes / (ms_per_step * 1e-3) / 1e9

    # ---- end to end through the host-buffer entry point (dense workloads) ----
    e2e = None
    if not args.no_e2e and not ragged:
        slab = min(n_cands, 32)
        staging = torch.empty(gv.gv_host_staging_bytes(wl.n, wl.dtype, slab), dtype=torch.uint8, device=device)
        href = wl.ref.cpu().pin_memory()
        hc = [c.cpu().pin_memory() for c in wl.cands]
        hres = np.zeros(n_cands, dtype=gv.RESULT_DTYPE)
        e2e_steps = max(1, min(args.steps, 5))
        gv.gv_verify_batch_host(href, hc, wl.atol, wl.rtol, wl.equal_nan, staging, results=hres)
        barrier()
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(e2e_steps):
            gv.gv_verify_batch_host(href, hc, wl.atol, wl.rtol, wl.equal_nan, staging, results=hres)
        t1.record(stream)
        barrier()
        e_ms = t0.elapsed_time(t1) / e2e_steps
        if dist is not None:
            e_ms = R.max_over_ranks(e_ms, device)
        same = hres.tobytes() == runner.records().tobytes()
        e2e = {"value": world * cand_bytes / (e_ms * 1e-3) / 1e9, "unit": "GB/s",
               "h2d_bytes_per_step": cand_bytes + ref_bytes, "d2h_bytes_per_step": 64 * n_cands + 8,
               "ms_per_step": e_ms, "steps": e2e_steps, "records_equal_device_path": bool(same),
               "api": "gv_verify_batch_host (pinned host buffers, slabs of %d candidates)" % slab}
        del staging, hc, href

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    algo_bytes = runner.algo_bytes
    achieved = algo_bytes / (ms_per_step * 1e-3) / 1e9
    first = step_ms[:20]
    roofline = {"bound": "hbm",
                "co_bound": {"kind": "alu", "peak_GB/s": {"f16": 5430.0, "bf16": 5640.0, "f32": 5800.0},
                             "what": "vectors identical to the reference stream at HBM rate; vectors that differ pay two splitmix64 "
                                     "evaluations and an fp32 compare per 16 bytes, whose arithmetic alone (registers only, 16 warps "
                                     "per SM) sustains these rates: profiles/compare_ceiling_b200.md"},
                "kernel": "ragged_kernel" if ragged else "dense_kernel",
                "achieved": achieved, "peak": peak, "peak_kind": peak_kind + " (STREAM-style copy)",
                "unit": "GB/s", "frac": achieved / peak, "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                "algorithmic_bytes_per_launch": algo_bytes,
                "achieved_first_20_steps": algo_bytes / (sum(first) / len(first) * 1e-3) / 1e9,
                "achieved_median_step": algo_bytes / (statistics.median(step_ms) * 1e-3) / 1e9,
                "note": "duration = CUDA-event span of the K timed steps / K on the launch stream (the same statistic as `value`; "
                        "each step = init, sampling and verify kernels); the first-20-steps and median-step figures show the "
                        "effect of the power cap on a long run"}

    cpu_baseline = None
    if not args.no_cpu_baseline:
        v, sample = time_oracle_sample(wl, 15.0)
        cpu_baseline = {"value": v, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample}
        if extras:
            nthr = host_threads()
            v_all, sample_all = time_oracle_sample(wl, 10.0, threads=nthr)
            cpu_baseline["all_cores"] = {"value": v_all, "unit": "GB/s", "cores": nthr, "sample": sample_all}

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "strong" if sharded else "weak",
        "vs_baseline": None, "dtype": dtype_name(wl), "data": "synthetic",
        "config": {"workload": wl.name, "candidates": n_cands, "candidate_bytes_per_step": cand_bytes,
                   "reference_bytes": ref_bytes, "atol": wl.atol, "rtol": wl.rtol, "equal_nan": wl.equal_nan,
                   "l2": "inputs larger than L2 (no flush needed)" if cand_bytes > (1 << 28) else "fits L2: not a bandwidth number",
                   "parallelism": ("one batch, candidates split over the GPUs, records gathered" if sharded else
                                   "independent replicas per GPU") if world > 1 else "one GPU"},
        "frac_of_measured_hbm": value / world / peak, "frac_of_nominal_8000": value / world / 8000.0,
        "clocks": clocks, "e2e": e2e, "gpu_launches": runner.launches_per_step * args.steps,
        "roofline": roofline, "cpu_baseline": cpu_baseline,
    }

    if extras:
        # ---- read-only bandwidth beside the copy peak ----
        ro = read_only_peak(device, stream, gv)
        roofline["peak_read_only"] = ro["GB/s"]
        roofline["peak_read_only_detail"] = ro
        roofline["frac_of_read_only"] = achieved / ro["GB/s"]

        # ---- the headline workload by candidate class (so that the aggregate is not flattered by copies) ----
        per_class = {}
        for cls in sorted({f["class"] for f in wl.facts}):
            keep = [j for j, f in enumerate(wl.facts) if f["class"] == cls]
            sub = W.DenseWorkload(name=wl.name + ":" + cls, dtype=wl.dtype, ref=wl.ref, cands=[wl.cands[j] for j in keep],
                                  atol=wl.atol, rtol=wl.rtol, equal_nan=wl.equal_nan, facts=[wl.facts[j] for j in keep])
            r = measure_config(Runner(sub, device), stream, local_rank, peak, target_s=0.3, check_oracle=False)
            r["frac_of_read_only"] = r["GB/s"] / ro["GB/s"]
            per_class[cls] = r
        line["per_class"] = per_class

        # ---- the content hash as a call of its own (every byte hashed: arithmetic-bound, not a copy) ----
        line["hash"] = bench_hash(gv, stream, device, peak)

        # ---- follow-on stages on the headline's records (outside the timed step) ----
        line["grouping"] = bench_grouping(gv, runner, stream, device, not args.no_cpu_baseline)
        line["error_profile"] = bench_error_profile(gv, wl, stream, device, peak)

        # ---- every workload of the recipe (the headline's first, while its tensors are still resident) ----
        per_config = {}
        del runner
        for name in ["cfg2"] + [w for w in ALL_WORKLOADS if w != "cfg2"]:
            if name != "cfg2":
                wl = None
                torch.cuda.empty_cache()
                wl = build_workload(name, device)
            r = measure_config(Runner(wl, device), stream, local_rank, peak, target_s=0.5)
            r["frac_of_read_only"] = r["GB/s"] / ro["GB/s"]
            r["traffic"] = NCU_TRAFFIC_BYTES.get(name)
            per_config[name] = r
        per_config = {k: per_config[k] for k in ALL_WORKLOADS}
        line["per_config"] = per_config
        line["fits_in_driver_run"] = True

    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def bench_hash(gv, stream, device, peak):
    out = {}
    buf = torch.empty((2 << 30) // 8, dtype=torch.int64, device=device)
    buf.random_()
    h = torch.empty(1, dtype=torch.int64, device=device)
    for label, n_words in (("256MiB", (256 << 20) // 8), ("2GiB", (2 << 30) // 8)):
        view = buf[:n_words]
        for name, fn in (("gv_hash", gv.gv_hash), ("gv_hash2", gv.gv_hash2)):
            for _ in range(3):
                fn(view, h)
            ms, _ = timed_steps(lambda: fn(view, h), 10, stream)
            gbs = n_words * 8 / (statistics.median(ms) * 1e-3) / 1e9
            out[f"{name}_{label}"] = {"GB/s": gbs, "frac_of_measured_hbm": gbs / peak}
    out["note"] = ("two splitmix64 evaluations per 16 bytes on every byte; the 256 MiB buffer is not much larger than L2 and a call "
                   "is a memset plus one launch")
    del buf
    return out


def bench_grouping(gv, runner, stream, device, with_oracle: bool):
    res = runner.res
    n_rec = res.shape[0]
    gws = torch.empty(gv.gv_group_workspace_bytes(n_rec), dtype=torch.uint8, device=device)
    gid = torch.empty(max(n_rec, 1), dtype=torch.int32, device=device)
    gcnt = torch.empty(max(n_rec, 1), dtype=torch.int32, device=device)
    gn = torch.empty(1, dtype=torch.int32, device=device)
    call = lambda: gv.gv_group_candidates(res, gid, gcnt, gn, gws)
    for _ in range(3):
        call()
    ms, _ = timed_steps(call, 20, stream)
    out = {"records": n_rec, "groups": int(gn.cpu()[0]), "us_per_call": 1e3 * statistics.median(ms),
           "launches_per_call": 1 if n_rec <= 2048 else 3}
    if with_oracle:
        from oracle import gv_oracle as O
        rec_np = gv.results_to_numpy(res)[:min(n_rec, 4096)]
        t0 = time.perf_counter()
        O.group(rec_np)
        out["cpu_oracle_us"] = 1e6 * (time.perf_counter() - t0)
        out["cpu_oracle_records"] = int(rec_np.shape[0])
    return out


def bench_error_profile(gv, wl, stream, device, peak):
    from paper_2507_23194_b200 import workloads as W
    j_bad = next((j for j, f in enumerate(wl.facts) if f["class"] != "copy"), 0)
    pws = torch.empty(gv.gv_profile_workspace_bytes(), dtype=torch.uint8, device=device)
    pout = torch.empty(gv.PROFILE_DTYPE.itemsize, dtype=torch.uint8, device=device)
    prow = torch.empty((wl.n + 4095) // 4096, dtype=torch.int32, device=device)
    call = lambda: gv.gv_error_profile(wl.ref, wl.cands[j_bad], wl.atol, wl.rtol, wl.equal_nan, 4096, pout, prow, pws)
    for _ in range(3):
        call()
    ms, _ = timed_steps(call, 10, stream)
    p_ms = statistics.median(ms)
    pbytes = 2 * wl.n * W.ELEM_SIZE[wl.dtype]
    return {"candidate": j_bad, "class": wl.facts[j_bad]["class"], "us_per_call": 1e3 * p_ms,
            "bytes_read": pbytes, "GB/s": pbytes / (p_ms * 1e-3) / 1e9,
            "frac_of_measured_hbm": pbytes / (p_ms * 1e-3) / 1e9 / peak,
            "note": "one candidate + the reference, both read once; fits L2 when the pair is below 126 MB"}


if __name__ == "__main__":
    main()
