#!/usr/bin/env python
"""Benchmark of the batched output verifier: GB/s of candidate outputs verified.

One "step" is one pass of the whole hot path (result init + the fused verify kernel) over one batch
of synthetic candidates: by default the dense bf16 workload (a 4096x4096 reference, 256 candidates,
8 GiB of candidate data per step, far larger than L2, so no cache flush is needed between steps).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3|cfg4|cfg4w|cfg5|cfg1]
    python bench.py --impl reference ...     # the CPU oracle on a bounded sample, for context

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

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "GB/s of candidate outputs verified (fraction of B200 HBM peak)"
FALLBACK_HBM_GBS = 6650.0

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
    "cfg2": _scaled(2.181e9 + 4.3e6, 33554432, 64, 256, cap_chunks=1, full_chunks=1),   # profiles/dense_kernel_bf16_cfg2.md (reference stays in L2)
    "cfg3": _scaled(5.100e9 + 4.1e6, 268435456, 16, 32, cap_chunks=3, full_chunks=2),   # profiles/dense_kernel_f16_cfg3.md
    "cfg4": _scaled(4.564e9 + 5.1e6, 268435456, 16, 64),      # profiles/dense_kernel_i32_cfg4.md
    "cfg5": (2.292e9 + 11.1e6) * 10000 / 2000,                # profiles/ragged_kernel_cfg5.md (2000 of 10000 tensors)
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

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
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
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


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


def time_oracle_sample(wl, budget_s: float = 15.0):
    """The oracle, as it stands, single-threaded, on as many whole candidates of the workload as
    fit the time budget (at least one). Returns (GB/s, description)."""
    from oracle import gv_oracle as O
    O.build()
    from paper_2507_23194_b200 import workloads as W
    if isinstance(wl, W.RaggedWorkload):
        # a prefix of the tensors, all four candidates each
        take = max(1, wl.T // 64)
        ro, co = wl.ref_off[:take + 1].cpu().numpy(), wl.cand_off[:take * wl.N].cpu().numpy()
        rb, cb = wl.ref_buf.cpu().numpy(), wl.cand_buf.cpu().numpy()
        dt, ne = wl.dtypes[:take].cpu().numpy(), wl.n_elems_t[:take].cpu().numpy()
        t0 = time.perf_counter()
        O.verify_ragged(rb, ro, cb, co, dt, wl.N, wl.atol, wl.rtol, wl.equal_nan, n_elems=ne)
        dt_s = time.perf_counter() - t0
        nbytes = int(sum(int(n) * W.ELEM_SIZE[int(d)] for n, d in zip(ne, dt))) * wl.N
        return nbytes / dt_s / 1e9, f"first {take} of {wl.T} tensors x {wl.N} candidates"
    ref = host_bytes(wl.ref)
    per = wl.n * W.ELEM_SIZE[wl.dtype]
    done, spent = 0, 0.0
    for j in range(len(wl.cands)):
        c = host_bytes(wl.cands[j])
        t0 = time.perf_counter()
        O.verify(ref, c, wl.dtype, wl.atol, wl.rtol, wl.equal_nan)
        spent += time.perf_counter() - t0
        done += 1
        if spent > budget_s:
            break
    return done * per / spent / 1e9, f"first {done} of {len(wl.cands)} candidates, all {wl.n} elements each"


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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
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

    from paper_2507_23194_b200 import gv, workloads as W
    wl = build_workload(args.workload, device, args.cands, args.tensors)
    ragged = isinstance(wl, W.RaggedWorkload)
    if args.only_class and not ragged:
        keep = [j for j, f in enumerate(wl.facts) if f["class"] == args.only_class]
        wl.cands = [wl.cands[j] for j in keep]
        wl.facts = [wl.facts[j] for j in keep]
        wl.name += ":" + args.only_class
    sharded = args.shard == "candidates" and world > 1 and not ragged
    shard_counts = None
    if sharded:
        # one batch, candidates split among the ranks; every rank holds the (seeded, identical) reference
        from paper_2507_23194_b200 import replicas as R
        n_all = len(wl.cands)
        shard_counts = [len(R.shard_candidates(n_all, world, r)) for r in range(world)]
        mine = R.shard_candidates(n_all, world, rank)
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
    if ragged:
        count = wl.T * wl.N
        res = torch.empty((count, 64), dtype=torch.uint8, device=device)
        ws = torch.empty(gv.gv_workspace_bytes(wl.T, wl.N), dtype=torch.uint8, device=device)

        def step():
            gv.gv_verify_ragged(wl.ref_buf, wl.ref_off, wl.cand_buf, wl.cand_off, wl.dtypes, wl.N, wl.atol,
                                wl.rtol, wl.equal_nan, n_elems=wl.n_elems_t, results=res, workspace=ws)
        launches_per_step = 3
        ref_bytes = wl.cand_bytes // wl.N
        n_cands = wl.N
    else:
        n_cands = len(wl.cands)
        res = torch.empty((n_cands, 64), dtype=torch.uint8, device=device)
        ws = torch.empty(gv.gv_workspace_bytes(0, n_cands), dtype=torch.uint8, device=device)
        rh = torch.zeros(1, dtype=torch.int64, device=device)
        ptrs = (ctypes.c_void_p * n_cands)(*[c.data_ptr() for c in wl.cands])

        def step():
            gv.gv_verify_batch(wl.ref, wl.cands, wl.atol, wl.rtol, wl.equal_nan, results=res, ref_hash=rh,
                               workspace=ws, cand_ptrs=ptrs)
        launches_per_step = 1 + 2 * ((n_cands + 255) // 256)      # init + (classify + verify) per 256 candidates
        ref_bytes = wl.n * W.ELEM_SIZE[wl.dtype]
    cand_bytes = wl.cand_bytes

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    ev[0].record(stream)
    for i in range(args.steps):
        step()
        ev[i + 1].record(stream)
    barrier()
    total_ms = ev[0].elapsed_time(ev[-1])
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    clocks = sampler.stop() if rank == 0 else None
    if gv.gv_check(ws) != gv.GV_OK:
        raise SystemExit("device status word reports an error")
    if dist is not None:
        t = torch.tensor([total_ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    job_bytes = world * cand_bytes
    if sharded:
        t = torch.tensor([cand_bytes], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        job_bytes = float(t.item())                       # the one batch, all shards
        from paper_2507_23194_b200 import replicas as R
        all_records = R.gather_records(res, shard_counts)
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
            t = torch.tensor([e_ms], dtype=torch.float64, device=device)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e_ms = float(t.item())
        same = hres.tobytes() == gv.results_to_numpy(res).tobytes()
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
    algo_bytes = cand_bytes + ref_bytes + 64 * (wl.T * wl.N if ragged else n_cands)
    kernel_ms = statistics.median(step_ms)
    achieved = algo_bytes / (kernel_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "co_bound": "alu (vectors identical to the reference stream at HBM rate; vectors that differ pay the integer work of the content hash, about 7.3 TB/s for the hash alone, and the compare: see profiles/instruction_rates_b200.md)",
                "kernel": "ragged_kernel" if ragged else "dense_kernel",
                "achieved": achieved, "peak": peak, "peak_kind": peak_kind + " (STREAM-style copy)",
                "unit": "GB/s", "frac": achieved / peak, "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                "algorithmic_bytes_per_launch": algo_bytes,
                "note": "duration = median CUDA-event time of one call (init, classify and verify kernels) on the launch stream"}

    cpu_baseline = None
    if not args.no_cpu_baseline:
        v, sample = time_oracle_sample(wl, 15.0)
        cpu_baseline = {"value": v, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample}

    # ---- duplicate groups of the step's records (follow-on stage; outside the timed step) ----
    n_rec = res.shape[0]
    gws = torch.empty(gv.gv_group_workspace_bytes(n_rec), dtype=torch.uint8, device=device)
    gid = torch.empty(max(n_rec, 1), dtype=torch.int32, device=device)
    gcnt = torch.empty(max(n_rec, 1), dtype=torch.int32, device=device)
    gn = torch.empty(1, dtype=torch.int32, device=device)
    for _ in range(3):
        gv.gv_group_candidates(res, gid, gcnt, gn, gws)
    torch.cuda.synchronize()
    g_ev = [torch.cuda.Event(enable_timing=True) for _ in range(21)]
    g_ev[0].record(stream)
    for i in range(20):
        gv.gv_group_candidates(res, gid, gcnt, gn, gws)
        g_ev[i + 1].record(stream)
    torch.cuda.synchronize()
    grouping = {"records": n_rec, "groups": int(gn.cpu()[0]),
                "us_per_call": 1e3 * statistics.median(g_ev[i].elapsed_time(g_ev[i + 1]) for i in range(20)),
                "launches_per_call": 1 if n_rec <= 2048 else 3}
    if not args.no_cpu_baseline:
        from oracle import gv_oracle as O
        rec_np = gv.results_to_numpy(res)[:min(n_rec, 4096)]
        t0 = time.perf_counter()
        O.group(rec_np)
        grouping["cpu_oracle_us"] = 1e6 * (time.perf_counter() - t0)
        grouping["cpu_oracle_records"] = int(rec_np.shape[0])

    # ---- error profile of one failing candidate (follow-on stage; outside the timed step) ----
    error_profile = None
    if not ragged:
        j_bad = next((j for j, f in enumerate(wl.facts) if f["class"] != "copy"), 0)
        pws = torch.empty(gv.gv_profile_workspace_bytes(), dtype=torch.uint8, device=device)
        pout = torch.empty(gv.PROFILE_DTYPE.itemsize, dtype=torch.uint8, device=device)
        prow = torch.empty((wl.n + 4095) // 4096, dtype=torch.int32, device=device)
        for _ in range(3):
            gv.gv_error_profile(wl.ref, wl.cands[j_bad], wl.atol, wl.rtol, wl.equal_nan, 4096, pout, prow, pws)
        torch.cuda.synchronize()
        p_ev = [torch.cuda.Event(enable_timing=True) for _ in range(11)]
        p_ev[0].record(stream)
        for i in range(10):
            gv.gv_error_profile(wl.ref, wl.cands[j_bad], wl.atol, wl.rtol, wl.equal_nan, 4096, pout, prow, pws)
            p_ev[i + 1].record(stream)
        torch.cuda.synchronize()
        p_ms = statistics.median(p_ev[i].elapsed_time(p_ev[i + 1]) for i in range(10))
        pbytes = 2 * wl.n * W.ELEM_SIZE[wl.dtype]
        error_profile = {"candidate": j_bad, "class": wl.facts[j_bad]["class"], "us_per_call": 1e3 * p_ms,
                         "bytes_read": pbytes, "GB/s": pbytes / (p_ms * 1e-3) / 1e9,
                         "frac_of_measured_hbm": pbytes / (p_ms * 1e-3) / 1e9 / peak,
                         "note": "one candidate + the reference, both read once; fits L2 when the pair is below 126 MB"}

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
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline, "cpu_baseline": cpu_baseline, "grouping": grouping,
        "error_profile": error_profile,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
