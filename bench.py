"""Benchmark of the MMEE search path: candidate mappings evaluated per second on B200.

A step is one pass of the whole hot path over one workload: for each search of the workload the plan
is decoded, every mapping's cost bounded or evaluated, capacity-pruned and reduced to the optimum on
the device, in one kernel launch per search.  The default workload is the largest single-GPU
configuration: grouped-query attention (batch 4, 32 query heads on 8 KV heads, S = 8192, d = 128) on
the cloud accelerator, latency-driven then energy-delay-product-driven, 3.39e9 mappings per search.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints one JSON line.  With N > 1 (under torchrun) every rank runs an independent replica on its
own GPU: the search is launched per workload and does not shard in this build.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import mmee_inputs as mi  # noqa: E402

METRIC = "candidate mappings evaluated/sec"
UNIT = "candidates/s"
OBJ_NAMES = {0: "energy", 1: "latency", 2: "edp", 3: "energy_lcap", 4: "latency_ecap"}

# Algorithmic work of the search kernels, per TESTED ROW (a row is the nine mappings that share tiling, order
# and buffering levels; the kernel reports how many rows it tested, the others lay in tilings, middle levels
# or groups that a coarser capacity test showed not to fit).  The least key of a row's nine mappings is its
# row sum plus the least stationary-pair term, which is taken once per tiling, so a row needs one test.
# Energy / latency, in thread-level 32-bit integer instructions: capacity difference of Eq. (4), its sign mask,
# the feasible count, the masked row term, and 2/5 of a three-input minimum (five rows share two).
# Energy-delay product: two capacity compares, their AND, the feasible count, and the single-precision row
# bound (two adds, a max, a multiply, a compare, the predicate merge).
ALG_OPS_PER_ROW = {0: 4.4, 1: 4.4, 2: 10.0}
LANES_PER_SM = 64          # 4 sub-partitions x 16 lanes: width of the integer-ALU pipe, the busiest pipe of these kernels
# dram__bytes_read.sum + dram__bytes_write.sum per launch, recorded from the ncu captures summarised under
# profiles/ (not measured in this run); workload -> objective -> bytes.  None where no capture backs it.
NCU_DRAM_BYTES_PER_LAUNCH = {"gqa": {1: 199680, 2: 193024}, "llama": {0: 207360, 1: 198400},
                             "bert": {0: 182272, 1: 201216}}


WORKLOADS = {"tiny": mi.config1, "bert": mi.config2, "llama": mi.config3, "gqa": mi.config4}


def workload_jobs(name):
    """(workload name, [(problem, search), ...]): one step runs every listed search once.
    The default, "gqa", is the largest single-GPU configuration; "sweep" is the 28-point
    sequence-length sweep (one energy search per point)."""
    if name == "sweep":
        pts = mi.config5()
        return "sweep_s1k_to_64k", [(c, c["searches"][0]) for c in pts]
    if name == "ffn":
        pts = mi.ffn_dram_sweep_configs()
        return "ffn_gpt3_dram_vs_buffer", [(c, c["searches"][0]) for c in pts]
    if name == "beyond":
        pts = mi.beyond_attention_configs()
        return "two_gemm_and_conv_chains", [(c, c["searches"][0]) for c in pts]
    if name == "reconfig":
        cfg, _ = mi.reconfigurable_array_designs()
        return "reconfigurable_arrays_" + cfg["name"], [(cfg, cfg["searches"][0])]
    cfg = WORKLOADS[name]()
    return cfg["name"], [(cfg, s) for s in cfg["searches"]]


class ClockSampler:
    """nvidia-smi clocks / throttle reasons of one GPU, sampled every 200 ms in the background."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.25)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t0 - 0.2 <= t <= t1 + 0.2] or [r for _, r in self.rows]
        sm, mx, reasons = [], [], set()
        for r in rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def cpu_baseline(cfg, obj, budget_s: float = 12.0):
    """The oracle as it stands on the host cores, on a bounded tiling sub-range of the workload; then the same
    on one core, on a quarter-size budget."""
    import oracle
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    probe = max(1, min(p.T, 40))
    t0 = time.perf_counter()
    oracle.search(oracle.make_problem(cfg["workload"], cfg["arch"], dict(obj, t_begin=0, t_end=probe)))
    rate = probe / max(time.perf_counter() - t0, 1e-6)
    n_t = int(max(probe, min(p.T, rate * budget_s)))
    lo = (p.T - n_t) // 2
    q = oracle.make_problem(cfg["workload"], cfg["arch"], dict(obj, t_begin=lo, t_end=lo + n_t))
    t0 = time.perf_counter()
    res = oracle.search(q)
    dt = time.perf_counter() - t0
    cores = oracle.threads_used()
    n_1 = max(1, int(n_t / max(cores, 1) / 4))
    q1 = oracle.make_problem(cfg["workload"], cfg["arch"], dict(obj, t_begin=lo, t_end=lo + n_1))
    t0 = time.perf_counter()
    res1 = oracle.search(q1, threads=1)
    dt1 = time.perf_counter() - t0
    return dict(value=res.n_total / dt, unit=UNIT, cores=cores, kind="oracle",
                sample="%s objective, tilings [%d,%d) of %d (%d mappings, %.1f s)" %
                       (OBJ_NAMES[obj["objective"]], lo, lo + n_t, p.T, res.n_total, dt),
                one_core=dict(value=res1.n_total / dt1, unit=UNIT, cores=1,
                              sample="tilings [%d,%d) (%d mappings, %.1f s)" % (lo, lo + n_1, res1.n_total, dt1)))


def run_reference(args, rank):
    """The CPU oracle as the reference arm: each step a bounded sample of the same workload."""
    if rank != 0:
        return
    import oracle
    wname, jobs = workload_jobs(args.workload)
    cfg, obj = jobs[0]
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    n_t = max(1, min(p.T, 24))
    stride = max(1, (p.T - n_t) // max(1, args.steps + args.warmup))
    done, t_total = 0, 0.0
    for step in range(args.warmup + args.steps):
        lo = min(p.T - n_t, step * stride)
        q = oracle.make_problem(cfg["workload"], cfg["arch"], dict(obj, t_begin=lo, t_end=lo + n_t))
        t0 = time.perf_counter()
        res = oracle.search(q)
        dt = time.perf_counter() - t0
        if step >= args.warmup:
            done += res.n_total
            t_total += dt
    value = done / t_total
    sample = "%d tilings of %d per step, %s objective" % (n_t, p.T, OBJ_NAMES[obj["objective"]])
    print(json.dumps(dict(
        impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
        warmup=args.warmup, ms_per_step=1e3 * t_total / args.steps, higher_is_better=True, scaling="weak",
        vs_baseline=None, dtype="int64", data="synthetic",
        config=dict(workload=wname, note="CPU oracle on host cores; " + sample),
        cpu_baseline=dict(value=value, unit=UNIT, cores=oracle.threads_used(), kind="oracle", sample=sample),
        e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))))


def run_reconfig(args):
    """EDP-driven search over the four array designs of the reconfigurable-array comparison: one search per
    logical shape through mmee_search_shapes, host wall clock per design."""
    import torch
    import paper_2604_03446_b200 as mm
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    cfg, designs = mi.reconfigurable_array_designs()
    out, total_ms, total_cand = [], 0.0, 0
    for name, mask, shapes in designs:
        obj = dict(cfg["searches"][0], stationary_mask=mask)
        mm.mmee_search_shapes(cfg["workload"], cfg["arch"], obj, shapes)          # warm-up
        t0 = time.perf_counter()
        per_shape, best = mm.mmee_search_shapes(cfg["workload"], cfg["arch"], obj, shapes)
        ms = 1e3 * (time.perf_counter() - t0)
        r = per_shape[best]
        total_ms += ms
        total_cand += sum(p.n_total for p in per_shape)
        out.append(dict(design=name, shapes=len(shapes), best_shape=list(shapes[best]), edp_key=r.edp_key,
                        energy_pj=r.energy_pj, latency_cycles=r.latency_cycles, sm=list(r.sm), idx=r.idx, ms=ms))
    print(json.dumps(dict(metric=METRIC, value=total_cand / (total_ms * 1e-3), unit=UNIT, n_gpus=1, steps=1, warmup=1,
                          ms_per_step=total_ms, higher_is_better=True, scaling="weak", vs_baseline=None,
                          dtype="f64", data="synthetic",
                          config=dict(workload="reconfigurable_arrays_" + cfg["name"],
                                      note="host wall clock of mmee_search_shapes (plan + search + copy per shape)"),
                          designs=out)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="gqa", choices=sorted(WORKLOADS) + ["sweep", "ffn", "beyond", "reconfig"])
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.workload == "reconfig":
        if rank == 0:
            run_reconfig(args)
        return

    import torch
    import torch.distributed as dist
    import paper_2604_03446_b200 as mm

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    wname, jobs = workload_jobs(args.workload)
    searches = [s for _, s in jobs]
    handles = [mm.mmee_create(c["workload"], c["arch"], s) for c, s in jobs]
    for h in handles:
        mm.mmee_kernel_timing(h, True)
    outs = [(mm.result_buffer(1), mm.result_buffer(s["topk"])) for s in searches]
    n_cand = [(s, mm.mmee_num_candidates(h)) for s, h in zip(searches, handles)]
    cand_per_step = sum(n for _, n in n_cand)

    peaks = mm.mmee_alu_peak()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")   # larger than the 126 MB L2

    def one_step(timed):
        flush.fill_(1)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for h, (b, t) in zip(handles, outs):
            mm.mmee_search(h, b, t)
        ev1.record()
        torch.cuda.synchronize()
        if not timed:
            return None
        return ev0.elapsed_time(ev1), [mm.mmee_last_search_stats(h).search_ms for h in handles]

    for _ in range(args.warmup):
        one_step(False)

    sampler = ClockSampler(local_rank)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t_start = time.time()
    step_ms, kernel_ms = [], []
    for _ in range(args.steps):
        ms, ks = one_step(True)
        step_ms.append(ms)
        kernel_ms.append(ks)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t_end = time.time()
    clocks = sampler.stop(t_start, t_end)

    total_ms = sum(step_ms)
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())

    # parity of what was timed is the tests' job; here only the counters of the last step
    bests = [mm.read_results(b, 1)[0] for b, _ in outs]
    stats = [mm.mmee_last_search_stats(h) for h in handles]
    check_failures = sum(1 for b in bests if b.status == mm.ERR_CHECK)

    # time to optimum per search: host wall clock of mmee_search_host on the warm handle (launch, device
    # search, copy of the optimum record to host memory)
    tto_ms = []
    for h in handles:
        samples = []
        for _ in range(21):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            mm.mmee_search_host(h)
            samples.append(1e3 * (time.perf_counter() - t0))
        tto_ms.append(statistics.median(samples))

    # offline symbolic row pruning (single-optimum searches only): same optimum, fewer rows evaluated
    pruning = []
    for i, (c, s) in enumerate(jobs):
        if s["topk"] != 1 or len(jobs) > 4:
            continue
        hp = mm.mmee_create(c["workload"], c["arch"], dict(s, row_pruning=1))
        mm.mmee_kernel_timing(hp, True)
        bp = mm.result_buffer(1)
        ms = []
        for _ in range(13):
            mm.mmee_search(hp, bp, None)
            torch.cuda.synchronize()
            ms.append(mm.mmee_last_search_stats(hp).search_ms)
        st = mm.mmee_last_search_stats(hp)
        got = mm.read_results(bp, 1)[0]
        pruning.append(dict(problem=c["name"], objective=OBJ_NAMES[s["objective"]],
                            rows=st.rows_per_tiling, rows_kept=st.rows_evaluated_per_tiling,
                            kernel_ms=statistics.median(ms[3:]), same_optimum=bool(got.idx == bests[i].idx),
                            optimum=dict(idx=got.idx, bs_words=got.bs, dram_words=got.n[0],
                                         energy_pj=got.energy_pj, latency_cycles=got.latency_cycles)))
        mm.mmee_destroy(hp)

    # end to end through the host-buffer entry point: plan, allocate, launch, copy back, release, every step
    e2e_steps = max(3, min(args.steps, 30))
    h2d = d2h = 0
    for _ in range(2):
        for c, s in jobs:
            mm.mmee_solve_host(c["workload"], c["arch"], s)
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        h2d = d2h = 0
        for c, s in jobs:
            _, _, a, b = mm.mmee_solve_host(c["workload"], c["arch"], s)
            h2d += a
            d2h += b
    e2e_s = time.perf_counter() - t0
    if world > 1:
        t = torch.tensor([e2e_s], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())

    for h in handles:
        mm.mmee_destroy(h)

    if rank == 0:
        sm_mhz = clocks.get("sm_mhz") or peaks[3]
        n_sm = torch.cuda.get_device_properties(local_rank).multi_processor_count
        peak = n_sm * LANES_PER_SM * sm_mhz * 1e6 / 1e9
        per_kernel = []
        for i, (s, n) in enumerate(n_cand):
            ks = [k[i] for k in kernel_ms]
            sm = statistics.mean(ks)
            ops = stats[i].rows_tested * ALG_OPS_PER_ROW.get(s["objective"], 10.0)
            per_kernel.append(dict(
                kernel="search_kernel<%s>" % OBJ_NAMES[s["objective"]], objective=s["objective"], problem=jobs[i][0]["name"],
                avg_ms=sm, median_ms=statistics.median(ks), max_ms=max(ks), create_ms=stats[i].create_ms,
                candidates=n, feasible=bests[i].n_feasible, pruned_fraction=1.0 - bests[i].n_feasible / n,
                rows_tested=stats[i].rows_tested, rows_total=n // 9, exact_path_visits=stats[i].exact_path_visits,
                time_to_optimum_ms=tto_ms[i], candidates_per_s=n / (sm * 1e-3),
                evaluated_per_s=9 * stats[i].rows_tested / (sm * 1e-3),
                achieved_gops=ops / (sm * 1e-3) / 1e9, frac=ops / (sm * 1e-3) / 1e9 / peak))
        dom = max(per_kernel, key=lambda k: k["avg_ms"])
        traffic = NCU_DRAM_BYTES_PER_LAUNCH.get(args.workload, {}).get(dom["objective"])
        roofline = dict(bound="alu", kernel=dom["kernel"], achieved=dom["achieved_gops"], peak=peak,
                        unit="Gop/s (thread-level 32-bit instructions of the row tests)", frac=dom["achieved_gops"] / peak,
                        traffic=traffic,
                        traffic_note=("recorded from the ncu capture under profiles/, not measured in this run"
                                      if traffic is not None else "no capture of this kernel on this workload"),
                        peak_source="%d SMs x %d lanes of the integer-ALU pipe x %.0f MHz (clock sampled during the run)" %
                                    (n_sm, LANES_PER_SM, sm_mhz),
                        ops_per_tested_row=ALG_OPS_PER_ROW.get(dom["objective"], 10.0),
                        measured_rates_gops=dict(logic=peaks[0], add_logic=peaks[1], key_mix=peaks[2],
                                                 sm_mhz=peaks[3]))
        line = dict(
            metric=METRIC, value=world * cand_per_step * args.steps / (total_ms * 1e-3), unit=UNIT,
            n_gpus=world, steps=args.steps, warmup=args.warmup, ms_per_step=total_ms / args.steps,
            higher_is_better=True, scaling="weak", vs_baseline=None, dtype="int64", data="synthetic",
            config=dict(workload=wname, searches=[OBJ_NAMES[s["objective"]] for s in searches],
                        candidates_per_step=cand_per_step, parallelism="replicas only",
                        l2="flushed between steps (256 MB write); the path reads no HBM-resident input",
                        grid=stats[0].grid, block=stats[0].block, smem_bytes=stats[0].smem_bytes),
            clocks=clocks, gpu_launches=len(searches) * args.steps, check_failures=check_failures,
            e2e=dict(value=world * cand_per_step * e2e_steps / e2e_s, unit=UNIT, h2d_bytes_per_step=h2d,
                     d2h_bytes_per_step=d2h, ms_per_step=1e3 * e2e_s / e2e_steps,
                     note="mmee_solve_host: plan + allocate + launch + result copy to host buffers + release, host wall clock"),
            time_to_optimum_ms=tto_ms, create_ms=[k["create_ms"] for k in per_kernel],
            kernels=per_kernel, roofline=roofline, row_pruning=pruning)
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(*jobs[0])
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
