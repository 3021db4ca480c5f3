#!/usr/bin/env python
"""Benchmark of the planner hot path: candidate plans evaluated per second.

One step = one pass of the whole hot path over the workload's candidate space: layer costs
(Eq. 2 / Eq. 3) for every configuration, the pipeline dynamic program for every candidate
(no pruning), and the (cost, index) argmin.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload stress] [--impl reference]

With N > 1 (launched by torch.distributed.run) the candidate space is sharded over the ranks
in contiguous, work-balanced ranges and the ranks exchange one (cost, index) pair per step.
`--impl reference` times the CPU oracle (as it stands) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "candidate_plans_per_second"
UNIT = "candidates/s"
SM_COUNT, SCHEDULERS_PER_SM, LANES = 148, 4, 32
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0}

def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower() == "active":
                        reasons.add(name)
            os.unlink(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def cpu_cores() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def oracle_sample(pb, budget_s: float, threads: int):
    """Times the CPU oracle on every `stride`-th configuration so that the run takes about budget_s."""
    from oracle import Oracle
    o = Oracle(pb)
    probe = max(1, o.n_pconf // 64)
    t0 = time.perf_counter()
    done, _, _ = o.search_pconfs(0, probe, threads=threads)
    dt = max(time.perf_counter() - t0, 1e-6)
    est_full = dt * o.n_cand / max(done, 1)
    stride = max(1, int(round(est_full / budget_s)))
    t0 = time.perf_counter()
    done, bc, bi = o.search_pconfs(0, stride, threads=threads)
    dt = time.perf_counter() - t0
    return dict(value=done / dt, seconds=dt, candidates=done, stride=stride, n_pconf=o.n_pconf, n_cand=o.n_cand)


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from gen import problems
    pb = problems.make_problem(args.workload)
    threads = cpu_cores()
    budget = max(2.0, min(30.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(pb, budget / 4, threads)
    vals, secs, sample = [], [], None
    for _ in range(args.steps):
        sample = oracle_sample(pb, budget, threads)
        vals.append(sample["value"]); secs.append(sample["seconds"])
    value = statistics.median(vals)
    desc = (f"every {sample['stride']}-th of {sample['n_pconf']} configurations of {args.workload} "
            f"({sample['candidates']} of {sample['n_cand']} candidates) per step")
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1e3 * statistics.median(secs), higher_is_better=True,
                scaling="strong", vs_baseline=None, dtype="int64", data="synthetic",
                config=dict(workload=args.workload, n_candidates=sample["n_cand"], sample=desc),
                cpu_baseline=dict(value=value, unit=UNIT, cores=threads, kind="oracle", sample=desc),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="stress")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--timed-only", action="store_true",
                    help="run the warm-up and the timed steps and stop (for profiler captures): prints a reduced line")
    ap.add_argument("--search-only", action="store_true",
                    help="run warm-up + steps calls of hap_search_best (no pruning) on one GPU and stop (for profiler "
                         "captures of the search form of the kernels): prints a reduced line")
    ap.add_argument("--delta-q", type=int, default=None, help="override the load-balance window (1/1024; <0 = off)")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"],
                    help="torch.distributed backend of the (cost, index) exchange when launched with several ranks")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import numpy as np
    import torch
    import torch.distributed as dist
    import paper_2609_39350_b200 as hap
    from paper_2609_39350_b200.sharding import shard_ranges, exchange_minimum_tensor, recurrence_cells, NO_CANDIDATE
    from gen import problems

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    local_rank %= torch.cuda.device_count()
    torch.cuda.set_device(local_rank)
    if world > 1:
        if args.backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group("gloo")
    xdev = "cuda" if args.backend == "nccl" else "cpu"
    warmup = max(args.warmup, 3)

    pb = problems.make_problem(args.workload)
    if args.delta_q is not None:
        pb.delta_q = args.delta_q
    hp = hap.hap_problem_create(pb)
    n_pconf, n_cand = hap.hap_enumerate(hp)
    pconfs = hap.hap_get_pconfs(hp)
    first, count = shard_ranges(pconfs, len(pb.rc_masks), pb.N, world)[rank]
    stream = torch.cuda.current_stream()

    if args.search_only:
        ms = []
        for it in range(warmup + args.steps):
            flush_s = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if it == 0 else flush_s
            flush_s.fill_(1)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            plan, stats = hap.hap_search_best(hp)
            ms.append(1e3 * (time.perf_counter() - t0))
        print(json.dumps(dict(metric="search_ms", unit="ms", value=statistics.median(ms[warmup:]), n_gpus=1, steps=args.steps, warmup=warmup,
                              config=dict(workload=args.workload), best=dict(cost=plan["T_iter"], index=plan["index"]),
                              dp_phase_ms=stats["ms_dp"], note="hap_search_best only (--search-only)")))
        hap.hap_problem_destroy(hp)
        return

    out = {"cost": torch.empty(max(count, 1), dtype=torch.int64, device="cuda"),
           "bottleneck": torch.empty(max(count, 1), dtype=torch.int64, device="cuda")}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")     # larger than the 126 MB L2

    def step():
        hap.hap_pipeline_dp(hp, first, count, out=out)
        return hap.hap_argmin(hp, out["cost"][:count]) if count else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # clocks and throttle reasons are sampled from before the warm-up until after the timed steps; the timed
    # region lasts only milliseconds, so the same steps keep running (untimed) until a few samples exist
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(warmup):
        flush.fill_(1)
        step()
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    dp_ms, lc_ms, cells = [], [], 0
    best = None
    barrier()
    t_wall = time.perf_counter()
    for a, b in ev:
        flush.fill_(1)                       # untimed: evicts the previous step's data from L2
        a.record(stream)
        am = step()
        if world > 1:
            # one (cost, index) pair per rank, gathered and reduced on the device the backend talks on: no host
            # round trip inside the step (gloo has no device path: the pair goes through the host there)
            pair = am if am is not None else torch.tensor(NO_CANDIDATE, dtype=torch.int64, device="cuda")
            best_t = exchange_minimum_tensor(pair if xdev == "cuda" else pair.cpu(), first)
        b.record(stream)
        b.synchronize()
        lc, dpk, cells = hap.hap_get_timings(hp)
        lc_ms.append(lc); dp_ms.append(dpk)
    barrier()
    t_wall = time.perf_counter() - t_wall
    t_load = time.perf_counter()
    while time.perf_counter() - t_load < 0.8:              # untimed: the same load while the sampler takes its samples
        flush.fill_(1)
        step()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world == 1:
        c, i = (int(x) for x in am.tolist())
        best = (c, i + first)
    else:
        best = tuple(int(x) for x in best_t.tolist())

    step_ms = [a.elapsed_time(b) for a, b in ev]
    if args.timed_only:
        if rank == 0:
            print(json.dumps(dict(metric=METRIC, unit=UNIT, value=n_cand * args.steps / (sum(step_ms) * 1e-3), n_gpus=world,
                                  steps=args.steps, warmup=warmup, ms_per_step=sum(step_ms) / args.steps,
                                  config=dict(workload=args.workload), note="timed region only (--timed-only)")))
        hap.hap_problem_destroy(hp)
        if world > 1:
            dist.destroy_process_group()
        return
    total_ms = torch.tensor([sum(step_ms)], dtype=torch.float64, device=xdev)
    if world > 1:
        dist.all_reduce(total_ms, op=dist.ReduceOp.MAX)
    total_ms = float(total_ms.item())
    ms_per_step = total_ms / args.steps
    value = n_cand * args.steps / (total_ms * 1e-3)

    cells_finite = hap.hap_count_cells(hp, first, count)        # untimed instrumentation launch
    # untimed: the same pass through the counting form of the kernels -> splits evaluated after all early exits
    hp_cnt = hap.hap_problem_create(pb, flags=hap.OPT_COUNT_SPLITS)
    hap.hap_enumerate(hp_cnt)
    hap.hap_pipeline_dp(hp_cnt, first, count, out=out)
    torch.cuda.synchronize()
    cells = hap.hap_get_timings(hp_cnt)[2]
    hap.hap_problem_destroy(hp_cnt)

    # the layer-cost kernels alone (inside a pass the candidate decode of the classes runs beside them on other
    # streams, so the pass's own phase time is not the kernels' time), L2 flushed, CUDA events on the launching stream
    lc_alone = []
    c2_buf, coef_buf = hap.hap_eval_layer_costs(hp)
    for it in range(3 + max(5, min(args.steps, 20))):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        hap.hap_eval_layer_costs(hp, c2=c2_buf, coef=coef_buf)
        b.record(stream)
        b.synchronize()
        if it >= 3:
            lc_alone.append(a.elapsed_time(b))
    lc_alone_ms = statistics.median(lc_alone)
    # yardstick, not part of the path: a plain fill of the same c2 buffer under the same timing (what a kernel that
    # does nothing but write these bytes reaches at this size, launch latency included)
    fill_ms = []
    for it in range(8):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        c2_buf.zero_()
        b.record(stream)
        b.synchronize()
        if it >= 3:
            fill_ms.append(a.elapsed_time(b))
    fill_same_bytes_ms = statistics.median(fill_ms)
    del c2_buf, coef_buf

    # joint recurrence over the device state (all stage-type sequences at once), second call timed
    joint_ms = None
    if world == 1:
        hap.hap_joint_bottleneck(hp)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        flush.fill_(1)
        a.record(stream)
        jb = hap.hap_joint_bottleneck(hp)
        b.record(stream)
        b.synchronize()
        joint_ms = a.elapsed_time(b)

    # the same pass in fp64 mode (unrounded times; context, the bench line is the integer mode)
    fp64_ms = None
    if world == 1:
        ts = []
        for it in range(5):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            hap.hap_pipeline_dp_f64(hp, first, count)
            b.record(stream)
            b.synchronize()
            if it >= 2:
                ts.append(a.elapsed_time(b))
        fp64_ms = statistics.median(ts)

    # the same pass with the refinement (smallest stage-cost sum among the bottleneck-optimal partitions) and with
    # the exact optimisation of sum + (M-1) max (limit sweep); untimed extras
    extra_modes = {}
    for mode_name, flag in (("refined_pass", hap.OPT_REFINE), ("exact_pass", hap.OPT_EXACT),
                            ("uniform_partition_ablation", hap.OPT_UNIFORM)):
        hp_ref = hap.hap_problem_create(pb, flags=flag)
        hap.hap_enumerate(hp_ref)
        ref_ms = []
        for it in range(5):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            hap.hap_pipeline_dp(hp_ref, first, count, out=out)
            am_ref = hap.hap_argmin(hp_ref, out["cost"][:count])
            b.record(stream)
            b.synchronize()
            if it >= 2:
                ref_ms.append(a.elapsed_time(b))
        ref_best = [int(x) for x in am_ref.tolist()]
        extra_modes[mode_name] = dict(ms=statistics.median(ref_ms), best_cost=ref_best[0], best_index=ref_best[1] + first)
        if flag != hap.OPT_UNIFORM:
            # the search entry point under this objective, call to return: a plain pass bounds every candidate and the
            # refinement runs only where the bound can still beat the incumbent
            s_ms = []
            for it in range(4):
                flush.fill_(1)
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                plan_ref, stats_ref = hap.hap_search_range(hp_ref, first, count)
                s_ms.append(1e3 * (time.perf_counter() - t0))
            assert (plan_ref["T_iter"], plan_ref["index"]) == (ref_best[0], ref_best[1] + first)
            extra_modes[mode_name].update(search_ms=statistics.median(s_ms[1:]), search_evaluated=stats_ref["n_evaluated"],
                                          search_cut_by_bound=stats_ref["n_pruned"])
        if flag == hap.OPT_UNIFORM and world == 1:
            # predicted latency of the best uniform-split plan over the best non-uniform plan (planner-level mirror of
            # the paper's "non-uniform partitioning disabled" ablation; synthetic inputs, context only)
            extra_modes[mode_name]["latency_ratio_vs_non_uniform"] = ref_best[0] / best[0]
        hap.hap_problem_destroy(hp_ref)

    # Appendix B's latency expression for the winning plan, beside the closed form the search minimises (context)
    appb = None
    if world == 1:
        one = hap.hap_pipeline_dp(hp, best[1], 1, partition=True)
        ab = hap.hap_eval_appendix_b(hp, best[1], 1, one["partition"], one["recompute"], detail=True)
        torch.cuda.synchronize()
        edge, middle, smax = (int(x) for x in ab["detail"][0].tolist())
        appb = dict(T_iter_closed_form=best[0], T_iter_appendix_b=int(ab["t_iter"][0]), T_edge=edge, T_middle=middle, s_max=smax)
        # ... and the 1F1B schedule itself run for that plan (context: what the closed form leaves out)
        sim = hap.hap_simulate_1f1b(hp, best[1], 1, one["partition"], one["recompute"], detail=True)
        torch.cuda.synchronize()
        appb["T_iter_simulated_1f1b"] = int(sim["t_iter"][0])
        appb["T_pipe_simulated_1f1b"], appb["T_pipe_closed_form"] = (int(x) for x in sim["detail"][0].tolist())

    # full search through the search entry point (pruning allowed), wall clock call to return
    search_ms, pruned_ms = [], []
    hp_pr = hap.hap_problem_create(pb, prune=1)
    hap.hap_enumerate(hp_pr)
    for _ in range(3):
        flush.fill_(1)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        plan, stats = hap.hap_search_range(hp, first, count)
        search_ms.append(1e3 * (time.perf_counter() - t0))
        flush.fill_(1)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        plan_pr, stats_pr = hap.hap_search_range(hp_pr, first, count)
        pruned_ms.append(1e3 * (time.perf_counter() - t0))
    assert plan_pr == plan
    hap.hap_problem_destroy(hp_pr)

    # end to end through the C ABI from host buffers: create (H2D of the tables), enumerate (H2D of the
    # configuration table), search, read the plan back
    e2e_ms = []
    h2d = sum(int(getattr(pb, n).nbytes) for n in ("tdf", "tdb", "tff", "tfb", "tpre", "tpost")) + int(pconfs.nbytes)
    d2h = 8 * 2 + 8 * 4 + 200
    for _ in range(3):
        flush.fill_(1)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        hp2 = hap.hap_problem_create(pb)
        hap.hap_enumerate(hp2)
        plan2, _ = hap.hap_search_range(hp2, first, count)
        e2e_ms.append(1e3 * (time.perf_counter() - t0))
        hap.hap_problem_destroy(hp2)
    # the same once more with the library's cache of device memory emptied first (the allocations are then the driver's)
    hap.hap_release_cached_memory()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    hp2 = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp2)
    hap.hap_search_range(hp2, first, count)
    e2e_uncached_ms = 1e3 * (time.perf_counter() - t0)
    hap.hap_problem_destroy(hp2)
    e2e_t = torch.tensor([statistics.median(e2e_ms)], dtype=torch.float64, device=xdev)
    if world > 1:
        dist.all_reduce(e2e_t, op=dist.ReduceOp.MAX)
    e2e_value = n_cand / (float(e2e_t.item()) * 1e-3)

    if rank == 0:
        peaks, peak_kind = read_peaks()
        dp_med, lc_med = statistics.median(dp_ms), statistics.median(lc_ms)
        sm_mhz = clocks["sm_mhz"] or peaks.get("sm_max_mhz", 1965.0)
        # issue-slot peak at the clock sampled during the timed region
        alu_peak = SM_COUNT * SCHEDULERS_PER_SM * LANES * float(sm_mhz) * 1e6 / 1e12
        # Work of the DP phase, three ways, all at 4 semiring operations (prefix difference, max, min, arg-select)
        # per split: `executed` = the splits the kernels evaluated (counted by the kernels, after windows, bands,
        # shared stage prefixes and early exits) -- this is what the fraction reports; `finite` = the splits of the
        # recurrence whose stage cost is finite, per candidate, nothing shared; `plain` = the recurrence without
        # the window, 2w + (PP-2)w(w+1)/2 per candidate with w = N-PP+1.  The last two say how much work the tree
        # form avoids; they are not utilisation figures.
        cells_plain = float(sum(recurrence_cells(pb.N, int(r["PP"])) * int(r["nmap"]) * len(pb.rc_masks) for r in pconfs))
        achieved = 4.0 * cells / (dp_med * 1e-3) / 1e12
        units = n_pconf * hp.T * pb.N
        lc_gbs = 16.0 * units / (lc_alone_ms * 1e-3) / 1e9
        line = dict(
            metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=warmup,
            ms_per_step=ms_per_step, higher_is_better=True, scaling="strong", vs_baseline=None, dtype="int64",
            data="synthetic",
            config=dict(workload=args.workload, n_pconf=n_pconf, n_candidates=n_cand, layers=pb.N, devices=pb.W,
                        window_delta_q=int(pb.delta_q), l2="flushed between steps (256 MiB fill, untimed)",
                        timing="sum of per-step CUDA-event times, max over ranks",
                        parallelism=f"candidate ranges over {world} gpu(s)"),
            clocks=dict(sm_mhz=clocks["sm_mhz"], sm_max_mhz=clocks["sm_max_mhz"], reasons=clocks["reasons"]),
            e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                     ms=float(e2e_t.item()), ms_without_cached_device_memory=e2e_uncached_ms,
                     what="hap_problem_create + hap_enumerate + hap_search_best from host buffers (median of 3; the "
                          "process keeps freed device memory and the classes' prefix trees between problems)"),
            # per step: type_const, one decode and one tree-gather launch, one tree DP launch per PP class, argmin partial + final
            gpu_launches=hap.hap_launches_per_pass(hp) * args.steps,
            **extra_modes,
            joint_recurrence_ms=joint_ms,
            fp64_mode_pass_ms=fp64_ms,
            appendix_b_best_plan=appb,
            full_search_ms=statistics.median(search_ms),
            full_search_pruned=dict(ms=statistics.median(pruned_ms), n_pruned=stats_pr["n_pruned"],
                                    n_evaluated=stats_pr["n_evaluated"]),
            best=dict(cost=best[0], index=best[1], search_index=plan["index"]),
            kernels_ms=dict(type_constants=lc_med, pipeline_dp=dp_med),
            roofline=dict(bound="alu", kernel="trie_dp_kernel (one launch per PP class, concurrent streams)",
                          achieved=achieved, peak=alu_peak, unit="Tops/s", frac=achieved / alu_peak,
                          traffic=None, ops_per_split=4, splits_executed=cells,
                          effective_finite=dict(cells=cells_finite, tops=4.0 * cells_finite / (dp_med * 1e-3) / 1e12),
                          effective_plain_recurrence=dict(cells=cells_plain, tops=4.0 * cells_plain / (dp_med * 1e-3) / 1e12),
                          note="achieved = 4 ops x splits the kernels evaluated / CUDA-event time of the DP phase; the "
                               "effective_* figures divide the work of the per-candidate recurrence (finite-cost splits; "
                               "every split without the window) by the same time and measure what the shared prefix tree, "
                               "bands and early exits avoid, not utilisation; traffic: not measured by this run",
                          peak_source=f"{SM_COUNT} SMs x {SCHEDULERS_PER_SM} schedulers x {LANES} lanes x "
                          f"{sm_mhz} MHz (clock sampled during the timed region)", sm_mhz_seen=sm_mhz),
            roofline_layer_cost=dict(bound="hbm", kernel="type_const_kernel + layer_cost_kernel (hap_eval_layer_costs alone; "
                                     "the pass itself computes layer costs inside the DP blocks and writes none)",
                                     achieved=lc_gbs, peak=peaks["hbm_gbs"],
                                     unit="GB/s", frac=lc_gbs / peaks["hbm_gbs"], traffic=None,
                                     bytes_per_launch=16 * units, ms_alone=lc_alone_ms, ms_before_dp_in_pass=lc_med,
                                     ms_plain_fill_of_the_same_bytes=fill_same_bytes_ms,
                                     note="achieved = 16 B per (configuration, type, layer) unit written / time of the call "
                                          "alone after an L2 flush; the output may still sit in L2 when the call ends",
                                     peak_source=f"hbm_gbs ({peak_kind})"),
            wall_s=t_wall,
        )
        if world == 1 and not args.no_cpu_baseline:
            s = oracle_sample(pb, 15.0, cpu_cores())
            line["cpu_baseline"] = dict(value=s["value"], unit=UNIT, cores=cpu_cores(), kind="oracle",
                                        sample=f"every {s['stride']}-th of {s['n_pconf']} configurations of "
                                               f"{args.workload}: {s['candidates']} candidates in {s['seconds']:.1f} s")
        print(json.dumps(line))
    hap.hap_problem_destroy(hp)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
