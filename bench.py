#!/usr/bin/env python
"""Throughput of the DiSCo policy-evaluation path on B200: request-policy evaluations per second.

One step = one pass of the whole path over one synthetic workload: trace ingestion (ticks, p(l), sorted
F), Algorithms 1-3 for every policy, token-by-token play-out, per-pair evaluation (with the per-pair
arrays written for workloads 0 and 1), per-policy reductions and policy selection.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference] [--sharded]

The line's `value` is workload `--config` (default 4: 16 M requests x 1024 policies, six profile groups,
nothing materialised) with the trace arrays already resident in HBM; `e2e` goes through the same calls
with pinned host arrays (host->device copies and the statistics read-back inside the timed region).  At
one GPU the line also carries `per_config`: the same measurements for every workload 0-5, taken in the
same process.  With N > 1 (torchrun) every rank evaluates an independent trace of the same shape (weak
scaling, no collective on the data path); `--sharded` instead splits ONE trace into request ranges, one
per rank (strong scaling: the ranks exchange the tables of Algorithm 1 and add up their accumulators).
`--impl reference` times the CPU oracle on the host cores instead.
"""
import argparse
import json
import math
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "request-policy evaluations/s"
UNIT = "pairs/s"
PAIR_OUT_BYTES = 31          # four fp32, three u32, one u16, one u8 per pair
TRACE_BYTES = 9              # packed request: ticks, prompt, output length, group
# Lane-instructions one token-step of the play-out needs.  General form (both endpoints' streams share the
# hash draw): counter add 1, hash finaliser 8, two range maps (multiply-high) 2, tail mask 1, two sums and two
# maxima 4, loop 1.  When no interval can exceed the consumption interval (tau >= T + J for both endpoints of
# every group) only the stream of the endpoint that may hand over is summed: counter 1, hash 8, one range map
# 1, tail test 1, sum 1, loop 1.
PLAYOUT_INSTR_PER_TOKEN = 17
PLAYOUT_INSTR_PER_TOKEN_LEAN = 13
# Lane-instructions one (request, policy) pair needs in the reduction kernel, by the kind of policy.
# Algorithm 3 (no waits; the race at w = 0 is staged once per request): request vector load 1, length
# threshold 1, trigger compare and its conjunction 2, outcome index 2, TTFT select 1, row address 1, two row
# loads 2, six 32-bit sums (tokens on device, two prefills, TBTs in tau's bin, delayed tokens, the four
# byte-packed counts) and one 64-bit sum 8, staged histogram increment (address, atomic) 2, stall test shared
# by four pairs 1.
PAIR_INSTR_NOWAIT = 21
# Algorithm 2 (waits): load 1, wait map 4, start compare 1, w + T_d 1, win compare 1, minimum 1, trigger 3,
# outcome index 3, row address 1, two row loads 2, sums 8, histogram increment from the float bits (convert,
# small-value test and branch, offset 2, increment 3, address, atomic) 10, stall test 1.
PAIR_INSTR_WAIT = 37
# Lane-instructions the zone-by-zone reduction needs per request and policy FAMILY (up to 128 policies along a
# budget axis, whatever their number): request loads 6, device TTFT 1, projected saving 4, race at wait 0 (two
# compares, select, minimum) 4, trigger against the family's range 3, outcome select 2, the common outcome's
# addends 14, its ten sums 11, histogram bin and increment 6; the first run's outcome 8, its addends 14, ten
# differences to the common outcome 20, histogram bin and increment 6; loop 1.  The extra sweeps over requests
# whose prompt length is some policy's l* are not counted.
ZONE_INSTR_PER_REQUEST_FAMILY = 100
SCHEDULERS, LANES = 4, 32    # warp schedulers per multiprocessor, lanes per warp
MIN_WARMUP_SECONDS = 0.5     # untimed steps run until this much device time has passed (and at least --warmup)
MAX_WARMUP_STEPS = 200
# From the committed ncu captures (profiles/): DRAM bytes per launch of the bench's own launch shape, and the
# lane-slots the hardware executed per unit of work beside the algorithmic counts above.  None: not captured
# for the current kernel.
NCU_TRAFFIC_BYTES = {("k_pairs_rows", 1): 145709568, ("k_playout_fast", 1): 827904}
# issued lane-slots per token-step (play-out; the workload-3 figure is of a 200,000-request capture of its shape, the
# workload-4 figure of a 4,000,000-request one) and
# per request and policy family (zone kernel, workload 2 at full size)
NCU_EXECUTED_PER_UNIT = {("k_playout_fast", 1): 31.9, ("k_playout_fast", 3): 21.8, ("k_playout_fast", 4): 28.2,
                         ("k_pairs_zones+k_pairs_acc", 2): 269.0}
HEADLINE_CONFIG = 4
ALL_CONFIGS = (0, 1, 2, 3, 4, 5)


def env_rank():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU every 20 ms through NVML while the timed region runs
    (read-only queries)."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index):
        import threading
        self.index, self.samples, self.reasons, self.max_mhz = int(index), [], set(), None
        self._stop, self._ready = threading.Event(), threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)
        self.error = None

    def _run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while True:
                self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                mask = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                self._ready.set()
                if self._stop.wait(0.02):
                    break
        except Exception as e:                      # no NVML: report that rather than invent numbers
            self.error = repr(e)
            self._ready.set()

    def start(self):
        """Returns once the first sample is in, so that opening NVML stays outside the timed region."""
        self._thread.start()
        self._ready.wait(timeout=60)

    def stop(self):
        self._stop.set()
        self._thread.join(timeout=5)
        if self.error or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "samples": 0,
                    "reasons": ["clock sampling failed: %s" % self.error]}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz, "samples": len(self.samples),
                "reasons": sorted(self.reasons)}


def never_clamps(w):
    """True when every policy paces delivery and no endpoint's slowest interval T + J exceeds the consumption
    interval, in the tick arithmetic of the library (microseconds, ties to even)."""
    FLAG_PACING = 2
    tick = lambda x: int(round(x * 1e6))
    for pol in w.policies:
        if not (int(pol["flags"]) & FLAG_PACING):
            return False
        tau = tick(1.0 / float(np.float32(pol["r_c"])))
        for sv in w.servers:
            T = tick(float(np.float32(sv["tbt_s"])))
            if T + int(round(T * float(np.float32(sv["jitter"])))) > tau:
                return False
        for dv in w.devices:
            T = tick(1.0 / float(np.float32(dv["decode_tps"])))
            if T + int(round(T * float(np.float32(dv["jitter"])))) > tau:
                return False
    return True


def max_over_ranks(total_ms, dist, device):
    """The slowest rank's time decides a multi-GPU step (all-reduce MAX); a single process returns its own."""
    if dist is None:
        return total_ms
    import torch
    t = torch.tensor([total_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank, world, steps, total_ms):
    """Whole-job throughput: units of all ranks over the slowest rank's time."""
    return units_per_rank * world * steps / (total_ms * 1e-3)


def shard_bounds(n, world):
    """Contiguous request ranges, one per rank: rank r holds [bounds[r], bounds[r+1])."""
    return [n * r // world for r in range(world + 1)]


def exchange_group_tables(cnt, sorted_by_group, dist, device):
    """Whole-trace tables from the ranks' own: the length histograms add up (one all-reduce); every rank's
    sorted ticks of a group are gathered (padded to the longest run) and laid out group after group.  Returns
    (cnt int64 [G, 4097] on the host, ticks int32 tensor, n_ticks uint64 [G]); the ticks of a group are the
    ranks' sorted runs one after the other, which is what disco_set_group_tables takes.
    cnt: numpy int64 [G, 4097]; sorted_by_group: list of G int32 tensors on `device`."""
    import torch
    world = dist.get_world_size()
    G = len(sorted_by_group)
    c = torch.from_numpy(np.ascontiguousarray(cnt, dtype=np.int64)).to(device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    mine = torch.tensor([int(s.numel()) for s in sorted_by_group], dtype=torch.int64, device=device)
    sizes = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(sizes, mine)
    sizes = torch.stack(sizes).cpu().numpy()                               # [world, G]
    longest = int(sizes.max()) if sizes.size else 0
    pieces = []
    for g in range(G):
        pad = torch.zeros(max(longest, 1), dtype=torch.int32, device=device)
        pad[:sorted_by_group[g].numel()] = sorted_by_group[g]
        got = [torch.empty_like(pad) for _ in range(world)]
        dist.all_gather(got, pad)
        pieces += [got[r][:int(sizes[r, g])] for r in range(world)]
    ticks = torch.cat(pieces) if pieces else torch.empty(0, dtype=torch.int32, device=device)
    return c.cpu().numpy(), ticks.contiguous(), sizes.sum(axis=0).astype(np.uint64)


def oracle_sample_run(w, n_req, threads):
    """Times the oracle, as it stands, on the first n_req requests under every policy of w, one thread per
    contiguous request range.  Returns seconds."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import Oracle
    orc = oracle_sample_run.cache.get(id(w))
    if orc is None:
        oracle_sample_run.cache.clear()
        orc = Oracle.from_workload(w)
        oracle_sample_run.cache[id(w)] = orc
    threads = max(1, min(threads, n_req))
    bounds = [n_req * k // threads for k in range(threads + 1)]
    t0 = time.perf_counter()
    if threads == 1:
        orc.eval(w.policies, w.seed, 0, n_req, finish=False)
    else:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(lambda k: orc.eval(w.policies, w.seed, bounds[k], bounds[k + 1], finish=False),
                        range(threads)))
    return time.perf_counter() - t0


oracle_sample_run.cache = {}


def size_oracle_sample(w, threads, seconds):
    """Number of leading requests the oracle takes about `seconds` for on `threads` threads: probes grow until
    one took at least a fifth of the target (short runs are dominated by the per-call policy preparation and do
    not extrapolate), then scale linearly."""
    probe = min(w.n, max(threads * 4, 64))
    while True:
        t = oracle_sample_run(w, probe, threads)
        if probe >= w.n or t >= 0.2 * seconds:
            break
        probe = int(min(w.n, max(2 * probe, probe * 0.5 * seconds / max(t, 1e-3))))
    return int(min(w.n, max(threads, probe * seconds / max(t, 1e-4))))


def cpu_baseline_of(w, seconds):
    cores = os.cpu_count() or 1
    n_req = size_oracle_sample(w, cores, seconds)
    t = oracle_sample_run(w, n_req, cores)
    P = w.n_policies
    return {"value": n_req * P / t, "unit": UNIT, "cores": min(cores, n_req), "kind": "oracle",
            "sample": "first %d of %d requests x all %d policies, %.1f s" % (n_req, w.n, P, t),
            "token_steps_per_s": int((w.output_len[:n_req] - 1).sum()) * P / t}


def run_reference(args):
    rank, _, world = env_rank()
    if rank != 0:
        return 0
    from paper_2502_11417_b200 import synth
    w = synth.make_workload(args.config, n=args.requests, n_budgets=args.budgets)
    cores = os.cpu_count() or 1
    n_req = size_oracle_sample(w, cores, args.oracle_step_seconds)
    for _ in range(args.warmup):
        oracle_sample_run(w, n_req, cores)
    times = [oracle_sample_run(w, n_req, cores) for _ in range(args.steps)]
    pairs = n_req * w.n_policies
    toks = int((w.output_len[:n_req] - 1).sum()) * w.n_policies
    total = sum(times)
    value = pairs * args.steps / total
    sample = "first %d of %d requests x all %d policies per step" % (n_req, w.n, w.n_policies)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "sim_tokens_per_s": toks * args.steps / total,
            "config": {"workload": w.name, "requests": w.n, "policies": w.n_policies, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, n_req), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


PIPELINE_WORKERS = 3


class Bench:
    """The measurements of one workload on this rank's GPU."""

    def pipelined(self, w, host, pols, steps):
        """End-to-end steps from pinned host arrays by PIPELINE_WORKERS host threads, each with a context and a
        stream of its own, so that one worker's host-to-device transfer runs beside another's kernels.  Every step
        still moves its own inputs in and its statistics out.  Timed on the device from before the first step to
        after the last."""
        import threading
        import torch
        from paper_2502_11417_b200 import Trace
        from paper_2502_11417_b200.api import stats_view, select_policy
        cap_factor, slo = w.select["cost_cap_factor"], w.select["tbt_slo_s"]
        dev = torch.cuda.current_device()
        trs = [Trace() for _ in range(PIPELINE_WORKERS)]
        sts = [torch.cuda.Stream() for _ in range(PIPELINE_WORKERS)]

        def worker(tr, st, k):
            torch.cuda.set_device(dev)
            for _ in range(k):
                tr.load_trace(*host, w.servers, w.devices, stream=st, staged_copy=True)
                tr.eval_policies(pols, w.seed, None, stream=st)
                s = tr.reduce_stats(stream=st)
                select_policy(s, cap_factor * float(stats_view(s)["total_cost"].min()), slo)

        def run(k):
            th = [threading.Thread(target=worker, args=(t, s, k)) for t, s in zip(trs, sts)]
            for x in th:
                x.start()
            for x in th:
                x.join()

        run(2)
        torch.cuda.synchronize()
        main = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        per_worker = max(2, (steps + PIPELINE_WORKERS - 1) // PIPELINE_WORKERS)
        e0.record(main)
        for s in sts:
            s.wait_stream(main)
        run(per_worker)
        for s in sts:
            main.wait_stream(s)
        e1.record(main)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / (per_worker * PIPELINE_WORKERS)
        for t in trs:
            t.close()
        return {"workers": PIPELINE_WORKERS, "ms_per_step": ms, "value": w.n * w.n_policies / (ms * 1e-3), "unit": UNIT,
                "how": "host threads with a context and a stream each; the transfers use the copy engine"}

    def __init__(self, args, dist, rank, world, flush, peaks, alu_measured):
        self.args, self.dist, self.rank, self.world = args, dist, rank, world
        self.flush, self.peaks, self.alu_measured = flush, peaks, alu_measured

    def run(self, cfg, steps, warmup, oracle_seconds, sampler=None, sharded=False):
        import ctypes
        import torch
        from paper_2502_11417_b200 import synth, Trace
        from paper_2502_11417_b200.api import (policy_array, kernel_launch_count, PolicyStats, stats_view,
                                               select_policy)
        args, dist, world, flush = self.args, self.dist, self.world, self.flush
        stream = torch.cuda.current_stream()
        if sharded:
            whole = synth.make_workload(cfg, n=args.requests, n_budgets=args.budgets)
            b = shard_bounds(whole.n, world)
            lo, hi = b[self.rank], b[self.rank + 1]
            w = whole
        else:
            w = synth.make_workload(cfg, n=args.requests, n_budgets=args.budgets, replica=self.rank)
            lo, hi = 0, w.n
        P, n = w.n_policies, hi - lo
        G = len(w.servers) * len(w.devices)
        pols = policy_array(w.policies)
        cols = (w.prompt_len, w.output_len, w.server_ttft_s, w.server_profile, w.device_profile)
        host = [torch.from_numpy(np.ascontiguousarray(x[lo:hi])).pin_memory() for x in cols]
        dev = [x.cuda() for x in host]
        h2d = sum(x.numel() * x.element_size() for x in host) + P * ctypes.sizeof(pols[0])
        d2h = P * ctypes.sizeof(PolicyStats) + 8
        tr = Trace()
        tr.n = n
        out = None
        if w.materialise:
            tr.load_trace(*dev, w.servers, w.devices, first_index=lo)
            out = tr.alloc_pair_outputs(P)
        cap_factor, slo = w.select["cost_cap_factor"], w.select["tbt_slo_s"]
        words = None

        def step(arrays):
            nonlocal words
            tr.load_trace(*arrays, w.servers, w.devices, stream=stream, first_index=lo)
            if sharded:
                # exchange 1: every rank needs the whole trace's p(l) and F before Algorithms 1-3 run
                cnt = np.stack([tr.group_tables(g, n_sorted=0)[0] for g in range(G)])
                mine = [tr.sorted_ticks_device(g) for g in range(G)]
                tcnt, ticks, n_ticks = exchange_group_tables(cnt, mine, dist, "cuda")
                tr.set_group_tables(tcnt, ticks, n_ticks, stream=stream)
            tr.eval_policies(pols, w.seed, out, stream=stream)
            if sharded:
                # exchange 2: the accumulators are integer sums over requests
                if words is None:
                    words = torch.empty(tr.accumulator_words(), dtype=torch.int64, device="cuda")
                tr.export_accumulators(words, stream=stream)
                dist.all_reduce(words, op=dist.ReduceOp.SUM)
                tr.import_accumulators(words, stream=stream)
            st = tr.reduce_stats(stream=stream)
            cap = cap_factor * float(stats_view(st)["total_cost"].min())
            return select_policy(st, cap, slo)

        def run_steps(arrays, k, collect=None):
            """k steps, each between its own pair of events, L2 flushed before each; returns the summed device
            milliseconds of this rank (the flush is outside the events)."""
            evs = []
            for _ in range(k):
                flush.zero_()
                if collect is not None:
                    tr.set_timing(True)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                step(arrays)
                e1.record(stream)
                evs.append((e0, e1))
                if collect is not None:
                    collect.append(tr.timing())
            torch.cuda.synchronize()
            return sum(a.elapsed_time(b) for a, b in evs)

        def warm_up(arrays):
            """At least `warmup` steps and MIN_WARMUP_SECONDS of device time (the first steps of a fresh process
            run slower: clocks and caches settle); the same count on every rank."""
            done, ms = 0, 0.0
            while done < MAX_WARMUP_STEPS and (done < warmup or ms < 1e3 * args.min_warmup_seconds):
                k = max(1, min(warmup - done, 8)) if done < warmup else 4
                ms += run_steps(arrays, k)
                done += k
                if dist is not None:                 # all ranks stop together
                    t = torch.tensor([ms], device="cuda", dtype=torch.float64)
                    dist.all_reduce(t, op=dist.ReduceOp.MIN)
                    ms = float(t.item())
            return done

        def timed(arrays):
            torch.cuda.synchronize()
            if dist is not None:
                dist.barrier()
            tr.set_timing(False)
            ms = run_steps(arrays, steps)
            if dist is not None:
                dist.barrier()
            return max_over_ranks(ms, dist, "cuda")

        warm_dev = warm_up(dev)
        l0 = kernel_launch_count()
        if sampler is not None:
            sampler.start()
        total_ms = timed(dev)
        clocks = sampler.stop() if sampler is not None else None
        launches = kernel_launch_count() - l0
        # per-kernel durations: a pass of its own (the library's events around its big kernels keep neighbouring
        # launches from overlapping, which would slow the timed steps), one sample per step
        ktimes = []
        run_steps(dev, max(steps, 5), ktimes)
        tr.set_timing(False)
        warm_host = warm_up(host)
        e2e_ms = timed(host)
        piped = self.pipelined(w, host, pols, steps) if (world == 1 and not sharded and not w.materialise) else None

        units = (w.n if sharded else n * world) * P                      # pairs of the whole job per step
        value = units * steps / (total_ms * 1e-3)
        e2e_value = units * steps / (e2e_ms * 1e-3)
        token_steps = int((w.output_len[lo:hi] - 1).sum())
        n_classes = len({(float(np.float32(q["r_c"])), float(np.float32(q["t_m_s"])), int(q["flags"]) & 2)
                         for q in w.policies})
        job_token_steps = (int((w.output_len - 1).sum()) if sharded else token_steps * world) * n_classes

        # ---- rooflines of the timed kernels
        hbm_gbs, sm_max_mhz, src = self.peaks
        sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
        names = ["k_playout_fast", "k_playout", "k_pairs_acc", "k_pairs_rows"]
        kms = {nm: statistics.mean(t[i] for t in ktimes) for i, nm in enumerate(names)}
        alu_peak = sms * SCHEDULERS * LANES * sm_max_mhz * 1e6 / 1e12         # T lane-instructions/s
        alu_src = "%d SMs x %d schedulers x %d lanes x %.0f MHz (issue slots)" % (sms, SCHEDULERS, LANES, sm_max_mhz)
        alu_meas = self.alu_measured / 1e12 if self.alu_measured else None
        per_token = PLAYOUT_INSTR_PER_TOKEN_LEAN if never_clamps(w) else PLAYOUT_INSTR_PER_TOKEN
        full_size = not args.requests and not args.budgets

        def alu_roof(name, lane_instr, ms, **extra):
            ach = lane_instr / (ms * 1e-3) / 1e12
            r = {"kernel": name, "bound": "alu", "achieved": ach, "peak": alu_peak, "unit": "Tinstr/s",
                 "frac": ach / alu_peak, "traffic": NCU_TRAFFIC_BYTES.get((name, cfg)) if full_size else None,
                 "peak_source": alu_src,
                 # what the GPU sustains on the token loop's own instruction mix with every SM full
                 # (disco_measure_alu_peak, measured in this run)
                 "peak_measured": alu_meas, "frac_of_measured": ach / alu_meas if alu_meas else None,
                 "executed_lane_slots_per_unit": NCU_EXECUTED_PER_UNIT.get((name, cfg)),
                 "ms_per_launch": ms}
            r.update(extra)
            return r

        def roof_of(name):
            ms = kms[name]
            if ms <= 0.0:
                return None
            if name == "k_pairs_rows":
                if not w.materialise:
                    return None
                bytes_alg = n * P * PAIR_OUT_BYTES + n * TRACE_BYTES
                ach = bytes_alg / (ms * 1e-3) / 1e9
                return {"kernel": name, "bound": "hbm", "achieved": ach, "peak": hbm_gbs, "unit": "GB/s",
                        "frac": ach / hbm_gbs, "traffic": NCU_TRAFFIC_BYTES.get((name, cfg)) if full_size else None,
                        "peak_source": src, "algorithmic_bytes": bytes_alg, "ms_per_launch": ms}
            if name == "k_pairs_acc":
                # the two reduction kernels together (their events bracket both): requests settled zone by zone per
                # policy family, and the pairs left to the pair-by-pair kernel, by kind (a (group, policy) waits
                # when Algorithm 1 made the group device-constrained)
                zone_pairs, left_pairs, settled, sweeps = tr.work_counts()
                wait_pairs = 0
                for g in range(tr.n_groups):
                    n_g = tr.group_size(g)
                    wait_pairs += n_g * sum(1 for p in range(P) if tr.prep(g, p).device_constrained)
                wait_share = wait_pairs / float(max(n * P, 1))
                per_left_pair = wait_share * PAIR_INSTR_WAIT + (1.0 - wait_share) * PAIR_INSTR_NOWAIT
                lane_instr = settled * ZONE_INSTR_PER_REQUEST_FAMILY + left_pairs * per_left_pair
                return alu_roof("k_pairs_zones+k_pairs_acc", lane_instr, ms,
                                work={"pairs_by_zones": zone_pairs, "pairs_one_by_one": left_pairs,
                                      "requests_settled_per_family": settled, "segment_sweeps": sweeps},
                                instr={"per_request_family": ZONE_INSTR_PER_REQUEST_FAMILY,
                                       "per_pair_one_by_one": per_left_pair},
                                instr_per_pair_mean=lane_instr / float(max(n * P, 1)))
            if name == "k_playout_fast":
                return alu_roof(name, token_steps * per_token * n_classes, ms, token_steps=token_steps * n_classes,
                                instr_per_token_step=per_token)
            return None                       # k_playout: only the requests the clamp-free kernel listed

        roofs = [r for r in (roof_of(nm) for nm in names) if r is not None]
        roof = None
        if roofs:
            roof = dict(max(roofs, key=lambda r: r["ms_per_launch"]))
            roof["all_kernels"] = [{k: r.get(k) for k in ("kernel", "bound", "achieved", "peak", "unit", "frac",
                                                          "frac_of_measured", "ms_per_launch")} for r in roofs]
            roof["kernels_ms"] = kms
            roof["kernel_event_samples"] = len(ktimes)
        cpu = None
        if self.rank == 0 and world == 1 and oracle_seconds > 0:
            cpu = cpu_baseline_of(w, oracle_seconds)
        tr.close()
        res = {"value": value, "ms_per_step": total_ms / steps, "steps": steps, "warmup": warm_dev,
               # token-steps actually played per second: one play-out per request and timeline class (policies
               # that share the consumption rate, buffer size and pacing share it), whatever the number of policies
               "sim_tokens_per_s": job_token_steps * steps / (total_ms * 1e-3),
               # tokens of all (request, policy) pairs covered per second: each played token counted once for
               # every policy that shares its play-out
               "pair_tokens_per_s": job_token_steps / n_classes * P * steps / (total_ms * 1e-3),
               "config": {"workload": w.name, "requests_per_gpu": n, "policies": P, "groups": G,
                          "pairs_per_step": units, "per_pair_outputs": bool(w.materialise),
                          "l2": "flushed between steps (512 MB write)", "seed": w.seed,
                          "select": "cost cap %.2f x cheapest policy, P99 TBT <= %.2f s" % (cap_factor, slo)},
               "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "ms_per_step": e2e_ms / steps, "warmup": warm_host, "pipelined": piped},
               "gpu_launches": launches, "roofline": roof, "cpu_baseline": cpu}
        if clocks is not None:
            res["clocks"] = clocks
        return res


def run_ours(args):
    import torch
    rank, local_rank, world = env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if args.sharded and world == 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", str(29400 + os.getpid() % 500))
            dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", local_rank))
    from paper_2502_11417_b200.api import measure_alu_peak

    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")       # larger than the 126 MB L2
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    try:
        phys = int(vis.split(",")[local_rank]) if vis else local_rank
    except ValueError:
        phys = local_rank
    measure_alu_peak()                                                     # first call: module load, clocks
    alu = statistics.median(measure_alu_peak()[0] for _ in range(3))
    b = Bench(args, dist, rank, world, flush, measured_peaks(), alu)
    main = b.run(args.config, args.steps, args.warmup, args.oracle_seconds if world == 1 else 0.0,
                 sampler=ClockSampler(phys), sharded=args.sharded)
    per_config = None
    if world == 1 and not args.sharded and not args.no_per_config and not args.requests and not args.budgets:
        per_config = []
        for cfg in ALL_CONFIGS:
            if cfg == args.config:
                r = main
            else:
                # enough steps for a stable mean, bounded in time (a workload-3 step takes about 3 ms, a
                # workload-2 step under 2 ms, the others well under 1 ms)
                r = b.run(cfg, max(args.steps, 20), args.warmup, min(args.oracle_seconds, 3.0))
            keep = {k: r[k] for k in ("value", "ms_per_step", "steps", "warmup", "sim_tokens_per_s",
                                      "pair_tokens_per_s", "gpu_launches", "cpu_baseline")}
            keep["workload"] = r["config"]["workload"]
            keep["requests"], keep["policies"] = r["config"]["requests_per_gpu"], r["config"]["policies"]
            keep["e2e"] = {k: r["e2e"][k] for k in ("value", "ms_per_step")}
            keep["roofline"] = None if r["roofline"] is None else {
                "kernel": r["roofline"]["kernel"], "bound": r["roofline"]["bound"], "frac": r["roofline"]["frac"],
                "frac_of_measured": r["roofline"].get("frac_of_measured"), "all_kernels": r["roofline"]["all_kernels"]}
            per_config.append(keep)
    if rank == 0:
        line = {"metric": METRIC, "value": main["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": main["warmup"], "warmup_requested": args.warmup, "ms_per_step": main["ms_per_step"],
                "higher_is_better": True, "scaling": "strong" if args.sharded else "weak", "vs_baseline": None,
                "dtype": "int32", "data": "synthetic", "sim_tokens_per_s": main["sim_tokens_per_s"],
                "pair_tokens_per_s": main["pair_tokens_per_s"], "config": main["config"], "clocks": main["clocks"],
                "e2e": main["e2e"], "gpu_launches": main["gpu_launches"], "roofline": main["roofline"],
                "cpu_baseline": main["cpu_baseline"],
                "alu_peak_measured": {"lane_instr_per_s": alu, "how": "disco_measure_alu_peak: the token loop's "
                                      "13-instruction mix on every SM, median of 3"}}
        if args.sharded:
            line["config"]["split"] = "one trace in %d request ranges; tables all-gathered, accumulators all-reduced" % world
        if per_config is not None:
            line["per_config"] = per_config
        print(json.dumps(line))
    if dist is not None and dist.is_initialized():
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=HEADLINE_CONFIG, help="workload 0..5 (default: workload 4)")
    ap.add_argument("--requests", type=int, default=None, help="shrink the trace (profiling on a small case)")
    ap.add_argument("--budgets", type=int, default=None, help="shrink the budget axis (profiling on a small case)")
    ap.add_argument("--no-per-config", action="store_true", help="skip the other workloads' measurements")
    ap.add_argument("--min-warmup-seconds", type=float, default=MIN_WARMUP_SECONDS,
                    help="untimed steps go on until this much device time has passed (profiling runs pass 0)")
    ap.add_argument("--sharded", action="store_true",
                    help="N > 1: split one trace into request ranges instead of running N independent traces")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--oracle-seconds", type=float, default=15.0, help="CPU time of the oracle baseline sample")
    ap.add_argument("--oracle-step-seconds", type=float, default=3.0, help="--impl reference: CPU time per step")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
