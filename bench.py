#!/usr/bin/env python
"""Throughput of the DiSCo policy-evaluation path on B200: request-policy evaluations per second.

One step = one pass of the whole path over one synthetic workload: trace ingestion (ticks, p(l), sorted
F), Algorithms 1-3 for every policy, token-by-token play-out, per-pair evaluation with the per-pair
arrays written (workloads 0 and 1), per-policy reductions and policy selection.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

`value` is measured with the trace arrays already resident in HBM; `e2e` goes through the same calls with
pinned host arrays (host->device copies and the statistics read-back inside the timed region).  With
N > 1 (torchrun) every rank evaluates an independent trace of the same shape (weak scaling, no
collective on the data path).  `--impl reference` times the CPU oracle on the host cores instead.
"""
import argparse
import json
import os
import statistics
import subprocess
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
SM_COUNT, SCHEDULERS, LANES = 148, 4, 32
MIN_WARMUP = 100             # untimed steps before either timed region, at the least
KERNEL_EVENT_STRIDE = 8      # per-kernel CUDA events are recorded on every 8th timed step
# DRAM bytes per launch from the committed ncu capture of the dominant kernel (None until captured for
# the current kernel; see profiles/).
NCU_TRAFFIC_BYTES = {"k_pairs_rows": 148985344, "k_pairs_acc": None, "k_playout_fast": 828160, "k_playout": None}


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


def oracle_sample_run(w, n_req, threads):
    """Times the oracle, as it stands, on the first n_req requests under every policy of w, one thread per
    contiguous request range.  Returns seconds."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import Oracle
    orc = oracle_sample_run.cache.get(id(w))
    if orc is None:
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
    probe = min(w.n, max(threads * 64, 2048))
    t = oracle_sample_run(w, probe, threads)
    return int(min(w.n, max(probe, probe * seconds / max(t, 1e-4))))


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
    toks = int(w.output_len[:n_req].sum()) * w.n_policies
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
    from paper_2502_11417_b200 import synth, Trace
    from paper_2502_11417_b200.api import policy_array, kernel_launch_count, PolicyStats, stats_view
    import ctypes

    w = synth.make_workload(args.config, n=args.requests, n_budgets=args.budgets, replica=rank)
    P, n = w.n_policies, w.n
    pols = policy_array(w.policies)
    host = [torch.from_numpy(x).pin_memory() for x in (w.prompt_len, w.output_len, w.server_ttft_s,
                                                       w.server_profile, w.device_profile)]
    dev = [x.cuda() for x in host]
    h2d = sum(x.numel() * x.element_size() for x in host) + P * ctypes.sizeof(pols[0])
    d2h = P * ctypes.sizeof(PolicyStats) + 8
    tr = Trace()
    tr.n = n
    out = None
    if w.materialise:
        tr.load_trace(*dev, w.servers, w.devices)
        out = tr.alloc_pair_outputs(P)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")       # larger than the 126 MB L2
    stream = torch.cuda.current_stream()
    tr.load_trace(*dev, w.servers, w.devices)
    cap_factor, slo = w.select["cost_cap_factor"], w.select["tbt_slo_s"]

    def step(arrays):
        tr.load_trace(*arrays, w.servers, w.devices, stream=stream)
        tr.eval_policies(pols, w.seed, out, stream=stream)
        st = tr.reduce_stats(stream=stream)
        cap = cap_factor * float(stats_view(st)["total_cost"].min())
        return tr.select_policy(cap, slo, stream=stream)

    def timed(arrays, steps, warmup, collect=None):
        for _ in range(warmup):
            step(arrays)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        evs = []
        for i in range(steps):
            flush.zero_()
            # the library's own events around its four big kernels cost about 45 us a step at workload 1 (they
            # keep neighbouring launches from overlapping), so they are recorded on every KERNEL_EVENT_STRIDE-th
            # timed step only
            sample = collect is not None and i % KERNEL_EVENT_STRIDE == 0
            tr.set_timing(sample)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            step(arrays)
            e1.record(stream)
            evs.append((e0, e1))
            if sample:
                collect.append(tr.timing())
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        return max_over_ranks(sum(a.elapsed_time(b) for a, b in evs), dist, "cuda")

    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    try:
        phys = int(vis.split(",")[local_rank]) if vis else local_rank
    except ValueError:
        phys = local_rank
    sampler = ClockSampler(phys)
    ktimes = []
    l0 = kernel_launch_count()
    # the first 75 or so steps of a fresh process run about 10 % slower (clocks and caches settling): at least
    # MIN_WARMUP untimed steps are run, whatever --warmup says; `warmup_run` in the output says how many
    warm = max(args.warmup, args.min_warmup)
    timed(dev, 0, warm)
    l_warm = kernel_launch_count()
    sampler.start()
    total_ms = timed(dev, args.steps, 0, ktimes)
    clocks = sampler.stop()
    launches = kernel_launch_count() - l_warm
    e2e_ms = timed(host, args.steps, warm)

    pairs = n * P * world
    toks = int(w.output_len.sum()) * P * world          # approximate for N > 1: replicas have like shapes
    value = whole_job_rate(n * P, world, args.steps, total_ms)
    e2e_value = whole_job_rate(n * P, world, args.steps, e2e_ms)

    # ---- roofline of the dominant kernel of a step
    hbm_gbs, sm_max_mhz, src = measured_peaks()
    names = ["k_playout_fast", "k_playout", "k_pairs_acc", "k_pairs_rows"]
    kms = {nm: statistics.mean(t[i] for t in ktimes) for i, nm in enumerate(names)}
    token_steps = int((w.output_len - 1).sum())
    n_classes = len({(float(np.float32(q["r_c"])), float(np.float32(q["t_m_s"])), int(q["flags"]) & 2) for q in w.policies})
    alu_peak = SM_COUNT * SCHEDULERS * LANES * sm_max_mhz * 1e6 / 1e12         # T lane-instructions/s
    alu_src = "148 SMs x 4 schedulers x 32 lanes x %.0f MHz (issue slots)" % sm_max_mhz
    per_token = PLAYOUT_INSTR_PER_TOKEN_LEAN if never_clamps(w) else PLAYOUT_INSTR_PER_TOKEN

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
                    "frac": ach / hbm_gbs,
                    "traffic": NCU_TRAFFIC_BYTES[name] if args.config == 1 and not args.requests else None,
                    "peak_source": src, "algorithmic_bytes": bytes_alg, "ms_per_launch": ms}
        if name == "k_pairs_acc":
            # pairs by kind: a (group, policy) waits when Algorithm 1 made the group device-constrained
            lane_instr, wait_pairs = 0, 0
            for g in range(tr.n_groups):
                n_g = tr.group_size(g)
                n_wait = sum(1 for p in range(P) if tr.prep(g, p).device_constrained)
                wait_pairs += n_g * n_wait
                lane_instr += n_g * (n_wait * PAIR_INSTR_WAIT + (P - n_wait) * PAIR_INSTR_NOWAIT)
            ach = lane_instr / (ms * 1e-3) / 1e12
            return {"kernel": name, "bound": "alu", "achieved": ach, "peak": alu_peak, "unit": "Tinstr/s",
                    "frac": ach / alu_peak, "traffic": None, "peak_source": alu_src,
                    "instr_per_pair": {"no_wait": PAIR_INSTR_NOWAIT, "wait": PAIR_INSTR_WAIT,
                                       "mean": lane_instr / float(n * P)},
                    "pairs_with_waits": wait_pairs, "ms_per_launch": ms}
        if name == "k_playout_fast":
            ach = token_steps * per_token / (ms * 1e-3) / 1e12
            return {"kernel": name, "bound": "alu", "achieved": ach, "peak": alu_peak, "unit": "Tinstr/s",
                    "frac": ach / alu_peak,
                    "traffic": NCU_TRAFFIC_BYTES[name] if args.config == 1 and not args.requests else None,
                    "peak_source": alu_src, "token_steps": token_steps, "instr_per_token_step": per_token,
                    "ms_per_launch": ms}
        return None                       # k_playout: only the requests the clamp-free kernel listed

    roofs = [r for r in (roof_of(nm) for nm in names) if r is not None]
    roof = dict(max(roofs, key=lambda r: r["ms_per_launch"]))
    roof["all_kernels"] = [{k: r[k] for k in ("kernel", "bound", "achieved", "peak", "unit", "frac", "ms_per_launch")}
                           for r in roofs]
    roof["kernels_ms"] = kms

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0
    cpu = None
    if world == 1 and args.oracle_seconds > 0:
        cores = os.cpu_count() or 1
        n_req = size_oracle_sample(w, cores, args.oracle_seconds)
        t = oracle_sample_run(w, n_req, cores)
        cpu = {"value": n_req * P / t, "unit": UNIT, "cores": min(cores, n_req), "kind": "oracle",
               "sample": "first %d of %d requests x all %d policies, %.1f s" % (n_req, n, P, t),
               "sim_tokens_per_s": int(w.output_len[:n_req].sum()) * P / t}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "warmup_run": warm, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "sim_tokens_per_s": toks * args.steps / (total_ms * 1e-3),
            # token-steps actually played: one play-out per request and timeline class (policies that share the
            # consumption rate, buffer size and pacing share it), whatever the number of policies
            "useful_token_steps_per_s": token_steps * n_classes * world * args.steps / (total_ms * 1e-3),
            "config": {"workload": w.name, "requests_per_gpu": n, "policies": P, "pairs_per_step": pairs,
                       "per_pair_outputs": bool(w.materialise), "l2": "flushed between steps (512 MB write)",
                       "kernel_events": "every %d-th timed step (%d samples)" % (KERNEL_EVENT_STRIDE, len(ktimes)),
                       "seed": w.seed},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms / args.steps},
            "gpu_launches": launches,
            "roofline": roof, "cpu_baseline": cpu}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--config", type=int, default=1, help="workload 0..5 (default: workload 1)")
    ap.add_argument("--requests", type=int, default=None, help="shrink the trace (profiling on a small case)")
    ap.add_argument("--budgets", type=int, default=None, help="shrink the budget axis (profiling on a small case)")
    ap.add_argument("--min-warmup", type=int, default=MIN_WARMUP,
                    help="untimed steps run at the least, whatever --warmup says (profiling runs pass a small number)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--oracle-seconds", type=float, default=15.0, help="CPU time of the oracle baseline sample")
    ap.add_argument("--oracle-step-seconds", type=float, default=3.0, help="--impl reference: CPU time per step")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
