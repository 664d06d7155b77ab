#!/usr/bin/env python
"""Benchmark of the dynamic block-sparse attention request path on B200.

A *step* is one complete request through the C ABI: ``bsa_plan_create`` (mask
state, statistics copy, regime lookup, launch preparation) followed by
``bsa_forward`` (attention kernel + Split-K merge) on synthetic vDiT-shaped
inputs already resident in HBM.  ``value`` is the effective TFLOP/s over the
active token pairs (4*d flops per pair) of that whole step.  The default
workload is the largest single-GPU configuration (HunyuanVideo-shaped: 24 heads,
115200 tokens, d = 128).  The same JSON line carries the forward-only
("kernel") figure with its roofline, the request breakdown, the other named
configurations under ``others`` and the 50-request dynamic sweep under ``sweep``.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload hunyuan|mid|...]
    python bench.py --impl reference   # the fp64 CPU oracle on a bounded sample
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
METRIC = "effective TFLOP/s on active blocks (4*d flops per active token pair)"
# dram__bytes_read.sum + dram__bytes_write.sum of ONE attention-kernel launch, from the ncu captures summarised under
# profiles/: {workload: (bytes, how the figure was obtained)}.  The Hunyuan-shaped launch is too large to capture
# whole under the pool's size rule; its figure is a 4-head capture of the same shape scaled by heads (the plan keeps
# heads apart in the queue, so traffic grows in proportion to them).
NCU_TRAFFIC_BYTES = {
    "hunyuan": (6 * 798.2e6, "ncu capture of one launch of the same shape at 4 heads (682.3 MB read + 116.0 MB written), x 24/4"),
    "mid": (206.5e6, "one ncu capture of one launch of this workload"),
    "stress_a": (266.9e6, "one ncu capture of one launch of this workload (row-block kernel)"),
}
KERNEL_NAMES = {0: "bsa_attention_kernel<D,TK,false>", 1: "bsa_attention_pair_kernel<D,TK>", 2: "bsa_attention_cs_kernel<D,TK>",
                3: "bsa_attention_kernel<D,TK,true>", 4: "bsa_attention_pp_kernel<D,TK,F16>", 5: "bsa_attention_rb_kernel<D,CK>"}
TENSOR_FLOP_PER_CLK_PER_SM = 8192  # dense bf16, fp32 accumulate


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs: NVML polled about every millisecond from a thread
    (read-only queries), or, where the NVML binding is missing, `nvidia-smi -lms 100`."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.thread = None
        self.stop_flag = False
        self.sm, self.mx, self.power, self.reasons = [], [], [], set()

    def _physical_index(self):
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        ids = [x for x in vis.split(",") if x.strip() != ""]
        if ids and self.idx < len(ids) and ids[self.idx].strip().isdigit():
            return int(ids[self.idx])
        return self.idx

    def _poll(self, nv, handle):
        bits = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown, "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown, "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
        while not self.stop_flag:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(handle)
                for name, bit in bits.items():
                    if r & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(handle) / 1000.0)
            except Exception:
                pass
            time.sleep(0.001)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            handle = nv.nvmlDeviceGetHandleByIndex(self._physical_index())
            self.mx.append(float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM)))
            import threading
            self.thread = threading.Thread(target=self._poll, args=(nv, handle), daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.thread is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
            return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_min_mhz": min(self.sm) if self.sm else None,
                    "sm_max_mhz": max(self.mx) if self.mx else None, "samples": len(self.sm),
                    "power_w_max": max(self.power) if self.power else None, "reasons": sorted(self.reasons), "source": "nvml"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "source": "nvidia-smi"}


def make_request(workload: str, rank: int, heads: int = 0):
    """The named workload; `heads` > 0 overrides its head count (a reduced copy of the same shape, e.g. for a profiler
    capture that must stay small)."""
    from paper_2609_25869_b200 import inputs as I
    kw = {"H": heads} if heads > 0 else {}
    if workload.startswith("sweep"):
        req = I.config_sweep(int(workload[5:] or 0) + 50 * rank, **kw)
    else:
        req = I.CONFIGS[workload](**kw)
    if rank:
        req.qkv_seed += 7919 * rank
    return req


def count_active_pairs(req) -> int:
    """In-range token pairs of E(M): the work the metric counts (4*d flops each).  Only the last block row and the
    last block column can be ragged."""
    import numpy as np
    n_kv = req.N_kv if req.N_kv > 0 else req.N
    rq = np.minimum(req.B_Q, req.N - np.arange(req.nQb) * req.B_Q).astype(np.int64)
    last_short = req.B_KV - (n_kv - (req.nKb - 1) * req.B_KV)           # tokens the last block column lacks
    cnt = np.count_nonzero(req.mask, axis=2).astype(np.int64)          # [H, nQb]
    keys = cnt * req.B_KV - (req.mask[:, :, -1] != 0).astype(np.int64) * last_short
    return int((keys * rq[None, :]).sum())


def oracle_sample(req, qkv, nblocks: int, seed: int = 123):
    """Time the CPU oracle as it stands on a bounded sample of query blocks."""
    from oracle import oracle
    from paper_2609_25869_b200 import inputs as I
    import numpy as np
    Qb, Kb, Vb = (I.bf16_bits(t) for t in qkv)
    per_head = max(1, nblocks // req.H)
    smp = I.sample_query_blocks(seed, req.H, req.nQb, per_head)
    sel = [(h, int(b)) for h in range(req.H) for b in smp[h]]
    t0 = time.perf_counter()
    _, _, pairs = oracle.attention_blocks(req.mask, req.B_Q, req.B_KV, req.N, req.d, Qb, Kb, Vb, sel)
    dt = time.perf_counter() - t0
    return pairs, dt, len(sel), oracle.num_threads()


def run_reference(args):
    """--impl reference: the oracle, unmodified, on host cores; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import oracle
    req = make_request(args.workload, 0, args.heads)
    qkv = req.qkv()
    nblocks = args.ref_blocks
    oracle_sample(req, qkv, min(nblocks, 8))  # builds/loads the library
    for _ in range(args.warmup):
        oracle_sample(req, qkv, nblocks)
    times, pairs = [], 0
    for _ in range(args.steps):
        pairs, dt, nsel, thr = oracle_sample(req, qkv, nblocks)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    val = 4.0 * req.d * pairs / (ms * 1e-3) / 1e12
    line = {
        "impl": "reference", "metric": METRIC,
        "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(req, args.workload),
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": thr, "kind": "oracle",
                         "sample": f"{nsel} of {req.H * req.nQb} query blocks per step ({pairs} active pairs)"},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def _gen_sweep_request(job):
    """Worker of the mask-generation pool (host only, no CUDA): one sweep request."""
    r, heads = job
    from paper_2609_25869_b200 import inputs as I
    req = I.config_sweep(r, H=heads)
    return r, req, count_active_pairs(req)


def start_sweep_generation(n_requests: int, heads: int):
    """Generates the sweep's masks in worker processes (forked BEFORE this process touches CUDA) while the main
    benchmarks run; returns (pool, ordered result iterator)."""
    import multiprocessing as mp
    # at most half of the cores, at low priority: the timed host path (statistics poll, launches) must not wait for a core
    workers = max(1, min(8, (os.cpu_count() or 2) // 2, n_requests))
    pool = mp.get_context("fork").Pool(workers, initializer=os.nice, initargs=(15,))
    return pool, pool.imap(_gen_sweep_request, [(r, heads) for r in range(n_requests)])


def sweep_block(gen, n_requests: int, heads: int, peaks):
    """Dynamic-request sweep (Section 7.1 timing protocol, Table 7's cold / warm / amortized view): every request is a
    cold unique request (a new mask): latency = bsa_plan_create (mask state, statistics, lookup, launch preparation)
    + bsa_forward + stream sync, host clock.  Then the median of 5 warm forwards of the prepared plan (after 3 warm-up
    forwards), and the destroy.  Before the timed requests one untimed request of the largest mask format sizes the
    memory pool, so that no timed request pays the driver for a first arena."""
    import torch
    from paper_2609_25869_b200 import bsa, inputs as I
    rows = []
    qkv = None
    O = L = None
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for i in range(n_requests):
        r, req, pairs = next(gen)
        if qkv is None:
            qkv = tuple(t.cuda() for t in req.qkv())  # tensors are reused; only the mask changes per request
            O = torch.empty_like(qkv[0])
            L = torch.empty((req.H, req.N), dtype=torch.float32, device="cuda")
            warm = I.config_sweep(1000, H=heads, B=(32, 32), rho=0.6)   # largest structures of the sweep
            wm = torch.from_numpy(warm.mask).cuda()
            with bsa.plan_create(wm, warm.B_Q, warm.B_KV, warm.N, warm.H, warm.d) as wp:
                wp.forward(*qkv, O, L)
                torch.cuda.synchronize()
            del wm, warm
        q, k, v = qkv
        mask = torch.from_numpy(req.mask).cuda()
        flush.fill_(i & 0xFF)
        torch.cuda.synchronize()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        t0 = time.perf_counter()
        e0.record()
        plan = bsa.plan_create(mask, req.B_Q, req.B_KV, req.N, req.H, req.d)
        e1.record()  # behind the plan's last preparation kernel: the plan is ready on the GPU when this event is
        t1 = time.perf_counter()
        plan.forward(q, k, v, O, L)
        e2.record()
        torch.cuda.synchronize()
        t2 = time.perf_counter()
        planning_us = e0.elapsed_time(e1) * 1e3
        cold_forward_us = e1.elapsed_time(e2) * 1e3
        for _ in range(3):
            plan.forward(q, k, v, O, L)
        ts = []
        for _ in range(5):  # warm exact repeats (prepared plan reused)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            plan.forward(q, k, v, O, L)
            b.record()
            b.synchronize()
            ts.append(a.elapsed_time(b))
        inf = plan.info()
        assert inf["device_status"] == 0
        t3 = time.perf_counter()
        plan.destroy()
        t4 = time.perf_counter()
        kern_ms = statistics.median(ts)
        cold_us = (t2 - t0) * 1e6
        rows.append({"r": r, "B": [req.B_Q, req.B_KV], "density": round(inf["density"], 4), "skew": round(inf["skew"], 2),
                     "plan": inf["plan"]["name"], "lut_hit": inf["lut_hit"], "cold_request_us": round(cold_us, 1),
                     "plan_create_us": round((t1 - t0) * 1e6, 1), "lookup_us": round(inf["us_lookup"], 2),
                     "planning_us": round(planning_us, 1), "cold_forward_us": round(cold_forward_us, 1),
                     "warm_forward_us": round(kern_ms * 1e3, 1), "destroy_us": round((t4 - t3) * 1e6, 1),
                     "tflops_warm": round(4.0 * req.d * pairs / (kern_ms * 1e-3) / 1e12, 1),
                     "covered_over_active": round(inf["covered_pairs"] / max(1, pairs), 3)})
        del mask
    cold = sorted(x["cold_request_us"] for x in rows)
    warm = sorted(x["warm_forward_us"] for x in rows)
    frac = [x["planning_us"] / (x["planning_us"] + x["cold_forward_us"]) for x in rows]

    def pct(xs, p):
        return xs[min(len(xs) - 1, int(round(p * (len(xs) - 1))))]

    def gm(xs):
        import math
        return math.exp(sum(math.log(max(x, 1e-9)) for x in xs) / len(xs))

    by_geom = {}
    for x in rows:
        by_geom.setdefault("%dx%d" % tuple(x["B"]), []).append(x["tflops_warm"])
    return {"protocol": "cold unique requests (new mask each): host clock around plan create + forward + sync; CUDA events split "
                        "it into planning (request start until the plan's last preparation kernel has finished, the host's "
                        "wait for the statistics and the lookup included) and the cold forward; then median of 5 warm "
                        "forwards after 3 warm-ups; one untimed request sizes the memory pool first",
            "workload": f"{len(rows)} requests, heads={heads} N=75600 d=128, B and density drawn per request",
            "cold_request_us": {"mean": statistics.mean(cold), "gm": gm(cold), "p50": pct(cold, 0.5), "p95": pct(cold, 0.95),
                                "max": cold[-1]},
            "warm_forward_us": {"gm": gm(warm), "p50": pct(warm, 0.5), "p95": pct(warm, 0.95)},
            "cold_over_warm_gm": gm([x["cold_request_us"] / x["warm_forward_us"] for x in rows]),
            "amortized4_over_warm_gm": gm([(x["cold_request_us"] + 3 * x["warm_forward_us"]) / 4 / x["warm_forward_us"] for x in rows]),
            "plan_create_host_us": {"mean": statistics.mean(x["plan_create_us"] for x in rows),
                                    "max": max(x["plan_create_us"] for x in rows)},
            "lookup_us_mean": statistics.mean(x["lookup_us"] for x in rows),
            "planning_us": {"mean": statistics.mean(x["planning_us"] for x in rows), "max": max(x["planning_us"] for x in rows)},
            "planning_fraction": {"mean": statistics.mean(frac), "max": max(frac)},
            "destroy_us_mean": statistics.mean(x["destroy_us"] for x in rows),
            "tflops_warm_mean": statistics.mean(x["tflops_warm"] for x in rows),
            "tflops_warm_gm_by_geometry": {k: round(gm(v), 1) for k, v in sorted(by_geom.items())},
            "frac_of_peak_warm_mean": statistics.mean(x["tflops_warm"] for x in rows) / peaks["bf16_tflops"],
            "lut_hits": sum(x["lut_hit"] for x in rows), "requests": rows}


def run_sweep(args):
    """--workload sweep: the sweep block alone, as one JSON line."""
    pool, gen = start_sweep_generation(args.sweep_requests, args.sweep_heads)
    import torch
    from paper_2609_25869_b200 import bsa
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    bsa.lib()
    blk = sweep_block(gen, args.sweep_requests, args.sweep_heads, load_peaks())
    pool.terminate()
    line = {"metric": "per-request us incl. planning (cold unique requests), dynamic-request sweep", "unit": "us",
            "value": blk["cold_request_us"]["mean"], "higher_is_better": False, "n_gpus": 1, "dtype": "bf16",
            "data": "synthetic", "config": {"workload": "sweep: " + blk["workload"]}, "sweep": blk}
    print(json.dumps(line), flush=True)


def aggregate_over_ranks(step_ms: float, flops_per_rank: float, dist=None, device="cuda"):
    """Weak scaling by replication: every rank runs its own request, no data-path collective.
    The job's time is the MAX over ranks; the job's work is the SUM.  Returns (max_ms, total TFLOP/s)."""
    world = 1
    if dist is not None and dist.is_initialized():
        import torch
        world = dist.get_world_size()
        t = torch.tensor([step_ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        step_ms = float(t.item())
        f = torch.tensor([flops_per_rank], dtype=torch.float64, device=device)
        dist.all_reduce(f, op=dist.ReduceOp.SUM)
        total = float(f.item())
    else:
        total = flops_per_rank
    return step_ms, total / (step_ms * 1e-3) / 1e12, world


def workload_config(req, name):
    return {"workload": f"{name}: heads={req.H} N={req.N} d={req.d} B=({req.B_Q},{req.B_KV}) {req.note}",
            "l2": "256 MiB buffer written between timed iterations (L2 flush)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="hunyuan",
                    help="hunyuan (default: the largest single-GPU configuration), mid, tiny, stress_a, stress_b, sweepN, sweep")
    ap.add_argument("--plan", type=int, default=-1, help="force a catalog plan id (-1: Algorithm 2)")
    ap.add_argument("--heads", type=int, default=0, help="override the workload's head count (reduced copies for profiler captures)")
    ap.add_argument("--lut", default="", help="plan table to load instead of the packaged one")
    ap.add_argument("--ref-blocks", type=int, default=256, help="query blocks per reference step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--extra", default="tiny,mid,stress_a,stress_b", help="comma list of workloads reported under 'others'")
    ap.add_argument("--no-sweep", action="store_true", help="leave the dynamic-request sweep block out")
    ap.add_argument("--sweep-requests", type=int, default=50)
    ap.add_argument("--sweep-heads", type=int, default=24)
    ap.add_argument("--shard-heads", action="store_true",
                    help="strong scaling: ONE request, its heads split over the ranks (no collective on the data path)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return
    if args.workload == "sweep":
        run_sweep(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    # the sweep block and the other configurations belong to the single-GPU line only
    with_sweep = world == 1 and not args.no_sweep and not args.shard_heads and args.sweep_requests > 0
    pool = gen = None
    if with_sweep:
        pool, gen = start_sweep_generation(args.sweep_requests, args.sweep_heads)  # before CUDA is initialised

    import torch
    from paper_2609_25869_b200 import bsa
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    bsa.lib()  # fail loudly if the CUDA library is missing; loads the packaged plan table if it matches the catalog
    if args.lut:
        bsa.lut_load(args.lut)
    lut_regimes = int(bsa.lib().bsa_lut_num_regimes())
    peaks = load_peaks()
    num_sms = torch.cuda.get_device_properties(local_rank).multi_processor_count

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def bench_workload(name, steps, warmup, primary):
        req = make_request(name, 0 if args.shard_heads else rank, args.heads if primary else 0)
        q, k, v = req.qkv()
        if args.shard_heads:  # every rank builds the same request and keeps its own contiguous range of heads
            import dataclasses
            from paper_2609_25869_b200 import shard
            lo, hi = shard.head_range(req.H, rank, world)
            if hi == lo:
                raise SystemExit(f"--shard-heads: {req.H} heads cannot feed {world} ranks")
            q, k, v = (t[lo:hi].contiguous() for t in (q, k, v))
            req = dataclasses.replace(req, H=hi - lo, mask=req.mask[lo:hi].copy(),
                                      note=req.note + f"; heads {lo}-{hi - 1} of {req.H} on this rank")
        mask_d = torch.from_numpy(req.mask).cuda()
        qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
        O = torch.empty_like(qd)
        LSE = torch.empty((req.H, req.N), dtype=torch.float32, device="cuda")
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        stream = torch.cuda.current_stream()
        pairs = count_active_pairs(req)
        flops = 4.0 * req.d * pairs

        def step(ready=None):
            plan = bsa.plan_create(mask_d, req.B_Q, req.B_KV, req.N, req.H, req.d, plan_id=args.plan, stream=stream)
            if ready is not None:
                ready.record(stream)  # behind the plan's last preparation kernel
            plan.forward(qd, kd, vd, O, LSE, stream=stream)
            return plan

        for _ in range(warmup):
            step().destroy()
        barrier()
        sampler = ClockSampler(local_rank)
        sampler.start()
        launches0 = bsa.kernel_launch_count()
        ev = [tuple(torch.cuda.Event(enable_timing=True) for _ in range(2)) for _ in range(steps)]
        host_us, destroy_us = [], []
        plan = None
        for i in range(steps):
            flush.fill_(i & 0xFF)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            ev[i][0].record(stream)
            plan = step()
            ev[i][1].record(stream)
            ev[i][1].synchronize()
            t1 = time.perf_counter()
            host_us.append((t1 - t0) * 1e6)
            if i + 1 < steps:  # giving the plan back is not part of the request; its host cost is reported beside it
                plan.destroy()
                destroy_us.append((time.perf_counter() - t1) * 1e6)
        barrier()
        launches = bsa.kernel_launch_count() - launches0
        step_ms = [a.elapsed_time(b) for a, b in ev]
        info = plan.info()
        # Planning share: a few more requests with an event between create and forward (request start -> the plan's
        # last preparation kernel finished, the host's wait for the statistics and the lookup included).  Kept out of
        # the timed steps: an event in front of the attention kernel takes away its dependent-launch overlap.
        plan_ms = []
        for i in range(min(steps, 5)):
            flush.fill_(i & 0xFF)
            torch.cuda.synchronize()
            a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            p2 = step(c)
            c.synchronize()
            plan_ms.append(a.elapsed_time(c))
            torch.cuda.synchronize()
            p2.destroy()
        # forward only (warm plan): the attention kernel (+ merge) timed alone, L2 flushed in between
        kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for _ in range(3):
            plan.forward(qd, kd, vd, O, LSE)
        for i in range(steps):
            flush.fill_(i & 0xFF)
            kev[i][0].record(stream)
            plan.forward(qd, kd, vd, O, LSE)
            kev[i][1].record(stream)
        torch.cuda.synchronize()
        clocks = sampler.stop()
        k_ms = [a.elapsed_time(b) for a, b in kev]
        res = {"req": req, "pairs": pairs, "flops": flops, "step_ms": sum(step_ms) / len(step_ms),
               "step_ms_median": statistics.median(step_ms), "host_us": statistics.median(host_us),
               "planning_ms": statistics.median(plan_ms), "planning_ms_all": [round(x, 4) for x in plan_ms],
               "destroy_us": statistics.median(destroy_us) if destroy_us else None,
               "kernel_ms": sum(k_ms) / len(k_ms), "kernel_ms_median": statistics.median(k_ms), "info": info,
               "launches": launches, "clocks": clocks, "qkv": (q, k, v)}
        if info["plan"]["split_pmax"] > 1 and info["nsplit_rows"] > 0:
            # the Split-K reduction kernel alone (HBM-bound), over the partials the forwards above left behind
            mev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for i in range(steps):
                flush.fill_(i & 0xFF)
                mev[i][0].record(stream)
                plan.merge_only(O, LSE, stream=stream)
                mev[i][1].record(stream)
            torch.cuda.synchronize()
            m_ms = statistics.mean(a.elapsed_time(b) for a, b in mev)
            rows_total = req.H * info["nQt"] * info["member_words"]
            parts = info["nitems"] * info["member_words"] - (rows_total - info["nsplit_rows"])  # 128-row partial slots merged
            rd = parts * 128 * (req.d + 1) * 4
            wr = info["nsplit_rows"] * 128 * (2 * req.d + 4)
            res["merge"] = {"kernel": "bsa_merge_kernel<D>", "launch_ms": m_ms, "merged_tile_rows": info["nsplit_rows"],
                            "partials": parts, "algorithmic_bytes": rd + wr, "bound": "hbm",
                            "achieved": (rd + wr) / (m_ms * 1e-3) / 1e9, "unit": "GB/s", "peak": peaks["hbm_gbs"],
                            "frac": (rd + wr) / (m_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        if primary:
            # warm request: the mask repeats, the plan cache recognises it (statistics kernel with the mask
            # fingerprint) and only the forward follows.  Reported beside the cold request; `value` stays the cold one.
            cache = bsa.PlanCache(4)
            cache.get(mask_d, req.B_Q, req.B_KV, req.N, req.H, req.d, plan_id=args.plan)[0].destroy()
            wev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            hits = 0
            for i in range(steps + 3):
                flush.fill_(i & 0xFF)
                torch.cuda.synchronize()
                if i >= 3:
                    wev[i - 3][0].record(stream)
                wp, hit = cache.request(mask_d, req.B_Q, req.B_KV, req.N, req.H, req.d, qd, kd, vd, O, LSE,
                                        plan_id=args.plan, stream=stream)
                if i >= 3:
                    wev[i - 3][1].record(stream)
                hits += int(hit)
                wp.destroy()
            torch.cuda.synchronize()
            assert hits == steps + 3
            cache.destroy()
            w_ms = [a.elapsed_time(b) for a, b in wev]
            res["warm_ms"] = sum(w_ms) / len(w_ms)
        # Last, because it heats the GPU into its power cap: back-to-back forwards (no flush) for at least 250 ms with the
        # clock sampled underneath, for the fraction of the tensor pipe's issue capacity at the clock the kernel actually
        # ran at, whatever the power state.
        kern_s = res["kernel_ms"] * 1e-3
        reps = max(3, min(20000, int(0.25 / max(kern_s, 1e-6)) + 1))
        cs = ClockSampler(local_rank)
        torch.cuda.synchronize()
        cs.start()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            plan.forward(qd, kd, vd, O, LSE)
        b.record(stream)
        b.synchronize()
        cl = cs.stop()
        bb_ms = a.elapsed_time(b) / reps
        res["back_to_back"] = {"launch_ms": bb_ms, "launches": reps, "sm_mhz": cl.get("sm_mhz"),
                               "sm_min_mhz": cl.get("sm_min_mhz"), "power_w_max": cl.get("power_w_max"),
                               "reasons": cl.get("reasons"), "tflops": flops / (bb_ms * 1e-3) / 1e12}
        if cl.get("sm_mhz"):
            res["back_to_back"]["frac_of_tensor_issue_at_clock"] = flops / (
                bb_ms * 1e-3 * cl["sm_mhz"] * 1e6 * num_sms * TENSOR_FLOP_PER_CLK_PER_SM)
        info2 = plan.info()
        assert info2["device_status"] == 0, "a bounded device wait expired during the bench"
        plan.destroy()
        if primary:
            qp, kp, vp = q.pin_memory(), k.pin_memory(), v.pin_memory()
            Oh = torch.empty_like(q).pin_memory()
            Lh = torch.empty((req.H, req.N), dtype=torch.float32).pin_memory()
            mh = torch.from_numpy(req.mask).pin_memory()
            for _ in range(2):
                bsa.request_host(mh, req.B_Q, req.B_KV, req.N, req.H, req.d, qp, kp, vp, Oh, Lh, plan_id=args.plan)
            ts = []
            for _ in range(max(3, min(10, steps // 2))):
                barrier()
                t0 = time.perf_counter()
                bsa.request_host(mh, req.B_Q, req.B_KV, req.N, req.H, req.d, qp, kp, vp, Oh, Lh, plan_id=args.plan)
                ts.append(time.perf_counter() - t0)
            res["e2e_s"] = sum(ts) / len(ts)
            res["h2d"] = req.mask.nbytes + 3 * q.numel() * 2
            res["d2h"] = q.numel() * 2 + req.H * req.N * 4
            del qp, kp, vp, Oh, Lh, mh
        del mask_d, qd, kd, vd, O, LSE, flush
        torch.cuda.empty_cache()
        return res

    r = bench_workload(args.workload, args.steps, args.warmup, True)
    req = r["req"]

    def maxr(x):
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    step_ms, value, _ = aggregate_over_ranks(r["step_ms"], r["flops"], dist)
    kernel_ms = maxr(r["kernel_ms"])
    e2e_s = maxr(r["e2e_s"])
    kernel_tflops = r["flops"] / (kernel_ms * 1e-3) / 1e12
    inf = r["info"]
    # The kernel is timed alone, launch by launch, so the denominator is the burst figure; a ten-millisecond launch
    # runs under the 1 kW power cap like the seconds-long GEMM loop behind the "sustained" figure, which is given too.
    peak_key = "bf16_tflops"
    base_name = args.workload.rstrip("0123456789") if args.workload.startswith("sweep") else args.workload
    traffic = NCU_TRAFFIC_BYTES.get(base_name) if not args.heads and args.plan < 0 else None  # the captured launch only
    line = {
        "metric": METRIC,
        "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": step_ms, "higher_is_better": True, "scaling": "strong" if args.shard_heads else "weak",
        "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": workload_config(req, args.workload),
        "step": "one whole cold request: bsa_plan_create (mask state, statistics, lookup, launch preparation) + bsa_forward",
        "clocks": r["clocks"],
        "e2e": {"value": world * r["flops"] / e2e_s / 1e12, "unit": "TFLOP/s",
                "h2d_bytes_per_step": r["h2d"], "d2h_bytes_per_step": r["d2h"], "ms_per_request": e2e_s * 1e3},
        "gpu_launches": r["launches"],
        "roofline": {"bound": "tensor", "kernel": KERNEL_NAMES.get(inf["plan"]["kernel"], "?"), "plan": inf["plan"]["name"],
                     "achieved": kernel_tflops, "peak": peaks[peak_key], "unit": "TFLOP/s",
                     "frac": kernel_tflops / peaks[peak_key],
                     "peak_kind": "burst dense bf16 matmul, " + peaks["_source"],
                     "frac_of_burst": kernel_tflops / peaks["bf16_tflops"],
                     "frac_of_sustained": kernel_tflops / peaks["bf16_tflops_sustained"],
                     "traffic": traffic[0] if traffic else None, "traffic_source": traffic[1] if traffic else None,
                     "launch_ms": kernel_ms, "flops_per_launch": r["flops"],
                     "covered_over_active": inf["covered_pairs"] / max(1, r["pairs"]),
                     "back_to_back": r["back_to_back"]},
        "request": {"us_per_request_gpu": step_ms * 1e3, "us_per_request_host_median": r["host_us"],
                    "us_forward": kernel_ms * 1e3, "us_per_warm_request_gpu": maxr(r["warm_ms"]) * 1e3,
                    "warm_request_tflops": world * r["flops"] / (maxr(r["warm_ms"]) * 1e-3) / 1e12,
                    "us_plan_create_host": inf["us_total"], "us_plan_destroy_host": r["destroy_us"],
                    "us_mask_state": inf["us_mask_state"], "us_stats_sync": inf["us_stats_sync"],
                    "us_lookup": inf["us_lookup"], "us_launch_prep": inf["us_launch_prep"],
                    "us_planning_gpu": r["planning_ms"] * 1e3, "us_planning_gpu_samples": [x * 1e3 for x in r["planning_ms_all"]],
                    "planning_fraction": r["planning_ms"] / r["step_ms"],
                    "plan": inf["plan"]["name"], "lut_hit": inf["lut_hit"], "lut_regimes": lut_regimes,
                    "ntiles": inf["ntiles"],
                    "nitems": inf["nitems"], "active_pairs": r["pairs"], "covered_pairs": inf["covered_pairs"],
                    "density": inf["density"]},
    }
    if "merge" in r:
        line["merge"] = r["merge"]
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        nb = req.H * req.nQb if args.workload in ("tiny", "mid") else 2048
        pairs, dt, nsel, thr = oracle_sample(req, r["qkv"], nb)
        line["cpu_baseline"] = {"value": 4.0 * req.d * pairs / dt / 1e12, "unit": "TFLOP/s", "cores": thr,
                                "kind": "oracle", "seconds": dt,
                                "sample": f"{nsel} of {req.H * req.nQb} query blocks ({pairs} active pairs)"}
    r.pop("qkv", None)
    others = {}
    if world == 1 and not args.shard_heads:
        for name in [x for x in args.extra.split(",") if x and x != args.workload]:
            o = bench_workload(name, 10, 3, False)
            oi = o["info"]
            kt = o["flops"] / (o["kernel_ms"] * 1e-3) / 1e12
            others[name] = {"workload": workload_config(o["req"], name)["workload"],
                            "kernel_tflops": kt, "kernel_ms": o["kernel_ms"], "request_ms": o["step_ms"],
                            "request_tflops": o["flops"] / (o["step_ms"] * 1e-3) / 1e12,
                            "frac_of_burst": kt / peaks["bf16_tflops"],
                            "planning_fraction": o["planning_ms"] / o["step_ms"],
                            "covered_over_active": oi["covered_pairs"] / max(1, o["pairs"]),
                            "plan": oi["plan"]["name"], "us_plan_create_host": oi["us_total"], "us_lookup": oi["us_lookup"],
                            "sm_mhz": o["clocks"].get("sm_mhz"), "back_to_back": o["back_to_back"]}
            o.pop("qkv", None)
    if others:
        line["others"] = others
    if with_sweep:
        line["sweep"] = sweep_block(gen, args.sweep_requests, args.sweep_heads, peaks)
        pool.terminate()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
