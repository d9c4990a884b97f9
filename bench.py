#!/usr/bin/env python
"""Benchmark of the CO3 gradient pipeline on B200.

A step is one CO3 iteration of Algorithm 1 over one batch of synthetic gradients: co3_encode
(error-feedback add, float conversion, residual update, histogram and moments, GenNorm fit,
Huffman code build, bit packing) followed by co3_decode_aggregate (code rebuild from the header,
decode of all users, average).  The workload is the 8-user ResNet-18-sized configuration
(d = 11,173,962 per user, 62 layers, 8-bit format, gamma = 0.9).  `value` is measured with the bias of
every iteration taken from that iteration's own moments, as Algorithm 1 prints it; the library gets those
results without a statistics pass in every iteration (it converts under the previous bias and converts
again the layers whose bias changed).  The same steps with that pass in every iteration
(`current_two_pass`, the same bits) and with the bias lagging one iteration behind (`lagged_bias`)
are timed beside it.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Metric: GB/s of fp32 gradient consumed = 4 * d * U * steps / time, inputs resident in HBM.
With N > 1 (torchrun) every rank runs an independent replica of the workload: the path has no
exchange step, so there is no collective on the data path.
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "co3_encode_decode_fp32_gradient_throughput"
UNIT = "GB/s"
POOL = 4                      # distinct gradient batches cycled through (each > L2)
# algorithmic bytes per user-element of the fused convert pass: read g, m (8), write m (4), symbol (1)
CONVERT_BYTES_PER_ELEMENT = 13.0
CONVERT_TIMED_EVERY = 4          # the convert launches of the timed region that carry an event pair
SUSTAINED_MS = 2000.0             # device time of the sustained leg


def convert_dram_traffic(n_users):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the convert kernel, from the figures of
    the one-pass ncu capture on the full 8-user workload that are kept beside its summary; the traffic
    grows in proportion with the number of users.  None if the file is missing."""
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "dram_traffic_config1_8users.json")))
        return float(rec["convert_dram_bytes_per_launch"]) * n_users / float(rec["n_users"])
    except Exception:
        return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (earlier pool measurement)"


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake", 0x2: "applications_clocks_setting",
               0x100: "display_clock_setting", 0x10: "sync_boost"}

    def __init__(self, index, period=0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_min_mhz": min(self.samples),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def max_over_ranks(ms, world, device):
    """A job of independent replicas is as slow as its slowest one: the maximum over all ranks of a
    device-timed interval (milliseconds).  `device` is where the exchanged scalar lives ("cuda" under
    NCCL, "cpu" under gloo)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput_gbs(world, bytes_per_replica_step, steps, ms):
    """Whole-job GB/s: every replica processes bytes_per_replica_step per step in the same time."""
    return world * bytes_per_replica_step * steps / (ms * 1e-3) / 1e9


def replica_workload(rank, n_users=None):
    """Configuration 1 for replica `rank`: same shapes, its own users' gradients (seed offset)."""
    from paper_2203_09044_b200 import inputs
    wl = inputs.workload(1, n_users=n_users).align_rows()
    wl.index = wl.index + 100 * rank
    return wl


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2203_09044_b200 import binding, inputs

    binding.lib()                                      # no CUDA library -> raise, never fall back
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    wl = replica_workload(rank, args.users)            # a weak-scaling replica: its own users' gradients
    U, d = wl.n_users, wl.d
    mode = {"lagged": binding.BIAS_LAGGED, "current": binding.BIAS_CURRENT,
            "code-lagged": binding.CODE_LAGGED}[args.mode]
    plan = binding.Plan(d, U, wl.exp_bits, wl.mant_bits, wl.seg_offsets, gamma=wl.gamma,
                        bias_mode=mode, ld=wl.ld)
    out = plan.alloc_outputs()
    residual = torch.zeros((U, plan.ld), dtype=torch.float32, device="cuda")
    pool = [wl.gradient(t, device="cuda") for t in range(POOL)]
    torch.cuda.synchronize()

    def step(t):
        plan.encode(pool[t % POOL], residual, out)
        plan.decode_aggregate(out)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for t in range(args.warmup):
        step(t)
    barrier()
    flags, _ = plan.status(clear=True)
    assert flags == 0, f"status flags {flags} after warm-up"

    # ---- timed region: K steps, the dominant kernel traced with CUDA events --------------------
    # A steady-state step is a fixed sequence of memsets and kernels with no host decision in it, so
    # it is captured once per gradient batch in a CUDA graph.  Every CONVERT_TIMED_EVERY-th step of the
    # timed region is launched eagerly with an event pair around its convert launch (the roofline
    # figure); the steps between are graph replays, which save the launch gaps between the dependent
    # kernels.  --no-graph launches every step eagerly.
    graphs = None
    per_step_launches = 0
    if not args.no_graph:
        graphs = []
        for i in range(POOL):
            n0 = plan.launch_count()
            gr = torch.cuda.CUDAGraph()
            # thread_local: only this thread launches; another thread (NCCL's watchdog) may query events
            with torch.cuda.graph(gr, capture_error_mode="thread_local"):
                step(i)
            per_step_launches = plan.launch_count() - n0
            graphs.append(gr)
        barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_loop(n_steps, first_t):
        """n_steps steps between two events, the convert launch of every eager step event-timed, NVML
        clock samples taken meanwhile.  Returns (ms, launches, convert ms, convert launches timed, clocks)."""
        plan.profile_enable(["convert"], max_records=n_steps)
        plan.profile_stride(1 if graphs else CONVERT_TIMED_EVERY)
        sampler = ClockSampler(physical_gpu_index(local_rank))
        launches0 = plan.launch_count()
        replays = 0
        barrier()
        sampler.start()
        e0.record()
        for t in range(n_steps):
            if graphs is None or t % CONVERT_TIMED_EVERY == 0:
                step(first_t + t)
            else:
                graphs[(first_t + t) % POOL].replay()
                replays += 1
        e1.record()
        barrier()
        clk = sampler.stop()
        ms = e0.elapsed_time(e1)
        n_launch = plan.launch_count() - launches0 + replays * per_step_launches
        c_ms, c_n = plan.profile_collect()["convert"]
        f, _ = plan.status(clear=True)
        assert f == 0, f"status flags {f} in the timed region"
        return ms, n_launch, c_ms, c_n, clk

    elapsed_ms, launches, conv_ms, conv_n, clocks = timed_loop(args.steps, args.warmup)
    # ---- sustained leg: the same loop for about two seconds of device time --------------------
    # (a timed region of a few milliseconds is a burst figure and meets at most one clock sample)
    sus_steps = args.steps if args.short else max(args.steps, int(SUSTAINED_MS / max(elapsed_ms / args.steps, 1e-3)) + 1)
    sus_ms, _, sus_conv_ms, sus_conv_n, sus_clocks = timed_loop(sus_steps, args.warmup + args.steps)
    sus_ms = max_over_ranks(sus_ms, world, "cuda")
    code_bits = float(out["user_bits"].sum().item()) / (U * d)
    container_bits = (32.0 * float(out["chunk_off"][:, -1].sum().item()) + 16.0 * U * plan.n_sub
                      + 32.0 * U * (plan.n_chunks + 1) + 32.0 * plan.S) / (U * d)

    elapsed_ms = max_over_ranks(elapsed_ms, world, "cuda")

    # ---- per-kernel breakdown: the same steps again with every kernel class traced -----------
    plan.profile_stride(1)
    nb = min(args.steps, 50)
    plan.profile_enable(None, max_records=2 * nb + 4)
    for t in range(nb):
        step(args.warmup + args.steps + t)
    breakdown = {k: {"ms_per_step": v[0] / nb, "launches_per_step": v[1] / nb}
                 for k, v in plan.profile_collect().items() if v[1]}
    plan.profile_enable([], 0)

    # ---- the other bias mode, timed the same way (K steps, eager) ------------------------------
    other = None if args.short else {"current": "lagged", "lagged": "current"}.get(args.mode)
    other_rec = None
    two_pass_rec = None

    def timed_other(other, two_pass):
        """K steps of another bias mode (or of the current-moments bias in its two-pass form: a statistics pass
        in every iteration, CO3_TWO_PASS=1 when the plan is made), graph-replayed like the main loop."""
        if two_pass:
            os.environ["CO3_TWO_PASS"] = "1"
        try:
            plan_o = binding.Plan(d, U, wl.exp_bits, wl.mant_bits, wl.seg_offsets, gamma=wl.gamma,
                                  bias_mode={"lagged": binding.BIAS_LAGGED, "current": binding.BIAS_CURRENT}[other],
                                  ld=wl.ld)
        finally:
            os.environ.pop("CO3_TWO_PASS", None)
        res_o = torch.zeros_like(residual)
        for t in range(args.warmup):
            plan_o.encode(pool[t % POOL], res_o, out)
            plan_o.decode_aggregate(out)
        gr_o = []
        for i in range(POOL if not args.no_graph else 0):
            g_o = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_o, capture_error_mode="thread_local"):
                plan_o.encode(pool[i], res_o, out)
                plan_o.decode_aggregate(out)
            gr_o.append(g_o)
        barrier()
        e0.record()
        for t in range(args.steps):
            if gr_o:
                gr_o[t % POOL].replay()
            else:
                plan_o.encode(pool[t % POOL], res_o, out)
                plan_o.decode_aggregate(out)
        e1.record()
        barrier()
        o_ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
        assert plan_o.status(clear=True)[0] == 0
        rec = {"bias_mode": other, "ms_per_step": o_ms / args.steps,
               "value": job_throughput_gbs(world, 4.0 * d * U, args.steps, o_ms), "unit": UNIT,
               "launch": "replayed from one-step CUDA graphs" if gr_o else "launched eagerly"}
        if two_pass:
            rec["note"] = ("a statistics pass in every iteration (Algorithm 1 line 8 in its printed order); the same "
                           "bits as `value`, whose iterations convert under the previous bias and convert again "
                           "only the layers whose bias changed")
        del gr_o
        plan_o.close()
        del res_o
        return rec

    if other is not None:
        other_rec = timed_other(other, False)
        two_pass_rec = timed_other("current", True)

    # ---- the same steps replayed from a CUDA graph (one graph = one pass over the gradient pool) --
    # All steps from one graph, no eager step in between: what the loop costs without any launch gap.
    graph_ms = None
    if world == 1 and not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, capture_error_mode="thread_local"):
            for t in range(POOL):
                step(t)
        n_rep = max(1, args.steps // POOL)
        for _ in range(2):
            graph.replay()
        barrier()
        e0.record()
        for _ in range(n_rep):
            graph.replay()
        e1.record()
        barrier()
        graph_ms = e0.elapsed_time(e1) / (n_rep * POOL)
        flags, _ = plan.status(clear=True)
        assert flags == 0, f"status flags {flags} in the graph replay"

    # ---- end to end: host gradients in, host average out, through co3_iteration_host ---------
    ne = min(args.steps, 20)
    h_pool = [g.cpu().pin_memory() for g in pool[:2]]
    h_avg = torch.empty(d, dtype=torch.float32).pin_memory()
    d_grad = torch.empty((U, plan.ld), dtype=torch.float32, device="cuda")
    for t in range(3):
        plan.iteration_host(h_pool[t % 2], d_grad, residual, out, h_avg)
    barrier()
    e0.record()
    for t in range(ne):
        plan.iteration_host(h_pool[t % 2], d_grad, residual, out, h_avg)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms, world, "cuda")
    flags, _ = plan.status(clear=True)
    assert flags == 0

    in_bytes = 4.0 * d * U
    value = job_throughput_gbs(world, in_bytes, args.steps, elapsed_ms)
    e2e_value = job_throughput_gbs(world, in_bytes, ne, e2e_ms)
    peak, peak_src = measured_peaks()
    conv_avg_ms = conv_ms / max(conv_n, 1)
    # bytes the dominant kernel must move per user-element: g, m in, m out, and the symbol (two-pass
    # modes) or the packed codewords (single-pass mode) out
    conv_bytes = CONVERT_BYTES_PER_ELEMENT if args.mode != "code-lagged" else 12.0 + code_bits / 8.0
    achieved = conv_bytes * U * d / (conv_avg_ms * 1e-3) / 1e9
    # all passes of one iteration, E4M3: 13 + 1.9 (encode) + 0.87 (decode) per user-element + the average
    # (the current-moments bias pays a statistics pass at t = 0 only: later iterations run the lagged-bias
    # passes and convert again the layers whose bias changed -- on this workload five of 64-128 elements)
    per_ue = {"lagged": 15.9, "current": 15.9, "code-lagged": 12.0 + 4.0 * code_bits / 8.0}[args.mode]
    step_bytes = (per_ue * U + 4.0) * d

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "configs[1]: %d users x ResNet-18 (10-class head) gradient, d=11173962, "
                               "62 layers, iid GenNorm(beta=0.8) per layer, E4M3, gamma=0.9, %s" % (
                                   U, {"lagged": "lagged bias", "current": "bias from the current moments (Algorithm 1 as printed)",
                                       "code-lagged": "lagged bias and code (single-pass encode)"}[args.mode]),
                   "d": d, "n_users": U, "n_segments": plan.S, "format": "E4M3", "gamma": wl.gamma,
                   "bias_mode": args.mode, "replicas": world, "row_stride": plan.ld,
                   "launch": ("every step launched eagerly" if graphs is None else
                              "every %d-th step launched eagerly (its convert launch event-timed), the others "
                              "replayed from one-step CUDA graphs" % CONVERT_TIMED_EVERY),
                   "l2": "inputs larger than L2: %d MB of gradient+memory read per step, %d gradient "
                         "batches cycled" % (8 * U * d // 1000000, POOL)},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(4 * U * plan.ld),
                "d2h_bytes_per_step": int(4 * d), "steps": ne, "ms_per_step": e2e_ms / ne,
                "call": "co3_iteration_host (pinned host gradients in, host average out)"},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "ef_kernel<convert> (fused EF-add/convert/residual/histogram/moments)"
                               if args.mode != "code-lagged" else
                               "ef_kernel<convert+pack> (EF-add/convert/residual/histogram/moments/codeword packing)",
                     "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": peak_src,
                     "traffic": convert_dram_traffic(U) if args.mode != "code-lagged" else None,
                     "traffic_source": "profiles/dram_traffic_config1_8users.json (one-pass ncu capture, scaled by users)",
                     "algorithmic_bytes_per_launch": conv_bytes * U * d,
                     "avg_launch_ms": conv_avg_ms, "launches_timed": conv_n,
                     "timing": "cudaEvent pair around the convert launch of every %d-th step, on the launching "
                               "stream, inside the timed region" % CONVERT_TIMED_EVERY},
        "elements_per_s": world * U * d * args.steps / (elapsed_ms * 1e-3),
        "bits_per_element": {"code": code_bits, "container": container_bits},
        "whole_step_hbm": {"algorithmic_bytes_per_step": step_bytes,
                           "achieved_GBps": step_bytes * args.steps / (elapsed_ms * 1e-3) / 1e9,
                           "frac_of_peak": step_bytes * args.steps / (elapsed_ms * 1e-3) / 1e9 / peak},
        "kernels": breakdown,
        "kernels_note": "a separate eager pass with every kernel class traced: each traced launch carries two "
                        "event records, so the classes add up to a few per cent more than ms_per_step",
        "sustained": {"steps": sus_steps, "ms_per_step": sus_ms / sus_steps,
                      "value": job_throughput_gbs(world, in_bytes, sus_steps, sus_ms), "unit": UNIT,
                      "device_seconds": sus_ms * 1e-3, "clocks": sus_clocks,
                      "roofline": {"achieved": conv_bytes * U * d / (sus_conv_ms / max(sus_conv_n, 1) * 1e-3) / 1e9,
                                   "frac": conv_bytes * U * d / (sus_conv_ms / max(sus_conv_n, 1) * 1e-3) / 1e9 / peak,
                                   "avg_launch_ms": sus_conv_ms / max(sus_conv_n, 1), "launches_timed": sus_conv_n}},
    }
    if other_rec is not None:
        result["lagged_bias" if other == "lagged" else "current_bias"] = other_rec
    if two_pass_rec is not None:
        result["current_two_pass"] = two_pass_rec
    if graph_ms is not None:
        result["graph_replay"] = {"ms_per_step": graph_ms, "value": job_throughput_gbs(1, in_bytes, 1, graph_ms),
                                  "unit": UNIT, "note": "the same steps replayed from one captured CUDA graph"}
    if rank == 0:
        if not args.no_cpu_baseline:
            result["cpu_baseline"] = cpu_baseline(wl_index=1, budget_s=25.0)
        print(json.dumps(result), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_sliced(args):
    """--slices: the SAME total workload (configuration 1) cut into slices of d, one per rank, with the
    all-reduce of the per-layer moment sums between the phases (strong scaling; not the default arm)."""
    import torch
    import torch.distributed as dist
    from paper_2203_09044_b200 import binding, inputs, sharded

    binding.lib()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if "RANK" in os.environ:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    wl = inputs.workload(1, n_users=args.users)
    U, d = wl.n_users, wl.d
    lay = sharded.SliceLayout(d, wl.seg_offsets, rank, world)
    ld = inputs.aligned_ld(lay.hi - lay.lo)
    sp = sharded.ShardedPlan(d, U, wl.exp_bits, wl.mant_bits, wl.seg_offsets, rank, world, ld=ld, gamma=wl.gamma)
    out = sp.plan.alloc_outputs()
    residual = torch.zeros((U, ld), dtype=torch.float32, device="cuda")
    pool = []
    for t in range(POOL):                               # every rank draws the whole batch and keeps its slice
        g = wl.gradient(t, device="cuda")
        x = torch.zeros((U, ld), dtype=torch.float32, device="cuda")
        x[:, :lay.hi - lay.lo] = g[:, lay.lo:lay.hi]
        pool.append(x)
        del g
    torch.cuda.synchronize()

    def step(t):
        sp.encode(pool[t % POOL], residual, out)
        sp.decode_aggregate(out)

    def barrier():
        if dist.is_initialized():
            dist.barrier()
        torch.cuda.synchronize()

    for t in range(args.warmup):
        step(t)
    barrier()
    assert sp.plan.status(clear=True)[0] == 0
    sampler = ClockSampler(physical_gpu_index(local_rank))
    launches0 = sp.plan.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    e0.record()
    for t in range(args.steps):
        step(args.warmup + t)
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
    launches = sp.plan.launch_count() - launches0
    assert sp.plan.status()[0] == 0
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": 4.0 * d * U * args.steps / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "configs[1] cut into %d slices of d (one per rank), moment sums all-reduced "
                                   "twice at t = 0 and once per iteration after" % world,
                       "d": d, "n_users": U, "slice_of_rank_0": [lay.lo, lay.hi], "row_stride": ld,
                       "launch": "every step launched eagerly (the all-reduce sits between the phases)",
                       "l2": "%d MB of gradient+memory read per step and rank, %d batches cycled"
                             % (8 * U * (lay.hi - lay.lo) // 1000000, POOL)},
            "clocks": clocks, "gpu_launches": launches}), flush=True)
    if dist.is_initialized():
        barrier()
        dist.destroy_process_group()


def oracle_sample_step(orc, wl, g, m):
    """One CO3 iteration of the oracle (encode + decode-aggregate) on host arrays."""
    r = orc.encode(g, m)
    rc, avg, _ = orc.decode_aggregate(r.payload, r.sub_bits, r.chunk_off, r.hdr)
    assert rc == 0
    return r


def cpu_baseline(wl_index, budget_s):
    """The oracle as it stands, single-threaded, on a bounded sample of the same workload."""
    import numpy as np
    from oracle import co3_oracle
    from paper_2203_09044_b200 import inputs
    full = inputs.workload(wl_index)
    per_elem = 2.0e-7                                   # rough oracle cost per user-element
    users = max(1, min(full.n_users, int(budget_s / (per_elem * full.d))))
    wl = inputs.workload(wl_index, n_users=users)
    g = wl.gradient(0).numpy()
    m = np.zeros_like(g)
    orc = co3_oracle.OracleCO3(wl.d, users, wl.exp_bits, wl.mant_bits, wl.seg_offsets, gamma=wl.gamma)
    t0 = time.perf_counter()
    oracle_sample_step(orc, wl, g, m)
    dt = time.perf_counter() - t0
    out = {"value": 4.0 * wl.d * users / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"1 iteration (encode + decode-aggregate) of {users} of the {full.n_users} users "
                     f"at full d={wl.d}, {dt:.1f} s",
           "host_cores_available": os.cpu_count()}
    del g, m, orc
    out["all_cores"] = cpu_baseline_all_cores(wl_index, full.n_users)
    return out


def cpu_baseline_all_cores(wl_index, n_users):
    """The same oracle, one process per user side by side (the users' streams are independent; each
    process fits its own user's moments, which is the same amount of work): what the host cores of
    this box deliver together.  value = the users' bytes / the slowest process's iteration time."""
    import subprocess
    procs = min(n_users, os.cpu_count() or 1)
    cmd = [sys.executable, os.path.abspath(__file__), "--oracle-worker"]
    ps = [subprocess.Popen(cmd + [f"{wl_index}:{u}"], stdout=subprocess.PIPE, text=True) for u in range(procs)]
    times, d = [], 0
    for pr in ps:
        try:
            line = pr.communicate(timeout=300)[0].strip().splitlines()[-1]
            rec = json.loads(line)
            times.append(rec["seconds"])
            d = rec["d"]
        except Exception:                               # a worker that failed: no figure, not a wrong one
            pr.kill()
            return {"unavailable": "an oracle worker process failed"}
    dt = max(times)
    return {"value": 4.0 * d * procs / dt / 1e9, "unit": UNIT, "cores": procs,
            "sample": f"{procs} processes, each 1 iteration of 1 user at full d={d}; slowest {dt:.1f} s"}


def oracle_worker(spec):
    """Child process of cpu_baseline_all_cores: one oracle iteration on one user's gradient."""
    import numpy as np
    from oracle import co3_oracle
    from paper_2203_09044_b200 import inputs
    wl_index, u = (int(x) for x in spec.split(":"))
    wl = inputs.workload(wl_index, n_users=1)
    g = wl.gradient(0, users=[u]).numpy()
    m = np.zeros_like(g)
    orc = co3_oracle.OracleCO3(wl.d, 1, wl.exp_bits, wl.mant_bits, wl.seg_offsets, gamma=wl.gamma)
    t0 = time.perf_counter()
    oracle_sample_step(orc, wl, g, m)
    print(json.dumps({"seconds": time.perf_counter() - t0, "d": wl.d}), flush=True)


def run_reference(args):
    """The reference arm: the CPU oracle timed on this machine's host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from oracle import co3_oracle
    from paper_2203_09044_b200 import inputs
    full = inputs.workload(1)
    total = max(1, args.steps + args.warmup)
    per_elem = 2.0e-7
    n = int(min(full.n_users * full.d, max(65536, 150.0 / (total * per_elem))))   # user-elements per step
    users = max(1, min(full.n_users, n // 65536, 8))
    d_s = max(4096, min(full.d, n // users))
    wl = inputs.workload(1, d=None if d_s >= full.d else d_s, n_users=users)
    # the bias mode of this arm's config (`--mode`, default: from the current moments, as `value` is measured)
    orc = co3_oracle.OracleCO3(wl.d, users, wl.exp_bits, wl.mant_bits, wl.seg_offsets, gamma=wl.gamma,
                               mode={"current": co3_oracle.MODE_CURRENT, "lagged": co3_oracle.MODE_LAGGED,
                                     "code-lagged": co3_oracle.MODE_LAGGED_CODE}[args.mode])
    grads = [wl.gradient(t).numpy() for t in range(2)]
    m = np.zeros_like(grads[0])
    for t in range(args.warmup):
        oracle_sample_step(orc, wl, grads[t % 2], m)
    t0 = time.perf_counter()
    for t in range(args.steps):
        oracle_sample_step(orc, wl, grads[t % 2], m)
    dt = time.perf_counter() - t0
    value = 4.0 * wl.d * users * args.steps / dt / 1e9
    sample = (f"each step = 1 iteration (encode + decode-aggregate) on {users} users x d={wl.d} of the "
              f"workload's {full.n_users} x {full.d} (same 62-layer size mix)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": "configs[1] (8 users x ResNet-18 gradient, E4M3, gamma=0.9), sampled",
                   "d": wl.d, "n_users": users},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--users", type=int, default=None,
                    help="override the number of simulated users (profiling a smaller case); default 8")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay leg")
    ap.add_argument("--short", action="store_true",
                    help="profiling runs: the sustained leg repeats only --steps steps, the other bias mode is not timed")
    ap.add_argument("--mode", default="current", choices=["lagged", "current", "code-lagged"],
                    help="bias/code mode behind `value` (default: current, the bias of Algorithm 1 as printed; "
                         "the lagged bias is timed beside it)")
    ap.add_argument("--slices", action="store_true",
                    help="cut the one workload into slices of d, one per rank (strong scaling), instead of replicas")
    ap.add_argument("--oracle-worker", default=None, help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.oracle_worker:
        oracle_worker(args.oracle_worker)
        return
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.slices:
        run_sliced(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
