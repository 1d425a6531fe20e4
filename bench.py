#!/usr/bin/env python
"""Benchmark of the LAQ re-eviction step (Section 4.3, Eq. 4) on B200.

One step = one ``laq_evict`` call over every layer / batch item / KV head of a Llama-3-8B-shaped
long-context cache (32 layers, 32/8 heads, batch 4, L = 32768, W = 32, pool kernel 7, budget
2048), on seeded synthetic tensors already resident in HBM. Prints ONE JSON line:

  value        prompt tokens evicted per second (Bt*L / step time, whole job)
  roofline     the scoring kernel's algorithmic bytes / its CUDA-event time vs the measured HBM peak
  e2e          the same metric through ``laq_evict_host`` (host buffers, copies inside the timing)
  cpu_baseline the fp64 CPU oracle timed on this machine's cores on a sample of the same units

``--impl reference`` times the CPU oracle instead (it is the only reference this method has).
With ``--gpus N`` (N > 1) the script starts N ranks itself, one per GPU, through
``torch.distributed.run`` (or runs as one of them when a launcher has already set WORLD_SIZE).
The units are independent, so there is no data-path collective; only the timing is reduced over
ranks. ``--scaling weak`` (default): every rank evicts its own cache of the full size;
``--scaling strong``: the layers of one cache are split over the ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "prompt KV tokens evicted/sec (all layers/heads)"
UNIT = "prompt_tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one score_tc_kernel launch, from the ncu capture
# of the 2-layer slice of config 3 summarised under profiles/ (64 units; 1000 tasks, far more than
# the distance between the two sweeps, so the L2 reuse is that of the full launch). The traffic
# grows in proportion to the units, which is how it is scaled to the launch that is timed.
NCU_SMALL_CASE_UNITS = 64
NCU_SMALL_CASE_DRAM_BYTES = 631.73e6 + 18.13e6
NCU_TRAFFIC_BYTES_RAW = 8.68e9  # score_raw_d128_kernel on the full workload (--score-mode raw; quoted, one-pass capture)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="laq", choices=["laq", "reference"])
    ap.add_argument("--config", type=int, default=3, help="workload (3 = the headline config)")
    ap.add_argument("--budget", type=int, default=2048)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (profiling)")
    ap.add_argument("--prompt-len", type=int, default=0, help="override the prompt length (profiling)")
    ap.add_argument("--window", type=int, default=0,
                    help="override W, the lookahead queries per head (Section 6.2 ablates 1, 2 and 8 steps)")
    ap.add_argument("--local-window", type=int, default=0,
                    help="LAQ++ (Eq. 5): this many of the window's queries are causal local queries")
    ap.add_argument("--score-mode", default="softmax", choices=["softmax", "raw"],
                    help="raw = Eq. 4 read literally (sums of raw logits, one pass over K)")
    ap.add_argument("--pool-mode", default="avg", choices=["avg", "max"])
    ap.add_argument("--ragged", action="store_true",
                    help="prompt b of the batch holds only L*(b+1)/batch positions (per-prompt lengths)")
    ap.add_argument("--seq-lens", default="", help="explicit per-prompt lengths, comma separated")
    ap.add_argument("--graph", action="store_true",
                    help="time the steps as replays of one captured CUDA graph (launch-bound small workloads)")
    ap.add_argument("--tiles-per-task", type=int, default=0)
    ap.add_argument("--lag-tasks", type=int, default=0)
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="N > 1: weak = one full-size cache per rank, strong = one cache's layers split over the ranks")
    ap.add_argument("--stub-step", action="store_true",
                    help="host-logic check of the multi-rank path without a GPU: gloo backend, the step is a "
                         "timed sleep (used by the CPU tests; the line it prints is not a measurement)")
    return ap.parse_args()


def spawn_ranks(args) -> int:
    """--gpus N without a launcher: re-run this script as N ranks of one node."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
           f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1", "--master-port", str(port),
           os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def run_stub(args):
    """The multi-rank plumbing of main() on CPU: process group, barrier, per-rank shard, MAX over
    ranks of the step time, one JSON line from rank 0."""
    import torch.distributed as dist
    from paper_2505_20334_b200 import multi, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    cfg = workload(args)
    layers = multi.shard_units(cfg.n_layers, world, rank) if args.scaling == "strong" else (0, cfg.n_layers)
    tokens = cfg.batch * cfg.prompt_len
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.002 * (rank + 1))  # the last rank is the slow one
    my_ms = (time.perf_counter() - t0) * 1e3 / max(1, args.steps)
    ms = multi.max_over_ranks(my_ms)
    if world > 1:
        dist.barrier()
    if rank == 0:
        per_step = tokens * world if args.scaling == "weak" else tokens
        print(json.dumps({"metric": METRIC, "value": per_step / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                          "higher_is_better": True, "scaling": args.scaling, "stub": True,
                          "layers_of_rank0": list(layers), "config": config_dict(cfg, args.budget, args)}))
    if world > 1:
        dist.destroy_process_group()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.power_w, self.reasons, self.max_mhz = [], [], set(), None
        self._stop_evt = threading.Event()
        self.handle = None
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.handle = None

    def run(self):
        if self.handle is None:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                try:
                    self.power_w.append(nv.nvmlDeviceGetPowerUsage(self.handle) / 1000.0)
                except Exception:
                    pass
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = None
        if self.samples:
            s = sorted(self.samples)
            med = s[len(s) // 2]
        return {"sm_mhz": med, "sm_min_mhz": min(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "power_w_max": max(self.power_w) if self.power_w else None,
                "samples": len(self.samples)}


def workload(args):
    from paper_2505_20334_b200 import synth

    cfg = synth.CONFIGS[args.config]
    if args.layers:
        cfg = cfg.scaled(n_layers=args.layers)
    if args.batch:
        cfg = cfg.scaled(batch=args.batch)
    if args.prompt_len:
        cfg = cfg.scaled(prompt_len=args.prompt_len)
    if args.window:
        cfg = cfg.scaled(window_len=args.window)  # the retained tail keeps its size
    return cfg


def algorithmic_bytes(cfg, B, mean_len=None):
    """Bytes the method must move per step: K once + Q for scoring; kept K/V rows read and written,
    the kept positions written (fp32 column sums and a second K sweep are overhead, not counted)."""
    D2 = 2 * cfg.head_dim
    score = cfg.units * (D2 * (cfg.prompt_len if mean_len is None else mean_len) + D2 * cfg.rows)
    gather = cfg.units * (2 * D2 * B + 2 * D2 * B + 4 * B)
    return score, gather


def cpu_baseline(cfg, inputs, B, budget_s=20.0):
    """The fp64 oracle, as it stands, on a sample of this workload's units (about 20 per host
    thread, which is 10-20 s of CPU work for the long-context workload)."""
    import torch
    from oracle import laq_oracle as orc
    from paper_2505_20334_b200 import synth

    cores = os.cpu_count() or 1
    n = max(1, min(cores * 20, cfg.units, 384))
    units = synth.sample_units(cfg, n)[:n]
    qs, ks, vs = [], [], []
    for u in units:
        q, k, v = synth.unit_slices(cfg, inputs, u)
        qs.append(q[0])
        ks.append(k[0])
        vs.append(v[0])
    q, k, v = torch.stack(qs), torch.stack(ks), torch.stack(vs)  # [n,1,G,W,D], [n,1,1,L,D]
    t0 = time.perf_counter()
    out = orc.evict(q, k, v, cfg.keep_tail, cfg.pool_kernel, B)
    dt = time.perf_counter() - t0
    tokens = cfg.batch * cfg.prompt_len * (len(units) / cfg.units)
    return {"value": tokens / dt, "unit": UNIT, "cores": int(out["threads"]), "kind": "oracle",
            "sample": f"{len(units)} of {cfg.units} (layer,batch,kv-head) units of the same "
                      f"workload spread over the OpenMP threads, {dt:.1f} s; tokens scaled by the unit fraction",
            "seconds": dt}


def run_reference(args):
    """--impl reference: the CPU oracle (the only reference this method has) on host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    if "WORLD_SIZE" in os.environ:
        # a launcher pins every rank to one OpenMP thread; here rank 0 alone works, on all host cores
        os.environ["OMP_NUM_THREADS"] = str(os.cpu_count() or 1)
    import torch
    from oracle import laq_oracle as orc
    from paper_2505_20334_b200 import synth

    cfg = workload(args)
    B = args.budget
    cores = os.cpu_count() or 1
    # one unit of the workload per step and per thread, generated on the host
    n = max(1, min(cores, 16))
    small = cfg.scaled(n_layers=1, batch=1, n_kv_heads=1, n_q_heads=cfg.group)
    qs, ks, vs = [], [], []
    for i in range(n):
        inp = synth.make_inputs(small.scaled(cfg_id=cfg.cfg_id + 100 * (i + 1)), "cpu")
        qs.append(inp["q"][0])
        ks.append(inp["k"][0])
        vs.append(inp["v"][0])
    q, k, v = torch.stack(qs), torch.stack(ks), torch.stack(vs)
    threads = 1
    for _ in range(args.warmup):
        threads = orc.evict(q[:1], k[:1], v[:1], cfg.keep_tail, cfg.pool_kernel, B)["threads"]
    t0 = time.perf_counter()
    for _ in range(args.steps):
        threads = orc.evict(q, k, v, cfg.keep_tail, cfg.pool_kernel, B)["threads"]
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    tokens = cfg.batch * cfg.prompt_len * (n / cfg.units)
    value = tokens / dt
    sample = (f"each step = {n} units (1 layer x 1 batch x 1 kv head each) of {cfg.units} in the "
              f"workload; tokens scaled by that fraction")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_dict(cfg, B, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": int(threads), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def config_dict(cfg, B, args, lens=None):
    """The workload and every option that changes it; the same keys in both arms."""
    return {"workload": f"config {cfg.cfg_id}: {cfg.name}", "score_mode": args.score_mode,
            "pool_mode": args.pool_mode, "local_window": args.local_window, "seq_lens": lens,
            "cuda_graph": bool(args.graph), "n_layers": cfg.n_layers,
            "batch": cfg.batch, "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads,
            "head_dim": cfg.head_dim, "prompt_len": cfg.prompt_len, "window_len": cfg.window_len,
            "keep_tail": cfg.keep_tail, "pool_kernel": cfg.pool_kernel, "budget": B,
            "units": cfg.units, "parallelism": "independent units, no collective",
            "l2": "inputs (K+V) far larger than the 126 MB L2; no flush needed"}


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    if args.impl == "reference":
        run_reference(args)
        return
    if args.stub_step:
        run_stub(args)
        return

    import torch
    import torch.distributed as dist

    from paper_2505_20334_b200 import build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if rank == 0:
        build.build_liblaq()
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    from paper_2505_20334_b200 import binding as laq
    from paper_2505_20334_b200 import multi, synth

    cfg_full = cfg = workload(args)
    if world > 1 and args.scaling == "strong":
        # one cache, its layers split over the ranks (units are independent: no exchange)
        lo, hi = multi.shard_units(cfg.n_layers, world, rank)
        if hi <= lo:
            raise SystemExit("--scaling strong needs at least one layer per rank")
        cfg = cfg.scaled(n_layers=hi - lo, cfg_id=cfg.cfg_id + 1000 * rank)
    elif world > 1:
        cfg = cfg.scaled(cfg_id=cfg.cfg_id + 1000 * rank)  # every rank draws its own cache
    B = args.budget
    inputs = synth.make_inputs(cfg, dev)
    q, k, v = inputs["q"], inputs["k"], inputs["v"]
    NL, Bt, Hkv, D, L = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.prompt_len
    k_out = torch.empty((NL, Bt, Hkv, B, D), dtype=torch.bfloat16, device=dev)
    v_out = torch.empty_like(k_out)
    idx = torch.empty((NL, Bt, Hkv, B), dtype=torch.int32, device=dev)
    p = laq.params_for(q, k, cfg.keep_tail, cfg.pool_kernel, B, v=v, out=k_out)
    p.tiles_per_task, p.sched_lag_tasks = args.tiles_per_task, args.lag_tasks
    p.local_window = args.local_window
    p.score_mode = laq.LAQ_SCORE_RAW if args.score_mode == "raw" else laq.LAQ_SCORE_SOFTMAX
    p.pool_mode = laq.LAQ_POOL_MAX if args.pool_mode == "max" else laq.LAQ_POOL_AVG
    lens = [max(B + 1, L * (b + 1) // Bt) for b in range(Bt)] if args.ragged else None
    if args.seq_lens:
        lens = [int(x) for x in args.seq_lens.split(",")]
    p.set_seq_lens(lens)
    tokens_per_step = sum(lens) if lens else Bt * L
    ws = laq.alloc_workspace(p, dev)

    def step():
        laq.laq_evict(p, q, k, v, k_out, v_out, idx, None, ws)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    if laq.laq_last_device_status(p, ws) != laq.LAQ_OK:
        raise RuntimeError("laq_evict reported a device-side error during warm-up")
    launches_per_step = laq.laq_last_launch_count()

    K = args.steps
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b in ev:  # create the underlying CUDA events
        a.record()
        b.record()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    start.record()
    for i in range(K):
        laq.laq_set_stage_events(ev[i][0], ev[i][1])
        step()
    stop.record()
    laq.laq_set_stage_events(None, None)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.finish()
    total_ms = start.elapsed_time(stop)
    score_ms = sum(a.elapsed_time(b) for a, b in ev) / K
    if args.graph:
        # the same K steps as replays of one captured step (the eager run above keeps the
        # per-kernel times; the step time reported is the replayed one)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            step()
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                step()
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        start.record()
        for _ in range(K):
            graph.replay()
        stop.record()
        torch.cuda.synchronize()
        total_ms = start.elapsed_time(stop)
    if laq.laq_last_device_status(p, ws) != laq.LAQ_OK:
        raise RuntimeError("laq_evict reported a device-side error")
    # what the scoring kernel of the last step recorded about itself: SM cycles and wall time of
    # its first block, i.e. the SM clock it really ran at (the board lowers it under load)
    kernel_cycles, kernel_ns = laq.laq_last_kernel_clock(ws)
    total_ms = multi.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / K
    # weak: every rank evicts tokens_per_step prompt tokens (all layers); strong: the ranks share
    # the layers of one cache, so the job as a whole evicts tokens_per_step per step
    value = multi.whole_job_tokens_per_s(tokens_per_step, world if args.scaling == "weak" else 1,
                                         ms_per_step)

    peak, peak_src = measured_peaks()
    score_bytes, gather_bytes = algorithmic_bytes(cfg, B, tokens_per_step / Bt)
    achieved = score_bytes / (score_ms * 1e-3) / 1e9
    raw = args.score_mode == "raw"
    # the ncu figures belong to config 3's geometry (any number of layers)
    captured = args.config == 3 and not (args.batch or args.prompt_len or lens or args.window or
                                         args.local_window)
    if raw:
        traffic = NCU_TRAFFIC_BYTES_RAW if captured and not args.layers else None
    else:
        traffic = NCU_SMALL_CASE_DRAM_BYTES * cfg.units / NCU_SMALL_CASE_UNITS if captured else None
    roofline = {"bound": "hbm", "kernel": "score_raw_d128_kernel" if raw else "score_tc_kernel",
                "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
                "traffic_source": None if traffic is None else (
                    "ncu on the full launch (one pass)" if raw else
                    f"ncu --set full on a {NCU_SMALL_CASE_UNITS}-unit slice, scaled by the units"),
                "peak_source": peak_src, "algorithmic_bytes_per_launch": score_bytes,
                "kernel_ms": score_ms, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}
    if kernel_ns > 0 and not raw:
        sms_ = torch.cuda.get_device_properties(dev).multi_processor_count
        tile_sweeps = 2.0 * NL * Hkv * sum(-(-x // 128) for x in (lens or [L] * Bt)) / sms_
        roofline["in_kernel"] = {"sm_mhz": kernel_cycles / kernel_ns * 1e3, "sm_cycles": kernel_cycles,
                                 "cycles_per_128key_tile_and_sweep_per_sm": kernel_cycles / tile_sweeps,
                                 "source": "clock64 / globaltimer of the kernel's first block, last step"}
    # The scoring kernel's busiest unit is the MUFU: two base-2 exponentials per (row, key) pair
    # (one per sweep) at 16 per clock and SM.
    n_exp = 2.0 * NL * Hkv * cfg.rows * tokens_per_step
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    mufu_peak = 16.0 * sms * (clocks.get("sm_max_mhz") or 1965) * 1e6
    if not raw:
        roofline["mufu"] = {"bound": "alu", "achieved": n_exp / (score_ms * 1e-3), "peak": mufu_peak,
                            "unit": "ex2/s", "frac": n_exp / (score_ms * 1e-3) / mufu_peak,
                            "peak_source": "16 ex2 per clock and SM (measured) x SMs x max SM clock"}
    step_gbs = (score_bytes + gather_bytes) / (ms_per_step * 1e-3) / 1e9
    step_roofline = {"algorithmic_bytes_per_step": score_bytes + gather_bytes, "achieved": step_gbs,
                     "unit": "GB/s", "frac_of_measured": step_gbs / peak,
                     "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS}

    e2e = None
    if not args.no_e2e and rank == 0:
        hq = torch.empty(q.shape, dtype=q.dtype, pin_memory=True).copy_(q)
        hk = torch.empty(k.shape, dtype=k.dtype, pin_memory=True).copy_(k)
        hv = torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v)
        del inputs, q, k, v, k_out, v_out
        torch.cuda.empty_cache()
        he = laq.HostEvictor(tuple(hq.shape), tuple(hk.shape), B, cfg.pool_kernel, cfg.keep_tail, dev)
        he.params.tiles_per_task, he.params.sched_lag_tasks = args.tiles_per_task, args.lag_tasks
        he.params.local_window, he.params.score_mode, he.params.pool_mode = (
            p.local_window, p.score_mode, p.pool_mode)
        he.params.set_seq_lens(lens)
        he.run(hq, hk, hv)
        torch.cuda.synchronize()
        n_e2e = 3
        s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s2.record()
        for _ in range(n_e2e):
            he.run(hq, hk, hv)
        e2.record()
        torch.cuda.synchronize()
        e2e_ms = s2.elapsed_time(e2) / n_e2e
        same = bool((he.h_idx.to(dev) == idx).all().item())
        e2e = {"value": tokens_per_step / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": he.h2d_bytes, "d2h_bytes_per_step": he.d2h_bytes,
               "ms_per_step": e2e_ms, "steps": n_e2e, "api": "laq_evict_host",
               "matches_device_run": same}
        inputs_host = {"q": hq, "k": hk, "v": hv}
    else:
        inputs_host = inputs

    cpu = None
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        cpu = cpu_baseline(cfg, inputs_host, B)

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": args.scaling, "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": config_dict(cfg_full, B, args, lens),
            "kv_entries_per_s": cfg_full.n_layers * Hkv * tokens_per_step *
                                (world if args.scaling == "weak" else 1) / (ms_per_step * 1e-3),
            "roofline": roofline, "step_roofline": step_roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": launches_per_step * K, "clocks": clocks,
        }))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
