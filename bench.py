#!/usr/bin/env python
"""Throughput of the per-layer cache look-up on B200: one JSON line per run.

A step is one pass of the whole hot path over one batch of synthetic requests.  The default workload is the
four-stage ResNet-18/CIFAR-10-shaped cascade (bf16 caches of 10,000 entries with 65536 / 32768 / 16384 / 8192
values per entry, batch 1,024, k = 5, misses compacted between stages); `--workload` also offers the large-cache
layer (200,000 x 8192, batch 8,192, k = 10) and the latency layer (50,000 x 16384, batch 1 / 4 / 16, k = 1).

`value` is queries/s with every input already resident in HBM; `e2e` is the same metric through the host-buffer
entry point of the C ABI (pinned host activations copied in, results copied out, every step).  With --gpus N
every rank holds its own caches and its own batch (the look-ups of different requests are independent, so
ranks never exchange data): weak scaling.

The default run (config 2, one GPU) also measures, in the same process, the configurations the two numeric targets
sit on and puts them into the same JSON line under "targets": config 3 (tensor-core bound), config 5 at batch 1, 4
and 16 (HBM bound, device-timed latency percentiles) and config 4's per-stage rates, each with its own clock record.

`--gpus N` with N > 1 and no WORLD_SIZE in the environment starts the N ranks itself (torch.distributed.run, one
process per GPU, rendezvous on 127.0.0.1); started under torchrun it uses the ranks it is given.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3|cfg4|cfg5|...] [--impl ours|reference]
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "cache-lookup queries/sec per layer (1 B200) and % of bf16 TC peak / HBM BW"
UNIT = "queries/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}


L2_BYTES = 126 << 20


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"]))}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def captured_traffic(kernel: str, workload: str):
    """(DRAM bytes per launch of `kernel` on `workload` from the committed ncu summary, where the figure comes from);
    the figure is None when there is no capture or the kernel's source has changed since (the summary line carries the
    source file's sha256).  Nothing is measured here: a run under a profiler is never a bench run."""
    import hashlib
    src = {"gemm_select_kernel": "fi_gemm.cu", "stream_lookup_kernel": "fi_stream.cu"}.get(kernel)
    try:
        with open(os.path.join(ROOT, "paper_2002_02645_b200", "csrc", src), "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 4 and not line.startswith("#") and parts[0] == kernel and parts[1] == workload \
                        and parts[3] == digest:
                    return float(parts[2]), ("replayed from profiles/dram_traffic.txt (ncu capture of this kernel on this "
                                             f"workload; source sha256 {digest[:12]} unchanged since)")
    except Exception:
        pass
    return None, "no ncu capture of the kernel as it stands"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
                for name, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        busy = [v for v in sm if v > 0.5 * max(sm)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    return rank, local, world


def launch_ranks(n: int) -> int:
    """Start this script again as n ranks of one node (one process per GPU) and return their exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ)
    # the communicator's own start-up log shows how many ranks joined and which transport they use
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def init_group(local: int, world: int):
    """Process group of the ranks torchrun started: NCCL on GPUs (barrier, timing reduction and, for a row-sharded
    cache, the one all-gather), gloo where there is no GPU (the launcher check only).  Returns the torch device."""
    import torch
    import torch.distributed as dist
    if torch.cuda.is_available():
        torch.cuda.set_device(local)
        dev = torch.device("cuda", local)
        if world > 1 and not dist.is_initialized():
            dist.init_process_group("nccl", device_id=dev)
        return dev
    if world > 1 and not dist.is_initialized():
        dist.init_process_group("gloo")
    return torch.device("cpu")


def run_launch_check(args):
    """Starts nothing on the data path: forms the process group, runs the barrier and the max / sum reduction of the
    timing on made-up numbers (rank r reports r + 1 ms and 10 units), and has rank 0 print what came out."""
    import torch.distributed as dist
    from paper_2002_02645_b200 import sharding
    rank, local, world = dist_env()
    dev = init_group(local, world)
    if world > 1:
        dist.barrier()
    ms, units = sharding.reduce_timing(float(rank + 1), 10.0, dev)
    if rank == 0:
        print(json.dumps({"check": "launch", "n_gpus": world, "requested": args.gpus, "max_ms": ms, "units": units,
                          "backend": dist.get_backend() if world > 1 else None, "device": dev.type}))
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------- workloads

def build_workload(name: str, seed: int, query_seed=None, batch=16):
    from paper_2002_02645_b200 import datagen as dg
    if name == "cfg2":
        return dg.config2(seed=seed, query_seed=query_seed)
    if name == "cfg3":
        return dg.config3(seed=seed, query_seed=query_seed)
    if name == "cfg5":
        return dg.config5(seed=seed, batch=batch, query_seed=query_seed)
    if name == "cfg4":
        return dg.config4(seed=seed, query_seed=query_seed)
    if name == "cfg4-s0":          # first stage of cfg4 alone (100,000 x 256, batch 4,096): the select-bound case
        w = dg.config4(seed=seed, query_seed=query_seed, stages=1)
        w.name = "cfg4_stage0_only"
        return w
    if name == "cfg3-quarter":     # config 3 with a quarter of the entries (50,000) under the full batch: for profiler captures
        w = dg.config3(seed=seed, query_seed=query_seed, n_cache=50000)
        w.name = "cfg3_quarter_cache"
        return w
    if name == "cfg4-s3":          # last stage of cfg4 alone (100,000 x 2,048, batch 4,096): the pair kernel's case
        w = dg.config4(seed=seed, query_seed=query_seed, stages=1, first_stage=3)
        w.name = "cfg4_stage3_only"
        return w
    if name == "cfg2-small":       # same recipe, 1/16 of the sizes: a quick functional run
        return dg.config2(seed=seed, shrink=16, query_seed=query_seed)
    if name == "cfg2-s0":          # first stage of cfg2 alone (10,000 x 65536, batch 1,024): the dominant GEMM
        w = dg.config2(seed=seed, query_seed=query_seed, stages=1)
        w.name = "cfg2_stage0_only"
        return w
    raise SystemExit(f"unknown workload {name}")


def to_dev(a, dev):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a))
    return t.view(torch.int16).to(dev).view(torch.bfloat16) if a.dtype == np.uint16 else t.to(dev)


def to_pinned(a):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.uint16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.pin_memory()


def calibrate(cache, calib_dev, percentile):
    """THRESHOLDS[layer] for the synthetic data: the given percentile of the confidences the library itself
    returns for a separate calibration batch (offline phase, Sec. 3.1 (ii), with a percentile in place of the
    validation-error rule because synthetic requests have no model prediction to disagree with)."""
    import torch
    cache.set_threshold(0.0)
    out = cache.lookup_batch(calib_dev, with_topk=False)
    torch.cuda.synchronize()
    conf = out.conf.cpu().numpy().astype(np.float64)
    conf = conf[np.isfinite(conf)]
    tau = float(np.float32(np.percentile(conf, percentile)))
    cache.set_threshold(tau)
    return tau


def measure_e2e(args, w, caches, cascade, fence, dev):
    """The same metric through the host-buffer entry point: pinned host activations copied in, results copied out,
    every step."""
    import torch
    from paper_2002_02645_b200 import binding as fb
    from paper_2002_02645_b200 import sharding
    b0 = w.stages[0].queries.shape[0]
    host_acts = [to_pinned(st.queries) for st in w.stages]
    h_label = torch.empty(b0, dtype=torch.int32).pin_memory()
    h_stage = torch.empty(b0, dtype=torch.int32).pin_memory()
    h_conf = torch.empty(b0, dtype=torch.float32).pin_memory()
    h_out = fb.LookupOut(b0, w.k, "cpu", with_topk=False)
    for name in ("label", "conf", "hit"):
        setattr(h_out, name, getattr(h_out, name).pin_memory())

    def e2e_step():
        if cascade:
            fb.cascade_run_host(caches, host_acts, h_label, h_stage, h_conf)
        else:
            caches[0].lookup_batch_host(host_acts[0], h_out)

    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        e2e_step()
    fence()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    fence()
    e2e_s = time.perf_counter() - t0
    e2e_s, e2e_served = sharding.reduce_timing(e2e_s, b0 * e2e_steps, dev)
    h2d = sum(int(a.numel() * a.element_size()) for a in host_acts)
    d2h = b0 * 12 if cascade else b0 * 9
    return {"value": e2e_served / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": 1e3 * e2e_s / e2e_steps}



def measure_ours(args, workload, batch, *, full=True):
    """One workload on this rank's GPU; returns the JSON line as a dict (rank 0) or None (other ranks).
    full=False leaves out the end-to-end leg and the CPU baseline (the "targets" entries of the default run)."""
    import torch
    import torch.distributed as dist

    from paper_2002_02645_b200 import binding as fb
    from paper_2002_02645_b200 import build as fbuild
    from paper_2002_02645_b200 import sharding

    rank, local, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    dev = init_group(local, world)
    if rank == 0:
        fbuild.build_library()
    if world > 1:
        dist.barrier()
    fb.load_library()

    t_gen = time.time()
    # every rank serves its own requests: same caches, batch drawn from the rank's own seed
    w = build_workload(workload, seed=0, query_seed=None if (rank == 0 or args.same_batch) else 1000 + rank,
                       batch=batch)
    t_gen = time.time() - t_gen

    n_stage = len(w.stages)
    b0 = w.stages[0].queries.shape[0]
    cascade = n_stage > 1
    rule = fb.FI_HIT_CONF_GT if w.meta.get("rule", "conf_gt") == "conf_gt" else fb.FI_HIT_DIST_LE
    caches, acts, taus = [], [], []
    for s_i, st in enumerate(w.stages):
        c = fb.FreezeCache(dim=st.dim, capacity=st.cache_vecs.shape[0], num_classes=w.num_classes, k=w.k,
                           dtype=fb.FI_BF16 if st.dtype == "bf16" else fb.FI_F32, rule=rule, device=local,
                           max_batch=max(b0, 0 if st.calib is None else st.calib.shape[0]))
        # insert in slices so the staging copy on the device stays small
        n = st.cache_vecs.shape[0]
        step_rows = max(1, (512 << 20) // (st.dim * 2))
        for lo in range(0, n, step_rows):
            hi = min(n, lo + step_rows)
            c.insert(to_dev(st.cache_vecs[lo:hi], dev), torch.from_numpy(st.cache_labels[lo:hi]).to(dev))
        torch.cuda.synchronize()
        if rule == fb.FI_HIT_CONF_GT and st.calib is not None:
            taus.append(calibrate(c, to_dev(st.calib, dev), w.meta["percentiles"][s_i]))
        else:
            # fixed threshold: 20th percentile of nearest-neighbour squared distances of the batch itself
            c.set_threshold(float("inf"))
            out = c.lookup_batch(to_dev(st.queries, dev))
            torch.cuda.synchronize()
            tau = float(np.float32(np.percentile(out.topk_dist[:, 0].cpu().numpy(), 20.0)))
            c.set_threshold(tau)
            taus.append(tau)
        caches.append(c)
        acts.append(to_dev(st.queries, dev))

    state = fb.CascadeState(b0, dev)
    out_single = fb.LookupOut(b0, w.k, dev, with_topk=False)

    def step():
        if cascade:
            fb.cascade_init(state, n_stage)
            for l in range(n_stage):
                fb.cascade_step(caches[l], acts[l], state, l)
        else:
            caches[0].lookup_batch(acts[0], out=out_single)

    def fence():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    fence()
    for c in caches:
        c.poll_status()

    # per-stage arrivals (what the cascade actually does on this data): one extra pass, read after every stage
    arrivals = [b0]
    if cascade:
        fb.cascade_init(state, n_stage)
        for l in range(n_stage):
            fb.cascade_step(caches[l], acts[l], state, l)
            arrivals.append(int(state.survivors(l)[1].item()))
        fence()

    for c in caches:
        c.set_profiling(True)
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    launches0 = fb.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fence()
    cache_bytes = sum(s.cache_vecs.nbytes for s in w.stages)
    flush_l2 = cache_bytes < 2 * L2_BYTES          # a step that does not cycle L2 by itself: evict between iterations
    ms_warm = None
    if flush_l2:
        evict = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for e0, e1 in pairs:
            evict.zero_()                          # untimed: overwrites twice the L2 capacity
            e0.record()
            step()
            e1.record()
        fence()
        ms_total = sum(e0.elapsed_time(e1) for e0, e1 in pairs)
        launches = fb.launch_count() - launches0
        prof = [c.read_profile() for c in caches]
        for c in caches:
            c.set_profiling(False)
        ev0.record()
        for _ in range(args.steps):
            step()
        ev1.record()
        fence()
        ms_warm = ev0.elapsed_time(ev1) / args.steps
    else:
        ev0.record()
        for _ in range(args.steps):
            step()
        ev1.record()
        fence()
        launches = fb.launch_count() - launches0
        ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    if not flush_l2:
        prof = [c.read_profile() for c in caches]
    for c in caches:
        c.set_profiling(False)
        c.poll_status()
    # whole-job figures: slowest rank's time, all ranks' requests
    ms_total, served = sharding.reduce_timing(ms_total, b0 * args.steps, dev)
    ms_per_step = ms_total / args.steps
    value = served / (ms_total * 1e-3)

    # ---- per-look-up device latency (latency workload): every look-up between its own pair of events
    latency = None
    if workload == "cfg5":
        n_lat = max(1000, args.steps)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_lat)]
        fence()
        for e0, e1 in evs:
            e0.record()
            step()
            e1.record()
        fence()
        lat = sorted(e0.elapsed_time(e1) * 1e3 for e0, e1 in evs)
        latency = {"lookups": n_lat, "p50_us": lat[len(lat) // 2], "p99_us": lat[int(len(lat) * 0.99)],
                   "min_us": lat[0], "max_us": lat[-1]}

    e2e = None
    if full:
        e2e = measure_e2e(args, w, caches, cascade, fence, dev)

    # ---- roofline of the dominant kernel: the distance kernel of the first (largest) stage
    peaks, peak_src = load_peaks()
    st0 = w.stages[0]
    n0, d0 = st0.cache_vecs.shape
    ms0, n_launch0 = prof[0]
    roofline = None
    if n_launch0 > 0 and ms0 > 0:
        avg_s = ms0 / n_launch0 * 1e-3
        flops = 2.0 * b0 * n0 * d0
        nbytes = n0 * d0 * st0.cache_vecs.itemsize + b0 * d0 * st0.cache_vecs.itemsize + 4.0 * n0
        gemm = st0.dtype == "bf16" and b0 > 1      # the library's own rule: single requests and fp32 caches stream
        # the events bracket the distance kernel of a look-up: gemm_select_kernel (followed, where tiles were cut along the row length, by
        # piece_select_kernel) or stream_lookup_kernel
        kernel = "gemm_select_kernel" if gemm else "stream_lookup_kernel"
        # the slower of the flops at the tensor peak and the bytes at the copy bandwidth bounds the launch
        tensor_bound = gemm and flops / (peaks["bf16_tflops"] * 1e12) > nbytes / (peaks["hbm_gbs"] * 1e9)
        if tensor_bound:
            achieved = flops / avg_s / 1e12
            roofline = {"bound": "tensor", "kernel": kernel + " (stage 0)", "achieved": achieved,
                        "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                        "peak_source": f"cuBLAS bf16 burst, {peak_src} (timed region well under a second)"}
        else:
            achieved = nbytes / avg_s / 1e9
            roofline = {"bound": "hbm", "kernel": kernel + " (stage 0)", "achieved": achieved,
                        "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                        "peak_source": f"copy bandwidth, {peak_src}"}
        # the nominal figures next to the measured ones: 2.25 PFLOP/s dense bf16 and "about 8 TB/s"
        roofline["frac_of_nominal"] = achieved / (2250.0 if tensor_bound else 8000.0)
        roofline["nominal_peak"] = 2250.0 if tensor_bound else 8000.0
        traffic, traffic_src = captured_traffic(kernel, w.name)
        roofline.update({"traffic": traffic, "traffic_source": traffic_src, "avg_launch_ms": avg_s * 1e3,
                         "launches": n_launch0, "algorithmic_flops": flops, "algorithmic_bytes": nbytes})
    stage_info = []
    for l, (ms_l, n_l) in enumerate(prof):
        if n_l:
            nl, dl = w.stages[l].cache_vecs.shape
            bl = arrivals[l] if cascade else b0
            stage_info.append({"stage": l, "arrivals": bl, "distance_kernel_ms": ms_l / n_l,
                               "tflops": 2.0 * bl * nl * dl / (ms_l / n_l * 1e-3) / 1e12})

    # ---- the oracle on the host cores, bounded sample (rank 0, single GPU runs only)
    cpu_baseline = None
    if rank == 0 and world == 1 and full and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(w, taus, args.cpu_sample)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if st0.dtype == "bf16" else "f32",
                "data": "synthetic",
                "config": {"workload": w.name, "stages": n_stage, "batch": b0, "k": w.k,
                           "cache_entries": int(n0), "dims": [s.dim for s in w.stages],
                           "thresholds": taus, "arrivals": arrivals,
                           "l2": ("L2 evicted before every timed iteration by an untimed %d MB write (caches %.3f GB)"
                                  % (2 * L2_BYTES >> 20, cache_bytes / 1e9)) if flush_l2 else
                                 "inputs larger than L2 (caches %.2f GB)" % (cache_bytes / 1e9),
                           "parallelism": f"replicas x{world}", "datagen_s": round(t_gen, 1)},
                "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline,
                "stages": stage_info, "cpu_baseline": cpu_baseline}
        if ms_warm is not None:
            line["ms_per_step_l2_warm"] = ms_warm
        if latency is not None:
            line["latency"] = latency
    else:
        line = None
    for c in caches:
        c.close()
    del caches, acts, state, out_single
    torch.cuda.empty_cache()
    return line


def run_ours(args):
    import torch.distributed as dist
    rank, _, world = dist_env()
    line = measure_ours(args, args.workload, args.batch)
    if rank == 0 and world == 1 and args.workload == "cfg2" and not args.no_targets:
        line["targets"] = measure_targets(args)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def measure_targets(args):
    """The configurations the two numeric targets sit on, measured in this process after the headline workload:
    config 3 (largest batch: fraction of the bf16 tensor peak), config 5 at batch 1 / 4 / 16 (fraction of the HBM
    bandwidth, device-timed latency percentiles over >= 1,000 look-ups) and config 4's per-stage rates.  Every entry
    carries the clocks sampled during its own timed region."""
    peaks, peak_src = load_peaks()
    out = {"peaks": {"source": peak_src, **peaks, "nominal_bf16_tflops": 2250.0, "nominal_hbm_gbs": 8000.0}}

    def brief(line):
        r = line["roofline"] or {}
        d = {"workload": line["config"]["workload"], "batch": line["config"]["batch"], "ms_per_step": line["ms_per_step"],
             "queries_per_s": line["value"], "kernel": r.get("kernel"), "kernel_ms": r.get("avg_launch_ms"),
             "bound": r.get("bound"), "achieved": r.get("achieved"), "unit": r.get("unit"),
             "frac_of_measured": r.get("frac"), "frac_of_nominal": r.get("frac_of_nominal"),
             "clocks": line["clocks"], "gpu_launches": line["gpu_launches"]}
        if r.get("bound") == "tensor":
            d["frac_of_measured_sustained"] = r["achieved"] / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
        return d

    l3 = measure_ours(args, "cfg3", 16, full=False)
    out["config3_batch8192"] = brief(l3)
    for b in (1, 4, 16):
        l5 = measure_ours(args, "cfg5", b, full=False)
        d = brief(l5)
        d.update({"p50_us": l5["latency"]["p50_us"], "p99_us": l5["latency"]["p99_us"], "lookups_timed": l5["latency"]["lookups"]})
        out[f"config5_batch{b}"] = d
    l4 = measure_ours(args, "cfg4", 16, full=False)
    d = brief(l4)
    d["arrivals"] = l4["config"]["arrivals"]
    d["stages"] = [{"stage": s["stage"], "arrivals": s["arrivals"], "distance_kernel_ms": s["distance_kernel_ms"],
                    "tflops": s["tflops"], "frac_of_measured": s["tflops"] / peaks["bf16_tflops"]} for s in l4["stages"]]
    out["config4_batch4096"] = d
    return out


# ---------------------------------------------------------------------------------------------- CPU oracle leg

def oracle_sample_step(w, taus, sample):
    from oracle import fi_oracle as fo
    rule = fo.RULE_CONF_GT if w.meta.get("rule", "conf_gt") == "conf_gt" else fo.RULE_DIST_LE
    qs = [s.queries[:sample] for s in w.stages]
    if len(w.stages) > 1:
        fo.cascade(qs, [s.cache_vecs for s in w.stages], [s.cache_labels for s in w.stages], taus, k=w.k, rule=rule)
    else:
        s = w.stages[0]
        fo.lookup(qs[0], s.cache_vecs, s.cache_labels, k=w.k, tau=taus[0], rule=rule)


def default_cpu_sample(w, reference_arm=False):
    """Requests whose oracle look-ups cost about 3e11 (baseline leg) or 5e10 (per reference step) multiply-adds."""
    per_query = sum(s.cache_vecs.shape[0] * s.dim for s in w.stages)
    budget = 5e10 if reference_arm else 3e11
    return int(max(1, min(w.stages[0].queries.shape[0], budget // per_query)))


def time_oracle(w, taus, sample):
    from oracle import fi_oracle as fo
    cores = len(os.sched_getaffinity(0))
    sample = min(sample or default_cpu_sample(w), w.stages[0].queries.shape[0])
    fo.set_threads(cores)
    t0 = time.perf_counter()
    oracle_sample_step(w, taus, sample)
    dt = time.perf_counter() - t0
    # the paper's prototype looks up on a single CPU thread (Sec. 5): the same oracle on one thread, smaller sample
    one = max(1, sample // cores)
    fo.set_threads(1)
    t1 = time.perf_counter()
    oracle_sample_step(w, taus, one)
    dt1 = time.perf_counter() - t1
    fo.set_threads(cores)
    return {"value": sample / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {sample} requests of the batch through all {len(w.stages)} stage(s) against the full "
                      f"caches, fp64, OpenMP over queries; {dt:.1f} s",
            "single_thread": {"value": one / dt1, "unit": UNIT, "cores": 1,
                              "sample": f"first {one} requests, same oracle on one thread; {dt1:.1f} s"}}


def run_reference(args):
    """The oracle as it stands, on the host cores, on a bounded sample of the same workload per step."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    w = build_workload(args.workload, seed=0, batch=args.batch)
    from oracle import fi_oracle as fo
    taus = []
    for s, p in zip(w.stages, w.meta.get("percentiles", [50.0] * len(w.stages))):
        if w.meta.get("rule", "conf_gt") == "conf_gt":
            conf = fo.lookup(s.calib[:32], s.cache_vecs, s.cache_labels, k=w.k, tau=0.0).conf
            taus.append(float(np.float32(np.percentile(conf, p))))
        else:
            taus.append(float("inf"))
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    fo.set_threads(len(os.sched_getaffinity(0)))      # a launcher may have set OMP_NUM_THREADS=1 for its ranks
    if args.cpu_sample:
        sample = args.cpu_sample
    else:
        # size the per-step sample from a short probe so that warm-up + K steps take about a minute
        probe = min(8, w.stages[0].queries.shape[0])
        t0 = time.perf_counter()
        oracle_sample_step(w, taus, probe)
        rate = probe / (time.perf_counter() - t0)
        sample = int(max(1, min(w.stages[0].queries.shape[0], rate * 60.0 / (steps + warmup))))
    for _ in range(warmup):
        oracle_sample_step(w, taus, sample)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_sample_step(w, taus, sample)
    dt = time.perf_counter() - t0
    cores = len(os.sched_getaffinity(0))
    value = sample * steps / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": 1e3 * dt / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "stages": len(w.stages), "batch": sample, "k": w.k},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"first {sample} requests per step through all stages against the full caches"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_kmeans(args):
    """One Lloyd iteration at the paper's scale (Sec. 2.1 / Sec. 4): 40,000 cached points per layer reduced to 1024
    dimensions, 200 clusters; reports points/s of fi_kmeans_step (assignment look-ups + update kernel)."""
    import torch
    from paper_2002_02645_b200 import binding as fb
    from paper_2002_02645_b200 import build as fbuild
    from paper_2002_02645_b200 import datagen as dg
    fbuild.build_library()
    dev = torch.device("cuda", 0)
    n, d, clusters = 40000, 1024, 200
    w = dg.single_layer(name="kmeans_40000x1024_200", n_cache=n, n_query=clusters, dim=d, num_classes=10, dtype="bf16",
                        sigma=0.5, k=1, seed=0)
    st = w.stages[0]
    pts, labs = to_dev(st.cache_vecs, dev), torch.from_numpy(st.cache_labels).to(dev)
    cache = fb.FreezeCache(dim=d, capacity=clusters, num_classes=10, k=1, dtype=fb.FI_BF16, max_batch=n)
    cache.insert(to_dev(st.queries, dev), torch.zeros(clusters, dtype=torch.int32, device=dev))
    for _ in range(max(args.warmup, 3)):
        cache.kmeans_step(pts, labs)
    torch.cuda.synchronize()
    l0 = fb.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        cache.kmeans_step(pts, labs)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    # the point of the k-means cache (Sec. 4, Table 1): a look-up against 200 tagged centres instead of 40,000 points
    centres, counts, major, frac = cache.kmeans_step(pts, labs)[1:5]
    km = fb.FreezeCache(dim=d, capacity=clusters, num_classes=10, k=1, dtype=fb.FI_BF16, max_batch=1024)
    keep = counts > 0
    km.insert(centres[keep].contiguous(), major[keep].contiguous(), frac[keep].contiguous())
    full = fb.FreezeCache(dim=d, capacity=n, num_classes=10, k=1, dtype=fb.FI_BF16, max_batch=1024)
    full.insert(pts, labs)
    reqs = to_dev(dg.single_layer(name="q", n_cache=8, n_query=1024, dim=d, num_classes=10, dtype="bf16", sigma=0.5, k=1,
                                  seed=0, query_seed=7).stages[0].queries, dev)
    lookup_ms = {}
    for name, cc in (("kmeans_cache_200", km), ("full_cache_40000", full)):
        out = fb.LookupOut(1024, 1, dev, with_topk=False)
        for _ in range(3):
            cc.lookup_batch(reqs, out=out)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.steps):
            cc.lookup_batch(reqs, out=out)
        b.record()
        torch.cuda.synchronize()
        lookup_ms[name] = a.elapsed_time(b) / args.steps
    km.close()
    full.close()
    peaks, src = load_peaks()
    nbytes = 2.0 * n * d * 2          # the points are read once by the assignment and once by the update
    print(json.dumps({"metric": "k-means Lloyd iteration, points/s", "value": n / (ms * 1e-3), "unit": "points/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                      "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": w.name, "points": n, "dim": d, "clusters": clusters,
                                 "l2": "points (82 MB) fit in L2: figures are L2-warm",
                                 "lookup_ms_batch_1024": lookup_ms},
                      "gpu_launches": fb.launch_count() - l0,
                      "roofline": {"bound": "hbm", "achieved": nbytes / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                                   "unit": "GB/s", "frac": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                   "peak_source": f"copy bandwidth, {src}", "traffic": None}}))
    cache.close()


def run_tau_sweep(args):
    """Frozen share against agreement with the request's class as the thresholds move (the axes of the paper's
    threshold study, Sec. 5), on the 4-stage synthetic cascade: every stage's threshold is set to the p-th percentile
    of the library's confidences on the calibration batch, p swept; one more point uses ComputeThresholds (Pseudocode 1)
    with the calibration requests' classes standing in for the model's predictions."""
    import torch
    from paper_2002_02645_b200 import binding as fb
    from paper_2002_02645_b200 import build as fbuild
    fbuild.build_library()
    dev = torch.device("cuda", 0)
    w = build_workload("cfg2", seed=0)
    b0, n_stage = w.stages[0].queries.shape[0], len(w.stages)
    caches, acts, calib_conf = [], [], []
    for st in w.stages:
        c = fb.FreezeCache(dim=st.dim, capacity=st.cache_vecs.shape[0], num_classes=w.num_classes, k=w.k, dtype=fb.FI_BF16,
                           max_batch=max(b0, st.calib.shape[0]))
        c.insert(to_dev(st.cache_vecs, dev), torch.from_numpy(st.cache_labels).to(dev))
        c.set_threshold(0.0)
        conf = c.lookup_batch(to_dev(st.calib, dev), with_topk=False).conf.cpu().numpy().astype(np.float64)
        calib_conf.append(conf[np.isfinite(conf)])
        caches.append(c)
        acts.append(to_dev(st.queries, dev))
    state = fb.CascadeState(b0, dev)
    classes = w.query_classes.astype(np.int64)

    def run(taus):
        for c, t in zip(caches, taus):
            c.set_threshold(float(t))
        fb.cascade_init(state, n_stage)
        for l in range(n_stage):
            fb.cascade_step(caches[l], acts[l], state, l)
        torch.cuda.synchronize()
        stage = state.exit_stage.cpu().numpy()[:b0]
        label = state.final_label.cpu().numpy()[:b0]
        frozen = stage < n_stage
        return {"thresholds": [float(t) for t in taus], "frozen_share": float(frozen.mean()),
                "frozen_by_stage": [int((stage == l).sum()) for l in range(n_stage)],
                "agreement_of_frozen": float((label[frozen] == classes[frozen]).mean()) if frozen.any() else None}

    points = []
    for p in (5, 10, 20, 30, 40, 50, 60, 70, 80, 90, 95, 99):
        r = run([np.float32(np.percentile(cc, p)) for cc in calib_conf])
        r["percentile"] = p
        points.append(r)
    computed = []
    for c, st in zip(caches, w.stages):
        tau, wrong = c.compute_threshold(to_dev(st.calib, dev), torch.from_numpy(w.calib_classes.astype(np.int32)).to(dev))
        computed.append({"tau": tau, "wrong_lookups": wrong})
    r = run([x["tau"] for x in computed])
    r["rule"] = "ComputeThresholds"
    r["wrong_lookups_on_calibration"] = [x["wrong_lookups"] for x in computed]
    print(json.dumps({"study": "threshold sweep", "config": {"workload": w.name, "batch": b0, "stages": n_stage},
                      "data": "synthetic", "points": points, "compute_thresholds": r}))
    for c in caches:
        c.close()


def run_projected(args):
    """The 4-stage cascade as the paper runs it (Sec. 3): every layer's activation is first reduced to 1,024 dimensions
    by that layer's one-layer network, and the caches hold reduced vectors.  Random weights stand in for the trained
    ones.  A step = cascade_init + 4 x (projection of the survivors + look-up + compaction)."""
    import torch
    from paper_2002_02645_b200 import binding as fb
    from paper_2002_02645_b200 import build as fbuild
    from paper_2002_02645_b200 import datagen as dg
    fbuild.build_library()
    dev = torch.device("cuda", 0)
    out_dim = 1024
    w = build_workload("cfg2", seed=0)
    b0, n_stage = w.stages[0].queries.shape[0], len(w.stages)
    projs, caches, acts, taus = [], [], [], []
    for l, st in enumerate(w.stages):
        w_bits, bias = dg.projection_weights(st.dim, out_dim, seed=0, stage=l)
        p = fb.Projection(in_dim=st.dim, out_dim=out_dim, max_batch=b0)
        p.set_weights(to_dev(w_bits, dev), torch.from_numpy(bias).to(dev))
        c = fb.FreezeCache(dim=out_dim, capacity=st.cache_vecs.shape[0], num_classes=w.num_classes, k=w.k,
                           dtype=fb.FI_BF16, max_batch=max(b0, st.calib.shape[0]))
        for lo in range(0, st.cache_vecs.shape[0], b0):
            hi = min(st.cache_vecs.shape[0], lo + b0)
            c.insert(p.apply(to_dev(st.cache_vecs[lo:hi], dev)), torch.from_numpy(st.cache_labels[lo:hi]).to(dev))
        taus.append(calibrate(c, p.apply(to_dev(st.calib, dev)), w.meta["percentiles"][l]))
        projs.append(p)
        caches.append(c)
        acts.append(to_dev(st.queries, dev))
    state = fb.CascadeState(b0, dev)

    def step():
        fb.cascade_init(state, n_stage)
        for l in range(n_stage):
            fb.cascade_step_projected(caches[l], projs[l], acts[l], state, l)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    arrivals = [b0]
    fb.cascade_init(state, n_stage)
    for l in range(n_stage):
        fb.cascade_step_projected(caches[l], projs[l], acts[l], state, l)
        arrivals.append(int(state.survivors(l)[1].item()))
    for o in projs + caches:
        o.set_profiling(True)
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.25)
    l0 = fb.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    launches = fb.launch_count() - l0
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    prof_p = [p.read_profile() for p in projs]
    prof_c = [c.read_profile() for c in caches]
    for o in projs + caches:
        o.set_profiling(False)
        o.poll_status()

    # end to end: host activations in pinned memory, copied in every step; results read back every step
    host_acts = [to_pinned(st.queries) for st in w.stages]
    dev_acts = [torch.empty_like(a) for a in acts]
    h_label = torch.empty(b0, dtype=torch.int32).pin_memory()
    h_stage = torch.empty(b0, dtype=torch.int32).pin_memory()

    def e2e_step():
        for d, h in zip(dev_acts, host_acts):
            d.copy_(h, non_blocking=True)
        fb.cascade_init(state, n_stage)
        for l in range(n_stage):
            fb.cascade_step_projected(caches[l], projs[l], dev_acts[l], state, l)
        h_label.copy_(state.final_label[:b0], non_blocking=True)
        h_stage.copy_(state.exit_stage[:b0], non_blocking=True)
        torch.cuda.synchronize()

    for _ in range(2):
        e2e_step()
    n_e2e = max(3, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(n_e2e):
        e2e_step()
    e2e_s = time.perf_counter() - t0
    h2d = sum(int(a.numel() * a.element_size()) for a in host_acts)

    peaks, src = load_peaks()
    d0 = w.stages[0].dim
    flops = 2.0 * b0 * out_dim * d0
    avg_s = prof_p[0][0] / max(1, prof_p[0][1]) * 1e-3
    achieved = flops / avg_s / 1e12
    print(json.dumps({
        "metric": METRIC, "value": b0 / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name + "_projected_to_1024", "stages": n_stage, "batch": b0, "k": w.k,
                   "cache_entries": int(w.stages[0].cache_vecs.shape[0]), "dims": [s.dim for s in w.stages],
                   "reduced_dim": out_dim, "thresholds": taus, "arrivals": arrivals,
                   "l2": "inputs larger than L2 (activations and weights %.2f GB per step)"
                         % (sum(2.0 * s.dim * (b0 + out_dim) for s in w.stages) / 1e9)},
        "e2e": {"value": b0 * n_e2e / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": b0 * 8,
                "steps": n_e2e, "ms_per_step": 1e3 * e2e_s / n_e2e},
        "gpu_launches": int(launches), "clocks": clocks,
        "roofline": {"bound": "tensor", "kernel": "gemm_select_kernel in product mode + product_reduce_kernel (stage 0)",
                     "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": achieved / peaks["bf16_tflops"], "peak_source": f"cuBLAS bf16 burst, {src}",
                     "frac_of_nominal": achieved / 2250.0, "traffic": None, "avg_launch_ms": avg_s * 1e3,
                     "algorithmic_flops": flops, "algorithmic_bytes": 2.0 * d0 * (b0 + out_dim) + 2.0 * b0 * out_dim},
        "stages": [{"stage": l, "arrivals": arrivals[l], "projection_ms": prof_p[l][0] / max(1, prof_p[l][1]),
                    "distance_kernel_ms": prof_c[l][0] / max(1, prof_c[l][1])} for l in range(n_stage)],
        "cpu_baseline": None}))
    for o in projs + caches:
        o.close()


def run_overlap(args):
    """Look-ups pipelined with the forward pass (Sec. 5): stage l's look-up runs on its own stream while the main stream
    already computes layer l + 1.  The layers are stood in for by the caller's own work (one bf16 matrix product per
    stage on the main stream); the look-up kernels can be limited to a share of the SMs so that both streams make
    progress.  Two regimes: the config-2 cascade (batch 1,024: the look-ups are tensor-core work themselves) and the
    config-5 latency look-up (batch 16: the look-up streams the cache at the HBM rate and leaves the tensor cores
    idle).  Reports, per SM share, the step time against the serial schedule and the fraction of the look-up time
    that disappears behind the layers."""
    import torch
    from paper_2002_02645_b200 import binding as fb
    from paper_2002_02645_b200 import build as fbuild
    fbuild.build_library()
    dev = torch.device("cuda", 0)
    main, side = torch.cuda.Stream(), torch.cuda.Stream()

    def timed(fn):
        with torch.cuda.stream(main):
            for _ in range(max(args.warmup, 3)):
                fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(main):
            e0.record(main)
            for _ in range(args.steps):
                fn()
            e1.record(main)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    def study(name, caches, begin, lookup, n_stage, m, shares):
        layer_a = torch.randn(m, m, device=dev, dtype=torch.bfloat16)
        layer_b = torch.randn(m, m, device=dev, dtype=torch.bfloat16)
        layer_out = torch.empty(m, m, device=dev, dtype=torch.bfloat16)
        done = [torch.cuda.Event() for _ in range(n_stage)]

        def layers_only():
            for _ in range(n_stage):
                torch.matmul(layer_a, layer_b, out=layer_out)

        def lookups_only():
            begin()
            for l in range(n_stage):
                lookup(l)

        def serial():
            begin()
            for l in range(n_stage):
                torch.matmul(layer_a, layer_b, out=layer_out)       # layer l produces the activations ...
                lookup(l)                                           # ... which are looked up before layer l + 1 starts

        def pipelined():
            with torch.cuda.stream(side):
                side.wait_stream(main)
                begin()
            for l in range(n_stage):
                torch.matmul(layer_a, layer_b, out=layer_out)
                done[l].record(main)
                with torch.cuda.stream(side):
                    side.wait_event(done[l])                        # layer l's activations exist
                    lookup(l)                                       # runs while the main stream computes layer l + 1
            main.wait_stream(side)

        t_layers = timed(layers_only)
        rows = []
        for sms in shares:
            for c in caches:
                c.set_sm_limit(sms)
            t_look, t_serial, t_pipe = timed(lookups_only), timed(serial), timed(pipelined)
            rows.append({"lookup_sms": sms or "all", "lookups_alone_ms": t_look, "serial_ms": t_serial, "pipelined_ms": t_pipe,
                         "lookup_time_hidden": (t_serial - t_pipe) / t_look})
        for c in caches:
            c.set_sm_limit(0)
            c.poll_status()
        return {"regime": name, "stages": n_stage, "layer_stand_in": f"one {m}^3 bf16 matrix product per stage on the caller's stream",
                "layers_alone_ms": t_layers, "schedules": rows}

    sampler = ClockSampler(0)
    sampler.start()
    out = []
    # ---- config 2: the 4-stage cascade at batch 1,024
    w = build_workload("cfg2", seed=0)
    b0, n_stage = w.stages[0].queries.shape[0], len(w.stages)
    caches, acts = [], []
    for s_i, st in enumerate(w.stages):
        c = fb.FreezeCache(dim=st.dim, capacity=st.cache_vecs.shape[0], num_classes=w.num_classes, k=w.k, dtype=fb.FI_BF16,
                           max_batch=max(b0, st.calib.shape[0]))
        c.insert(to_dev(st.cache_vecs, dev), torch.from_numpy(st.cache_labels).to(dev))
        calibrate(c, to_dev(st.calib, dev), w.meta["percentiles"][s_i])
        caches.append(c)
        acts.append(to_dev(st.queries, dev))
    state = fb.CascadeState(b0, dev)
    out.append(study("config 2 cascade, batch 1024 (look-ups bound by the tensor cores)", caches,
                     lambda: fb.cascade_init(state, n_stage), lambda l: fb.cascade_step(caches[l], acts[l], state, l),
                     n_stage, 6144, (0, 96, 64)))
    for c in caches:
        c.close()
    del caches, acts, w
    torch.cuda.empty_cache()
    # ---- config 5: one cache, batch 16, the same look-up after each of four layers
    w = build_workload("cfg5", seed=0, batch=16)
    st = w.stages[0]
    c5 = fb.FreezeCache(dim=st.dim, capacity=st.cache_vecs.shape[0], num_classes=w.num_classes, k=w.k, dtype=fb.FI_BF16,
                        rule=fb.FI_HIT_DIST_LE, max_batch=16)
    c5.insert(to_dev(st.cache_vecs, dev), torch.from_numpy(st.cache_labels).to(dev))
    c5.set_threshold(float("inf"))
    q5 = to_dev(st.queries, dev)
    o5 = fb.LookupOut(16, w.k, dev, with_topk=False)
    out.append(study("config 5 look-up, batch 16 (bound by HBM)", [c5], lambda: None, lambda l: c5.lookup_batch(q5, out=o5),
                     4, 5120, (0, 96, 64, 32, 16)))
    c5.close()
    clocks = sampler.stop()
    print(json.dumps({"study": "look-ups pipelined with the forward pass", "data": "synthetic", "steps": args.steps,
                      "regimes": out, "clocks": clocks}))


def run_rowshard(args):
    """The 200,000-entry single-layer workload with the cache ROWS split over the ranks (strong scaling: the same
    8,192 requests and the same entries at every N).  Every rank looks all requests up in its rows, one all-gather
    moves batch x k x 16 bytes per rank, every rank merges and votes.  At N=1 this is the plain look-up plus the two
    small kernels of the exchange."""
    import torch
    import torch.distributed as dist
    from paper_2002_02645_b200 import binding as fb
    from paper_2002_02645_b200 import build as fbuild
    from paper_2002_02645_b200 import sharding
    rank, local, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        fbuild.build_library()
    if world > 1:
        dist.barrier()
    w = build_workload("cfg3", seed=0)
    st = w.stages[0]
    n, b0 = st.cache_vecs.shape[0], st.queries.shape[0]
    lo, hi = sharding.shard_bounds(n, world, rank)
    cache = fb.FreezeCache(dim=st.dim, capacity=hi - lo, num_classes=w.num_classes, k=w.k, dtype=fb.FI_BF16, device=local,
                           max_batch=max(b0, st.calib.shape[0]))
    rows = max(1, (512 << 20) // (st.dim * 2))
    for a in range(lo, hi, rows):
        b = min(hi, a + rows)
        cache.insert(to_dev(st.cache_vecs[a:b], dev), torch.from_numpy(st.cache_labels[a:b]).to(dev))
    cache.set_threshold(0.0)
    conf = sharding.sharded_lookup(cache, to_dev(st.calib, dev), lo).conf.cpu().numpy().astype(np.float64)
    tau = float(np.float32(np.percentile(conf[np.isfinite(conf)], w.meta["percentiles"][0])))
    cache.set_threshold(tau)
    q = to_dev(st.queries, dev)

    def fence():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        out = sharding.sharded_lookup(cache, q, lo)
    fence()
    cache.poll_status()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    l0 = fb.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fence()
    e0.record()
    for _ in range(args.steps):
        out = sharding.sharded_lookup(cache, q, lo)
    e1.record()
    fence()
    launches = fb.launch_count() - l0
    clocks = sampler.stop()
    cache.poll_status()
    ms_total, _ = sharding.reduce_timing(e0.elapsed_time(e1), 0, dev)
    ms = ms_total / args.steps
    if rank == 0:
        peaks, src = load_peaks()
        tf = 2.0 * b0 * n * st.dim / (ms * 1e-3) / 1e12 / world          # per GPU, whole step as the duration
        print(json.dumps({"metric": METRIC, "value": b0 / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                          "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16",
                          "data": "synthetic",
                          "config": {"workload": w.name + "_row_sharded", "batch": b0, "entries": n, "dim": st.dim,
                                     "k": w.k, "rows_per_rank": hi - lo, "exchange_bytes_per_rank": b0 * w.k * 16,
                                     "hit_rate": float(out.hit.float().mean().item()),
                                     "l2": "inputs larger than L2"},
                          "gpu_launches": launches, "clocks": clocks,
                          "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops_sustained"],
                                       "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops_sustained"],
                                       "peak_source": f"cuBLAS bf16 sustained, {src}; whole step as the duration",
                                       "traffic": None}}))
    cache.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg3", "cfg3-quarter", "cfg4", "cfg5", "cfg2-small", "cfg2-s0", "cfg4-s0", "cfg4-s3", "kmeans", "cfg3-rows", "tau-sweep", "cfg2-proj", "launch-check", "overlap"])
    ap.add_argument("--no-targets", action="store_true",
                    help="default workload only: skip the config 3 / 4 / 5 measurements that follow the headline")
    ap.add_argument("--cpu-sample", type=int, default=0,
                    help="requests per oracle timing (0: sized for 10-30 s of CPU work)")
    ap.add_argument("--batch", type=int, default=16, help="batch of the latency workload (cfg5): 1, 4 or 16")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--same-batch", action="store_true", help="every rank serves the same batch")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_ranks(args.gpus))
    if args.workload == "launch-check":
        run_launch_check(args)
    elif args.workload == "kmeans":
        run_kmeans(args)
    elif args.workload == "cfg2-proj" and args.impl == "ours":
        run_projected(args)
    elif args.workload == "tau-sweep":
        run_tau_sweep(args)
    elif args.workload == "overlap":
        run_overlap(args)
    elif args.workload == "cfg3-rows" and args.impl == "ours":
        run_rowshard(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
