#!/usr/bin/env python
"""Benchmark of the DIVISION compress / decompress pair on B200.

One "step" = one pass of the whole hot path over the ResNet-50 / ImageNet-shaped activation set
(batch 64, fp32, B = 8, Q = 2; five maps): every map is compressed (Algorithm 1, forward loop), then
every map is decompressed (Algorithm 1, backward loop).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is GB of activation taken through the pair per second
(raw activation bytes / (compress time + decompress time)), inputs resident in HBM.
`--impl reference` times the CPU checker (oracle/) on host cores instead.
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
sys.path.insert(0, ROOT)

METRIC = "compress+decompress GB/s of activation"
UNIT = "GB/s"
WORKLOAD = "config2: ResNet-50 ImageNet-shaped set, batch 64 fp32, B=8, Q=2, fp32 LFC (5 maps, 590 MB)"
MIN_TIMED_MS = 1000.0        # device time the headline rests on (the timed loop of --steps steps is repeated)
MAX_REPEATS = 2000
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# DRAM bytes per launch of profiled kernels come from profiles/traffic.json (written next to the ncu summaries):
# each entry names the kernel, the map, dram__bytes_read.sum / dram__bytes_write.sum of one capture and the
# SHA-256 over the kernel's source files at capture time.  An entry whose sources have changed since is not used.
def ncu_traffic(kernel: str, map_label: str):
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            table = json.load(f)
        e = table[f"{kernel} on {map_label}"]
        h = hashlib.sha256()
        for rel in e["sources"]:
            with open(os.path.join(ROOT, rel), "rb") as f:
                h.update(f.read())
        if h.hexdigest() != e["sources_sha256"]:
            return None
        return int(e["dram_bytes_read"]) + int(e["dram_bytes_write"])
    except Exception:
        return None


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 6:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
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
            except ValueError:
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def aggregate_over_ranks(local_ms: float, local_units: float, dist=None, device=None):
    """Whole-job figures: time = max over ranks, units = sum over ranks (replicas: no data-path collective)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    import torch
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ----------------------------------------------------------------------------------------------
# reference arm / CPU baseline: the checker as it stands, on host cores
# ----------------------------------------------------------------------------------------------
REFERENCE_SAMPLES_PER_MAP = 2


def oracle_step_inputs(samples_per_map: int):
    from paper_2208_04187_b200 import synth
    import numpy as np
    out = []
    for spec in synth.config_specs(2):
        x = np.concatenate([synth.make_sample(spec, i) for i in range(samples_per_map)])
        out.append((spec, x))
    return out


def oracle_step(inputs):
    from oracle import division_oracle as orc
    nbytes = 0
    for spec, x in inputs:
        comp = orc.compress(x, spec.block, spec.qbits, 0, spec.x_dtype, spec.lfc_dtype)
        orc.decompress(comp)
        nbytes += x.nbytes
    return nbytes


def cpu_threads_used() -> int:
    # the checker is plain NumPy elementwise code: one call runs on one thread
    return 1


_POOL_INPUTS = None


def _oracle_task(task):
    """One (map, sample) unit of the workload in a worker process (inputs inherited by fork, not pickled)."""
    from oracle import division_oracle as orc
    m, i = task
    spec, x = _POOL_INPUTS[m]
    comp = orc.compress(x[i:i + 1], spec.block, spec.qbits, 0, spec.x_dtype, spec.lfc_dtype, first_sample=i)
    orc.decompress(comp)
    return x[i:i + 1].nbytes


def time_oracle_all_cores(inputs):
    """The checker as it stands, samples dealt to one worker process per host core (samples are independent units)."""
    import multiprocessing as mp
    global _POOL_INPUTS
    _POOL_INPUTS = inputs
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    tasks = [(m, i) for m, (spec, x) in enumerate(inputs) for i in range(x.shape[0])]
    tasks.sort(key=lambda t: -inputs[t[0]][1][t[1]:t[1] + 1].nbytes)          # large units first
    with mp.get_context("fork").Pool(cores) as pool:
        pool.map(_oracle_task, tasks[:cores])                                  # start-up and imports, untimed
        t0 = time.perf_counter()
        nbytes = sum(pool.map(_oracle_task, tasks, chunksize=1))
        dt = time.perf_counter() - t0
    _POOL_INPUTS = None
    return nbytes / dt / 1e9, cores


def time_oracle(steps: int, warmup: int, samples_per_map: int):
    inputs = oracle_step_inputs(samples_per_map)
    for _ in range(warmup):
        oracle_step(inputs)
    t0 = time.perf_counter()
    nbytes = 0
    for _ in range(steps):
        nbytes += oracle_step(inputs)
    dt = time.perf_counter() - t0
    return nbytes / dt / 1e9, dt * 1e3 / max(steps, 1)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    gbs, ms = time_oracle(args.steps, args.warmup, REFERENCE_SAMPLES_PER_MAP)
    sample = (f"first {REFERENCE_SAMPLES_PER_MAP} samples of each of the 5 maps per step "
              f"({REFERENCE_SAMPLES_PER_MAP}/64 of the workload)")
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "CPU checker (oracle/), NumPy, untuned; " + sample},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cpu_threads_used(), "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def measure_train_step(device, ev, barrier, batch=64, steps=3):
    """Forward + backward of a randomly initialised torchvision ResNet-50 on synthetic images, with plain autograd
    and with the activation cache of Algorithm 1; memory in the paper's way (allocated after forward minus after
    backward), time with CUDA events.  The model is a stand-in for the paper's workload; its kernels are torch's."""
    import torch
    import torchvision

    from paper_2208_04187_b200 import autograd as dv

    torch.manual_seed(0)
    x = torch.randn(batch, 3, 224, 224, device=device)

    def run(model, make_cache):
        model.zero_grad(set_to_none=True)
        barrier()
        base = torch.cuda.memory_allocated(device)
        t0, t1 = ev(), ev()
        t0.record()
        cache = make_cache()
        if cache is None:
            loss = model(x).square().mean()
        else:
            with cache:
                loss = model(x).square().mean()
        barrier()
        after_fwd = torch.cuda.memory_allocated(device)
        loss.backward()
        t1.record()
        barrier()
        after_bwd = torch.cuda.memory_allocated(device)
        grads = sum(p.grad.numel() * p.grad.element_size() for p in model.parameters() if p.grad is not None)
        del loss
        return {"ms": t0.elapsed_time(t1), "activation_bytes": after_fwd - base, "after_bwd_minus_grads": after_bwd - base - grads,
                "cache": cache}

    out = {}
    for name in ("plain", "division"):
        model = torchvision.models.resnet50(weights=None).to(device).train()
        make_cache = lambda: None
        if name == "division":
            dv.to_division_modules(model)
            make_cache = lambda: dv.DivisionCache(block=8, qbits=2, seed=1)
        for _ in range(2):
            run(model, make_cache)
        rs = [run(model, make_cache) for _ in range(steps)]
        out[name] = {"ms_per_step": statistics.mean(r["ms"] for r in rs),
                     "activation_bytes_after_forward": int(statistics.mean(r["activation_bytes"] for r in rs))}
        if name == "division":
            c = rs[-1]["cache"]
            out[name].update({"maps_compressed": c.maps, "raw_bytes_of_those_maps": c.raw_bytes, "cached_bytes": c.cached_bytes,
                              "ratio_of_those_maps": c.raw_bytes / max(c.cached_bytes, 1)})
        del model, rs
        torch.cuda.empty_cache()
    out["what"] = (f"torchvision ResNet-50 (random init), batch {batch} x 3 x 224 x 224 fp32 synthetic, forward + backward; "
                   "activation bytes = allocated after forward - before the step (the paper's MEM_after_fwd - MEM_after_bwd, "
                   "gradients excluded); division = DivisionCache(B=8, Q=2) + ReLU with packed 1-bit masks")
    out["activation_memory_ratio"] = out["plain"]["activation_bytes_after_forward"] / max(out["division"]["activation_bytes_after_forward"], 1)
    out["time_ratio_division_over_plain"] = out["division"]["ms_per_step"] / out["plain"]["ms_per_step"]
    return out


def measure_configs(device, ev, barrier, configs, peak, names, dec_names):
    """The other workload configurations (seeded synthetic maps shaped like the paper's ResNet-18 / WRN-28-10 /
    DenseNet-121 activations): every tensor compressed and decompressed on its own, back-to-back calls between two
    CUDA events.  A tensor smaller than the L2 rotates over a pool of copies larger than twice the L2, inputs and
    outputs alike, so that no call finds its data there."""
    import torch

    from paper_2208_04187_b200 import binding, synth

    L2_BYTES = 126 * 2 ** 20
    out = {}
    for cfg in configs:
        rows = []
        raw_total, c_total, d_total = 0, 0.0, 0.0
        for spec in synth.config_specs(cfg):
            x = torch.from_numpy(synth.make_input(spec))
            if spec.x_dtype == "bf16":
                x = x.view(torch.bfloat16)
            x = x.to(device)
            nbytes = x.numel() * x.element_size()
            pool = 2 if nbytes > L2_BYTES else int(2 * L2_BYTES // nbytes) + 2
            xs = [x] + [x.clone() for _ in range(pool - 1)]
            outs = [torch.empty_like(x) for _ in range(pool)]
            codec = binding.Codec(*spec.shape, spec.block, spec.qbits, spec.x_dtype, spec.lfc_dtype, device=device)
            plan = codec.plan()
            algo = int(codec.layout.raw_bytes) + int(codec.layout.closed_form_bytes)
            reps = max(10, min(60, int(2e9 // algo)))
            for k in range(3):
                codec.compress(xs[k % pool], seed=0)
                codec.decompress(out=outs[k % pool])
            barrier()
            a, b = ev(), ev()
            a.record()
            for k in range(reps):
                codec.compress(xs[k % pool], seed=0)
            b.record()
            barrier()
            c_us = a.elapsed_time(b) * 1e3 / reps
            assert codec.device_status() == binding.DIV_OK
            a, b = ev(), ev()
            a.record()
            for k in range(reps):
                codec.decompress(out=outs[k % pool])
            b.record()
            barrier()
            d_us = a.elapsed_time(b) * 1e3 / reps
            rows.append({"map": "x".join(map(str, spec.shape)) + f" {spec.x_dtype} {spec.kind} B{spec.block} Q{spec.qbits}",
                         "MB": round(nbytes / 1e6, 1), "pool": pool, "calls": reps,
                         "compress_kernel": names[int(plan.fused)], "compress_us": round(c_us, 1),
                         "compress_GBps": round(algo / c_us / 1e3, 1), "compress_frac": round(algo / c_us / 1e3 / peak, 3),
                         "decompress_kernel": dec_names[int(plan.decompress_fast)], "decompress_us": round(d_us, 1),
                         "decompress_GBps": round(algo / d_us / 1e3, 1), "decompress_frac": round(algo / d_us / 1e3 / peak, 3)})
            raw_total += nbytes
            c_total += c_us
            d_total += d_us
            del xs, outs, x, codec
            torch.cuda.empty_cache()
        out[f"config{cfg}"] = {"tensors": len(rows), "raw_MB": round(raw_total / 1e6, 1),
                               "compress_us_sum": round(c_total, 1), "decompress_us_sum": round(d_total, 1),
                               "GBps_of_activation": round(raw_total / (c_total + d_total) / 1e3, 1), "per_tensor": rows}
    out["what"] = ("every tensor of the configuration on its own: back-to-back calls through the C ABI between two CUDA events, "
                   "inputs and outputs rotating over a pool of copies > 2 x L2 where the tensor is smaller than the L2; us per call "
                   "include the launch cost a caller sees (the smallest maps are bound by it); GBps = algorithmic bytes "
                   "(raw + closed-form compressed) / time; frac = GBps / measured HBM peak")
    return out


# ----------------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------------
def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2208_04187_b200 import binding, build, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    build.build()
    binding.lib()

    kernel_names_all = {8: "line_fused_kernel", 7: "plane_fused_kernel", 6: "staged_kernel", 5: "line_stats_kernel + line_quant_kernel", 4: "plane_stats_kernel + plane_quant_kernel",
                        3: "lagged_kernel", 2: "fused_v_kernel", 1: "fused_compress_kernel", 0: "lfc_stats_kernel + quant_pack_kernel"}
    dec_names_all = {1: "decompress_quad_kernel", 2: "decompress_flat_kernel", 3: "decompress_line_kernel", 0: "decompress_general_kernel"}
    specs = synth.config_specs(2)
    if args.maps:
        specs = [specs[int(i)] for i in args.maps.split(",")]
    host_x = [torch.from_numpy(synth.make_input(s)).pin_memory() for s in specs]
    dev_x = [h.to(device, non_blocking=True) for h in host_x]
    codecs = [binding.Codec(*s.shape, s.block, s.qbits, s.x_dtype, s.lfc_dtype, device=device) for s in specs]
    dev_out = [torch.empty_like(x) for x in dev_x]
    plans = [c.plan(args.compress_flags) for c in codecs]
    raw_bytes = sum(int(c.layout.raw_bytes) for c in codecs)
    comp_bytes = sum(int(c.layout.closed_form_bytes) for c in codecs)
    kernels_per_step = sum((2 if p.fused in (0, 4, 5) else 1) + 1 for p in plans)      # compress launches + one decompress launch
    torch.cuda.synchronize()

    def step(record=None):
        for i, c in enumerate(codecs):
            if record is not None:
                record[0][i][0].record()
            c.compress(dev_x[i], seed=0, flags=args.compress_flags)
            if record is not None:
                record[0][i][1].record()
        for i, c in enumerate(codecs):
            if record is not None:
                record[1][i][0].record()
            c.decompress(out=dev_out[i])
            if record is not None:
                record[1][i][1].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    for c in codecs:
        assert c.device_status() == binding.DIV_OK

    ev = lambda: torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    barrier()
    # the timed region: exactly args.steps steps between two events, nothing else on the stream; repeated (same
    # number of steps each time) until at least MIN_TIMED_MS of device time has been measured, so that a short
    # --steps still rests on a second of samples.  ms_per_step is the median over the repeats.
    rep_ms = []
    while True:
        t_start, t_end = ev(), ev()
        t_start.record()
        for k in range(args.steps):
            step()
        t_end.record()
        barrier()
        rep_ms.append(t_start.elapsed_time(t_end))
        if sum(rep_ms) >= MIN_TIMED_MS or len(rep_ms) >= args.max_repeats:
            break
    total_ms = statistics.median(rep_ms)
    # a second, instrumented pass for the per-call figures (an event pair around every call costs a few us per
    # call, which is why it is kept out of the timed region above)
    rec_steps = max(3, min(args.steps, 100))
    records = [[[(ev(), ev()) for _ in codecs] for _ in range(2)] for _ in range(rec_steps)]
    for k in range(rec_steps):
        step(records[k])
    barrier()
    clocks = sampler.stop()

    comp_ms = [statistics.mean(records[k][0][i][0].elapsed_time(records[k][0][i][1]) for k in range(rec_steps))
               for i in range(len(codecs))]
    dec_ms = [statistics.mean(records[k][1][i][0].elapsed_time(records[k][1][i][1]) for k in range(rec_steps))
              for i in range(len(codecs))]

    # ---- the dominant kernel alone: back-to-back launches of the slowest compress call, two input buffers
    # ---- alternating (410 MB, far above the L2), no events between the calls
    dom = max(range(len(specs)), key=lambda i: comp_ms[i])
    alt = torch.empty_like(dev_x[dom]).copy_(dev_x[dom])
    dom_n = max(20, min(args.steps, 100))
    for k in range(3):
        codecs[dom].compress(alt if k % 2 else dev_x[dom], seed=0, flags=args.compress_flags)
    barrier()
    d0, d1 = ev(), ev()
    d0.record()
    for k in range(dom_n):
        codecs[dom].compress(alt if k % 2 else dev_x[dom], seed=0, flags=args.compress_flags)
    d1.record()
    barrier()
    dom_ms = d0.elapsed_time(d1) / dom_n
    del alt

    # ---- end to end through the C ABI with host buffers: H2D of x, compress, decompress, D2H of x_hat ----
    host_out = [torch.empty_like(h).pin_memory() for h in host_x]
    e2e_steps = max(2, min(args.steps, 5))

    # three streams, so that the two PCIe directions and the kernels overlap: copy-in -> (compress, decompress) -> copy-out
    # per map, each stage ordered after its predecessor by events; a buffer is reused only after its last reader is done
    s_main = torch.cuda.current_stream(device)
    s_in, s_out = torch.cuda.Stream(device), torch.cuda.Stream(device)
    ev_in = [torch.cuda.Event() for _ in codecs]       # x[i] has arrived on the device
    ev_done = [torch.cuda.Event() for _ in codecs]     # compress + decompress of map i have run (x[i] may be overwritten)
    ev_out = [torch.cuda.Event() for _ in codecs]      # x_hat[i] has reached the host (dev_out[i] may be overwritten)

    def e2e_step(first=False):
        for i, c in enumerate(codecs):
            with torch.cuda.stream(s_in):
                if not first:
                    s_in.wait_event(ev_done[i])
                dev_x[i].copy_(host_x[i], non_blocking=True)
                ev_in[i].record(s_in)
            s_main.wait_event(ev_in[i])
            if not first:
                s_main.wait_event(ev_out[i])
            c.compress(dev_x[i], seed=0, flags=args.compress_flags)
            c.decompress(out=dev_out[i])
            ev_done[i].record(s_main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i])
                host_out[i].copy_(dev_out[i], non_blocking=True)
                ev_out[i].record(s_out)

    def e2e_join():
        for e in ev_out:
            s_main.wait_event(e)

    e2e_step(first=True)
    e2e_join()
    barrier()
    e0, e1 = ev(), ev()
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e2e_join()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps

    # ---- the per-plane form (one bfloat16 (delta, Delta) pair per plane): same maps, same order, own timed loop ----
    plane_groups = None
    if not args.no_plane_groups:
        pg = [binding.PlaneGroupCodec(*s.shape, s.block, s.qbits, s.x_dtype, s.lfc_dtype, device=device) for s in specs]
        pg_plans = [c.plan() for c in pg]
        pg_steps = max(3, min(args.steps, 100))

        def pg_step(record=None):
            for i, c in enumerate(pg):
                if record is not None:
                    record[0][i][0].record()
                c.compress(dev_x[i], seed=0)
                if record is not None:
                    record[0][i][1].record()
            for i, c in enumerate(pg):
                if record is not None:
                    record[1][i][0].record()
                c.decompress(out=dev_out[i])
                if record is not None:
                    record[1][i][1].record()

        for _ in range(3):
            pg_step()
        barrier()
        p0, p1 = ev(), ev()
        p0.record()
        for k in range(pg_steps):
            pg_step()
        p1.record()
        barrier()
        pg_ms = p0.elapsed_time(p1) / pg_steps
        pg_rec = [[[(ev(), ev()) for _ in pg] for _ in range(2)] for _ in range(pg_steps)]
        for k in range(pg_steps):
            pg_step(pg_rec[k])
        barrier()
        pg_comp = [statistics.mean(pg_rec[k][0][i][0].elapsed_time(pg_rec[k][0][i][1]) for k in range(pg_steps))
                   for i in range(len(pg))]
        pg_dec = [statistics.mean(pg_rec[k][1][i][0].elapsed_time(pg_rec[k][1][i][1]) for k in range(pg_steps))
                  for i in range(len(pg))]
        pg_names = {1: "pg_strip_kernel", 2: "pg_small_kernel", 0: "pg_general_kernel"}
        pg_dec_names = {1: "pg_decompress_quad_kernel", 2: "pg_decompress_flat_kernel", 0: "pg_decompress_general_kernel"}
        pg_algo = [int(c.layout.raw_bytes) + int(c.layout.closed_form_bytes) for c in pg]
        pg_dom = max(range(len(pg)), key=lambda i: pg_comp[i])
        pg_peak, pg_peak_kind = measured_peak()
        pg_dom_gbs = pg_algo[pg_dom] / (pg_comp[pg_dom] * 1e-3) / 1e9
        plane_groups = {
            "what": "the same step with one bfloat16 (delta, Delta) pair per (sample, channel) plane "
                    "(div_planegroup_compress / div_planegroup_decompress), this rank",
            "value": raw_bytes / (pg_ms * 1e-3) / 1e9, "unit": UNIT, "steps": pg_steps, "ms_per_step": pg_ms,
            "compression_ratio": raw_bytes / sum(int(c.layout.closed_form_bytes) for c in pg),
            "gpu_launches": 2 * len(pg) * pg_steps,
            "per_map": [{"map": "x".join(map(str, s.shape)), "compress_kernel": pg_names[int(p.fused)],
                         "decompress_kernel": pg_dec_names[int(p.decompress_fast)],
                         "compress_us": round(cm * 1e3, 2), "compress_GBps": round(b / cm / 1e6, 1),
                         "decompress_us": round(dm * 1e3, 2), "decompress_GBps": round(b / dm / 1e6, 1)}
                        for s, p, cm, dm, b in zip(specs, pg_plans, pg_comp, pg_dec, pg_algo)],
            "roofline": {"bound": "hbm", "kernel": pg_names[int(pg_plans[pg_dom].fused)] + " on " +
                         "x".join(map(str, specs[pg_dom].shape)), "achieved": pg_dom_gbs, "peak": pg_peak,
                         "unit": "GB/s", "frac": pg_dom_gbs / pg_peak, "peak_kind": f"of {pg_peak_kind}",
                         "traffic": ncu_traffic(pg_names[int(pg_plans[pg_dom].fused)], "x".join(map(str, specs[pg_dom].shape))),
                         "algorithmic_bytes_per_launch": pg_algo[pg_dom]},
        }

    # ---- ReLU / dropout operators with a packed 1-bit mask, on the largest map of the set (this rank) ----
    mask_ops = None
    if not args.no_masks:
        big = max(range(len(specs)), key=lambda i: dev_x[i].numel())
        xs, ys = dev_x[big], dev_out[big]
        total = xs.numel()
        mbytes = binding.div_mask_bytes(total)
        mbuf = torch.zeros(mbytes, dtype=torch.uint8, device=device)
        # a second pair of buffers, so that successive calls do not find their input in the 126 MB L2
        xs2, ys2 = torch.empty_like(xs).copy_(xs), torch.empty_like(xs)
        pairs = [(xs, ys), (xs2, ys2)]
        stream = binding.current_stream_handle()
        dt = specs[big].x_dtype
        calls = {
            "relu_forward": lambda a, b: binding.div_relu_forward(a.data_ptr(), b.data_ptr(), mbuf.data_ptr(), mbytes, total, dt, stream),
            "dropout_forward": lambda a, b: binding.div_dropout_forward(a.data_ptr(), b.data_ptr(), mbuf.data_ptr(), mbytes, total, 1, 6554, dt, stream),
            "mask_backward": lambda a, b: binding.div_mask_backward(mbuf.data_ptr(), mbytes, a.data_ptr(), b.data_ptr(), total, dt, stream),
        }
        m_steps = max(4, min(args.steps, 50))
        m_peak, m_peak_kind = measured_peak()
        algo = 2 * total * xs.element_size() + total // 8
        mask_ops = {"what": "mask operators on " + "x".join(map(str, specs[big].shape)) + " (two buffer pairs alternate: inputs never L2-resident)",
                    "algorithmic_bytes_per_launch": algo, "steps": m_steps, "kernels": {}}
        for name, fn in calls.items():
            for k in range(3):
                fn(*pairs[k % 2])
            barrier()
            evs = [(ev(), ev()) for _ in range(m_steps)]
            for k in range(m_steps):
                evs[k][0].record()
                fn(*pairs[k % 2])
                evs[k][1].record()
            barrier()
            us = statistics.mean(a.elapsed_time(b) for a, b in evs) * 1e3
            gbs = algo / (us * 1e-6) / 1e9
            mask_ops["kernels"][name] = {"us": round(us, 2), "roofline": {"bound": "hbm", "achieved": gbs, "peak": m_peak, "unit": "GB/s",
                                                                         "frac": gbs / m_peak, "peak_kind": f"of {m_peak_kind}", "traffic": None}}
        mask_ops["gpu_launches"] = 3 * (m_steps + 3)
        del xs2, ys2

    # ---- 1-D maps (token activations; N x C x 1 x W descriptors), three transformer / MLP-shaped tensors ----
    one_d = None
    if not args.no_one_d:
        shapes_1d = [("32x512x768 B=8 Q=4", (32, 512, 768), 8, 4), ("64x196x768 B=16 Q=2", (64, 196, 768), 16, 2),
                     ("64x784x192 B=64 Q=2", (64, 784, 192), 64, 2)]
        gen = torch.Generator(device=device).manual_seed(11)
        t_x = [torch.randn(m, c, 1, n, device=device, generator=gen) for _, (m, c, n), _, _ in shapes_1d]
        t_out = [torch.empty_like(x) for x in t_x]
        t_codec = [binding.Codec(m, c, 1, n, b, q, device=device) for _, (m, c, n), b, q in shapes_1d]
        t_steps = max(4, min(args.steps, 50))

        def t_step(record=None):
            for i, c in enumerate(t_codec):
                if record is not None:
                    record[0][i][0].record()
                c.compress(t_x[i], seed=0)
                if record is not None:
                    record[0][i][1].record()
            for i, c in enumerate(t_codec):
                if record is not None:
                    record[1][i][0].record()
                c.decompress(out=t_out[i])
                if record is not None:
                    record[1][i][1].record()

        for _ in range(3):
            t_step()
        barrier()
        q0, q1 = ev(), ev()
        q0.record()
        for k in range(t_steps):
            t_step()
        q1.record()
        barrier()
        t_ms = q0.elapsed_time(q1) / t_steps
        t_rec = [[[(ev(), ev()) for _ in t_codec] for _ in range(2)] for _ in range(t_steps)]
        for k in range(t_steps):
            t_step(t_rec[k])
        barrier()
        t_raw = sum(int(c.layout.raw_bytes) for c in t_codec)
        t_peak, t_peak_kind = measured_peak()
        rows = []
        for i, (name, _, _, _) in enumerate(shapes_1d):
            cm = statistics.mean(t_rec[k][0][i][0].elapsed_time(t_rec[k][0][i][1]) for k in range(t_steps))
            dm = statistics.mean(t_rec[k][1][i][0].elapsed_time(t_rec[k][1][i][1]) for k in range(t_steps))
            b = int(t_codec[i].layout.raw_bytes) + int(t_codec[i].layout.closed_form_bytes)
            rows.append({"map": name, "compress_kernel": kernel_names_all[int(t_codec[i].plan().fused)],
                         "compress_us": round(cm * 1e3, 2), "compress_GBps": round(b / cm / 1e6, 1),
                         "compress_frac_of_peak": round(b / cm / 1e6 / t_peak, 3),
                         "decompress_us": round(dm * 1e3, 2), "decompress_GBps": round(b / dm / 1e6, 1),
                         "decompress_frac_of_peak": round(b / dm / 1e6 / t_peak, 3)})
        one_d = {"what": "1-D maps (Minibatch x Channel x N as N x C x 1 x W), compress then decompress of three tensors per step, this rank",
                 "value": t_raw / (t_ms * 1e-3) / 1e9, "unit": UNIT, "steps": t_steps, "ms_per_step": t_ms,
                 "peak": t_peak, "peak_kind": f"of {t_peak_kind}", "gpu_launches": 9 * (t_steps + 3), "per_map": rows}
        del t_x, t_out, t_codec

    # ---- one 3-D map (Minibatch x Channel x D x H x W) ----
    three_d = None
    if not args.no_one_d:
        shp, b3, q3 = (8, 64, 16, 56, 56), 8, 2
        desc3 = binding.make_desc_3d(*shp, b3, q3)
        lo3 = binding.div_compressed_bytes_3d(desc3)
        gen = torch.Generator(device=device).manual_seed(12)
        pairs3 = [(torch.randn(*shp, device=device, generator=gen), torch.empty(shp, device=device)) for _ in range(2)]
        blob3 = torch.empty(int(lo3.total_bytes), dtype=torch.uint8, device=device)
        ws3 = torch.empty(int(lo3.workspace_bytes), dtype=torch.uint8, device=device)
        stream = binding.current_stream_handle()
        n3 = max(4, min(args.steps, 20))
        ce3 = [(ev(), ev()) for _ in range(n3)]
        de3 = [(ev(), ev()) for _ in range(n3)]
        for k in range(-3, n3):
            xin, xout = pairs3[k % 2]
            if k >= 0:
                ce3[k][0].record()
            binding.div_compress_3d(desc3, xin.data_ptr(), blob3.data_ptr(), blob3.numel(), ws3.data_ptr(), ws3.numel(), 0, stream)
            if k >= 0:
                ce3[k][1].record()
                de3[k][0].record()
            binding.div_decompress_3d(desc3, blob3.data_ptr(), blob3.numel(), xout.data_ptr(), stream)
            if k >= 0:
                de3[k][1].record()
        barrier()
        c_us = statistics.mean(a.elapsed_time(b) for a, b in ce3) * 1e3
        d_us = statistics.mean(a.elapsed_time(b) for a, b in de3) * 1e3
        b3y = int(lo3.raw_bytes) + int(lo3.closed_form_bytes)
        pk3, pk3_kind = measured_peak()
        three_d = {"what": "3-D map " + "x".join(map(str, shp)) + f" fp32, B={b3}, Q={q3}, this rank",
                   "compression_ratio": int(lo3.raw_bytes) / int(lo3.closed_form_bytes), "steps": n3,
                   "compress_kernel": "lfc_stats3d_strip_kernel + quant3d_strip_kernel", "compress_us": round(c_us, 1),
                   "compress_GBps": round(b3y / c_us / 1e3, 1), "compress_frac_of_peak": round(b3y / c_us / 1e3 / pk3, 3),
                   "decompress_kernel": "decompress3d_strip_kernel", "decompress_us": round(d_us, 1),
                   "decompress_GBps": round(b3y / d_us / 1e3, 1), "decompress_frac_of_peak": round(b3y / d_us / 1e3 / pk3, 3),
                   "peak_kind": f"of {pk3_kind}", "gpu_launches": 3 * (n3 + 3)}
        del pairs3, blob3, ws3

    # ---- the other workload configurations, tensor by tensor ----
    other_configs = None
    if args.configs and not args.maps and rank == 0:
        dev_x.clear()                   # hand the benchmark's device buffers back first
        dev_out.clear()
        for c in codecs:
            c.blob = c.workspace = None
        torch.cuda.empty_cache()
        cfg_peak, _ = measured_peak()
        other_configs = measure_configs(device, ev, barrier, [int(c) for c in args.configs.split(",")], cfg_peak,
                                        kernel_names_all, dec_names_all)

    # ---- Algorithm 1 around a synthetic ResNet-50 step: activation memory (after forward - after backward) and
    # ---- forward+backward time, plain autograd against the cache (B=8, Q=2; ReLU with packed masks) ----
    train_step = None
    if not args.no_train_step and not args.maps:
        dev_x.clear()                   # hand the benchmark's device buffers back before the model allocates
        dev_out.clear()
        for c in codecs:
            c.blob = c.workspace = None
        torch.cuda.empty_cache()
        try:
            train_step = measure_train_step(device, ev, barrier)
        except Exception as exc:       # the headline line must not depend on torchvision or on free memory
            train_step = {"error": f"{type(exc).__name__}: {exc}"}

    ms_per_step = total_ms / args.steps
    job_ms, job_bytes = aggregate_over_ranks(ms_per_step, float(raw_bytes), dist if world > 1 else None, device)
    e2e_job_ms, _ = aggregate_over_ranks(e2e_ms, float(raw_bytes), dist if world > 1 else None, device)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    algo_bytes = [int(c.layout.raw_bytes) + int(c.layout.closed_form_bytes) for c in codecs]
    comp_gbs = sum(algo_bytes) / (sum(comp_ms) * 1e-3) / 1e9
    dec_gbs = sum(algo_bytes) / (sum(dec_ms) * 1e-3) / 1e9
    kernel_names = kernel_names_all
    per_map = [{"map": "x".join(map(str, s.shape)), "compress_kernel": kernel_names[int(p.fused)],
                "compress_us": round(cm * 1e3, 2), "compress_GBps": round(b / cm / 1e6, 1),
                "decompress_us": round(dm * 1e3, 2), "decompress_GBps": round(b / dm / 1e6, 1)}
               for s, p, cm, dm, b in zip(specs, plans, comp_ms, dec_ms, algo_bytes)]
    # dominant kernel: the compress kernel with the largest share of the step's device time, timed alone above
    dom_gbs = algo_bytes[dom] / (dom_ms * 1e-3) / 1e9

    # CPU baseline: the checker on the whole workload once (after one warm-up on a slice)
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        inputs = [(sp, h.numpy()) for sp, h in zip(specs, host_x)]
        time_oracle(1, 0, 1)
        gbs1, _ = time_oracle(1, 0, 8)
        gbs, cores = time_oracle_all_cores(inputs)
        cpu = {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "the whole config-2 workload (5 maps, 64 samples each), one pass, NumPy checker as it stands, "
                         "samples dealt to one process per host core",
               "single_thread": {"value": gbs1, "cores": cpu_threads_used(), "sample": "first 8 samples of each of the 5 maps"}}

    line = {
        "metric": METRIC, "value": job_bytes / (job_ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": job_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD + (f" [maps {args.maps} only]" if args.maps else ""), "maps": [m["map"] for m in per_map],
                   "l2": "working set 1.2 GB per step, every buffer touched once per step: far above the 126 MB L2",
                   "order": "compress maps 0..4, then decompress maps 0..4",
                   "timing": f"value / ms_per_step: median of {len(rep_ms)} repeats of {args.steps} steps between two CUDA events "
                             f"(min {min(rep_ms) / args.steps:.4f} ms, max {max(rep_ms) / args.steps:.4f} ms per step), nothing else on the "
                             f"stream; per_map: a second pass of {rec_steps} steps with an event pair around every call; roofline: the "
                             "dominant kernel alone, back to back",
                   "ms_per_step_min": min(rep_ms) / args.steps, "ms_per_step_max": max(rep_ms) / args.steps, "repeats": len(rep_ms),
                   "multi_gpu": "replicas only: each rank runs the same set on its own GPU, no collective",
                   "compression_ratio": raw_bytes / comp_bytes, "per_map": per_map},
        "roofline": {"bound": "hbm", "kernel": kernel_names[int(plans[dom].fused)] + " on " + per_map[dom]["map"] +
                     f" ({dom_n} back-to-back calls between two CUDA events on its stream, two inputs alternating; "
                     "the span includes the 2-us workspace clear)",
                     "achieved": dom_gbs, "peak": peak, "unit": "GB/s", "frac": dom_gbs / peak, "us_per_launch": dom_ms * 1e3,
                     "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBps": dom_gbs / NOMINAL_HBM_GBS,
                     "traffic": ncu_traffic(kernel_names[int(plans[dom].fused)], per_map[dom]["map"]),
                     "algorithmic_bytes_per_launch": algo_bytes[dom]},
        "roofline_all_compress": {"bound": "hbm", "kernel": "all compress calls of the step", "achieved": comp_gbs,
                                  "peak": peak, "unit": "GB/s", "frac": comp_gbs / peak, "peak_kind": f"of {peak_kind}"},
        "roofline_all_decompress": {"bound": "hbm", "kernel": "all decompress calls of the step", "achieved": dec_gbs,
                                    "peak": peak, "unit": "GB/s", "frac": dec_gbs / peak, "peak_kind": f"of {peak_kind}"},
        "cpu_baseline": cpu,
        "plane_groups": plane_groups,
        "mask_ops": mask_ops,
        "one_d": one_d,
        "three_d": three_d,
        "configs": other_configs,
        "train_step": train_step,
        "e2e": {"value": raw_bytes * world / (e2e_job_ms * 1e-3) / 1e9, "unit": UNIT,
                "h2d_bytes_per_step": raw_bytes, "d2h_bytes_per_step": raw_bytes, "ms_per_step": e2e_job_ms,
                "steps": e2e_steps,
                "how": "pinned host buffers; per map: copy-in, compress, decompress, copy-out, on three streams ordered by "
                       "events so that the two PCIe directions and the kernels overlap"},
        "gpu_launches": kernels_per_step * args.steps * len(rep_ms),
        "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-plane-groups", action="store_true", help="skip the extra timed loop of the per-plane form")
    ap.add_argument("--no-train-step", action="store_true", help="skip the ResNet-50 forward+backward memory / time measurement")
    ap.add_argument("--no-one-d", action="store_true", help="skip the timing of the 1-D and 3-D maps")
    ap.add_argument("--no-masks", action="store_true", help="skip the timing of the ReLU / dropout mask operators")
    ap.add_argument("--max-repeats", type=int, default=MAX_REPEATS,
                    help="upper bound on the repeats of the timed loop (1 for a short run under a profiler)")
    ap.add_argument("--configs", default="0,1,3,4",
                    help="other workload configurations to time tensor by tensor (empty: none); config 2 is the headline")
    ap.add_argument("--maps", default="", help="comma-separated indices of the config-2 maps to run (profiling aid)")
    ap.add_argument("--compress-flags", type=int, default=0,
                    help="DIV_FLAG_* bits passed to div_compress_ex (profiling aid: 4 = strip ring kernel instead of the lagged one)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
