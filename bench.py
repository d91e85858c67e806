#!/usr/bin/env python
"""Benchmark of the sparse-convolution hot path (kernel-map build + forward) on B200.

One "step" is one pass of the whole hot path over one synthetic LiDAR sweep: build the kernel map of a
submanifold 3x3x3 layer from the voxel coordinates (hash insert, probe, pair compaction, tile plan) and run
the 64->64 bf16 forward on it.  The headline `value` is voxels per second through that pass with all
inputs resident in HBM; `e2e` is the same pass through the host-buffer entry point with the host<->device
copies inside the timed region.  The forward kernel is additionally timed alone (CUDA events on the launch
stream) for the roofline entry, in the same launch configuration.  Instead of flushing L2 between steps a rank
rotates over eight different sweeps, whose arrays together are about three times the size of L2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 runs one rank per GPU under torchrun (started by the caller, or by this script itself when it is run
plainly with --gpus N); each rank processes its own sweeps (seed = rank), no data-path collective (sweeps are
independent: coordinates with different batch indices never pair).
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2402_07710_b200 import workloads as wl  # noqa: E402

METRIC = "SubM3 64->64 bf16 layer on one LiDAR sweep (kmap build + forward) throughput"
UNIT = "Mvoxels/s"
WORKLOAD = "config 3: synthetic 64-beam LiDAR sweep, 1408x1600x41 grid, SubM 3x3x3, Cin=Cout=64, bf16"
CIN = COUT = 64
KVOL = 27
DTYPE = "bf16"
REFERENCE_SAMPLE_VOXELS = 10**9   # the oracle finishes the whole sweep in a fraction of a second: no sub-sampling
# DRAM bytes (read + write) of one forward launch on sweep 0, from one profiler capture of this kernel
# (dram__bytes_read.sum + dram__bytes_write.sum with the profiler's cache flush before the launch).  It is a
# recorded figure, not measured by this script: the line says so in `traffic_source`.
FORWARD_DRAM_TRAFFIC_BYTES = 15_232_512
FORWARD_DRAM_TRAFFIC_SOURCE = ("one profiler capture of k_forward_tc<64,64> on sweep 0 (DRAM bytes read + written per launch, "
                               "caches flushed before the launch); recorded, not measured in this run")
# Our kernels launched per step: k_fill_regions (table, filter, totals), k_insert, k_probe_rows (every offset of a row
# per thread), k_subm_emit (on a second
# stream), k_sort_rows_coop (row keys + radix sort, one cooperative launch), k_tile_plan_rows (its last block also
# orders the tiles and reports to the host) for the kernel map, + k_forward_tc.
OUR_LAUNCHES_PER_STEP = 7
ROTATION = 8   # sweeps a rank rotates over (about 45 MB of arrays each)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


def kmap_algorithmic_bytes(n, pairs):
    """Compulsory bytes of one submanifold kernel-map build: read the coordinates (16 B per row), fill and write a
    location table of two slots of 12 bytes per row (keys + rows), write the offset table (4 * K^3 B per row) and
    the pair lists (8 B per pair)."""
    return n * (16 + 2 * 2 * 12 + 4 * KVOL) + 8 * pairs


def forward_algorithmic_bytes(n_in, n_out, pairs):
    """Compulsory HBM bytes of one forward launch: read every input row once, write every output row once,
    read the weights once, read the kernel map once in its cheaper form (pairs or dense table)."""
    e = 2
    return n_in * CIN * e + n_out * COUT * e + KVOL * CIN * COUT * e + min(8 * pairs, 4 * KVOL * n_out)


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def count(self) -> int:
        """Samples written so far."""
        try:
            with open(self.file.name) as f:
                return sum(1 for line in f if line.count(",") >= 8)
        except OSError:
            return 0

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file.read().splitlines():
            f = [v.strip() for v in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.file.name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def time_oracle(coords, seed, sample_voxels):
    """The oracle as it stands on a bounded sample: the first `sample_voxels` voxels in lexicographic order
    (a contiguous x-slab of the sweep, so the neighbourhood structure is kept)."""
    import oracle
    order = np.lexsort((coords[:, 3], coords[:, 2], coords[:, 1], coords[:, 0]))
    sub = np.ascontiguousarray(coords[order[:sample_voxels]])
    x = wl.features(len(sub), CIN, DTYPE, seed)
    w = wl.weights(KVOL, CIN, COUT, DTYPE, seed)
    t0 = time.perf_counter()
    km = oracle.build_kmap(sub, 3, 1, 1, True)
    t1 = time.perf_counter()
    ref = oracle.forward(x, w, km["oft"])
    t2 = time.perf_counter()
    return len(sub), t1 - t0, t2 - t1, oracle.num_threads(), dict(coords=sub, x=x, w=w, ref=ref, pairs=len(km["pair_in"]))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    coords = wl.lidar_sweep(0)
    total = 0.0
    n = 0
    threads = 1
    for i in range(args.warmup + args.steps):
        n, tk, tf, threads, _ = time_oracle(coords, 0, REFERENCE_SAMPLE_VOXELS)
        if i >= args.warmup:
            total += tk + tf
    ms = 1e3 * total / args.steps
    value = n / (ms * 1e-3) / 1e6
    sample = f"the whole config-3 sweep ({n} voxels), kmap build + forward per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2402_07710_b200 import binding, sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU path"
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    binding.load()

    def barrier():
        if world > 1:
            dist.barrier()

    # Weak scaling: every rank owns its own sweeps.  A rank rotates over ROTATION different sweeps, so that the
    # arrays a step touches (coordinates, features, output, and for the forward-alone loop the kernel maps:
    # about 45 MB per sweep, 360 MB in all) were last used 315 MB of traffic ago and are no longer in the
    # 126 MB L2 when the step runs: inputs larger than L2 instead of a flush between steps.
    seed = sharding.sweep_seed(rank)
    sweeps = []
    for j in range(ROTATION):
        sj = seed + 1000 * j
        cj = wl.lidar_sweep(sj)
        sweeps.append(dict(seed=sj, coords_np=cj, n=len(cj), coords=torch.from_numpy(cj).cuda(),
                           x=torch.from_numpy(wl.features(len(cj), CIN, DTYPE, sj)).to(torch.bfloat16).cuda(),
                           out=torch.empty(len(cj), COUT, dtype=torch.bfloat16, device="cuda")))
    coords_np, n = sweeps[0]["coords_np"], sweeps[0]["n"]
    x_np = wl.features(n, CIN, DTYPE, seed)
    w_np = wl.weights(KVOL, CIN, COUT, DTYPE, seed)
    w = torch.from_numpy(w_np).to(torch.bfloat16).cuda()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # > 126 MB of L2 (profiler and single-launch paths)
    stream = torch.cuda.current_stream()
    coords, x, out = sweeps[0]["coords"], sweeps[0]["x"], sweeps[0]["out"]

    def step(j=0):   # one pass of the hot path: kernel map and forward of the layer, one call through the C ABI
        sw = sweeps[j % ROTATION]
        km, _ = binding.spconv_layer(sw["coords"], sw["x"], w, 1, 1, 3, True, out=sw["out"])
        return km

    km0 = step()
    pairs, n_tiles, blocks = km0.total_pairs, km0.n_tiles, km0.tile_blocks
    if args.only:   # short launch sequences for profiler captures; prints no bench line
        for _ in range(3):
            if args.only == "forward":
                flush.zero_()
                binding.spconv_forward(x, w, km0, out=out)
            else:
                step().close()
        torch.cuda.synchronize()
        print(json.dumps({"only": args.only, "n_voxels": n, "pairs": int(pairs), "tiles": int(n_tiles), "tile_blocks": int(blocks)}))
        return
    # The timed region lasts milliseconds, less than one nvidia-smi sampling period, so the clock sampler brackets
    # it with the same load: it starts before the warm-up, the warm-up goes on (beyond its W steps, untimed) until
    # the first sample is in, and after the timed region the same steps keep the GPU busy until three more are.
    sampler = ClockSampler(local_rank)
    sampler.start()
    warm = max(args.warmup, 3)
    for i in range(warm - 1):
        step(1 + i).close()
    t_hold = time.perf_counter()
    while sampler.proc is not None and sampler.count() < 1 and time.perf_counter() - t_hold < 2.0:
        step().close()
    torch.cuda.synchronize()
    samples_before = sampler.count()

    # ---------------- timed region: K steps over rotating sweeps, device-timed per step
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier(); torch.cuda.synchronize()
    t_wall0 = time.perf_counter()
    voxels_timed = 0
    for i in range(args.steps):
        sw = sweeps[(warm + i) % ROTATION]
        voxels_timed += sw["n"]
        ev[i][0].record(stream)
        km, _ = binding.spconv_layer(sw["coords"], sw["x"], w, 1, 1, 3, True, out=sw["out"])
        ev[i][1].record(stream)
        km.close()
    torch.cuda.synchronize(); barrier()
    wall = time.perf_counter() - t_wall0
    t_hold = time.perf_counter()
    while sampler.proc is not None and sampler.count() < samples_before + 3 and time.perf_counter() - t_hold < 2.0:
        step().close()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    clocks["window"] = "continuous load of the same steps from the warm-up through the timed region and on until three further samples"
    step_ms = [e[0].elapsed_time(e[1]) for e in ev]
    total_ms = sum(step_ms)

    # ---------------- the two stages separately (two calls, the host in between): kernel-map build, then forward
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
            torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for i in range(args.steps):
        sw = sweeps[(warm + i) % ROTATION]
        ev2[i][0].record(stream)
        km = binding.spconv_build_kmap(sw["coords"], 1, 1, 3, True)
        ev2[i][1].record(stream)
        binding.spconv_forward(sw["x"], w, km, out=sw["out"])
        ev2[i][2].record(stream)
        km.close()
    torch.cuda.synchronize()
    kmap_ms = [e[0].elapsed_time(e[1]) for e in ev2]
    fwd_cold_ms = [e[1].elapsed_time(e[2]) for e in ev2]
    two_call_ms = [e[0].elapsed_time(e[2]) for e in ev2]

    # ---------------- forward kernel alone, same launch configuration
    # (a) back to back over the rotating sweeps: every launch finds its features, kernel map and output out of L2
    kms = [binding.spconv_build_kmap(sw["coords"], 1, 1, 3, True) for sw in sweeps]
    rot_pairs = [int(k.total_pairs) for k in kms]
    for j in range(ROTATION):
        binding.spconv_forward(sweeps[j]["x"], w, kms[j], out=sweeps[j]["out"])
    torch.cuda.synchronize()
    rounds = 6

    def graph_time(launch_all, launches):
        """Device time per launch of a captured launch sequence (a CUDA graph replays it without the host's
        per-call latency, which otherwise exceeds the kernel's duration)."""
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            launch_all()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        graph.replay()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / launches

    def rotate_all():
        for _ in range(rounds):
            for j in range(ROTATION):
                binding.spconv_forward(sweeps[j]["x"], w, kms[j], out=sweeps[j]["out"])

    fwd_rot_ms = graph_time(rotate_all, rounds * ROTATION)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    rotate_all()
    b.record(stream)
    torch.cuda.synchronize()
    fwd_rot_host_ms = a.elapsed_time(b) / (rounds * ROTATION)   # the same sequence launched call by call from Python
    rot_n = sum(sw["n"] for sw in sweeps) / ROTATION
    rot_pairs_mean = sum(rot_pairs) / ROTATION
    for j in range(ROTATION):
        assert binding.spconv_last_device_status(kms[j]) == 0
    # (b) one launch at a time after a 256 MiB flush (also evicts the kernel's code and page tables)
    km = km0
    fwd_ms = []
    for i in range(8):
        flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        binding.spconv_forward(x, w, km, out=out)
        b.record(stream)
        torch.cuda.synchronize()
        if i >= 3:
            fwd_ms.append(a.elapsed_time(b))
    # (c) back-to-back launches on one sweep (L2-warm)
    reps = 50

    def same_sweep():
        for _ in range(reps):
            binding.spconv_forward(x, w, km, out=out)

    fwd_warm_ms = graph_time(same_sweep, reps)
    assert binding.spconv_last_device_status(km) == 0
    for k in kms:
        k.close()

    # ---------------- end to end from pinned host buffers through the host entry point
    hc = torch.from_numpy(coords_np).pin_memory()
    hx = torch.from_numpy(x_np).to(torch.bfloat16).pin_memory()
    hw = torch.from_numpy(w_np).to(torch.bfloat16).pin_memory()
    ho = torch.empty(n, COUT, dtype=torch.bfloat16).pin_memory()
    hoc = torch.empty(n, 4, dtype=torch.int32).pin_memory()
    for _ in range(3):
        binding.spconv_layer_host(hc, hx, hw, 1, 1, 3, True, ho, hoc)
    barrier(); torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(args.steps):
        binding.spconv_layer_host(hc, hx, hw, 1, 1, 3, True, ho, hoc)
    b.record(stream)
    torch.cuda.synchronize(); barrier()
    e2e_ms = a.elapsed_time(b) / args.steps
    h2d = hc.numel() * 4 + hx.numel() * 2 + hw.numel() * 2
    d2h = ho.numel() * 2 + hoc.numel() * 4

    # ---------------- max over ranks of the time, sum over ranks of the work
    total_ms_max, voxels_all = sharding.combine(total_ms, float(voxels_timed), device="cuda")
    _, voxels_e2e = sharding.combine(total_ms, float(n), device="cuda")
    e2e_ms_max, _ = sharding.combine(e2e_ms, float(n), device="cuda")
    value = voxels_all / (total_ms_max * 1e-3) / 1e6
    e2e_value = voxels_e2e / (e2e_ms_max * 1e-3) / 1e6

    if rank == 0:
        peaks = measured_peaks()
        fwd = fwd_rot_ms
        alg_bytes = forward_algorithmic_bytes(rot_n, rot_n, rot_pairs_mean)
        flops = 2.0 * rot_pairs_mean * CIN * COUT
        achieved = alg_bytes / (fwd * 1e-3) / 1e9
        t_hbm_us = alg_bytes / (peaks["hbm_gbs"] * 1e9) * 1e6
        t_mma_us = flops / (peaks["bf16_tflops"] * 1e12) * 1e6
        cpu_n, cpu_tk, cpu_tf, cpu_threads, sample = time_oracle(coords_np, seed, REFERENCE_SAMPLE_VOXELS)
        # Parity of the timed call on the timed workload (outside the timed region): the same spconv_layer call on the
        # oracle's inputs, every output row against the oracle's fp64 result.
        pk, py = binding.spconv_layer(torch.from_numpy(sample["coords"]).cuda(), torch.from_numpy(sample["x"]).to(torch.bfloat16).cuda(),
                                      w, 1, 1, 3, True)
        torch.cuda.synchronize()
        p_status = binding.spconv_last_device_status(pk)
        p_err = float(np.abs(py.float().cpu().numpy().astype(np.float64) - sample["ref"]).max() / np.abs(sample["ref"]).max())
        parity = {"max_rel_err": p_err, "rows": int(py.shape[0]), "tolerance": 2e-2, "pairs_match": int(pk.total_pairs) == sample["pairs"],
                  "device_status": p_status, "ok": bool(p_err <= 2e-2 and int(pk.total_pairs) == sample["pairs"] and p_status == 0),
                  "what": "spconv_layer on sweep 0, all rows, vs the fp64 oracle (max-abs error / max |ref|)"}
        pk.close()
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": total_ms_max / args.steps, "ms_per_step_min": min(step_ms), "ms_per_step_median": statistics.median(step_ms),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "n_voxels": n, "pairs": int(pairs), "tiles": int(n_tiles),
                       "tile_blocks": int(blocks), "seed": seed,
                       "l2": f"no flush: inputs larger than L2, each rank rotates over {ROTATION} sweeps (about 360 MB of arrays)",
                       "voxels_per_sweep": [sw["n"] for sw in sweeps],
                       "sharding": "one independent sweep per GPU, no collective"},
            "layer": {"kmap_build_ms": statistics.mean(kmap_ms), "forward_ms_after_build_separate_call": statistics.mean(fwd_cold_ms),
                      "step_ms_as_two_calls": statistics.mean(two_call_ms),
                      "forward_ms_l2_cold": fwd, "forward_ms_l2_cold_python_launches": fwd_rot_host_ms,
                      "forward_ms_flushed_single_launch": statistics.mean(fwd_ms),
                      "forward_ms_l2_warm": fwd_warm_ms,
                      "eff_tflops_l2_cold": flops / (fwd * 1e-3) / 1e12, "eff_tflops_l2_warm": flops / (fwd_warm_ms * 1e-3) / 1e12,
                      "kmap_build_ms_min": min(kmap_ms), "kmap_build_ms_median": statistics.median(kmap_ms),
                      "kmap_build_mvoxels_s": rot_n / (statistics.mean(kmap_ms) * 1e-3) / 1e6,
                      "kmap_algorithmic_bytes": kmap_algorithmic_bytes(rot_n, rot_pairs_mean),
                      "kmap_roofline_frac": kmap_algorithmic_bytes(rot_n, rot_pairs_mean) / (peaks["hbm_gbs"] * 1e9) / (statistics.mean(kmap_ms) * 1e-3),
                      "kmap_share_of_step": statistics.mean(kmap_ms) / statistics.mean(two_call_ms),
                      "t_hbm_us": t_hbm_us, "t_mma_us": t_mma_us,
                      "roofline_frac_l2_cold": max(t_hbm_us, t_mma_us) / (fwd * 1e3),
                      "roofline_frac_l2_warm": max(t_hbm_us, t_mma_us) / (fwd_warm_ms * 1e3)},
            "roofline": {"kernel": "k_forward_tc<64,64>", "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": FORWARD_DRAM_TRAFFIC_BYTES,
                         "traffic_source": FORWARD_DRAM_TRAFFIC_SOURCE,
                         "frac_single_launch_after_flush": alg_bytes / (statistics.mean(fwd_ms) * 1e-3) / 1e9 / peaks["hbm_gbs"],
                         "frac_note": "frac uses the period of back-to-back launches over rotating (L2-cold) sweeps, where a launch's set-up overlaps "
                                      "the tail of the launch before; frac_single_launch_after_flush is one isolated launch",
                         "peak_source": peaks["source"], "algorithmic_bytes": alg_bytes, "ms": fwd},
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms_max, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h},
            "parity": parity,
            "gpu_launches": OUR_LAUNCHES_PER_STEP * args.steps,
            "clocks": clocks,
            "wall_s": wall,
            "cpu_baseline": {"value": cpu_n / (cpu_tk + cpu_tf) / 1e6, "unit": UNIT, "cores": cpu_threads, "kind": "oracle",
                             "sample": f"the whole sweep ({cpu_n} voxels), once: "
                                       f"kmap {cpu_tk * 1e3:.0f} ms + forward {cpu_tf * 1e3:.0f} ms"},
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_survey(args):
    """Per-layer table over all five workloads (not the bench line): kernel-map build and forward time of every
    layer, L2 flushed before every timed launch, with the layer's roofline from the measured peaks."""
    import torch

    from paper_2402_07710_b200 import binding

    torch.cuda.set_device(0)
    peaks = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    rows = []

    def timed(fn, reps):
        ms = []
        for i in range(reps + 2):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            r = fn()
            b.record(stream)
            torch.cuda.synchronize()
            if i >= 2:
                ms.append(a.elapsed_time(b))
            if hasattr(r, "close"):
                r.close()
        return statistics.mean(ms)

    for index in (1, 2, 3, 4, 5):
        cfg = wl.config(index)
        coords = torch.from_numpy(cfg["coords"]).cuda()
        x = None
        for li, layer in enumerate(cfg["layers"]):
            subm = layer["kind"] == "subm"
            K, s, cin, cout, dtype = layer["kernel"], layer["stride"], layer["cin"], layer["cout"], layer["dtype"]
            td = binding.DTYPE_BY_NAME[dtype]
            e = 4 if dtype == "f32" else 2
            km = binding.spconv_build_kmap(coords, s, 1, K, subm)
            if x is None or x.shape[1] != cin or x.shape[0] != km.n_in:
                x = torch.from_numpy(wl.features(km.n_in, cin, dtype, li)).to(td).cuda()
            w = torch.from_numpy(wl.weights(K ** 3, cin, cout, dtype, li)).to(td).cuda()
            out = torch.empty(km.n_out, cout, dtype=td, device="cuda")
            t_build = timed(lambda: binding.spconv_build_kmap(coords, s, 1, K, subm), args.steps)
            t_fwd = timed(lambda: binding.spconv_forward(x, w, km, out=out), args.steps)
            P, kvol = km.total_pairs, K ** 3
            byts = km.n_in * cin * e + km.n_out * cout * e + kvol * cin * cout * e + min(8 * P, 4 * kvol * km.n_out)
            flops = 2.0 * P * cin * cout
            t_hbm = byts / (peaks["hbm_gbs"] * 1e9) * 1e3
            t_mma = flops / (peaks["bf16_tflops"] * 1e12) * 1e3 if dtype != "f32" else flops / 74e12 * 1e3
            rows.append(dict(config=index, layer=li, kind=layer["kind"], kernel=K, stride=s, cin=cin, cout=cout, dtype=dtype,
                             n_in=km.n_in, n_out=km.n_out, pairs=int(P), tile_blocks=km.tile_blocks,
                             kmap_build_ms=t_build, kmap_mvoxels_s=km.n_in / (t_build * 1e-3) / 1e6, forward_ms=t_fwd,
                             eff_tflops=flops / (t_fwd * 1e-3) / 1e12, t_hbm_ms=t_hbm, t_mma_ms=t_mma,
                             roofline_frac=max(t_hbm, t_mma) / t_fwd))
            if not subm and index == 5:        # encoder stack: the strided layer's outputs are the next level's inputs
                coords = km.out_coords.clone()
            x = out if index == 5 else None
            km_keep = km                       # keep the handle alive while `coords` may view its memory
        del km_keep
    print(json.dumps({"survey": rows, "peaks": peaks}))


def run_options(args):
    """The measured options of the path (not the bench line), one JSON line: row order of the tile plan x offsets per
    pipeline step of the tensor-core forward; hash table against dense-array location table; the voxeliser."""
    import numpy as np
    import torch

    from paper_2402_07710_b200 import binding

    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream()

    def build_time(fn, reps=20):          # median of event-timed calls through the Python binding, microseconds
        ts = []
        for i in range(reps + 3):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            r = fn()
            b.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b) * 1e3)
            if hasattr(r, "close"):
                r.close()
        return statistics.median(ts)

    def graph_time(fn, launches=20):      # microseconds per launch, CUDA-graph replay on L2-warm arrays
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for _ in range(launches):
                fn()
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            g.replay()
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) / launches * 1e3)
        return statistics.median(ts)

    def z_order(c):                        # rows sorted along a Z-order curve (batch-major)
        def spread(v):
            v = v.astype(np.uint64) & np.uint64(0x1fffff)
            v = (v | (v << np.uint64(32))) & np.uint64(0x1f00000000ffff)
            v = (v | (v << np.uint64(16))) & np.uint64(0x1f0000ff0000ff)
            v = (v | (v << np.uint64(8))) & np.uint64(0x100f00f00f00f00f)
            v = (v | (v << np.uint64(4))) & np.uint64(0x10c30c30c30c30c3)
            v = (v | (v << np.uint64(2))) & np.uint64(0x1249249249249249)
            return v
        key = (c[:, 0].astype(np.uint64) << np.uint64(60)) | (spread(c[:, 1]) << np.uint64(2)) | (spread(c[:, 2]) << np.uint64(1)) | spread(c[:, 3])
        return np.ascontiguousarray(c[np.argsort(key, kind="stable")])

    c3, c2 = wl.config(3)["coords"], wl.config(2)["coords"]
    cases = [("config 3, rows as generated (scan order)", c3, 3, 1, True, 64, 64),
             ("config 3, rows shuffled", wl.shuffle_rows(c3, seed=1), 3, 1, True, 64, 64),
             ("config 3, rows in Z-order", z_order(c3), 3, 1, True, 64, 64),
             ("config 2, rows as generated", c2, 3, 1, True, 32, 32),
             ("config 2, rows in Z-order", z_order(c2), 3, 1, True, 32, 32),
             ("config 4 L0 (K3 s2)", c3, 3, 2, False, 64, 128),
             ("config 4 L1 (K2 s2)", c3, 2, 2, False, 64, 64)]
    row_options = []
    for name, coords, K, s, subm, cin, cout in cases:
        t = torch.from_numpy(np.ascontiguousarray(coords)).cuda()
        for order, oname in ((binding.ROWS_BY_OFFSET_SET, "by offset set"), (binding.ROWS_AS_GIVEN, "as given")):
            km = binding.spconv_build_kmap(t, s, 1, K, subm, row_order=order)
            tb = build_time(lambda: binding.spconv_build_kmap(t, s, 1, K, subm, row_order=order))
            x = torch.randn(km.n_in, cin, device="cuda").bfloat16()
            w = torch.randn(K ** 3, cin, cout, device="cuda").bfloat16()
            out = torch.empty(km.n_out, cout, device="cuda", dtype=torch.bfloat16)
            tg = graph_time(lambda: binding.spconv_forward(x, w, km, algo="tcgen05", out=out))
            ts = graph_time(lambda: binding.spconv_forward(x, w, km, algo="tcgen05_single", out=out))
            row_options.append(dict(case=name, rows=km.n_out, order=oname, tile_blocks=km.tile_blocks, kmap_build_us=tb,
                                    forward_us_offsets_grouped=tg, forward_us_one_offset_per_step=ts))
            km.close()
    tables = []
    c1 = torch.from_numpy(wl.config(1)["coords"]).cuda()
    blob = torch.from_numpy(wl.shuffle_rows(wl.random_blob(60000, 50, seed=3, batches=2), seed=1)).cuda()
    for name, c, grid in (("config 1 (%d voxels), grid 1 x 64^3" % len(c1), c1, (1, 64, 64, 64)),
                          ("blob (%d voxels), grid 2 x 128^3" % len(blob), blob, (2, 128, 128, 128))):
        tables.append(dict(input=name, hash_table_build_us=build_time(lambda: binding.spconv_build_kmap(c, 1, 1, 3, True)),
                           dense_array_build_us=build_time(lambda: binding.spconv_build_kmap_dense(c, grid, 1, 3))))
    pts = torch.from_numpy(wl.lidar_points(0, n_feat=4)).cuda()
    vc, _ = binding.spconv_voxelize(pts, 4, 0, wl.LIDAR_ORIGIN, wl.LIDAR_VOXEL, wl.LIDAR_GRID)
    vox = dict(points=len(pts), n_feat=4, voxels=len(vc),
               us=build_time(lambda: binding.spconv_voxelize(pts, 4, 0, wl.LIDAR_ORIGIN, wl.LIDAR_VOXEL, wl.LIDAR_GRID)[0]))
    print(json.dumps({"row_options": row_options, "location_table": tables, "voxelize": vox}))


def respawn_under_torchrun(args):
    """`python bench.py --gpus N` with N > 1 and no launcher around it: start the N ranks here (one per GPU, NCCL
    rendezvous on 127.0.0.1) and pass their output through."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__), "--gpus", str(args.gpus), "--steps", str(args.steps),
           "--warmup", str(args.warmup), "--impl", args.impl]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--only", choices=("forward", "kmap"), default=None,
                    help="run three launches of one stage and exit (for profiler captures)")
    ap.add_argument("--survey", action="store_true", help="per-layer table over all five workloads (one JSON line)")
    ap.add_argument("--options", action="store_true",
                    help="row order x offsets per step, hash table vs dense array, voxeliser (one JSON line)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.survey and not args.options and not args.only:
        sys.exit(respawn_under_torchrun(args))
    if args.survey:
        run_survey(args)
    elif args.options:
        run_options(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
