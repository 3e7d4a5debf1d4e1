#!/usr/bin/env python
"""Throughput of the pattern-sparse 3x3 convolution path on synthetic VGG-16-shaped layers.

One step = one pass of the whole path over one batch: for each of the 13 VGG-16 conv layers, pattern
selection + connectivity pruning (pat_project), packing (pat_pack) and the convolution itself
(pat_conv3x3; the first layer, C = 3, is dense: pat_conv3x3_dense).  Every layer has its own seeded input
tensor of that layer's shape (batch 64, fp16 storage, fp32 accumulation), all resident in HBM before the
timed region; the working set (about 3.4 GB) is far larger than L2, so nothing is reused across steps.

Prints one JSON line.  `--impl reference` times the CPU oracle on the host cores instead (a bounded sample).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2001_07710_b200 import workloads  # noqa: E402

METRIC = "pattern-sparse conv images/s"
UNIT = "images/s"
SM_COUNT, FMA_LANES, SM_MAX_MHZ = 148, 128, 1965.0
FMA_PEAK_TFLOPS = 2 * FMA_LANES * SM_COUNT * SM_MAX_MHZ * 1e6 / 1e12     # 74.45: fp32 FMA, no tensor cores
DEFAULT_CONFIG = 3
# DRAM traffic of the convolution path (ncu counters of a small case), written by `bench.py --write-traffic` and
# valid only for the kernel sources it was captured from
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic_conv_f16_img_conv6_b32.json")
TRAFFIC_SOURCES = ["conv_f16_img.cu", "f16_tile.cuh", "common.cuh", "img_geometry.cuh"]


def kernel_source_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for f in TRAFFIC_SOURCES:
        h.update(open(os.path.join(ROOT, "paper_2001_07710_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def write_traffic(csv_path: str):
    """Turns an ncu launch list with dram__bytes_read.sum / dram__bytes_write.sum of the three launches of the conv6
    path (batch 32) into TRAFFIC_FILE.  The bytes the path wrote but that were still in L2 when a launch ended are
    added from what the launches are known to write (stage images, outputs)."""
    import csv
    unit = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    rows = [r for r in csv.reader(open(csv_path)) if len(r) > 5]
    hdr = rows[0]
    ki, mi, ui, vi = hdr.index("Kernel Name"), hdr.index("Metric Name"), hdr.index("Metric Unit"), hdr.index("Metric Value")
    kernels = {}
    for r in rows[1:]:
        name = "stage" if "k_stage_images" in r[ki] else "conv" if "k_conv_f16_img" in r[ki] else "reduce" if "k_reduce_parts" in r[ki] else None
        if name is None or not r[mi].startswith("dram__bytes_"):
            continue
        key = "read" if "read" in r[mi] else "write"
        kernels.setdefault(name, {})[key] = float(r[vi].replace(",", "")) * unit[r[ui]]
    cfg = workloads.configs()[3]
    L = [l for l in cfg.layers if l.name == "conv6"][0]
    from paper_2001_07710_b200 import binding
    lib = binding.load()
    images = lib.pat_conv3x3_workspace(L.F, L.C, 1, 32, L.H, L.W, 1) - 256 * 32 * 56 * 32 * 4     # stage images without the partial tiles
    known_writes = images + 32 * L.Ho * L.Wo * L.F * 2
    pending = max(0.0, known_writes - sum(k.get("write", 0.0) for k in kernels.values()))
    out = {"workload": "config 3 layer conv6 (56x56x256 -> 256, keep 12.5 %), fp16 storage, batch 32",
           "source_sha16": kernel_source_hash(), "sources": TRAFFIC_SOURCES, "batch": 32, "kernels": kernels,
           "written_still_in_l2": pending, "algorithmic_bytes": L.compulsory_bytes(32, 2)}
    json.dump(out, open(TRAFFIC_FILE, "w"), indent=1)
    print(json.dumps(out))


def traffic_field(N: int, cfg_no: int):
    """roofline.traffic for the benchmark's batch, or None when the counters do not belong to the current kernels."""
    if cfg_no != 3 or not os.path.exists(TRAFFIC_FILE):
        return None, "no counters for this workload"
    t = json.load(open(TRAFFIC_FILE))
    if t.get("source_sha16") != kernel_source_hash():
        return None, "the kernel sources changed since the counters in %s were taken" % os.path.basename(TRAFFIC_FILE)
    scale = N / float(t["batch"])
    dram = sum(k.get("read", 0.0) + k.get("write", 0.0) for k in t["kernels"].values()) + t.get("written_still_in_l2", 0.0)
    note = ("DRAM read + write of the three launches of one layer's path (stage images, convolution, reduce) on %s "
            "(ncu), plus the %.1f MB the launches wrote that were still in L2 when they ended, scaled by batch/%d; "
            "algorithmic bytes of that layer at this batch: %d (traffic / algorithmic = %.2f)"
            % (t["workload"], t.get("written_still_in_l2", 0.0) / 1e6, t["batch"], int(t["algorithmic_bytes"] * scale),
               dram / t["algorithmic_bytes"]))
    return dram * scale, note


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return json.load(open(p)), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


# ----------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if sm:
            out["sm_mhz"] = float(np.median(sm)); out["sm_max_mhz"] = float(max(mx)); out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------------------------- GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2001_07710_b200 as pc

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")     # the communicator's own log (rings, NVLS) goes to stderr
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    pc.load()

    cfg = workloads.configs()[args.config]
    N = cfg.N if args.batch is None else args.batch
    if args.strong and world > 1:
        # strong scaling: the configuration's batch is cut into contiguous slices, one per rank (no data-path
        # collective: images are independent); every rank draws the tensors of a batch of its slice's size
        from paper_2001_07710_b200.sharding import shard_batch
        lo, hi = shard_batch(N, world, rank)
        if hi == lo:
            raise SystemExit("bench.py --strong: more ranks than images in the batch")
        N = hi - lo
    dtype = cfg.dtype
    tdt = torch.float16 if dtype == "f16" else torch.float32
    elem = 2 if dtype == "f16" else 4
    masks = {K: pc.pat_library_builtin(K) for K in (4, 8, 12)}
    stream = torch.cuda.current_stream()

    # ---- seeded host tensors (pinned: they are also the source of the end-to-end copies)
    layers = []
    cfg_layers = [L for L in cfg.layers if args.layers is None or L.name in args.layers.split(",")]
    for L in cfg_layers:
        w_np, x_np = workloads.make_layer_tensors(cfg.number, L, N)
        hw = torch.from_numpy(w_np).pin_memory()
        hx = torch.from_numpy(x_np).to(tdt).pin_memory()
        del x_np
        hy = torch.empty((N, L.Ho, L.Wo, L.F), dtype=tdt).pin_memory()
        st = dict(L=L, hw=hw, hx=hx, hy=hy,
                  w=hw.cuda(), x=hx.cuda(), y=torch.empty((N, L.Ho, L.Wo, L.F), dtype=tdt, device="cuda"))
        if not L.dense:
            st["pid"] = torch.empty((L.F, L.C), dtype=torch.uint8, device="cuda")
            st["wm"] = torch.empty((L.F, L.C, 3, 3), dtype=torch.float32, device="cuda")
            st["ws"] = torch.empty(pc.pat_project_workspace(L.F, L.C), dtype=torch.uint8, device="cuda")
            st["blob"] = torch.empty(pc.pat_pack_size(L.F, L.C, L.K, L.n_keep, dtype), dtype=torch.uint8, device="cuda")
        layers.append(st)
    # one workspace for the stage images of pat_conv3x3_ws, sized for the largest layer (layers run one after another)
    cws_bytes = max([pc.pat_conv3x3_workspace(L.F, L.C, dtype, N, L.H, L.W, L.stride) for L in cfg_layers if not L.dense] + [0])
    cws = torch.empty(max(cws_bytes, 256), dtype=torch.uint8, device="cuda")

    # Projection and packing of a layer depend on its weights only: every pruned layer gets a stream of its own for
    # them, forked from the main stream at the start of the step, and an event orders the layer's convolution after
    # its own packing.  The chains of small kernels (a dozen launches per layer) then run side by side while the
    # first layers convolve, instead of one after another in the gaps between the convolution kernels.
    sides = [torch.cuda.Stream(priority=-1) for _ in layers]    # their small blocks go first whenever an SM has room
    packed_ev = [torch.cuda.Event() for _ in layers]

    def step(conv_events=None, overlap=True):
        overlap = overlap and not args.no_overlap
        main = torch.cuda.current_stream()
        for i, st in enumerate(layers):
            L = st["L"]
            if L.dense:
                continue
            prep = sides[i] if overlap else main
            if overlap:
                prep.wait_stream(main)             # the previous step no longer reads this layer's blob
            with torch.cuda.stream(prep):
                pc.pat_project(st["w"], masks[L.K], L.n_keep, st["pid"], st["wm"], st["ws"])
                pc.pat_pack(st["wm"], st["pid"], masks[L.K], L.n_keep, dtype, st["blob"])
                if overlap:
                    packed_ev[i].record(prep)
        for i, st in enumerate(layers):
            L = st["L"]
            if conv_events is not None: conv_events[i][0].record(main)
            if L.dense:
                pc.pat_conv3x3_dense(st["w"], dtype, st["x"], L.stride, y=st["y"])
            else:
                if overlap:
                    main.wait_event(packed_ev[i])  # joins the layer's stream: every fork is waited for within the step
                pc.pat_conv3x3(st["blob"], L.F, L.C, masks[L.K], L.n_keep, dtype, st["x"], L.stride, y=st["y"], workspace=cws)
            if conv_events is not None: conv_events[i][1].record(main)

    # End to end: every step copies its weights and inputs from pinned host memory and reads all outputs back.  The
    # copies run on streams of their own (host-to-device, device-to-host: the link is full duplex) and overlap the
    # compute stream layer by layer; events order copy-in -> compute -> copy-out per layer, and a step begins only
    # when the previous step's kernels no longer read the device buffers it overwrites.
    h2d, d2h = torch.cuda.Stream(), torch.cuda.Stream()
    in_ev = [torch.cuda.Event() for _ in layers]
    out_ev = [torch.cuda.Event() for _ in layers]

    def step_e2e():
        main = torch.cuda.current_stream()
        h2d.wait_stream(main)                      # the previous step has consumed w and x
        with torch.cuda.stream(h2d):
            for i, st in enumerate(layers):
                st["w"].copy_(st["hw"], non_blocking=True)
                st["x"].copy_(st["hx"], non_blocking=True)
                in_ev[i].record(h2d)
        for i, st in enumerate(layers):
            L = st["L"]
            main.wait_event(in_ev[i])
            if L.dense:
                pc.pat_conv3x3_dense(st["w"], dtype, st["x"], L.stride, y=st["y"])
            else:
                pc.pat_project(st["w"], masks[L.K], L.n_keep, st["pid"], st["wm"], st["ws"])
                pc.pat_pack(st["wm"], st["pid"], masks[L.K], L.n_keep, dtype, st["blob"])
                pc.pat_conv3x3(st["blob"], L.F, L.C, masks[L.K], L.n_keep, dtype, st["x"], L.stride, y=st["y"], workspace=cws)
            out_ev[i].record(main)
            with torch.cuda.stream(d2h):
                d2h.wait_event(out_ev[i])
                st["hy"].copy_(st["y"], non_blocking=True)
        main.wait_stream(d2h)                      # the results are on the host before the step counts as done

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    from paper_2001_07710_b200.sharding import job_throughput

    # ---- warm-up
    for _ in range(max(args.warmup, 3)):
        step()
    assert pc.pat_query_status() == 0

    # ---- the step as a CUDA graph: the ~200 small launches of a step (projection and packing kernels of twelve
    # layers) are then issued by the GPU front end without a host round trip each
    launches0 = pc.pat_launch_count()
    if args.no_graph:                  # plain launches (for profilers, which see one kernel per launch that way)
        step()
        run_step = step
    else:
        gstream = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(gstream):
            with torch.cuda.graph(graph, stream=gstream):
                step()
        run_step = graph.replay
    launches_per_step = pc.pat_launch_count() - launches0
    # clocks are sampled from here on (two more untimed steps, then the timed region): nvidia-smi needs some tens of
    # milliseconds before its first sample, more than a short timed region lasts
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(2):
        run_step()
    barrier()

    # ---- timed region: device-resident inputs, K replays of the step
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for k in range(args.steps):
        run_step()
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = launches_per_step * args.steps
    value, ms_total, _ = job_throughput(float(N * args.steps), e0.elapsed_time(e1), "cuda")   # weak scaling: N images per rank
    ms_step = ms_total / args.steps
    assert pc.pat_query_status() == 0

    # per-layer convolution times: plain launches with events around every convolution (mean over three passes;
    # outside the timed region)
    nrep = 3
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in layers]
          for _ in range(nrep)]
    for k in range(nrep):
        step(ev[k], overlap=False)     # one stream: nothing else runs beside the timed convolutions
    barrier()
    conv_ms = [float(np.mean([ev[k][i][0].elapsed_time(ev[k][i][1]) for k in range(nrep)])) for i in range(len(layers))]

    # ---- end to end: host buffers, copies inside the timed region
    e2e_steps = max(1, min(args.steps, 3))
    step_e2e()
    barrier()
    e0.record(stream)
    for _ in range(e2e_steps):
        step_e2e()
    e1.record(stream)
    barrier()
    e2e_value, ms_e2e, _ = job_throughput(float(N * e2e_steps), e0.elapsed_time(e1), "cuda")
    h2d = sum(st["hw"].numel() * 4 + st["hx"].numel() * elem for st in layers)
    d2h = sum(st["hy"].numel() * elem for st in layers)
    assert pc.pat_query_status() == 0

    # ---- roofline of the dominant kernel (the sparse convolution), and per layer
    traffic, traffic_note = traffic_field(N, cfg.number)
    fma_measured = pc.pat_measure_fma_peak(1 if dtype == "f16" else 0)
    peaks, peak_kind = measured_peaks()
    hbm = peaks["hbm_gbs"]
    per_layer = []
    sparse_flop = sparse_ms = 0.0
    for st, ms in zip(layers, conv_ms):
        L = st["L"]
        flop = L.useful_flop(N)
        byts = L.compulsory_bytes(N, elem)
        # sparse layers: fp32 FMA pipe or HBM; the dense first layer runs on the tensor cores (fp16 inputs), where its
        # 27 x 64 contraction per pixel is negligible against writing the output: HBM or the measured bf16 tensor rate
        p_flop = (peaks["bf16_tflops"] if (L.dense and dtype == "f16") else FMA_PEAK_TFLOPS) * 1e12
        t_roof_us = max(flop / p_flop, byts / (hbm * 1e9)) * 1e6
        per_layer.append({"layer": L.name, "shape": f"{L.H}x{L.W}x{L.C}->{L.F}", "n_keep": L.n_keep,
                          "conv_us": round(ms * 1e3, 2), "eff_tflops": round(flop / (ms * 1e-3) / 1e12, 3),
                          "roof_us": round(t_roof_us, 2), "roof_frac": round(t_roof_us / (ms * 1e3), 4)})
        if not L.dense:
            sparse_flop += flop; sparse_ms += ms
    achieved = sparse_flop / (sparse_ms * 1e-3) / 1e12 if sparse_ms > 0 else 0.0
    total_flop = sum(st["L"].useful_flop(N) for st in layers)

    touched = sum((st["x"].numel() + st["y"].numel()) * elem for st in layers)
    l2_note = (f"inputs and outputs larger than L2 ({touched / 1e9:.2f} GB touched per step)" if touched > 4 * 126e6 else
               f"inputs and outputs of a step ({touched / 1e6:.1f} MB) are not much larger than the 126 MB L2: no flush between steps, warm-cache numbers")
    out = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 4), "higher_is_better": True, "scaling": "strong" if (args.strong and world > 1) else "weak",
        "vs_baseline": None, "dtype": "f16 storage, f32 accumulate" if dtype == "f16" else "f32", "data": "synthetic",
        "config": {"workload": f"config {cfg.number}: {cfg.name}", "batch_per_gpu": N,
                   "layers": len(layers), "step": "project + pack + conv for every layer" + ("" if args.no_overlap else ", projection / packing of each layer on a stream of its own")
                           + ("" if args.no_graph else ", replayed as one CUDA graph"),
                   "l2": l2_note, "seed": workloads.BASE_SEED},
        "effective_gflops": round(total_flop * world * args.steps / (ms_total * 1e-3) / 1e9, 1),
        "conv_only_images_per_s": round(world * N / (sum(conv_ms) * 1e-3), 2),
        "roofline": {"bound": "alu", "kernel": "sparse convolution path of the pruned layers (stage images + convolution + reduce launches)", "achieved": round(achieved, 3),
                     "peak": round(FMA_PEAK_TFLOPS, 2), "unit": "TFLOP/s", "frac": round(achieved / FMA_PEAK_TFLOPS, 4),
                     "peak_kind": "derived: 2 x 128 fp32 lanes x 148 SMs x 1.965 GHz",
                     "traffic": traffic, "traffic_note": traffic_note,
                     "peak_measured": round(fma_measured, 2),
                     "peak_measured_kind": "fma.rn.f32.f16 chains on all SMs, best of three, this run (pat_measure_fma_peak)",
                     "hbm_peak_gbs": hbm, "hbm_peak_kind": peak_kind,
                     "min_layer_frac": min([p["roof_frac"] for p in per_layer if p["layer"] != "conv1"] + [1.0])},
        "layers": per_layer,
        "e2e": {"value": round(e2e_value, 2), "unit": UNIT,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if world == 1 and cfg.number == 3 and not args.no_other_configs:
        out["fused_pooling"] = fused_pooling(pc, torch, layers, masks, dtype, cws, N)
    if world == 1 and not args.no_other_configs and args.batch is None and args.layers is None:
        # the other four configurations: short measurements of their own, after the main timed region
        out["other_configs"] = {str(c): quick_config(pc, torch, c, peaks) for c in range(5) if c != cfg.number}
    if world == 1 and not args.no_other_configs and args.batch is None and args.layers is None:
        out["admm_primitives"] = admm_primitives(pc, torch, peaks, with_cpu=not args.no_cpu)
    if rank == 0 and world == 1 and not args.no_cpu:
        out["cpu_baseline"] = cpu_baseline(cfg, budget_s=args.cpu_seconds)
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def fused_pooling(pc, torch, layers, masks, dtype, cws, N, reps: int = 5):
    """The five layers of the VGG-16 stack that are followed by the rectifier and 2x2 max pooling: the convolution
    with both fused into its epilogue (pat_conv3x3_ws_act, act = 2: the pooled image is the only output) next to the
    convolution followed by pat_relu_maxpool as a pass of its own.  Plain launches on one stream, CUDA events,
    two warm-up calls; the inputs and packed weights are those of the step (already resident)."""
    res = {}
    for st in layers:
        L = st["L"]
        if L.dense or L.name not in ("conv2", "conv4", "conv7", "conv10", "conv13"):
            continue
        yp = torch.empty((N, L.H // 2, L.W // 2, L.F), dtype=st["y"].dtype, device="cuda")

        def two_pass():
            pc.pat_conv3x3(st["blob"], L.F, L.C, masks[L.K], L.n_keep, dtype, st["x"], 1, y=st["y"], workspace=cws)
            pc.pat_relu_maxpool(st["y"], dtype, True, yp)

        def fused():
            pc.pat_conv3x3(st["blob"], L.F, L.C, masks[L.K], L.n_keep, dtype, st["x"], 1, y=yp, workspace=cws, pool=True)

        t = []
        for fn in (two_pass, fused):
            for _ in range(2):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            t.append(e0.elapsed_time(e1) / reps * 1e3)
        res[L.name] = {"conv_then_relu_maxpool_us": round(t[0], 1), "fused_us": round(t[1], 1), "speedup": round(t[0] / t[1], 3)}
        del yp
    assert pc.pat_query_status() == 0
    return res


def admm_primitives(pc, torch, peaks, with_cpu: bool, reps: int = 10):
    """The training-side primitives on the kernels of a 512 x 512 layer with the full library of 126 masks (the
    start of the library extraction): simplex projection and binarisation of 262 144 vectors of 126 entries (132 MB
    in, 132 MB out: larger than L2), and one reduction step 126 -> 12 of the library.  CUDA events, after three
    warm-up calls; the oracle is timed beside them on a bounded sample."""
    import itertools
    n, K = 512 * 512, 126
    rng = np.random.default_rng(20200107)
    d_np = (rng.standard_normal((n, K)) * 0.3 + 1.0 / K).astype(np.float32)
    w_np = workloads.make_weights(rng, 512, 512)
    masks = np.array([sum(1 << b for b in c) for c in itertools.combinations(range(9), 4)], dtype=np.uint16)
    d = torch.from_numpy(d_np).cuda()
    u = torch.empty_like(d)
    idx = torch.empty(n, dtype=torch.uint8, device="cuda")
    w = torch.from_numpy(w_np).cuda()
    mout = torch.empty(12, dtype=torch.int16, device="cuda")
    counts = torch.empty(K, dtype=torch.int64, device="cuda")
    st = torch.cuda.current_stream()

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(reps):
            fn()
        e1.record(st)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e-3

    hbm = peaks["hbm_gbs"]
    t_sp = timed(lambda: pc.pat_simplex_project(d, u))
    t_am = timed(lambda: pc.pat_argmax_binarize(u, idx, want_onehot=False))
    t_ex = timed(lambda: pc.pat_extract_library(w, masks, 12, mout, counts))
    res = {"workload": "262144 vectors / kernels (a 512 x 512 layer), library of 126 masks; inputs and outputs larger than L2",
           "simplex_project": {"ms": round(t_sp * 1e3, 4), "GB/s": round(8.0 * n * K / t_sp / 1e9, 1),
                               "roofline": {"bound": "hbm", "peak": hbm, "frac": round(8.0 * n * K / t_sp / 1e9 / hbm, 4)},
                               "bytes": "read once + written once, 8 per entry"},
           "argmax_binarize": {"ms": round(t_am * 1e3, 4), "GB/s": round((4.0 * n * K + n) / t_am / 1e9, 1),
                               "roofline": {"bound": "hbm", "peak": hbm, "frac": round((4.0 * n * K + n) / t_am / 1e9 / hbm, 4)},
                               "bytes": "read once, one index byte per vector"},
           "extract_library_126_to_12": {"ms": round(t_ex * 1e3, 4), "kernels_per_s": round(n / t_ex, 0),
                                         "note": "a memset and two launches; 126 mask energies per kernel (fp32, exact fp64 fallback): arithmetic, not memory"}}
    # the rectifier and 2x2 max pooling after the second VGG-16 layer: 64 x 224 x 224 x 64 fp16 in, a quarter out
    xa = torch.randn((64, 224, 224, 64), dtype=torch.float16, device="cuda")
    ya = torch.empty((64, 112, 112, 64), dtype=torch.float16, device="cuda")
    t_rp = timed(lambda: pc.pat_relu_maxpool(xa, "f16", True, ya))
    by = (xa.numel() + ya.numel()) * 2.0
    res["relu_maxpool_vgg_conv2_output"] = {"ms": round(t_rp * 1e3, 4), "GB/s": round(by / t_rp / 1e9, 1),
                                            "roofline": {"bound": "hbm", "peak": hbm, "frac": round(by / t_rp / 1e9 / hbm, 4)},
                                            "bytes": "input read once, output written once (514 MB)"}
    del xa, ya
    if with_cpu:
        import oracle
        m = 8192                                      # a bounded sample of the same vectors / kernels
        t0 = time.perf_counter(); oracle.simplex_project(d_np[:m]); t1 = time.perf_counter()
        oracle.argmax_binarize(d_np[:m]); t2 = time.perf_counter()
        oracle.extract_library(w_np.reshape(-1, 3, 3)[:m], masks, 12); t3 = time.perf_counter()
        res["cpu_oracle"] = {"sample": f"{m} vectors / kernels, one thread", "simplex_project_vectors_per_s": round(m / (t1 - t0), 0),
                             "argmax_binarize_vectors_per_s": round(m / (t2 - t1), 0), "extract_library_kernels_per_s": round(m / (t3 - t2), 0),
                             "gpu_simplex_project_vectors_per_s": round(n / t_sp, 0)}
    del d, u, w
    torch.cuda.empty_cache()
    return res


def quick_config(pc, torch, cfg_no: int, peaks, steps: int = 10):
    """One of the other configurations: the same step (project + pack + convolution of every layer) on one stream,
    `steps` times after three warm-up steps, CUDA events around the steps and around every convolution call."""
    cfg = workloads.configs()[cfg_no]
    N, dtype = cfg.N, cfg.dtype
    tdt = torch.float16 if dtype == "f16" else torch.float32
    elem = 2 if dtype == "f16" else 4
    masks = {K: pc.pat_library_builtin(K) for K in (4, 8, 12)}
    layers = []
    for L in cfg.layers:
        w_np, x_np = workloads.make_layer_tensors(cfg.number, L, N)
        st = dict(L=L, w=torch.from_numpy(w_np).cuda(), x=torch.from_numpy(x_np).to(tdt).cuda(),
                  y=torch.empty((N, L.Ho, L.Wo, L.F), dtype=tdt, device="cuda"))
        if not L.dense:
            st["pid"] = torch.empty((L.F, L.C), dtype=torch.uint8, device="cuda")
            st["wm"] = torch.empty((L.F, L.C, 3, 3), dtype=torch.float32, device="cuda")
            st["ws"] = torch.empty(pc.pat_project_workspace(L.F, L.C), dtype=torch.uint8, device="cuda")
            st["blob"] = torch.empty(pc.pat_pack_size(L.F, L.C, L.K, L.n_keep, dtype), dtype=torch.uint8, device="cuda")
        layers.append(st)
    cws = torch.empty(max([pc.pat_conv3x3_workspace(L.F, L.C, dtype, N, L.H, L.W, L.stride) for L in cfg.layers if not L.dense] + [256]),
                      dtype=torch.uint8, device="cuda")
    main = torch.cuda.current_stream()
    sides = [torch.cuda.Stream(priority=-1) for _ in layers]
    packed_ev = [torch.cuda.Event() for _ in layers]

    def step(ev=None):
        # ev given: one stream, events around every convolution; otherwise projection / packing of every layer on a
        # stream of its own, as in the main run
        cur = torch.cuda.current_stream()
        for i, st in enumerate(layers):
            L = st["L"]
            if L.dense:
                continue
            prep = cur if ev is not None else sides[i]
            if ev is None:
                prep.wait_stream(cur)
            with torch.cuda.stream(prep):
                pc.pat_project(st["w"], masks[L.K], L.n_keep, st["pid"], st["wm"], st["ws"])
                pc.pat_pack(st["wm"], st["pid"], masks[L.K], L.n_keep, dtype, st["blob"])
                if ev is None:
                    packed_ev[i].record(prep)
        for i, st in enumerate(layers):
            L = st["L"]
            if ev is not None: ev[i][0].record(cur)
            if L.dense:
                pc.pat_conv3x3_dense(st["w"], dtype, st["x"], L.stride, y=st["y"])
            else:
                if ev is None:
                    cur.wait_event(packed_ev[i])
                pc.pat_conv3x3(st["blob"], L.F, L.C, masks[L.K], L.n_keep, dtype, st["x"], L.stride, y=st["y"], workspace=cws)
            if ev is not None: ev[i][1].record(cur)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    gstream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(gstream):
        with torch.cuda.graph(graph, stream=gstream):
            step()
        graph.replay()
        gstream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(gstream)
        for _ in range(steps):
            graph.replay()
        e1.record(gstream)
        gstream.synchronize()
        ms_step = e0.elapsed_time(e1) / steps
        touched = sum((st["x"].numel() + st["y"].numel()) * elem for st in layers)
        ms_cold = None
        if touched <= 4 * 126e6:
            # working set inside L2: also a cold figure, every step after a buffer larger than L2 has been written
            flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
            pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for a, b in pairs:
                flush.fill_(1)
                a.record(gstream)
                graph.replay()
                b.record(gstream)
            gstream.synchronize()
            ms_cold = float(np.mean([a.elapsed_time(b) for a, b in pairs]))
            del flush
    del graph
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in layers] for _ in range(3)]
    for k in range(3):
        step(ev[k])
    torch.cuda.synchronize()
    assert pc.pat_query_status() == 0
    conv_ms = [float(np.mean([ev[k][i][0].elapsed_time(ev[k][i][1]) for k in range(3)])) for i in range(len(layers))]
    fracs, flop_s, ms_s, roof_s = [], 0.0, 0.0, 0.0
    for st, ms in zip(layers, conv_ms):
        L = st["L"]
        flop = L.useful_flop(N)
        p_flop = (peaks["bf16_tflops"] if (L.dense and dtype == "f16") else FMA_PEAK_TFLOPS) * 1e12
        roof_us = max(flop / p_flop, L.compulsory_bytes(N, elem) / (peaks["hbm_gbs"] * 1e9)) * 1e6
        roof_s += roof_us
        if not L.dense:
            fracs.append(roof_us / (ms * 1e3)); flop_s += flop; ms_s += ms
    res = {"workload": f"config {cfg.number}: {cfg.name}", "batch": N, "dtype": dtype, "steps": steps,
           "images_per_s": round(N / (ms_step * 1e-3), 1), "ms_per_step": round(ms_step, 4),
           "conv_ms_per_step": round(sum(conv_ms), 4),
           "sparse_conv_tflops": round(flop_s / (ms_s * 1e-3) / 1e12, 3),
           "roof_frac": round(roof_s / (sum(conv_ms) * 1e3), 4), "min_layer_frac": round(min(fracs), 4),
           "timing": "step: CUDA-graph replays, projection / packing of each layer on a stream of its own; convolution times: plain launches on one stream",
           "l2": "inputs and outputs larger than L2" if touched > 4 * 126e6 else "warm L2 (working set %.0f MB, no flush between steps)" % (touched / 1e6)}
    if ms_cold is not None:
        res["ms_per_step_cold"] = round(ms_cold, 4)
        res["images_per_s_cold"] = round(N / (ms_cold * 1e-3), 1)
        res["cold"] = "a 512 MB buffer is written before every step (L2 flushed)"
    del layers, cws
    torch.cuda.empty_cache()
    return res


# ----------------------------------------------------------------------------------------------- CPU oracle
class OracleSample:
    """A bounded sample of the workload for the CPU oracle: a seeded fraction of the outputs of one image
    of every layer, each computed by the oracle's direct float64 definition over the masked weights."""

    def __init__(self, cfg, frac: float):
        import oracle
        self.oracle = oracle
        self.cfg = cfg
        self.frac = frac
        self.items = []
        rng = np.random.default_rng(1234)
        for L in cfg.layers:
            w, x = workloads.make_layer_tensors(cfg.number, L, cfg.N, n_limit=1)
            if cfg.dtype == "f16":
                x = x.astype(np.float16)
            if L.dense:
                wm = w
            else:
                _, wm, _ = oracle.project(w, oracle.library(L.K), L.n_keep)
            if cfg.dtype == "f16":
                wm = wm.astype(np.float16)
            total = L.Ho * L.Wo * L.F
            n = max(1, int(round(total * frac)))
            flat = rng.choice(total, size=n, replace=False) if n < total else np.arange(total)
            coords = np.stack([np.zeros(n, dtype=np.int64), flat // (L.Wo * L.F), (flat // L.F) % L.Wo, flat % L.F], axis=1).astype(np.int32)
            self.items.append((L, wm.astype(np.float64), x, coords))

    def run(self):
        acc = 0.0
        for L, wm, x, coords in self.items:
            acc += float(self.oracle.conv3x3_at(wm, x, coords, L.stride).sum())
        return acc


def _omp_threads() -> int:
    v = os.environ.get("OMP_NUM_THREADS")
    if v:
        return int(v)
    return len(os.sched_getaffinity(0))


def _calibrate(cfg, budget_s: float) -> float:
    """Fraction of one image's outputs the oracle can compute in about budget_s seconds."""
    probe = OracleSample(cfg, 0.002)
    t = time.perf_counter(); probe.run(); dt = time.perf_counter() - t
    return float(min(1.0, 0.002 * budget_s / max(dt, 1e-6)))


def cpu_baseline(cfg, budget_s: float = 20.0):
    frac = _calibrate(cfg, budget_s)
    s = OracleSample(cfg, frac)
    t = time.perf_counter(); s.run(); dt = time.perf_counter() - t
    reps = 1
    while dt < 0.5 * budget_s and reps < 16:          # fast hosts: repeat the sample to reach the time budget
        t = time.perf_counter(); s.run(); dt += time.perf_counter() - t
        reps += 1
    return {"value": round(frac * reps / dt, 5), "unit": UNIT, "cores": _omp_threads(), "kind": "oracle",
            "sample": f"{frac * 100:.2f}% of the outputs of one image of all {len(cfg.layers)} layers, {reps} time(s) "
                      f"(direct dense float64 convolution of the masked weights), {dt:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = workloads.configs()[args.config]
    total = args.steps + args.warmup
    per_step = max(2.0, min(20.0, 150.0 / max(total, 1)))
    frac = _calibrate(cfg, per_step)
    s = OracleSample(cfg, frac)
    for _ in range(args.warmup):
        s.run()
    t = time.perf_counter()
    for _ in range(args.steps):
        s.run()
    dt = time.perf_counter() - t
    value = frac * args.steps / dt
    sample = (f"{frac * 100:.3f}% of the outputs of one image of all {len(cfg.layers)} layers per step, "
              f"direct dense float64 convolution of the masked weights")
    out = {"impl": "reference", "metric": METRIC, "value": round(value, 5), "unit": UNIT,
           "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": round(dt / args.steps * 1e3, 2), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"config {cfg.number}: {cfg.name}", "sample": sample, "seed": workloads.BASE_SEED},
           "cpu_baseline": {"value": round(value, 5), "unit": UNIT, "cores": _omp_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": round(value, 5), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=DEFAULT_CONFIG, help="workload number (3 = VGG-16 batch 64 fp16 storage)")
    ap.add_argument("--strong", action="store_true", help="with N > 1 ranks: shard the configuration's batch over the ranks (strong scaling) instead of one whole batch per rank")
    ap.add_argument("--batch", type=int, default=None, help="override the batch size (profiling small cases)")
    ap.add_argument("--layers", default=None, help="comma-separated layer names: run only these (profiling one layer)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--admm-only", action="store_true", help="only the training-side primitives (simplex projection, binarisation, library extraction): prints their JSON object")
    ap.add_argument("--no-overlap", action="store_true", help="projection / packing on the same stream as the convolutions")
    ap.add_argument("--no-graph", action="store_true", help="time plain launches instead of CUDA-graph replays")
    ap.add_argument("--cpu-seconds", type=float, default=20.0)
    ap.add_argument("--no-other-configs", action="store_true", help="skip the short measurements of the other four configurations")
    ap.add_argument("--fma-peak", action="store_true", help="only measure and print the device's multiply-add rate")
    ap.add_argument("--write-traffic", default=None, metavar="NCU_CSV",
                    help="turn an ncu launch list with the DRAM byte counters of the conv6 path into " + os.path.relpath(TRAFFIC_FILE, ROOT))
    args = ap.parse_args()
    if args.write_traffic:
        write_traffic(args.write_traffic)
        return
    if args.impl == "reference":
        run_reference(args)
        return
    world = int(os.environ.get("WORLD_SIZE", "0"))
    if world == 0 and args.gpus > 1:
        # no launcher around us: start one rank per GPU on this node ourselves
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 2000), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if world > 0 and world != args.gpus:
        sys.exit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if args.fma_peak:
        import torch
        import paper_2001_07710_b200 as pc
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
        print(json.dumps({"fma_rn_f32_tflops": round(pc.pat_measure_fma_peak(0), 2), "fma_rn_f32_f16_tflops": round(pc.pat_measure_fma_peak(1), 2),
                          "derived_tflops": round(FMA_PEAK_TFLOPS, 2)}))
        return
    if args.admm_only:
        import torch
        import paper_2001_07710_b200 as pc
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
        print(json.dumps(admm_primitives(pc, torch, measured_peaks()[0], with_cpu=not args.no_cpu)))
        return
    run_ours(args)


if __name__ == "__main__":
    main()
