#!/usr/bin/env python
"""Benchmark of the column-wise N:M sparse-convolution hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload: every convolution of ResNet-50 at 224x224, batch 64 per GPU (53 layers; the 7x7 stem
keeps all its columns, every other layer is pruned column-wise 2:4), seeded synthetic inputs
(activations N(0,1), Kaiming-normal weights, bias N(0,1)); each layer runs on its own input
tensor of the right shape.  One step = one pass over all 53 layers through the C ABI.

Prints ONE JSON line: images/s over all GPUs (inputs resident in HBM), the same through the
host-buffer entry point (`e2e`), a roofline object (algorithmic bytes per step / measured time
against the measured HBM copy peak), the CPU checker timed on a bounded sample (`cpu_baseline`),
clocks sampled during the timed region, and a per-layer table (time, useful TFLOP/s, fraction of
max(kept FLOPs / TF32 peak, bytes / HBM peak)).  `--impl reference` times the CPU checker instead.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2507_17301_b200 import inputs  # noqa: E402

METRIC = "resnet50_conv_stack_images_per_s"
UNIT = "images/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
TF32_OVER_BF16 = 1.1 / 2.25   # nominal dense tensor peaks: 1.1 PFLOP/s TF32, 2.25 PFLOP/s bf16
KERNEL_OF_VARIANT = {1: "k_conv_gather", 2: "k_conv_slab", 3: "k_conv_stream", 4: "k_conv_expand", 5: "k_conv_rowrun",
                     6: "k_conv_window", 7: "k_conv_pair", 8: "k_conv_select", 9: "k_conv_planes"}
KERNEL_SOURCE = {"k_conv_gather": "nm_conv_gather.cu", "k_conv_slab": "nm_conv_slab.cu", "k_conv_stream": "nm_conv_stream.cu",
                 "k_conv_expand": "nm_conv_expand.cu", "k_conv_rowrun": "nm_conv_rowrun.cu", "k_conv_window": "nm_conv_window.cu",
                 "k_conv_pair": "nm_conv_pair.cu", "k_conv_select": "nm_conv_select.cu", "k_conv_planes": "nm_conv_planes.cu"}
KEPT_ONLY_VARIANTS = (1, 2, 3, 8)   # kernels that contract over the retained columns only (Algorithm 1 proper)
PLAN_FIELDS = ("variant", "bn", "stages", "split", "kblk", "loads", "issuers", "ksplit")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS, "source": "fallback"}


def source_digest(kernel: str) -> str:
    """Digest of the kernel's source file: DRAM counters taken from an ncu capture are only quoted
    while the kernel is unchanged since."""
    import hashlib
    path = os.path.join(ROOT, "paper_2507_17301_b200", "csrc", KERNEL_SOURCE[kernel])
    with open(path, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def recorded_traffic(kernel: str):
    """DRAM bytes (read + write) per algorithmic byte of `kernel`, from the committed summary of single-layer ncu
    captures (profiles/dram_traffic_<kernel>.txt: key = value lines); None if there is no summary or the kernel
    source has changed since it was taken.  A launch's traffic is this ratio times its algorithmic bytes (the
    captured layers' traffic grows with their bytes).  Output lines still dirty in the L2 when a kernel ends are
    not in ncu's per-kernel write counter, so the figure bounds re-reads, not total writes."""
    path = os.path.join(ROOT, "profiles", f"dram_traffic_{kernel}.txt")
    if not os.path.exists(path):
        return None
    kv = {}
    with open(path) as f:
        for line in f:
            if "=" in line and not line.lstrip().startswith("#"):
                k, v = line.split("=", 1)
                kv[k.strip()] = v.strip()
    try:
        if kv["source_sha256_16"] != source_digest(kernel):
            return None
        return float(kv["dram_bytes_per_algorithmic_byte"])
    except (KeyError, ValueError):
        return None


def algorithmic_bytes(s: inputs.ConvShape) -> int:
    """Bytes one layer must move, each distinct byte once: input touched + output + compressed
    weights + indices + bias.  A strided 1x1 conv touches only the pixels it samples."""
    if s.kh == 1 and s.kw == 1 and s.stride > 1:
        in_elems = s.pixels * s.c_in
    else:
        in_elems = s.batch * s.h * s.w * s.c_in
    n_tiles = -(-s.c_out // s.tile_t)
    return 4 * in_elems + 4 * s.pixels * s.c_out + 4 * s.c_out * s.kk + 2 * n_tiles * s.kk + 4 * s.c_out


def useful_flops(s: inputs.ConvShape) -> int:
    return 2 * s.pixels * s.c_out * s.kk


WORKLOAD = {"depth": 50, "n": 2, "m": 4, "tile": 64}   # the headline configuration; --depth / --nm / --tile change it


def workload(batch: int):
    if WORKLOAD.get("net") == "mobilenet_v2":
        layers = inputs.mobilenet_v2_pointwise(batch, WORKLOAD["n"], WORKLOAD["m"], tile_t=WORKLOAD["tile"])
    else:
        layers = inputs.resnet_conv_stack(WORKLOAD["depth"], batch, WORKLOAD["n"], WORKLOAD["m"], tile_t=WORKLOAD["tile"])
    r = WORKLOAD.get("adaptive")
    if r is not None:
        # the paper's adaptive setting (Sec. 3.1): a group spans a layer's input channels, N = (1 - sparsity) * M
        layers = [s if s.n_keep == s.m_group else s.with_(m_group=s.c_in, n_keep=max(1, round(s.c_in * (1.0 - r))))
                  for s in layers]
    return layers


def workload_name(batch: int) -> str:
    pat = f"{WORKLOAD['n']}of{WORKLOAD['m']}" if WORKLOAD.get("adaptive") is None else f"adaptiveM_sparsity{WORKLOAD['adaptive']}"
    if WORKLOAD.get("net") == "mobilenet_v2":
        return f"mobilenet_v2_pointwise_convs_b{batch}_224_{pat}"
    return f"resnet{WORKLOAD['depth']}_conv_stack_b{batch}_224_{pat}"


class ClockSampler:
    """Polls nvidia-smi for SM clock and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        busy = [v for v in sm if v > 0.5 * (max(mx) if mx else 1)] or sm
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return world, rank, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


def replica_seed(layer: int, rank: int) -> int:
    """Seed of a replica's activations for one layer: every rank draws its own batch."""
    return 1 + 1000 * layer + 7919 * rank


def aggregate_images_per_s(batch_per_gpu: int, world: int, ms_step_max: float) -> float:
    """Whole-job throughput of `world` replicas: all images of a step over the slowest rank's step time."""
    return world * batch_per_gpu / (ms_step_max * 1e-3)


def max_over_ranks(value: float, world: int, device: str = "cuda") -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def measure_tf32_peak() -> float:
    """Dense TF32 matmul throughput (library GEMM, 8192^3, best of 10): the tensor roof per layer."""
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        n = 8192
        a = torch.randn(n, n, device="cuda")
        b = torch.randn(n, n, device="cuda")
        for _ in range(3):
            a @ b
        best = 1e9
        for _ in range(10):
            e0, e1 = torch.cuda.Event(True), torch.cuda.Event(True)
            e0.record()
            a @ b
            e1.record()
            e1.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return 2 * n ** 3 / (best * 1e-3) / 1e12
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old


def run_reference(args):
    """The CPU checker, as it stands, on a bounded sample: image 0 of every layer of the stack."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    layers = workload(1)
    prepared = []
    for li, s in enumerate(layers):
        w = inputs.make_weights(s, li)
        values, indices = oracle.prune(w.numpy(), s.n_keep, s.m_group, s.tile_t)
        prepared.append((s, values, indices, inputs.make_activations(s, li, batch=1).numpy(), inputs.make_bias(s, li).numpy()))

    def step():
        for s, values, indices, x, b in prepared:
            oracle.conv2d(values, indices, s.kh, s.kw, s.c_in, s.tile_t, x, (s.stride,) * 2, (s.pad,) * 2,
                          (s.dil,) * 2, b, s.relu)

    steps = max(1, min(args.steps, 5))
    for _ in range(min(args.warmup, 1)):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    value = 1.0 / dt
    sample = f"image 0 of each of the {len(layers)} layers per step (1 image of the batch)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(64), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


REL_FRO_TOL = 2e-3      # relative Frobenius error allowed under TF32
MAX_ABS_TOL = 1e-2      # max-abs error allowed, as a fraction of max|ref|


def parity_and_cpu_baseline(nm, state):
    """Every layer under the plan that is about to be timed against the CPU checker on the bench's own
    tensors: pruning bit for bit, image 0 of the output within the TF32 tolerance.  The checker's
    convolutions are timed on the way: they are the `cpu_baseline` sample.  Runs outside the timed region."""
    import numpy as np
    import oracle
    worst_rel, worst_abs, t_total = 0.0, 0.0, 0.0
    failed, prune_ok = [], True
    for li, (s, hnd, x, bias, y, plan) in enumerate(state):
        nm.nm_conv2d(hnd, x, s.kh, s.kw, s.stride, s.pad, s.dil, bias, s.relu, y=y, plan=plan)
        nm.nm_weights_check(hnd)
        v, i = nm.nm_weights_export(hnd)
        torch.cuda.synchronize()
        vr, ir = oracle.prune(inputs.make_weights(s, li).numpy(), s.n_keep, s.m_group, s.tile_t)
        if not (np.array_equal(i.cpu().numpy(), ir) and np.array_equal(v.cpu().numpy().view(np.uint32), vr.view(np.uint32))):
            prune_ok = False
            failed.append(s.name + " (pruning)")
        x0, b0 = x[0:1].cpu().numpy(), bias.cpu().numpy()
        t0 = time.perf_counter()
        yr = oracle.conv2d(vr, ir, s.kh, s.kw, s.c_in, s.tile_t, x0, (s.stride,) * 2, (s.pad,) * 2, (s.dil,) * 2, b0, s.relu)
        t_total += time.perf_counter() - t0
        d = y[0:1].cpu().numpy().astype(np.float64) - yr.astype(np.float64)
        ref_n = float(np.sqrt((yr.astype(np.float64) ** 2).sum()))
        rel = float(np.sqrt((d ** 2).sum())) / max(ref_n, 1e-30)
        mx = float(np.abs(d).max()) / max(float(np.abs(yr).max()), 1e-30)
        worst_rel, worst_abs = max(worst_rel, rel), max(worst_abs, mx)
        if not (np.isfinite(d).all() and rel <= REL_FRO_TOL and mx <= MAX_ABS_TOL):
            failed.append(s.name)
    sample = f"image 0 of each of the {len(state)} layers (1 image of the batch), the bench's own tensors"
    parity = {"layers": len(state), "max_rel_fro": worst_rel, "max_abs_over_ref": worst_abs, "prune_bit_exact": prune_ok,
              "ok": not failed, "failed": failed, "tolerance": {"rel_fro": REL_FRO_TOL, "max_abs_over_ref": MAX_ABS_TOL},
              "sample": "image 0 of every layer's output under the plan that is timed, against the CPU checker on the same input"}
    baseline = {"value": 1.0 / t_total, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample}
    return parity, baseline


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--no-extras", action="store_true", help="skip e2e, cpu baseline, cuDNN and per-layer passes")
    ap.add_argument("--layer", default=None, help="run only the layers whose name contains this text (profiling aid)")
    ap.add_argument("--variant", type=int, default=None, help="force a kernel variant instead of auto-tuning")
    ap.add_argument("--bn", type=int, default=0, help="with --variant: output channels per CTA")
    ap.add_argument("--stages", type=int, default=0, help="with --variant: ring depth")
    ap.add_argument("--split", type=int, default=0, help="with --variant: the plan's split field")
    ap.add_argument("--kblk", type=int, default=0, help="with --variant: 32-column blocks per pipeline stage")
    ap.add_argument("--loads", type=int, default=0, help="with --variant 8: 1 = im2col loads, 2 = patch loads")
    ap.add_argument("--issuers", type=int, default=0, help="with --variant 8: MMA issuer threads")
    ap.add_argument("--ksplit", type=int, default=0, help="with --variant 8: ranges of the reduction axis")
    ap.add_argument("--depth", type=int, default=50, choices=[18, 34, 50, 101, 152], help="ResNet depth of the conv stack")
    ap.add_argument("--net", default="resnet", choices=["resnet", "mobilenet_v2"],
                    help="mobilenet_v2: its pointwise (1x1) convolutions only, the layers the paper prunes there")
    ap.add_argument("--nm", default="2:4", help="N:M pattern of the pruned layers, e.g. 1:4 or 2:8")
    ap.add_argument("--tile", type=int, default=64, help="pruning tile width T")
    ap.add_argument("--adaptive", type=float, default=None,
                    help="sparsity in (0, 1): groups span a layer's input channels (M = C_in, N = (1 - sparsity) * M)")
    ap.add_argument("--json-out", default=None, help="also write the result, indented, to this file")
    ap.add_argument("--save-plans", default=None, help="write the auto-tuned plans to this JSON file")
    ap.add_argument("--load-plans", default=None, help="use the plans of this JSON file instead of auto-tuning")
    args = ap.parse_args()
    WORKLOAD.update(depth=args.depth, n=int(args.nm.split(":")[0]), m=int(args.nm.split(":")[1]), tile=args.tile,
                    adaptive=args.adaptive, net=args.net)
    if args.impl == "reference":
        return run_reference(args)
    if args.warmup < 3:
        args.warmup = 3

    world, rank, local = dist_setup(args.gpus)
    from paper_2507_17301_b200 import build
    if rank == 0:
        build.build()
    barrier(world)
    from paper_2507_17301_b200 import nm  # fails loudly if the CUDA library is missing

    pk = peaks()
    layers = workload(args.batch)
    if args.layer:
        layers = [s for s in layers if args.layer in s.name]
        assert layers, f"no layer matches {args.layer!r}"
    dev = torch.device("cuda", local if world > 1 else 0)
    loaded = None
    if args.load_plans:
        with open(args.load_plans) as f:
            loaded = json.load(f)
    state = []
    for li, s in enumerate(layers):
        w = inputs.make_weights(s, li).to(dev)
        hnd = nm.nm_prune(w, s.n_keep, s.m_group, s.tile_t)
        del w
        g = torch.Generator(device="cpu").manual_seed(replica_seed(li, rank))
        # activations ~ N(0,1): drawn on the host in slices to bound pinned/pageable staging
        x = torch.empty((s.batch, s.h, s.w, s.c_in), dtype=torch.float32, device=dev)
        for b0 in range(0, s.batch, 8):
            x[b0:b0 + 8] = torch.randn((min(8, s.batch - b0), s.h, s.w, s.c_in), generator=g).to(dev)
        bias = inputs.make_bias(s, li).to(dev)
        y = torch.empty((s.batch, s.ho, s.wo, s.c_out), dtype=torch.float32, device=dev)
        if loaded is not None and s.name in loaded:
            plan = nm.nm_plan_t()
            for k in PLAN_FIELDS:
                setattr(plan, k, int(loaded[s.name].get(k, 0)))
            nm.nm_weights_reserve(hnd, nm.nm_plan_scratch_bytes(hnd, x.shape, s.stride, s.pad, s.dil, plan))
        elif args.variant is None:
            plan, _ = nm.nm_autotune(hnd, x, s.stride, s.pad, s.dil, bias, s.relu, y_scratch=y, kh=s.kh, kw=s.kw)
        else:
            plan = nm.nm_plan_t()
            plan.variant, plan.bn, plan.stages, plan.split = args.variant, args.bn, args.stages, args.split
            plan.kblk, plan.loads, plan.issuers, plan.ksplit = args.kblk, args.loads, args.issuers, args.ksplit
            nm.nm_weights_reserve(hnd, nm.nm_plan_scratch_bytes(hnd, x.shape, s.stride, s.pad, s.dil, plan))
        state.append((s, hnd, x, bias, y, plan))

    if args.save_plans and rank == 0:
        with open(args.save_plans, "w") as f:
            json.dump({s.name: plan.as_dict() for s, _, _, _, _, plan in state}, f, indent=1)

    def step():
        for s, hnd, x, bias, y, plan in state:
            nm.nm_conv2d(hnd, x, s.kh, s.kw, s.stride, s.pad, s.dil, bias, s.relu, y=y, plan=plan)

    parity = baseline = None
    if rank == 0 and world == 1 and not args.no_extras:
        parity, baseline = parity_and_cpu_baseline(nm, state)

    for _ in range(args.warmup):
        step()
    barrier(world)
    sampler = ClockSampler(local if world > 1 else 0)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if not args.no_extras:
        for _ in range(200):   # about half a second of untimed steps so that the clock sampler sees the load
            step()
    launches0 = nm.nm_launch_count()
    barrier(world)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier(world)
    ms_total = max_over_ranks(e0.elapsed_time(e1), world)
    launches = nm.nm_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    for s, hnd, *_ in state:
        nm.nm_weights_check(hnd)
    ms_step = ms_total / args.steps
    value = aggregate_images_per_s(args.batch, world, ms_step)

    bytes_step = sum(algorithmic_bytes(s) for s in layers)
    flops_step = sum(useful_flops(s) for s in layers)
    achieved_gbs = bytes_step / (ms_step * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "tf32",
        "data": "synthetic",
        "config": {"workload": workload_name(args.batch) + (f" [only {args.layer}]" if args.layer else ""),
                   "layers": len(layers), "batch_per_gpu": args.batch,
                   "tile_t": WORKLOAD["tile"], "plans": "per layer by nm_autotune" if args.variant is None and not args.load_plans else "given", "cache": f"inputs larger than L2 ({bytes_step / 1e9:.1f} GB touched per step, one buffer per layer)",
                   "parallelism": f"replicas x{world}"},
        "useful_tflops": flops_step / (ms_step * 1e-3) / 1e12,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": achieved_gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved_gbs / pk["hbm_gbs"], "traffic": None, "peak_source": pk["source"],
                     "kernel": "conv kernels of the whole stack (53 launches per step)"},
    }

    if rank == 0 and not args.no_extras and world == 1:
        # the same step recorded once as a CUDA graph and replayed: what the GPU does when the host's launch
        # calls are out of the way (matters for networks of small layers)
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    step()
            torch.cuda.current_stream().wait_stream(side)
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(True), torch.cuda.Event(True)
            a.record()
            for _ in range(args.steps):
                graph.replay()
            b.record()
            b.synchronize()
            g_ms = a.elapsed_time(b) / args.steps
            out["graph_replay"] = {"value": args.batch / (g_ms * 1e-3), "unit": UNIT, "ms_per_step": g_ms,
                                   "note": "the timed step captured in one CUDA graph and replayed"}
            del graph
        except Exception as e:
            out["graph_replay"] = {"unavailable": f"{type(e).__name__}: {e}"[:300]}
            torch.cuda.synchronize()
        # tensor roof: the measured bf16 GEMM peak scaled by the nominal TF32 : bf16 ratio; the library
        # TF32 GEMM timed here is context
        tf32_peak = pk["bf16_tflops"] * TF32_OVER_BF16
        out["tf32_peak_tflops"] = tf32_peak
        out["tf32_peak_source"] = f"{pk['source']} bf16 GEMM peak x nominal TF32/bf16 ratio (1.1 / 2.25)"
        out["tf32_cublas_tflops_measured"] = measure_tf32_peak()
        # per-layer pass: each layer launched back to back on rotating (input, output) buffer sets whose
        # total exceeds twice the L2 capacity, so that every launch finds its data in HBM, and timed as a
        # whole (events around single launches would add the event overhead and forbid launch overlap)
        L2_BYTES = 126e6
        per = []
        for s, hnd, x, bias, y, plan in state:
            set_bytes = (x.numel() + y.numel()) * 4
            n_sets = int(max(2, min(24, -(-2.2 * L2_BYTES // set_bytes))))
            xs = [x] + [x.clone() for _ in range(n_sets - 1)]
            ys = [y] + [torch.empty_like(y) for _ in range(n_sets - 1)]
            launches = max(20, 2 * n_sets)

            def burst():
                for k in range(launches):
                    nm.nm_conv2d(hnd, xs[k % n_sets], s.kh, s.kw, s.stride, s.pad, s.dil, bias, s.relu,
                                 y=ys[k % n_sets], plan=plan)

            # the burst is recorded once as a CUDA graph and replayed, so that small layers are timed at the
            # GPU's pace and not at the pace of the host's launch calls; if the capture is refused the burst
            # is launched directly
            replay = burst
            try:
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    with torch.cuda.graph(graph, stream=side):
                        burst()
                torch.cuda.current_stream().wait_stream(side)
                replay = graph.replay
                per_layer_mode = "graph replay"
            except Exception:
                torch.cuda.synchronize()
                per_layer_mode = "direct launches"
            samples = []
            for rep in range(3):
                for k in range(n_sets):   # also evicts what the previous repetition left in L2 in order
                    nm.nm_conv2d(hnd, xs[k], s.kh, s.kw, s.stride, s.pad, s.dil, bias, s.relu, y=ys[k], plan=plan)
                a, b = torch.cuda.Event(True), torch.cuda.Event(True)
                a.record()
                replay()
                b.record()
                b.synchronize()
                samples.append(a.elapsed_time(b) / launches)
            # the same layer on ONE buffer pair, back to back: operands that fit stay in the L2 ("warm"; context only,
            # the roofline fractions use the cold figure)
            warm_ms = None
            try:
                def warm_burst():
                    for _k in range(launches):
                        nm.nm_conv2d(hnd, xs[0], s.kh, s.kw, s.stride, s.pad, s.dil, bias, s.relu, y=ys[0], plan=plan)
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                wgraph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    with torch.cuda.graph(wgraph, stream=side):
                        warm_burst()
                torch.cuda.current_stream().wait_stream(side)
                wgraph.replay()
                a, b = torch.cuda.Event(True), torch.cuda.Event(True)
                a.record()
                wgraph.replay()
                b.record()
                b.synchronize()
                warm_ms = a.elapsed_time(b) / launches
                del wgraph
            except Exception:
                torch.cuda.synchronize()
            per.append((samples, warm_ms))
            del replay, xs, ys
        table, t_roof_sum = [], 0.0
        for (s, hnd, x, bias, y, plan), (ts, warm_ms) in zip(state, per):
            ms = statistics.median(ts)
            t_tc = useful_flops(s) / (tf32_peak * 1e12) * 1e3
            t_hbm = algorithmic_bytes(s) / (pk["hbm_gbs"] * 1e9) * 1e3
            t_roof = max(t_tc, t_hbm)
            t_roof_sum += t_roof
            table.append({"layer": s.name, "shape": f"{s.c_in}->{s.c_out} {s.kh}x{s.kw}/{s.stride} @{s.h}",
                          "ms": round(ms, 4), "ms_warm": round(warm_ms, 4) if warm_ms is not None else None,
                          "kept_columns_only": plan.variant in KEPT_ONLY_VARIANTS or s.n_keep == s.m_group,
                          "useful_tflops": round(useful_flops(s) / (ms * 1e-3) / 1e12, 2),
                          "gbs": round(algorithmic_bytes(s) / (ms * 1e-3) / 1e9, 1),
                          "bound": "tensor" if t_tc > t_hbm else "hbm", "roofline_frac": round(t_roof / ms, 3),
                          "plan": plan.as_dict()})
        out["stack_roofline_frac"] = t_roof_sum / ms_step
        out["stack_roofline_note"] = ("sum over layers of max(kept FLOPs / TF32 peak, algorithmic bytes / HBM peak) "
                                      "divided by the measured time of a step")
        out["per_layer"] = table
        out["per_layer_mode"] = per_layer_mode
        out["per_layer_note"] = ("ms: cold (rotating buffer sets larger than twice the L2, every launch finds its operands in HBM); "
                                 "ms_warm: the same launch repeated on one buffer pair (operands that fit stay in L2)")
        out["layers_at_half_roofline"] = sum(1 for r in table if r["roofline_frac"] >= 0.5)
        out["launches_kept_columns_only"] = sum(1 for r in table if r["kept_columns_only"])
        # tile width as a tuning knob (Sec. 3.3, Sec. 4.4) on the tensor-bound layers: per candidate T the fastest plan,
        # the fastest plan among the kernels that skip the pruned columns, and the share of the L1 mass the
        # pruning retains (the accuracy proxy: wider tiles share a kept set among more rows and retain less)
        if args.variant is None and not args.load_plans and not args.layer:
            choice = []
            for li, ((s, hnd, x, bias, y, plan), row) in enumerate(zip(state, table)):
                if row["bound"] != "tensor" or s.n_keep == s.m_group:
                    continue
                w = inputs.make_weights(s, li).to(dev)
                cands = []
                for t in (64, 128, 256):
                    if s.c_out % t != 0:
                        continue
                    h_t = nm.nm_prune(w, s.n_keep, s.m_group, t)
                    kept, total = nm.nm_weights_retained_l1(h_t)
                    p_all, ms_all = nm.nm_autotune(h_t, x, s.stride, s.pad, s.dil, bias, s.relu, y_scratch=y, kh=s.kh, kw=s.kw)
                    os.environ["NM_AUTOTUNE_VARIANTS"] = ",".join(str(v) for v in KEPT_ONLY_VARIANTS)
                    p_kept, ms_kept = nm.nm_autotune(h_t, x, s.stride, s.pad, s.dil, bias, s.relu, y_scratch=y, kh=s.kh, kw=s.kw)
                    del os.environ["NM_AUTOTUNE_VARIANTS"]
                    cands.append({"tile_t": t, "retained_l1": round(kept / total, 4), "ms": round(ms_all, 4),
                                  "variant": p_all.variant, "ms_kept_columns_only": round(ms_kept, 4),
                                  "variant_kept_columns_only": p_kept.variant})
                    h_t.free()
                best = min(cands, key=lambda c: c["ms"])
                choice.append({"layer": s.name, "candidates": cands, "fastest_tile_t": best["tile_t"]})
                del w
            out["tile_choice"] = {"layers": choice,
                                  "note": "single cold launches timed by nm_autotune (median of 9); the headline keeps T = "
                                          f"{WORKLOAD['tile']} for every layer"}
        # roofline object: the kernel that takes the largest share of a step, over all its launches
        by_kernel = {}
        for (s, hnd, x, bias, y, plan), row in zip(state, table):
            k = KERNEL_OF_VARIANT.get(plan.variant, "library default")
            acc = by_kernel.setdefault(k, {"ms": 0.0, "bytes": 0, "flops": 0, "launches": 0, "roof_ms": 0.0})
            acc["roof_ms"] += row["ms"] * row["roofline_frac"]
            acc["ms"] += row["ms"]
            acc["bytes"] += algorithmic_bytes(s)
            acc["flops"] += useful_flops(s)
            acc["launches"] += 1
        total_ms = sum(v["ms"] for v in by_kernel.values())
        out["kernel_shares"] = {k: {"launches": v["launches"], "ms": round(v["ms"], 4), "share": round(v["ms"] / total_ms, 3)}
                                for k, v in by_kernel.items()}
        dom = max(by_kernel, key=lambda k: by_kernel[k]["ms"])
        d = by_kernel[dom]
        dom_gbs = d["bytes"] / (d["ms"] * 1e-3) / 1e9
        traffic = recorded_traffic(dom) if dom in KERNEL_SOURCE else None
        out["roofline"] = {
            "bound": "hbm", "achieved": dom_gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": dom_gbs / pk["hbm_gbs"],
            # per launch: DRAM bytes per algorithmic byte from single-layer ncu captures x this kernel's algorithmic bytes
            # per launch (null once the kernel source has changed since the capture)
            "traffic": traffic * d["bytes"] / d["launches"] if traffic else None,
            "traffic_note": "scaled from single-layer captures (profiles/dram_traffic_<kernel>.txt); output lines still "
                            "dirty in L2 at kernel end are not counted by the per-kernel write counter",
            "peak_source": pk["source"] + " (burst copy figure)",
            "kernel": dom, "launches_per_step": d["launches"], "avg_launch_ms": d["ms"] / d["launches"],
            "algorithmic_bytes_per_launch": d["bytes"] / d["launches"],
            "share_of_step": d["ms"] / total_ms,
            "useful_tflops": d["flops"] / (d["ms"] * 1e-3) / 1e12,
            "time_frac_of_layer_rooflines": d["roof_ms"] / d["ms"],   # some of its layers are tensor-bound, not HBM-bound
            "note": "algorithmic bytes of the layers this kernel runs / their summed launch times (per layer: median of 3 runs "
                    "of >= 20 back-to-back launches, recorded as a CUDA graph and replayed, on rotating buffers larger "
                    "than twice the L2)",
        }

        # the same stack restricted to the kernels that contract over the retained columns only (variants
        # 1-3 and 8: Algorithm 1 proper, kept FLOPs only); the headline lets the auto-tuner also take the
        # expanded-operand kernels, which multiply the zeros
        if args.variant is None and not args.load_plans and not args.layer:
            os.environ["NM_AUTOTUNE_VARIANTS"] = ",".join(str(v) for v in KEPT_ONLY_VARIANTS)
            gplans = []
            for s, hnd, x, bias, y, plan in state:
                if s.n_keep == s.m_group:     # an unpruned layer (the stem) has no pruned columns to skip: any kernel qualifies
                    gplans.append(plan)
                    continue
                gp, _ = nm.nm_autotune(hnd, x, s.stride, s.pad, s.dil, bias, s.relu, y_scratch=y, kh=s.kh, kw=s.kw)
                gplans.append(gp)
            del os.environ["NM_AUTOTUNE_VARIANTS"]

            def gather_step():
                for (s, hnd, x, bias, y, plan), gp in zip(state, gplans):
                    nm.nm_conv2d(hnd, x, s.kh, s.kw, s.stride, s.pad, s.dil, bias, s.relu, y=y, plan=gp)
            for _ in range(3):
                gather_step()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(True), torch.cuda.Event(True)
            a.record()
            for _ in range(args.steps):
                gather_step()
            b.record()
            b.synchronize()
            g_ms = a.elapsed_time(b) / args.steps
            out["gather_only"] = {"value": args.batch / (g_ms * 1e-3), "unit": UNIT, "ms_per_step": g_ms,
                                  "useful_tflops": flops_step / (g_ms * 1e-3) / 1e12,
                                  "variants": {str(v): sum(1 for gp in gplans if gp.variant == v) for v in sorted({gp.variant for gp in gplans})},
                                  "note": "plans restricted to the kernels that contract over the retained columns only "
                                          "(variants 1-3 and 8: Algorithm 1 proper); unpruned layers (the stem) keep their plan, "
                                          "they have no pruned column; the headline lets the tuner also take the "
                                          "expanded-operand kernels, which multiply the zeros of the pruned columns"}

        # the same layers chained as the network's dataflow: stem -> max-pool -> residual blocks, every
        # layer reading its predecessor's output, shortcut additions fused into the last conv of a block
        if not args.layer and args.net == "resnet":
            idx = {s.name: i for i, (s, *_rest) in enumerate(state)}
            pool_out = torch.empty((args.batch, state[1][0].h, state[1][0].w, 64), dtype=torch.float32, device=dev)
            prefixes = []
            for s, *_rest in state[1:]:
                pre = s.name.rsplit("_", 1)[0]
                if pre not in prefixes:
                    prefixes.append(pre)

            def conv(i, x_in, relu, residual=None):
                s, hnd, _x, bias, y, plan = state[i]
                nm.nm_conv2d(hnd, x_in, s.kh, s.kw, s.stride, s.pad, s.dil, bias, relu, y=y, plan=plan, residual=residual)
                return y

            branch = torch.cuda.Stream()          # a block's projection shortcut runs beside its main path
            ev_fork, ev_join = torch.cuda.Event(), torch.cuda.Event()

            def chained_step(x_in=None, before_last=None):
                main = torch.cuda.current_stream()
                cur = conv(0, state[0][2] if x_in is None else x_in, True)
                cur = nm.nm_maxpool2d(cur, 3, 2, 1, y=pool_out)
                for pre in prefixes:
                    if before_last is not None and pre == prefixes[-1]:
                        before_last()    # the last block writes the step's output buffer
                    forked = pre + "_ds" in idx
                    if forked:
                        ev_fork.record(main)
                        branch.wait_event(ev_fork)
                        with torch.cuda.stream(branch):
                            shortcut = conv(idx[pre + "_ds"], cur, False)
                            ev_join.record(branch)
                    else:
                        shortcut = cur
                    t = conv(idx[pre + "_c1"], cur, True)
                    if pre + "_c3" in idx:                       # bottleneck block
                        t = conv(idx[pre + "_c2"], t, True)
                        if forked:
                            main.wait_event(ev_join)
                        cur = conv(idx[pre + "_c3"], t, True, residual=shortcut)
                    else:                                        # basic block
                        if forked:
                            main.wait_event(ev_join)
                        cur = conv(idx[pre + "_c2"], t, True, residual=shortcut)
                return cur

            for _ in range(3):
                last = chained_step()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(True), torch.cuda.Event(True)
            a.record()
            for _ in range(args.steps):
                chained_step()
            b.record()
            b.synchronize()
            c_ms = a.elapsed_time(b) / args.steps
            out["chained"] = {"value": args.batch / (c_ms * 1e-3), "unit": UNIT, "ms_per_step": c_ms,
                              "finite": bool(torch.isfinite(last).all()),
                              "note": "conv backbone in dataflow order: stem, 3x3/2 max-pool, residual blocks with the "
                                      "shortcut addition fused into the block's last convolution, projection "
                                      "shortcuts on a second stream beside the block's main path"}
            # ... fed from the host: images copied in from pinned memory and the final feature map copied back,
            # every step, inside the timed region (what an inference loop around the backbone moves over PCIe)
            x0 = state[0][2]
            x_host = torch.empty(x0.shape, dtype=torch.float32, pin_memory=True).copy_(x0.cpu())
            y_host = torch.empty(last.shape, dtype=torch.float32, pin_memory=True)
            xin = [x0, torch.empty_like(x0)]
            s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
            ev_in = [torch.cuda.Event(), torch.cuda.Event()]
            ev_comp = [torch.cuda.Event(), torch.cuda.Event()]
            ev_out = torch.cuda.Event()

            def fed_from_host(n):
                """n chained steps; step i + 1's images are uploaded and step i - 1's output is downloaded
                while step i computes (two input buffers, three streams)."""
                main = torch.cuda.current_stream()
                s_in.wait_stream(main)
                with torch.cuda.stream(s_in):
                    xin[0].copy_(x_host, non_blocking=True)
                    ev_in[0].record(s_in)
                for i in range(n):
                    cur_buf = i & 1
                    if i + 1 < n:
                        with torch.cuda.stream(s_in):
                            if i >= 1:
                                s_in.wait_event(ev_comp[(i - 1) & 1])   # that step read the buffer about to be refilled
                            xin[(i + 1) & 1].copy_(x_host, non_blocking=True)
                            ev_in[(i + 1) & 1].record(s_in)
                    main.wait_event(ev_in[cur_buf])
                    y_dev = chained_step(xin[cur_buf], (lambda: main.wait_event(ev_out)) if i > 0 else None)
                    ev_comp[cur_buf].record(main)
                    with torch.cuda.stream(s_out):
                        s_out.wait_event(ev_comp[cur_buf])
                        y_host.copy_(y_dev, non_blocking=True)
                        ev_out.record(s_out)
                main.wait_stream(s_out)

            fed_from_host(3)
            torch.cuda.synchronize()
            fed_ok = bool(torch.equal(y_host, last.cpu()))
            a, b = torch.cuda.Event(True), torch.cuda.Event(True)
            a.record()
            fed_from_host(args.steps)
            b.record()
            b.synchronize()
            h_ms = a.elapsed_time(b) / args.steps
            out["chained_from_host"] = {"value": args.batch / (h_ms * 1e-3), "unit": UNIT, "ms_per_step": h_ms,
                                        "h2d_bytes_per_step": x_host.numel() * 4, "d2h_bytes_per_step": y_host.numel() * 4,
                                        "same_output_as_resident": fed_ok,
                                        "note": "the chained step with its input images copied from pinned host memory and its "
                                                "output copied back every step, inside the timed region; uploads and downloads "
                                                "overlap the neighbouring steps (two input buffers, three streams)"}
            del x_host, y_host, xin
            # the same step recorded once as a CUDA graph and replayed (no per-launch host work in the timed region)
            try:
                ref = last.clone()
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    with torch.cuda.graph(graph, stream=side):
                        g_last = chained_step()
                torch.cuda.current_stream().wait_stream(side)
                for _ in range(3):
                    graph.replay()
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(True), torch.cuda.Event(True)
                a.record()
                for _ in range(args.steps):
                    graph.replay()
                b.record()
                b.synchronize()
                g_ms = a.elapsed_time(b) / args.steps
                out["chained_graph"] = {"value": args.batch / (g_ms * 1e-3), "unit": UNIT, "ms_per_step": g_ms,
                                        "same_output_as_launches": bool(torch.equal(g_last, ref)),
                                        "note": "the chained step captured in one CUDA graph and replayed"}
                for _s, hnd, *_r in state:
                    nm.nm_weights_check(hnd)
            except Exception as e:  # a capture the runtime refuses is reported, not fatal
                out["chained_graph"] = {"unavailable": f"{type(e).__name__}: {e}"[:300]}
                torch.cuda.synchronize()

        # cuDNN dense convolution on the same shapes (context, unpruned weights, TF32 allowed)
        try:
            torch.backends.cudnn.allow_tf32 = True
            torch.backends.cudnn.benchmark = True
            dense = []
            for li, (s, hnd, x, bias, y, plan) in enumerate(state):
                w = inputs.make_weights(s, li).to(dev).permute(0, 3, 1, 2).contiguous(memory_format=torch.channels_last)
                dense.append((s, x.permute(0, 3, 1, 2), w, bias))
            def dense_step():
                for s, xx, w, b in dense:
                    torch.nn.functional.conv2d(xx, w, b, stride=s.stride, padding=s.pad, dilation=s.dil)
            for _ in range(3):
                dense_step()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(True), torch.cuda.Event(True)
            a.record()
            for _ in range(5):
                dense_step()
            b.record()
            b.synchronize()
            out["cudnn_dense_images_per_s"] = args.batch / (a.elapsed_time(b) / 5 * 1e-3)
            del dense
        except Exception as exc:  # context only
            out["cudnn_dense_images_per_s"] = f"unavailable: {exc}"

        # end to end through the host-buffer entry point: pinned host x / y per layer
        host = []
        h2d = d2h = 0
        for s, hnd, x, bias, y, plan in state:
            xh = torch.empty(x.shape, dtype=torch.float32).pin_memory()
            xh.copy_(x)
            yh = torch.empty(y.shape, dtype=torch.float32).pin_memory()
            bh = bias.cpu().pin_memory()
            host.append((xh, bh, yh))
            h2d += xh.numel() * 4 + bh.numel() * 4
            d2h += yh.numel() * 4
        # the layers are independent (own buffers), so they are issued round-robin on three streams: one
        # layer's upload, another's kernel and a third's download overlap (PCIe is full duplex)
        e2e_streams = [torch.cuda.Stream() for _ in range(3)]

        def e2e_step():
            for i, ((s, hnd, x, bias, y, plan), (xh, bh, yh)) in enumerate(zip(state, host)):
                with torch.cuda.stream(e2e_streams[i % 3]):
                    nm.nm_conv2d_host(hnd, xh, x, s.stride, s.pad, s.dil, bh, bias, s.relu, yh, y, plan=plan)

        def e2e_join():
            for st in e2e_streams:
                torch.cuda.current_stream().wait_stream(st)

        torch.cuda.synchronize()
        e2e_step()
        torch.cuda.synchronize()
        n_e2e = max(1, min(args.steps, 3))
        a, b = torch.cuda.Event(True), torch.cuda.Event(True)
        for st in e2e_streams:
            st.wait_stream(torch.cuda.current_stream())
        a.record()
        for st in e2e_streams:
            st.wait_event(a)
        for _ in range(n_e2e):
            e2e_step()
        e2e_join()
        b.record()
        b.synchronize()
        out["e2e"] = {"value": args.batch / (a.elapsed_time(b) / n_e2e * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e,
                      "note": "every layer's input copied from pinned host memory and every output copied back "
                              "(nm_conv2d_host per layer, three streams)"}
        del host
        out["cpu_baseline"] = baseline
        out["parity"] = parity

    if rank == 0:
        if args.json_out:
            with open(args.json_out, "w") as f:
                json.dump(out, f, indent=1)
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    if parity is not None and not parity["ok"]:
        sys.exit(1)   # a timed plan whose output is wrong is not a result


if __name__ == "__main__":
    main()
