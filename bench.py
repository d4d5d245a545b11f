"""Benchmark of the integer-convolution hot path on B200.

One "step" is one forward of the ResNet-50-shaped int8 network (batch 256, 224x224x3
synthetic images, random-init weights quantised per layer): every convolution with its
fused bias / residual rescale / BReLU / requantisation epilogue, the max-pool, the integer
average pool and the fully connected layer.  Prints ONE JSON line:

  value      images/s with the batch resident in HBM (CUDA events over exactly K steps,
             max over ranks);
  e2e        the same metric through the network's host-buffer entry: every step copies
             the batch from pinned host memory and reads the logits back;
  roofline   the tensor-core convolution kernel's achieved int8 TOP/s (true MACs of its
             launches / their summed CUDA-event duration in the timed region) against
             2 x the measured dense bf16 peak;
  cpu_baseline  the CPU oracle timed on a bounded sample of the same workload.

``--impl reference`` times the CPU oracle instead (the paper ships no code to install).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "ResNet-50 int8 images/sec"
UNIT = "images/s"
WORKLOAD = "resnet50_b256_224x224x3"
# the other full-size configurations can be timed the same way (--workload); the default and the
# metric of record is the ResNet-50 one
WORKLOADS = {"resnet50": ("ResNet-50 int8 images/sec", "resnet50_b256_224x224x3"),
             "resnet18": ("ResNet-18 int8 images/sec", "resnet18_b256_224x224x3"),
             "resnet152": ("ResNet-152 int8 images/sec", "resnet152_b128_224x224x3"),
             "vdsr": ("VDSR int8 images/sec", "vdsr_16x256x256x1"),
             "vrcnn": ("VRCNN int8 images/sec", "vrcnn_16x512x512x1"),
             "vrcnn_hd": ("VRCNN int8 images/sec", "vrcnn_1x1600x2560x1"),
             "vdsr_hd": ("VDSR int8 images/sec", "vdsr_1x1080x1920x1")}
# DRAM bytes (read + written) per tensor-core launch of one forward, from a one-pass ncu capture
# of the full workload (command and per-kernel figures: profiles/dram_traffic_resnet50_b256.md),
# valid only for the kernel source it was taken on: {workload: (bytes per launch, sha256 of
# csrc/kernel_umma.cu)}.  A changed kernel reports null until the counters are taken again.
DRAM_TRAFFIC = {"resnet50": (93223973, "dd97c3edb066cdea6a601480599b4600effab8ca5c46244dff8b114cbb5b85ab")}
NOMINAL_INT8_TOPS = 4500.0      # NVIDIA's dense INT8 figure for B200 (context only)
INT8_OVER_BF16 = 2.0            # nominal dense ratio 4.5 / 2.25 PFLOP/s


def measured_peaks():
    """(int8 TOP/s peak, HBM GB/s peak, label).  Dense int8 = 2 x the measured bf16 rate; the
    sustained figure is used because the kernel is timed inside a long step."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return INT8_OVER_BF16 * float(m["bf16_tflops_sustained"]), float(m["hbm_gbs"]), "measured"
    return INT8_OVER_BF16 * 1400.0, 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.thread = [], None, None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "25"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r for t, r in self.rows if t0 <= t <= t1 + 0.1] or [r for _, r in self.rows]
        sm, reasons, sm_max = [], set(), None
        for r in rows:
            try:
                sm.append(float(r[0]))
                sm_max = float(r[1])
            except (ValueError, IndexError):
                continue
            for name, col in (("hw_slowdown", 3), ("hw_thermal_slowdown", 4), ("sw_thermal_slowdown", 5),
                              ("sw_power_cap", 6)):
                if len(r) > col and r[col] == "Active":
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": sm_max, "reasons": sorted(reasons),
                "samples": len(sm)}


def probe_mma_rate(block_n: int = 256, iters: int = 100000):
    """(whole-GPU int8 TOP/s, cycles per instruction) of back-to-back tcgen05.mma kind::i8: the
    benchmark's own measurement aid, a small library of its own built next to the layer's."""
    import ctypes as C
    from paper_2006_11735_b200 import build as lib_build
    lib = C.CDLL(lib_build.PROBE_LIB)
    lib.probe_mma_rate.argtypes = [C.c_int32, C.c_int32, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    lib.probe_mma_rate.restype = C.c_int
    tops, cyc = C.c_double(), C.c_double()
    rc = lib.probe_mma_rate(block_n, iters, C.byref(tops), C.byref(cyc))
    if rc != 0:
        raise RuntimeError("probe_mma_rate failed with status %d" % rc)
    return tops.value, cyc.value


def oracle_images_per_s(n_images: int, repeats: int = 1, first: int = 0):
    """Times the CPU oracle, as it stands, on n_images of the workload (forward only)."""
    from oracle import networks as ON
    from workloads.params import load_params
    from workloads import networks as N
    net = N.resnet50()
    params = load_params("resnet50")
    x = ON.net_input(net, first, n_images)
    weights = {op.name: ON.layer_weights(net, op, params[op.name]["delta"]) for op in net.convs()}
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        ON.forward(net, params, x, weights)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return n_images / best, best


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count()
    sample = 2 if args.steps <= 40 else 1       # images per step: the whole run stays within a few minutes
    for _ in range(args.warmup):
        oracle_images_per_s(1)
    t0 = time.perf_counter()
    from oracle import networks as ON
    from workloads.params import load_params
    from workloads import networks as N
    net = N.resnet50()
    params = load_params("resnet50")
    x = ON.net_input(net, 0, sample)
    weights = {op.name: ON.layer_weights(net, op, params[op.name]["delta"]) for op in net.convs()}
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ON.forward(net, params, x, weights)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": "%d images per step" % sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "%d images per step, %d steps" % (sample, args.steps)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--per-layer", action="store_true", help="print the per-layer table to stderr")
    ap.add_argument("--workload", default="resnet50", choices=sorted(WORKLOADS))
    ap.add_argument("--batch", type=int, default=0,
                    help="images per GPU; 0 = the full workload (256). Smaller batches are for profiler "
                         "captures only and are named in config.workload")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    import numpy as np
    import torch

    from paper_2006_11735_b200 import binding as B          # raises if the CUDA library is missing
    from paper_2006_11735_b200 import dist as D
    from paper_2006_11735_b200.network import Network, load_params, net_input
    from workloads import networks as N

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    rank, local_rank, size = D.world()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    D.init("nccl")

    metric, full_name = WORKLOADS[args.workload]
    full = N.by_name(args.workload)
    net = N.by_name(args.workload, n=args.batch) if args.batch > 0 else full   # the full batch per GPU (weak scaling)
    workload = full_name if net.n == full.n else "%s with batch %d (reduced batch: profiling only)" % (full_name, net.n)
    params = load_params(args.workload)
    g = Network(net, params, device=dev)
    x_host = torch.from_numpy(net_input(net)).pin_memory()
    x_dev = x_host.to(dev, non_blocking=True)
    t_out = net.tensors[net.output]
    logits_host = torch.empty((net.n, t_out.h, t_out.w, t_out.c),
                              dtype=torch.int32 if t_out.dtype == "i32" else torch.uint8).pin_memory()
    stream = torch.cuda.current_stream(dev)
    kernels = g.kernels()
    described = g.describe()
    macs = g.conv_macs()
    abytes = g.algorithmic_bytes()

    for _ in range(args.warmup):
        g.forward(x_dev)
    B.iconv_check(stream.cuda_stream)

    # ---- device-resident timing: exactly K steps between two events ----
    D.barrier()
    torch.cuda.synchronize(dev)
    sampler = ClockSampler(local_rank)
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    all_marks = []
    t_wall0 = time.time()
    e0.record(stream)
    for _ in range(args.steps):
        marks = []
        g.forward(x_dev, marks=marks)
        all_marks.append(marks)
    e1.record(stream)
    torch.cuda.synchronize(dev)
    D.barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    ms_local = e0.elapsed_time(e1)
    ms = D.max_over_ranks(ms_local, dev)
    B.iconv_check(stream.cuda_stream)
    # the stem is two launches (repack + GEMM), every other step one
    launches = (len(g.steps) + sum(1 for k in kernels.values() if k == "stem")) * args.steps

    # per-kernel-family time inside the timed region
    fam_ms, fam_macs, fam_bytes, layer_ms = {}, {}, {}, {}
    for marks in all_marks:
        for (_, prev), (name, ev) in zip(marks[:-1], marks[1:]):
            dt = prev.elapsed_time(ev)
            fam = kernels.get(name, "pool")
            fam_ms[fam] = fam_ms.get(fam, 0.0) + dt
            fam_macs[fam] = fam_macs.get(fam, 0) + macs.get(name, 0)
            fam_bytes[fam] = fam_bytes.get(fam, 0) + abytes.get(name, 0)
            layer_ms[name] = layer_ms.get(name, 0.0) + dt / args.steps
    int8_peak, hbm_peak, peak_kind = measured_peaks()
    issue_tops, issue_cycles = probe_mma_rate(256, 100000)             # outside every timed region
    umma_launches = sum(1 for k in kernels.values() if k == "umma") * args.steps
    umma_tops = 2.0 * fam_macs.get("umma", 0) / (fam_ms.get("umma", 1e-9) * 1e-3) / 1e12
    traffic = None
    if args.workload in DRAM_TRAFFIC and net.n == full.n:
        import hashlib
        src = os.path.join(os.path.dirname(os.path.abspath(__file__)), "paper_2006_11735_b200", "csrc", "kernel_umma.cu")
        with open(src, "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() == DRAM_TRAFFIC[args.workload][1]:
                traffic = DRAM_TRAFFIC[args.workload][0]
    roofline = {"kernel": "umma_conv_kernel + umma_window_kernel", "bound": "tensor", "achieved": umma_tops, "peak": int8_peak,
                "unit": "TOP/s", "frac": umma_tops / int8_peak, "traffic": traffic, "peak_kind": peak_kind + " 2 x bf16 sustained",
                "launches": umma_launches, "avg_launch_ms": fam_ms.get("umma", 0.0) / max(1, umma_launches),
                "frac_of_nominal_4500": umma_tops / NOMINAL_INT8_TOPS,
                "issue_rate_peak": issue_tops, "frac_of_issue_rate_peak": umma_tops / issue_tops,
                "time_share": {k: v / sum(fam_ms.values()) for k, v in fam_ms.items()}}
    # the same launches against the memory roofline: most layers of this workload are bound by it
    umma_gbs = fam_bytes.get("umma", 0) / (fam_ms.get("umma", 1e-9) * 1e-3) / 1e9
    roofline_hbm = {"kernel": "umma_conv_kernel + umma_window_kernel", "bound": "hbm", "achieved": umma_gbs, "peak": hbm_peak,
                    "unit": "GB/s", "frac": umma_gbs / hbm_peak, "traffic": traffic,
                    "algorithmic_bytes_per_launch": fam_bytes.get("umma", 0) / max(1, umma_launches), "peak_kind": peak_kind + " copy bandwidth",
                    "algorithmic_bytes_per_step": int(sum(abytes.values())),
                    "whole_step_gbs": sum(abytes.values()) / (ms / args.steps * 1e-3) / 1e9}

    # ---- end to end: pinned host input in, logits out, every step ----
    D.barrier()
    torch.cuda.synchronize(dev)
    # Two device input buffers and a copy stream, as a serving loop would run it: the batch of
    # step i+1 crosses PCIe while step i computes.  Every step's input still comes from pinned
    # host memory inside the timed region, and every step's result goes back to the host.
    x_bufs = [x_dev, torch.empty_like(x_dev)]
    copy_stream = torch.cuda.Stream(dev)
    copied = [torch.cuda.Event() for _ in range(args.steps)]
    consumed = [torch.cuda.Event() for _ in range(args.steps)]
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record(stream)
    copy_stream.wait_stream(stream)
    for i in range(args.steps):
        with torch.cuda.stream(copy_stream):
            if i >= 2:
                copy_stream.wait_event(consumed[i - 2])       # the buffer's previous batch has been read
            x_bufs[i % 2].copy_(x_host, non_blocking=True)
            copied[i].record(copy_stream)
        stream.wait_event(copied[i])
        out = g.forward(x_bufs[i % 2])
        consumed[i].record(stream)
        logits_host.copy_(out, non_blocking=True)
    e3.record(stream)
    torch.cuda.synchronize(dev)
    ms_e2e = D.max_over_ranks(e2.elapsed_time(e3), dev)
    B.iconv_check(stream.cuda_stream)

    if args.per_layer and rank == 0:
        for op in net.ops:
            m = macs.get(op.name, 0)
            t = layer_ms.get(op.name, 0.0)
            sys.stderr.write("%-14s %-6s %8.4f ms %8.1f TOP/s  %s\n" % (op.name, kernels.get(op.name, "pool"), t,
                                                                          2.0 * m / max(t, 1e-9) / 1e9, described.get(op.name, "")))

    cpu = None
    if rank == 0 and size == 1 and not args.no_cpu_baseline and args.workload == "resnet50":
        n_s = 8
        v, dt = oracle_images_per_s(n_s)
        cpu = {"value": v, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
               "sample": "%d images of the same batch, one forward, %.1f s" % (n_s, dt)}

    if rank == 0:
        total_images = net.n * size * args.steps
        line = {"metric": metric, "value": total_images / (ms * 1e-3), "unit": UNIT, "n_gpus": size,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
                "config": {"workload": workload, "global_batch": net.n * size, "parallelism": "dp%d" % size,
                           "l2": "per-step algorithmic traffic (%.1f GB) far exceeds the 126 MB L2" % (sum(abytes.values()) / 1e9),
                           "timing_note": "the timed region carries one CUDA event per layer (the per-kernel durations of "
                                          "`roofline`); the end-to-end loop carries none, which is worth 1-2 %",
                           "int8_tops_whole_step": 2.0 * sum(macs.values()) / (ms / args.steps * 1e-3) / 1e12},
                "clocks": clocks,
                "e2e": {"value": total_images / (ms_e2e * 1e-3), "unit": UNIT,
                        "h2d_bytes_per_step": int(x_host.numel()), "d2h_bytes_per_step": int(logits_host.numel() * logits_host.element_size()),
                        "overlap": "the input copy of step i+1 runs under the compute of step i (two device buffers, one copy stream)"},
                "gpu_launches": launches, "roofline": roofline, "roofline_hbm": roofline_hbm, "cpu_baseline": cpu}
        print(json.dumps(line))
    g.close()
    D.finish()


if __name__ == "__main__":
    main()
