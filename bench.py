"""Benchmark of the integer-convolution hot path on B200.

One "step" is one forward of the ResNet-50-shaped int8 network (batch 256, 224x224x3
synthetic images, random-init weights quantised per layer): every convolution with its
fused bias / residual rescale / BReLU / requantisation epilogue, the max-pool, the integer
average pool and the fully connected layer.  Prints ONE JSON line:

  value      images/s with the batch resident in HBM (CUDA events over exactly K steps,
             max over ranks);
  e2e        the same metric through the network's host-buffer entry: every step copies
             the batch from pinned host memory and reads the logits back;
  roofline   the tensor-core convolution kernels' achieved int8 TOP/s (true MACs of their
             launches / their summed CUDA-event duration in the timed region) against
             2 x the measured dense bf16 peak (burst and sustained, both printed);
  roofline_hbm  the same launches' algorithmic bytes per second against the measured copy rate;
  per_layer  every layer: time, TOP/s, GB/s, percent of each peak, the bound that binds it;
  elementwise  the bandwidth-bound kernels (pools, stand-alone add, thin layers, calibration)
             timed alone through the C ABI, GB/s against the measured copy rate;
  vdsr       the second target workload (VDSR-shaped, 16 x 256 x 256) timed the same way;
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
# DRAM bytes (read + written) per launch of the dominant kernel, from an ncu capture of that
# kernel's launches in one forward (two one-pass counters): {workload: (bytes per launch, kernel,
# sha256 of the kernel's source the counters were taken on, that source file)}.  A changed kernel
# reports null until the counters are taken again.
DRAM_TRAFFIC = {"resnet50": (46245691, "umma_conv_kernel (cta pairs)", "62e1eff8a847e6eaaa5fff8f3f2d34a89c64c72bed6fa101b64178549eee88af",
                             "umma_device.cuh")}
NOMINAL_INT8_TOPS = 4500.0      # NVIDIA's dense INT8 figure for B200 (context only)
INT8_OVER_BF16 = 2.0            # nominal dense ratio 4.5 / 2.25 PFLOP/s


def measured_peaks():
    """(int8 burst TOP/s, int8 sustained TOP/s, HBM GB/s, label).  Dense int8 = 2 x the measured
    bf16 rate (nominal ratio 4.5 : 2.25); burst = a kernel timed at full clocks, sustained = inside
    a long power-capped loop."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return (INT8_OVER_BF16 * float(m["bf16_tflops"]), INT8_OVER_BF16 * float(m["bf16_tflops_sustained"]),
                float(m["hbm_gbs"]), "measured")
    return INT8_OVER_BF16 * 1590.0, INT8_OVER_BF16 * 1400.0, 6650.0, "fallback"


def tensor_roofline(tops: float, clocks: dict, issue_tops: float) -> dict:
    """Fractions of every int8 peak in use, and which measured one applies to this run: the burst
    figure when the median SM clock under load stayed within 5 % of its maximum (the condition that
    figure was measured under), else the sustained one (measured at about 1.35 GHz under the power cap)."""
    burst, sustained, _, kind = measured_peaks()
    held = bool(clocks.get("sm_mhz")) and bool(clocks.get("sm_max_mhz")) and clocks["sm_mhz"] >= 0.95 * clocks["sm_max_mhz"]
    peak = burst if held else sustained
    return {"bound": "tensor", "achieved": tops, "peak": peak, "unit": "TOP/s", "frac": tops / peak,
            "peak_kind": "%s 2 x bf16 %s (of %s)" % (kind, "burst: the median SM clock stayed within 5 % of its maximum" if held else "sustained: the SM clock fell under the power cap", kind),
            "frac_of_burst": tops / burst, "frac_of_sustained": tops / sustained, "peak_burst": burst, "peak_sustained": sustained,
            "frac_of_nominal_4500": tops / NOMINAL_INT8_TOPS, "issue_rate_peak": issue_tops,
            "frac_of_issue_rate_peak": tops / issue_tops if issue_tops else None}


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


def probe_mma_rate_rows(block_n: int, row_bytes: int, a_group_stride: int, iters: int = 50000):
    """The same probe with operand rows of row_bytes (32 / 64 / 128, the swizzle width) and A's 8-row groups
    a_group_stride bytes apart: the operand forms of narrow layers and of the window kernel's block tiling."""
    import ctypes as C
    from paper_2006_11735_b200 import build as lib_build
    lib = C.CDLL(lib_build.PROBE_LIB)
    lib.probe_mma_rate_rows.argtypes = [C.c_int32] * 4 + [C.POINTER(C.c_double)] * 2
    lib.probe_mma_rate_rows.restype = C.c_int
    tops, cyc = C.c_double(), C.c_double()
    rc = lib.probe_mma_rate_rows(block_n, row_bytes, a_group_stride, iters, C.byref(tops), C.byref(cyc))
    if rc != 0:
        raise RuntimeError("probe_mma_rate_rows failed with status %d" % rc)
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


def time_network(g, x_dev, steps, stream, sampler_index):
    """Exactly K forwards between two events (nothing else on the stream, so consecutive kernels
    overlap their set-up with the tail of the one before, as in deployment), then a second pass of
    up to 20 forwards with one event after every layer for the per-kernel durations (an event
    between two kernels keeps the second from starting early, so that pass is a little slower and
    is not the reported step time).  Returns (ms of the K steps, marks, steps of the marks pass, clocks)."""
    import torch
    sampler = ClockSampler(sampler_index)
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record(stream)
    for _ in range(steps):
        g.forward(x_dev)
    e1.record(stream)
    torch.cuda.synchronize()
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    all_marks = []
    for _ in range(min(steps, 20)):
        marks = []
        g.forward(x_dev, marks=marks)
        all_marks.append(marks)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1), all_marks, len(all_marks), clocks


def layer_table(g, net, all_marks, steps, kernels, macs, abytes, int8_peak, hbm_peak):
    """Per layer: time, TOP/s, GB/s, percent of each peak and the bound that binds it (the larger of
    the time at the int8 peak and the time at the copy bandwidth)."""
    layer_ms = {}
    for marks in all_marks:
        for (_, prev), (name, ev) in zip(marks[:-1], marks[1:]):
            layer_ms[name] = layer_ms.get(name, 0.0) + prev.elapsed_time(ev) / steps
    rows = []
    for op in net.ops:
        if op.name not in layer_ms:
            continue
        t = layer_ms[op.name]
        ops = 2.0 * macs.get(op.name, 0)
        b = abytes.get(op.name, 0)
        t_tensor, t_hbm = ops / (int8_peak * 1e12) * 1e3, b / (hbm_peak * 1e9) * 1e3
        rows.append({"layer": op.name, "kernel": kernels.get(op.name, "pool"), "ms": round(t, 5),
                     "tops": round(ops / (t * 1e-3) / 1e12, 2) if t > 0 else None,
                     "gbs": round(b / (t * 1e-3) / 1e9, 1) if t > 0 else None,
                     "pct_int8_peak": round(100.0 * t_tensor / t, 1) if t > 0 else None,
                     "pct_hbm_peak": round(100.0 * t_hbm / t, 1) if t > 0 else None,
                     "bound": "tensor" if t_tensor >= t_hbm else "hbm",
                     "roofline_frac": round(max(t_tensor, t_hbm) / t, 3) if t > 0 else None})
    return rows, layer_ms


def family_sums(all_marks, kernels, macs, abytes):
    fam_ms, fam_macs, fam_bytes = {}, {}, {}
    for marks in all_marks:
        for (_, prev), (name, ev) in zip(marks[:-1], marks[1:]):
            fam = kernels.get(name, "pool")
            fam_ms[fam] = fam_ms.get(fam, 0.0) + prev.elapsed_time(ev)
            fam_macs[fam] = fam_macs.get(fam, 0) + macs.get(name, 0)
            fam_bytes[fam] = fam_bytes.get(fam, 0) + abytes.get(name, 0)
    return fam_ms, fam_macs, fam_bytes


def elementwise_kernels(dev, hbm_peak, peak_kind, iters_default=10):
    """The bandwidth-bound kernels, each timed alone through the C ABI on tensors of the paper's
    shapes: CUDA events around every call, a 256 MB write between calls so that nothing is served
    from L2.  Algorithmic bytes = every input and output once."""
    import numpy as np
    import torch
    from paper_2006_11735_b200 import binding as B
    st = torch.cuda.current_stream(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    rng = np.random.default_rng(7)
    out = {}

    def timed(name, nbytes, fn, iters=None):
        iters = iters or iters_default
        for _ in range(3):
            fn()
        ms = 0.0
        for _ in range(iters):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            fn()
            e1.record(st)
            torch.cuda.synchronize(dev)
            ms += e0.elapsed_time(e1)
        ms /= iters
        gbs = nbytes / (ms * 1e-3) / 1e9
        out[name] = {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak, "ms": ms,
                     "algorithmic_bytes": int(nbytes), "peak_kind": peak_kind + " copy bandwidth", "traffic": None}

    def u8(*shape):
        return torch.randint(0, 256, shape, dtype=torch.uint8, device=dev)

    # stand-alone add with ratio synchronisation: two 205 MB activations (stage 1 of the ResNet-50 batch)
    n = 256 * 56 * 56 * 256
    a, b, o = u8(n), u8(n), torch.empty(n, dtype=torch.uint8, device=dev)
    timed("add_requant_kernel", 3 * n, lambda: B.iadd_requant(a.data_ptr(), b.data_ptr(), o.data_ptr(), st.cuda_stream, n_elems=n, a_dtype=B.U8,
                                                              b_dtype=B.U8, out_dtype=B.U8, a_zero=0, b_zero=0, mul_a=3, sh_a=1, mul_b=5, sh_b=2,
                                                              brelu=1, h_i=400, mul=160, shift=8, out_zero=0, out_lo=0, out_hi=255))
    del a, b, o
    # 3x3 / 2 max-pool of the stem output, global average of the last stage
    x = u8(256, 112, 112, 64)
    o = torch.empty((256, 56, 56, 64), dtype=torch.uint8, device=dev)
    timed("maxpool_3x3s2_kernel", x.numel() + o.numel(), lambda: B.ipool_max(x.data_ptr(), o.data_ptr(), 256, 112, 112, 64, 3, 2, 1, st.cuda_stream))
    x = u8(256, 7, 7, 2048)
    o = torch.empty((256, 1, 1, 2048), dtype=torch.uint8, device=dev)
    timed("avgpool16_kernel", x.numel() + o.numel(), lambda: B.ipool_avg_requant(x.data_ptr(), o.data_ptr(), 256, 7, 7, 2048, 1337, 16, 255, st.cuda_stream))
    # the thin layers of the VDSR shape on the CUDA-core kernels (forced; the plan prefers the tensor cores)
    W = rng.integers(-127, 128, size=(64, 3, 3, 1), dtype=np.int8)
    plan = B.iconv_plan(n=16, h=256, w=256, c_in=1, c_out=64, kh=3, kw=3, pad=1, in_dtype=B.U8_RAW128, weights=W,
                        bias=np.zeros(64, np.int32), mul=[200], shift=[16], h_i=[80000], kernel=B.KERNEL_THIN)
    x = u8(16, 256, 256, 1)
    o = torch.empty((16, 256, 256, 64), dtype=torch.uint8, device=dev)
    timed("thin_in_kernel", x.numel() + o.numel(), lambda: B.iconv_forward(plan, x.data_ptr(), None, o.data_ptr(), None, st.cuda_stream))
    B.iconv_plan_destroy(plan)
    W = rng.integers(-127, 128, size=(1, 3, 3, 64), dtype=np.int8)
    plan = B.iconv_plan(n=16, h=256, w=256, c_in=64, c_out=1, kh=3, kw=3, pad=1, weights=W, bias=np.zeros(1, np.int32), mul=[200], shift=[16],
                        h_i=[0], brelu=0, out_zero=128, skip_dtype=B.U8_RAW128, skip_c_total=1, skip_mul=3, skip_shift=1, kernel=B.KERNEL_THIN)
    x = u8(16, 256, 256, 64)
    sk = u8(16, 256, 256, 1)
    o = torch.empty((16, 256, 256, 1), dtype=torch.uint8, device=dev)
    timed("thin_out_kernel", x.numel() + sk.numel() + o.numel(), lambda: B.iconv_forward(plan, x.data_ptr(), sk.data_ptr(), o.data_ptr(), None, st.cuda_stream))
    B.iconv_plan_destroy(plan)
    # the n-sigma bound of a 256 MB int32 feature map: four passes over the data
    y = torch.randint(-200000, 200000, (64 << 20,), dtype=torch.int32, device=dev)
    timed("select_hist_kernel (iq_sigma_bound, 4 passes)", 4 * y.numel() * 4, lambda: B.iq_sigma_bound(y.data_ptr(), y.numel(), 0.0015, st.cuda_stream), iters=max(1, iters_default // 2))
    del y, flush
    torch.cuda.empty_cache()
    return out


def bench_network(name, args, dev, local_rank, rank, size, with_e2e=True):
    """Times one workload; returns the dict of its figures (the caller prints the line)."""
    import torch
    from paper_2006_11735_b200 import binding as B
    from paper_2006_11735_b200 import dist as D
    from paper_2006_11735_b200.network import Network, net_input
    from workloads import networks as N
    from workloads.params import load_params

    metric, full_name = WORKLOADS[name]
    full = N.by_name(name)
    net = N.by_name(name, n=args.batch) if args.batch > 0 else full       # the full batch per GPU (weak scaling)
    workload = full_name if net.n == full.n else "%s with batch %d (reduced batch: profiling only)" % (full_name, net.n)
    strips = None
    if args.row_shard:
        # one picture over the ranks: every rank convolves the strip it owns (plus the halo)
        from paper_2006_11735_b200 import rowshard as RS
        t_in = full.tensors[full.input]
        strips = RS.partition(t_in.h, size, RS.halo_rows(full))
        net = N.by_name(name, h=max(1, strips[rank].rows), w=t_in.w)
        workload = "%s, rows sharded over %d ranks with a halo of %d rows" % (full_name, size, RS.halo_rows(full))
    params = load_params(name)
    g = Network(net, params, device=dev)
    if strips is not None:
        x_np = net_input(full)[:, strips[rank].in0:strips[rank].in1]
    else:
        x_np = net_input(net)
    x_host = torch.from_numpy(x_np.copy()).pin_memory()
    x_dev = x_host.to(dev, non_blocking=True)
    t_out = net.tensors[net.output]
    out_host = torch.empty((net.n, t_out.h, t_out.w, t_out.c), dtype=torch.int32 if t_out.dtype == "i32" else torch.uint8).pin_memory()
    stream = torch.cuda.current_stream(dev)
    kernels, macs, abytes = g.kernels(), g.conv_macs(), g.algorithmic_bytes()

    for _ in range(args.warmup):
        g.forward(x_dev)
    B.iconv_check(stream.cuda_stream)

    D.barrier()
    torch.cuda.synchronize(dev)
    ms_local, all_marks, mark_steps, clocks = time_network(g, x_dev, args.steps, stream, local_rank)
    D.barrier()
    ms = D.max_over_ranks(ms_local, dev)
    B.iconv_check(stream.cuda_stream)
    # the repacked first layers are two launches (repack + GEMM), every other step one
    launches = (len(g.steps) + sum(1 for k in kernels.values() if k == "stem")) * args.steps

    burst, sustained, hbm_peak, peak_kind = measured_peaks()
    fam_ms, fam_macs, fam_bytes = family_sums(all_marks, kernels, macs, abytes)
    issue_tops, _ = probe_mma_rate(256, 100000)             # outside every timed region
    issue64_tops, issue64_cycles = probe_mma_rate_rows(64, 64, 512, 50000)
    umma_launches = sum(1 for k in kernels.values() if k == "umma") * mark_steps
    umma_tops = 2.0 * fam_macs.get("umma", 0) / (fam_ms.get("umma", 1e-9) * 1e-3) / 1e12
    traffic = None     # the aggregate over several kernels has no single capture behind it: see roofline_dominant
    roofline = tensor_roofline(umma_tops, clocks, issue_tops)
    # what a stream of N = 64 instructions reaches (layers with at most 64 output channels): an instruction with
    # N <= 64 occupies the pipe about as long as one with N = 128
    roofline.update({"issue_rate_peak_n64": issue64_tops, "cycles_per_instruction_n64": issue64_cycles})
    roofline.update({"kernel": "umma_conv_kernel + umma_window_kernel", "traffic": traffic, "launches": umma_launches,
                     "avg_launch_ms": fam_ms.get("umma", 0.0) / max(1, umma_launches),
                     "time_share": {k: v / sum(fam_ms.values()) for k, v in fam_ms.items()}})
    umma_gbs = fam_bytes.get("umma", 0) / (fam_ms.get("umma", 1e-9) * 1e-3) / 1e9
    roofline_hbm = {"kernel": "umma_conv_kernel + umma_window_kernel", "bound": "hbm", "achieved": umma_gbs, "peak": hbm_peak,
                    "unit": "GB/s", "frac": umma_gbs / hbm_peak, "traffic": traffic,
                    "algorithmic_bytes_per_launch": fam_bytes.get("umma", 0) / max(1, umma_launches), "peak_kind": peak_kind + " copy bandwidth",
                    "algorithmic_bytes_per_step": int(sum(abytes.values())),
                    "whole_step_gbs": sum(abytes.values()) / (ms / args.steps * 1e-3) / 1e9,
                    "whole_step_frac": sum(abytes.values()) / (ms / args.steps * 1e-3) / 1e9 / hbm_peak}
    table, layer_ms = layer_table(g, net, all_marks, mark_steps, kernels, macs, abytes, roofline["peak"], hbm_peak)
    # the kernel with the largest share of the step, by itself against the roofline that binds it
    groups = {}
    for row in table:
        desc = g.describe().get(row["layer"], "")
        kname = ("umma_chain_kernel" if "chain" in desc else "umma_window_kernel" if "window" in desc else
                 "umma_conv_kernel (cta pairs)" if "cta pairs" in desc else "umma_conv_kernel" if row["kernel"] == "umma" else row["kernel"])
        gr = groups.setdefault(kname, {"ms": 0.0, "bytes": 0, "ops": 0.0, "launches": 0})
        gr["ms"] += row["ms"]; gr["bytes"] += abytes.get(row["layer"], 0); gr["ops"] += 2.0 * macs.get(row["layer"], 0); gr["launches"] += 1
    dom = max(groups, key=lambda k: groups[k]["ms"])
    gd = groups[dom]
    t_tensor, t_hbm = gd["ops"] / (roofline["peak"] * 1e12) * 1e3, gd["bytes"] / (hbm_peak * 1e9) * 1e3
    dom_traffic = None
    if name in DRAM_TRAFFIC and net.n == full.n and DRAM_TRAFFIC[name][1] == dom:
        import hashlib
        with open(os.path.join(ROOT, "paper_2006_11735_b200", "csrc", DRAM_TRAFFIC[name][3]), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() == DRAM_TRAFFIC[name][2]:
                dom_traffic = DRAM_TRAFFIC[name][0]
    if t_hbm >= t_tensor:
        dominant = {"kernel": dom, "bound": "hbm", "achieved": gd["bytes"] / (gd["ms"] * 1e-3) / 1e9, "peak": hbm_peak, "unit": "GB/s",
                    "frac": t_hbm / gd["ms"], "traffic": dom_traffic, "peak_kind": peak_kind + " copy bandwidth"}
    else:
        dominant = {"kernel": dom, "bound": "tensor", "achieved": gd["ops"] / (gd["ms"] * 1e-3) / 1e12, "peak": roofline["peak"], "unit": "TOP/s",
                    "frac": t_tensor / gd["ms"], "traffic": dom_traffic, "peak_kind": roofline["peak_kind"]}
    dominant.update({"launches_per_step": gd["launches"], "avg_launch_ms": gd["ms"] / gd["launches"],
                     "algorithmic_bytes_per_launch": gd["bytes"] / gd["launches"], "share_of_step": gd["ms"] / sum(v["ms"] for v in groups.values()),
                     "shares": {k: round(v["ms"] / sum(x["ms"] for x in groups.values()), 4) for k, v in groups.items()}})

    res = {"metric": metric, "workload": workload, "net": net, "ms": ms, "clocks": clocks, "launches": launches, "roofline": roofline,
           "roofline_dominant": dominant,
           "roofline_hbm": roofline_hbm, "per_layer": table, "macs": macs, "abytes": abytes, "kernels": kernels, "described": g.describe(),
           "layer_ms": layer_ms, "images": (1 if strips is not None else net.n * size) * args.steps, "e2e": None,
           "scaling": "strong" if strips is not None else "weak"}

    if with_e2e:
        # ---- end to end: pinned host input in, result out, every step ----
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
            out_host.copy_(out, non_blocking=True)
        e3.record(stream)
        torch.cuda.synchronize(dev)
        ms_e2e = D.max_over_ranks(e2.elapsed_time(e3), dev)
        B.iconv_check(stream.cuda_stream)
        res["e2e"] = {"value": res["images"] / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(x_host.numel()),
                      "d2h_bytes_per_step": int(out_host.numel() * out_host.element_size()),
                      "overlap": "the input copy of step i+1 runs under the compute of step i (two device buffers, one copy stream)"}
    g.close()
    del g
    torch.cuda.empty_cache()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the VDSR leg and the element-wise kernels (profiler captures)")
    ap.add_argument("--elementwise-iters", type=int, default=10, help="timed calls per element-wise kernel (1 for profiler captures)")
    ap.add_argument("--per-layer", action="store_true", help="also print the per-layer table to stderr")
    ap.add_argument("--workload", default="resnet50", choices=sorted(WORKLOADS))
    ap.add_argument("--row-shard", action="store_true",
                    help="one picture (vrcnn_hd, vdsr_hd) with its rows sharded over the ranks instead of one batch per rank")
    ap.add_argument("--batch", type=int, default=0,
                    help="images per GPU; 0 = the full workload. Smaller batches are for profiler captures only and are "
                         "named in config.workload")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    import torch

    from paper_2006_11735_b200 import binding as B          # noqa: F401  (raises if the CUDA library is missing)
    from paper_2006_11735_b200 import dist as D

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    rank, local_rank, size = D.world()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    D.init("nccl")
    if args.row_shard and args.workload not in ("vrcnn_hd", "vdsr_hd"):
        raise SystemExit("--row-shard applies to the single-picture workloads (vrcnn_hd, vdsr_hd)")

    r = bench_network(args.workload, args, dev, local_rank, rank, size)
    ms, net = r["ms"], r["net"]
    extras = rank == 0 and size == 1 and not args.no_extras and args.batch == 0 and args.workload == "resnet50"
    vdsr = elementwise = None
    if extras:
        v = bench_network("vdsr", args, dev, local_rank, rank, size)
        vdsr = {"metric": v["metric"], "value": v["images"] / (v["ms"] * 1e-3), "unit": UNIT, "ms_per_step": v["ms"] / args.steps,
                "workload": v["workload"], "clocks": v["clocks"], "e2e": v["e2e"], "roofline": v["roofline"], "roofline_hbm": v["roofline_hbm"],
                "roofline_dominant": v["roofline_dominant"],
                "int8_tops_whole_step": 2.0 * sum(v["macs"].values()) / (v["ms"] / args.steps * 1e-3) / 1e12, "per_layer": v["per_layer"]}
        _, _, hbm_peak, peak_kind = measured_peaks()
        elementwise = elementwise_kernels(dev, hbm_peak, peak_kind, args.elementwise_iters)
        # the repacked stem (repack kernel + GEMM) as one step of the timed forward
        stem_ms = r["layer_ms"].get("stem")
        if stem_ms and r["kernels"].get("stem") == "stem":
            t = net.tensors
            scratch = net.n * (t["stem"].h + 3) * (t["stem"].w + 3) * 16
            nbytes = net.n * t["x0"].h * t["x0"].w * 3 + 2 * scratch + net.n * t["stem"].h * t["stem"].w * t["stem"].c
            elementwise["stem_repack_kernel + umma_window_kernel (7x7/2 stem)"] = {
                "bound": "hbm", "achieved": nbytes / (stem_ms * 1e-3) / 1e9, "peak": hbm_peak, "unit": "GB/s",
                "frac": nbytes / (stem_ms * 1e-3) / 1e9 / hbm_peak, "ms": stem_ms, "algorithmic_bytes": int(nbytes),
                "peak_kind": peak_kind + " copy bandwidth", "traffic": None,
                "note": "image in, repacked copy written and read once, activations out"}

    if args.per_layer and rank == 0:
        for row in r["per_layer"]:
            sys.stderr.write("%-14s %-6s %8.4f ms %8.1f TOP/s %8.1f GB/s  %5.1f %% int8  %5.1f %% hbm  %-6s %s\n" % (
                row["layer"], row["kernel"], row["ms"], row["tops"] or 0.0, row["gbs"] or 0.0, row["pct_int8_peak"] or 0.0,
                row["pct_hbm_peak"] or 0.0, row["bound"], r["described"].get(row["layer"], "")))

    cpu = None
    if rank == 0 and size == 1 and not args.no_cpu_baseline and args.workload == "resnet50":
        n_s = 8
        v, dt = oracle_images_per_s(n_s)
        cpu = {"value": v, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
               "sample": "%d images of the same batch, one forward, %.1f s" % (n_s, dt)}

    if rank == 0:
        abytes, macs = r["abytes"], r["macs"]
        line = {"metric": r["metric"], "value": r["images"] / (ms * 1e-3), "unit": UNIT, "n_gpus": size,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
                "scaling": r["scaling"], "vs_baseline": None, "dtype": "int8", "data": "synthetic",
                "config": {"workload": r["workload"], "global_batch": net.n * size if r["scaling"] == "weak" else net.n,
                           "parallelism": ("dp%d" if r["scaling"] == "weak" else "rows%d") % size,
                           "l2": "per-step algorithmic traffic (%.1f GB) far exceeds the 126 MB L2" % (sum(abytes.values()) / 1e9),
                           "timing_note": "value: exactly K forwards between two CUDA events; the per-kernel durations of `roofline`, "
                                          "`roofline_hbm` and `per_layer` come from a second pass with one event after every layer",
                           "int8_tops_whole_step": 2.0 * sum(macs.values()) / (ms / args.steps * 1e-3) / 1e12},
                "clocks": r["clocks"], "e2e": r["e2e"], "gpu_launches": r["launches"], "roofline": r["roofline"],
                "roofline_hbm": r["roofline_hbm"], "roofline_dominant": r["roofline_dominant"], "cpu_baseline": cpu, "per_layer": r["per_layer"], "elementwise": elementwise, "vdsr": vdsr}
        print(json.dumps(line))
    D.finish()


if __name__ == "__main__":
    main()
