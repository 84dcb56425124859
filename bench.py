#!/usr/bin/env python
"""Benchmark of the binarised-DNN forward pass on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config wsj]

One step = one whole forward pass (every layer, through one bnn_forward call of the C ABI)
over one batch of seeded synthetic frames.  Prints ONE JSON line on rank 0.
With --impl reference the plain CPU oracle is timed instead (a slow, obviously correct
program: a reported baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "frames/sec for 6x2048 binarized DNN forward on 1 B200; XNOR-GEMM binary-op/s vs roofline"
UNIT = "frames/s"
L2_BYTES = 126 * 1024 * 1024
SMS = 148


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="wsj", choices=["tiny", "wsj", "wsj_bw", "ami", "wsj_mixed"])
    ap.add_argument("--frames", type=int, default=None, help="override the batch size (frames per step)")
    ap.add_argument("--cpu-frames", type=int, default=16384, help="frames of the workload the CPU oracle is timed on")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--xnor-prepared", default="auto", choices=["auto", "stream", "resident"],
                    help="kernel for hidden layers with prepared weights (see BNN_OPT_XNOR_PREPARED)")
    ap.add_argument("--act-values", default="pm1", choices=["pm1", "01"],
                    help="what the binary activations stand for: (-1,+1) or (0,1)")
    ap.add_argument("--splice", action="store_true",
                    help="feed one 40-dim frame per row and let the first layer form the context window "
                         "(11 or 15 frames) instead of reading an already spliced input")
    ap.add_argument("--no-stack", action="store_true",
                    help="one launch per binary hidden layer instead of one launch for the run of equal layers")
    ap.add_argument("--no-follow", action="store_true",
                    help="run the log-softmax after the top layer's kernel instead of behind it (overlapped)")
    ap.add_argument("--no-graph", action="store_true",
                    help="launch every step's kernels from the host instead of replaying a captured CUDA graph")
    ap.add_argument("--sweep", action="store_true",
                    help="isolated XNOR GEMM sweep (M x K x N x bit density), one JSON line per point")
    ap.add_argument("--sweep-quick", action="store_true", help="only the corner points of the sweep")
    ap.add_argument("--pipe-rates", action="store_true",
                    help="measure the rates of the pipes that bound the kernels (popc, lop3, iadd, fadd, ffma, "
                         "4-bit and fp16 tensor-core MMA, L2 reads); one JSON line per pipe")
    ap.add_argument("--real-path", default="tensor", choices=["tensor", "fp32"],
                    help="kernel of the real-valued layers: tcgen05 with split operands or the FP32 pipe")
    ap.add_argument("--xnor-path", default="tensor", choices=["tensor", "tensor-unprepared", "popc"],
                    help="kernel of the binary hidden layers: tcgen05 tensor core or integer-pipe popcount")
    return ap.parse_args()


def workload_name(cfg, frames):
    return "%s: %d frames x %d -> %d x %d -> %d log-softmax, %s" % (
        cfg.name, frames, cfg.in_dim, cfg.n_hidden, cfg.hidden, cfg.classes,
        "binary weights+activations" if cfg.act == 1 else "binary weights, hardtanh activations")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    sm_max_mhz=p.get("sm_max_mhz", 1965.0), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, sm_max_mhz=1965.0,
                source="fallback")


# ------------------------------------------------------------------ CPU oracle arm
def oracle_step(cfg, net, X):
    from oracle import bnn_oracle as o
    if getattr(cfg, "mixed", False):
        return o.forward_mixed(X, net.W, net.scale, net.shift, net.Wout, net.bout, o.SIGN_ZERO_POS)
    return o.forward(X, net.W, net.scale, net.shift, net.Wout, net.bout,
                     o.ACT_SIGN if cfg.act == 1 else o.ACT_HARDTANH, o.SIGN_ZERO_POS)


def run_reference(args):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import bnn_oracle as o
    from paper_1706_09453_b200 import workloads as wl
    cfg = wl.CONFIGS[args.config]
    frames = args.frames or cfg.frames
    sample = min(frames, 256)       # frames per step: ~1.2 s of CPU work at WSJ scale on 8 cores
    net = wl.make_model(cfg)
    X = wl.make_frames(cfg, sample)
    steps, warmup = max(1, min(args.steps, 40)), max(1, min(args.warmup, 3))
    for _ in range(warmup):
        oracle_step(cfg, net, X)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(cfg, net, X)
    dt = time.perf_counter() - t0
    fps = sample * steps / dt
    desc = "first %d frames of the batch per step, %d steps" % (sample, steps)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": fps, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt / steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg, frames), "sample": desc},
        "cpu_baseline": {"value": fps, "unit": UNIT, "cores": o.num_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": fps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, torch, device_index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = torch.cuda.get_device_properties(device_index).uuid
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-%s" % uuid).encode())
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # NVML missing: report that, do not guess
            self.nv, self.err = None, repr(e)

    def _loop(self):
        nv = self.nv
        # NVML clocks-event (throttle) reason bits
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                 0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self.nv:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread:
            self._stop.set()
            self._thread.join()

    def summary(self):
        if not self.nv:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "error": self.err}
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": float(self.max_mhz), "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------ roofline bookkeeping
def xnor_kernel_name(k, xnor_path, prepared, stacked=True):
    """The kernel bnn_forward runs for a binary hidden layer of fan-in k (see bnn_api.cu); `stacked`: the
    layer is one of a run of equal layers that goes out as one launch."""
    if xnor_path == "popc":
        return "xnor_popc_kernel"
    if xnor_path == "tensor-unprepared":
        return "xnor_tc_kernel"
    if prepared == "stream":
        return "xnor_img_kernel"
    if k <= 2048 or (k <= 3072 and (prepared == "resident" or stacked)):
        return "xnor_res_kernel"
    return "xnor_tc_kernel"


def choose_tensor_regime(peaks, clocks, timed_s):
    """Which measured bf16 figure applies to this run: the burst figure when the SM clock sampled
    under load stayed at (or within 5 % of) its maximum or the timed region is shorter than a
    second; the sustained figure when the samples show the power-capped regime."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz") or peaks["sm_max_mhz"]
    if mhz is not None and mhz < 0.95 * mx and timed_s >= 1.0:
        return "sustained", peaks["bf16_tflops_sustained"], "median SM clock %.0f of %.0f MHz over a %.2f s timed region" % (mhz, mx, timed_s)
    why = "timed region %.3f s" % timed_s if timed_s < 1.0 else "median SM clock %.0f of %.0f MHz" % (mhz or -1, mx)
    return "burst", peaks["bf16_tflops"], why


def layer_table(cfg, frames, peaks, sm_mhz, xnor_path="tensor", real_path="tensor", prepared="auto", stacked=True):
    """Per layer: algorithmic work, the pipe that bounds the kernel and its peak.

    peaks["bf16"] is the bf16 figure chosen for this run (burst or sustained); peaks["mxf4"] the
    rate of a bare kind::mxf4 MMA loop measured in this process (falls back to 4 x bf16).

    Algorithmic work: 2 binary ops per bit-MAC for XNOR layers, 2 flop per add/sub or MAC for
    the real-valued layers.  Peaks of the integer / FP32 pipes are derived from unit counts:
    per SM and clock 16 popcount lanes (x 32 bits x 2 bop) and 128 FP32 FMA lanes (x 2 flop),
    at the maximum SM clock.
    """
    clk = peaks["sm_max_mhz"] * 1e6
    popc_peak = SMS * 16 * 32 * 2 * clk / 1e12      # Tbop/s on the popcount pipe
    fp32_peak = SMS * 128 * 2 * clk / 1e12          # TFLOP/s on the FP32 pipe
    rows = []
    k = cfg.in_dim
    mixed = getattr(cfg, "mixed", False)
    for l in range(cfg.n_hidden):
        xnor = cfg.act == 1 and l > (1 if mixed else 0)
        work = 2.0 * frames * cfg.hidden * k
        if mixed and l == 0:
            # real-valued Sigmoid layer: both operands in two fp16 terms, three MMAs per step
            if real_path == "tensor":
                rows.append(dict(name="real_1", kernel="h_split_kernel+outf_tc_kernel", work=work, unit="TFLOP/s",
                                 bound="tensor", peak=peaks["bf16"], passes=3))
            else:
                rows.append(dict(name="real_1", kernel="real_gemm_kernel", work=work, unit="TFLOP/s", bound="alu",
                                 peak=fp32_peak))
        elif xnor and mixed and l == cfg.n_hidden - 1 and xnor_path != "popc":
            # binary layer with Sigmoid units: int32 dot products, then one pass that applies the Sigmoid and
            # writes the top layer's fp16 activation image
            rows.append(dict(name="xnor_%d" % (l + 1), kernel="xnor_tc_kernel+h_split_kernel", work=work,
                             unit="Tbop/s", bound="tensor", peak=peaks["mxf4"], peak_nominal_ratio=4.0 * peaks["bf16"]))
        elif xnor and xnor_path in ("tensor", "tensor-unprepared"):
            # 4-bit (e2m1, kind::mxf4) tensor-core MACs, 1 bit-MAC = 2 bop.  Peak: the rate of a bare
            # kind::mxf4 MMA loop measured in this process (the stricter denominator); beside it the
            # figure 4 x bf16 (nominal ratio 9 : 2.25 PFLOP/s applied to the measured bf16 peak).
            # smem_bytes: what the kernel moves through the SM's shared
            # memory per launch (per bit of the unit operand and tile visit 4 bits stored + 4 bits
            # read by the tensor core; the packed bits of both operands staged by TMA and read
            # back once; the widened frame operand goes to tensor memory instead).
            tiles_m, tiles_n = -(-frames // 128), -(-cfg.hidden // 192)
            kpad = -(-k // 256) * 256
            smem_bytes = tiles_m * tiles_n * kpad * (192 * (0.5 + 0.5 + 0.125 + 0.125) + 128 * (0.125 + 0.125))
            kern = xnor_kernel_name(k, xnor_path, prepared, stacked and cfg.n_hidden > 2)
            if kern == "xnor_img_kernel":
                # weights prepared once: their widened image arrives by bulk copies (4 bits written,
                # 4 bits read by the tensor core per weight bit and tile visit); nothing else
                smem_bytes = tiles_m * tiles_n * kpad * (192 * (0.5 + 0.5) + 128 * (0.125 + 0.125))
            elif kern == "xnor_res_kernel":
                # weights resident: written once per CTA, read by the tensor core on every tile visit
                bn = 192 if k <= 2048 else 128
                tiles_n = -(-cfg.hidden // bn)
                smem_bytes = tiles_m * tiles_n * kpad * (bn * 0.5 + 128 * (0.125 + 0.125)) + SMS * kpad * bn * 0.5
            rows.append(dict(name="xnor_%d" % (l + 1), kernel=kern, work=work, unit="Tbop/s",
                             bound="tensor", peak=peaks["mxf4"], peak_nominal_ratio=4.0 * peaks["bf16"],
                             smem_bytes=smem_bytes))
        elif xnor:
            rows.append(dict(name="xnor_%d" % (l + 1), kernel="xnor_popc_kernel", work=work, unit="Tbop/s",
                             bound="alu", peak=popc_peak))
        elif real_path == "tensor":
            # bf16 tensor-core MMAs, one pass per bf16 term of the real operand (2 terms);
            # algorithmic flops count the product once
            # (a sign-weight layer fed by another one finds its split-activation image written by that
            # layer's epilogue: no split launch of its own)
            chained = l > 0 and not mixed
            rows.append(dict(name="signw_%d" % (l + 1), kernel="signw_img_kernel" if chained else "x_split_kernel+signw_img_kernel",
                             work=work, unit="TFLOP/s", bound="tensor", peak=peaks["bf16"], passes=2))
        else:
            rows.append(dict(name="signw_%d" % (l + 1), kernel="real_gemm_kernel", work=work, unit="TFLOP/s",
                             bound="alu", peak=fp32_peak))
        k = cfg.hidden
    owork = 2.0 * frames * cfg.classes * cfg.hidden
    if real_path == "tensor" and cfg.act == 1 and not mixed:
        rows.append(dict(name="output_gemm", kernel="out_tc_kernel", work=owork, unit="TFLOP/s", bound="tensor",
                         peak=peaks["bf16"], passes=2))
    elif real_path == "tensor":
        # fp32 activations: both operands in two fp16 terms, three MMAs per step
        # (its fp16 activation image comes from the epilogue of the layer before: no split launch)
        rows.append(dict(name="output_gemm", kernel="outf_tc_kernel", work=owork, unit="TFLOP/s",
                         bound="tensor", peak=peaks["bf16"], passes=3))
    else:
        rows.append(dict(name="output_gemm", kernel="real_gemm_kernel", work=owork, unit="TFLOP/s", bound="alu",
                         peak=fp32_peak))
    if frames <= 16 and cfg.act == 1 and not mixed and xnor_path != "popc":
        # a handful of frames: bnn_forward runs the matrix-vector kernels (one warp per unit), which
        # are bound by reading each layer's weights once
        for r in rows:
            if r["name"].startswith("signw"):
                r.update(kernel="small_signw_kernel", bound="alu", peak=fp32_peak, passes=1)
            elif r["name"].startswith("xnor"):
                r.update(kernel="small_xnor_kernel", bound="alu", peak=popc_peak)
                r.pop("smem_bytes", None)
            elif r["name"] == "output_gemm":
                r.update(kernel="small_out_kernel", bound="hbm", unit="GB/s", peak=peaks["hbm_gbs"], scale=1e9, passes=1,
                         work=4.0 * cfg.classes * cfg.hidden + 4.0 * frames * cfg.classes)
    # log-softmax: one read and one write of the [frames][classes] fp32 matrix
    rows.append(dict(name="log_softmax", kernel="log_softmax_rows_reg_kernel", work=2.0 * frames * cfg.classes * 4,
                     unit="GB/s", bound="hbm", peak=peaks["hbm_gbs"], scale=1e9))
    return rows


def hbm_bytes_per_step(cfg, frames):
    """Algorithmic HBM bytes of one forward: input, log-probs, weights once, activations."""
    from paper_1706_09453_b200 import workloads as wl
    b = frames * cfg.in_dim * 4 + frames * cfg.classes * 4
    k = cfg.in_dim
    for _ in range(cfg.n_hidden):
        b += cfg.hidden * ((k + 31) // 32) * 4
        b += 2 * frames * (cfg.hidden // 8 if cfg.act == wl.ACT_SIGN else cfg.hidden * 4)
        k = cfg.hidden
    b += cfg.classes * cfg.hidden * 4 + cfg.classes * 4
    return b


def ncu_traffic(kernel, workload):
    """DRAM bytes (read + write) per launch of `kernel` from the committed ncu capture, or None when
    there is none for this workload's shapes or the kernel's source has changed since it was taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None
    table = json.load(open(path))
    total = 0.0
    for part in kernel.split("+"):      # a row of two launches (split + GEMM): the sum of both
        rec = table.get(part)
        if not rec or workload not in rec.get("workloads", []):
            return None
        src = os.path.join(ROOT, "paper_1706_09453_b200", "csrc", rec["source"])
        if not os.path.exists(src) or hashlib.sha256(open(src, "rb").read()).hexdigest() != rec["source_sha256"]:
            return None
        total += rec["dram_bytes_per_launch"]
    return total


# ------------------------------------------------------------------ GPU arm
def run_ours(args):
    import torch
    from paper_1706_09453_b200 import build
    build.build()
    from paper_1706_09453_b200 import binding as B, model, workloads as wl

    from paper_1706_09453_b200 import dist as D
    rank, world, local = D.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    dist = D.init("nccl", torch.device(dev))

    cfg = wl.CONFIGS[args.config]
    frames = args.frames or cfg.frames
    net = wl.make_model(cfg)
    B.bnn_set_xnor_path(B.XNOR_POPC if args.xnor_path == "popc" else B.XNOR_TENSOR)
    B.bnn_set_option(B.OPT_REAL_PATH, B.PATH_TENSOR if args.real_path == "tensor" else B.PATH_CUDA_CORE)
    B.bnn_set_option(B.OPT_XNOR_PREPARED, {"auto": 0, "stream": 1, "resident": 2}[args.xnor_prepared])
    if args.no_stack:
        B.bnn_set_option(B.OPT_XNOR_STACK, 0)
    if args.no_follow:
        B.bnn_set_option(B.OPT_SOFTMAX_FOLLOW, 0)
    dn = model.DeviceNet(net, device=dev, prepare_xnor=args.xnor_path == "tensor",
                         act_values=B.VALUES_01 if args.act_values == "01" else B.VALUES_PM1,
                         splice=((cfg.in_dim // 40) // 2, (cfg.in_dim // 40) // 2) if args.splice else (0, 0))
    # Frames are independent, so ranks shard them with no exchange: each rank owns its own batch.
    Xh = wl.make_frames(cfg, frames, seed=D.frames_seed(cfg.seed, rank))
    if args.splice:   # the same draws, read as unspliced 40-dim frames
        Xh = np.ascontiguousarray(Xh[:, :40])
    set_bytes = frames * (Xh.shape[1] + cfg.classes) * 4
    nsets = max(2, -(-2 * L2_BYTES // set_bytes))          # rotate over > 2 x L2 of inputs/outputs
    Xd = [model.to_dev(Xh, dev) for _ in range(nsets)]
    Ld = [torch.empty((frames, cfg.classes), dtype=torch.float32, device=dev) for _ in range(nsets)]
    ws = dn.workspace(frames)
    K, W = args.steps, max(args.warmup, 3)

    def step(i):
        B.bnn_forward(dn.desc, Xd[i % nsets], Ld[i % nsets], ws)

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(W):
        step(i)
    # bnn_forward only enqueues kernels on the caller's stream, so a caller can capture it: one
    # CUDA graph per buffer set (one bnn_forward each), replayed in turn.  The device then starts
    # each kernel of a step without a host launch in between.
    graphs = None
    if not args.no_graph:
        torch.cuda.synchronize()
        side = torch.cuda.Stream(dev)
        side.wait_stream(torch.cuda.current_stream())
        graphs = []
        with torch.cuda.stream(side):
            for b in range(nsets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    step(b)
                graphs.append(g)
        torch.cuda.current_stream().wait_stream(side)
        for b in range(min(nsets, W)):
            graphs[b].replay()

    def timed_step(i):
        if graphs:
            graphs[i % nsets].replay()
        else:
            step(i)

    clocks = ClockSampler(torch, local)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    clocks.start()
    e0.record()
    for i in range(K):
        timed_step(i)
    e1.record()
    barrier()
    clocks.stop()
    total_ms = D.max_over_ranks(dist, e0.elapsed_time(e1), dev)

    # ---- per-layer device time over the same steps (events recorded inside the C-ABI call)
    nl = cfg.n_hidden + 1
    Kp = min(K, 50)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(nl + 2)] for _ in range(Kp)]
    for row in evs:
        for e in row:
            e.record()
    torch.cuda.synchronize()
    for i in range(Kp):
        B.bnn_forward_events(dn.desc, Xd[i % nsets], Ld[i % nsets], ws, evs[i])
    torch.cuda.synchronize()
    # event order in time: 0 .. nl-1 (before each layer), nl+1 (after the top GEMM), nl (end)
    order = list(range(nl)) + [nl + 1, nl]
    layer_ms = [float(np.mean([evs[i][order[l]].elapsed_time(evs[i][order[l + 1]]) for i in range(Kp)]))
                for l in range(nl + 1)]

    # ---- end to end: pinned host input -> device, forward, log-probs -> pinned host, every step.
    # The three legs run on three streams (copy-in of step i+1, forward of step i and copy-out of
    # step i-1 overlap, as a serving loop would run them); buffers rotate over the nsets device
    # sets and two pinned result buffers, each reuse ordered by events.
    Ke = max(3, min(K, 20))
    Xp = torch.from_numpy(Xh).pin_memory()
    Lps = [torch.empty((frames, cfg.classes), dtype=torch.float32).pin_memory() for _ in range(2)]
    Lp = Lps[0]
    s_in, s_fw, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)

    def e2e_run(n):
        ev_in = [torch.cuda.Event() for _ in range(n)]
        ev_fw = [torch.cuda.Event() for _ in range(n)]
        ev_out = [torch.cuda.Event() for _ in range(n)]
        for i in range(n):
            b = i % nsets
            with torch.cuda.stream(s_in):
                if i >= nsets:
                    s_in.wait_event(ev_fw[i - nsets])        # the forward that read this input set is done
                Xd[b].copy_(Xp, non_blocking=True)
                ev_in[i].record(s_in)
            with torch.cuda.stream(s_fw):
                s_fw.wait_event(ev_in[i])
                if i >= nsets:
                    s_fw.wait_event(ev_out[i - nsets])       # the copy-out of this output set is done
                step(i)
                ev_fw[i].record(s_fw)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_fw[i])
                Lps[i % 2].copy_(Ld[b], non_blocking=True)   # copies on one stream run in order
                ev_out[i].record(s_out)
        return ev_out[-1]

    e2e_run(3)
    torch.cuda.synchronize()
    barrier()
    for st in (s_in, s_fw, s_out):
        st.wait_stream(torch.cuda.current_stream())
    e0.record()
    s_in.wait_event(e0)
    last = e2e_run(Ke)
    torch.cuda.current_stream().wait_event(last)
    e1.record()
    barrier()
    e2e_fps = D.aggregate_rate(frames, world, Ke, D.max_over_ranks(dist, e0.elapsed_time(e1), dev))

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    ck = clocks.summary()
    regime, bf16_peak, regime_why = choose_tensor_regime(peaks, ck, total_ms * 1e-3)
    peaks["bf16"] = bf16_peak
    # rate of a bare kind::mxf4 MMA loop (192-unit tiles, A operand in tensor memory, as the hidden-layer
    # kernel issues them), measured here with the library's micro-benchmark launch
    mxf4_rate = None
    if args.xnor_path != "popc":
        kind = B.RATE_KINDS["mma_mxf4_n192_atmem"]
        scratch = torch.zeros(max(256, B.bnn_pipe_rate_scratch_bytes(kind)), dtype=torch.uint8, device=dev)
        B.bnn_pipe_rate(kind, 512, scratch)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(3):
            work = B.bnn_pipe_rate(kind, 512, scratch)
        e1.record()
        torch.cuda.synchronize()
        mxf4_rate = work / (e0.elapsed_time(e1) / 3 * 1e-3) / 1e12
    peaks["mxf4"] = mxf4_rate or 4.0 * bf16_peak
    rows = layer_table(cfg, frames, peaks, ck.get("sm_mhz"), args.xnor_path, args.real_path, args.xnor_prepared,
                       stacked=not args.no_stack)
    assert len(rows) == len(layer_ms)
    for r, t in zip(rows, layer_ms):
        r["ms"] = t
    # A run of equal binary hidden layers is ONE launch (its events are recorded before the run):
    # the run is reported as one row, time and work summed.
    if not args.no_stack and frames > 16:
        merged = []
        for r in rows:
            if (merged and r["kernel"] == "xnor_res_kernel" and merged[-1]["kernel"] == "xnor_res_kernel"
                    and r["work"] == merged[-1]["work_per_layer"]):
                m = merged[-1]
                m["ms"] += r["ms"]; m["work"] += r["work"]; m["layers"] += 1
                m["name"] = m["first_name"] + ".." + r["name"].split("_")[1]
                if "smem_bytes" in m:
                    m["smem_bytes"] += r["smem_bytes"]
            else:
                r = dict(r, work_per_layer=r["work"], first_name=r["name"], layers=1)
                merged.append(r)
        rows = merged
    for r in rows:
        t = r["ms"]
        r["achieved"] = r["work"] / (t * 1e-3) / r.get("scale", 1e12)
        r["frac"] = r["achieved"] / r["peak"]
        if "peak_nominal_ratio" in r:
            r["frac_nominal_ratio"] = r["achieved"] / r["peak_nominal_ratio"]
        r["pipe_util"] = r["frac"] * r.get("passes", 1)
        if "smem_bytes" in r:
            # fraction of the SMs' shared-memory bandwidth (128 B per clock and SM at the maximum clock)
            r["smem_pipe_util"] = r["smem_bytes"] / (r["ms"] * 1e-3) / (SMS * 128 * peaks["sm_max_mhz"] * 1e6)
    # dominant KERNEL: group the layers by the kernel that runs them (the five binary hidden
    # layers are five launches of one kernel) and take the largest share of the step
    groups = {}
    for r in rows:
        gk = groups.setdefault(r["kernel"], dict(ms=0.0, work=0.0, n=0, row=r))
        gk["ms"] += r["ms"]; gk["work"] += r["work"]; gk["n"] += 1
    dk, dg = max(groups.items(), key=lambda kv: kv[1]["ms"])
    dom = dg["row"]
    achieved = dg["work"] / (dg["ms"] * 1e-3) / dom.get("scale", 1e12)
    if dk in ("xnor_tc_kernel", "xnor_img_kernel", "xnor_res_kernel"):
        peak_source = ("rate of a bare kind::mxf4 MMA loop measured in this run (%.0f Tbop/s); 4 x the %s bf16 figure of "
                       "MEASURED_PEAKS.json (%s) would be %.0f; of measured" % (peaks["mxf4"], regime, peaks["source"], 4 * bf16_peak))
    elif dom["bound"] == "tensor":
        peak_source = "bf16_tflops%s of MEASURED_PEAKS.json (%s), %s regime: %s; of measured" % (
            "" if regime == "burst" else "_sustained", peaks["source"], regime, regime_why)
    elif dom["bound"] == "hbm":
        peak_source = "hbm_gbs of MEASURED_PEAKS.json (%s); of measured" % peaks["source"]
    else:
        peak_source = "derived from unit counts x max SM clock (%.0f MHz)" % peaks["sm_max_mhz"]
    roofline = {"kernel": dk, "launches_per_step": dg["n"], "bound": dom["bound"],
                "achieved": achieved, "peak": dom["peak"], "unit": dom["unit"],
                "frac": achieved / dom["peak"], "traffic": ncu_traffic(dk, cfg.name if frames == cfg.frames else None),
                "peak_source": peak_source,
                "algorithmic_work_per_launch": dg["work"] / dg["n"],
                "share_of_step": dg["ms"] / sum(layer_ms), "avg_launch_ms": dg["ms"] / dg["n"]}
    if dom["bound"] == "tensor" and "peak_nominal_ratio" not in dom:
        roofline["frac_burst"] = achieved / peaks["bf16_tflops"]
        roofline["frac_sustained"] = achieved / peaks["bf16_tflops_sustained"]
    # whole-step roofline: every stage at the peak of the pipe that bounds it, (a) counting the
    # algorithmic work once, (b) counting the work the split-precision layers really execute
    t_alg = sum(r["work"] / (r["peak"] * r.get("scale", 1e12)) for r in rows)
    t_exe = sum(r["work"] * r.get("passes", 1) / (r["peak"] * r.get("scale", 1e12)) for r in rows)
    step_s = total_ms / K * 1e-3
    forward_roofline = {"t_roof_algorithmic_ms": t_alg * 1e3, "frac_algorithmic": t_alg / step_s,
                        "t_roof_executed_ms": t_exe * 1e3, "frac_executed": t_exe / step_s,
                        "target_frac_algorithmic": 0.60, "target_met": bool(t_alg / step_s >= 0.60),
                        "tensor_regime": regime, "bf16_peak_tflops": bf16_peak, "mxf4_peak_tbops": peaks["mxf4"],
                        "note": "sum over layers of algorithmic work / peak of the bounding pipe (bf16: %s figure, %s; 4-bit: "
                                "measured bare MMA rate); 'executed' also counts the extra passes of the split-precision "
                                "real-valued layers" % (regime, regime_why)}
    fps = D.aggregate_rate(frames, world, K, total_ms)
    xnor_work = sum(r["work"] for r in rows if r["name"].startswith("xnor"))
    xnor_ms = sum(r["ms"] for r in rows if r["name"].startswith("xnor"))
    hbm = hbm_bytes_per_step(cfg, frames)
    out = {
        "metric": METRIC, "value": fps, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "%s (hidden layers) + %s (first and top layer)"
                 % ("e2m1 (mxf4) tensor-core MMA, f32 accumulate, exact" if args.xnor_path != "popc" else "int32 popcount",
                    "split bf16/fp16 tensor-core MMA, f32 accumulate" if args.real_path == "tensor" else "f32"),
        "device_status": B.bnn_device_status(), "data": "synthetic",
        "config": {"workload": workload_name(cfg, frames), "frames_per_gpu": frames,
                   "launch": "host launches" if args.no_graph else "one captured CUDA graph per step (a single bnn_forward call each)", "l2": "inputs/outputs rotate over %d buffer sets (%.0f MB > 2 x L2); weights stay hot"
                         % (nsets, nsets * set_bytes / 1e6),
                   "log_softmax": ("after the top layer's kernel" if args.no_follow else
                                   "launched behind the top layer's tensor-core kernel and overlapped with it where that "
                                   "kernel has more than one wave of tiles (log_softmax_rows_follow_kernel); the "
                                   "per-layer rows time the two kernels apart (log_softmax_rows_reg_kernel)"),
                   "sign_zero": "+1", "act_values": "(0,1)" if args.act_values == "01" else "(-1,+1)",
                   "input": "one 40-dim frame per row, context window formed in the first layer" if args.splice else "spliced", "seed": cfg.seed},
        "clocks": ck,
        "e2e": {"value": e2e_fps, "unit": UNIT, "h2d_bytes_per_step": int(Xp.numel() * 4),
                "d2h_bytes_per_step": int(Lp.numel() * 4), "steps": Ke,
                "overlap": "copy-in, forward and copy-out of consecutive steps on three streams"},
        # per step: the kernels named in the layer table (one per binary hidden layer, two per
        # sign-weight layer: split + GEMM, top-layer GEMM, log-softmax)
        "gpu_launches": K * (sum(r["kernel"].count("+") + 1 for r in rows)),
        "paths": {"xnor": args.xnor_path, "real": args.real_path},
        "roofline": roofline,
        "forward_roofline": forward_roofline,
        "layers": [{k: r[k] for k in ("name", "kernel", "layers", "bound", "ms", "achieved", "peak", "unit", "frac", "frac_nominal_ratio", "pipe_util", "smem_pipe_util") if k in r}
                   for r in rows],
        "xnor_tbops": (xnor_work / (xnor_ms * 1e-3) / 1e12) if xnor_ms else None,
        "hbm": {"algorithmic_bytes_per_step": hbm, "achieved_gbs": hbm / (total_ms / K * 1e-3) / 1e9,
                "peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"]},
    }
    if world == 1 and not args.no_cpu_baseline:
        from oracle import bnn_oracle as o
        n = min(frames, args.cpu_frames)
        # The oracle pass that is timed also checks the log-probs of the last timed step.  For the
        # binary networks it continues from the library's own first-layer bits (units whose
        # pre-activation lies inside the float tolerance may binarise either way), after which every
        # later bit must be equal; those bits come from one more forward on the same input.
        last = (K - 1) % nsets
        g1, outs = None, None
        mixed = getattr(cfg, "mixed", False)
        plain = args.act_values == "pm1" and not args.splice
        binary = cfg.act == 1 and not mixed and plain
        if (binary or mixed) and plain:
            outs = dn.layer_out_buffers(frames)
            chk = torch.empty_like(Ld[last])
            B.bnn_forward(dn.desc, Xd[last], chk, ws, layer_out=outs)
            torch.cuda.synchronize()
            # the first layer with Sign units: layer 1, or layer 2 of the mixed topology
            g1 = model.words_to_numpy(outs[1 if mixed else 0][:n], cfg.hidden)
            same_logp = bool(torch.equal(chk, Ld[last]))
        t0 = time.perf_counter()
        if binary:
            ref = o.forward(Xh[:n], net.W, net.scale, net.shift, net.Wout, net.bout, o.ACT_SIGN, o.SIGN_ZERO_POS,
                            layer1_bits=g1)
        elif mixed and plain:
            ref = o.forward_mixed(Xh[:n], net.W, net.scale, net.shift, net.Wout, net.bout, o.SIGN_ZERO_POS, layer2_bits=g1)
        else:
            ref = oracle_step(cfg, net, Xh[:n])
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": n / dt, "unit": UNIT, "cores": o.num_threads(), "kind": "oracle",
                               "sample": "first %d frames of the batch, one pass (%.1f s)" % (n, dt)}
        if plain:
            got = Ld[last][:n].cpu().numpy()
            par = {"frames": n, "max_abs_dlogp": float(np.abs(got - ref["logp"]).max()), "tolerance_logp": 1e-4}
            if binary:
                band = 1e-4 * np.abs(net.scale[0])[None, :] * ref["sumabs"][:, None]
                decided = np.abs(ref["pre"][0]) > band
                par["layer1_bits_equal_outside_tolerance_band"] = bool(
                    (o.unpack_pm1(g1, cfg.hidden)[decided] == o.unpack_pm1(ref["bits_own_layer1"], cfg.hidden)[decided]).all())
                par["layer1_units_inside_band"] = int((~decided).sum())
                par["hidden_bits_equal"] = bool(all(
                    (model.words_to_numpy(outs[l][:n], cfg.hidden) == ref["bits"][l]).all() for l in range(1, cfg.n_hidden)))
                par["timed_step_logp_equal_to_checked_forward"] = same_logp
            elif mixed:
                band = 1e-4 * np.abs(net.scale[1])[None, :] * ref["sumabs2"][:, None]
                decided = np.abs(ref["pre2"]) > band
                par["layer2_bits_equal_outside_tolerance_band"] = bool(
                    (o.unpack_pm1(g1, cfg.hidden)[decided] == o.unpack_pm1(ref["bits_own_layer2"], cfg.hidden)[decided]).all())
                par["hidden_bits_equal"] = bool(all(
                    (model.words_to_numpy(outs[l][:n], cfg.hidden) == ref["bits"][l - 1]).all() for l in range(2, cfg.n_hidden - 1)))
                par["timed_step_logp_equal_to_checked_forward"] = same_logp
            par["ok"] = bool(par["max_abs_dlogp"] <= 1e-4 and par.get("hidden_bits_equal", True)
                             and par.get("layer1_bits_equal_outside_tolerance_band", True)
                             and par.get("layer2_bits_equal_outside_tolerance_band", True))
            out["parity"] = par
    print(json.dumps(out))
    if dist:
        dist.destroy_process_group()


def run_sweep(args):
    """Isolated XNOR-popcount GEMM, int32 output, on both kernels; binary-op/s and GB/s per point
    against max(bytes / HBM bandwidth, bops / tensor peak).  Inputs are drawn on the device and
    packed with the library's own bnn_binarize_pack; a few rows of every point are checked
    against the CPU oracle."""
    import torch
    from paper_1706_09453_b200 import build
    build.build()
    from paper_1706_09453_b200 import binding as B, model, workloads as wl
    from oracle import bnn_oracle as o
    peaks = load_peaks()
    dev = "cuda:0"
    Ms, Ks, Ns = wl.SWEEP_M, wl.SWEEP_K, wl.SWEEP_N
    if args.sweep_quick:
        Ms, Ks, Ns = (Ms[0], Ms[-1]), (Ks[0], Ks[-1]), (Ns[0], Ns[-1])
    gen = torch.Generator(device=dev)

    def planes(rows, k, p, seed):
        gen.manual_seed(seed)
        out = model.packed_empty(rows, k, dev)
        step = max(1, (1 << 28) // k)      # pack in slabs of <= 1 GiB of floats
        for r0 in range(0, rows, step):
            r1 = min(rows, r0 + step)
            x = torch.rand((r1 - r0, k), device=dev, generator=gen)
            x = (p - x)                      # >= 0 with probability p  ->  bit 1
            B.bnn_binarize_pack(x, out[r0:r1], B.SIGN_ZERO_NEG)
        return out

    def timeit(fn, n):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    for p in wl.SWEEP_P:
        for M in Ms:
            for K in Ks:
                A = planes(M, K, p, 1000 + M + K)
                for N in Ns:
                    W = planes(N, K, p, 2000 + N + K)
                    # rotate over enough output buffers that C is never found in L2
                    cbytes = M * N * 4
                    nbuf = max(1, min(4, -(-2 * L2_BYTES // cbytes)))
                    Cs = [torch.empty((M, N), dtype=torch.int32, device=dev) for _ in range(nbuf)]
                    bops = 2.0 * M * N * K
                    nbytes = M * K / 8 + N * K / 8 + cbytes
                    rec = {"sweep": True, "M": M, "K": K, "N": N, "p": p, "bops": bops, "bytes": nbytes}
                    it = [0]
                    for name, path in (("tensor", B.XNOR_TENSOR), ("popc", B.XNOR_POPC)):
                        B.bnn_set_xnor_path(path)
                        def call():
                            B.bnn_xnor_gemm(A, W, K, C_out=Cs[it[0] % nbuf]); it[0] += 1
                        reps = 5 if bops > 1e12 else 20
                        if name == "popc" and bops > 2e12:
                            reps = 2
                        ms = timeit(call, reps)
                        rec[name] = {"ms": ms, "tbops": bops / ms / 1e9, "gbs": nbytes / ms / 1e6}
                    t_roof = max(nbytes / (peaks["hbm_gbs"] * 1e9), bops / (4 * peaks["bf16_tflops"] * 1e12))
                    rec["bound"] = "hbm" if nbytes / (peaks["hbm_gbs"] * 1e9) > bops / (4 * peaks["bf16_tflops"] * 1e12) else "tensor"
                    rec["roofline_frac_tensor_kernel"] = t_roof / (rec["tensor"]["ms"] * 1e-3)
                    # parity on sampled rows (first, last, two in between)
                    B.bnn_set_xnor_path(B.XNOR_TENSOR)
                    B.bnn_xnor_gemm(A, W, K, C_out=Cs[0])
                    rows = sorted({0, M // 3, (2 * M) // 3, M - 1})
                    got = Cs[0][rows].cpu().numpy()
                    want = o.xnor_gemm(model.words_to_numpy(A[rows], K), model.words_to_numpy(W, K), K)
                    rec["parity_rows_checked"] = len(rows)
                    rec["parity_ok"] = bool((got == want).all())
                    rec["device_status"] = B.bnn_device_status()
                    print(json.dumps(rec), flush=True)
                    del Cs, W
                del A


def run_pipe_rates(args):
    """Rates of the execution pipes the kernels are bound by, measured with the library's own
    micro-benchmark launches (bnn_pipe_rate), each timed with CUDA events after a warm-up launch;
    SM clock and throttle reasons sampled meanwhile."""
    import torch
    from paper_1706_09453_b200 import build
    build.build()
    from paper_1706_09453_b200 import binding as B
    dev = "cuda:0"
    torch.cuda.set_device(0)
    peaks = load_peaks()
    scratch = torch.zeros(max(B.bnn_pipe_rate_scratch_bytes(k) for k in B.RATE_KINDS.values()), dtype=torch.uint8, device=dev)
    plan = [("popc", 256, "Tbop/s", 1e12), ("lop3", 256, "Tinst/s", 1e12), ("iadd", 256, "Tinst/s", 1e12),
            ("fadd", 256, "Tinst/s", 1e12), ("ffma", 256, "TFLOP/s", 1e12),
            ("mma_mxf4_n256", 512, "Tbop/s", 1e12), ("mma_mxf4_n192", 512, "Tbop/s", 1e12),
            ("mma_mxf4_n192_atmem", 512, "Tbop/s", 1e12), ("mma_f16_n256", 512, "TFLOP/s", 1e12),
            ("l2_read", 4, "GB/s", 1e9)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, repeat, unit, scale in plan:
        kind = B.RATE_KINDS[name]
        B.bnn_pipe_rate(kind, repeat, scratch)          # warm-up
        torch.cuda.synchronize()
        sampler = ClockSampler(torch, 0)
        sampler.start()
        reps = 10
        e0.record()
        for _ in range(reps):
            work = B.bnn_pipe_rate(kind, repeat, scratch)
        e1.record()
        torch.cuda.synchronize()
        sampler.stop()
        ms = e0.elapsed_time(e1) / reps
        rec = {"pipe_rate": name, "rate": work / (ms * 1e-3) / scale, "unit": unit, "ms_per_launch": ms,
               "work_per_launch": work, "launches": reps, "clocks": sampler.summary(),
               "device_status": B.bnn_device_status()}
        if name.startswith("mma_mxf4"):
            rec["vs_4x_bf16_burst"] = rec["rate"] / (4 * peaks["bf16_tflops"])
        if name == "mma_f16_n256":
            rec["vs_bf16_burst"] = rec["rate"] / peaks["bf16_tflops"]
        print(json.dumps(rec), flush=True)


if __name__ == "__main__":
    a = parse_args()
    if a.pipe_rates:
        run_pipe_rates(a)
    elif a.sweep:
        run_sweep(a)
    elif a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
