#!/usr/bin/env python
"""Benchmark of the MicroQonv hot path on B200.

A step is one pass of the whole path over one batch of synthetic input of the workload
(default: the single 3x3 MXFP4 layer N=32, 64->128 channels, 80x80): mq_quantize on X, W and dY
(once each), mq_cbf_im2col, mq_conv_fwd, mq_conv_bwd_data, mq_conv_bwd_weight.  The headline value
is the layer's useful convolution FLOPs (3 GEMMs) divided by the whole step time, with inputs
resident in HBM; `e2e` is the same through mq_conv_layer_host with pinned host buffers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config2|config1|config4_3x3|...]
    python bench.py --impl reference ...      # times the CPU oracle on a bounded sample

Multi-GPU (torchrun): each rank runs the layer on its own batch (weak scaling, batch shards in
units of 32 samples) and the weight gradients are summed with one NCCL all-reduce per step.
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2609_28358_b200 import inputs  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
FMT_NAME = {0: "e4m3", 1: "e5m2", 2: "e2m1", 3: "e3m2", 4: "e2m3"}
FMT_BITS = {0: 8, 1: 8, 2: 4, 3: 8, 4: 8}   # stored bits per code (the 6-bit formats sit one per byte and run at the 8-bit tensor rate)
# nominal dense tensor-core ratio to bf16 for the operand formats of a GEMM
TENSOR_RATIO = {8: 2.0, 4: 4.0}

# dram__bytes_read.sum + dram__bytes_write.sum per call from ncu captures of the call's kernels on the named
# workload (profiles/*_config2.md), summed over the kernels one call launches.  Config 2's tensors are of the size
# of the 126 MB L2, so part of every output is still cached when the kernel ends: these figures are below the
# algorithmic bytes for the write-heavy calls and are kept as measured.
NCU_TRAFFIC = {
    ("config2", "quantize_x"): 52442112 + 322560,
    ("config2", "quantize_dy"): 104871680 + 6986496,
    ("config2", "cbf_im2col"): 6600960 + 4038400,
    ("config2", "conv_fwd"): 6650880 + 52783872,          # conv_tc_halo_kernel<fwd>
    ("config2", "conv_bwd_data"): 13218560 + 4152832,     # conv_tc_halo_kernel<bwd_data>; weight_transpose_kernel not captured
    ("config2", "conv_bwd_weight"): 19756544 + 26230272,   # wgrad_flat_prep_kernel + wgrad_tc_kernel; the reduce not captured
}


def workloads():
    w = {}
    for cfg in ("config1", "config2", "config4"):
        for l in inputs.CONFIGS[cfg]():
            w[l.name] = l
    w["config1"] = inputs.config1()[0]
    w["config2"] = inputs.config2()[0]
    for l in inputs.config5():
        w[l.name] = l
    for l in inputs.config3():
        w["cfg3_" + l.name] = l
    for l in inputs.fp6_layers():
        w[l.name] = l
    return w


def layer_flops(d):
    ho, wo = inputs.out_hw(d)
    return 2.0 * d.N * ho * wo * d.C_out * d.C_in * d.Kh * d.Kw


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            m = json.load(f)
        return {"hbm_gbs": float(m["hbm_gbs"]), "bf16_tflops": float(m["bf16_tflops"]),
                "bf16_tflops_sustained": float(m.get("bf16_tflops_sustained", m["bf16_tflops"]))}, "measured"
    return dict(FALLBACK_PEAKS, bf16_tflops_sustained=1400.0), "fallback"


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.stop_flag, self.max_mhz, self.err = index, [], set(), False, None, None

    def run(self):
        try:
            import pynvml as nv

            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                     "hw_power_brake_slowdown": 0x80}
            while not self.stop_flag:
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(h) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
                time.sleep(0.002)
        except Exception as e:  # NVML missing: report it, do not fail the bench
            self.err = repr(e)

    def result(self):
        self.stop_flag = True
        self.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "error": self.err}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------ ours
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2609_28358_b200 import mq

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    mq.lib()  # fail loudly if the CUDA library is missing

    layer = workloads()[args.workload]
    d = layer.desc
    fmts = (layer.fmt_x, layer.fmt_w, layer.fmt_dy)
    roles = (mq.ROLE_X, mq.ROLE_W, mq.ROLE_DY)
    seed = layer.seed + 1000 * rank
    x, w, g = (inputs.make_x(d, seed, layer.x_kind), inputs.make_w(d, layer.seed, layer.w_kind), inputs.make_dy(d, seed, layer.dy_kind))
    src = [torch.from_numpy(t).cuda() for t in (x, w, g)]
    q = [mq.empty_qtensor(d, r, f) for r, f in zip(roles, fmts)]
    icb, isb = mq.im2col_sizes(d, fmts[0])
    ic = torch.empty(icb, dtype=torch.uint8, device="cuda")
    isc = torch.empty(isb, dtype=torch.uint8, device="cuda")
    ho, wo = inputs.out_hw(d)
    y = torch.empty((d.N, d.C_out, ho, wo), dtype=torch.float32, device="cuda")
    dx = torch.empty((d.N, d.C_in, d.H, d.W), dtype=torch.float32, device="cuda")
    dw = torch.empty((d.C_out, d.C_in, d.Kh, d.Kw), dtype=torch.float32, device="cuda")
    ws_bytes = max(mq.workspace_size(d, op, a, b) for op, a, b in
                   ((mq.OP_FWD, fmts[0], fmts[1]), (mq.OP_BWD_DATA, fmts[1], fmts[2]), (mq.OP_BWD_WEIGHT, fmts[0], fmts[2])))
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")  # > 126 MB L2

    calls = [
        ("quantize_x", lambda: mq.quantize(d, roles[0], fmts[0], src[0], out=q[0])),
        ("quantize_w", lambda: mq.quantize(d, roles[1], fmts[1], src[1], out=q[1])),
        ("quantize_dy", (lambda: mq.quantize_sr(d, roles[2], fmts[2], src[2], 1234, out=q[2])) if args.dy_rounding == "stochastic" else
         (lambda: mq.quantize(d, roles[2], fmts[2], src[2], out=q[2]))),
        ("cbf_im2col", lambda: mq.cbf_im2col(d, q[0], ic, isc)),
        ("conv_fwd", lambda: mq.conv_fwd(d, q[0], q[1], y=y, workspace=ws)),
        ("conv_bwd_data", lambda: mq.conv_bwd_data(d, q[1], q[2], dx=dx, workspace=ws)),
        ("conv_bwd_weight", lambda: mq.conv_bwd_weight(d, q[0], q[2], dw=dw, workspace=ws)),
    ]

    def step():
        for _, fn in calls:
            fn()
        if world > 1:
            dist.all_reduce(dw)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()

    # Optionally the step's launches are captured once into a CUDA graph and replayed: the same kernels with the same
    # arguments, without the per-call host work (small layers are bound by it).  Single GPU only; any failure to
    # capture falls back to plain launches and is reported.
    run_step, graph_note, launches_per_step = step, "off", None
    if args.cuda_graph and world == 1:
        try:
            c0 = mq.kernel_launch_count()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            launches_per_step = mq.kernel_launch_count() - c0
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            graph.replay()
            torch.cuda.synchronize()
            if mq.last_device_status() != 0:
                raise RuntimeError("device status after replay")
            run_step, graph_note = graph.replay, "on"
        except Exception as exc:  # noqa: BLE001
            torch.cuda.synchronize()
            run_step, graph_note, launches_per_step = step, f"capture failed ({type(exc).__name__}), plain launches", None

    # ---- timed region: K steps, L2 flushed between steps (flush outside the event pairs)
    K = args.steps
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    barrier()
    launches0 = mq.kernel_launch_count()
    for s, e in ev:
        flush.zero_()
        s.record()
        run_step()
        e.record()
    barrier()
    launches = mq.kernel_launch_count() - launches0   # kernels of this library inside the timed region
    if launches_per_step is not None:
        launches = launches_per_step * K               # replayed launches are not counted by the library's host-side counter
    ms_total = sum(s.elapsed_time(e) for s, e in ev)

    # ---- per-call durations over K more steps (same stream, same flush), for the roofline
    names = [n for n, _ in calls]
    per = {n: [] for n in names}
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)] for _ in range(K)]
    for m in marks:
        flush.zero_()
        m[0].record()
        for i, (_, fn) in enumerate(calls):
            fn()
            m[i + 1].record()
    torch.cuda.synchronize()
    for m in marks:
        for i, n in enumerate(names):
            per[n].append(m[i].elapsed_time(m[i + 1]))
    dev_status = mq.last_device_status()
    # kernels one call launches (the library's own count): conv_bwd_weight is a re-layout, a GEMM and a reduction
    n_launch = {}
    for n, fn in calls:
        c0 = mq.kernel_launch_count()
        fn()
        n_launch[n] = max(1, mq.kernel_launch_count() - c0)
    torch.cuda.synchronize()

    # ---- the same step with channel-fastest fp32 tensors ([H][W][N][C] / [Cout][Kh][Kw][Cin]): the order the
    # convolution entry points emit when layers chain.  Reported beside the headline, which keeps NCHW / OIHW.
    src_cl = [src[0].permute(2, 3, 0, 1).contiguous(), src[1].permute(0, 2, 3, 1).contiguous(), src[2].permute(2, 3, 0, 1).contiguous()]
    y_cl = torch.empty((ho, wo, d.N, d.C_out), dtype=torch.float32, device="cuda")
    dx_cl = torch.empty((d.H, d.W, d.N, d.C_in), dtype=torch.float32, device="cuda")
    dw_cl = torch.empty((d.C_out, d.Kh, d.Kw, d.C_in), dtype=torch.float32, device="cuda")
    calls_cl = [
        ("quantize_x", lambda: mq.quantize(d, roles[0], fmts[0], src_cl[0], out=q[0], src_layout=mq.HWNC)),
        ("quantize_w", lambda: mq.quantize(d, roles[1], fmts[1], src_cl[1], out=q[1], src_layout=mq.HWNC)),
        ("quantize_dy", (lambda: mq.quantize_sr(d, roles[2], fmts[2], src_cl[2], 1234, out=q[2], src_layout=mq.HWNC)) if args.dy_rounding == "stochastic"
         else (lambda: mq.quantize(d, roles[2], fmts[2], src_cl[2], out=q[2], src_layout=mq.HWNC))),
        ("cbf_im2col", lambda: mq.cbf_im2col(d, q[0], ic, isc)),
        ("conv_fwd", lambda: mq.conv_fwd(d, q[0], q[1], y=y_cl, layout=mq.HWNC, workspace=ws)),
        ("conv_bwd_data", lambda: mq.conv_bwd_data(d, q[1], q[2], dx=dx_cl, layout=mq.HWNC, workspace=ws)),
        ("conv_bwd_weight", lambda: mq.conv_bwd_weight(d, q[0], q[2], dw=dw_cl, layout=mq.HWNC, workspace=ws)),
    ]
    for _ in range(3):
        for _, fn in calls_cl:
            fn()
    torch.cuda.synchronize()
    Kc = max(3, min(K, 20))
    ev_cl = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(Kc)]
    for s_, e_ in ev_cl:
        flush.zero_()
        s_.record()
        for _, fn in calls_cl:
            fn()
        e_.record()
    torch.cuda.synchronize()
    ms_cl = sum(s_.elapsed_time(e_) for s_, e_ in ev_cl) / Kc
    per_cl = {n: [] for n, _ in calls_cl}
    for _ in range(Kc):
        flush.zero_()
        m = [torch.cuda.Event(enable_timing=True) for _ in range(len(calls_cl) + 1)]
        m[0].record()
        for i, (_, fn) in enumerate(calls_cl):
            fn()
            m[i + 1].record()
        torch.cuda.synchronize()
        for i, (n, _) in enumerate(calls_cl):
            per_cl[n].append(m[i].elapsed_time(m[i + 1]))
    # leave the NCHW-quantized tensors in place for what follows
    for n, fn in calls[:3]:
        fn()
    torch.cuda.synchronize()

    # ---- end to end: pinned host buffers through mq_conv_layer_host, copies inside the timed region
    hx, hw_, hg = [torch.from_numpy(t).pin_memory() for t in (x, w, g)]
    hy = torch.empty(y.shape, dtype=torch.float32).pin_memory()
    hdx = torch.empty(dx.shape, dtype=torch.float32).pin_memory()
    hdw = torch.empty(dw.shape, dtype=torch.float32).pin_memory()
    arena = torch.empty(mq.conv_layer_host_arena_size(d, *fmts), dtype=torch.uint8, device="cuda")
    Ke = max(3, min(K, 20))
    for _ in range(2):
        mq.conv_layer_host(d, fmts, hx, hw_, hg, hy, hdx, hdw, arena)
    barrier()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(Ke):
        mq.conv_layer_host(d, fmts, hx, hw_, hg, hy, hdx, hdw, arena)
        if world > 1:
            pass  # the host-buffer call returns per-rank gradients; the reduction is the device path's
    t1.record()
    barrier()
    e2e_ms = t0.elapsed_time(t1) / Ke
    clocks = sampler.result()

    if world > 1:
        t = torch.tensor([ms_total, e2e_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total, e2e_ms = float(t[0]), float(t[1])

    flops = 3.0 * layer_flops(d) * world
    ms_step = ms_total / K
    value = flops / (ms_step * 1e-3) / 1e12

    # ---- roofline of the dominant kernel
    pk, pk_src = peaks()
    nelem = {"quantize_x": x.size, "quantize_w": w.size, "quantize_dy": g.size}
    qbytes = {n: nelem[n] * 4.0 + sum(t.numel() for t in (qt.codes, qt.scales)) for n, qt in zip(("quantize_x", "quantize_w", "quantize_dy"), q)}
    alg_bytes = dict(qbytes)
    alg_bytes["cbf_im2col"] = float(q[0].codes.numel() + q[0].scales.numel() + icb + isb)
    gemm_bits = {"conv_fwd": max(FMT_BITS[fmts[0]], FMT_BITS[fmts[1]]), "conv_bwd_data": max(FMT_BITS[fmts[1]], FMT_BITS[fmts[2]]),
                 "conv_bwd_weight": max(FMT_BITS[fmts[0]], FMT_BITS[fmts[2]])}
    # GEMMs: the binding roof is the slower of tensor time and HBM time for the kernel's algorithmic bytes
    qb = {r: float(qt.codes.numel() + qt.scales.numel()) for r, qt in zip(("x", "w", "dy"), q)}
    gemm_bytes = {"conv_fwd": qb["x"] + qb["w"] + 4.0 * y.numel(), "conv_bwd_data": qb["w"] + qb["dy"] + 4.0 * dx.numel(),
                  "conv_bwd_weight": qb["dy"] + qb["x"] + 4.0 * dw.numel()}
    kern = {}
    for n in names:
        ms = float(np.mean(per[n]))
        if n in alg_bytes:
            ach = alg_bytes[n] / (ms * 1e-3) / 1e9
            kern[n] = {"ms": ms, "bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"]}
        else:
            peak_t = pk["bf16_tflops"] * TENSOR_RATIO[gemm_bits[n]]
            t_tensor = layer_flops(d) / (peak_t * 1e12)
            t_hbm = gemm_bytes[n] / (pk["hbm_gbs"] * 1e9)
            if t_tensor >= t_hbm:
                ach = layer_flops(d) / (ms * 1e-3) / 1e12
                kern[n] = {"ms": ms, "bound": "tensor", "achieved": ach, "peak": peak_t, "unit": "TFLOP/s", "frac": ach / peak_t}
            else:
                ach = gemm_bytes[n] / (ms * 1e-3) / 1e9
                kern[n] = {"ms": ms, "bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"]}
            kern[n]["tflops"] = layer_flops(d) / (ms * 1e-3) / 1e12
    # dominant KERNEL: the largest time per launch (a call's time over the kernels it launches), not the longest call
    for n in names:
        kern[n]["launches"] = n_launch[n]
    dom = max(names, key=lambda n: kern[n]["ms"] / n_launch[n])
    roof = {k: kern[dom][k] for k in ("bound", "achieved", "peak", "unit", "frac")}
    roof.update({"kernel": dom, "peak_source": pk_src + (" (bf16 burst x%g nominal ratio)" % TENSOR_RATIO[gemm_bits[dom]] if roof["bound"] == "tensor" else " copy bandwidth"),
                 "traffic": NCU_TRAFFIC.get((args.workload, dom))})
    qi_bytes = sum(alg_bytes[n] for n in alg_bytes)
    qi_ms = sum(kern[n]["ms"] for n in alg_bytes)

    out = {
        "metric": "MX conv fwd+bwd TFLOPS (whole layer step: quantize x3 + CBF-im2col + fwd + dX + dW)",
        "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "+".join(FMT_NAME[f] for f in fmts) + " (fp32 accumulate)", "data": "synthetic",
        "config": {"workload": args.workload, "layer": dict(d._asdict()), "formats": [FMT_NAME[f] for f in fmts], "dy_rounding": args.dy_rounding, "cuda_graph": graph_note,
                   "global_batch": d.N * world, "parallelism": "dp%d" % world if world > 1 else "single", "l2": "flushed between steps (512 MiB write)"},
        "clocks": clocks,
        "e2e": {"value": flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOPS", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int((x.size + w.size + g.size) * 4), "d2h_bytes_per_step": int((y.numel() + dx.numel() + dw.numel()) * 4)},
        "gpu_launches": launches,
        "roofline": roof,
        "quantize_im2col_gbs": {"value": qi_bytes / (qi_ms * 1e-3) / 1e9, "frac_of_hbm_peak": qi_bytes / (qi_ms * 1e-3) / 1e9 / pk["hbm_gbs"]},
        "kernels": kern,
        "channel_fastest_fp32": {"note": "same step with fp32 tensors in [H][W][N][C] / [Cout][Kh][Kw][Cin] order (MQ_HWNC)",
                                 "value": 3.0 * layer_flops(d) / (ms_cl * 1e-3) / 1e12, "unit": "TFLOPS", "ms_per_step": ms_cl,
                                 "ms_per_call": {n: float(np.mean(v)) for n, v in per_cl.items()}},
        "device_status": dev_status,
        "quantization_accounting": quantization_accounting(d, fmts),
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(layer, budget_s=args.cpu_budget)
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def quantization_accounting(d, fmts):
    """Counts of the kind the paper tabulates (Table I): elements that pass through a quantizer per training step of the
    layer, and bytes of the activation kept for the backward pass, for this library's path (square tiles: each tensor
    quantized once, usable in both contraction directions) next to two stand-ins built from their descriptions in the
    paper - a line-block scheme (blocks along one contraction axis only, so every tensor is quantized again for its
    second GEMM and the activation is kept in fp32 for that) and a scheme that quantizes the expanded im2col matrix and
    keeps it.  Pure arithmetic on the layer shape; nothing here is measured."""
    ho, wo = inputs.out_hw(d)
    nx, nw, ng = d.N * d.C_in * d.H * d.W, d.C_out * d.C_in * d.Kh * d.Kw, d.N * d.C_out * ho * wo
    nxp = ho * wo * d.N * d.Kh * d.Kw * d.C_in                      # elements of the expanded X'
    bx = FMT_BITS[fmts[0]] / 8.0
    return {
        "unit": {"quantized_elements": "elements per fwd+bwd step", "activation_kept": "bytes"},
        "square_tiles_once": {"quantized_elements": nx + nw + ng, "activation_kept": nx * bx * (1 + 1 / 1024)},
        "line_blocks_requantize": {"quantized_elements": 2 * (nx + nw + ng), "activation_kept": nx * 4.0},
        "quantize_expanded_im2col": {"quantized_elements": nxp + nw + ng, "activation_kept": nxp * bx * (1 + 1 / 32)},
        "expansion_factor": nxp / nx,
    }


# ----------------------------------------------------------------------------------- CPU oracle
def oracle_step(layer, ns):
    """One pass of the whole path in the oracle on the first `ns` samples of the layer's batch."""
    import oracle

    d0 = layer.desc
    d = d0._replace(N=ns)
    x = inputs.make_x(d0, layer.seed, layer.x_kind)[:ns]
    w = inputs.make_w(d0, layer.seed, layer.w_kind)
    g = inputs.make_dy(d0, layer.seed, layer.dy_kind)[:ns]
    t0 = time.perf_counter()
    fm = (layer.fmt_x, layer.fmt_w, layer.fmt_dy)
    q = [oracle.quantize(d, r, f, t) for r, f, t in zip((0, 1, 2), fm, (x, w, g))]
    oracle.cbf_im2col(d, fm[0], *q[0])
    xh, wh, gh = [oracle.dequant(d, r, f, c, s) for r, f, (c, s) in zip((0, 1, 2), fm, q)]
    oracle.conv_fwd(d, xh, wh)
    oracle.conv_bwd_data(d, wh, gh)
    oracle.conv_bwd_weight(d, gh, xh)
    return time.perf_counter() - t0, 3.0 * layer_flops(d)


def pick_sample(layer, budget_s):
    import oracle

    oracle.build()
    t1, _ = oracle_step(layer, 1)
    ns = int(max(1, min(layer.desc.N, budget_s / max(t1, 1e-3))))
    return ns


def cpu_baseline(layer, budget_s=15.0):
    import oracle

    ns = pick_sample(layer, budget_s)
    t, fl = oracle_step(layer, ns)
    return {"value": fl / t / 1e12, "unit": "TFLOPS", "cores": oracle.num_threads(), "kind": "oracle", "seconds": t,
            "sample": f"first {ns} of {layer.desc.N} samples of the batch, whole path (quantize x3, im2col, fwd, dX, dW) in the fp64 oracle"}


def run_reference(args):
    import oracle

    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    layer = workloads()[args.workload]
    K, W = args.steps, max(args.warmup, 0)
    ns = pick_sample(layer, 150.0 / (K + W + 1))
    for _ in range(W):
        oracle_step(layer, ns)
    t = 0.0
    fl = 0.0
    for _ in range(K):
        dt, f = oracle_step(layer, ns)
        t += dt
        fl += f
    value = fl / t / 1e12
    d = layer.desc
    fmts = (layer.fmt_x, layer.fmt_w, layer.fmt_dy)
    sample = f"first {ns} of {d.N} samples of the batch per step, whole path in the fp64 oracle"
    print(json.dumps({
        "impl": "reference",
        "metric": "MX conv fwd+bwd TFLOPS (whole layer step: quantize x3 + CBF-im2col + fwd + dX + dW)",
        "value": value, "unit": "TFLOPS", "n_gpus": int(os.environ.get("WORLD_SIZE", 1)), "steps": K, "warmup": W,
        "ms_per_step": t / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "layer": dict(d._asdict()), "formats": [FMT_NAME[f] for f in fmts], "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOPS", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cuda-graph", action="store_true", help="replay the step's launches from a CUDA graph (single GPU)")
    ap.add_argument("--dy-rounding", default="nearest", choices=["nearest", "stochastic"],
                    help="rounding of the gradient's quantizer in the device-timed step (the host-buffer call keeps nearest)")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
