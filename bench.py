#!/usr/bin/env python
"""Benchmark of the MicroQonv hot path on B200.

A step is one pass of the whole path over one batch of synthetic input of the workload: mq_quantize on X, W and
dY (once each), mq_cbf_im2col, mq_conv_fwd, mq_conv_bwd_data, mq_conv_bwd_weight.  The headline value is the
layer's useful convolution FLOPs (3 GEMMs) divided by the whole step time, with inputs resident in HBM; `e2e` is
the same through mq_conv_layer_host with pinned host buffers.

The default workload is the largest single-GPU point of the throughput sweep (N = 256, 512 -> 512 channels, 56 x 56,
3x3, MXFP8 E4M3: 3.79 TFLOP per GEMM, 1.64 GB of fp32 per activation tensor), where the GEMMs are tensor-bound and
the quantizer works at HBM scale.  The same step is also timed on three more workloads (the MXFP4 twin of the
default, the latent-replay 3x3 layer, and the small outlier layer) and reported under `more_workloads`.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--more a,b,c | --more none]
    python bench.py --impl reference ...      # times the CPU oracle on a bounded sample

Multi-GPU (torchrun): each rank runs the layer on its own batch (weak scaling, batch shards in units of 32
samples) and the weight gradients are summed with one NCCL all-reduce per step.
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

DEFAULT_WORKLOAD = "cfg5_e4m3_k3s1_c512_hw56"
# a name + "+ts16": the same layer in the paper's own number format (fp32 tensor scale, E4M3 scale per 16 x 16 block, E2M1; Eq. 4-6)
MORE_WORKLOADS = ("cfg5_e2m1_k3s1_c512_hw56", "cfg5_e2m1_k3s1_c512_hw56+ts16", "cfg4_3x3", "config2")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
# published dense figures (NVIDIA's B200 / HGX B200 data sheet, per GPU, without sparsity): context beside the measured roofs
PUBLISHED = {"hbm_gbs": 7700.0, "tensor_tflops": {8: 4500.0, 4: 9000.0}}
FMT_NAME = {0: "e4m3", 1: "e5m2", 2: "e2m1", 3: "e3m2", 4: "e2m3", 5: "e3m2_p6", 6: "e2m3_p6"}
FMT_BITS = {0: 8, 1: 8, 2: 4, 3: 8, 4: 8, 5: 8, 6: 8}   # tensor-core rate class of a code (the 6-bit formats run at the 8-bit rate, one per byte or packed)
PACKED6 = {3: 5, 4: 6}                       # name + "+p6": the layer's 6-bit tensors in packed storage (16 codes in 12 bytes)
# nominal dense tensor-core ratio to bf16 for the operand formats of a GEMM
TENSOR_RATIO = {8: 2.0, 4: 4.0}
CALLS = ("quantize_x", "quantize_w", "quantize_dy", "cbf_im2col", "conv_fwd", "conv_bwd_data", "conv_bwd_weight")

# dram__bytes_read.sum + dram__bytes_write.sum of the main kernel of a call, per launch, from ncu captures summarised
# under profiles/ (captured on the workload named in the first field; `scale` = units of the bench workload per unit
# of the captured one, traffic being proportional to the units processed).
NCU_TRAFFIC = {
    # (bench workload, call): (captured workload, bytes per launch there, scale)
    ("cfg5_e4m3_k3s1_c512_hw56", "conv_fwd"): ("cfg5_e4m3_k3s1_c512_hw28", 117502208 + 356616960, 4.0),       # conv_tc_kernel<fwd>
    ("cfg5_e4m3_k3s1_c512_hw56", "conv_bwd_data"): ("cfg5_e4m3_k3s1_c512_hw28", 117229568 + 356492544, 4.0),  # conv_tc_kernel<bwd_data>
    ("cfg5_e4m3_k3s1_c512_hw56", "quantize_x"): ("cfg5_e4m3_k3s1_c512_hw28", 420059648 + 81590016, 4.0),      # quantize_tma_kernel
    ("cfg5_e4m3_k3s1_c512_hw56", "quantize_dy"): ("cfg5_e4m3_k3s1_c512_hw28", 423871488 + 81877248, 4.0),
    ("cfg5_e4m3_k3s1_c512_hw28", "conv_fwd"): ("cfg5_e4m3_k3s1_c512_hw28", 117502208 + 356616960, 1.0),
}


class _WorkloadTable(dict):
    """name -> layer; a "+ts16" / "+p6" suffix selects the number format / the storage, not the layer"""

    def __missing__(self, name):
        if name.endswith("+ts16") and name[:-5] in self:
            return self[name[:-5]]
        if name.endswith("+p6") and name[:-3] in self:
            return self[name[:-3]]
        raise KeyError(name)


def workloads():
    w = _WorkloadTable()
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


def touched_fraction(d):
    """Fraction of the input pixels that some (output pixel, tap) pair reads: 1 unless the stride exceeds the kernel."""
    ho, wo = inputs.out_hw(d)
    th = len({o * d.stride_h + k - d.pad_h for o in range(ho) for k in range(d.Kh)} & set(range(d.H)))
    tw = len({o * d.stride_w + k - d.pad_w for o in range(wo) for k in range(d.Kw)} & set(range(d.W)))
    return th * tw / float(d.H * d.W)


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
class Workload:
    """Device buffers and the seven calls of one layer step."""

    def __init__(self, name, layer, rank, dy_rounding="nearest", fp32_layout="nchw"):
        import torch

        from paper_2609_28358_b200 import mq

        self.name, self.layer = name, layer
        d = self.d = layer.desc
        self.fmts = fmts = tuple(PACKED6.get(f, f) if name.endswith("+p6") else f for f in (layer.fmt_x, layer.fmt_w, layer.fmt_dy))
        blk = self.block = mq.TS16 if name.endswith("+ts16") else mq.TILE32
        assert blk == mq.TILE32 or all(f == mq.E2M1 for f in fmts), "the paper's own format has E2M1 elements"
        roles = (mq.ROLE_X, mq.ROLE_W, mq.ROLE_DY)
        seed = layer.seed + 1000 * rank
        self.host = (inputs.make_x(d, seed, layer.x_kind), inputs.make_w(d, layer.seed, layer.w_kind), inputs.make_dy(d, seed, layer.dy_kind))
        src = self.src = [torch.from_numpy(t).cuda() for t in self.host]
        hwnc = fp32_layout == "hwnc"     # fp32 tensors in the channel-fastest order the convolution calls can emit when layers chain
        sl = ol = mq.HWNC if hwnc else mq.NCHW
        if hwnc:
            src = self.src = [src[0].permute(2, 3, 0, 1).contiguous(), src[1].permute(0, 2, 3, 1).contiguous(), src[2].permute(2, 3, 0, 1).contiguous()]
        q = self.q = [mq.empty_qtensor(d, r, f, block=blk) for r, f in zip(roles, fmts)]
        self.icb, self.isb = mq.im2col_sizes(d, fmts[0], blk)
        ic = torch.empty(self.icb, dtype=torch.uint8, device="cuda")
        isc = torch.empty(self.isb, dtype=torch.uint8, device="cuda")
        ho, wo = inputs.out_hw(d)
        self.y = y = torch.empty((ho, wo, d.N, d.C_out) if hwnc else (d.N, d.C_out, ho, wo), dtype=torch.float32, device="cuda")
        self.dx = dx = torch.empty((d.H, d.W, d.N, d.C_in) if hwnc else (d.N, d.C_in, d.H, d.W), dtype=torch.float32, device="cuda")
        self.dw = dw = torch.empty((d.C_out, d.Kh, d.Kw, d.C_in) if hwnc else (d.C_out, d.C_in, d.Kh, d.Kw), dtype=torch.float32, device="cuda")
        ws_bytes = max(mq.workspace_size(d, op, a, b, blk) for op, a, b in
                       ((mq.OP_FWD, fmts[0], fmts[1]), (mq.OP_BWD_DATA, fmts[1], fmts[2]), (mq.OP_BWD_WEIGHT, fmts[0], fmts[2])))
        self.ws = ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
        self.calls = [
            ("quantize_x", lambda: mq.quantize(d, roles[0], fmts[0], src[0], out=q[0], src_layout=sl, block=blk)),
            ("quantize_w", lambda: mq.quantize(d, roles[1], fmts[1], src[1], out=q[1], src_layout=sl, block=blk)),
            ("quantize_dy", (lambda: mq.quantize_sr(d, roles[2], fmts[2], src[2], 1234, out=q[2], src_layout=sl, block=blk)) if dy_rounding == "stochastic" else
             (lambda: mq.quantize(d, roles[2], fmts[2], src[2], out=q[2], src_layout=sl, block=blk))),
            ("cbf_im2col", lambda: mq.cbf_im2col(d, q[0], ic, isc)),
            ("conv_fwd", lambda: mq.conv_fwd(d, q[0], q[1], y=y, layout=ol, workspace=ws)),
            ("conv_bwd_data", lambda: mq.conv_bwd_data(d, q[1], q[2], dx=dx, layout=ol, workspace=ws)),
            ("conv_bwd_weight", lambda: mq.conv_bwd_weight(d, q[0], q[2], dw=dw, layout=ol, workspace=ws)),
        ]

    def step(self):
        for _, fn in self.calls:
            fn()

    def algorithmic_bytes(self):
        """Bytes each call must move (what the method itself reads and writes, each byte once)."""
        d, q = self.d, self.q
        x, w, g = self.host
        qb = [float(t.codes.numel() + t.scales.numel()) for t in q]
        tf = touched_fraction(d)
        return {
            "quantize_x": 4.0 * x.size + qb[0], "quantize_w": 4.0 * w.size + qb[1], "quantize_dy": 4.0 * g.size + qb[2],
            "cbf_im2col": tf * qb[0] + self.icb + self.isb,
            "conv_fwd": tf * qb[0] + qb[1] + 4.0 * self.y.numel(),
            "conv_bwd_data": qb[1] + qb[2] + 4.0 * self.dx.numel(),
            "conv_bwd_weight": qb[2] + tf * qb[0] + 4.0 * self.dw.numel(),
        }

    def gemm_bits(self):
        f = self.fmts
        return {"conv_fwd": max(FMT_BITS[f[0]], FMT_BITS[f[1]]), "conv_bwd_data": max(FMT_BITS[f[1]], FMT_BITS[f[2]]),
                "conv_bwd_weight": max(FMT_BITS[f[0]], FMT_BITS[f[2]])}


def fused_epilogue_times(wl, flush, K, kern, pk):
    """mq_conv_fwd_mx (ReLU, emitting the next layer's activation tensor in X's format) and mq_conv_bwd_data_mx (emitting the
    previous layer's gradient tensor in dY's format) on the workload's quantized operands."""
    import torch

    from paper_2609_28358_b200 import mq

    d, q, f = wl.d, wl.q, wl.fmts
    if wl.block == mq.TS16:
        # the paper's own format: mq_conv_fwd_ts / mq_conv_bwd_data_ts, the emitted tensors' maxima supplied (here: the true ones,
        # taken from the fp32 outputs of the step that has just run, as an earlier step's statistics would be)
        am_y = wl.y.abs().max().reshape(1).float()
        am_dx = wl.dx.abs().max().reshape(1).float()
        ws = torch.empty(max(mq.conv_ts_workspace_size(d, mq.OP_FWD), mq.conv_ts_workspace_size(d, mq.OP_BWD_DATA), 16), dtype=torch.uint8, device="cuda")
        yq = mq.conv_fwd_ts(d, q[0], q[1], am_y, mq.ACT_RELU, workspace=ws)
        dxq = mq.conv_bwd_data_ts(d, q[1], q[2], am_dx, workspace=ws)
        calls = {"conv_fwd_ts": (lambda: mq.conv_fwd_ts(d, q[0], q[1], am_y, mq.ACT_RELU, yq=yq, workspace=ws), "conv_fwd", 4),
                 "conv_bwd_data_ts": (lambda: mq.conv_bwd_data_ts(d, q[1], q[2], am_dx, dxq=dxq, workspace=ws), "conv_bwd_data", 4)}
    else:
        ws = torch.empty(max(mq.conv_mx_workspace_size(d, mq.OP_FWD, f[0], f[1]), mq.conv_mx_workspace_size(d, mq.OP_BWD_DATA, f[1], f[2]), 16),
                         dtype=torch.uint8, device="cuda")
        yq = mq.conv_fwd_mx(d, q[0], q[1], f[0], mq.ACT_RELU, workspace=ws)
        dxq = mq.conv_bwd_data_mx(d, q[1], q[2], f[2], workspace=ws)
        calls = {"conv_fwd_mx": (lambda: mq.conv_fwd_mx(d, q[0], q[1], f[0], mq.ACT_RELU, yq=yq, workspace=ws), "conv_fwd", max(FMT_BITS[f[0]], FMT_BITS[f[1]])),
                 "conv_bwd_data_mx": (lambda: mq.conv_bwd_data_mx(d, q[1], q[2], f[2], dxq=dxq, workspace=ws), "conv_bwd_data", max(FMT_BITS[f[1]], FMT_BITS[f[2]]))}
    res = {}
    for name, (fn, plain, bits) in calls.items():
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for s, e in ev:
            flush.zero_()
            s.record()
            fn()
            e.record()
        torch.cuda.synchronize()
        ms = sum(s.elapsed_time(e) for s, e in ev) / K
        tf = layer_flops(d) / (ms * 1e-3) / 1e12
        peak = pk["bf16_tflops"] * TENSOR_RATIO[bits]
        res[name] = {"ms": ms, "tflops": tf, "frac": tf / peak, "frac_of_published": tf / PUBLISHED["tensor_tflops"][bits],
                     "fp32_output_call_ms": kern[plain]["ms"], "activation": "relu" if plain == "conv_fwd" else "none",
                     "emits": FMT_NAME[f[0] if plain == "conv_fwd" else f[2]] + (" (16x16 blocks, E4M3 scales, supplied maximum)" if wl.block == mq.TS16 else "")}
    if wl.block == mq.TS16:
        # the quantizer itself with the maximum supplied (Sec. VII-B): one pass that also records the tensor's own maximum
        src = wl.src[0]
        sl = mq.HWNC if tuple(src.shape) != (d.N, d.C_in, d.H, d.W) else mq.NCHW
        am_x = src.abs().max().reshape(1).float()
        fn = lambda: mq.quantize_ts(d, mq.ROLE_X, src, out=q[0], src_layout=sl, amax_in=am_x)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for s, e in ev:
            flush.zero_()
            s.record()
            fn()
            e.record()
        torch.cuda.synchronize()
        ms = sum(s.elapsed_time(e) for s, e in ev) / K
        nbytes = wl.algorithmic_bytes()["quantize_x"]
        res["quantize_x_supplied_maximum"] = {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "frac": nbytes / (ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                                              "own_maximum_call_ms": kern["quantize_x"]["ms"]}
    res["device_status"] = mq.last_device_status()
    return res


def time_per_call(wl, flush, K):
    """Mean duration of each call over K steps (CUDA events on the launching stream, L2 flushed before each step) and
    the number of kernels each call launches (the library's own count)."""
    import torch

    from paper_2609_28358_b200 import mq

    per = {n: [] for n, _ in wl.calls}
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(len(wl.calls) + 1)] for _ in range(K)]
    for m in marks:
        flush.zero_()
        m[0].record()
        for i, (_, fn) in enumerate(wl.calls):
            fn()
            m[i + 1].record()
    torch.cuda.synchronize()
    for m in marks:
        for i, (n, _) in enumerate(wl.calls):
            per[n].append(m[i].elapsed_time(m[i + 1]))
    n_launch = {}
    for n, fn in wl.calls:
        c0 = mq.kernel_launch_count()
        fn()
        n_launch[n] = max(1, mq.kernel_launch_count() - c0)
    torch.cuda.synchronize()
    return {n: float(np.mean(v)) for n, v in per.items()}, n_launch


def roofline_table(wl, ms, n_launch, pk):
    """Per call: the binding roof (HBM for quantize / im2col; for a GEMM the slower of tensor time and HBM time of its
    algorithmic bytes), the achieved rate, its fraction of the measured roof and of the published one."""
    d = wl.d
    alg = wl.algorithmic_bytes()
    bits = wl.gemm_bits()
    kern = {}
    for n in CALLS:
        t = ms[n] * 1e-3
        if n in bits:
            peak_t = pk["bf16_tflops"] * TENSOR_RATIO[bits[n]]
            tensor_bound = layer_flops(d) / (peak_t * 1e12) >= alg[n] / (pk["hbm_gbs"] * 1e9)
        else:
            tensor_bound = False
        if tensor_bound:
            ach = layer_flops(d) / t / 1e12
            kern[n] = {"ms": ms[n], "bound": "tensor", "achieved": ach, "peak": peak_t, "unit": "TFLOP/s", "frac": ach / peak_t,
                       "frac_of_published": ach / PUBLISHED["tensor_tflops"][bits[n]]}
        else:
            ach = alg[n] / t / 1e9
            kern[n] = {"ms": ms[n], "bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                       "frac_of_published": ach / PUBLISHED["hbm_gbs"]}
        if n in bits:
            kern[n]["tflops"] = layer_flops(d) / t / 1e12
        kern[n]["launches"] = n_launch[n]
        kern[n]["algorithmic_bytes"] = alg[n]
    qi = ("quantize_x", "quantize_w", "quantize_dy", "cbf_im2col")
    qi_gbs = sum(alg[n] for n in qi) / (sum(ms[n] for n in qi) * 1e-3) / 1e9
    return kern, {"value": qi_gbs, "frac_of_hbm_peak": qi_gbs / pk["hbm_gbs"], "frac_of_published": qi_gbs / PUBLISHED["hbm_gbs"]}


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

    all_wl = workloads()
    wl = Workload(args.workload, all_wl[args.workload], rank, args.dy_rounding, args.fp32_layout)
    d, fmts = wl.d, wl.fmts
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")  # > 126 MB L2

    def step():
        wl.step()
        if world > 1:
            dist.all_reduce(wl.dw)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()

    # ---- timed region: K steps, L2 flushed between steps (flush outside the event pairs)
    K = args.steps
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    barrier()
    launches0 = mq.kernel_launch_count()
    for s, e in ev:
        flush.zero_()
        s.record()
        step()
        e.record()
    barrier()
    launches = mq.kernel_launch_count() - launches0   # kernels of this library inside the timed region
    ms_total = sum(s.elapsed_time(e) for s, e in ev)

    # ---- per-call durations over K more steps (same stream, same flush), for the roofline
    per_ms, n_launch = time_per_call(wl, flush, K)
    dev_status = mq.last_device_status()

    # ---- end to end: pinned host buffers through mq_conv_layer_host, copies inside the timed region
    hx, hw_, hg = [torch.from_numpy(t).pin_memory() for t in wl.host]
    hy = torch.empty(wl.y.shape, dtype=torch.float32).pin_memory()
    hdx = torch.empty(wl.dx.shape, dtype=torch.float32).pin_memory()
    hdw = torch.empty(wl.dw.shape, dtype=torch.float32).pin_memory()
    arena = torch.empty(mq.conv_layer_host_arena_size(d, *fmts), dtype=torch.uint8, device="cuda")
    Ke = max(3, min(K, 10))
    for _ in range(2):
        mq.conv_layer_host(d, fmts, hx, hw_, hg, hy, hdx, hdw, arena)
    barrier()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(Ke):
        mq.conv_layer_host(d, fmts, hx, hw_, hg, hy, hdx, hdw, arena)   # per-rank gradients; the reduction is the device path's
    t1.record()
    barrier()
    e2e_ms = t0.elapsed_time(t1) / Ke
    clocks = sampler.result()
    del arena, hx, hg, hy, hdx

    if world > 1:
        t = torch.tensor([ms_total, e2e_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total, e2e_ms = float(t[0]), float(t[1])

    flops = 3.0 * layer_flops(d) * world
    ms_step = ms_total / K
    value = flops / (ms_step * 1e-3) / 1e12

    # ---- roofline of the dominant kernel
    pk, pk_src = peaks()
    kern, qi = roofline_table(wl, per_ms, n_launch, pk)
    # the dominant kernel = the main kernel of the call that takes longest (a GEMM call's other launch, the expansion of its
    # scale chunks, is a few microseconds; the call's whole time is charged to the main kernel)
    dom = max(CALLS, key=lambda n: kern[n]["ms"])
    roof = {k: kern[dom][k] for k in ("bound", "achieved", "peak", "unit", "frac", "frac_of_published")}
    traffic = NCU_TRAFFIC.get((args.workload, dom))
    roof.update({"kernel": dom,
                 "peak_source": pk_src + (" bf16 burst x%g (nominal ratio)" % TENSOR_RATIO[wl.gemm_bits()[dom]] if roof["bound"] == "tensor" else " copy bandwidth"),
                 "traffic": None if traffic is None else traffic[1] * traffic[2],
                 "traffic_source": None if traffic is None else "ncu on %s, x%g" % (traffic[0], traffic[2])})

    out = {
        "metric": "MX conv fwd+bwd TFLOPS (whole layer step: quantize x3 + CBF-im2col + fwd + dX + dW)",
        "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "+".join(FMT_NAME[f] for f in fmts) + " (fp32 accumulate)", "data": "synthetic",
        "config": {"workload": args.workload, "layer": dict(d._asdict()), "formats": [FMT_NAME[f] for f in fmts], "dy_rounding": args.dy_rounding, "fp32_layout": args.fp32_layout,
                   "global_batch": d.N * world, "parallelism": "dp%d" % world if world > 1 else "single", "l2": "flushed between steps (512 MiB write)"},
        "clocks": clocks,
        "e2e": {"value": flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOPS", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(sum(t.size for t in wl.host) * 4), "d2h_bytes_per_step": int((wl.y.numel() + wl.dx.numel() + wl.dw.numel()) * 4)},
        "gpu_launches": launches,
        "roofline": roof,
        "quantize_im2col_gbs": qi,
        "kernels": kern,
        "device_status": dev_status,
    }

    # ---- the two GEMMs with the quantizing producer epilogue (the next tensor leaves the chip in its stored MX form instead of
    # fp32): per-call times beside the fp32-output calls and the quantizer call they replace
    if world == 1 and not any(f in PACKED6.values() for f in fmts):   # (the quantizing epilogue does not emit packed 6-bit storage)
        out["fused_epilogue"] = fused_epilogue_times(wl, flush, max(3, min(K, 10)), kern, pk)

    # ---- the same step on further workloads (device-timed step and per-call roofline only)
    more = [] if args.more == "none" else [m for m in args.more.split(",") if m and m != args.workload]
    if world == 1 and more:
        del wl
        torch.cuda.empty_cache()
        out["more_workloads"] = {}
        Km = max(3, min(K, 20))
        for name in more:
            w2 = Workload(name, all_wl[name], rank, args.dy_rounding, args.fp32_layout)
            for _ in range(3):
                w2.step()
            torch.cuda.synchronize()
            ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(Km)]
            for s, e in ev2:
                flush.zero_()
                s.record()
                w2.step()
                e.record()
            torch.cuda.synchronize()
            ms2 = sum(s.elapsed_time(e) for s, e in ev2) / Km
            per2, nl2 = time_per_call(w2, flush, Km)
            k2, qi2 = roofline_table(w2, per2, nl2, pk)
            out["more_workloads"][name] = {
                "layer": dict(w2.d._asdict()), "formats": [FMT_NAME[f] for f in w2.fmts],
                "blocks": "16x16, E4M3 block scale, fp32 tensor scale" if name.endswith("+ts16") else "32x32, E8M0 scale", "steps": Km, "ms_per_step": ms2,
                "value": 3.0 * layer_flops(w2.d) / (ms2 * 1e-3) / 1e12, "unit": "TFLOPS", "quantize_im2col_gbs": qi2,
                "kernels": {n: {k: v for k, v in k2[n].items() if k != "algorithmic_bytes"} for n in CALLS},
                "device_status": mq.last_device_status()}
            if name.endswith("+ts16"):
                out["more_workloads"][name]["fused_epilogue"] = fused_epilogue_times(w2, flush, max(3, min(Km, 10)), k2, pk)
            del w2
            torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_accounting:
        out["quantization_accounting"] = quantization_accounting(all_wl[args.workload], flush)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(all_wl[args.workload], budget_s=args.cpu_budget)
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def quantization_accounting(layer, flush, reps=5):
    """Measured counterpart of the paper's Table I (Sec. IV-C) on one layer: elements that pass through a quantizer per
    forward + backward step, bytes those quantizer calls move, their time, and the bytes of activation kept for the
    backward pass - for this library's path and for two stand-ins built from the library's own kernels:
      square_blocks_once          X, W, G_Y quantized once each in 32 x 32 blocks (usable by both of their GEMMs); Q(X) kept;
      line_blocks_expanded_twice  the scheme the paper compares with first: one-directional (line) blocks on the im2col-EXPANDED
                                  activation, quantized for the forward pass and again, in the other direction, for the
                                  backward pass (the library's line quantizer stands in for that second direction at the same
                                  element count), W and G_Y likewise twice; the fp32 activation is what is kept;
      square_blocks_on_expanded   the second comparison: the expanded activation quantized once in square blocks and kept.
    The expanded fp32 matrix X' is produced by torch's unfold (glue, not timed).  Every count is the numel of a tensor
    actually handed to mq_quantize; bytes are the sizes of the buffers those calls read and wrote."""
    import torch
    import torch.nn.functional as F

    from paper_2609_28358_b200 import mq

    d = layer.desc
    fmts = (layer.fmt_x, layer.fmt_w, layer.fmt_dy)
    ho, wo = inputs.out_hw(d)
    x, w, g = [torch.from_numpy(t).cuda() for t in (inputs.make_x(d, layer.seed, layer.x_kind), inputs.make_w(d, layer.seed, layer.w_kind),
                                                     inputs.make_dy(d, layer.seed, layer.dy_kind))]
    xe = F.unfold(x, (d.Kh, d.Kw), padding=(d.pad_h, d.pad_w), stride=(d.stride_h, d.stride_w)).reshape(d.N, d.C_in * d.Kh * d.Kw, ho, wo).contiguous()
    de = d._replace(C_in=d.C_in * d.Kh * d.Kw, H=ho, W=wo, Kh=1, Kw=1, stride_h=1, stride_w=1, pad_h=0, pad_w=0)   # X' as a 1x1 layer's input

    def run(calls):
        """calls: (desc, role, fmt, tensor, block); returns elements, bytes moved, ms per pass, size of the first call's stored tensor."""
        outs = [mq.empty_qtensor(dd, r, f, block=b) for dd, r, f, t, b in calls]
        fns = [lambda dd=dd, r=r, f=f, t=t, o=o, b=b: mq.quantize(dd, r, f, t, out=o, block=b) for (dd, r, f, t, b), o in zip(calls, outs)]
        for fn in fns:
            fn()
        torch.cuda.synchronize()
        ms = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for fn in fns:
                fn()
            e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        elems = sum(t.numel() for _, _, _, t, _ in calls)
        moved = sum(4 * t.numel() for _, _, _, t, _ in calls) + sum(o.codes.numel() + o.scales.numel() for o in outs)
        return elems, moved, float(np.median(ms)), outs[0].codes.numel() + outs[0].scales.numel()

    T, L = mq.TILE32, mq.LINE32
    ours = run([(d, 0, fmts[0], x, T), (d, 1, fmts[1], w, T), (d, 2, fmts[2], g, T)])
    line2 = run([(de, 0, fmts[0], xe, L), (d, 1, fmts[1], w, L), (d, 2, fmts[2], g, L)] * 2)
    sq_e = run([(de, 0, fmts[0], xe, T), (d, 1, fmts[1], w, T), (d, 2, fmts[2], g, T)])
    res = {
        "layer": dict(d._asdict()), "formats": [FMT_NAME[f] for f in fmts],
        "square_blocks_once": {"quantized_elements": ours[0], "quantizer_bytes_moved": ours[1], "quantizer_ms": ours[2], "activation_kept_bytes": ours[3]},
        "line_blocks_expanded_twice": {"quantized_elements": line2[0], "quantizer_bytes_moved": line2[1], "quantizer_ms": line2[2],
                                       "activation_kept_bytes": 4 * x.numel()},
        "square_blocks_on_expanded": {"quantized_elements": sq_e[0], "quantizer_bytes_moved": sq_e[1], "quantizer_ms": sq_e[2],
                                      "activation_kept_bytes": sq_e[3]},
    }
    res["activation_elements_ratio"] = {"line_blocks_expanded_twice": 2.0 * xe.numel() / x.numel(), "square_blocks_on_expanded": xe.numel() / x.numel()}
    res["activation_kept_ratio"] = {"line_blocks_expanded_twice": 4.0 * x.numel() / ours[3], "square_blocks_on_expanded": sq_e[3] / ours[3]}
    return res


# ----------------------------------------------------------------------------------- CPU oracle
def oracle_step(layer, ns, tensors=None):
    """One pass of the whole path in the oracle on the first `ns` samples of the layer's batch."""
    import oracle

    d0 = layer.desc
    d = d0._replace(N=ns)
    x, w, g = tensors if tensors is not None else sample_tensors(layer, ns)
    t0 = time.perf_counter()
    fm = (layer.fmt_x, layer.fmt_w, layer.fmt_dy)
    q = [oracle.quantize(d, r, f, t) for r, f, t in zip((0, 1, 2), fm, (x[:ns], w, g[:ns]))]
    oracle.cbf_im2col(d, fm[0], *q[0])
    xh, wh, gh = [oracle.dequant(d, r, f, c, s) for r, f, (c, s) in zip((0, 1, 2), fm, q)]
    oracle.conv_fwd(d, xh, wh)
    oracle.conv_bwd_data(d, wh, gh)
    oracle.conv_bwd_weight(d, gh, xh)
    return time.perf_counter() - t0, 3.0 * layer_flops(d)


def sample_tensors(layer, ns):
    """The layer's tensors restricted to a batch of `ns` samples (same distributions; the sample's own draws)."""
    d = layer.desc._replace(N=ns)
    return (inputs.make_x(d, layer.seed, layer.x_kind), inputs.make_w(d, layer.seed, layer.w_kind), inputs.make_dy(d, layer.seed, layer.dy_kind))


def pick_sample(layer, budget_s):
    import oracle

    oracle.build()
    t1, _ = oracle_step(layer, 1)
    return int(max(1, min(layer.desc.N, budget_s / max(t1, 1e-3))))


def cpu_baseline(layer, budget_s=15.0):
    import oracle

    ns = pick_sample(layer, budget_s)
    t, fl = oracle_step(layer, ns)
    return {"value": fl / t / 1e12, "unit": "TFLOPS", "cores": oracle.num_threads(), "kind": "oracle", "seconds": t,
            "sample": f"a batch of {ns} samples of the layer instead of {layer.desc.N} (TFLOPS is a rate: the full batch would take "
                      f"about x{layer.desc.N / ns:.0f} as long), whole path (quantize x3, im2col, fwd, dX, dW) in the fp64 oracle"}


def run_reference(args):
    import oracle

    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    layer = workloads()[args.workload]
    K, W = args.steps, max(args.warmup, 0)
    ns = pick_sample(layer, 150.0 / (K + W + 1))
    tensors = sample_tensors(layer, ns)
    for _ in range(W):
        oracle_step(layer, ns, tensors)
    t = 0.0
    fl = 0.0
    for _ in range(K):
        dt, f = oracle_step(layer, ns, tensors)
        t += dt
        fl += f
    value = fl / t / 1e12
    d = layer.desc
    fmts = (layer.fmt_x, layer.fmt_w, layer.fmt_dy)
    sample = f"a batch of {ns} samples of the layer instead of {d.N} per step, whole path in the fp64 oracle"
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
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--more", default=",".join(MORE_WORKLOADS), help="further workloads timed after the main one (comma-separated, or 'none')")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-accounting", action="store_true", help="skip the measured Table-I style quantization accounting")
    ap.add_argument("--dy-rounding", default="nearest", choices=["nearest", "stochastic"],
                    help="rounding of the gradient's quantizer in the device-timed step (the host-buffer call keeps nearest)")
    ap.add_argument("--fp32-layout", default="nchw", choices=["nchw", "hwnc"],
                    help="order of the fp32 tensors in the device-timed step: NCHW / OIHW (the layout of record) or channel-fastest [H][W][N][C] / [Cout][Kh][Kw][Cin]")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
