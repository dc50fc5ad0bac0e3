"""The N>1 path on CPU: two gloo ranks, each holding a shard of the batch in units of 32 samples.

Checks what the data-parallel mode relies on: (1) a rank's quantized shard is bit-identical to the
corresponding slice of the single-rank quantization (no tile straddles two ranks), so forward and
input-gradient need no communication; (2) the weight gradient is the sum over ranks, i.e. one
all-reduce of the per-rank G_W reproduces the single-rank G_W."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from oracle import E4M3, E5M2, ROLE_DY, ROLE_X
from paper_2609_28358_b200 import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        oracle.build()
        d = inputs.conv_desc(64, 40, 6, 6, 48, 3, 1, 1)           # global batch 64 = 2 ranks x 32
        x, w, g = inputs.make_x(d, 3), inputs.make_w(d, 3), inputs.make_dy(d, 3, "gauss")
        nl = d.N // world
        dl = d._replace(N=nl)
        xs, gs = x[rank * nl:(rank + 1) * nl], g[rank * nl:(rank + 1) * nl]
        # (1) shard quantization == slice of the full quantization
        cx, sx = oracle.quantize(d, ROLE_X, E4M3, x)
        cxl, sxl = oracle.quantize(dl, ROLE_X, E4M3, xs)
        Cp = 64
        full_codes = cx.reshape(d.H * d.W, d.N, Cp)[:, rank * nl:(rank + 1) * nl]
        full_scales = sx.reshape(d.H * d.W, d.N // 32, Cp // 32)[:, rank * nl // 32:(rank + 1) * nl // 32]
        ok = np.array_equal(cxl.reshape(d.H * d.W, nl, Cp), full_codes) and np.array_equal(sxl.reshape(full_scales.shape), full_scales)
        # (2) all-reduce of the per-rank weight gradients == single-rank weight gradient
        cg, sg = oracle.quantize(dl, ROLE_DY, E5M2, gs)
        xh = oracle.dequant(dl, ROLE_X, E4M3, cxl, sxl)
        gh = oracle.dequant(dl, ROLE_DY, E5M2, cg, sg)
        gw, _ = oracle.conv_bwd_weight(dl, gh, xh)
        t = torch.from_numpy(gw)
        dist.all_reduce(t)
        if rank == 0:
            cgf, sgf = oracle.quantize(d, ROLE_DY, E5M2, g)
            gw_full, gwa = oracle.conv_bwd_weight(d, oracle.dequant(d, ROLE_DY, E5M2, cgf, sgf), oracle.dequant(d, ROLE_X, E4M3, cx, sx))
            ok = ok and bool((np.abs(t.numpy() - gw_full) <= 1e-12 * gwa + 1e-300).all())
        flag = torch.tensor([1 if ok else 0])
        dist.all_reduce(flag, op=dist.ReduceOp.MIN)
        if rank == 0:
            out.put(int(flag.item()))
    finally:
        dist.destroy_process_group()


def test_batch_sharding_and_weight_gradient_allreduce_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    assert out.get() == 1
