"""`bench.py --parallelism ep`: the expert-parallel forward timed over the ranks of a torchrun job.

The global layer is the configuration as given (total work fixed as ranks are added: strong
scaling); every rank draws its own groups and its own experts.  Timing as in the replica bench: CUDA
events on the launching stream between barriers, maximum over ranks."""
from __future__ import annotations

import json

import torch
import torch.distributed as dist

from . import binding as B
from . import ep
from .inputs import _normal


def run(args, cfg, dev, world, rank, metric, unit, sampler):
    train = bool(getattr(cfg, "backward", False))            # a training-step configuration: forward + backward
    shape = B.make_shape(cfg, flags=args.flags | (B.GSHARD_FLAG_SAVE_FOR_BACKWARD if train else 0))
    layout = B.gshard_moe_ep_plan(shape, rank, world)
    Gl, El, dt = layout.groups_local, layout.experts_local, cfg.torch_dtype
    gen = torch.Generator(device=dev).manual_seed(cfg.seed)              # wg is replicated: same draw everywhere
    wg = _normal((cfg.M, cfg.E), cfg.M ** -0.5, gen, dev, dt)
    gen.manual_seed(cfg.seed + 1000 + rank)                              # this rank's groups and experts
    x = _normal((Gl, cfg.S, cfg.M), 1.0, gen, dev, dt)
    u = torch.rand(Gl, cfg.S, generator=gen, device=dev, dtype=torch.float32)
    wi = _normal((El, cfg.M, cfg.H), cfg.M ** -0.5, gen, dev, dt)
    wo = _normal((El, cfg.H, cfg.M), cfg.H ** -0.5, gen, dev, dt)
    y = torch.empty_like(x)
    l_aux = torch.zeros(1, dtype=torch.float32, device=dev)
    ws = torch.empty(B.gshard_moe_ep_workspace_bytes(shape, world), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    # exchange: NCCL called from inside the library (default), torch.distributed through callbacks, or
    # fused into the dispatch and combine kernels (peer stores and loads on symmetric memory)
    mode = getattr(args, "ep_comm", "nccl")
    if train and mode == "p2p":
        raise SystemExit("--ep-comm p2p is the forward only; use nccl or torch for a training-step configuration")
    comm = ep.NcclComm(rank, world) if (world > 1 and mode in ("nccl", "p2p")) else None
    exchange = ep.SymmetricExchange(shape, rank, world) if mode == "p2p" else None
    if train:
        ctx = torch.empty(B.gshard_moe_ep_context_bytes(shape, world), dtype=torch.uint8, device=dev)
        wsb = torch.empty(B.gshard_moe_ep_backward_workspace_bytes(shape, world), dtype=torch.uint8, device=dev)
        dy = _normal((Gl, cfg.S, cfg.M), 1.0, gen, dev, dt)
        dx, dwi, dwo = torch.empty_like(x), torch.empty_like(wi), torch.empty_like(wo)
        dwg = torch.empty(cfg.M, cfg.E, dtype=torch.float32, device=dev)

    def step():
        if exchange is not None:
            ep.forward_p2p(shape, rank, world, x, wg, wi, wo, u, y, l_aux, exchange, None, ws, comm=comm)
        elif train:
            ep.forward(shape, rank, world, x, wg, wi, wo, u, y, l_aux, None, ws, comm=comm, context=ctx)
            ep.backward(shape, rank, world, x, wg, wi, wo, ctx, dy, cfg.k_aux, dx, dwg, dwi, dwo, wsb, comm=comm)
        else:
            ep.forward(shape, rank, world, x, wg, wi, wo, u, y, l_aux, None, ws, comm=comm)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    if B.gshard_moe_last_device_status(ws) != B.GSHARD_OK:
        raise SystemExit("device status is not OK after warm-up")
    launches = B.gshard_moe_last_launch_count()
    if train:                                                 # the counter restarts in every call: add the forward's
        ep.forward(shape, rank, world, x, wg, wi, wo, u, y, l_aux, None, ws, comm=comm, context=ctx)
        launches += B.gshard_moe_last_launch_count()
        barrier()
    sampler.start()
    sampler.wait_first_sample()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms = torch.tensor([e0.elapsed_time(e1) / args.steps], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    sampler.stop()
    status = B.gshard_moe_last_device_status(ws)
    if status != B.GSHARD_OK:
        raise SystemExit("device status is not OK after the timed steps")
    if rank == 0:
        ms_per_step = float(ms.item())
        line = {"metric": metric, "value": cfg.N / (ms_per_step * 1e-3), "unit": unit, "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
                "config": {"workload": cfg.name, "G": cfg.G, "S": cfg.S, "M": cfg.M, "H": cfg.H, "E": cfg.E, "C": cfg.C,
                           "parallelism": f"ep{world}: {Gl} groups and {El} experts per GPU, "
                                          f"{layout.bytes_per_peer} bytes per peer before and after the expert FFN, "
                                          + ("stored and loaded peer to peer by the dispatch and combine kernels"
                                             if exchange is not None else f"all-to-all ({mode})"),
                           "step": "forward + backward" if train else "forward", "l2": "inputs larger than L2"},
                "roofline": None, "cpu_baseline": None, "e2e": None, "gpu_launches": launches * args.steps,
                "clocks": sampler.summary(), "device_status": status}
        print(json.dumps(line))
