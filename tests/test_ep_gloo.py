"""The expert-parallel partitioning on CPU: `gloo` ranks (world 2 and 4) exchange slabs with
all_to_all_single exactly as the GPU path does, with the slab sizes and the regrouping permutation
taken from the library's own host functions (gshard_moe_ep_plan, gshard_moe_ep_regroup_host - the
same index arithmetic as the device-side regroup).  Each rank routes its own groups and evaluates
its own experts with the oracle; the reassembled routing and y must equal the oracle's single-process
result for the whole layer bit for bit, and the backward, walked back through the same exchanges
(gshard_moe_top2_backward_ep's data flow), the oracle's gradients."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2006_16668_b200 import MoEConfig, make_inputs        # noqa: E402
from paper_2006_16668_b200 import binding as B                  # noqa: E402
from paper_2006_16668_b200.build import build_library           # noqa: E402

CFG = MoEConfig("ep_cpu", G=8, S=40, M=16, H=24, E=12, C=5, dtype="f32", seed=77, backward=True, k_aux=0.01)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_forward(rank, world, inp):
    """What gshard_moe_top2_forward_ep does on one rank, with the oracle in place of the kernels and
    CPU tensors in place of device buffers; returns this rank's (expert_idx, slot, y, l_aux share)."""
    from oracle import gshard_oracle as orc
    cfg = CFG
    shape = B.make_shape(cfg)
    lay = B.gshard_moe_ep_plan(shape, rank, world)
    gs = slice(lay.group_begin, lay.group_begin + lay.groups_local)
    es = slice(lay.expert_begin, lay.expert_begin + lay.experts_local)
    x = inp["x"][gs].numpy()
    u = inp["u"][gs].numpy()
    wg = inp["wg"].numpy()
    Gl, El, C, M, E = lay.groups_local, lay.experts_local, cfg.C, cfg.M, cfg.E
    assert lay.rows_local == Gl * C and lay.bytes_per_peer == El * Gl * C * M * 4
    # 1. gating + Algorithm 1 over the local groups
    f = orc.forward(x, wg, None, None, u, C, want_y=False)
    # 2. dispatch into the send buffer [E, Gl*C, M] (fp64 rows here: the exchange moves bytes)
    send = torch.zeros(E, Gl * C, M, dtype=torch.float64)
    for e in range(E):
        for g in range(Gl):
            for c in range(C):
                s = f.slot_token[e, g, c]
                if s >= 0:
                    send[e, g * C + c] = torch.from_numpy(x[g, s].astype(np.float64))
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send)                         # slab d of send -> rank d
    ffn_in = torch.empty_like(recv)
    B.gshard_moe_ep_regroup_host(lay, recv, ffn_in)            # [W][El][rows] -> [El][W*rows]
    ffn_in = ffn_in.view(El, world * Gl * C, M)
    # 3. the local experts over all groups' rows
    ffn_out = torch.zeros_like(ffn_in)
    wi, wo = inp["wi"][es].numpy(), inp["wo"][es].numpy()
    for el in range(El):
        rows = ffn_in[el].numpy()
        filled = np.abs(rows).sum(axis=1) > 0
        if filled.any():
            out = orc.ffn_rows(rows[filled].astype(np.float32), wi[el], wo[el])
            ffn_out[el][torch.from_numpy(filled)] = torch.from_numpy(out)
    # 4. back: inverse regroup, AllToAll
    back = torch.empty_like(recv)
    B.gshard_moe_ep_regroup_host(lay, ffn_out.view_as(recv).contiguous(), back, inverse=True)
    out_local = torch.empty_like(send)
    dist.all_to_all_single(out_local, back)
    # 5. combine (eq. (3)) in the oracle's order: first choice, then second
    y = np.zeros((Gl, cfg.S, M))
    for g in range(Gl):
        for s in range(cfg.S):
            for k in range(2):
                pos = f.slot[g, s, k]
                if pos >= 0:
                    y[g, s] += f.weight[g, s, k] * out_local[f.expert_idx[g, s, k], g * C + pos].numpy()
    l_share = torch.tensor([f.l_aux_group.sum() / cfg.G])
    dist.all_reduce(l_share)
    state = dict(f=f, lay=lay, x=x, wg=wg, wi=wi, wo=wo, ffn_in=ffn_in, out_local=out_local, gs=gs)
    return f.expert_idx, f.slot, y, float(l_share), state


def _rank_backward(rank, world, inp, st):
    """What gshard_moe_top2_backward_ep does on one rank, again with the oracle's per-row and per-token
    routines in place of the kernels: combine backward over the local groups, AllToAll + regroup of the
    expert-output gradients, expert FFN backward over the local experts, the way back for the
    expert-input gradients, gating backward over the local groups, all-reduce of dwg."""
    from oracle import gshard_oracle as orc
    cfg, f, lay = CFG, st["f"], st["lay"]
    x, wg, wi, wo = st["x"], st["wg"], st["wi"], st["wo"]
    Gl, El, C, M, E, S = lay.groups_local, lay.experts_local, cfg.C, cfg.M, cfg.E, cfg.S
    dy = inp["dy"][st["gs"]].numpy().astype(np.float64)
    out_local = st["out_local"].numpy()
    # 1. combine backward: dw per choice, dout per slot (local layout [E, Gl*C, M])
    dw = np.zeros((Gl, S, 2))
    dout = torch.zeros(E, Gl * C, M, dtype=torch.float64)
    for g in range(Gl):
        for s in range(S):
            for k in range(2):
                pos = f.slot[g, s, k]
                if pos >= 0:
                    e = f.expert_idx[g, s, k]
                    dw[g, s, k] = float(dy[g, s] @ out_local[e, g * C + pos])
                    dout[e, g * C + pos] = torch.from_numpy(f.weight[g, s, k] * dy[g, s])
    # 2. to the experts' owners
    recv = torch.empty_like(dout)
    dist.all_to_all_single(recv, dout)
    dout_ffn = torch.empty_like(recv)
    B.gshard_moe_ep_regroup_host(lay, recv, dout_ffn)
    dout_ffn = dout_ffn.view(El, world * Gl * C, M)
    # 3. expert FFN backward over the local experts (rows of all groups)
    ffn_in = st["ffn_in"]
    dbuf_ffn = torch.zeros_like(ffn_in)
    dwi = np.zeros((El, M, cfg.H))
    dwo = np.zeros((El, cfg.H, M))
    for el in range(El):
        rows = ffn_in[el].numpy()
        filled = np.abs(rows).sum(axis=1) > 0
        if filled.any():
            dxr, dwi[el], dwo[el] = orc.ffn_rows_backward(rows[filled].astype(np.float32), dout_ffn[el].numpy()[filled],
                                                          wi[el], wo[el])
            dbuf_ffn[el][torch.from_numpy(filled)] = torch.from_numpy(dxr)
    # 4. back to the groups' owners
    back = torch.empty_like(recv)
    B.gshard_moe_ep_regroup_host(lay, dbuf_ffn.view_as(recv).contiguous(), back, inverse=True)
    dbuf = torch.empty_like(dout)
    dist.all_to_all_single(dbuf, back)
    dbuf = dbuf.numpy()
    # 5. gating backward and dx over the local groups (l_aux averages over the GLOBAL group count)
    dx = np.zeros((Gl, S, M))
    dwg = np.zeros((M, E))
    for g in range(Gl):
        _, p = orc.gates(x[g], wg)
        for s in range(S):
            e1, e2 = f.expert_idx[g, s]
            dl = orc.gate_row_backward(p[s], e1, e2, dw[g, s, 0], dw[g, s, 1], f.first_count[g], S, cfg.G, cfg.k_aux)
            dwg += np.outer(x[g, s].astype(np.float64), dl)
            dx[g, s] = wg.astype(np.float64) @ dl
            for k in range(2):
                pos = f.slot[g, s, k]
                if pos >= 0:
                    dx[g, s] += dbuf[f.expert_idx[g, s, k], g * C + pos]
    dwg_t = torch.from_numpy(dwg)
    dist.all_reduce(dwg_t)                                     # wg is replicated: its gradient is the sum over ranks
    return dx, dwg_t.numpy(), dwi, dwo


def _worker(rank, world, port, out_dir):
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    inp = make_inputs(CFG, "cpu")
    ei, slot, y, l_aux, state = _rank_forward(rank, world, inp)
    dx, dwg, dwi, dwo = _rank_backward(rank, world, inp, state)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), ei=ei, slot=slot, y=y, l_aux=l_aux, dx=dx, dwg=dwg, dwi=dwi,
             dwo=dwo)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_expert_parallel_partitioning_matches_single_process(world, tmp_path):
    from oracle import gshard_oracle as orc
    build_library()
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    inp = make_inputs(CFG, "cpu")
    ref = orc.forward(inp["x"].numpy(), inp["wg"].numpy(), inp["wi"].numpy(), inp["wo"].numpy(), inp["u"].numpy(), CFG.C)
    parts = [np.load(os.path.join(str(tmp_path), f"rank{r}.npz")) for r in range(world)]
    assert np.array_equal(np.concatenate([p["ei"] for p in parts]), ref.expert_idx)
    assert np.array_equal(np.concatenate([p["slot"] for p in parts]), ref.slot)
    y = np.concatenate([p["y"] for p in parts])
    assert np.array_equal(y, ref.y), "reassembled y differs from the single-process oracle"
    assert (ref.slot >= 0).any() and (ref.slot < 0).any()
    for p in parts:
        assert float(p["l_aux"]) == pytest.approx(ref.l_aux, rel=1e-12)
    # the backward, partitioned the same way, against the oracle's single-process gradients (fp64
    # throughout; only the order of the sums differs)
    rdx, rdwg, rdwi, rdwo = orc.backward(inp["x"].numpy(), inp["wg"].numpy(), inp["wi"].numpy(), inp["wo"].numpy(), ref,
                                         inp["dy"].numpy(), CFG.k_aux)
    np.testing.assert_allclose(np.concatenate([p["dx"] for p in parts]), rdx, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(np.concatenate([p["dwi"] for p in parts]), rdwi, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(np.concatenate([p["dwo"] for p in parts]), rdwo, rtol=1e-10, atol=1e-12)
    for p in parts:
        np.testing.assert_allclose(p["dwg"], rdwg, rtol=1e-10, atol=1e-12)
    assert np.abs(rdwg).max() > 0 and np.abs(rdwi).max() > 0


def test_plan_arithmetic_and_rejections():
    build_library()
    shape = B.make_shape(G=8, S=64, M=64, H=128, E=16, C=8, dtype="bf16")
    lay = B.gshard_moe_ep_plan(shape, 3, 4)
    assert (lay.groups_local, lay.experts_local, lay.group_begin, lay.expert_begin) == (2, 4, 6, 12)
    assert lay.rows_local == 16 and lay.row_bytes == 128 and lay.bytes_per_peer == 4 * 16 * 128
    assert (lay.local.G, lay.local.E, lay.ffn.G, lay.ffn.E) == (2, 16, 8, 4)
    assert B.gshard_moe_ep_workspace_bytes(shape, 4) > 0
    for rank, world, code in [(0, 3, B.GSHARD_ERR_UNSUPPORTED_SHAPE), (4, 4, B.GSHARD_ERR_INVALID_ARG),
                              (-1, 2, B.GSHARD_ERR_INVALID_ARG), (0, 0, B.GSHARD_ERR_INVALID_ARG)]:
        with pytest.raises(B.GshardError) as e:
            B.gshard_moe_ep_plan(shape, rank, world)
        assert e.value.code == code
    assert B.gshard_moe_ep_workspace_bytes(shape, 3) == 0
    # the regroup permutation and its inverse: every row lands where the index rule says, and back
    rows = lay.world * lay.experts_local * lay.rows_local
    src = torch.arange(rows * 4, dtype=torch.int32).view(rows, 4)
    dst, back = torch.empty_like(src), torch.empty_like(src)
    B.gshard_moe_ep_regroup_host(lay, src, dst)
    B.gshard_moe_ep_regroup_host(lay, dst, back, inverse=True)
    assert torch.equal(back, src)
    v = dst.view(lay.experts_local, lay.world, lay.rows_local, 4)
    s = src.view(lay.world, lay.experts_local, lay.rows_local, 4)
    assert torch.equal(v, s.transpose(0, 1))
