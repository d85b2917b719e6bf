"""Helpers of the GPU parity tests: the oracle's routing for one group with the near-tie
replay, and error measures.  Expected values always come from ``oracle/``; the CUDA path
only ever supplies the values under test."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from oracle import gshard_oracle as orc

MARGIN = 1e-6          # tokens whose oracle top-2 or random-routing margin is below this are
                       # excluded from the decision comparison (counted and reported)


def to_np(t: torch.Tensor) -> np.ndarray:
    """Exact float32 / integer numpy copy of a tensor (bf16 is widened, never re-rounded)."""
    t = t.detach()
    if t.dtype == torch.bfloat16:
        t = t.float()
    return t.cpu().numpy()


def rel_fro(got: np.ndarray, ref: np.ndarray) -> float:
    den = np.linalg.norm(ref.astype(np.float64).ravel())
    num = np.linalg.norm(got.astype(np.float64).ravel() - ref.astype(np.float64).ravel())
    return float(num / den) if den > 0 else float(num)


@dataclass
class GroupCheck:
    excluded: int            # |F|
    flips: int               # decisions inside F where the GPU differs from the oracle
    routing: orc.GroupRouting
    e1: np.ndarray
    e2: np.ndarray
    m: np.ndarray
    p: np.ndarray


def check_group_routing(x_g, wg, u_g, C, gpu_expert_idx, gpu_flags, variant_a=False) -> GroupCheck:
    """Oracle routing of one group, compared with the GPU's decisions under the replay protocol.

    Outside the near-tie set F the GPU's (e1, e2, random-test outcome) must equal the oracle's.
    Inside F the GPU's decisions are substituted and the oracle's capacity loops are replayed,
    so that the returned routing is the one every slot, flag and count must match bit-exactly.
    """
    S = x_g.shape[0]
    _, p = orc.gates(x_g, wg)
    m = orc.mean_gates(p)
    e1, e2, g1, g2, g3 = orc.top2(p)
    w2 = g2 / (g1 + g2)
    margin_top = np.where(g3 >= 0, np.minimum(g1 - g2, g2 - g3), g1 - g2)
    margin_rnd = np.abs(2.0 * w2 - u_g.astype(np.float64))
    F = (margin_top < MARGIN) | (margin_rnd < MARGIN)
    o_pass = (2.0 * w2 > u_g.astype(np.float64))
    g_e1 = gpu_expert_idx[:, 0].astype(np.int32)
    g_e2 = gpu_expert_idx[:, 1].astype(np.int32)
    g_pass = (gpu_flags & 2) != 0
    ok = ~F
    assert np.array_equal(g_e1[ok], e1[ok]), "first expert differs outside the near-tie set"
    assert np.array_equal(g_e2[ok], e2[ok]), "second expert differs outside the near-tie set"
    assert np.array_equal(g_pass[ok], o_pass[ok]), "random-routing test differs outside the near-tie set"
    flips = int(((g_e1 != e1) | (g_e2 != e2) | (g_pass != o_pass))[F].sum())
    e1r = np.where(F, g_e1, e1).astype(np.int32)
    e2r = np.where(F, g_e2, e2).astype(np.int32)
    idx = np.arange(S)
    g1r, g2r = p[idx, e1r], p[idx, e2r]
    override = np.where(F, g_pass.astype(np.int8), np.int8(-1)).astype(np.int8)
    routing = orc.capacity(p.shape[1], C, e1r, e2r, g1r, g2r, u_g, m, pass_override=override,
                           variant_a=variant_a)
    return GroupCheck(int(F.sum()), flips, routing, e1r, e2r, m, p)


def slot_token_from(routing: orc.GroupRouting, e1, e2, E, C) -> np.ndarray:
    """[E,C] inverse list of one group built from the oracle's slots."""
    st = np.full((E, C), -1, np.int32)
    for k, ek in ((0, e1), (1, e2)):
        kept = routing.slot[:, k] >= 0
        st[ek[kept], routing.slot[kept, k]] = np.nonzero(kept)[0]
    return st


def oracle_token_output(x_row, kept, experts, weights, fetch_expert) -> np.ndarray:
    """Eq. (3) for one token: sum over kept choices of weight * FFN_e(x).  fetch_expert(e)
    returns (wi_e [M,H], wo_e [H,M]) as float32 numpy arrays."""
    y = np.zeros(x_row.shape[0], np.float64)
    for k in range(2):
        if not kept[k]:
            continue
        wi_e, wo_e = fetch_expert(int(experts[k]))
        y += weights[k] * orc.ffn_rows(x_row[None, :], wi_e, wo_e)[0]
    return y
