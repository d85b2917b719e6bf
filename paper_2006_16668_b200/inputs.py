"""Seeded synthetic inputs for the top-2 MoE layer.

This module is the one piece shared by the CUDA path's tests/benchmark and the CPU
oracle's tests.  It holds NO arithmetic of the method: it only draws random tensors
with the shapes and value distributions of the paper's MoE(128E/512E/2048E) layers
(model dimension 1024, expert hidden dimension 8192; Appendix "Model details" and
the model-family table), which stand in for the paper's non-public training data
and trained weights.

Recipe (one seed per configuration, one rounding to the configuration's dtype):
    x  ~ N(0, 1)            [G,S,M]
    wg ~ N(0, var 1/M)      [M,E]     (unit-variance logits)
    wi ~ N(0, var 1/M)      [E,M,H]
    wo ~ N(0, var 1/H)      [E,H,M]
    u  ~ U[0, 1) float32    [G,S]     (the noise of the random-routing test)
    dy ~ N(0, 1)            [G,S,M]   (training-step configuration only)
The "skew" configuration adds the constant vector 3*v/|v|, v = sum of wg columns
0..7, to every token before rounding, so that experts 0..7 overflow.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class MoEConfig:
    name: str
    G: int
    S: int
    M: int
    H: int
    E: int
    C: int
    dtype: str = "bf16"          # "f32" | "bf16": x, wg, wi, wo, y share it
    seed: int = 20200630
    skew: bool = False
    backward: bool = False
    k_aux: float = 0.01

    @property
    def N(self) -> int:
        return self.G * self.S

    @property
    def rows_per_expert(self) -> int:
        return self.G * self.C

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def scaled(self, **kw) -> "MoEConfig":
        return replace(self, **kw)


CONFIGS = {
    # configs[0]: the tiny case the oracle finishes in milliseconds
    "c1_tiny": MoEConfig("c1_tiny", G=2, S=64, M=64, H=256, E=8, C=16, dtype="f32", seed=20200631),
    # configs[1..3]: MoE(128E/512E/2048E)-shaped forward
    "c2_128e": MoEConfig("c2_128e", G=16, S=4096, M=1024, H=8192, E=128, C=64, seed=20200632),
    "c3_512e_skew": MoEConfig("c3_512e_skew", G=16, S=4096, M=1024, H=8192, E=512, C=16,
                              seed=20200633, skew=True),
    "c4_2048e": MoEConfig("c4_2048e", G=32, S=4096, M=1024, H=8192, E=2048, C=4, seed=20200634),
    # configs[4]: training step
    "c5_512e_train": MoEConfig("c5_512e_train", G=16, S=4096, M=1024, H=8192, E=512, C=16,
                               seed=20200635, backward=True),
}


def _normal(shape, std, gen, device, dtype, chunk_elems=1 << 26):
    """N(0, std^2) rounded once to dtype; generated in fp32 chunks to bound the temporary."""
    n = 1
    for d in shape:
        n *= d
    out = torch.empty(n, device=device, dtype=dtype)
    for lo in range(0, n, chunk_elems):
        hi = min(n, lo + chunk_elems)
        t = torch.randn(hi - lo, generator=gen, device=device, dtype=torch.float32)
        out[lo:hi] = (t * std).to(dtype)
    return out.view(*shape)


def make_inputs(cfg: MoEConfig, device="cpu", with_experts: bool = True) -> dict:
    """Return {'x','wg','wi','wo','u'[, 'dy']} on `device` in the configuration's dtype.

    The CPU and CUDA generators of torch give different streams: a comparison must
    generate once and copy the same bytes to the other side.
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed)
    dt = cfg.torch_dtype
    out = {}
    out["wg"] = _normal((cfg.M, cfg.E), cfg.M ** -0.5, gen, dev, dt)
    x32 = torch.randn(cfg.G, cfg.S, cfg.M, generator=gen, device=dev, dtype=torch.float32)
    if cfg.skew:
        v = out["wg"][:, :8].float().sum(dim=1)
        x32 += 3.0 * v / v.norm()
    out["x"] = x32.to(dt)
    del x32
    out["u"] = torch.rand(cfg.G, cfg.S, generator=gen, device=dev, dtype=torch.float32)
    if cfg.backward:
        out["dy"] = _normal((cfg.G, cfg.S, cfg.M), 1.0, gen, dev, dt)
    if with_experts:
        out["wi"] = _normal((cfg.E, cfg.M, cfg.H), cfg.M ** -0.5, gen, dev, dt)
        out["wo"] = _normal((cfg.E, cfg.H, cfg.M), cfg.H ** -0.5, gen, dev, dt)
    return out
