"""The dense Transformer feed-forward sub-layer (section 2.1; eq. (2) with one expert that sees
every token) against the oracle's FFN rows."""
import numpy as np
import pytest
import torch

from oracle import gshard_oracle as orc
from paper_2006_16668_b200 import binding as B
from parity_util import rel_fro, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,M,H,dtype", [
    (50, 64, 256, "f32"), (128, 128, 512, "bf16"), (1000, 256, 1024, "bf16"), (130, 64, 192, "bf16"),
    (4100, 1024, 2048, "bf16"),
])
def test_dense_ffn_against_oracle(n, M, H, dtype):
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    gen = torch.Generator(device="cuda").manual_seed(n + M)
    x = torch.randn(n, M, generator=gen, device="cuda").to(tdt)
    wi = (torch.randn(M, H, generator=gen, device="cuda") * M ** -0.5).to(tdt)
    wo = (torch.randn(H, M, generator=gen, device="cuda") * H ** -0.5).to(tdt)
    y = torch.empty_like(x)
    code = B.GSHARD_BF16 if dtype == "bf16" else B.GSHARD_F32
    ws = torch.empty(B.gshard_dense_ffn_workspace_bytes(n, M, H, code), dtype=torch.uint8, device="cuda")
    B.gshard_dense_ffn_forward(x, wi, wo, y, ws)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
    rows = np.unique(np.concatenate([np.arange(min(n, 40)), np.arange(max(0, n - 40), n),
                                     np.random.default_rng(n).integers(0, n, 64)]))
    ref = orc.ffn_rows(to_np(x)[rows], to_np(wi), to_np(wo))
    err = rel_fro(to_np(y)[rows], ref)
    assert err < (1e-5 if dtype == "f32" else 1e-2), err


@pytest.mark.parametrize("n,M,H", [(50, 64, 256), (300, 40, 72), (1000, 256, 1024), (4100, 1024, 2048)])
def test_dense_ffn_tf32_against_oracle(n, M, H):
    """fp32 tensors with both contractions on the tensor cores in TF32: within 1e-2 of the oracle
    (the achieved error, a few 1e-4, is printed), and much closer to it than bf16 would be."""
    gen = torch.Generator(device="cuda").manual_seed(n + M + 1)
    x = torch.randn(n, M, generator=gen, device="cuda")
    wi = torch.randn(M, H, generator=gen, device="cuda") * M ** -0.5
    wo = torch.randn(H, M, generator=gen, device="cuda") * H ** -0.5
    y = torch.empty_like(x)
    ws = torch.empty(B.gshard_dense_ffn_workspace_bytes(n, M, H, B.GSHARD_F32), dtype=torch.uint8, device="cuda")
    B.gshard_dense_ffn_forward(x, wi, wo, y, ws, flags=B.GSHARD_FLAG_TF32_EXPERTS)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
    assert B.gshard_moe_last_launch_count() == 4          # two weight transposes, two tensor-core GEMMs
    rows = np.unique(np.concatenate([np.arange(min(n, 40)), np.arange(max(0, n - 40), n),
                                     np.random.default_rng(n).integers(0, n, 64)]))
    ref = orc.ffn_rows(to_np(x)[rows], to_np(wi), to_np(wo))
    err = rel_fro(to_np(y)[rows], ref)
    print(f"\n[dense FFN tf32 n={n} M={M} H={H}] rel. Frobenius error {err:.3e}")
    assert 1e-6 < err < 2e-3, err


def test_dense_ffn_full_size_sampled_rows():
    """The adjacent Transformer layer's FFN at the MoE(2048E) batch: 131072 tokens, M=1024, H=8192."""
    n, M, H = 131072, 1024, 8192
    gen = torch.Generator(device="cuda").manual_seed(11)
    x = torch.randn(n, M, generator=gen, device="cuda").bfloat16()
    wi = (torch.randn(M, H, generator=gen, device="cuda") * M ** -0.5).bfloat16()
    wo = (torch.randn(H, M, generator=gen, device="cuda") * H ** -0.5).bfloat16()
    y = torch.empty_like(x)
    ws = torch.empty(B.gshard_dense_ffn_workspace_bytes(n, M, H, B.GSHARD_BF16), dtype=torch.uint8, device="cuda")
    B.gshard_dense_ffn_forward(x, wi, wo, y, ws)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
    rows = np.unique(np.concatenate([np.arange(0, 8), np.arange(n - 8, n), np.arange(65528, 65544),
                                     np.random.default_rng(3).integers(0, n, 96)]))
    idx = torch.from_numpy(rows).cuda()
    ref = orc.ffn_rows(to_np(x[idx]), to_np(wi), to_np(wo))
    assert rel_fro(to_np(y[idx]), ref) < 1e-2


def test_dense_ffn_bad_arguments():
    lib = B.load()
    assert B.gshard_dense_ffn_workspace_bytes(0, 64, 64, B.GSHARD_F32) == 0
    assert B.gshard_dense_ffn_workspace_bytes(8, 60, 64, B.GSHARD_F32) == 0
    assert B.gshard_dense_ffn_workspace_bytes(8, 72, 64, B.GSHARD_BF16) == 0
    fake = 0x10000
    assert lib.gshard_dense_ffn_forward(0, 64, 64, 0, 0, fake, fake, fake, fake, fake, 1 << 30, None) == B.GSHARD_ERR_INVALID_ARG
    assert lib.gshard_dense_ffn_forward(8, 72, 64, 1, 0, fake, fake, fake, fake, fake, 1 << 30, None) == B.GSHARD_ERR_UNSUPPORTED_SHAPE
    assert lib.gshard_dense_ffn_forward(8, 64, 64, 0, 0, fake, fake, None, fake, fake, 1 << 30, None) == B.GSHARD_ERR_INVALID_ARG
    assert lib.gshard_dense_ffn_forward(8, 64, 64, 0, 0, fake, fake, fake, fake, fake, 16, None) == B.GSHARD_ERR_WORKSPACE_TOO_SMALL
