"""Pins for the oracle's layer output and gradients through a second formulation:
the dense einsum program of Algorithm 2 (combine_weights [G,S,E,C], dispatch mask,
five library einsums) in torch float64, with its autograd giving the gradients,
plus central finite differences.  The only thing taken from the oracle here is
the integer routing (which expert, which buffer position) - the values of the
combine weights are recomputed from a torch softmax so that autograd sees them.
"""
import numpy as np
import pytest
import torch

from oracle import gshard_oracle as orc


def _rand_layer(seed, G, S, M, H, E):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((G, S, M)).astype(np.float32)
    wg = (rng.standard_normal((M, E)) / np.sqrt(M) * 2).astype(np.float32)
    wi = (rng.standard_normal((E, M, H)) / np.sqrt(M)).astype(np.float32)
    wo = (rng.standard_normal((E, H, M)) / np.sqrt(H)).astype(np.float32)
    u = rng.random((G, S)).astype(np.float32)
    dy = rng.standard_normal((G, S, M)).astype(np.float32)
    return x, wg, wi, wo, u, dy


def _dense_algorithm2(x, wg, wi, wo, f, C, k_aux):
    """Algorithm 2 with einsums; returns y, l_aux, loss pieces as torch float64 tensors."""
    G, S, M = x.shape
    E = wg.shape[1]
    gates = torch.softmax(torch.einsum("gsm,me->gse", x, wg), dim=-1)
    ei = torch.from_numpy(f.expert_idx.astype(np.int64))
    slot = torch.from_numpy(f.slot.astype(np.int64))
    g12 = torch.gather(gates, 2, ei)                          # raw top-2 gates [G,S,2]
    w = g12 / g12.sum(dim=-1, keepdim=True)
    combine = torch.zeros(G, S, E, C, dtype=torch.float64)
    gi, si = torch.meshgrid(torch.arange(G), torch.arange(S), indexing="ij")
    for k in range(2):
        kept = slot[..., k] >= 0
        combine = combine.index_put(
            (gi[kept], si[kept], ei[..., k][kept], slot[..., k][kept]), w[..., k][kept])
    dispatch = (combine != 0).to(torch.float64)
    dispatched = torch.einsum("gsec,gsm->egcm", dispatch, x)
    h = torch.relu(torch.einsum("egcm,emh->egch", dispatched, wi))
    expert_out = torch.einsum("egch,ehm->gecm", h, wo)
    y = torch.einsum("gsec,gecm->gsm", combine, expert_out)
    c1 = torch.from_numpy(f.first_count.astype(np.float64))   # constant (non-differentiable)
    l_aux = ((c1 / S) * gates.mean(dim=1)).mean(dim=1).mean()
    return y, l_aux, combine


CASES = [(21, 2, 24, 6, 10, 4, 8, False), (22, 1, 40, 5, 7, 6, 3, False),
         (23, 3, 16, 4, 6, 3, 4, True), (24, 2, 32, 8, 12, 8, 2, False)]


@pytest.mark.parametrize("seed,G,S,M,H,E,C,variant_a", CASES)
def test_forward_matches_dense_einsum_program(seed, G, S, M, H, E, C, variant_a):
    x, wg, wi, wo, u, _ = _rand_layer(seed, G, S, M, H, E)
    f = orc.forward(x, wg, wi, wo, u, C, variant_a=variant_a)
    t = [torch.from_numpy(a.astype(np.float64)) for a in (x, wg, wi, wo)]
    y, l_aux, combine = _dense_algorithm2(*t, f, C, 0.0)
    np.testing.assert_allclose(f.y, y.numpy(), rtol=1e-9, atol=1e-11)
    assert f.l_aux == pytest.approx(float(l_aux), rel=1e-12)
    # at most two non-zeros per token; dropped tokens produce exactly zero
    assert int((combine != 0).sum(dim=(2, 3)).max()) <= 2
    both_dropped = (f.slot < 0).all(axis=-1)
    assert np.all(f.y[both_dropped] == 0.0)
    # some case must actually exercise drops and skips
    if seed == 24:
        assert both_dropped.any() and (f.slot[..., 0] < 0).any() and (f.flags & 2 == 0).any()


@pytest.mark.parametrize("seed,G,S,M,H,E,C,variant_a", CASES)
def test_backward_matches_autograd(seed, G, S, M, H, E, C, variant_a):
    k_aux = 0.37
    x, wg, wi, wo, u, dy = _rand_layer(seed, G, S, M, H, E)
    f = orc.forward(x, wg, wi, wo, u, C, variant_a=variant_a)
    dx, dwg, dwi, dwo = orc.backward(x, wg, wi, wo, f, dy, k_aux)
    t = [torch.from_numpy(a.astype(np.float64)).requires_grad_(True) for a in (x, wg, wi, wo)]
    y, l_aux, _ = _dense_algorithm2(*t, f, C, k_aux)
    loss = (y * torch.from_numpy(dy.astype(np.float64))).sum() + k_aux * l_aux
    loss.backward()
    for got, ref in zip((dx, dwg, dwi, dwo), t):
        ref = ref.grad.numpy()
        assert np.linalg.norm(got - ref) <= 1e-10 * max(1.0, np.linalg.norm(ref))


def test_backward_aux_only_and_finite_differences():
    # k*l_aux alone: the gradient reaches only x and wg, through the dense mean-gate term.
    seed, G, S, M, H, E, C = 31, 2, 12, 4, 5, 3, 5
    x, wg, wi, wo, u, dy = _rand_layer(seed, G, S, M, H, E)
    f = orc.forward(x, wg, wi, wo, u, C)
    dx, dwg, dwi, dwo = orc.backward(x, wg, wi, wo, f, np.zeros_like(dy), 1.0)
    assert np.all(dwi == 0) and np.all(dwo == 0) and np.abs(dwg).max() > 0

    # central differences on L(wg) = <dy, y> + k l_aux with the routing frozen:
    # y and l_aux are re-evaluated from the definitions with the SAME integer routing.
    k_aux = 0.5
    dx, dwg, dwi, dwo = orc.backward(x, wg, wi, wo, f, dy, k_aux)

    def loss(wg_):
        tot = 0.0
        for g in range(G):
            _, p = orc.gates(x[g], wg_)
            m = p.mean(0)
            tot += k_aux * float(((f.first_count[g] / S) * m).mean()) / G
            for s in range(S):
                a, b = p[s, f.expert_idx[g, s, 0]], p[s, f.expert_idx[g, s, 1]]
                for k, wk in ((0, a / (a + b)), (1, b / (a + b))):
                    if f.slot[g, s, k] >= 0:
                        e = f.expert_idx[g, s, k]
                        o = orc.ffn_rows(x[g, s:s + 1], wi[e], wo[e])[0]
                        tot += wk * float(dy[g, s].astype(np.float64) @ o)
        return tot

    rng = np.random.default_rng(0)
    for _ in range(6):
        i, j = int(rng.integers(M)), int(rng.integers(E))
        eps = 2.0 ** -10                       # exactly representable step in float32
        wp, wm = wg.copy(), wg.copy()
        wp[i, j] += eps
        wm[i, j] -= eps
        fd = (loss(wp) - loss(wm)) / (float(wp[i, j]) - float(wm[i, j]))
        assert dwg[i, j] == pytest.approx(fd, rel=2e-4, abs=1e-7)
