"""Host-buffer entry points: the synchronous call and the pipelined (three-stream, slotted) call
must give exactly the bits of the device-buffer forward on the same inputs."""
import pytest
import torch

from paper_2006_16668_b200 import MoEConfig, make_inputs
from paper_2006_16668_b200 import binding as B

pytestmark = pytest.mark.gpu


def _device_forward(cfg, shape, inp, x, u):
    ws = B.alloc_workspace(shape)
    y = torch.empty_like(x)
    l_aux = torch.zeros(1, device="cuda")
    B.gshard_moe_top2_forward(shape, x, inp["wg"], inp["wi"], inp["wo"], u, y, l_aux, None, None, ws)
    torch.cuda.synchronize()
    return y.cpu(), float(l_aux)


@pytest.mark.parametrize("dtype,H", [("f32", 128), ("bf16", 1024)])
def test_host_calls_match_device_call(dtype, H):
    cfg = MoEConfig("host", G=2, S=256, M=128, H=H, E=16, C=32, dtype=dtype, seed=91)
    inp = make_inputs(cfg, "cuda")
    shape = B.make_shape(cfg)
    steps = 5
    gen = torch.Generator(device="cuda").manual_seed(7)
    xs = [torch.randn(cfg.G, cfg.S, cfg.M, generator=gen, device="cuda").to(cfg.torch_dtype) for _ in range(steps)]
    us = [torch.rand(cfg.G, cfg.S, generator=gen, device="cuda") for _ in range(steps)]
    ref = [_device_forward(cfg, shape, inp, xs[i], us[i]) for i in range(steps)]

    # synchronous host call
    ws = B.alloc_workspace(shape, host_staging=True)
    xh, uh = xs[0].cpu().pin_memory(), us[0].cpu().pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    lh = torch.zeros(1).pin_memory()
    B.gshard_moe_top2_forward_host(shape, xh, inp["wg"], inp["wi"], inp["wo"], uh, yh, lh, None, ws)
    assert torch.equal(yh.view(torch.uint8), ref[0][0].view(torch.uint8)) and float(lh) == ref[0][1]

    # pipelined call: two slots in rotation, every step its own pinned host buffers
    ws2 = B.alloc_workspace(shape)
    nslots = 2
    stg = [torch.empty(B.gshard_moe_top2_host_staging_bytes(shape), dtype=torch.uint8, device="cuda")
           for _ in range(nslots)]
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    events = [[torch.cuda.Event() for _ in range(3)] for _ in range(nslots)]
    for evs in events:
        for e in evs:
            e.record()                                   # materialise the handles
    torch.cuda.synchronize()
    xhs = [x.cpu().pin_memory() for x in xs]
    uhs = [u.cpu().pin_memory() for u in us]
    yhs = [torch.empty_like(x).pin_memory() for x in xhs]
    lhs = [torch.zeros(1).pin_memory() for _ in range(steps)]
    for i in range(steps):
        k = i % nslots
        B.gshard_moe_top2_forward_host_async(shape, xhs[i], inp["wg"], inp["wi"], inp["wo"], uhs[i], yhs[i], lhs[i],
                                             None, ws2, stg[k], s_in, s_cmp, s_out, *events[k])
    torch.cuda.synchronize()
    assert B.gshard_moe_last_device_status(ws2, s_cmp) == B.GSHARD_OK
    for i in range(steps):
        assert torch.equal(yhs[i].view(torch.uint8), ref[i][0].view(torch.uint8)), f"step {i}"
        assert float(lhs[i]) == ref[i][1]


def test_forward_replays_from_a_cuda_graph():
    """The device-buffer forward only enqueues work on the caller's stream (no allocation, no
    synchronisation), so it can be captured once and replayed on new inputs in the same buffers."""
    cfg = MoEConfig("graph", G=2, S=256, M=256, H=1024, E=32, C=16, dtype="bf16", seed=93)
    inp = make_inputs(cfg, "cuda")
    shape = B.make_shape(cfg)
    ws = B.alloc_workspace(shape)
    x, u = inp["x"].clone(), inp["u"].clone()
    y = torch.empty_like(x)
    l_aux = torch.zeros(1, device="cuda")
    # eager reference on two different inputs
    gen = torch.Generator(device="cuda").manual_seed(11)
    x2 = torch.randn(cfg.G, cfg.S, cfg.M, generator=gen, device="cuda").to(torch.bfloat16)
    u2 = torch.rand(cfg.G, cfg.S, generator=gen, device="cuda")
    refs = []
    for xi, ui in ((inp["x"], inp["u"]), (x2, u2)):
        yi = torch.empty_like(xi)
        li = torch.zeros(1, device="cuda")
        B.gshard_moe_top2_forward(shape, xi, inp["wg"], inp["wi"], inp["wo"], ui, yi, li, None, None, ws)
        torch.cuda.synchronize()
        refs.append((yi.clone(), float(li)))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        B.gshard_moe_top2_forward(shape, x, inp["wg"], inp["wi"], inp["wo"], u, y, l_aux, None, None, ws,
                                  torch.cuda.current_stream())
    for (xi, ui), (y_ref, l_ref) in zip(((inp["x"], inp["u"]), (x2, u2)), refs):
        x.copy_(xi); u.copy_(ui)
        graph.replay()
        torch.cuda.synchronize()
        assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
        assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16)) and float(l_aux) == l_ref
