"""The library's calls can be captured into a CUDA graph and replayed: they allocate nothing, synchronise nothing
and keep no host state a replay would need (the counters the kernels use are reset by the kernels themselves, and a
captured launch gets counters that no other launch is ever given, so a replay may overlap other launches of the
library on another stream).

One step of the hot path (fused fake-quant forward + backward of three tensors, then their static W8A8 linears in one
call, then a decode-sized linear) is run eagerly, captured, and replayed on new input values written into the same
buffers; every replay must be bit-identical to the eager result on the same values.
"""
import pytest
import torch

import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu


def test_step_replays_from_a_cuda_graph_bit_identically():
    dev = torch.device("cuda")
    shapes = [(384, 520, 256), (300, 264, 512), (260, 1024, 128)]          # (T, N, K)
    xs = [torch.empty((T, K), dtype=torch.bfloat16, device=dev) for T, _, K in shapes]
    gs = [torch.empty_like(x) for x in xs]
    ys, dxs = [torch.empty_like(x) for x in xs], [torch.empty_like(x) for x in xs]
    ws = [torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev) for _, N, K in shapes]
    wsc = [torch.rand(N, device=dev) * 1e-2 + 1e-3 for _, N, _ in shapes]
    outs = [torch.empty((T, N), dtype=torch.bfloat16, device=dev) for T, N, _ in shapes]
    scales = torch.tensor([0.05, 0.03, 0.08], device=dev)
    grads = torch.zeros(3, device=dev)
    xd = torch.empty((8, 512), dtype=torch.bfloat16, device=dev)           # a decode-sized linear on its own
    wd = torch.randint(-127, 128, (1024, 512), dtype=torch.int8, device=dev)
    wdsc = torch.full((1024,), 2e-3, device=dev)
    outd = torch.empty((8, 1024), dtype=torch.bfloat16, device=dev)
    q_ws = torch.empty(P.sasq_fakequant_multi_workspace(3), dtype=torch.uint8, device=dev)
    l_ws = torch.empty(P.sasq_static_w8a8_linear_multi_workspace(shapes), dtype=torch.uint8, device=dev)
    d_ws = torch.empty(P.sasq_static_w8a8_linear_workspace(8, 1024, 512), dtype=torch.uint8, device=dev)
    quant = P.QuantTensors([(xs[i], gs[i], ys[i], dxs[i], i) for i in range(3)])
    linears = P.LinearProblems([(xs[i], ws[i], wsc[i], scales[i:i + 1], outs[i]) for i in range(3)])

    def fill(seed):
        for i, (T, _, K) in enumerate(shapes):
            xs[i].copy_(W.activations(T, K, torch.bfloat16, seed + i, device=dev))
            gs[i].copy_(W.upstream_grad(T, K, torch.bfloat16, seed + i, device=dev))
        xd.copy_(W.activations(8, 512, torch.bfloat16, seed + 9, device=dev))

    def step():
        P.sasq_fakequant_fwd_bwd_multi(quant, scales, grads, q_ws, 8)
        P.sasq_static_w8a8_linear_multi(linears, l_ws)
        P.sasq_static_w8a8_linear(xd, wd, wdsc, scales[0:1], outd, workspace=d_ws)

    def snapshot():
        torch.cuda.synchronize()
        return [t.clone() for t in ys + dxs + outs + [outd, grads]]

    fill(100)
    step()                                   # eager warm-up: one-time attribute set-up happens outside the capture
    torch.cuda.synchronize()
    want = {}
    for seed in (100, 200, 300):
        fill(seed)
        step()
        want[seed] = snapshot()

    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fill(100)
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()

    for seed in (200, 300, 100, 200):
        fill(seed)
        graph.replay()
        got = snapshot()
        assert P.sasq_device_status() == 0
        for a, b in zip(got, want[seed]):
            if a.dtype == torch.float32:
                assert torch.equal(a, b)
            else:
                assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_graph_replay_overlapping_direct_launches_on_another_stream():
    """A replayed graph keeps the counter addresses of its capture.  Launches made directly on another stream while
    the graph replays must not share them: both streams' results stay bit-identical to their serial results."""
    dev = torch.device("cuda")
    T, N, K = 512, 1032, 512
    n = 1_000_003

    def make(seed):
        x = W.activations(T, K, torch.bfloat16, seed, device=dev)
        w = torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev,
                          generator=torch.Generator(device=dev).manual_seed(seed))
        wsc = torch.full((N,), 3e-3, device=dev)
        out = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
        l_ws = torch.empty(P.sasq_static_w8a8_linear_workspace(T, N, K), dtype=torch.uint8, device=dev)
        qx = (torch.randn(n, device=dev, generator=torch.Generator(device=dev).manual_seed(seed + 7)) * 3).bfloat16()
        qg = torch.randn(n, device=dev, generator=torch.Generator(device=dev).manual_seed(seed + 8)).bfloat16()
        qy, qdx, ds = torch.empty_like(qx), torch.empty_like(qx), torch.zeros(1, device=dev)
        q_ws = torch.empty(P.sasq_fakequant_bwd_workspace(n), dtype=torch.uint8, device=dev)
        sc = torch.tensor([0.04], device=dev)
        return dict(x=x, w=w, wsc=wsc, out=out, l_ws=l_ws, qx=qx, qg=qg, qy=qy, qdx=qdx, ds=ds, q_ws=q_ws, sc=sc)

    def step(c, stream=None):
        P.sasq_fakequant_fwd_bwd(c["qx"], c["qg"], c["qy"], c["qdx"], c["ds"], c["sc"], c["q_ws"], 8, stream=stream)
        P.sasq_static_w8a8_linear(c["x"], c["w"], c["wsc"], c["sc"], c["out"], workspace=c["l_ws"], stream=stream)

    def results(c):
        return [c["qy"].clone(), c["qdx"].clone(), c["ds"].clone(), c["out"].clone()]

    a, b = make(41), make(42)            # a: captured and replayed; b: launched directly on another stream
    step(a); step(b)
    torch.cuda.synchronize()
    want_a, want_b = results(a), results(b)
    graph = torch.cuda.CUDAGraph()
    s_a, s_b = torch.cuda.Stream(), torch.cuda.Stream()
    s_a.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s_a):
        with torch.cuda.graph(graph, stream=s_a):
            step(a)
    torch.cuda.synchronize()
    for rep in range(20):
        for t in (a["qy"], a["qdx"], a["out"], b["qy"], b["qdx"], b["out"]):
            t.zero_()
        torch.cuda.synchronize()
        with torch.cuda.stream(s_a):
            graph.replay()
        with torch.cuda.stream(s_b):
            step(b, s_b)
            step(b, s_b)
        torch.cuda.synchronize()
        assert P.sasq_device_status() == 0
        for got, want in zip(results(a) + results(b), want_a + want_b):
            assert torch.equal(got.view(torch.int16) if got.dtype != torch.float32 else got,
                               want.view(torch.int16) if want.dtype != torch.float32 else want), rep
