"""Linears submitted from two streams at once.

Kernels with the activation quantizer inside have CTAs that wait for other CTAs of the same launch.  By default
such launches are co-operative grids, which the driver starts only when all their CTAs can be resident, so launches
that overlap on different streams cannot starve each other; sasq_set_gang_launch(0) makes them plain launches for
callers that keep to one stream.  The test checks that the setting changes no bit of any result and that interleaved
launches on two streams (default setting) all complete with the right outputs.
"""
import pytest
import torch

import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu


def make(T, N, K, seed):
    dev = torch.device("cuda")
    x = W.activations(T, K, torch.bfloat16, seed, device=dev)
    w = torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev,
                      generator=torch.Generator(device=dev).manual_seed(seed))
    wsc = torch.rand(N, device=dev, generator=torch.Generator(device=dev).manual_seed(seed + 1)) * 1e-2 + 1e-3
    sc = torch.tensor([0.04], device=dev)
    ws = torch.empty(max(16, P.sasq_static_w8a8_linear_workspace(T, N, K)), dtype=torch.uint8, device=dev)
    return dict(x=x, w=w, wsc=wsc, sc=sc, ws=ws, T=T, N=N)


def run(pr, stream=None):
    y = torch.empty((pr["T"], pr["N"]), dtype=torch.bfloat16, device="cuda")
    P.sasq_static_w8a8_linear(pr["x"], pr["w"], pr["wsc"], pr["sc"], y, workspace=pr["ws"], stream=stream)
    return y


def test_gang_launch_changes_no_result_and_streams_can_overlap():
    cases = [make(700, 1032, 512, 31), make(16, 4096, 1024, 32), make(2048, 4096, 1024, 33), make(1, 2048, 4096, 34)]
    previous = P.sasq_set_gang_launch(False)          # plain launches, one stream: the reference results
    assert previous is True                           # co-operative launches are the default
    try:
        want = [run(pr) for pr in cases]
        torch.cuda.synchronize()
        assert P.sasq_device_status() == 0
    finally:
        P.sasq_set_gang_launch(True)
    try:
        for pr, ref in zip(cases, want):                       # same bits with co-operative launches
            assert torch.equal(run(pr).view(torch.int16), ref.view(torch.int16))
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        s1.wait_stream(torch.cuda.current_stream())
        s2.wait_stream(torch.cuda.current_stream())
        # every case has its own workspace, so the two streams share nothing but the GPU
        outs = []
        for rep in range(10):
            for i, pr in enumerate(cases):
                stream = s1 if (i + rep) % 2 == 0 else s2
                with torch.cuda.stream(stream):
                    outs.append((i, run(pr, stream)))
            s1.synchronize()              # a case's workspace is free again before its next launch
            s2.synchronize()
        torch.cuda.synchronize()
        assert P.sasq_device_status() == 0
        for i, y in outs:
            assert torch.equal(y.view(torch.int16), want[i].view(torch.int16)), i
    finally:
        P.sasq_set_gang_launch(True)
