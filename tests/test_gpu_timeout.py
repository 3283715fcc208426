"""The give-up path of the GEMM kernels' bounded waits, made to happen on purpose without hanging anything: with the
wait limit set to zero cycles the producer stops waiting for the activation quantizer as soon as it polls (the rows
cannot be ready that early), the kernel winds down in order, and the host reads SASQ_ERR_TIMEOUT.  Afterwards, with
the default limit back, the same call gives the right answer: nothing was left behind in the library's counters."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu
SASQ_ERR_TIMEOUT = 5


@pytest.mark.parametrize("T", [2048, 16])
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_clean(T):
    tag, N, K = oracle.BF16, 1024, 4096
    x = W.activations(T, K, torch.bfloat16, 9900 + T, device="cuda")
    w_int = torch.randint(-127, 128, (N, K), dtype=torch.int8, device="cuda")
    w_scale = torch.full((N,), 1e-3, device="cuda")
    sc = torch.tensor([0.05], device="cuda")
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(P.sasq_static_w8a8_linear_workspace(T, N, K), dtype=torch.uint8, device="cuda")
    assert P.sasq_device_status() == 0
    old = P.sasq_debug_set_wait_limit(0)
    try:
        P.sasq_static_w8a8_linear(x, w_int, w_scale, sc, y, workspace=ws)
        status = P.sasq_device_status()
    finally:
        P.sasq_debug_set_wait_limit(-1)
    assert old == 1 << 31
    assert status == SASQ_ERR_TIMEOUT
    assert P.sasq_device_status() == 0                       # sticky word cleared by the read
    # the same call with the default limit: bit-exact on sampled rows
    P.sasq_static_w8a8_linear(x, w_int, w_scale, sc, y, workspace=ws)
    assert P.sasq_device_status() == 0
    rows = [0, T // 2, T - 1]
    idx = torch.tensor(rows, device="cuda")
    xb = oracle.bits_of(x[idx].cpu())[0]
    y_o, _, _ = oracle.w8a8_linear(xb, tag, w_int.cpu().numpy(), w_scale.cpu().numpy(), 0.05, 8)
    assert np.array_equal(oracle.bits_of(y[idx].cpu())[0], y_o)


def test_give_up_path_of_a_multi_problem_launch_and_of_the_grouped_form():
    """The same for a launch that carries several problems and for the grouped (Eq. 3) kernel: the wait runs out,
    the status word says so, and the next call with the default limit matches an untouched reference run."""
    dev = torch.device("cuda")
    shapes = [(300, 520, 512), (700, 264, 1024)]
    probs = []
    for i, (T, N, K) in enumerate(shapes):
        probs.append((W.activations(T, K, torch.bfloat16, 9950 + i, device=dev),
                      torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev),
                      torch.full((N,), 1e-3, device=dev), torch.tensor([0.05], device=dev),
                      torch.empty((T, N), dtype=torch.bfloat16, device=dev)))
    ws = torch.empty(P.sasq_static_w8a8_linear_multi_workspace(shapes), dtype=torch.uint8, device=dev)
    T, N, K, group = 300, 264, 1024, 256
    xg = W.activations(T, K, torch.bfloat16, 9960, device=dev)
    wg = torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev)
    wsg = torch.full((N,), 1e-3, device=dev)
    sg = torch.full((K // group,), 0.05, device=dev)
    yg = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
    wsp = torch.empty(P.sasq_static_w8a8_linear_grouped_workspace(T, N, K), dtype=torch.uint8, device=dev)

    def run_all():
        P.sasq_static_w8a8_linear_multi(probs, ws)
        P.sasq_static_w8a8_linear_grouped(xg, wg, wsg, sg, group, yg, workspace=wsp)

    run_all()
    assert P.sasq_device_status() == 0
    want = [pr[4].clone() for pr in probs] + [yg.clone()]
    for call in (lambda: P.sasq_static_w8a8_linear_multi(probs, ws),
                 lambda: P.sasq_static_w8a8_linear_grouped(xg, wg, wsg, sg, group, yg, workspace=wsp)):
        P.sasq_debug_set_wait_limit(0)
        try:
            call()
            status = P.sasq_device_status()
        finally:
            P.sasq_debug_set_wait_limit(-1)
        assert status == SASQ_ERR_TIMEOUT
    run_all()
    assert P.sasq_device_status() == 0
    for got, ref in zip([pr[4] for pr in probs] + [yg], want):
        assert torch.equal(got.view(torch.int16), ref.view(torch.int16))
