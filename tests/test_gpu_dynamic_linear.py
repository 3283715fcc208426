"""GPU parity of the dynamic per-token W8A8 linear (the generation phase of phased quantization, Sec. 4.4) against the
CPU oracle: per-row factors, int32 accumulators and 16-bit outputs bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu
DT = {oracle.F16: torch.float16, oracle.BF16: torch.bfloat16}


def run(xb, tag, w_int, w_scale, bits=8, bias_bits=None, want_scales=True):
    T, K = xb.shape
    N = w_int.shape[0]
    x = oracle.tensor_of(xb, tag).cuda()
    y = torch.empty((T, N), dtype=DT[tag], device="cuda")
    acc = torch.empty((T, N), dtype=torch.int32, device="cuda")
    rs = torch.zeros(T, device="cuda") if want_scales else None
    bias = None if bias_bits is None else oracle.tensor_of(bias_bits, tag).cuda()
    ws = torch.empty(P.sasq_dynamic_w8a8_linear_workspace(T, N, K), dtype=torch.uint8, device="cuda")
    P.sasq_dynamic_w8a8_linear(x, torch.from_numpy(w_int).cuda(), torch.from_numpy(w_scale).cuda(), y, bias=bias,
                               row_scale_out=rs, acc_out=acc, workspace=ws, bits=bits)
    assert P.sasq_device_status() == 0
    return oracle.bits_of(y.cpu())[0], acc.cpu().numpy(), (None if rs is None else rs.cpu().numpy())


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("T,N,K", [(1, 8, 16), (1, 4096, 4096), (16, 264, 144), (40, 1024, 11008), (128, 512, 512),
                                   (130, 776, 400), (300, 256, 1040)])
def test_parity_decode_and_small_prefill(tag, T, N, K):
    x = W.activations(T, K, DT[tag], 9500 + T + N + K)
    if T > 2:
        x[1] = 0                                   # an all-zero row takes factor 1
    xb = oracle.bits_of(x)[0]
    w_int, w_scale = oracle.quantize_weight(W.weights_fp32(N, K, 9600 + N).numpy(), 8)
    y_o, acc_o, s_o = oracle.w8a8_linear_dynamic(xb, tag, w_int, w_scale)
    y, acc, s = run(xb, tag, w_int, w_scale)
    assert np.array_equal(s, s_o)
    assert np.array_equal(acc, acc_o)
    assert np.array_equal(y, y_o)
    # no row clips: every row's factor is its own maximum over Qp
    assert np.abs(acc).max() > 0


def test_bias_low_bits_and_factors_kept_in_the_workspace():
    tag, T, N, K = oracle.BF16, 9, 520, 384
    xb = oracle.bits_of(W.activations(T, K, torch.bfloat16, 9700))[0]
    w_int, w_scale = oracle.quantize_weight(W.weights_fp32(N, K, 9701).numpy(), 8)
    bias = oracle.bits_of((torch.randn(N, generator=torch.Generator().manual_seed(4)) * 0.5).to(torch.bfloat16))[0]
    for bits in (8, 4):
        y_o, acc_o, _ = oracle.w8a8_linear_dynamic(xb, tag, w_int, w_scale, bits, bias)
        y, acc, _ = run(xb, tag, w_int, w_scale, bits, bias, want_scales=False)
        assert np.array_equal(acc, acc_o) and np.array_equal(y, y_o)


def test_dynamic_equals_static_with_the_same_factor_on_one_row():
    """On a single row the dynamic factor is the static per-tensor factor of Eq. 1: both entry points agree."""
    tag, N, K = oracle.BF16, 1024, 2048
    x = W.activations(1, K, torch.bfloat16, 9800)
    xb = oracle.bits_of(x)[0]
    w_int, w_scale = oracle.quantize_weight(W.weights_fp32(N, K, 9801).numpy(), 8)
    y_d, acc_d, s = run(xb, tag, w_int, w_scale)
    xd = x.cuda()
    y = torch.empty((1, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(P.sasq_static_w8a8_linear_workspace(1, N, K), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear(xd, torch.from_numpy(w_int).cuda(), torch.from_numpy(w_scale).cuda(),
                              torch.from_numpy(s).cuda(), y, workspace=ws)
    assert np.array_equal(oracle.bits_of(y.cpu())[0], y_d)
