"""GPU parity: the static W8A8 linear in the grouped form of Eq. 3 (one static activation factor per group of K
columns, int32 partial products per group, fp32 accumulation in group order) against the CPU oracle.

Bar: the 16-bit output bit-exact.  Both sides form fl32(acc_g) * fl32(s_g * s_w[n]) and add the groups in ascending
order in fp32 without FMA, so nothing is left to rounding order.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu

DT = {oracle.F16: torch.float16, oracle.BF16: torch.bfloat16}


def host_bits(t):
    return oracle.bits_of(t.cpu())[0]


def make_case(T, N, K, group, tag, seed, bits=8, factor=0.6):
    xb = oracle.bits_of(W.activations(T, K, DT[tag], seed))[0]
    w_int, w_scale = oracle.quantize_weight(W.weights_fp32(N, K, seed + 1).numpy(), 8)
    calib = xb[:min(T, W.CALIBRATION_TOKENS)]
    # Eq. 1 on each group's columns of the calibration rows, shrunk so that outliers are clipped
    s_group = np.array([float(oracle.absmax_scale(np.ascontiguousarray(calib[:, g * group:(g + 1) * group]), tag, bits))
                        * factor for g in range(K // group)], np.float32)
    return xb, w_int, w_scale, s_group


def run_gpu(xb, tag, w_int, w_scale, s_group, group, bits=8, bias_bits=None):
    T, K = xb.shape
    N = w_int.shape[0]
    x = oracle.tensor_of(xb, tag).cuda()
    y = torch.full((T, N), 7.0, dtype=DT[tag], device="cuda")
    bias = None if bias_bits is None else oracle.tensor_of(bias_bits, tag).cuda()
    ws = torch.empty(max(16, P.sasq_static_w8a8_linear_grouped_workspace(T, N, K)), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear_grouped(x, torch.from_numpy(w_int).cuda(), torch.from_numpy(w_scale).cuda(),
                                      torch.from_numpy(s_group).cuda(), group, y, bias=bias, workspace=ws, bits=bits)
    assert P.sasq_device_status() == 0
    return host_bits(y)


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("T,N,K,group", [(1, 136, 256, 128), (128, 128, 1024, 256), (200, 264, 512, 128),
                                         (257, 1024, 2048, 512), (300, 520, 1152, 384), (130, 4104, 384, 128)])
def test_parity_grouped_shapes(tag, T, N, K, group):
    xb, w_int, w_scale, s_group = make_case(T, N, K, group, tag, 8000 + T + N + K)
    y_g = run_gpu(xb, tag, w_int, w_scale, s_group, group)
    y_o, _ = oracle.w8a8_linear_grouped(xb, tag, w_int, w_scale, s_group, group)
    assert np.array_equal(y_g, y_o)


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
def test_parity_with_bias_negative_factor_and_low_bits(tag):
    T, N, K, group = 70, 520, 768, 256
    xb, w_int, w_scale, s_group = make_case(T, N, K, group, tag, 8100, bits=4)
    s_group[1] = -s_group[1]
    bias = oracle.bits_of((torch.randn(N, generator=torch.Generator().manual_seed(5)) * 0.5).to(DT[tag]))[0]
    y_g = run_gpu(xb, tag, w_int, w_scale, s_group, group, bits=4, bias_bits=bias)
    y_o, _ = oracle.w8a8_linear_grouped(xb, tag, w_int, w_scale, s_group, group, bits=4, bias=bias)
    assert np.array_equal(y_g, y_o)


def test_one_group_is_the_per_tensor_linear():
    """With a single group Eq. 3 is Eq. 2: the grouped entry point and the plain one give the same bits."""
    tag, T, N, K = oracle.BF16, 300, 520, 384
    xb, w_int, w_scale, s_group = make_case(T, N, K, K, tag, 8200)
    y_g = run_gpu(xb, tag, w_int, w_scale, s_group, K)
    y_o, _, _ = oracle.w8a8_linear(xb, tag, w_int, w_scale, float(s_group[0]), 8)
    assert np.array_equal(y_g, y_o)


def test_many_groups_and_several_tiles_per_cta():
    """More tiles than SMs (each CTA walks several tiles, so the accumulator buffers and the fp32 sums are reused)
    and 32 groups of 128 columns; sampled rows against the oracle."""
    tag, T, N, K, group = oracle.BF16, 1024, 4096, 4096, 128
    x = W.activations(T, K, torch.bfloat16, 8300, device="cuda")
    w = W.weights_fp32(N, K, 8301, device="cuda")
    w_int = torch.empty((N, K), dtype=torch.int8, device="cuda")
    w_scale = torch.empty(N, dtype=torch.float32, device="cuda")
    P.sasq_quantize_weight(w, w_int, w_scale, 8)
    calib = oracle.bits_of(x[:W.CALIBRATION_TOKENS].cpu())[0]
    s_group = np.array([float(oracle.absmax_scale(np.ascontiguousarray(calib[:, g * group:(g + 1) * group]), tag, 8)) * 0.5
                        for g in range(K // group)], np.float32)
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(P.sasq_static_w8a8_linear_grouped_workspace(T, N, K), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear_grouped(x, w_int, w_scale, torch.from_numpy(s_group).cuda(), group, y, workspace=ws)
    assert P.sasq_device_status() == 0
    rows = [0, 1, 127, 128, 129, 511, 640, 1023]
    idx = torch.tensor(rows, device="cuda")
    y_o, _ = oracle.w8a8_linear_grouped(oracle.bits_of(x[idx].cpu())[0], tag, w_int.cpu().numpy(),
                                        w_scale.cpu().numpy(), s_group, group)
    assert np.array_equal(host_bits(y[idx]), y_o)


def test_unsupported_group_sizes_and_bad_factor():
    tag, T, N, K = oracle.BF16, 64, 128, 256
    xb, w_int, w_scale, s_group = make_case(T, N, K, 128, tag, 8400)
    x = oracle.tensor_of(xb, tag).cuda()
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(P.sasq_static_w8a8_linear_grouped_workspace(T, N, K), dtype=torch.uint8, device="cuda")
    w, wsc = torch.from_numpy(w_int).cuda(), torch.from_numpy(w_scale).cuda()
    with pytest.raises(RuntimeError):            # groups are whole 128-column blocks
        P.sasq_static_w8a8_linear_grouped(x, w, wsc, torch.ones(4, device="cuda"), 64, y, workspace=ws)
    with pytest.raises(RuntimeError):            # workspace too small
        P.sasq_static_w8a8_linear_grouped(x, w, wsc, torch.ones(2, device="cuda"), 128, y, workspace=ws[:64])
    P.sasq_static_w8a8_linear_grouped(x, w, wsc, torch.tensor([0.05, 0.0], device="cuda"), 128, y, workspace=ws)
    assert P.sasq_device_status() != 0           # a zero factor is reported through the status word
    assert P.sasq_device_status() == 0           # ... and reading it clears it
