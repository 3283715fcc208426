"""GPU parity of the static W8A8 linear with one activation factor per channel (folded into the weights ahead of
time) against the CPU oracle: int32 accumulators and outputs bit-exact, for the decode, general small-T and CTA-pair
kernels; and a sanity bound against the float64 product, which shows that the folding really represents x W^T."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu
DT = {oracle.F16: torch.float16, oracle.BF16: torch.bfloat16}


def make(T, N, K, tag, seed, bits=8, shrink=1.0):
    x = W.activations(T, K, DT[tag], seed)
    xb = oracle.bits_of(x)[0]
    qp = 2 ** (bits - 1) - 1
    amax = np.abs(oracle.widen(xb, tag)).max(axis=0)
    s = (np.maximum(amax, 1e-3) / qp * shrink).astype(np.float32)           # Eq. 1 per channel (x shrink: "learned")
    w_fp = W.weights_fp32(N, K, seed + 1).numpy()
    w_int, w_scale = oracle.quantize_weight(w_fp * s[None, :], 8)            # factors folded into the frozen weights
    return xb, s, w_fp, w_int, w_scale


def run(xb, tag, s, w_int, w_scale, bits=8, bias_bits=None):
    T, K = xb.shape
    N = w_int.shape[0]
    x = oracle.tensor_of(xb, tag).cuda()
    y = torch.empty((T, N), dtype=DT[tag], device="cuda")
    acc = torch.empty((T, N), dtype=torch.int32, device="cuda")
    bias = None if bias_bits is None else oracle.tensor_of(bias_bits, tag).cuda()
    ws = torch.empty(P.sasq_static_w8a8_linear_per_channel_workspace(T, N, K), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear_per_channel(x, torch.from_numpy(w_int).cuda(), torch.from_numpy(w_scale).cuda(),
                                          torch.from_numpy(s).cuda(), y, bias=bias, acc_out=acc, workspace=ws,
                                          bits=bits)
    assert P.sasq_device_status() == 0
    return oracle.bits_of(y.cpu())[0], acc.cpu().numpy()


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("T,N,K", [(1, 8, 16), (16, 264, 144), (128, 512, 512), (130, 776, 400), (300, 256, 1040),
                                   (520, 1024, 2048), (24, 19200, 80)])
def test_parity_all_three_kernels(tag, T, N, K):
    xb, s, _, w_int, w_scale = make(T, N, K, tag, 9950 + T + N + K, shrink=0.7)
    y_o, acc_o = oracle.w8a8_linear_per_channel(xb, tag, w_int, w_scale, s)
    y, acc = run(xb, tag, s, w_int, w_scale)
    assert np.array_equal(acc, acc_o)
    assert np.array_equal(y, y_o)


def test_bias_and_four_bits():
    tag, T, N, K = oracle.BF16, 70, 520, 384
    xb, s, _, w_int, w_scale = make(T, N, K, tag, 9960, bits=4)
    bias = oracle.bits_of((torch.randn(N, generator=torch.Generator().manual_seed(3)) * 0.5).to(torch.bfloat16))[0]
    y_o, acc_o = oracle.w8a8_linear_per_channel(xb, tag, w_int, w_scale, s, 4, bias)
    y, acc = run(xb, tag, s, w_int, w_scale, 4, bias)
    assert np.array_equal(acc, acc_o) and np.array_equal(y, y_o)


def test_folded_factors_reproduce_the_float_product_on_outlier_channels():
    """The folded form really computes x W^T: the W8A8 result stays within a few percent of the float64 product (the
    outlier channels' large factors now sit in the weight rows, which costs weight resolution), and well below the
    error of one factor for the whole tensor on the same data."""
    tag, T, N, K = oracle.BF16, 256, 512, 1024
    xb, s, w_fp, w_int, w_scale = make(T, N, K, tag, 9970)
    y, _ = run(xb, tag, s, w_int, w_scale)
    ref = oracle.widen(xb, tag).astype(np.float64) @ w_fp.astype(np.float64).T
    err_pc = np.linalg.norm(oracle.widen(y, tag) - ref) / np.linalg.norm(ref)
    s_t = float(oracle.absmax_scale(xb, tag, 8))
    w_int_t, w_scale_t = oracle.quantize_weight(w_fp, 8)
    y_t, _, _ = oracle.w8a8_linear(xb, tag, w_int_t, w_scale_t, s_t, 8)
    err_pt = np.linalg.norm(oracle.widen(y_t, tag) - ref) / np.linalg.norm(ref)
    assert err_pc < 0.07 and err_pc < 0.7 * err_pt, (err_pc, err_pt)


def test_a_zero_factor_is_reported():
    x = torch.ones((4, 32), dtype=torch.bfloat16, device="cuda")
    w = torch.ones((8, 32), dtype=torch.int8, device="cuda")
    sc = torch.ones(32, device="cuda")
    sc[7] = 0.0
    y = torch.empty((4, 8), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(P.sasq_static_w8a8_linear_per_channel_workspace(4, 8, 32), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear_per_channel(x, w, torch.ones(8, device="cuda"), sc, y, workspace=ws)
    assert P.sasq_device_status() == 4
    assert P.sasq_device_status() == 0
