"""GPU parity: the "FP weights" form of the linear (Table 3; fake-quantized activations times 16-bit weights)
against the CPU oracle.

The fake-quantized activations are bit-exact (checked through the workspace).  The contraction accumulates in fp32
on the tensor cores in an order the hardware chooses, so the output is compared with the oracle's float64 result
within a bound derived from the arithmetic: one rounding to the 16-bit output (2^-9 relative for bf16, 2^-12 for
fp16, doubled for the boundary cases) plus K fp32 roundings of partial sums, each at most 2^-23 of
sum_k |x'[t,k] w[n,k]| (the products themselves are exact in fp32).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu

DT = {oracle.F16: torch.float16, oracle.BF16: torch.bfloat16}
OUT_RTOL = {oracle.F16: 2.0 ** -11, oracle.BF16: 2.0 ** -8}


def run_case(T, N, K, tag, seed, bits=8, with_bias=False):
    xb = oracle.bits_of(W.activations(T, K, DT[tag], seed))[0]
    wb = oracle.bits_of((W.weights_fp32(N, K, seed + 1) * 10.0).to(DT[tag]))[0]
    s = float(oracle.absmax_scale(xb[:min(T, W.CALIBRATION_TOKENS)], tag, bits)) * 0.6
    bias = None
    if with_bias:
        bias = oracle.bits_of((torch.randn(N, generator=torch.Generator().manual_seed(seed + 2)) * 0.5).to(DT[tag]))[0]
    x = oracle.tensor_of(xb, tag).cuda()
    y = torch.full((T, N), 7.0, dtype=DT[tag], device="cuda")
    ws = torch.zeros(P.sasq_fakequant_linear_fp_weights_workspace(T, N, K), dtype=torch.uint8, device="cuda")
    P.sasq_fakequant_linear_fp_weights(x, oracle.tensor_of(wb, tag).cuda(), torch.tensor([s], device="cuda"), y,
                                       bias=None if bias is None else oracle.tensor_of(bias, tag).cuda(),
                                       workspace=ws, bits=bits)
    assert P.sasq_device_status() == 0
    # the fake-quantized activations in the workspace (behind the alignment slack): bit-exact
    base = (-ws.data_ptr()) % 128
    xq_gpu = ws[base:base + T * K * 2].view(torch.int16).cpu().numpy().view(np.uint16).reshape(T, K)
    assert np.array_equal(xq_gpu, oracle.fakequant_fwd(xb, tag, s, bits)[0])
    y64, mag = oracle.fp_weights_linear(xb, tag, wb, s, bits, bias)
    got = oracle.widen(oracle.bits_of(y.cpu())[0], tag).astype(np.float64)
    bound = OUT_RTOL[tag] * np.abs(y64) + K * 2.0 ** -23 * mag + 1e-30
    worst = np.max(np.abs(got - y64) / bound)
    assert worst <= 1.0, worst
    return got, y64


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("T,N,K", [(1, 8, 8), (16, 256, 64), (127, 264, 136), (128, 512, 512), (300, 776, 400),
                                   (257, 1024, 2048)])
def test_parity_fp_weights_shapes(tag, T, N, K):
    run_case(T, N, K, tag, 8500 + T + N + K)


@pytest.mark.parametrize("bits", [8, 4])
def test_parity_with_bias_and_low_bits(bits):
    run_case(200, 520, 384, oracle.BF16, 8600 + bits, bits=bits, with_bias=True)


def test_exact_on_small_integers():
    """Operands whose products and sums are exactly representable: the result must be exact, whatever the order."""
    tag, T, N, K = oracle.BF16, 130, 264, 192
    codes = ((np.arange(T)[:, None] * 5 + np.arange(K)[None, :] * 3) % 15 - 7).astype(np.float32)
    w = ((np.arange(N)[:, None] + np.arange(K)[None, :] * 7) % 5 - 2).astype(np.float32)
    x = torch.from_numpy(codes).to(torch.bfloat16).cuda()
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(P.sasq_fakequant_linear_fp_weights_workspace(T, N, K), dtype=torch.uint8, device="cuda")
    P.sasq_fakequant_linear_fp_weights(x, torch.from_numpy(w).to(torch.bfloat16).cuda(), torch.tensor([1.0], device="cuda"),
                                       y, workspace=ws)
    assert P.sasq_device_status() == 0
    want = torch.from_numpy(codes @ w.T).to(torch.bfloat16)            # |sums| < 2^12: exact in fp32, then one narrowing
    assert torch.equal(y.cpu().view(torch.int16), want.view(torch.int16))


def test_llama_shape_sampled():
    got, y64 = run_case(512, 4096, 4096, oracle.BF16, 8700)
    assert np.isfinite(got).all()
