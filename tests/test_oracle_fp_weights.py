"""Pins of the oracle's "FP weights" form (Table 3; Eq. 5 / 6): Y = g(X) W^T with 16-bit floating-point weights.

The routine composes the pinned fake-quant forward with a float64 library matmul; what is pinned here is the
composition: operand order (W is [N, K], one row per output channel), the use of the fake-quantized and not the raw
activations, and the bias.
"""
from fractions import Fraction

import numpy as np
import torch

import oracle
import sasq_workloads as W


def case(T, N, K, tag, seed):
    dt = torch.float16 if tag == oracle.F16 else torch.bfloat16
    xb = oracle.bits_of(W.activations(T, K, dt, seed))[0]
    wb = oracle.bits_of(W.weights_fp32(N, K, seed + 1).to(dt))[0]
    s = float(oracle.absmax_scale(xb, tag, 8)) * 0.5
    return xb, wb, s


def test_brute_force_on_a_tiny_case_with_exact_rationals():
    tag, T, N, K = oracle.BF16, 3, 5, 7
    xb, wb, s = case(T, N, K, tag, 41)
    bias = oracle.bits_of(torch.tensor([0.5, -1.25, 3.0, 0.0, -0.75]).to(torch.bfloat16))[0]
    y, mag = oracle.fp_weights_linear(xb, tag, wb, s, 8, bias)
    xq = oracle.widen(oracle.fakequant_fwd(xb, tag, s, 8)[0], tag)
    w = oracle.widen(wb, tag)
    b = oracle.widen(bias, tag)
    for t in range(T):
        for n in range(N):
            exact = sum(Fraction(float(xq[t, k])) * Fraction(float(w[n, k])) for k in range(K)) + Fraction(float(b[n]))
            assert abs(Fraction(float(y[t, n])) - exact) <= abs(exact) * Fraction(1, 10 ** 12) + Fraction(1, 10 ** 15)
            assert mag[t, n] >= abs(y[t, n]) - 1e-12


def test_uses_the_fake_quantized_activations_not_the_raw_ones():
    tag, T, N, K = oracle.F16, 4, 6, 16
    xb, wb, s = case(T, N, K, tag, 42)
    y, _ = oracle.fp_weights_linear(xb, tag, wb, s, 4)              # 4 bits: X' differs visibly from X
    raw = oracle.widen(xb, tag).astype(np.float64) @ oracle.widen(wb, tag).astype(np.float64).T
    xq = oracle.widen(oracle.fakequant_fwd(xb, tag, s, 4)[0], tag).astype(np.float64)
    assert np.allclose(y, xq @ oracle.widen(wb, tag).astype(np.float64).T, rtol=0, atol=0)
    assert not np.allclose(y, raw, rtol=1e-3, atol=1e-6)


def test_operand_orientation_with_structured_weights():
    """W rows that pick single columns of X': a transposed operand or a wrong row/column shows up at once."""
    tag, T, N, K = oracle.BF16, 5, 8, 8
    codes = (np.arange(T)[:, None] * 3 + np.arange(K)[None, :] - 10).astype(np.float32)      # small integers
    xb = oracle.bits_of(torch.from_numpy(codes).to(torch.bfloat16))[0]
    w = np.zeros((N, K), np.float32)
    pick = (np.arange(N) * 3 + 1) % K
    w[np.arange(N), pick] = 2.0
    wb = oracle.bits_of(torch.from_numpy(w).to(torch.bfloat16))[0]
    y, _ = oracle.fp_weights_linear(xb, tag, wb, 1.0, 8)            # s = 1: integers within the code range pass
    assert np.array_equal(y, 2.0 * codes[:, pick].astype(np.float64))
