"""Pins for the CPU oracle's static W8A8 linear (Eq. 2), grouped form (Eq. 3),
weight quantizer (Eq. 1 per output channel) and dequantisation.

The integer GEMM is checked against numpy's int64 matmul (an independent
library routine), against the oracle's own 64-bit brute-force twin, and on
structured operands with known answers; the epilogue against exact small
integers and float64.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import BF16, F16

TAGS = [F16, BF16]
TDT = {F16: torch.float16, BF16: torch.bfloat16}


def to_bits(vals, tag):
    return oracle.bits_of(torch.as_tensor(np.asarray(vals, dtype=np.float64)).to(TDT[tag]))[0]


def from_bits(bits, tag):
    return oracle.tensor_of(bits, tag).to(torch.float64).numpy()


def _rand_int8(rng, shape, full_range=True):
    lo, hi = (-128, 128) if full_range else (-20, 21)
    return rng.integers(lo, hi, size=shape, dtype=np.int64).astype(np.int8)


@pytest.mark.parametrize("T,N,K", [(1, 1, 1), (3, 5, 7), (17, 33, 129), (64, 48, 512)])
def test_int_gemm_vs_numpy_int64_and_brute_force(T, N, K):
    rng = np.random.default_rng(100 + T)
    x = _rand_int8(rng, (T, K))
    w = _rand_int8(rng, (N, K))
    acc = oracle.int_gemm(x, w)
    ref = x.astype(np.int64) @ w.astype(np.int64).T
    assert np.array_equal(acc.astype(np.int64), ref)
    assert np.array_equal(oracle.int_gemm_i64(x, w), ref)
    assert np.abs(acc).max() <= K * 128 * 128


def test_int_gemm_extreme_values_do_not_overflow():
    K = 11008
    x = np.full((2, K), -128, np.int8)
    w = np.full((3, K), -128, np.int8)
    w[1] = 127
    acc = oracle.int_gemm(x, w)
    assert acc[0, 0] == K * 16384 and acc[0, 1] == -K * 128 * 127


def test_int_gemm_structured_operands():
    rng = np.random.default_rng(7)
    K = 96
    x = _rand_int8(rng, (10, K))
    eye = np.eye(K, dtype=np.int8)
    assert np.array_equal(oracle.int_gemm(x, eye), x.astype(np.int32))            # W = I copies the row
    ones = np.ones((4, K), np.int8)
    assert np.array_equal(oracle.int_gemm(x, ones), np.repeat(x.astype(np.int32).sum(1, keepdims=True), 4, 1))
    # transposed operands would break this: a one-hot W row n picks column n+1 of x
    pick = np.zeros((K - 1, K), np.int8)
    pick[np.arange(K - 1), np.arange(1, K)] = 1
    assert np.array_equal(oracle.int_gemm(x, pick), x[:, 1:].astype(np.int32))


def test_int_gemm_rows_are_independent_and_row_range_is_respected():
    rng = np.random.default_rng(8)
    x = _rand_int8(rng, (12, 40))
    w = _rand_int8(rng, (9, 40))
    full = oracle.int_gemm(x, w)
    part = oracle.int_gemm(x, w, 3, 7)
    assert np.array_equal(part[3:7], full[3:7])
    assert not part[:3].any() and not part[7:].any()
    x2 = x.copy()
    x2[5] = 0
    chg = oracle.int_gemm(x2, w)
    assert np.array_equal(np.delete(chg, 5, 0), np.delete(full, 5, 0)) and not chg[5].any()


@pytest.mark.parametrize("tag", TAGS)
def test_dequant_unit_scales_is_exact_for_small_integers(tag):
    lim = 2 ** 11 if tag == F16 else 2 ** 8
    acc = np.arange(-lim, lim + 1, dtype=np.int32).reshape(1, -1)
    N = acc.shape[1]
    y, y32 = oracle.dequant(acc, np.ones(N, np.float32), 1.0, tag)
    assert np.array_equal(y32, acc.astype(np.float32))
    assert np.array_equal(from_bits(y, tag), acc.astype(np.float64))


@pytest.mark.parametrize("tag", TAGS)
def test_dequant_vs_float64(tag):
    rng = np.random.default_rng(9)
    T, N = 7, 300
    acc = rng.integers(-2**27, 2**27, size=(T, N)).astype(np.int32)
    ws = (rng.random(N) * 1e-3 + 1e-5).astype(np.float32)
    sx = np.float32(0.0173)
    bias = to_bits(rng.standard_normal(N), tag)
    y, y32 = oracle.dequant(acc, ws, float(sx), tag)
    ref = acc.astype(np.float64) * (float(sx) * ws.astype(np.float64))[None, :]
    assert np.all(np.abs(y32 - ref) <= 3 * 2.0 ** -24 * np.abs(ref))       # int->fp32, scale product, final product
    ulp = 2.0 ** -10 if tag == F16 else 2.0 ** -7
    assert np.all(np.abs(from_bits(y, tag) - ref) <= (ulp / 2 + 1e-6) * np.abs(ref))
    # bias is added in fp32 before the single narrowing (Sec. 3: bias is not quantized)
    yb, yb32 = oracle.dequant(acc, ws, float(sx), tag, bias=bias)
    refb = ref + from_bits(bias, tag)[None, :]
    assert np.all(np.abs(yb32 - refb) <= 4 * 2.0 ** -24 * (np.abs(ref) + np.abs(refb)))
    # channel n uses w_scale[n]: a permuted scale vector must change the answer
    y_perm, _ = oracle.dequant(acc, ws[::-1].copy(), float(sx), tag)
    assert not np.array_equal(y_perm, y)


def test_weight_quantizer_invariants():
    rng = np.random.default_rng(10)
    N, K = 37, 200
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    w[5] = 0.0
    w[6, 3] = 1.0     # a dominant element
    w_int, ws = oracle.quantize_weight(w)
    amax = np.abs(w).max(1)
    nz = amax > 0
    assert np.array_equal(ws[nz], (amax[nz] / np.float32(127)).astype(np.float32))
    assert ws[5] == 1.0 and not w_int[5].any()
    assert np.array_equal(np.abs(w_int.astype(np.int32)).max(1)[nz], np.full(nz.sum(), 127))   # Eq. 1: max maps to Qp
    assert w_int[6, 3] == 127
    err = np.abs(w.astype(np.float64) - w_int.astype(np.float64) * ws[:, None].astype(np.float64))
    assert np.all(err <= ws[:, None] / 2 * (1 + 1e-5))
    # per output channel means per ROW of w[N, K]: scaling one row changes only that row's factor
    w2 = w.copy()
    w2[9] *= 3
    _, ws2 = oracle.quantize_weight(w2)
    assert ws2[9] != ws[9] and np.array_equal(np.delete(ws2, 9), np.delete(ws, 9))


@pytest.mark.parametrize("tag", TAGS)
def test_w8a8_linear_is_the_composition_and_tracks_the_float_product(tag):
    rng = np.random.default_rng(11)
    T, N, K = 9, 40, 256
    xv = rng.standard_normal((T, K))
    x = to_bits(xv, tag)
    xv = from_bits(x, tag)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    w_int, ws = oracle.quantize_weight(w)
    s = float(oracle.absmax_scale(x, tag, 8))
    y, y32, acc = oracle.w8a8_linear(x, tag, w_int, ws, s)
    codes = oracle.quantize_act(x, tag, s)
    assert np.array_equal(acc, oracle.int_gemm(codes, w_int))
    y_c, y32_c = oracle.dequant(acc, ws, s, tag)
    assert np.array_equal(y, y_c) and np.array_equal(y32, y32_c)
    # Eq. 2: the quantized product approximates X W^T
    ref = xv @ w.astype(np.float64).T
    rel = np.linalg.norm(y32 - ref) / np.linalg.norm(ref)
    assert rel < 0.02
    # row range
    yp, _, accp = oracle.w8a8_linear(x, tag, w_int, ws, s, row_begin=2, row_end=5)
    assert np.array_equal(yp[2:5], y[2:5]) and not accp[:2].any() and not accp[5:].any()


@pytest.mark.parametrize("tag", TAGS)
def test_grouped_form_reduces_to_eq2_and_matches_float64_eq3(tag):
    rng = np.random.default_rng(12)
    T, N, K, group = 5, 24, 128, 32
    x = to_bits(rng.standard_normal((T, K)) * 2, tag)
    w_int = _rand_int8(rng, (N, K))
    ws = (rng.random(N) * 1e-3 + 1e-4).astype(np.float32)
    s = 0.031
    # one group spanning K is Eq. 2
    y1, y32_1 = oracle.w8a8_linear_grouped(x, tag, w_int, ws, np.array([s], np.float32), K)
    y2, y32_2, _ = oracle.w8a8_linear(x, tag, w_int, ws, s)
    assert np.array_equal(y32_1, y32_2) and np.array_equal(y1, y2)
    # several groups with distinct factors: float64 evaluation of Eq. 3 from the per-group codes
    sg = np.array([0.031, 0.5, 0.0077, 0.12], np.float32)
    y, y32 = oracle.w8a8_linear_grouped(x, tag, w_int, ws, sg, group)
    ref = np.zeros((T, N))
    for gi in range(K // group):
        sl = slice(gi * group, (gi + 1) * group)
        codes = oracle.quantize_act(np.ascontiguousarray(x[:, sl]), tag, float(sg[gi]))
        ref += float(sg[gi]) * (codes.astype(np.int64) @ w_int[:, sl].astype(np.int64).T) * ws[None, :].astype(np.float64)
    assert np.all(np.abs(y32 - ref) <= 1e-5 * np.abs(ref).max())


def test_dynamic_per_token_linear_against_numpy_on_small_inputs():
    """Sec. 4.4 generation phase: every row has its own max-based factor.  Checked against the definition typed in
    numpy float32 / int64 (power-of-two-free data, so rounding decisions are generic), plus the all-zero row."""
    rng = np.random.default_rng(11)
    T, K, N = 5, 48, 24
    x = (rng.normal(0, 2, (T, K))).astype(np.float32)
    x[3] = 0.0
    xb = oracle.bits_of(torch.from_numpy(x).to(torch.bfloat16))[0]
    xw = oracle.widen(xb, oracle.BF16)                      # the bf16 values as float32
    w_int = rng.integers(-127, 128, (N, K)).astype(np.int8)
    w_scale = rng.uniform(1e-3, 2e-3, N).astype(np.float32)
    y, acc, s = oracle.w8a8_linear_dynamic(xb, oracle.BF16, w_int, w_scale)
    for t in range(T):
        amax = np.abs(xw[t]).max()
        st = np.float32(amax) / np.float32(127) if amax > 0 else np.float32(1)
        assert s[t] == st
        inv = np.float32(1) / st
        codes = np.clip(np.rint((xw[t] * inv).astype(np.float32)), -128, 127).astype(np.int64)
        a = codes @ w_int.astype(np.int64).T
        assert np.array_equal(acc[t], a)
        y32 = a.astype(np.float32) * (st * w_scale).astype(np.float32)
        assert np.array_equal(y[t], oracle.narrow(y32.astype(np.float32), oracle.BF16))
    assert not acc[3].any() and np.abs(np.clip(acc, None, None)).max() > 0
    assert np.abs(oracle.quantize_act(xb[0:1], oracle.BF16, float(s[0]), 8)).max() == 127     # the row maximum maps to Qp


@pytest.mark.parametrize("tag", TAGS)
def test_per_channel_linear_with_a_constant_factor_is_eq2_on_folded_weights(tag):
    """Sec. 5.1 granularity (per-channel activations), static form: with the same factor c on every channel,
    folding it into the frozen weights (w' = w*c, quantized per output channel) and then leaving the activation
    factor out of the epilogue must give the per-tensor Eq. 2 result on the same folded weights with s_x = 1
    in the epilogue but codes taken with c, bit for bit.  The per-tensor pieces are pinned above."""
    rng = np.random.default_rng(21)
    T, N, K = 6, 24, 96
    x = to_bits(rng.standard_normal((T, K)) * 3, tag)
    c = np.float32(0.043)
    w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    w_int, ws = oracle.quantize_weight((w * c).astype(np.float32))
    y, acc = oracle.w8a8_linear_per_channel(x, tag, w_int, ws, np.full(K, c, np.float32))
    codes = oracle.quantize_act(x, tag, float(c))                       # Eq. 1 with the common factor
    acc_ref = oracle.int_gemm(codes, w_int)
    assert np.array_equal(acc, acc_ref)
    y_ref, _ = oracle.dequant(acc_ref, ws, 1.0, tag)
    assert np.array_equal(y, y_ref)
    # the per-tensor linear applies s_x in its epilogue: on the folded weights that would count c twice
    y_twice, _, acc_t = oracle.w8a8_linear(x, tag, w_int, ws, float(c))
    assert np.array_equal(acc_t, acc) and not np.array_equal(y_twice, y)


@pytest.mark.parametrize("tag", TAGS)
def test_per_channel_linear_against_exact_arithmetic_on_tiny_operands(tag):
    """Eq. 1 per channel + Eq. 2 with the activation factors inside the weights, evaluated exactly: power-of-two
    factors make every code an exact integer computed with Fractions, the accumulators are exact integer sums, and
    with power-of-two w_scale the product acc*w_scale[n] is exact in fp32 (under 24 bits), so the output is that
    rational number narrowed once (torch's conversion, an independent library routine).  A wrong output factor
    (any activation factor left in the epilogue), a factor taken from the wrong channel or a transposed weight
    fails here."""
    from fractions import Fraction
    rng = np.random.default_rng(22)
    T, N, K = 4, 5, 6
    s_vec = np.array([0.5, 0.25, 2.0, 1.0, 0.125, 4.0], np.float32)
    # values on a 1/16 grid: exactly representable in both 16-bit types, with ties and clipping among them
    xv = rng.integers(-64, 65, size=(T, K)) / 16.0
    xv[0, 0] = 0.25          # 0.25/0.5 = 0.5  -> tie, rounds to 0
    xv[0, 1] = 0.375         # 0.375/0.25 = 1.5 -> tie, rounds to 2
    xv[1, 4] = 40.0          # 40/0.125 = 320 -> clips to 127
    xv[2, 4] = -40.0         # clips to -128
    x = to_bits(xv, tag)
    w_int = rng.integers(-5, 6, size=(N, K)).astype(np.int8)
    ws = np.array([1.0, 0.5, 2.0, 0.25, 4.0], np.float32)
    y, acc = oracle.w8a8_linear_per_channel(x, tag, w_int, ws, s_vec)

    def rne(fr):
        fl = fr.numerator // fr.denominator
        rem = fr - fl
        if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
            return fl + 1
        return fl

    codes = [[min(max(rne(Fraction(float(xv[t, k])) / Fraction(float(s_vec[k]))), -128), 127) for k in range(K)]
             for t in range(T)]
    assert codes[0][0] == 0 and codes[0][1] == 2 and codes[1][4] == 127 and codes[2][4] == -128
    for t in range(T):
        for n in range(N):
            a = sum(codes[t][k] * int(w_int[n, k]) for k in range(K))
            assert int(acc[t, n]) == a
            exact = Fraction(a) * Fraction(float(ws[n]))
            assert abs(a) < 2 ** 24 and Fraction(float(exact)) == exact       # exact in fp32 and in a double
            want = torch.tensor([float(exact)], dtype=torch.float32).to(TDT[tag]).to(torch.float64).item()
            assert float(from_bits(y[t:t + 1, n:n + 1], tag)[0, 0]) == want


def test_per_channel_linear_planted_mistakes_fail_the_pins():
    """What the two pins above catch, shown on the CPU: an activation factor left in the epilogue, and the
    factors applied to the wrong channels."""
    rng = np.random.default_rng(23)
    T, N, K = 3, 4, 8
    tag = BF16
    s_vec = (2.0 ** rng.integers(-3, 3, K)).astype(np.float32)
    x = to_bits(rng.integers(-64, 65, size=(T, K)) / 16.0, tag)
    w_int = rng.integers(-5, 6, size=(N, K)).astype(np.int8)
    ws = np.ones(N, np.float32)
    y, acc = oracle.w8a8_linear_per_channel(x, tag, w_int, ws, s_vec)
    _, codes = oracle.fakequant_fwd_per_channel(x, tag, s_vec)
    y_bad, _ = oracle.dequant(oracle.int_gemm(codes.astype(np.int8), w_int), ws, 0.5, tag)
    assert not np.array_equal(y_bad, y)
    _, acc_rev = oracle.w8a8_linear_per_channel(x, tag, w_int, ws, s_vec[::-1].copy())
    assert not np.array_equal(acc_rev, acc)
