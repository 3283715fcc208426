"""GPU parity: the static W8A8 linear (through the C ABI) against the CPU oracle.

Bars: int32 accumulators bit-exact; the 16-bit output bit-exact as well, because
the epilogue order is fixed (fl32(acc) * fl32(s_x * s_w[n]), bias in fp32, one
narrowing) -- which implies the stated 1e-6 relative bound on the fp32 value.
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


def make_case(T, N, K, tag, seed, spec=W.NORMAL_OUTLIERS, scale_factor=0.6, bits=8):
    x = W.activations(T, K, DT[tag], seed, spec)
    w = W.weights_fp32(N, K, seed + 1)
    xb = oracle.bits_of(x)[0]
    w_int, w_scale = oracle.quantize_weight(w.numpy(), 8)
    calib = xb[:min(T, W.CALIBRATION_TOKENS)]
    s = float(oracle.absmax_scale(calib, tag, bits)) * scale_factor     # a "learned" factor that truncates outliers
    return xb, w_int, w_scale, s


def run_gpu(xb, tag, w_int, w_scale, s, bits=8, bias_bits=None, want_acc=True):
    T, K = xb.shape
    N = w_int.shape[0]
    x = oracle.tensor_of(xb, tag).cuda()
    w = torch.from_numpy(w_int).cuda()
    ws = torch.from_numpy(w_scale).cuda()
    sc = torch.tensor([s], dtype=torch.float32, device="cuda")
    y = torch.empty((T, N), dtype=DT[tag], device="cuda")
    acc = torch.empty((T, N), dtype=torch.int32, device="cuda") if want_acc else None
    bias = None if bias_bits is None else oracle.tensor_of(bias_bits, tag).cuda()
    wsp = torch.empty(max(16, P.sasq_static_w8a8_linear_workspace(T, N, K)), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear(x, w, ws, sc, y, bias=bias, acc_out=acc, workspace=wsp, bits=bits)
    assert P.sasq_device_status() == 0
    return host_bits(y), (None if acc is None else acc.cpu().numpy())


def check(xb, tag, w_int, w_scale, s, bits=8, bias_bits=None, rows=None):
    T = xb.shape[0]
    y_g, acc_g = run_gpu(xb, tag, w_int, w_scale, s, bits, bias_bits)
    if rows is None:
        y_o, y32_o, acc_o = oracle.w8a8_linear(xb, tag, w_int, w_scale, s, bits, bias_bits)
        assert np.array_equal(acc_g, acc_o)
        assert np.array_equal(y_g, y_o)
    else:
        for r0, r1 in rows:
            y_o, y32_o, acc_o = oracle.w8a8_linear(xb, tag, w_int, w_scale, s, bits, bias_bits, row_begin=r0, row_end=r1)
            assert np.array_equal(acc_g[r0:r1], acc_o[r0:r1])
            assert np.array_equal(y_g[r0:r1], y_o[r0:r1])
    # stated tolerance on the value before narrowing: implied by bit equality of y, checked on the widened output
    return y_g, acc_g


def test_structured_operands_locate_layout_mistakes():
    """W rows that pick single columns of x: a wrong swizzle, descriptor or transpose shows up as a wrong column."""
    tag, T, K, N = oracle.BF16, 128, 256, 256
    codes = ((np.arange(T)[:, None] * 3 + np.arange(K)[None, :] * 7) % 255 - 127).astype(np.float32)
    xb = oracle.bits_of(torch.from_numpy(codes).to(torch.bfloat16))[0]       # integers < 256: exact in bf16
    w_int = np.zeros((N, K), np.int8)
    w_int[np.arange(N), (np.arange(N) * 5 + 3) % K] = 1
    w_scale = np.ones(N, np.float32)
    y_g, acc_g = run_gpu(xb, tag, w_int, w_scale, 1.0)
    want = codes[:, (np.arange(N) * 5 + 3) % K].astype(np.int32)
    assert np.array_equal(acc_g, want)
    assert np.array_equal(oracle.widen(y_g, tag), want.astype(np.float32))


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("T,N,K", [(1, 8, 16), (16, 256, 128), (127, 264, 144), (128, 512, 512), (129, 256, 1040),
                                   (300, 776, 400), (257, 1024, 2048)])
def test_parity_small_and_ragged_shapes(tag, T, N, K):
    xb, w_int, w_scale, s = make_case(T, N, K, tag, 7000 + T + N + K)
    check(xb, tag, w_int, w_scale, s)


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
def test_parity_with_bias_and_negative_scale(tag):
    T, N, K = 70, 520, 384
    xb, w_int, w_scale, s = make_case(T, N, K, tag, 7100)
    bias = oracle.bits_of((torch.randn(N, generator=torch.Generator().manual_seed(3)) * 0.5).to(DT[tag]))[0]
    check(xb, tag, w_int, w_scale, s, bias_bits=bias)
    check(xb, tag, w_int, w_scale, -s, bias_bits=bias)


@pytest.mark.parametrize("bits", [4, 2])
def test_parity_low_bit_activations(bits):
    tag, T, N, K = oracle.BF16, 64, 256, 256
    xb, w_int, w_scale, s = make_case(T, N, K, tag, 7200, bits=bits)
    check(xb, tag, w_int, w_scale, s, bits=bits)


def test_saturating_operands_reach_the_int32_extremes():
    tag, T, N, K = oracle.BF16, 128, 256, 11008
    xb = oracle.bits_of(torch.full((T, K), -1000.0).to(torch.bfloat16))[0]     # every code is -128
    w_int = np.full((N, K), -128, np.int8)
    w_int[1::2] = 127
    y_g, acc_g = run_gpu(xb, tag, w_int, np.ones(N, np.float32), 1.0)
    assert np.all(acc_g[:, 0::2] == K * 128 * 128) and np.all(acc_g[:, 1::2] == -K * 128 * 127)


def test_config1_single_linear_full_check():
    """T=128, K=N=4096, fp16, weights N(0, 0.02) quantized per output channel, s = max|x[0:64]|/127."""
    tag, T, N, K = oracle.F16, 128, 4096, 4096
    x = W.activations(T, K, torch.float16, W.seed_of(1, 0))
    w = W.weights_fp32(N, K, W.seed_of(1, 1))
    xb = oracle.bits_of(x)[0]
    w_int, w_scale = oracle.quantize_weight(w.numpy(), 8)
    s = float(oracle.absmax_scale(xb[:W.CALIBRATION_TOKENS], tag, 8))
    check(xb, tag, w_int, w_scale, s)


@pytest.mark.parametrize("T", [1, 16, 2048])
def test_llama7b_shapes_sampled_rows(T):
    """q_proj (4096 -> 4096) and down_proj (11008 -> 4096) at decode / prefill token counts, with a learned
    factor that saturates outliers; every row for small T, 3 row bands otherwise."""
    tag = oracle.BF16
    for li, (K, N) in enumerate([(4096, 4096), (11008, 4096)]):
        x = W.activations(T, K, torch.bfloat16, W.seed_of(3, li))
        xb = oracle.bits_of(x)[0]
        w = W.weights_fp32(N, K, W.seed_of(3, 10 + li))
        w_int, w_scale = oracle.quantize_weight(w.numpy(), 8)
        s = float(oracle.absmax_scale(xb[:min(T, 64)], tag, 8)) * W.learned_scale_factor(W.seed_of(3, li))
        rows = None if T <= 16 else [(0, 8), (1021, 1029), (T - 8, T)]
        check(xb, tag, w_int, w_scale, s, rows=rows)


def test_more_channel_tiles_than_sms_takes_the_general_small_t_kernel():
    """T <= 128 with more 128-channel tiles than the chip has SMs (N = 19200 > 148 x 128): the clustered small-T
    kernel does not apply (its in-kernel quantizer needs every CTA resident), the 128 x 256-tile kernel with the
    quantizer as a launch of its own does."""
    tag, T, N, K = oracle.BF16, 24, 19200, 80
    xb, w_int, w_scale, s = make_case(T, N, K, tag, 7400)
    check(xb, tag, w_int, w_scale, s)


def test_output_is_deterministic():
    tag, T, N, K = oracle.BF16, 256, 512, 1024
    xb, w_int, w_scale, s = make_case(T, N, K, tag, 7300)
    a = run_gpu(xb, tag, w_int, w_scale, s)
    b = run_gpu(xb, tag, w_int, w_scale, s)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_unsupported_shapes_and_bad_scale_are_reported():
    x = torch.zeros((4, 24), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((8, 24), dtype=torch.int8, device="cuda")
    ws = torch.ones(8, device="cuda")
    sc = torch.ones(1, device="cuda")
    y = torch.empty((4, 8), dtype=torch.bfloat16, device="cuda")
    wsp = torch.empty(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(P.SasqError) as e:
        P.sasq_static_w8a8_linear(x, w, ws, sc, y, workspace=wsp)        # K % 16 != 0
    assert e.value.status == 2
    x = torch.zeros((4, 32), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((8, 32), dtype=torch.int8, device="cuda")
    with pytest.raises(P.SasqError) as e:
        P.sasq_static_w8a8_linear(x, w, ws, sc, y, workspace=None)       # workspace missing
    assert e.value.status == 3
    sc.zero_()
    P.sasq_static_w8a8_linear(x, w, ws, sc, y, workspace=wsp)
    assert P.sasq_device_status() == 4
    assert P.sasq_device_status() == 0


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("T,N,K,bits", [(1, 136, 144, 8), (5, 264, 1040, 8), (16, 520, 400, 8), (9, 4096, 11008, 8),
                                        (16, 1032, 2064, 4), (3, 11008, 4096, 8), (17, 264, 1040, 8), (32, 520, 400, 8)])
def test_parity_decode_sizes_with_ragged_k_and_bias(tag, T, N, K, bits):
    """Up to 16 rows every CTA of the small-T kernel quantizes its own K slice into shared memory (K not a multiple of
    128, rows padded to 16, slices of unequal length); 17 and 32 rows take the path through global memory.  All rows
    and all accumulators against the oracle, with a bias and with a negative factor."""
    xb, w_int, w_scale, s = make_case(T, N, K, tag, 7300 + T + N, bits=bits)
    bias = oracle.bits_of((torch.randn(N, generator=torch.Generator().manual_seed(T)) * 0.5).to(DT[tag]))[0]
    check(xb, tag, w_int, w_scale, s, bits=bits)
    check(xb, tag, w_int, w_scale, -s, bits=bits, bias_bits=bias)
