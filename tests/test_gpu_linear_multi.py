"""GPU parity of sasq_static_w8a8_linear_multi: several independent static W8A8 linears submitted together.

Problems with T > 128 share launches of the CTA-pair kernel (one tile list and one quantizer chunk list over all of
them); the others run on their own.  The bar is that of the single linear: every output bit-exact against the CPU
oracle (small shapes, every element) and, at the sizes of a LLaMA-2-7B layer, bit-identical to separate calls
plus oracle rows.
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


def make_problem(T, N, K, tag, seed, with_bias=False, bits=8):
    w = W.weights_fp32(N, K, seed + 1)
    xb = oracle.bits_of(W.activations(T, K, DT[tag], seed))[0] if T > 0 else np.zeros((0, K), np.uint16)
    w_int, w_scale = oracle.quantize_weight(w.numpy(), 8)
    if T > 0:
        s = float(oracle.absmax_scale(xb[:min(T, W.CALIBRATION_TOKENS)], tag, bits)) * 0.6
    else:
        s = 1.0
    bias = None
    if with_bias:
        bias = oracle.bits_of((torch.randn(N, generator=torch.Generator().manual_seed(seed + 2)) * 0.5).to(DT[tag]))[0]
    return dict(T=T, N=N, K=K, xb=xb, w_int=w_int, w_scale=w_scale, s=s, bias=bias)


def run_multi(problems, tag, bits=8):
    dev = []
    for pr in problems:
        x = oracle.tensor_of(pr["xb"], tag).cuda() if pr["T"] > 0 else torch.empty((0, pr["K"]), dtype=DT[tag],
                                                                                    device="cuda")
        y = torch.full((pr["T"], pr["N"]), 7.0, dtype=DT[tag], device="cuda")
        bias = None if pr["bias"] is None else oracle.tensor_of(pr["bias"], tag).cuda()
        dev.append((x, torch.from_numpy(pr["w_int"]).cuda(), torch.from_numpy(pr["w_scale"]).cuda(),
                    torch.tensor([pr["s"]], dtype=torch.float32, device="cuda"), y, bias))
    need = P.sasq_static_w8a8_linear_multi_workspace([(pr["T"], pr["N"], pr["K"]) for pr in problems])
    ws = torch.empty(max(16, need), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear_multi(dev, ws, bits=bits)
    assert P.sasq_device_status() == 0
    return [host_bits(d[4]) for d in dev]


def check_against_oracle(problems, tag, bits=8):
    ys = run_multi(problems, tag, bits)
    for i, (pr, y_g) in enumerate(zip(problems, ys)):
        if pr["T"] == 0:
            continue
        y_o, _, _ = oracle.w8a8_linear(pr["xb"], tag, pr["w_int"], pr["w_scale"], pr["s"], bits, pr["bias"])
        assert np.array_equal(y_g, y_o), i


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
def test_group_of_ragged_problems_matches_the_oracle(tag):
    """Different T, N and K in one launch: ragged row blocks, 16-column tails, one problem with a bias."""
    problems = [make_problem(300, 264, 256, tag, 9100),
                make_problem(129, 512, 128, tag, 9110),
                make_problem(700, 136, 320, tag, 9120, with_bias=True),
                make_problem(513, 776, 400, tag, 9130)]
    check_against_oracle(problems, tag)


def test_single_problem_and_empty_call():
    tag = oracle.BF16
    check_against_oracle([make_problem(260, 520, 144, tag, 9200)], tag)
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear_multi([], ws)                     # nothing to do is not an error
    assert P.sasq_device_status() == 0


def test_small_t_and_empty_problems_between_larger_ones():
    """A run with T <= 128 problems whose tiles do not fill the chip is launched problem by problem, in order; a
    T = 0 problem is skipped."""
    tag = oracle.BF16
    problems = [make_problem(257, 256, 256, tag, 9300),
                make_problem(64, 264, 144, tag, 9310),
                make_problem(0, 128, 64, tag, 9320),
                make_problem(1, 136, 528, tag, 9330, with_bias=True),
                make_problem(384, 128, 1040, tag, 9340),
                make_problem(200, 520, 96, tag, 9350)]
    assert P.sasq_static_w8a8_linear_multi_launches([(pr["T"], pr["N"], pr["K"]) for pr in problems]) == 5
    check_against_oracle(problems, tag)


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
def test_small_t_problems_that_fill_the_chip_share_one_launch(tag):
    """Decode-sized problems (T = 1, 16, 128) with enough output tiles for every CTA pair, and a T > 128 problem
    among them, run in ONE launch of the CTA-pair kernel; every element against the oracle."""
    problems = [make_problem(16, 11008, 256, tag, 9700),
                make_problem(1, 4096, 144, tag, 9710, with_bias=True),
                make_problem(128, 11008, 128, tag, 9720),
                make_problem(300, 520, 96, tag, 9730),
                make_problem(77, 4104, 64, tag, 9740)]
    assert P.sasq_static_w8a8_linear_multi_launches([(pr["T"], pr["N"], pr["K"]) for pr in problems]) == 1
    check_against_oracle(problems, tag)


def test_single_row_block_problems_take_the_cost_dealt_tile_lists():
    """Problems of up to 256 rows (one row block each) with different K: their tiles are dealt out by cost instead
    of round-robin; with more than 32 rows the launch keeps the five-stage layout."""
    tag = oracle.BF16
    problems = [make_problem(200, 11008, 128, tag, 9800),
                make_problem(256, 11008, 64, tag, 9810, with_bias=True),
                make_problem(130, 4096, 320, tag, 9820),
                make_problem(33, 4104, 48, tag, 9830)]
    assert P.sasq_static_w8a8_linear_multi_launches([(pr["T"], pr["N"], pr["K"]) for pr in problems]) == 1
    check_against_oracle(problems, tag)


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("T", [1, 16, 100])
def test_same_t_small_problems_share_a_launch_of_the_small_t_kernel(tag, T):
    """Too few tiles for the CTA pairs, but all 128-channel tiles fit the device: one launch of the small-T kernel
    over three problems with different N and K (the K split is limited by the shortest), one with a bias."""
    problems = [make_problem(T, 1032, 512, tag, 9900 + T),
                make_problem(T, 520, 2048, tag, 9910 + T, with_bias=True),
                make_problem(T, 2048, 256, tag, 9920 + T)]
    assert P.sasq_static_w8a8_linear_multi_launches([(pr["T"], pr["N"], pr["K"]) for pr in problems]) == 1
    check_against_oracle(problems, tag)


def test_llama7b_qkv_at_decode_size_share_a_small_t_launch():
    tag, T = oracle.BF16, 16
    problems = [make_problem(T, 4096, 4096, tag, 9950 + i) for i in range(3)]
    assert P.sasq_static_w8a8_linear_multi_launches([(pr["T"], pr["N"], pr["K"]) for pr in problems]) == 1
    check_against_oracle(problems, tag)


def test_llama7b_layer_at_decode_size_in_one_launch():
    """The seven linears of a LLaMA-2-7B layer at T = 16: one launch, every output row against the oracle for three
    of them, all seven bit-identical to separate calls (which take the small-T kernel)."""
    tag, T = oracle.BF16, 16
    probs, singles = [], []
    for li, (name, K, N) in enumerate(W.LLAMA2_7B_LINEARS):
        x = W.activations(T, K, torch.bfloat16, W.seed_of(3, 60 + li), device="cuda")
        w = W.weights_fp32(N, K, W.seed_of(3, 70 + li), device="cuda")
        w_int = torch.empty((N, K), dtype=torch.int8, device="cuda")
        w_scale = torch.empty(N, dtype=torch.float32, device="cuda")
        P.sasq_quantize_weight(w, w_int, w_scale, 8)
        s = float(oracle.absmax_scale(oracle.bits_of(x.cpu())[0], tag, 8)) * W.learned_scale_factor(W.seed_of(3, li))
        sc = torch.tensor([s], dtype=torch.float32, device="cuda")
        y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
        probs.append((x, w_int, w_scale, sc, y))
        y1 = torch.empty_like(y)
        ws1 = torch.empty(P.sasq_static_w8a8_linear_workspace(T, N, K), dtype=torch.uint8, device="cuda")
        P.sasq_static_w8a8_linear(x, w_int, w_scale, sc, y1, workspace=ws1)
        singles.append((y1, s))
    shapes = [(T, N, K) for _, K, N in W.LLAMA2_7B_LINEARS]
    assert P.sasq_static_w8a8_linear_multi_launches(shapes) == 1
    ws = torch.empty(P.sasq_static_w8a8_linear_multi_workspace(shapes), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear_multi(probs, ws)
    assert P.sasq_device_status() == 0
    for li, ((x, w_int, w_scale, sc, y), (y1, s)) in enumerate(zip(probs, singles)):
        assert torch.equal(y.view(torch.int16), y1.view(torch.int16)), li
        if li in (0, 5, 6):
            y_o, _, _ = oracle.w8a8_linear(oracle.bits_of(x.cpu())[0], tag, w_int.cpu().numpy(), w_scale.cpu().numpy(),
                                           s, 8)
            assert np.array_equal(host_bits(y), y_o), li


def test_more_problems_than_one_launch_holds():
    tag = oracle.BF16
    problems = [make_problem(130 + 37 * i, 128 + 8 * i, 64 + 16 * i, tag, 9400 + 10 * i) for i in range(11)]
    assert P.sasq_static_w8a8_linear_multi_launches([(pr["T"], pr["N"], pr["K"]) for pr in problems]) == 2
    check_against_oracle(problems, tag)


def test_low_bit_group():
    tag = oracle.BF16
    problems = [make_problem(300, 256, 256, tag, 9500, bits=4), make_problem(140, 264, 128, tag, 9510, bits=4)]
    check_against_oracle(problems, tag, bits=4)


def test_llama7b_layer_group_equals_separate_calls_and_oracle_rows():
    """The seven linears of a LLaMA-2-7B layer at T = 2048 in one call: bit-identical to seven separate calls, and
    sampled rows of every output bit-exact against the oracle."""
    tag, T = oracle.BF16, 2048
    rows = [0, 1, 255, 256, 257, 1023, 1024, T - 1]
    idx = torch.tensor(rows, device="cuda")
    probs, singles = [], []
    for li, (name, K, N) in enumerate(W.LLAMA2_7B_LINEARS):
        x = W.activations(T, K, torch.bfloat16, W.seed_of(3, 40 + li), device="cuda")
        w = W.weights_fp32(N, K, W.seed_of(3, 50 + li), device="cuda")
        w_int = torch.empty((N, K), dtype=torch.int8, device="cuda")
        w_scale = torch.empty(N, dtype=torch.float32, device="cuda")
        P.sasq_quantize_weight(w, w_int, w_scale, 8)
        calib = oracle.bits_of(x[:W.CALIBRATION_TOKENS].cpu())[0]
        s = float(oracle.absmax_scale(calib, tag, 8)) * W.learned_scale_factor(W.seed_of(3, li))
        sc = torch.tensor([s], dtype=torch.float32, device="cuda")
        y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
        probs.append((x, w_int, w_scale, sc, y))
        y1 = torch.empty_like(y)
        ws1 = torch.empty(P.sasq_static_w8a8_linear_workspace(T, N, K), dtype=torch.uint8, device="cuda")
        P.sasq_static_w8a8_linear(x, w_int, w_scale, sc, y1, workspace=ws1)
        singles.append((y1, s))
    need = P.sasq_static_w8a8_linear_multi_workspace([(T, N, K) for _, K, N in W.LLAMA2_7B_LINEARS])
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    assert P.sasq_static_w8a8_linear_multi_launches([(T, N, K) for _, K, N in W.LLAMA2_7B_LINEARS]) == 1
    P.sasq_static_w8a8_linear_multi(probs, ws)
    assert P.sasq_device_status() == 0
    for li, ((x, w_int, w_scale, sc, y), (y1, s)) in enumerate(zip(probs, singles)):
        assert torch.equal(y.view(torch.int16), y1.view(torch.int16)), li
        if li in (0, 4, 6):
            xb = oracle.bits_of(x[idx].cpu())[0]
            y_o, _, _ = oracle.w8a8_linear(xb, tag, w_int.cpu().numpy(), w_scale.cpu().numpy(), s, 8)
            assert np.array_equal(host_bits(y[idx]), y_o), li


def test_argument_errors_are_reported_before_any_launch():
    tag = oracle.BF16
    good = make_problem(256, 128, 64, tag, 9600)
    x = oracle.tensor_of(good["xb"], tag).cuda()
    w = torch.from_numpy(good["w_int"]).cuda()
    wsc = torch.from_numpy(good["w_scale"]).cuda()
    sc = torch.tensor([good["s"]], dtype=torch.float32, device="cuda")
    y = torch.full((256, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(P.sasq_static_w8a8_linear_multi_workspace([(256, 128, 64)] * 2), dtype=torch.uint8, device="cuda")
    # second problem has K % 16 != 0
    xbad = torch.zeros((256, 24), dtype=torch.bfloat16, device="cuda")
    wbad = torch.zeros((128, 24), dtype=torch.int8, device="cuda")
    with pytest.raises(RuntimeError):
        P.sasq_static_w8a8_linear_multi([(x, w, wsc, sc, y), (xbad, wbad, wsc, sc, y)], ws)
    torch.cuda.synchronize()
    assert bool((y == 7.0).all())                  # the first problem was not launched either
    with pytest.raises(RuntimeError):              # workspace too small
        P.sasq_static_w8a8_linear_multi([(x, w, wsc, sc, y), (x, w, wsc, sc, y)], ws[:1024])
