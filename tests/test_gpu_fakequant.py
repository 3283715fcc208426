"""GPU parity: the CUDA fake-quant path (through the C ABI) against the CPU oracle,
element by element on the same seeded bytes.

Bars: y and dx bit-exact (16-bit patterns); the reduced scale gradient within
1e-4 relative of the oracle's double-precision sum and bit-identical from run to
run.  The tolerance on ds is the stated bar of the library; the arithmetic
(fp32 products, fp32 trees of 8, double accumulation) keeps the error near
1e-7 * sum|g * term|.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu

DT = {oracle.F16: torch.float16, oracle.BF16: torch.bfloat16}
DS_RTOL = 1e-4


def dev(bits_arr, tag):
    return oracle.tensor_of(bits_arr, tag).cuda()


def host_bits(t):
    return oracle.bits_of(t.cpu())[0]


def ds_close(got, want, sum_abs=None):
    tol = DS_RTOL * abs(want)
    if sum_abs is not None:
        tol += 4 * 2.0 ** -24 * sum_abs     # floor for sums that cancel to ~0
    return abs(float(got) - want) <= tol + 1e-30


def rand_bits(n, tag, seed, scale=3.0, outliers=True):
    g = torch.Generator().manual_seed(seed)
    v = torch.randn(n, generator=g) * scale
    if outliers and n >= 50:
        idx = torch.randint(0, n, (n // 50,), generator=g)
        v[idx] *= 40.0
    return oracle.bits_of(v.to(DT[tag]))[0]


def run_all(xb, gb, tag, s, bits):
    """Returns dict of GPU results from the separate and the fused entry points."""
    x, g = dev(xb, tag), dev(gb, tag)
    sc = torch.tensor([s], dtype=torch.float32, device="cuda")
    ws = torch.empty(P.sasq_fakequant_bwd_workspace(x.numel()), dtype=torch.uint8, device="cuda")
    y = torch.empty_like(x); dx = torch.empty_like(x); ds = torch.full((1,), 7.0, device="cuda")
    P.sasq_fakequant_fwd(x, y, sc, bits)
    P.sasq_fakequant_bwd(x, g, dx, ds, sc, ws, bits)
    y2 = torch.empty_like(x); dx2 = torch.empty_like(x); ds2 = torch.full((1,), -3.0, device="cuda")
    P.sasq_fakequant_fwd_bwd(x, g, y2, dx2, ds2, sc, ws, bits)
    assert P.sasq_device_status() == 0
    return dict(y=host_bits(y), dx=host_bits(dx), ds=ds.item(), y2=host_bits(y2), dx2=host_bits(dx2), ds2=ds2.item())


SIZES = [1, 7, 8, 9, 255, 2048, 65536 + 3, 1_000_003]


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("n", SIZES)
def test_parity_sizes_with_ragged_tails(tag, n):
    s, bits = 0.0371, 8
    xb, gb = rand_bits(n, tag, 100 + n), rand_bits(n, tag, 200 + n, scale=1.0, outliers=False)
    y_o, _ = oracle.fakequant_fwd(xb, tag, s, bits)
    dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, s, bits)
    r = run_all(xb, gb, tag, s, bits)
    assert np.array_equal(r["y"], y_o) and np.array_equal(r["y2"], y_o)
    assert np.array_equal(r["dx"], dx_o) and np.array_equal(r["dx2"], dx_o)
    sum_abs = float(np.abs(oracle.widen(gb, tag)).sum()) * 128
    assert ds_close(r["ds"], ds_o, sum_abs) and ds_close(r["ds2"], ds_o, sum_abs)
    assert r["ds"] == r["ds2"]                     # the fused pass reduces in the same order


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("bits,s", [(8, -0.05), (4, 0.4), (4, -0.7), (2, 1.3), (3, 0.9), (8, 1.0 / 3.0)])
def test_parity_bit_widths_and_negative_scales(tag, bits, s):
    n = 300_007
    xb, gb = rand_bits(n, tag, 31), rand_bits(n, tag, 32, scale=1.0, outliers=False)
    y_o, _ = oracle.fakequant_fwd(xb, tag, s, bits)
    dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, s, bits)
    r = run_all(xb, gb, tag, s, bits)
    assert np.array_equal(r["y2"], y_o) and np.array_equal(r["dx2"], dx_o)
    assert np.array_equal(r["y"], y_o) and np.array_equal(r["dx"], dx_o)
    assert ds_close(r["ds2"], ds_o) and ds_close(r["ds"], ds_o)


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
def test_degenerate_all_clipped_and_none_clipped(tag):
    n = 50_001
    gb = rand_bits(n, tag, 5, scale=1.0, outliers=False)
    big = oracle.bits_of(torch.where(torch.arange(n) % 3 == 0, 900.0, -900.0).to(DT[tag]))[0]
    r = run_all(big, gb, tag, 0.5, 8)
    dx_o, ds_o = oracle.fakequant_bwd(big, gb, tag, 0.5, 8)
    assert not r["dx2"].any() and np.array_equal(r["dx2"], dx_o)
    assert ds_close(r["ds2"], ds_o)
    small = oracle.bits_of((torch.linspace(-1, 1, n)).to(DT[tag]))[0]
    r = run_all(small, gb, tag, 1.0, 8)
    y_o, _ = oracle.fakequant_fwd(small, tag, 1.0, 8)
    dx_o, ds_o = oracle.fakequant_bwd(small, gb, tag, 1.0, 8)
    assert np.array_equal(r["dx2"], gb) and np.array_equal(r["y2"], y_o)
    assert ds_close(r["ds2"], ds_o, float(np.abs(oracle.widen(gb, tag)).sum()))


def test_special_values_follow_the_header():
    """+-Inf saturates with m = 0; NaN gives code -Qn with m = 0; +-0 and subnormals pass through."""
    tag = oracle.F16
    vals = torch.tensor([float("inf"), float("-inf"), float("nan"), 0.0, -0.0, 6e-8, -6e-8, 65504.0, -65504.0, 0.26],
                        dtype=torch.float16)
    xb = oracle.bits_of(vals)[0]
    gb = oracle.bits_of(torch.ones(10, dtype=torch.float16))[0]
    r = run_all(xb, gb, tag, 0.5, 8)
    y_o, codes = oracle.fakequant_fwd(xb, tag, 0.5, 8)
    dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, 0.5, 8)
    assert codes[:3].tolist() == [127, -128, -128]
    assert np.array_equal(r["y2"], y_o) and np.array_equal(r["dx2"], dx_o)
    assert ds_close(r["ds2"], ds_o)


def test_config1_single_linear_input_full_check():
    """T=128, K=4096 fp16, N(0,1) with 1% of channels x50, s = max|x[0:64]|/127 (Eq. 1), upstream grad N(0,1)."""
    T, K = 128, 4096
    x = W.activations(T, K, torch.float16, W.seed_of(1, 0))
    g = W.upstream_grad(T, K, torch.float16, W.seed_of(1, 0))
    xb, tag = oracle.bits_of(x)
    gb, _ = oracle.bits_of(g)
    s = float(oracle.absmax_scale(xb[:W.CALIBRATION_TOKENS], tag, 8))
    y_o, _ = oracle.fakequant_fwd(xb, tag, s, 8)
    dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, s, 8)
    r = run_all(xb.reshape(-1), gb.reshape(-1), tag, s, 8)
    assert np.array_equal(r["y2"], y_o.reshape(-1)) and np.array_equal(r["dx2"], dx_o.reshape(-1))
    assert np.array_equal(r["y"], y_o.reshape(-1)) and np.array_equal(r["dx"], dx_o.reshape(-1))
    assert ds_close(r["ds2"], ds_o) and ds_close(r["ds"], ds_o)
    assert (dx_o == 0).sum() > 0      # the calibration slice does not cover every outlier: some clipping


def test_scale_gradient_is_bit_identical_run_to_run_and_accumulates():
    tag, n, s = oracle.BF16, 3_000_001, 0.02
    x, g = dev(rand_bits(n, tag, 77), tag), dev(rand_bits(n, tag, 78, scale=1.0, outliers=False), tag)
    sc = torch.tensor([s], dtype=torch.float32, device="cuda")
    ws = torch.empty(P.sasq_fakequant_bwd_workspace(n), dtype=torch.uint8, device="cuda")
    y, dx = torch.empty_like(x), torch.empty_like(x)
    outs = []
    for i in range(5):
        ds = torch.zeros(1, device="cuda")
        ws.fill_(i * 37 % 251)                       # workspace contents must not matter
        P.sasq_fakequant_fwd_bwd(x, g, y, dx, ds, sc, ws, 8)
        outs.append(ds.cpu().numpy().view(np.uint32)[0])
    assert len(set(outs)) == 1
    base = torch.tensor([1000.0], device="cuda")
    P.sasq_fakequant_fwd_bwd(x, g, y, dx, base, sc, ws, 8, accumulate=True)
    one = np.array([outs[0]], np.uint32).view(np.float32)[0]
    assert base.item() == float(np.float32(1000.0) + one)


def test_in_place_aliasing_is_allowed():
    tag, n, s = oracle.BF16, 100_003, 0.03
    xb, gb = rand_bits(n, tag, 91), rand_bits(n, tag, 92, scale=1.0, outliers=False)
    y_o, _ = oracle.fakequant_fwd(xb, tag, s, 8)
    dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, s, 8)
    x, g = dev(xb, tag), dev(gb, tag)
    sc = torch.tensor([s], dtype=torch.float32, device="cuda")
    ws = torch.empty(P.sasq_fakequant_bwd_workspace(n), dtype=torch.uint8, device="cuda")
    ds = torch.zeros(1, device="cuda")
    P.sasq_fakequant_fwd_bwd(x, g, x, g, ds, sc, ws, 8)       # y over x, grad_x over grad_y
    assert np.array_equal(host_bits(x), y_o) and np.array_equal(host_bits(g), dx_o)
    assert ds_close(ds.item(), ds_o)


def _layer_tensors(shapes, tag, seed0):
    xs, gs = [], []
    for i, (T, K) in enumerate(shapes):
        xs.append(oracle.bits_of(W.activations(T, K, DT[tag], seed0 + i))[0])
        gs.append(oracle.bits_of(W.upstream_grad(T, K, DT[tag], seed0 + i))[0])
    return xs, gs


@pytest.mark.parametrize("bits", [8, 4])
def test_multi_tensor_per_tensor_and_per_layer_scales(bits):
    """Seven linear inputs of a (scaled-down) decoder layer in one call: seven factors, then one shared factor."""
    tag = oracle.BF16
    shapes = [(33, 512)] * 6 + [(33, 1376 + 8)]
    xs, gs = _layer_tensors(shapes, tag, 4000)
    scal = [float(oracle.absmax_scale(x[:16], tag, bits)) * (0.5 + 0.07 * i) for i, x in enumerate(xs)]
    xd = [dev(x, tag) for x in xs]
    gd = [dev(g, tag) for g in gs]
    yd = [torch.empty_like(t) for t in xd]
    dxd = [torch.empty_like(t) for t in xd]
    ws = torch.empty(P.sasq_fakequant_multi_workspace(7), dtype=torch.uint8, device="cuda")
    # per-tensor
    scales = torch.tensor(scal, dtype=torch.float32, device="cuda")
    grads = torch.full((7,), 5.0, device="cuda")
    P.sasq_fakequant_fwd_bwd_multi([(xd[i], gd[i], yd[i], dxd[i], i) for i in range(7)], scales, grads, ws, bits)
    assert P.sasq_device_status() == 0
    for i in range(7):
        y_o, _ = oracle.fakequant_fwd(xs[i], tag, scal[i], bits)
        dx_o, ds_o = oracle.fakequant_bwd(xs[i], gs[i], tag, scal[i], bits)
        assert np.array_equal(host_bits(yd[i]), y_o) and np.array_equal(host_bits(dxd[i]), dx_o)
        assert ds_close(grads[i].item(), ds_o)
    # per-layer: one factor shared by the seven quantizers, ds = sum over all seven tensors
    s_layer = float(np.mean(scal))
    scales1 = torch.tensor([s_layer], dtype=torch.float32, device="cuda")
    grads1 = torch.zeros(1, device="cuda")
    P.sasq_fakequant_fwd_bwd_multi([(xd[i], gd[i], yd[i], dxd[i], 0) for i in range(7)], scales1, grads1, ws, bits)
    total = 0.0
    for i in range(7):
        y_o, _ = oracle.fakequant_fwd(xs[i], tag, s_layer, bits)
        dx_o, ds_o = oracle.fakequant_bwd(xs[i], gs[i], tag, s_layer, bits)
        total += ds_o
        assert np.array_equal(host_bits(yd[i]), y_o) and np.array_equal(host_bits(dxd[i]), dx_o)
    assert ds_close(grads1.item(), total)
    # mixed index map: q/k/v share, gate/up share
    idx = [0, 0, 0, 1, 2, 2, 3]
    sc4 = [0.05, 0.04, 0.03, 0.06]
    scales4 = torch.tensor(sc4, dtype=torch.float32, device="cuda")
    grads4 = torch.zeros(4, device="cuda")
    P.sasq_fakequant_fwd_bwd_multi([(xd[i], gd[i], yd[i], dxd[i], idx[i]) for i in range(7)], scales4, grads4, ws, bits)
    want = [0.0] * 4
    for i in range(7):
        want[idx[i]] += oracle.fakequant_bwd(xs[i], gs[i], tag, sc4[idx[i]], bits)[1]
    for k in range(4):
        assert ds_close(grads4[k].item(), want[k])


def test_multi_more_descriptors_than_one_launch_holds():
    tag, bits = oracle.F16, 8
    n_t = 70
    xs = [rand_bits(1000 + 13 * i, tag, 500 + i) for i in range(n_t)]
    gs = [rand_bits(1000 + 13 * i, tag, 900 + i, scale=1.0, outliers=False) for i in range(n_t)]
    idx = [i % 5 for i in range(n_t)]
    sc = [0.03, 0.05, 0.02, 0.07, 0.011]
    xd, gd = [dev(x, tag) for x in xs], [dev(g, tag) for g in gs]
    yd, dxd = [torch.empty_like(t) for t in xd], [torch.empty_like(t) for t in xd]
    ws = torch.empty(P.sasq_fakequant_multi_workspace(n_t), dtype=torch.uint8, device="cuda")
    scales = torch.tensor(sc, dtype=torch.float32, device="cuda")
    grads = torch.full((5,), 123.0, device="cuda")
    P.sasq_fakequant_fwd_bwd_multi([(xd[i], gd[i], yd[i], dxd[i], idx[i]) for i in range(n_t)], scales, grads, ws, bits)
    want = [0.0] * 5
    for i in range(n_t):
        y_o, _ = oracle.fakequant_fwd(xs[i], tag, sc[idx[i]], bits)
        dx_o, ds_o = oracle.fakequant_bwd(xs[i], gs[i], tag, sc[idx[i]], bits)
        want[idx[i]] += ds_o
        assert np.array_equal(host_bits(yd[i]), y_o) and np.array_equal(host_bits(dxd[i]), dx_o)
    for k in range(5):
        assert abs(grads[k].item() - want[k]) <= 2e-4 * abs(want[k]) + 1e-3   # three float adds across chunks


def test_multi_forward_only_and_backward_only():
    tag, bits, s = oracle.BF16, 8, 0.04
    xb, gb = rand_bits(77_777, tag, 1), rand_bits(77_777, tag, 2, scale=1.0, outliers=False)
    x, g = dev(xb, tag), dev(gb, tag)
    y, dx = torch.empty_like(x), torch.empty_like(x)
    scales = torch.tensor([s], dtype=torch.float32, device="cuda")
    P.sasq_fakequant_fwd_bwd_multi([(x, None, y, None, 0)], scales, None, None, bits)
    assert np.array_equal(host_bits(y), oracle.fakequant_fwd(xb, tag, s, bits)[0])
    ws = torch.empty(P.sasq_fakequant_multi_workspace(1), dtype=torch.uint8, device="cuda")
    grads = torch.zeros(1, device="cuda")
    P.sasq_fakequant_fwd_bwd_multi([(x, g, None, dx, 0)], scales, grads, ws, bits)
    dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, s, bits)
    assert np.array_equal(host_bits(dx), dx_o) and ds_close(grads.item(), ds_o)


def test_empty_tensor_is_ok_and_zeroes_the_gradient():
    x = torch.empty(0, dtype=torch.bfloat16, device="cuda")
    sc = torch.ones(1, device="cuda")
    ws = torch.empty(P.sasq_fakequant_bwd_workspace(0), dtype=torch.uint8, device="cuda")
    ds = torch.full((1,), 9.0, device="cuda")
    P.sasq_fakequant_fwd(x, x, sc, 8)
    P.sasq_fakequant_fwd_bwd(x, x, x, x, ds, sc, ws, 8)
    assert ds.item() == 0.0
    ds.fill_(9.0)
    P.sasq_fakequant_fwd_bwd(x, x, x, x, ds, sc, ws, 8, accumulate=True)
    assert ds.item() == 9.0


@pytest.mark.parametrize("bad", [0.0, float("nan"), float("inf"), 1e-45])
def test_bad_scale_sets_the_sticky_status(bad):
    x = torch.ones(1024, dtype=torch.bfloat16, device="cuda")
    y = torch.empty_like(x)
    sc = torch.tensor([bad], dtype=torch.float32, device="cuda")
    assert P.sasq_device_status() == 0
    P.sasq_fakequant_fwd(x, y, sc, 8)
    assert P.sasq_device_status() == 4      # SASQ_ERR_BAD_SCALE
    assert P.sasq_device_status() == 0      # cleared by the read


def test_llama7b_layer_shapes_full_size_launch_sampled_tensor():
    """The benchmark's launch configuration (seven tensors, T=2048, one call): every element of the
    down_proj input (K=11008) and of one K=4096 input is checked; ds of all seven."""
    tag, bits, T = oracle.BF16, 8, 2048
    xs, gs, sc = [], [], []
    for i, (_, K, _) in enumerate(W.LLAMA2_7B_LINEARS):
        xs.append(W.activations(T, K, torch.bfloat16, W.seed_of(2, i), device="cuda"))
        gs.append(W.upstream_grad(T, K, torch.bfloat16, W.seed_of(2, i), device="cuda"))
        xb = oracle.bits_of(xs[i][:W.CALIBRATION_TOKENS].cpu())[0]
        sc.append(float(oracle.absmax_scale(xb, tag, bits)))
    ys, dxs = [torch.empty_like(t) for t in xs], [torch.empty_like(t) for t in xs]
    scales = torch.tensor(sc, dtype=torch.float32, device="cuda")
    grads = torch.zeros(7, device="cuda")
    ws = torch.empty(P.sasq_fakequant_multi_workspace(7), dtype=torch.uint8, device="cuda")
    P.sasq_fakequant_fwd_bwd_multi([(xs[i], gs[i], ys[i], dxs[i], i) for i in range(7)], scales, grads, ws, bits)
    assert P.sasq_device_status() == 0
    for i in range(7):
        xb, gb = host_bits(xs[i]), host_bits(gs[i])
        dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, sc[i], bits)
        assert ds_close(grads[i].item(), ds_o), i
        if i in (2, 6):
            y_o, _ = oracle.fakequant_fwd(xb, tag, sc[i], bits)
            assert np.array_equal(host_bits(ys[i]), y_o) and np.array_equal(host_bits(dxs[i]), dx_o)
