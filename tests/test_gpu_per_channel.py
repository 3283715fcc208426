"""GPU parity of the per-channel fake-quant operator (one factor per column of x[T, K], the granularity of the
paper's experiments) against the CPU oracle, through the C ABI.  y and dx bit-exact; every channel's factor
gradient within 1e-4 relative of the oracle's double sum (with the rounding floor of the fp32 products where a
column's sum cancels), bit-identical from run to run."""
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


def make(T, K, tag, seed, bits=8, negative=False):
    x = W.activations(T, K, DT[tag], seed)
    g = W.upstream_grad(T, K, DT[tag], seed)
    xb, gb = oracle.bits_of(x)[0], oracle.bits_of(g)[0]
    # a "learned" factor per channel: the channel's own max over the first rows, shrunk so that clipping occurs
    qp = 2 ** (bits - 1) - 1
    amax = np.abs(oracle.widen(xb[:max(1, min(T, 64))], tag)).max(axis=0)
    rng = np.random.default_rng(seed)
    s = (np.maximum(amax, 1e-3) / qp * rng.uniform(0.3, 1.0, K)).astype(np.float32)
    if negative:
        s[::3] *= -1.0
    return xb, gb, s


def run(xb, gb, tag, s, bits, fwd=True, bwd=True, accumulate=False, grads_init=0.0):
    x, g = oracle.tensor_of(xb, tag).cuda(), oracle.tensor_of(gb, tag).cuda()
    T, K = x.shape
    sc = torch.from_numpy(s).cuda()
    y = torch.empty_like(x) if fwd else None
    dx = torch.empty_like(x) if bwd else None
    grads = torch.full((K,), grads_init, device="cuda") if bwd else None
    ws = torch.empty(max(16, P.sasq_fakequant_per_channel_workspace(T, K)), dtype=torch.uint8, device="cuda")
    P.sasq_fakequant_fwd_bwd_per_channel(x, g if bwd else None, y, dx, grads, sc, ws, bits, accumulate=accumulate)
    assert P.sasq_device_status() == 0
    return (None if y is None else host_bits(y), None if dx is None else host_bits(dx),
            None if grads is None else grads.cpu().numpy())


def check_ds(got, want, gb, tag, bits):
    floor = 4 * 2.0 ** -24 * np.abs(oracle.widen(gb, tag)).sum(axis=0) * 2 ** (bits - 1)
    assert np.all(np.abs(got.astype(np.float64) - want) <= 1e-4 * np.abs(want) + floor + 1e-30)


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("T,K", [(1, 8), (7, 16), (33, 520), (300, 4096), (64, 11008), (1000, 2056)])
def test_parity_shapes(tag, T, K):
    xb, gb, s = make(T, K, tag, 9000 + T + K)
    y_o, _ = oracle.fakequant_fwd_per_channel(xb, tag, s, 8)
    dx_o, ds_o = oracle.fakequant_bwd_per_channel(xb, gb, tag, s, 8)
    y, dx, ds = run(xb, gb, tag, s, 8)
    assert np.array_equal(y, y_o) and np.array_equal(dx, dx_o)
    check_ds(ds, ds_o, gb, tag, 8)
    assert (dx_o == 0).sum() > 0 or T * K < 100


@pytest.mark.parametrize("bits", [4, 2])
def test_low_bit_widths_and_negative_factors(bits):
    tag, T, K = oracle.BF16, 257, 1032
    xb, gb, s = make(T, K, tag, 9100 + bits, bits=bits, negative=True)
    y_o, _ = oracle.fakequant_fwd_per_channel(xb, tag, s, bits)
    dx_o, ds_o = oracle.fakequant_bwd_per_channel(xb, gb, tag, s, bits)
    y, dx, ds = run(xb, gb, tag, s, bits)
    assert np.array_equal(y, y_o) and np.array_equal(dx, dx_o)
    check_ds(ds, ds_o, gb, tag, bits)


def test_forward_only_backward_only_and_accumulate():
    tag, T, K = oracle.F16, 130, 264
    xb, gb, s = make(T, K, tag, 9200)
    y_o, _ = oracle.fakequant_fwd_per_channel(xb, tag, s, 8)
    dx_o, ds_o = oracle.fakequant_bwd_per_channel(xb, gb, tag, s, 8)
    y, _, _ = run(xb, gb, tag, s, 8, bwd=False)
    assert np.array_equal(y, y_o)
    _, dx, ds = run(xb, gb, tag, s, 8, fwd=False)
    assert np.array_equal(dx, dx_o)
    check_ds(ds, ds_o, gb, tag, 8)
    _, _, ds2 = run(xb, gb, tag, s, 8, accumulate=True, grads_init=10.0)
    assert np.array_equal(ds2, (np.float32(10.0) + ds).astype(np.float32))


def test_full_size_llama_tensor_is_deterministic():
    """down_proj input of the benchmark layer (T=2048, K=11008): every element, every channel, twice."""
    tag, T, K = oracle.BF16, 2048, 11008
    xb, gb, s = make(T, K, tag, W.seed_of(2, 6))
    y_o, _ = oracle.fakequant_fwd_per_channel(xb, tag, s, 8)
    dx_o, ds_o = oracle.fakequant_bwd_per_channel(xb, gb, tag, s, 8)
    y, dx, ds = run(xb, gb, tag, s, 8)
    assert np.array_equal(y, y_o) and np.array_equal(dx, dx_o)
    check_ds(ds, ds_o, gb, tag, 8)
    _, _, ds_again = run(xb, gb, tag, s, 8)
    assert np.array_equal(ds.view(np.uint32), ds_again.view(np.uint32))


def test_errors_and_edge_cases():
    x = torch.zeros((4, 12), dtype=torch.bfloat16, device="cuda")
    sc = torch.ones(12, device="cuda")
    ws = torch.empty(P.sasq_fakequant_per_channel_workspace(4, 16), dtype=torch.uint8, device="cuda")
    with pytest.raises(P.SasqError) as e:
        P.sasq_fakequant_fwd_bwd_per_channel(x, None, torch.empty_like(x), None, None, sc, ws, 8)    # K % 8 != 0
    assert e.value.status == 2
    x = torch.zeros((4, 16), dtype=torch.bfloat16, device="cuda")
    sc = torch.ones(16, device="cuda")
    with pytest.raises(P.SasqError) as e:
        P.sasq_fakequant_fwd_bwd_per_channel(x, x, None, torch.empty_like(x), torch.zeros(16, device="cuda"), sc,
                                             None, 8)                                                  # no workspace
    assert e.value.status == 3
    sc[5] = 0.0
    P.sasq_fakequant_fwd_bwd_per_channel(x, None, torch.empty_like(x), None, None, sc, ws, 8)
    assert P.sasq_device_status() == 4
    assert P.sasq_device_status() == 0
    # no rows: gradients are zeroed, nothing is launched
    e0 = torch.empty((0, 16), dtype=torch.bfloat16, device="cuda")
    grads = torch.full((16,), 7.0, device="cuda")
    sc.fill_(1.0)
    P.sasq_fakequant_fwd_bwd_per_channel(e0, e0, e0, e0, grads, sc, ws, 8)
    assert float(grads.abs().sum()) == 0.0


def test_multi_tensor_launch_matches_the_oracle_per_tensor():
    """The seven linear inputs of a (scaled-down) decoder layer in one launch, plus an empty tensor."""
    tag, bits = oracle.BF16, 8
    shapes = [(67, 512)] * 3 + [(67, 1376), (5, 264), (0, 16), (300, 2056)]
    cases = [make(max(T, 1), K, tag, 9300 + i) for i, (T, K) in enumerate(shapes)]
    tensors, keep = [], []
    total_k = sum(K for _, K in shapes)
    for (T, K), (xb, gb, s) in zip(shapes, cases):
        xb, gb = xb[:T], gb[:T]
        x = oracle.tensor_of(xb, tag).cuda().reshape(T, K)
        g = oracle.tensor_of(gb, tag).cuda().reshape(T, K)
        y, dx = torch.empty_like(x), torch.empty_like(x)
        sc, gs = torch.from_numpy(s).cuda(), torch.full((K,), 3.0, device="cuda")
        tensors.append((x, g, y, dx, sc, gs))
        keep.append((xb, gb, s))
    ws = torch.empty(P.sasq_fakequant_per_channel_multi_workspace(total_k), dtype=torch.uint8, device="cuda")
    P.sasq_fakequant_fwd_bwd_per_channel_multi(tensors, ws, bits)
    assert P.sasq_device_status() == 0
    for (T, K), (x, g, y, dx, sc, gs), (xb, gb, s) in zip(shapes, tensors, keep):
        if T == 0:
            assert float(gs.abs().sum()) == 0.0
            continue
        y_o, _ = oracle.fakequant_fwd_per_channel(xb, tag, s, bits)
        dx_o, ds_o = oracle.fakequant_bwd_per_channel(xb, gb, tag, s, bits)
        assert np.array_equal(host_bits(y), y_o) and np.array_equal(host_bits(dx), dx_o)
        check_ds(gs.cpu().numpy(), ds_o, gb, tag, bits)
