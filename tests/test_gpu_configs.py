"""GPU parity at the full sizes of the five benchmark configurations, through the C ABI, in the launch shapes
the benchmark uses.  Where the CPU oracle cannot afford every output (the integer GEMM at thousands of tokens) it
checks whole sampled rows (first / last rows, rows around the 128- and 256-row tile edges, seeded random rows),
bit for bit; rows are independent of one another, so the oracle runs on the gathered rows alone.  The quantizer
outputs are cheap for the oracle and are checked in full on sampled tensors; every scale gradient is checked.

Bars as everywhere: codes / accumulators / y / dx bit-exact, scale gradient within 1e-4 relative.
Inputs are generated on the device (seeded) and copied to the host, so both sides consume the same bytes.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu
DS_RTOL = 1e-4


def host_bits(t):
    return oracle.bits_of(t.cpu())[0]


def sample_rows(T, seed, n_random=6):
    fixed = [0, 1, 127, 128, 129, 255, 256, 257, T // 2, T - 2, T - 1]
    g = torch.Generator().manual_seed(seed)
    rnd = torch.randint(0, T, (n_random,), generator=g).tolist()
    return sorted({r for r in fixed + rnd if 0 <= r < T})


def device_weights(N, K, seed):
    w = W.weights_fp32(N, K, seed, device="cuda")
    w_int = torch.empty((N, K), dtype=torch.int8, device="cuda")
    w_scale = torch.empty(N, dtype=torch.float32, device="cuda")
    P.sasq_quantize_weight(w, w_int, w_scale, 8)
    return w_int, w_scale


def check_linear_rows(x, w_int, w_scale, s, rows, bits=8, with_acc=True):
    """Runs the library on the full problem, the oracle on the gathered rows, and compares those rows."""
    T, K = x.shape
    N = w_int.shape[0]
    sc = torch.tensor([s], dtype=torch.float32, device="cuda")
    y = torch.empty((T, N), dtype=x.dtype, device="cuda")
    acc = torch.empty((T, N), dtype=torch.int32, device="cuda") if with_acc else None
    ws = torch.empty(max(16, P.sasq_static_w8a8_linear_workspace(T, N, K)), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear(x, w_int, w_scale, sc, y, acc_out=acc, workspace=ws, bits=bits)
    assert P.sasq_device_status() == 0
    idx = torch.tensor(rows, device="cuda")
    xb, tag = oracle.bits_of(x[idx].cpu())
    y_o, _, acc_o = oracle.w8a8_linear(xb, tag, w_int.cpu().numpy(), w_scale.cpu().numpy(), s, bits)
    if with_acc:
        assert np.array_equal(acc[idx].cpu().numpy(), acc_o)
    assert np.array_equal(host_bits(y[idx]), y_o)
    return y


# ---------------------------------------------------------------------------
# config 3: static W8A8 inference of the seven LLaMA-2-7B linears, decode through prefill
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("T", [1, 16, 128, 2048, 8192])
def test_config3_llama7b_linears_decode_through_prefill(T):
    tag = oracle.BF16
    for li, (name, K, N) in enumerate(W.LLAMA2_7B_LINEARS):
        if name in ("k_proj", "v_proj", "o_proj", "up_proj"):
            continue                      # same shapes as q_proj / gate_proj
        x = W.activations(T, K, torch.bfloat16, W.seed_of(3, li), device="cuda")
        w_int, w_scale = device_weights(N, K, W.seed_of(3, 10 + li))
        calib = oracle.bits_of(x[:min(T, W.CALIBRATION_TOKENS)].cpu())[0]
        s = float(oracle.absmax_scale(calib, tag, 8)) * W.learned_scale_factor(W.seed_of(3, li))
        rows = list(range(T)) if T <= 16 else sample_rows(T, 300 + li)
        check_linear_rows(x, w_int, w_scale, s, rows, with_acc=True)     # int32 accumulators at every size


# ---------------------------------------------------------------------------
# config 4: LLaMA-2-13B-shaped layer, T = 4096, heavy-tailed activations, 8 and 4 bits,
#           one factor per tensor and one factor per layer
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [8, 4])
def test_config4_llama13b_heavy_tailed_per_tensor_and_per_layer(bits):
    tag, T = oracle.BF16, 4096
    xs, gs = [], []
    for i, (_, K, _) in enumerate(W.LLAMA2_13B_LINEARS):
        xs.append(W.activations(T, K, torch.bfloat16, W.seed_of(4, i), W.HEAVY_TAILED, device="cuda"))
        gs.append(W.upstream_grad(T, K, torch.bfloat16, W.seed_of(4, i), device="cuda"))
    ys, dxs = [torch.empty_like(t) for t in xs], [torch.empty_like(t) for t in xs]
    xb = [host_bits(t) for t in xs]
    gb = [host_bits(t) for t in gs]
    scal = [float(oracle.absmax_scale(b[:W.CALIBRATION_TOKENS], tag, bits)) for b in xb]
    ws = torch.empty(P.sasq_fakequant_multi_workspace(7), dtype=torch.uint8, device="cuda")
    full = (1, 6)          # tensors whose y and dx are compared element by element: one K = 5120, the K = 13824 one

    # one factor per tensor
    scales = torch.tensor(scal, dtype=torch.float32, device="cuda")
    grads = torch.zeros(7, device="cuda")
    P.sasq_fakequant_fwd_bwd_multi([(xs[i], gs[i], ys[i], dxs[i], i) for i in range(7)], scales, grads, ws, bits)
    assert P.sasq_device_status() == 0
    clipped = 0
    for i in range(7):
        dx_o, ds_o = oracle.fakequant_bwd(xb[i], gb[i], tag, scal[i], bits)
        assert abs(grads[i].item() - ds_o) <= DS_RTOL * abs(ds_o), (i, grads[i].item(), ds_o)
        if i in full:
            y_o, _ = oracle.fakequant_fwd(xb[i], tag, scal[i], bits)
            assert np.array_equal(host_bits(ys[i]), y_o) and np.array_equal(host_bits(dxs[i]), dx_o)
            clipped += int((dx_o == 0).sum())
    assert clipped > 0            # the heavy tails do reach the clamp

    # one factor for the whole layer (all seven quantizers share it; ds is the sum over all seven tensors)
    s_layer = float(np.float32(np.mean(scal)))
    scales1 = torch.tensor([s_layer], dtype=torch.float32, device="cuda")
    grads1 = torch.zeros(1, device="cuda")
    P.sasq_fakequant_fwd_bwd_multi([(xs[i], gs[i], ys[i], dxs[i], 0) for i in range(7)], scales1, grads1, ws, bits)
    assert P.sasq_device_status() == 0
    total = 0.0
    for i in range(7):
        dx_o, ds_o = oracle.fakequant_bwd(xb[i], gb[i], tag, s_layer, bits)
        total += ds_o
        if i in full:
            y_o, _ = oracle.fakequant_fwd(xb[i], tag, s_layer, bits)
            assert np.array_equal(host_bits(ys[i]), y_o) and np.array_equal(host_bits(dxs[i]), dx_o)
    assert abs(grads1.item() - total) <= DS_RTOL * abs(total)


# ---------------------------------------------------------------------------
# config 5: 32 layers x 7 quantizers over 8 x 2048 tokens: one scale-only training step, then the static
#           W8A8 prefill of all 224 linears; activation buffers are reused layer by layer
# ---------------------------------------------------------------------------
def test_config5_full_stack_scale_only_step_then_static_prefill():
    tag, T, bits, layers = oracle.BF16, 8 * 2048, 8, 32
    checked_layers = {0: (0, 6), 13: (4,), 31: (6, 3)}      # layer -> tensors compared element by element
    shapes = [(K, N) for _, K, N in W.LLAMA2_7B_LINEARS]
    xs = [torch.empty((T, K), dtype=torch.bfloat16, device="cuda") for K, _ in shapes]
    gs = [torch.empty_like(t) for t in xs]
    ys, dxs = [torch.empty_like(t) for t in xs], [torch.empty_like(t) for t in xs]
    outs = {N: torch.empty((T, N), dtype=torch.bfloat16, device="cuda") for _, N in shapes}
    scales = torch.empty(layers * 7, dtype=torch.float32, device="cuda")
    grads = torch.full((layers * 7,), 3.0, device="cuda")
    q_ws = torch.empty(P.sasq_fakequant_multi_workspace(7), dtype=torch.uint8, device="cuda")
    cal_ws = torch.empty(P.sasq_absmax_scale_workspace(0), dtype=torch.uint8, device="cuda")
    l_ws = torch.empty(max(P.sasq_static_w8a8_linear_workspace(T, N, K) for K, N in shapes), dtype=torch.uint8,
                       device="cuda")
    ds_checked = 0
    for layer in range(layers):
        for i, (K, N) in enumerate(shapes):
            seed = W.seed_of(5, layer * 7 + i)
            xs[i].copy_(W.activations(T, K, torch.bfloat16, seed, device="cuda"))
            gs[i].copy_(W.upstream_grad(T, K, torch.bfloat16, seed, device="cuda"))
            q = layer * 7 + i
            P.sasq_absmax_scale(xs[i][:W.CALIBRATION_TOKENS], scales[q:q + 1], cal_ws, bits)   # Eq. 1, set-up
        # the scale-only training step of this layer: seven quantizers, one launch, seven slots of the 224
        P.sasq_fakequant_fwd_bwd_multi([(xs[i], gs[i], ys[i], dxs[i], layer * 7 + i) for i in range(7)], scales, grads,
                                       q_ws, bits)
        # properties that hold for every element, checked on the device for every layer:
        # dx is the upstream gradient or zero; y takes at most 2^b distinct values per tensor (zero with either sign)
        for i in (0, 6):
            d, g = dxs[i].view(torch.int16), gs[i].view(torch.int16)
            assert bool(((d == g) | (d == 0)).all())
            assert torch.unique(ys[i].view(torch.int16)).numel() <= 256 + 1
        # static prefill of the seven linears of this layer with frozen random-init int8 weights
        rows = sample_rows(T, 500 + layer, n_random=3)
        idx = torch.tensor(rows, device="cuda")
        for i, (K, N) in enumerate(shapes):
            w_int, w_scale = device_weights(N, K, W.seed_of(5, 1000 + layer * 7 + i))
            q = layer * 7 + i
            P.sasq_static_w8a8_linear(xs[i], w_int, w_scale, scales[q:q + 1], outs[N], workspace=l_ws, bits=bits)
            if layer in checked_layers and i in checked_layers[layer]:
                s = float(scales[q].item())
                xb_rows = oracle.bits_of(xs[i][idx].cpu())[0]
                y_o, _, _ = oracle.w8a8_linear(xb_rows, tag, w_int.cpu().numpy(), w_scale.cpu().numpy(), s, bits)
                assert np.array_equal(host_bits(outs[N][idx]), y_o), (layer, i)
        assert P.sasq_device_status() == 0
        if layer in checked_layers:
            for i in range(7):
                q = layer * 7 + i
                s = float(scales[q].item())
                xb, gb = host_bits(xs[i]), host_bits(gs[i])
                assert np.float32(s) == oracle.absmax_scale(xb[:W.CALIBRATION_TOKENS], tag, bits)
                dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, s, bits)
                assert abs(grads[q].item() - ds_o) <= DS_RTOL * abs(ds_o), (layer, i)
                ds_checked += 1
                if i in checked_layers[layer]:
                    y_o, _ = oracle.fakequant_fwd(xb, tag, s, bits)
                    assert np.array_equal(host_bits(ys[i]), y_o) and np.array_equal(host_bits(dxs[i]), dx_o)
    assert ds_checked == 21
    assert bool((grads != 3.0).all())          # every one of the 224 slots was written


def test_config5_one_layer_in_the_launch_configuration_the_benchmark_times():
    """One layer of config 5 (T = 16 384) submitted exactly as the benchmark's step submits it: the fused fake-quant
    forward + backward of the seven inputs as ONE prepared multi-tensor call, then the seven static linears in the
    groups a decoder layer's data flow allows (q/k/v | o | gate/up | down) as prepared multi-linear calls, plain
    (not co-operative) launches, raw stream handle.  Every scale gradient against the oracle's double sum, two
    tensors element by element, sampled rows of every linear bit for bit."""
    tag, T, bits = oracle.BF16, 8 * 2048, 8
    shapes = [(K, N) for _, K, N in W.LLAMA2_7B_LINEARS]
    xs = [W.activations(T, K, torch.bfloat16, W.seed_of(5, 500 + i), device="cuda") for i, (K, _) in enumerate(shapes)]
    gs = [W.upstream_grad(T, K, torch.bfloat16, W.seed_of(5, 500 + i), device="cuda") for i, (K, _) in enumerate(shapes)]
    ys, dxs = [torch.empty_like(t) for t in xs], [torch.empty_like(t) for t in xs]
    outs = [torch.empty((T, N), dtype=torch.bfloat16, device="cuda") for _, N in shapes]
    weights = [device_weights(N, K, W.seed_of(5, 600 + i)) for i, (K, N) in enumerate(shapes)]
    scales = torch.empty(7, dtype=torch.float32, device="cuda")
    grads = torch.zeros(7, dtype=torch.float32, device="cuda")
    cal_ws = torch.empty(P.sasq_absmax_scale_workspace(0), dtype=torch.uint8, device="cuda")
    for i in range(7):
        P.sasq_absmax_scale(xs[i][:W.CALIBRATION_TOKENS], scales[i:i + 1], cal_ws, bits)
    q_ws = torch.empty(P.sasq_fakequant_multi_workspace(7), dtype=torch.uint8, device="cuda")
    l_ws = torch.empty(P.sasq_static_w8a8_linear_multi_workspace([(T, N, K) for K, N in shapes]), dtype=torch.uint8,
                       device="cuda")
    quant = P.QuantTensors([(xs[i], gs[i], ys[i], dxs[i], i) for i in range(7)])
    calls = [P.LinearProblems([(xs[i], weights[i][0], weights[i][1], scales[i:i + 1], outs[i]) for i in call])
             for call in ([0, 1, 2], [3], [4, 5], [6])]
    handle = torch.cuda.current_stream().cuda_stream
    previous = P.sasq_set_gang_launch(False)
    try:
        for _ in range(2):                                  # twice: the second pass finds the counters as the first left them
            P.sasq_fakequant_fwd_bwd_multi(quant, scales, grads, q_ws, bits, stream=handle)
            for problems in calls:
                P.sasq_static_w8a8_linear_multi(problems, l_ws, bits=bits, stream=handle)
        assert P.sasq_device_status() == 0
    finally:
        P.sasq_set_gang_launch(previous)
    s_host = scales.cpu().numpy()
    for i, (K, N) in enumerate(shapes):
        s = float(s_host[i])
        xb, gb = host_bits(xs[i]), host_bits(gs[i])
        dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, s, bits)
        assert abs(grads[i].item() - ds_o) <= DS_RTOL * abs(ds_o), i
        if i in (1, 6):
            y_o, _ = oracle.fakequant_fwd(xb, tag, s, bits, want_codes=False)
            assert np.array_equal(host_bits(ys[i]), y_o) and np.array_equal(host_bits(dxs[i]), dx_o), i
        rows = sample_rows(T, 700 + i, n_random=3)
        idx = torch.tensor(rows, device="cuda")
        y_lin, _, _ = oracle.w8a8_linear(oracle.bits_of(xs[i][idx].cpu())[0], tag, weights[i][0].cpu().numpy(),
                                         weights[i][1].cpu().numpy(), s, bits)
        assert np.array_equal(host_bits(outs[i][idx]), y_lin), i
