"""Seeded random shapes through the static W8A8 linear, alone and in random groups through the multi entry, every
output bit-exact against the CPU oracle.  The draws cover what the planners branch on: T on both sides of 32, 128
and 256, widths that are not multiples of 16, 64 or 128 columns, K down to one 16-element group."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu


def draw_shapes(seed, count):
    rng = np.random.default_rng(seed)
    t_choices = [1, 2, 15, 16, 17, 31, 32, 33, 64, 127, 128, 129, 200, 255, 256, 257, 300, 511, 513, 600]
    shapes = []
    for _ in range(count):
        T = int(rng.choice(t_choices))
        N = int(rng.integers(1, 150)) * 8
        K = int(rng.integers(1, 70)) * 16
        shapes.append((T, N, K))
    return shapes


def make(T, N, K, seed):
    tag = oracle.BF16
    xb = oracle.bits_of(W.activations(T, K, torch.bfloat16, seed))[0]
    w_int, w_scale = oracle.quantize_weight(W.weights_fp32(N, K, seed + 1).numpy(), 8)
    s = float(oracle.absmax_scale(xb[:min(T, 64)], tag, 8)) * 0.55
    y_o, _, _ = oracle.w8a8_linear(xb, tag, w_int, w_scale, s, 8)
    dev = (oracle.tensor_of(xb, tag).cuda(), torch.from_numpy(w_int).cuda(), torch.from_numpy(w_scale).cuda(),
           torch.tensor([s], dtype=torch.float32, device="cuda"),
           torch.full((T, N), 7.0, dtype=torch.bfloat16, device="cuda"))
    return dev, y_o


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_shapes_alone_and_in_random_groups(seed):
    shapes = draw_shapes(seed, 14)
    cases = [make(T, N, K, 12000 + 100 * seed + i) for i, (T, N, K) in enumerate(shapes)]
    # alone
    for (dev, y_o), (T, N, K) in zip(cases, shapes):
        ws = torch.empty(max(16, P.sasq_static_w8a8_linear_workspace(T, N, K)), dtype=torch.uint8, device="cuda")
        P.sasq_static_w8a8_linear(*dev, workspace=ws)
        assert P.sasq_device_status() == 0
        assert np.array_equal(oracle.bits_of(dev[4].cpu())[0], y_o), (T, N, K)
        dev[4].fill_(7.0)
    # all of them in one call (the entry cuts the list into launches), then in a shuffled order
    rng = np.random.default_rng(seed + 50)
    for order in (list(range(len(cases))), list(rng.permutation(len(cases)))):
        problems = [cases[i][0] for i in order]
        need = P.sasq_static_w8a8_linear_multi_workspace([shapes[i] for i in order])
        ws = torch.empty(max(16, need), dtype=torch.uint8, device="cuda")
        P.sasq_static_w8a8_linear_multi(problems, ws)
        assert P.sasq_device_status() == 0
        for i in order:
            assert np.array_equal(oracle.bits_of(cases[i][0][4].cpu())[0], cases[i][1]), shapes[i]
            cases[i][0][4].fill_(7.0)
