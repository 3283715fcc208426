"""GPU parity of the PTQ-initialisation helpers (max-based factor, per-channel weight quantizer): bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,tag", [(torch.float16, oracle.F16), (torch.bfloat16, oracle.BF16)])
@pytest.mark.parametrize("n", [1, 7, 8, 1001, 64 * 4096, 3_000_005])
@pytest.mark.parametrize("bits", [8, 4])
def test_absmax_scale_matches_oracle(dtype, tag, n, bits):
    x = (torch.randn(n, generator=torch.Generator().manual_seed(n)) * 3).to(dtype)
    if n > 100:
        x[n // 3] = -77.0
    xb = oracle.bits_of(x)[0]
    out = torch.zeros(1, device="cuda")
    ws = torch.empty(P.sasq_absmax_scale_workspace(n), dtype=torch.uint8, device="cuda")
    P.sasq_absmax_scale(x.cuda(), out, ws, bits)
    assert np.float32(out.item()) == oracle.absmax_scale(xb, tag, bits)


@pytest.mark.parametrize("N,K", [(1, 16), (37, 200), (256, 4096), (300, 11008)])
@pytest.mark.parametrize("bits", [8, 4])
def test_weight_quantizer_matches_oracle(N, K, bits):
    w = W.weights_fp32(N, K, 5000 + N)
    if N > 5:
        w[5] = 0.0
    w_int_o, ws_o = oracle.quantize_weight(w.numpy(), bits)
    w_int = torch.empty((N, K), dtype=torch.int8, device="cuda")
    ws = torch.empty(N, device="cuda")
    P.sasq_quantize_weight(w.cuda(), w_int, ws, bits)
    assert np.array_equal(ws.cpu().numpy(), ws_o)
    assert np.array_equal(w_int.cpu().numpy(), w_int_o)
