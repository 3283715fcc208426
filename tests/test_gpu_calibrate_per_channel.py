"""GPU parity of the per-channel calibration helpers (Sec. 4.1 with the per-channel granularity of Sec. 5.1): the
max-based factor of every channel of a batch, bit for bit against the oracle's Eq. 1 applied to each column, and the
running mean over calibration batches against the float64 mean (fp32 on the device: 1e-6 relative)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P
import sasq_workloads as W

pytestmark = pytest.mark.gpu

DT = {oracle.F16: torch.float16, oracle.BF16: torch.bfloat16}


def oracle_channels(xb, tag, bits):
    return np.array([oracle.absmax_scale(np.ascontiguousarray(xb[:, k]), tag, bits) for k in range(xb.shape[1])],
                    np.float32)


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("T,K,bits", [(1, 8, 8), (37, 264, 8), (300, 520, 4), (1000, 4096, 8)])
def test_per_channel_factors_match_eq1_on_every_column(tag, T, K, bits):
    x = W.activations(T, K, DT[tag], 8800 + T + K)
    x[:, 3] = 0                                            # an all-zero channel gives 0
    xb = oracle.bits_of(x)[0]
    out = torch.full((K,), 7.0, device="cuda")
    P.sasq_absmax_scale_per_channel(x.cuda(), out, bits)
    torch.cuda.synchronize()
    want = oracle_channels(xb, tag, bits)
    assert want[3] == 0.0
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_empty_batch_gives_zeros_and_shape_errors_are_reported():
    out = torch.full((16,), 7.0, device="cuda")
    P.sasq_absmax_scale_per_channel(torch.empty((0, 16), dtype=torch.bfloat16, device="cuda"), out)
    torch.cuda.synchronize()
    assert bool((out == 0).all())
    with pytest.raises(RuntimeError):                      # K % 8 != 0
        P.sasq_absmax_scale_per_channel(torch.zeros((4, 12), dtype=torch.bfloat16, device="cuda"),
                                        torch.zeros(12, device="cuda"))


def test_running_mean_over_calibration_batches():
    tag, T, K, batches = oracle.BF16, 64, 512, 6
    mean = torch.full((K,), -3.0, device="cuda")           # whatever it held before the first batch is dropped
    value = torch.empty(K, device="cuda")
    per_batch = []
    for b in range(batches):
        x = W.activations(T, K, torch.bfloat16, 8900 + b)
        per_batch.append(oracle_channels(oracle.bits_of(x)[0], tag, 8).astype(np.float64))
        P.sasq_absmax_scale_per_channel(x.cuda(), value, 8)
        P.sasq_running_mean(mean, value, b + 1)
        if b == 0:
            torch.cuda.synchronize()
            assert torch.equal(mean, value)
    torch.cuda.synchronize()
    want = np.mean(per_batch, axis=0)
    got = mean.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - want) <= 1e-6 * np.abs(want))
    with pytest.raises(RuntimeError):
        P.sasq_running_mean(mean, value, 0)
