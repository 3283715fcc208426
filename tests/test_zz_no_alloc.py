"""The workspace-free fused call (sasq_fakequant_fwd_bwd_static) against the regular one.

Some users of this library run where device allocation is off limits -- an inference runtime's plugin hook, or a
process whose memory is wholly owned by another pool -- and cannot pass a workspace either.  For them the library
keeps the reduction scratch in a fixed device array.  This test calls that entry point through the C ABI twice in a
row (different data, different sizes, so stale scratch from the first call is in place for the second) and requires
the outputs to equal the regular entry point's bit for bit -- y, grad_x and grad_scale alike, since the header
promises that both calls reduce in the same order -- and, on the second call, the CPU oracle's: y and grad_x bit
for bit, grad_scale within the 1e-4 relative tolerance used for the scale gradient everywhere else.
Collected last on purpose: a failure here cannot hide another test's result under `pytest -x`.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P

pytestmark = pytest.mark.gpu


def _case(n, seed, dtype):
    g = torch.Generator().manual_seed(seed)
    x = (torch.randn(n, generator=g) * 3).to(dtype).cuda()
    gy = torch.randn(n, generator=g).to(dtype).cuda()
    return x, gy


def _bits(t):
    return t.cpu().view(torch.int16).numpy()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_static_scratch_call_matches_the_workspace_call_twice_in_a_row(dtype):
    scale = torch.tensor([0.037], dtype=torch.float32, device="cuda")
    for n, seed in [(3_000_005, 1), (70_001, 2)]:            # two calls in a row; the second is smaller
        x, gy = _case(n, seed, dtype)
        y_ref, dx_ref, ds_ref = torch.empty_like(x), torch.empty_like(x), torch.zeros(1, device="cuda")
        ws = torch.empty(P.sasq_fakequant_bwd_workspace(n), dtype=torch.uint8, device="cuda")
        P.sasq_fakequant_fwd_bwd(x, gy, y_ref, dx_ref, ds_ref, scale, ws, 8)
        y, dx, ds = torch.empty_like(x), torch.empty_like(x), torch.full((1,), 55.0, device="cuda")
        P.sasq_fakequant_fwd_bwd_static(x, gy, y, dx, ds, scale, 8)
        assert P.sasq_device_status() == 0
        assert np.array_equal(_bits(y), _bits(y_ref))
        assert np.array_equal(_bits(dx), _bits(dx_ref))
        assert ds.item() == ds_ref.item()                      # same reduction order, same bits
        # accumulate adds to what is there (one fp32 addition of the same value: exact doubling)
        P.sasq_fakequant_fwd_bwd_static(x, gy, y, dx, ds, scale, 8, accumulate=True)
        assert ds.item() == 2 * ds_ref.item()
    # the second call's results against the CPU oracle, on the same bytes
    xb, tag = oracle.bits_of(x.cpu())
    gb, _ = oracle.bits_of(gy.cpu())
    s = float(scale.item())
    y_o, _ = oracle.fakequant_fwd(xb, tag, s, 8, want_codes=False)
    dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, s, 8)
    assert np.array_equal(oracle.bits_of(y.cpu())[0], y_o)
    assert np.array_equal(oracle.bits_of(dx.cpu())[0], dx_o)
    assert abs(ds_ref.item() - ds_o) <= 1e-4 * abs(ds_o)


def test_static_scratch_call_rejects_oversized_tensors_without_launching():
    lib = P.load_library()
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    f = torch.ones(1, dtype=torch.float32, device="cuda")
    rc = lib.sasq_fakequant_fwd_bwd_static(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), f.data_ptr(), 0,
                                           (1 << 30) + 8, P.SASQ_BF16, f.data_ptr(), 8, None)
    assert rc == 2      # SASQ_ERR_UNSUPPORTED
    assert "UNSUPPORTED" in P.sasq_status_string(rc)
