"""The measurement aid behind the bench's tensor roofline: back-to-back int8 tensor-core instructions of the GEMM's
shape.  It must report a rate no tensor core can exceed (8192 multiply-accumulates per clock per SM) and close to it,
leave the device status clean, and leave the library usable (TMEM freed)."""
import pytest
import torch

import paper_2512_14481_b200 as P

pytestmark = pytest.mark.gpu


def test_issue_rate_is_close_to_and_not_above_the_hardware_rate():
    ops, mac = P.sasq_debug_int8_issue_rate(32 * 256, 256)
    assert 0.85 * 8192 <= mac <= 8192 * 1.001
    assert 1.0e15 < ops < 8192 * 2 * 148 * 2.2e9           # positive, below the rate at an impossible 2.2 GHz
    ops_narrow, mac_narrow = P.sasq_debug_int8_issue_rate(32 * 256, 128)
    assert 0 < mac_narrow <= 8192 * 1.001
    assert P.sasq_device_status() == 0
    # a linear right after it: tensor memory was given back
    x = torch.randn((300, 256), device="cuda").bfloat16()
    w = torch.randint(-127, 128, (264, 256), dtype=torch.int8, device="cuda")
    y = torch.empty((300, 264), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(P.sasq_static_w8a8_linear_workspace(300, 264, 256), dtype=torch.uint8, device="cuda")
    P.sasq_static_w8a8_linear(x, w, torch.full((264,), 1e-2, device="cuda"), torch.tensor([0.05], device="cuda"), y,
                              workspace=ws)
    assert P.sasq_device_status() == 0
