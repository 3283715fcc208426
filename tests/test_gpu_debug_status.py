"""SASQ_DEBUG_STATUS=1: the binding reads the device status word after every call, so a device-detected problem
(here a zero factor) raises at the call that caused it instead of at the caller's next sasq_device_status().
The switch is read when the binding is imported, so the check runs in a child process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, sys.argv[1])
import torch
import paper_2512_14481_b200 as P
x = torch.randn(4096, device="cuda").bfloat16()
y = torch.empty_like(x)
P.sasq_fakequant_fwd(x, y, torch.tensor([0.05], device="cuda"), 8)          # a good factor: no error
try:
    P.sasq_fakequant_fwd(x, y, torch.zeros(1, device="cuda"), 8)             # a zero factor
except P.SasqError as e:
    assert e.status == 4, e.status                                           # SASQ_ERR_BAD_SCALE
    assert P.sasq_device_status() == 0                                       # read and cleared by the binding
    print("raised at the call")
    sys.exit(0)
sys.exit(3)
"""


def test_device_errors_raise_at_the_call_in_debug_mode():
    env = dict(os.environ, SASQ_DEBUG_STATUS="1")
    r = subprocess.run([sys.executable, "-c", CHILD, ROOT], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "raised at the call" in r.stdout
