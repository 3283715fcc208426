"""GPU parity of Table 3's ablation variants of the fake-quant operator ("w/o round", "w/o clamp") and of the AdamW
step on the factors, against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2512_14481_b200 as P

pytestmark = pytest.mark.gpu
DT = {oracle.F16: torch.float16, oracle.BF16: torch.bfloat16}


def rand_bits(n, tag, seed, scale=3.0):
    g = torch.Generator().manual_seed(seed)
    v = torch.randn(n, generator=g) * scale
    if n >= 50:
        v[torch.randint(0, n, (n // 50,), generator=g)] *= 40.0
    return oracle.bits_of(v.to(DT[tag]))[0]


@pytest.mark.parametrize("tag", [oracle.F16, oracle.BF16])
@pytest.mark.parametrize("variant", [oracle.NO_ROUND, oracle.NO_CLAMP, oracle.FULL])
@pytest.mark.parametrize("bits,s", [(8, 0.0371), (4, -0.6)])
def test_ablation_variants_match_the_oracle(tag, variant, bits, s):
    n = 300_011
    xb, gb = rand_bits(n, tag, 41), rand_bits(n, tag, 42, scale=1.0)
    y_o, _ = oracle.fakequant_fwd(xb, tag, s, bits, variant=variant, want_codes=False)
    dx_o, ds_o = oracle.fakequant_bwd(xb, gb, tag, s, bits, variant=variant)
    x, g = oracle.tensor_of(xb, tag).cuda(), oracle.tensor_of(gb, tag).cuda()
    y, dx, ds = torch.empty_like(x), torch.empty_like(x), torch.zeros(1, device="cuda")
    sc = torch.tensor([s], dtype=torch.float32, device="cuda")
    ws = torch.empty(P.sasq_fakequant_bwd_workspace(n), dtype=torch.uint8, device="cuda")
    P.sasq_fakequant_fwd_bwd_ablation(x, g, y, dx, ds, sc, ws, variant, bits)
    assert P.sasq_device_status() == 0
    assert np.array_equal(oracle.bits_of(y.cpu())[0], y_o)
    assert np.array_equal(oracle.bits_of(dx.cpu())[0], dx_o)
    floor = 4 * 2.0 ** -24 * float(np.abs(oracle.widen(gb, tag)).sum()) * 2 ** (bits - 1)
    assert abs(ds.item() - ds_o) <= 1e-4 * abs(ds_o) + floor
    if variant == oracle.NO_CLAMP:
        assert np.array_equal(dx_o, gb)            # every element passes the gradient
    if variant == oracle.NO_ROUND:
        assert len(np.unique(y_o)) > 2 ** bits     # the output is no longer on the integer grid


def test_invalid_variant_is_rejected():
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    f = torch.ones(1, device="cuda")
    ws = torch.empty(P.sasq_fakequant_bwd_workspace(64), dtype=torch.uint8, device="cuda")
    with pytest.raises(P.SasqError) as e:
        P.sasq_fakequant_fwd_bwd_ablation(x, x, torch.empty_like(x), torch.empty_like(x), f.clone(), f, ws, 3)
    assert e.value.status == 1


def test_adamw_on_the_factors_follows_the_oracle_over_several_steps():
    """224 factors (7 per layer, 32 layers), gradients of the size the quantizer produces; fp32 on the device,
    float64 in the oracle: the factors agree to 1e-6 relative after every step."""
    rng = np.random.default_rng(5)
    n, steps = 224, 8
    s0 = rng.uniform(0.01, 0.2, n).astype(np.float32)
    s_dev = torch.from_numpy(s0.copy()).cuda()
    m_dev, v_dev = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    s, m, v = s0.astype(np.float64), np.zeros(n), np.zeros(n)
    # the hyper-parameters cross the C ABI as fp32: both sides get the same (fp32-representable) values
    hp = {k: float(np.float32(x)) for k, x in dict(lr=2e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01).items()}
    for t in range(1, steps + 1):
        g = rng.normal(0, 300, n).astype(np.float32)
        P.sasq_adamw_scales(s_dev, torch.from_numpy(g).cuda(), m_dev, v_dev, t, **hp)
        s, m, v = oracle.adamw_step(s, g, m, v, t, **hp)
        assert np.allclose(s_dev.cpu().numpy(), s, rtol=1e-6, atol=1e-9)
        # m is a signed sum of terms of the gradients' size: its fp32 rounding error scales with them, not with m
        assert np.allclose(m_dev.cpu().numpy(), m, rtol=1e-6, atol=1e-6 * float(np.abs(g).max()) * t)
        assert np.allclose(v_dev.cpu().numpy(), v, rtol=1e-5, atol=1e-7)
    assert np.abs(s - s0).max() > 1e-4          # the factors did move


def test_adamw_rejects_bad_arguments():
    t = torch.zeros(4, device="cuda")
    with pytest.raises(P.SasqError):
        P.sasq_adamw_scales(t, t.clone(), t.clone(), t.clone(), 0)          # steps count from 1
    with pytest.raises(P.SasqError):
        P.sasq_adamw_scales(t, t.clone(), t.clone(), t.clone(), 1, beta1=1.0)
