"""Pins for the CPU oracle's quantizer: checks against what the paper and the
mathematics fix, none of which re-type the oracle's own formula.

  * 16-bit conversions against numpy (binary16) and torch (bfloat16), exhaustively;
  * a hand-worked 4-bit example (tests/golden/quantizer_b4_s0p5.txt; Eq. 1, Eq. 4);
  * exact rational arithmetic on inputs where x/s is exact (tie rule, clamp ends);
  * invariants: idempotence, clip bounds, half-step error, power-of-two identity;
  * the scale gradient against fp64 central differences of the STE surrogate,
    against torch float64 autograd, and against closed forms;
  * Table 3's ablation variants against their closed forms.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import BF16, F16, FULL, NO_CLAMP, NO_ROUND

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
TAGS = [F16, BF16]
TDT = {F16: torch.float16, BF16: torch.bfloat16}


def to_bits(vals, tag):
    """python floats / fp32 array -> 16-bit patterns via torch's own rounding (not the oracle's)."""
    t = torch.as_tensor(np.asarray(vals, dtype=np.float64)).to(TDT[tag])
    return oracle.bits_of(t)[0]


def from_bits(bits, tag):
    return oracle.tensor_of(bits, tag).to(torch.float64).numpy()


# ---------------------------------------------------------------------------
# 16-bit conversions
# ---------------------------------------------------------------------------
def test_widen_half_exhaustive_vs_numpy():
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    got = oracle.widen(allbits, F16)
    ref = allbits.view(np.float16).astype(np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_widen_bf16_exhaustive_vs_torch():
    allbits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    got = oracle.widen(allbits, BF16)
    ref = oracle.tensor_of(allbits, BF16).to(torch.float32).numpy()
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def _narrow_cases():
    rng = np.random.default_rng(7)
    bits = rng.integers(0, 2**32, size=400_000, dtype=np.uint64).astype(np.uint32)
    rnd = bits.view(np.float32)
    small = (rng.standard_normal(200_000) * 10.0 ** rng.uniform(-9, 5, 200_000)).astype(np.float32)
    # every half-way point between adjacent binary16 values, and its two fp32 neighbours
    h = np.arange(0, 0x7C00, dtype=np.uint16)
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    mid = ((lo + hi) / 2).astype(np.float32)
    ties = np.concatenate([mid, np.nextafter(mid, np.float32(np.inf)), np.nextafter(mid, np.float32(-np.inf))])
    edge = np.array([0.0, -0.0, np.inf, -np.inf, 65504.0, 65519.9, 65520.0, 65536.0, 6e-8, 2.98e-8, 2.99e-8,
                     6.1e-5, 3.3895e38, 3.4e38, 1e-40, -1e-40], dtype=np.float32)
    return np.concatenate([rnd, small, ties, -ties, edge])


def test_narrow_half_vs_numpy():
    v = _narrow_cases()
    v = v[~np.isnan(v)]
    got = oracle.narrow(v, F16)
    with np.errstate(over="ignore"):
        ref = v.astype(np.float16).view(np.uint16)
    assert np.array_equal(got, ref)


def test_narrow_bf16_vs_torch():
    v = _narrow_cases()
    v = v[~np.isnan(v)]
    got = oracle.narrow(v, BF16)
    ref = oracle.bits_of(torch.from_numpy(v.copy()).to(torch.bfloat16))[0]
    assert np.array_equal(got, ref)


def test_narrow_nan_stays_nan():
    for tag in TAGS:
        out = oracle.narrow(np.array([np.nan, -np.nan], dtype=np.float32), tag)
        assert np.all(np.isnan(from_bits(out, tag)))


# ---------------------------------------------------------------------------
# hand-worked example
# ---------------------------------------------------------------------------
def _load_golden():
    rows = []
    with open(os.path.join(GOLDEN, "quantizer_b4_s0p5.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(v) for v in line.split()])
    a = np.array(rows)
    return dict(x=a[:, 0], g=a[:, 1], t=a[:, 2], r=a[:, 3], c=a[:, 4], inside=a[:, 5], y=a[:, 6], term=a[:, 7])


@pytest.mark.parametrize("tag", TAGS)
def test_golden_hand_worked_example(tag):
    G = _load_golden()
    x = to_bits(G["x"], tag)
    g = to_bits(G["g"], tag)
    assert np.array_equal(from_bits(x, tag), G["x"]) and np.array_equal(from_bits(g, tag), G["g"])
    y, codes = oracle.fakequant_fwd(x, tag, 0.5, bits=4)
    assert np.array_equal(codes, G["c"].astype(np.int32))
    assert np.array_equal(from_bits(y, tag), G["y"])
    dx, ds = oracle.fakequant_bwd(x, g, tag, 0.5, bits=4)
    assert np.array_equal(from_bits(dx, tag), G["g"] * G["inside"])
    assert ds == -23.75
    assert ds == float(np.sum(G["g"] * G["term"]))
    assert np.array_equal(oracle.quantize_act(x, tag, 0.5, bits=4), G["c"].astype(np.int8))


# ---------------------------------------------------------------------------
# exact rational arithmetic where x/s is exact (s a power of two)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("tag", TAGS)
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("s", [0.25, -0.125, 4.0])
def test_codes_vs_exact_rationals(tag, bits, s):
    qn, qp = 2 ** (bits - 1), 2 ** (bits - 1) - 1
    # a grid containing every tie (k + 1/2) * |s| and values far outside the range
    ks = np.arange(-4 * qn - 3, 4 * qn + 4)
    xs = np.concatenate([ks * abs(s) / 2, ks * abs(s) / 4, [1000.0 * abs(s), -1000.0 * abs(s)]])
    xb = to_bits(xs, tag)
    xv = from_bits(xb, tag)                # storage rounding may move a point; x/s stays exact (s = 2^k)
    _, codes = oracle.fakequant_fwd(xb, tag, s, bits=bits)
    want = [max(-qn, min(qp, round(Fraction(float(v)) / Fraction(s)))) for v in xv]   # Fraction rounds half to even
    assert codes.tolist() == want
    assert oracle.quantize_act(xb, tag, s, bits=bits).tolist() == want


# ---------------------------------------------------------------------------
# invariants on random data
# ---------------------------------------------------------------------------
def _rand_x(tag, n, seed, scale=3.0):
    rng = np.random.default_rng(seed)
    v = rng.standard_normal(n) * scale
    v[rng.integers(0, n, n // 50)] *= 40.0
    return to_bits(v, tag)


@pytest.mark.parametrize("tag", TAGS)
@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("s", [0.037, -0.21, 1.0 / 3.0])
def test_bounds_and_half_step_error(tag, bits, s):
    qn, qp = 2 ** (bits - 1), 2 ** (bits - 1) - 1
    x = _rand_x(tag, 20000, 11)
    y, codes = oracle.fakequant_fwd(x, tag, s, bits=bits)
    assert codes.min() >= -qn and codes.max() <= qp
    assert codes.min() == -qn and codes.max() == qp          # the data really saturates both ends
    xv, yv = from_bits(x, tag), from_bits(y, tag)
    ulp = 2.0 ** -10 if tag == F16 else 2.0 ** -7
    assert np.all(np.abs(yv) <= qn * abs(s) * (1 + ulp))
    s32 = float(np.float32(s))
    inside = (codes > -qn) & (codes < qp)
    # unclipped: |x - c*s| <= |s|/2 up to fp32 rounding of x/s and the output narrowing
    err = np.abs(xv - codes * s32)
    assert np.all(err[inside] <= abs(s32) / 2 * (1 + 1e-5) + np.abs(xv[inside]) * 2e-7)
    # y is c*s rounded once to the storage type
    assert np.all(np.abs(yv - codes * s32) <= np.abs(codes * s32) * ulp / 2 * (1 + 1e-6) + 1e-30)
    # clipped on the positive / negative side exactly when x/s is beyond the last half step
    u = xv / s32
    assert np.all(codes[u > qp + 0.5001] == qp) and np.all(codes[u < -qn - 0.5001] == -qn)


@pytest.mark.parametrize("bits", [4, 8])
def test_idempotence_fp16(bits):
    """Q(Q(x)) = Q(x) on fp16 storage: re-quantizing c*s gives c back."""
    s = 0.0371
    x = _rand_x(F16, 20000, 5)
    y, codes = oracle.fakequant_fwd(x, F16, s, bits=bits)
    y2, codes2 = oracle.fakequant_fwd(y, F16, s, bits=bits)
    assert np.array_equal(codes2, codes)
    assert np.array_equal(y2, y)


@pytest.mark.parametrize("bits", [4, 8])
def test_idempotence_bf16_representable_scale(bits):
    """bf16 keeps 8 significant bits, so c*s is stored exactly when s is a power of two."""
    s = 2.0 ** -4
    x = _rand_x(BF16, 20000, 6)
    y, codes = oracle.fakequant_fwd(x, BF16, s, bits=bits)
    y2, codes2 = oracle.fakequant_fwd(y, BF16, s, bits=bits)
    assert np.array_equal(codes2, codes) and np.array_equal(y2, y)


@pytest.mark.parametrize("tag", TAGS)
def test_power_of_two_grid_is_a_fixed_point(tag):
    s = 2.0 ** -3
    k = np.arange(-128, 128)
    x = to_bits(k * s, tag)
    y, codes = oracle.fakequant_fwd(x, tag, s, bits=8)
    assert np.array_equal(codes, k)
    assert np.array_equal(from_bits(y, tag), k * s)


@pytest.mark.parametrize("tag", TAGS)
def test_sign_symmetry_except_at_the_ends(tag):
    s = 0.05
    x = _rand_x(tag, 5000, 3)
    xn = (x ^ np.uint16(0x8000)).astype(np.uint16)
    _, c = oracle.fakequant_fwd(x, tag, s, bits=8)
    _, cn = oracle.fakequant_fwd(xn, tag, s, bits=8)
    sym = (c > -127) & (c < 127) & (cn > -127) & (cn < 127)
    assert np.array_equal(cn[sym], -c[sym])
    # a negative scale mirrors the codes the same way
    _, cs = oracle.fakequant_fwd(x, tag, -s, bits=8)
    assert np.array_equal(cs, cn)


def test_four_bit_has_at_most_16_levels():
    x = _rand_x(BF16, 50000, 9)
    y, codes = oracle.fakequant_fwd(x, BF16, 0.4, bits=4)
    assert len(np.unique(codes)) == 16
    assert len(np.unique(from_bits(y, BF16))) <= 16


@pytest.mark.parametrize("tag", TAGS)
def test_absmax_scale_vs_numpy(tag):
    x = _rand_x(tag, 4096, 21)
    for bits in (4, 8):
        qp = 2 ** (bits - 1) - 1
        want = np.float32(np.max(np.abs(from_bits(x, tag))).astype(np.float32) / np.float32(qp))
        assert oracle.absmax_scale(x, tag, bits) == want
    # with that factor nothing is clipped and the largest element maps to +-Qp (Eq. 1)
    s = float(oracle.absmax_scale(x, tag, 8))
    _, codes = oracle.fakequant_fwd(x, tag, s, bits=8)
    assert np.max(np.abs(codes)) == 127


# ---------------------------------------------------------------------------
# input gradient (Eq. 4)
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("tag", TAGS)
def test_dx_is_g_or_zero(tag):
    s, bits = 0.05, 8
    x = _rand_x(tag, 20000, 13)
    g = _rand_x(tag, 20000, 14, scale=1.0)
    dx, _ = oracle.fakequant_bwd(x, g, tag, s, bits=bits)
    u = from_bits(x, tag) / float(np.float32(s))
    sure_in = np.abs(u) < 126.0
    sure_out = (u > 127.6) | (u < -128.6)
    assert sure_in.sum() > 0 and sure_out.sum() > 0
    assert np.array_equal(dx[sure_in], g[sure_in])
    assert np.all(dx[sure_out] == 0)
    assert np.all((dx == g) | (dx == 0))
    # all inside -> dx == g ; all clipped -> dx == 0
    small = to_bits(np.linspace(-1, 1, 999), tag)
    gg = _rand_x(tag, 999, 15, scale=1.0)
    assert np.array_equal(oracle.fakequant_bwd(small, gg, tag, 1.0, bits=8)[0], gg)
    big = to_bits(np.where(np.arange(999) % 2 == 0, 300.0, -300.0), tag)
    assert np.all(oracle.fakequant_bwd(big, gg, tag, 1.0, bits=8)[0] == 0)


# ---------------------------------------------------------------------------
# scale gradient
# ---------------------------------------------------------------------------
def _ste_surrogate_fd(xv, gv, s, qn, qp, rel_h=1e-6):
    """fp64 central difference of f(s') = sum g * s' * clamp(x/s' + delta), delta = round(x/s) - x/s frozen at s.
    This is the function whose derivative the straight-through rules of Eq. 4 define."""
    u = xv / s
    delta = np.rint(u) - u

    def f(sp):
        return float(np.sum(gv * sp * np.clip(xv / sp + delta, -qn, qp)))

    h = abs(s) * rel_h
    return (f(s + h) - f(s - h)) / (2 * h)


@pytest.mark.parametrize("tag", TAGS)
@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("s", [0.25, -0.5])
def test_ds_vs_finite_differences_exact_grid(tag, bits, s):
    """x on a grid where x/s is exact in fp32, kept away from the clamp kinks."""
    qn, qp = 2 ** (bits - 1), 2 ** (bits - 1) - 1
    rng = np.random.default_rng(31)
    k = rng.integers(-3 * qn * 8, 3 * qn * 8, size=200)         # x = k * |s| / 8, then rounded to storage
    xb = to_bits(k * abs(s) / 8.0, tag)
    u = from_bits(xb, tag) / abs(s)                               # exact: s is a power of two
    # the surrogate has its kinks where the rounded value sits exactly on a clamp bound
    keep = (np.abs(np.abs(np.rint(u)) - qp) > 0.5) & (np.abs(np.abs(np.rint(u)) - qn) > 0.5) \
        & (np.abs(u - np.floor(u) - 0.5) > 0.05)
    xb = xb[keep]
    xv = from_bits(xb, tag)
    gv = rng.integers(-8, 9, size=xv.size) / 4.0
    gb = to_bits(gv, tag)
    _, ds = oracle.fakequant_bwd(xb, gb, tag, s, bits=bits)
    fd = _ste_surrogate_fd(xv, gv, s, qn, qp)
    assert abs(ds - fd) <= 1e-6 * max(1.0, abs(fd))
    assert (np.abs(xv / s) > qn + 1).sum() > 0                     # some elements really are clipped


@pytest.mark.parametrize("tag", TAGS)
def test_ds_vs_finite_differences_generic_scale(tag):
    qn, qp = 128, 127
    s = 0.0437
    rng = np.random.default_rng(32)
    xv = rng.standard_normal(64) * 3.0
    xv[:6] *= 5.0
    xb = to_bits(xv, tag)
    xv = from_bits(xb, tag)
    u = xv / float(np.float32(s))
    keep = (np.abs(np.abs(np.rint(u)) - 127) > 0.5) & (np.abs(np.abs(np.rint(u)) - 128) > 0.5) \
        & (np.abs(u - np.rint(u)) < 0.45)
    xb, xv = xb[keep], xv[keep]
    gv = rng.standard_normal(xv.size)
    gb = to_bits(gv, tag)
    gv = from_bits(gb, tag)
    _, ds = oracle.fakequant_bwd(xb, gb, tag, s, bits=8)
    fd = _ste_surrogate_fd(xv, gv, float(np.float32(s)), qn, qp)
    # fp32 evaluation of x/s differs from the fp64 one by ~1e-7 relative per element
    assert abs(ds - fd) <= 2e-5 * np.sum(np.abs(gv)) + 1e-6 * abs(fd)
    assert (np.abs(u[keep]) > 129).sum() > 0


@pytest.mark.parametrize("tag", TAGS)
@pytest.mark.parametrize("bits", [4, 8])
def test_ds_vs_torch_autograd_float64(tag, bits):
    """Composing clamp after a straight-through round with autograd gives Eq. 4's rules."""
    qn, qp = 2 ** (bits - 1), 2 ** (bits - 1) - 1
    s0 = 0.3 if bits == 4 else 0.02
    rng = np.random.default_rng(33)
    xs = rng.standard_normal(200) * 2.0
    s32 = float(np.float32(s0))
    # plant elements whose rounded value lands exactly on each clamp bound (inclusive in Eq. 4) and just beyond
    xs[:6] = np.array([qp - 0.3, qp + 0.3, qp + 0.7, -qn + 0.3, -qn - 0.3, -qn - 0.7]) * s32
    xb = to_bits(xs, tag)
    # x * fl32(1/s) and the exact quotient may fall on different sides of a tie: keep clear of ties
    uu = from_bits(xb, tag) / s32
    xb = xb[np.abs(uu - np.floor(uu) - 0.5) > 1e-3]
    assert np.array_equal(xb[:6], to_bits(xs[:6], tag))
    gb = to_bits(rng.standard_normal(xb.size), tag)
    xv = torch.from_numpy(from_bits(xb, tag))
    gv = torch.from_numpy(from_bits(gb, tag))
    s = torch.tensor(float(np.float32(s0)), dtype=torch.float64, requires_grad=True)
    xt = xv.clone().requires_grad_(True)
    u = xt / s
    r = (u.round() - u).detach() + u          # torch.round is half-to-even
    y = r.clamp(-qn, qp) * s
    y.backward(gv)
    dx, ds = oracle.fakequant_bwd(xb, gb, tag, s0, bits=bits)
    assert abs(ds - s.grad.item()) <= 2e-5 * float(gv.abs().sum()) + 1e-6 * abs(s.grad.item())
    assert np.array_equal(from_bits(dx, tag), xt.grad.numpy())
    assert (xt.grad == 0).sum() > 0 and (xt.grad != 0).sum() > 0
    # forward agrees as well, up to the storage rounding of y
    yb, _ = oracle.fakequant_fwd(xb, tag, s0, bits=bits)
    ulp = 2.0 ** -10 if tag == F16 else 2.0 ** -7
    assert np.allclose(from_bits(yb, tag), y.detach().numpy(), rtol=ulp, atol=0)


@pytest.mark.parametrize("tag", TAGS)
def test_ds_closed_forms(tag):
    s = 0.5
    rng = np.random.default_rng(34)
    gv = rng.integers(-8, 9, size=300) / 4.0
    gb = to_bits(gv, tag)
    # all on the grid and inside: r - t = 0 everywhere
    xb = to_bits(rng.integers(-128, 128, size=300) * s, tag)
    assert oracle.fakequant_bwd(xb, gb, tag, s, bits=8)[1] == 0.0
    # all clipped: ds = sum g * (+Qp or -Qn)
    sign = np.where(rng.random(300) < 0.5, 1.0, -1.0)
    xb = to_bits(sign * 200.0, tag)
    want = float(np.sum(gv * np.where(sign > 0, 127.0, -128.0)))
    assert oracle.fakequant_bwd(xb, gb, tag, s, bits=8)[1] == want
    # negative scale flips the side that clips
    want_neg = float(np.sum(gv * np.where(sign > 0, -128.0, 127.0)))
    assert oracle.fakequant_bwd(xb, gb, tag, -s, bits=8)[1] == want_neg
    # half-way inside: x = (k + 1/4) s -> r - t = -1/4
    xb = to_bits((rng.integers(-15, 16, size=300) + 0.25) * s, tag)     # exact in bf16 too
    assert oracle.fakequant_bwd(xb, gb, tag, s, bits=8)[1] == float(np.sum(gv) * -0.25)


def test_ds_is_linear_in_g_and_additive_over_rows():
    tag, s = BF16, 0.031
    x = _rand_x(tag, 6000, 41).reshape(6, 1000)
    g = _rand_x(tag, 6000, 42, scale=1.0).reshape(6, 1000)
    _, ds = oracle.fakequant_bwd(x, g, tag, s)
    parts = [oracle.fakequant_bwd(x[i], g[i], tag, s)[1] for i in range(6)]
    assert abs(ds - sum(parts)) <= 1e-12 * sum(abs(p) for p in parts)
    g2 = to_bits(2.0 * from_bits(g, tag), tag)
    assert abs(oracle.fakequant_bwd(x, g2, tag, s)[1] - 2 * ds) <= 1e-12 * abs(ds)


# ---------------------------------------------------------------------------
# Table 3 variants
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("tag", TAGS)
def test_variant_without_round(tag):
    """y = s*clamp(x/s): the identity inside the range (up to fp32 rounding), derivative wrt s zero there."""
    s = 0.25
    rng = np.random.default_rng(51)
    xv = rng.integers(-2000, 2000, size=500) / 16.0
    xb, gb = to_bits(xv, tag), to_bits(rng.integers(-8, 9, size=500) / 4.0, tag)
    xv = from_bits(xb, tag)                # the stored values; x/s is exact for s = 2^-2
    gv = from_bits(gb, tag)
    y, _ = oracle.fakequant_fwd(xb, tag, s, bits=8, variant=NO_ROUND)
    assert np.array_equal(from_bits(y, tag), np.clip(xv, -128 * s, 127 * s))
    dx, ds = oracle.fakequant_bwd(xb, gb, tag, s, bits=8, variant=NO_ROUND)
    u = xv / s
    assert np.array_equal(from_bits(dx, tag), gv * ((u >= -128) & (u <= 127)))
    assert ds == float(np.sum(gv * np.where(u > 127, 127.0, np.where(u < -128, -128.0, 0.0))))


@pytest.mark.parametrize("tag", TAGS)
def test_variant_without_clamp(tag):
    """y = s*round(x/s): nothing is masked; dy/ds = r - t everywhere."""
    s = 0.5
    rng = np.random.default_rng(52)
    xv = rng.integers(-4000, 4000, size=500) / 8.0
    xb, gb = to_bits(xv, tag), to_bits(rng.integers(-8, 9, size=500) / 4.0, tag)
    gv = from_bits(gb, tag)
    y, codes = oracle.fakequant_fwd(xb, tag, s, bits=8, variant=NO_CLAMP)
    want_r = np.array([round(Fraction(float(v)) / Fraction(s)) for v in from_bits(xb, tag)], dtype=np.float64)
    assert np.array_equal(codes, want_r.astype(np.int32))
    assert np.abs(codes).max() > 200
    dx, ds = oracle.fakequant_bwd(xb, gb, tag, s, bits=8, variant=NO_CLAMP)
    assert np.array_equal(dx, gb)
    assert ds == float(np.sum(gv * (want_r - from_bits(xb, tag) / s)))


# ---------------------------------------------------------------------------
# per-channel factors reduce to the per-tensor routine column by column
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("tag", TAGS)
def test_per_channel_reduces_to_per_tensor_on_each_column(tag):
    rows, cols = 37, 9
    x = _rand_x(tag, rows * cols, 61).reshape(rows, cols)
    g = _rand_x(tag, rows * cols, 62, scale=1.0).reshape(rows, cols)
    s = np.array([0.02, 0.5, -0.1, 0.033, 1.0, 0.25, 0.07, 2.0, 0.011], dtype=np.float32)
    y, codes = oracle.fakequant_fwd_per_channel(x, tag, s, bits=8)
    dx, ds = oracle.fakequant_bwd_per_channel(x, g, tag, s, bits=8)
    for c in range(cols):
        yc, cc = oracle.fakequant_fwd(np.ascontiguousarray(x[:, c]), tag, float(s[c]))
        dxc, dsc = oracle.fakequant_bwd(np.ascontiguousarray(x[:, c]), np.ascontiguousarray(g[:, c]), tag, float(s[c]))
        assert np.array_equal(y[:, c], yc) and np.array_equal(codes[:, c], cc)
        assert np.array_equal(dx[:, c], dxc)
        assert abs(ds[c] - dsc) <= 1e-12 * max(1.0, abs(dsc))


def test_rejects_bad_arguments():
    x = np.zeros(4, np.uint16)
    with pytest.raises(ValueError):
        oracle.fakequant_fwd(x, F16, 1.0, bits=9)
    with pytest.raises(ValueError):
        oracle.fakequant_fwd(x, F16, 1.0, bits=1)
    with pytest.raises(ValueError):
        oracle.fakequant_bwd(x, x, F16, 1.0, bits=8, variant=3)
