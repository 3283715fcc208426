"""Seeded synthetic inputs for the SASQ hot path.

This module only draws random numbers and names shapes; it contains none of the
method's arithmetic (no scale, no rounding, no clamp) so both the CPU oracle's
tests and the CUDA library's tests and benchmark can be fed from it.

The tensors take the shapes of LLaMA-2 linear-layer inputs and the
outlier-channel structure the paper attributes to LLaMA activations (Sec. 3,
"Outlier"; Fig. 3): a small seeded set of channels (columns) carries values tens
of times larger than the rest.  They stand in for real activations on
WikiText / Pile, which need trained weights and datasets.

Seeds: ``seed = 1000 * config + tensor_index``; the outlier channel set is the
first ``max(1, round(p * K))`` entries of a seeded permutation of ``range(K)``.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

# (name, K = in_features, N = out_features) of the seven linears of one decoder layer
LLAMA2_7B_LINEARS = (
    ("q_proj", 4096, 4096),
    ("k_proj", 4096, 4096),
    ("v_proj", 4096, 4096),
    ("o_proj", 4096, 4096),
    ("gate_proj", 4096, 11008),
    ("up_proj", 4096, 11008),
    ("down_proj", 11008, 4096),
)
LLAMA2_13B_LINEARS = (
    ("q_proj", 5120, 5120),
    ("k_proj", 5120, 5120),
    ("v_proj", 5120, 5120),
    ("o_proj", 5120, 5120),
    ("gate_proj", 5120, 13824),
    ("up_proj", 5120, 13824),
    ("down_proj", 13824, 5120),
)


@dataclass(frozen=True)
class ActSpec:
    """How one activation tensor is drawn."""
    dist: str = "normal"          # "normal" = N(0,1); "student_t3" = Student-t, 3 degrees of freedom
    outlier_frac: float = 0.01    # fraction of channels that are outliers
    outlier_gain: float = 50.0    # multiplier on those channels


NORMAL_OUTLIERS = ActSpec("normal", 0.01, 50.0)
HEAVY_TAILED = ActSpec("student_t3", 0.005, 100.0)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def outlier_channels(K: int, frac: float, seed: int) -> torch.Tensor:
    """Indices of the outlier channels (always drawn on the CPU so the set is device-independent)."""
    n = max(1, int(round(frac * K)))
    perm = torch.randperm(K, generator=_gen(seed ^ 0x5A5A, "cpu"))
    return perm[:n].clone()


def activations(T: int, K: int, dtype: torch.dtype, seed: int, spec: ActSpec = NORMAL_OUTLIERS,
                device="cpu", chunk_rows: int = 4096) -> torch.Tensor:
    """[T, K] activations of the given 16-bit dtype with seeded outlier channels."""
    out = torch.empty((T, K), dtype=dtype, device=device)
    g = _gen(seed, device)
    gain = torch.ones(K, dtype=torch.float32, device=device)
    gain[outlier_channels(K, spec.outlier_frac, seed).to(device)] = spec.outlier_gain
    for r0 in range(0, T, chunk_rows):
        r1 = min(T, r0 + chunk_rows)
        z = torch.randn((r1 - r0, K), generator=g, device=device, dtype=torch.float32)
        if spec.dist == "student_t3":
            chi2 = torch.zeros_like(z)
            for _ in range(3):
                n = torch.randn((r1 - r0, K), generator=g, device=device, dtype=torch.float32)
                chi2 += n * n
            z = z / torch.sqrt(chi2 / 3.0)
        elif spec.dist != "normal":
            raise ValueError(spec.dist)
        out[r0:r1] = (z * gain).to(dtype)
    return out


def upstream_grad(T: int, K: int, dtype: torch.dtype, seed: int, device="cpu", chunk_rows: int = 4096) -> torch.Tensor:
    """[T, K] upstream gradient ~ N(0,1) in the given 16-bit dtype."""
    out = torch.empty((T, K), dtype=dtype, device=device)
    g = _gen(seed ^ 0x0F0F0F, device)
    for r0 in range(0, T, chunk_rows):
        r1 = min(T, r0 + chunk_rows)
        out[r0:r1] = torch.randn((r1 - r0, K), generator=g, device=device, dtype=torch.float32).to(dtype)
    return out


def weights_fp32(N: int, K: int, seed: int, device="cpu", std: float = 0.02) -> torch.Tensor:
    """[N, K] fp32 weight ~ N(0, std^2) (nn.Linear layout: one row per output channel)."""
    g = _gen(seed ^ 0x77777, device)
    return torch.randn((N, K), generator=g, device=device, dtype=torch.float32) * std


def learned_scale_factor(seed: int) -> float:
    """Seeded factor in [0.25, 1] applied to a calibrated scale to stand in for a learned one
    (the paper's learned factors truncate outliers, so saturation must really occur)."""
    g = _gen(seed ^ 0x1234, "cpu")
    return float(0.25 + 0.75 * torch.rand((), generator=g).item())


def seed_of(config: int, index: int) -> int:
    return 1000 * int(config) + int(index)


CALIBRATION_TOKENS = 64   # rows of x the initial factor is taken from (one calibration batch)
