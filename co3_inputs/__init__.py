"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

Holds no arithmetic of the compression method: only random tensors with the shapes and
distributions of the paper's workloads (per-layer i.i.d. generalized-normal gradients,
Sec. II-C and Sec. III), the layer layout used by the multi-layer configurations, and the
per-layer parameters of each configuration.
"""
from __future__ import annotations

import math

import numpy as np
import torch

# Trainable tensors of an 18-layer residual network with a 10-class head (conv weights,
# batch-norm scale/shift pairs, projection shortcuts, classifier weight and bias), in
# forward order: 62 tensors, 11,181,642 elements.
RESNET18_LAYER_SIZES = (
    9408, 64, 64,
    36864, 64, 64, 36864, 64, 64, 36864, 64, 64, 36864, 64, 64,
    73728, 128, 128, 147456, 128, 128, 8192, 128, 128, 147456, 128, 128, 147456, 128, 128,
    294912, 256, 256, 589824, 256, 256, 32768, 256, 256, 589824, 256, 256, 589824, 256, 256,
    1179648, 512, 512, 2359296, 512, 512, 131072, 512, 512, 2359296, 512, 512, 2359296, 512, 512,
    5120, 10,
)
assert len(RESNET18_LAYER_SIZES) == 62 and sum(RESNET18_LAYER_SIZES) == 11_181_642


def gennorm_sigma(alpha: float, beta: float) -> float:
    """Standard deviation of GenNorm(0, alpha, beta): alpha * sqrt(Gamma(3/beta) / Gamma(1/beta))."""
    return alpha * math.sqrt(math.exp(math.lgamma(3.0 / beta) - math.lgamma(1.0 / beta)))


def gennorm(n: int, beta: float, alpha: float, seed: int, device: str = "cpu",
            outlier_frac: float = 0.0, outlier_mult: float = 1.0) -> torch.Tensor:
    """n i.i.d. GenNorm(0, alpha, beta) samples as fp32: sign * alpha * G^(1/beta), G ~ Gamma(1/beta, 1).

    With outlier_frac > 0 each position is independently (Bernoulli) redrawn at
    alpha * outlier_mult.  The stream depends on (seed, device type) only.
    """
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    out = torch.empty(n, dtype=torch.float32, device=device)
    step = 1 << 24
    for lo in range(0, n, step):
        k = min(step, n - lo)
        conc = torch.full((k,), 1.0 / beta, dtype=torch.float64, device=device)
        g = torch._standard_gamma(conc, generator=gen)
        mag = g.pow_(1.0 / beta)
        sign = torch.randint(0, 2, (k,), generator=gen, device=device, dtype=torch.int8)
        scale = torch.full((k,), alpha, dtype=torch.float64, device=device)
        if outlier_frac > 0.0:
            pick = torch.rand(k, generator=gen, device=device, dtype=torch.float64) < outlier_frac
            scale = torch.where(pick, scale * outlier_mult, scale)
        x = mag * scale
        x = torch.where(sign.bool(), x, -x)
        out[lo:lo + k] = x.to(torch.float32)
    return out


def layer_params(n_layers: int, seed: int, beta_range=(0.6, 1.2), log10_alpha_range=(-4.0, -2.0)):
    """Per-layer (beta, alpha): beta ~ U[beta_range], log10 alpha ~ U[log10_alpha_range], drawn once."""
    rng = np.random.default_rng(seed)
    beta = rng.uniform(beta_range[0], beta_range[1], size=n_layers)
    alpha = 10.0 ** rng.uniform(log10_alpha_range[0], log10_alpha_range[1], size=n_layers)
    return beta, alpha


def layered_gradient(sizes, beta, alpha, seed: int, device: str = "cpu") -> torch.Tensor:
    """One client's flat gradient: layer k is i.i.d. GenNorm(0, alpha[k], beta[k]); layers independent."""
    parts = [gennorm(int(n), float(beta[k]), float(alpha[k]), seed * 1_000_003 + k, device)
             for k, n in enumerate(sizes)]
    return torch.cat(parts) if parts else torch.empty(0, dtype=torch.float32, device=device)


def client_round_seed(base: int, client: int, rnd: int) -> int:
    """Seed of the gradient of one client in one round."""
    return base + 1000 * client + rnd


# ------------------------------------------------------------------------------------------------
# Format scale ("exponent bias") per layer.  The stored table holds, per format and shape value,
# the multiplier that minimises the expected squared conversion error for a unit-scale GenNorm;
# it is written by make_scale_table.py from the CPU oracle and only read here.
_SCALE_TABLE = None


def _scale_table() -> dict:
    global _SCALE_TABLE
    if _SCALE_TABLE is None:
        import json
        import os
        with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "scale_table.json")) as fh:
            _SCALE_TABLE = json.load(fh)
    return _SCALE_TABLE


def scale_log_table(formats) -> tuple[np.ndarray, float, float]:
    """(float32[len(formats)][n_beta] natural logarithms of the stored multipliers, beta0, dbeta) for the given
    (exp_bits, mant_bits) pairs: the table a data-driven fit of the multiplier interpolates in."""
    t = _scale_table()
    betas = np.asarray(t["betas"], dtype=np.float64)
    rows = [np.log(np.asarray(t["formats"]["%d,%d" % (E, M)], dtype=np.float64)) for (E, M) in formats]
    return np.asarray(rows, dtype=np.float32), float(betas[0]), float(betas[1] - betas[0])


def scale_for(exp_bits: int, mant_bits: int, beta: float, alpha: float) -> tuple[float, float]:
    """(scale, inv_scale) as fp32 values for a layer modelled as GenNorm(0, alpha, beta)."""
    _SCALE_TABLE = _scale_table()
    betas = np.asarray(_SCALE_TABLE["betas"], dtype=np.float64)
    row = np.asarray(_SCALE_TABLE["formats"]["%d,%d" % (exp_bits, mant_bits)], dtype=np.float64)
    b = min(max(float(beta), float(betas[0])), float(betas[-1]))
    s_unit = math.exp(float(np.interp(b, betas, np.log(row))))
    s = np.float32(s_unit / alpha)
    inv = np.float32(1.0) / s
    return float(s), float(inv)


# ------------------------------------------------------------------------------------------------
# The five workload configurations (sizes, shapes and distributions; synthetic stand-ins for the
# paper's training gradients).  `clients`, `rounds` and sizes are the full-size values; tests pass
# smaller ones through the same recipe.
def config(idx: int) -> dict:
    if idx == 1:
        return dict(name="cfg1_flat1M_fit_per_round", clients=1, sizes=(1_000_000,), beta=(1.0,), alpha=(1e-3,),
                    fmt=(4, 3), decay=0.9, rounds=10, seed=0, fit_per_round=True)
    if idx in (2, 3):
        beta, alpha = layer_params(len(RESNET18_LAYER_SIZES), seed=2)
        return dict(name="cfg2_resnet18_10clients" if idx == 2 else "cfg3_resnet18_100clients",
                    clients=10 if idx == 2 else 100, sizes=RESNET18_LAYER_SIZES, beta=tuple(beta),
                    alpha=tuple(alpha), fmt=(4, 3), decay=0.9, rounds=20 if idx == 2 else 1,
                    seed=2000 if idx == 2 else 3000, fit_per_round=False)
    if idx == 4:
        cells = [dict(fmt=f, beta=b, decay=d) for f in ((2, 1), (3, 0), (4, 3), (5, 2))
                 for b in (0.5, 1.0, 2.0) for d in (0.5, 0.9, 0.99)]
        return dict(name="cfg4_sweep_25p6M", clients=1, sizes=(25_600_000,), alpha=(1e-3,), rounds=5,
                    seed=4000, cells=cells, fit_per_round=False)
    if idx == 5:
        return dict(name="cfg5_1G_outliers", clients=1, sizes=(1_000_000_000,), beta=(0.8,), alpha=(1e-3,),
                    fmt=(4, 3), decay=0.9, rounds=3, seed=5000, outlier_frac=1e-4, outlier_mult=100.0,
                    fit_per_round=False,
                    part_b=dict(clients=8, sizes=(125_000_000,)))
    raise ValueError("config index 1..5")
