"""Variance compensation (section "Variance Align for Exposure Bias").  Test infrastructure.

Rescaling identity: if f ~ N(mu, sigma^2) then Y = mu + (sigma_new/sigma)(f - mu)
has variance sigma_new^2.  The method applies a per-step, per-channel factor
K in R^{St x C} to the intermediate sample:

    x~_t = mu_t + K_t . (x^_t - mu_t)          (channel-wise product)

and fits K_t by minimising rQNSR(x~_t, x'_t)^2 + MSE(x~_t, x'_t) against target
samples x'_t.

Readings (the paper leaves mu_t undefined, prints a garbled closed form, and
its derivation is in a supplement that is not available):
  * mu_t is the spatial mean of x^_t for each (sample, channel).
  * rQNSR^2 = sum ((x~ - x')/x')^2 and MSE = sum (x~ - x')^2 over the N elements
    (all samples and positions of the channel at that step).  With a = x^ - mu,
    b = x' - mu, setting the derivative to zero gives
        K = (sum a b + sum a b / x'^2) / (sum a^2 + sum a^2 / x'^2)
    ("derived" form, default).  The printed exponent "2+" is read as x'^2 + eps.
  * The form as printed has sum a / x' as the second numerator term ("printed").
  * "var_ratio" mode takes K from the rescaling identity itself:
    K = sqrt(target_var / (var(x^) + eps)) per (sample, channel).
"""
from __future__ import annotations

import numpy as np


def spatial_mean(x):
    """Per (sample, channel) mean over positions; x [B,C,H,W] -> [B,C,1,1]."""
    return np.asarray(x, dtype=np.float64).mean(axis=(2, 3), keepdims=True)


def apply(x, row, mode: str = "k_table", eps: float = 1e-6):
    """x~ = mu + K (x^ - mu) for one step.  row [C]: K values, or target variances in var_ratio mode."""
    x = np.asarray(x, dtype=np.float64)
    mu = spatial_mean(x)
    row = np.asarray(row, dtype=np.float64).reshape(1, -1, 1, 1)
    if mode == "k_table":
        K = row
    elif mode == "var_ratio":
        var = ((x - mu) ** 2).mean(axis=(2, 3), keepdims=True)
        K = np.sqrt(row / (var + eps))
    else:
        raise ValueError(mode)
    return mu + K * (x - mu)


def fit(x_hat, x_target, eps: float = 1e-6, form: str = "derived"):
    """Closed-form K[C] for one step from x_hat, x_target [Ncal, C, H, W]."""
    xh = np.asarray(x_hat, dtype=np.float64)
    xt = np.asarray(x_target, dtype=np.float64)
    mu = spatial_mean(xh)
    a = xh - mu
    b = xt - mu
    wgt = 1.0 / (xt ** 2 + eps)
    ax = (0, 2, 3)
    den = (a * a).sum(axis=ax) + (a * a * wgt).sum(axis=ax)
    if form == "derived":
        num = (a * b).sum(axis=ax) + (a * b * wgt).sum(axis=ax)
    elif form == "printed":
        num = (a * b).sum(axis=ax) + (a / xt).sum(axis=ax)
    else:
        raise ValueError(form)
    return num / den
