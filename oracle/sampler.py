"""Cached sampling loop: schedule, guidance, DDIM update, VC.  Test infrastructure.

Cache rule (Background, "Quantization and Cache"): with cache interval N the
features of all layers are computed and cached at the first step; at step t
with t mod N == 0 the model recomputes and refreshes the cache, and the next
N-1 steps reuse it.  Readings: t counts sampling steps i = 0, 1, ... from the
noise end; the schedule is global (all blocks together); what is cached is the
output of each block's self-attention branch and MLP branch ("store and reuse
outputs from self-attention and MLP layers") before the adaLN gate, which is
re-applied with the current step's conditioning.

Sampler: deterministic DDIM (eta = 0) over a 1000-step linear-beta schedule
(1e-4 .. 2e-2) with evenly spaced timesteps t_i = (S-1-i) * (1000 // S); after
the last step alpha_bar_prev = 1.  Classifier-free guidance evaluates the
network on [conditional; unconditional (label = num_classes)] and combines
eps = eps_u + g * (eps_c - eps_u) on the C noise channels.  VC (module vc) is
applied to the latent after every update.

The stochastic sampler of the Experimental Settings ("DDPM") is available as kind="ddpm": the ancestral step of
the cited DDPM / improved-DDPM papers on the same timestep subset, with the betas re-derived for the subset
(beta'_k = 1 - ab_k / ab_{k-1}), the mean from the predicted noise and the variance interpolated in the log
domain between beta'_k and the posterior variance by the network's second output group (the "learned sigma"
channels), v in [-1, 1].  The Gaussian noise of every step is an INPUT ([S, B, C, H, W]), so that both
implementations see the same numbers.  Readings: under guidance v is taken from the conditional half; no
clipping of the predicted x0.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

from . import dit, vc

TRAIN_STEPS = 1000


def should_refresh(step_index: int, interval: int) -> bool:
    """True when the cache is recomputed at sampling step `step_index` (0-based)."""
    if interval < 1:
        raise ValueError("cache interval must be >= 1")
    return step_index % interval == 0


def ddim_table(num_steps: int):
    """Per sampling step i: (t_i, sqrt(ab_t), sqrt(1-ab_t), sqrt(ab_prev), sqrt(1-ab_prev)), float64."""
    betas = np.linspace(1e-4, 2e-2, TRAIN_STEPS, dtype=np.float64)
    ab = np.cumprod(1.0 - betas)
    stride = TRAIN_STEPS // num_steps
    ts = [(num_steps - 1 - i) * stride for i in range(num_steps)]
    rows = []
    for i, t in enumerate(ts):
        ab_t = ab[t]
        ab_p = ab[ts[i + 1]] if i + 1 < num_steps else 1.0
        rows.append((t, np.sqrt(ab_t), np.sqrt(1 - ab_t), np.sqrt(ab_p), np.sqrt(1 - ab_p)))
    return rows


def ddpm_table(num_steps: int):
    """Per sampling step i (t descending): (t_i, 1/sqrt(ab), sqrt(1/ab - 1), coef_x0, coef_xt, log beta',
    log posterior variance (clipped at the last step), noise factor 0/1), float64, betas re-derived for the subset."""
    if num_steps < 2:
        raise ValueError("the stochastic sampler needs at least two steps")
    betas = np.linspace(1e-4, 2e-2, TRAIN_STEPS, dtype=np.float64)
    ab_full = np.cumprod(1.0 - betas)
    stride = TRAIN_STEPS // num_steps
    ts = np.array([k * stride for k in range(num_steps)])          # ascending
    ab = ab_full[ts]
    ab_prev = np.concatenate([[1.0], ab[:-1]])
    beta = 1.0 - ab / ab_prev
    post_var = beta * (1.0 - ab_prev) / (1.0 - ab)
    log_post = np.log(np.concatenate([post_var[1:2], post_var[1:]]))
    coef_x0 = beta * np.sqrt(ab_prev) / (1.0 - ab)
    coef_xt = (1.0 - ab_prev) * np.sqrt(1.0 - beta) / (1.0 - ab)
    rows = []
    for i in range(num_steps):
        k = num_steps - 1 - i
        rows.append((int(ts[k]), 1.0 / np.sqrt(ab[k]), np.sqrt(1.0 / ab[k] - 1.0), coef_x0[k], coef_xt[k],
                     np.log(beta[k]), log_post[k], 1.0 if k > 0 else 0.0))
    return rows


def ddpm_update(x, eps, v, row, noise):
    """x_prev = mean + [k > 0] exp(0.5 logvar) noise;  x0 = x/sqrt(ab) - sqrt(1/ab - 1) eps,
    mean = coef_x0 x0 + coef_xt x,  logvar = f log beta' + (1 - f) log beta~,  f = (v + 1)/2."""
    _, sr, srm1, c0, ct, lb, lp, nz = row
    x0 = sr * x - srm1 * eps
    mean = c0 * x0 + ct * x
    f = (np.asarray(v, dtype=np.float64) + 1.0) / 2.0
    logvar = f * lb + (1.0 - f) * lp
    return mean + nz * np.exp(0.5 * logvar) * np.asarray(noise, dtype=np.float64)


def cfg_combine(eps_both, guidance: float):
    """eps_both [2B,C,...] = [cond; uncond] -> eps_u + g*(eps_c - eps_u)  [B,C,...]."""
    B = eps_both.shape[0] // 2
    e_c, e_u = eps_both[:B], eps_both[B:]
    return e_u + guidance * (e_c - e_u)


def ddim_update(x, eps, row):
    """x_prev = sqrt(ab_prev) * x0 + sqrt(1-ab_prev) * eps with x0 = (x - sqrt(1-ab_t) eps)/sqrt(ab_t)."""
    _, sa, s1a, sap, s1ap = row
    x0 = (x - s1a * eps) / sa
    return sap * x0 + s1ap * eps


@dataclass
class SamplerConfig:
    num_steps: int
    cache_interval: int = 1
    guidance: Optional[float] = None      # None: no classifier-free guidance
    vc_table: Optional[np.ndarray] = None  # K[S,C]; None: no VC
    vc_mode: str = "k_table"               # or "var_ratio" (table = target variances)
    vc_eps: float = 1e-6
    use_cache: bool = True                 # False: plain un-cached loop (every step computes, nothing stored)
    kind: str = "ddim"                     # or "ddpm": stochastic ancestral step with learned variance
    noise: Optional[np.ndarray] = None     # ddpm: standard-normal noise [S, B, C, Hl, Wl]
    schedule: Optional[np.ndarray] = None  # [S, blocks, 2] booleans: per step, block and branch, True = reuse the
                                           # cached output (replaces the global rule "i mod N == 0 refreshes")


def sample(model: dit.QModel, ctx: dit.Context, scfg: SamplerConfig, latent, labels, on_step=None):
    """Run the whole trajectory; returns the final latent [B,C,Hl,Wl] (float64; float32-valued after each step)."""
    x = np.asarray(latent, dtype=np.float64)
    B, C = x.shape[0], model.cfg.channels
    labels = np.asarray(labels, dtype=np.int64)
    if scfg.kind not in ("ddim", "ddpm"):
        raise ValueError(scfg.kind)
    table = ddim_table(scfg.num_steps) if scfg.kind == "ddim" else ddpm_table(scfg.num_steps)
    cache = {} if scfg.use_cache else None
    for i, row in enumerate(table):
        t = np.full(B, row[0], dtype=np.float64)
        if scfg.guidance is not None:
            xin = np.concatenate([x, x], axis=0)
            tin = np.concatenate([t, t])
            yin = np.concatenate([labels, np.full(B, model.cfg.num_classes, dtype=np.int64)])
        else:
            xin, tin, yin = x, t, labels
        reuse = scfg.use_cache and not should_refresh(i, scfg.cache_interval)
        mask = None
        if scfg.use_cache and scfg.schedule is not None:
            mask = np.asarray(scfg.schedule, dtype=bool)[i]
            reuse = bool(mask.all())
        out = dit.forward(model, ctx, xin, tin, yin, cache=cache, reuse=reuse, mask=mask)
        eps = out[:, :C]
        v = out[:B, C:2 * C]                # learned-variance channels (of the conditional half under guidance)
        if scfg.guidance is not None:
            eps = cfg_combine(eps, scfg.guidance)
        if scfg.kind == "ddim":
            x = ddim_update(x, eps, row)
        else:
            x = ddpm_update(x, eps, v, row, scfg.noise[i])
        if scfg.vc_table is not None:
            x = vc.apply(x, scfg.vc_table[i], mode=scfg.vc_mode, eps=scfg.vc_eps)
        x = dit.store(x, "f32")            # the latent lives in float32 between steps
        if on_step is not None:
            on_step(i, x, reuse)
    return x
