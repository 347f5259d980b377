"""The DiT network the quantized linears sit in.  Test infrastructure.

The paper evaluates on class-conditional DiT-XL/2 (Experimental Settings) and
quantizes its linear layers to 8 bits (Table 1) without restating the
architecture; the block below is the adaLN-Zero DiT block of the cited DiT
paper, with these readings:

  * quantized layers: the block's modulation linear, QKV, attention projection,
    MLP fc1 and fc2.  Patch embedding, timestep/label embedders and the final
    layer stay in floating point.
  * modulation chunks in the order shift_msa, scale_msa, gate_msa, shift_mlp,
    scale_mlp, gate_mlp; QKV output laid out [3, heads, head_dim].
  * LayerNorm without affine parameters, eps 1e-6, biased variance.
  * GELU in its tanh form.
  * attention is not quantized; softmax(q k^T / sqrt(head_dim)) v.
  * storage formats are part of the function: the residual stream, Q/K/V and the
    cached branch outputs may be declared bfloat16 (`Storage`), in which case
    the value is rounded (nearest-even) at exactly that point; "exact" keeps
    float64.

Every function takes and returns float64 arrays unless it says otherwise.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Optional

import numpy as np

from .quant import F32, QParams, qparams_symmetric, quantize, quantize_weight_per_channel
from .linear import w8a8_linear

LN_EPS = 1e-6
LINEARS = ("ada", "qkv", "proj", "fc1", "fc2")


# ----------------------------------------------------------------------------- storage formats
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even), returned as float64."""
    f = np.ascontiguousarray(np.asarray(x, dtype=F32))
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    return r.astype(np.uint32).view(F32).astype(np.float64).reshape(np.shape(x))


@dataclass(frozen=True)
class Storage:
    resid: str = "bf16"   # residual stream between sub-layers
    qkv: str = "bf16"     # attention operands
    cache: str = "bf16"   # cached branch outputs

    @staticmethod
    def exact() -> "Storage":
        return Storage("exact", "exact", "exact")


def store(x: np.ndarray, fmt: str) -> np.ndarray:
    if fmt == "exact":
        return np.asarray(x, dtype=np.float64)
    if fmt == "bf16":
        return round_bf16(x)
    if fmt == "f32":
        return np.asarray(x, dtype=F32).astype(np.float64)
    raise ValueError(fmt)


# ----------------------------------------------------------------------------- elementary layers
def silu(x):
    return x / (1.0 + np.exp(-x))


def gelu_tanh(x):
    return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * (x * x * x))))


def layer_norm_modulate(x, shift, scale, tokens: int, eps: float = LN_EPS):
    """Row-wise LayerNorm (no affine) then y*(1+scale[b]) + shift[b], b = row // tokens."""
    x = np.asarray(x, dtype=np.float64)
    mu = x.mean(axis=1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=1, keepdims=True)
    y = (x - mu) / np.sqrt(var + eps)
    b = np.arange(x.shape[0]) // tokens
    return y * (1.0 + np.asarray(scale, dtype=np.float64)[b]) + np.asarray(shift, dtype=np.float64)[b]


def attention(q, k, v, scale: Optional[float] = None):
    """q,k,v [B,T,H,dh] -> [B,T,H,dh]; non-causal softmax attention."""
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    if scale is None:
        scale = 1.0 / np.sqrt(q.shape[-1])
    qh, kh, vh = (a.transpose(0, 2, 1, 3) for a in (q, k, v))    # [B,H,T,dh]
    s = (qh @ kh.transpose(0, 1, 3, 2)) * scale                  # [B,H,T,T] scores (library matrix product per head)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    return (p @ vh).transpose(0, 2, 1, 3)


# ----------------------------------------------------------------------------- quantized model
@dataclass
class QLinear:
    q: np.ndarray        # int8 codes [N,K]
    scale: np.ndarray    # float32 [N]
    colsum: np.ndarray   # int64 [N]
    bias: np.ndarray     # float32 [N]
    w: np.ndarray        # original float32 weights (un-quantized mode only)


def make_qlinear(w, b, bits: int = 8) -> QLinear:
    q, s, cs = quantize_weight_per_channel(w, bits)
    return QLinear(q.astype(np.int8), s, cs, np.asarray(b, dtype=F32), np.asarray(w, dtype=F32))


@dataclass
class QBlock:
    ada: QLinear
    qkv: QLinear
    proj: QLinear
    fc1: QLinear
    fc2: QLinear


def make_qblock(bw: dict, bits: int = 8) -> QBlock:
    return QBlock(*(make_qlinear(bw["w_" + n], bw["b_" + n], bits) for n in LINEARS))


@dataclass
class ActScales:
    """Static tensor-wise activation parameters: one for the shared modulation
    input SiLU(c), and per block one for each of the other four linears' inputs."""
    ada: QParams
    blocks: list  # list of dict name -> QParams for "qkv", "proj", "fc1", "fc2"


@dataclass
class Context:
    """How the forward treats quantizers, plus optional hooks.

    quant: "off" (float weights and activations), "static" (ActScales given),
           "dynamic" (each activation quantizer takes s = max|x| / 127 of its own input).
    tap:   called as tap(name, array) on named intermediates.
    """
    quant: str = "static"
    scales: Optional[ActScales] = None
    storage: Storage = field(default_factory=Storage)
    tap: Optional[Callable] = None
    reuse_walk: bool = False   # a fully skipped step walked block by block (each cached branch enters the residual
                               # stream with its own rounding, as in a computed step) instead of accumulated once

    def emit(self, name, arr):
        if self.tap is not None:
            self.tap(name, arr)


def _qlinear_apply(ctx: Context, lin: QLinear, x, qp: Optional[QParams], name: str):
    """One linear layer on a float input under the context's quantization mode."""
    ctx.emit(name + ".in", x)
    if ctx.quant == "off":
        return np.asarray(x, dtype=np.float64) @ lin.w.astype(np.float64).T + lin.bias.astype(np.float64)
    if ctx.quant == "dynamic":
        qp = qparams_symmetric(float(np.max(np.abs(np.asarray(x).astype(F32)))))
        ctx.emit(name + ".absmax", np.float64(qp.scale) * qp.qmax)
    qa = quantize(x, qp)
    ctx.emit(name + ".qa", qa)
    return w8a8_linear(qa, qp, _codes_f64(lin), lin.scale, lin.colsum, lin.bias)


def _codes_f64(lin: QLinear) -> np.ndarray:
    """The weight codes as the float64 array the integer product takes (same integers; converted once per layer
    instead of once per call)."""
    c = getattr(lin, "_q64", None)
    if c is None:
        c = np.asarray(lin.q, dtype=np.float64)
        lin._q64 = c
    return c


def modulation(ctx: Context, blk: QBlock, c, index: int):
    """mod[b,:] = Lin_ada(SiLU(c[b])) -> six [B,D] chunks."""
    qp = ctx.scales.ada if ctx.quant == "static" else None
    mod = _qlinear_apply(ctx, blk.ada, silu(np.asarray(c, dtype=np.float64)), qp, f"blk{index}.ada")
    ctx.emit(f"blk{index}.mod", mod)
    return np.split(mod, 6, axis=1)


def attn_branch(ctx: Context, blk: QBlock, x, shift, scale, tokens: int, heads: int, index: int):
    """LN-modulate -> QKV -> attention -> projection; returns the pre-gate branch output."""
    aq = ctx.scales.blocks[index] if ctx.quant == "static" else {}
    M, D = x.shape
    B, dh = M // tokens, D // heads
    h = layer_norm_modulate(x, shift, scale, tokens)
    qkv = _qlinear_apply(ctx, blk.qkv, h, aq.get("qkv"), f"blk{index}.qkv")
    qkv = store(qkv, ctx.storage.qkv)
    ctx.emit(f"blk{index}.qkv.out", qkv)
    qkv = qkv.reshape(B, tokens, 3, heads, dh)
    a = attention(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2]).reshape(M, D)
    ctx.emit(f"blk{index}.attn.out", a)
    return _qlinear_apply(ctx, blk.proj, a, aq.get("proj"), f"blk{index}.proj")


def mlp_branch(ctx: Context, blk: QBlock, x, shift, scale, tokens: int, index: int):
    """LN-modulate -> fc1 -> GELU -> fc2; returns the pre-gate branch output."""
    aq = ctx.scales.blocks[index] if ctx.quant == "static" else {}
    h = layer_norm_modulate(x, shift, scale, tokens)
    u = _qlinear_apply(ctx, blk.fc1, h, aq.get("fc1"), f"blk{index}.fc1")
    g = gelu_tanh(u)
    return _qlinear_apply(ctx, blk.fc2, g, aq.get("fc2"), f"blk{index}.fc2")


def gated_residual(ctx: Context, x, gate, branch, tokens: int):
    """x + gate[b] * branch, stored in the residual format."""
    b = np.arange(x.shape[0]) // tokens
    return store(x + np.asarray(gate, dtype=np.float64)[b] * branch, ctx.storage.resid)


def block_forward(ctx: Context, blk: QBlock, x, c, tokens: int, heads: int, index: int = 0, cache=None,
                  reuse_attn: bool = False, reuse_mlp: bool = False):
    """One DiT block.  If `cache` is a dict, the pre-gate branch outputs are written
    to cache[(index, "attn")] and cache[(index, "mlp")] in the cache storage format.
    reuse_attn / reuse_mlp (per-block, per-branch cache schedules): the branch is not evaluated; its cached
    output enters the residual under the current step's gate, and the cache entry is left as it is."""
    sh_a, sc_a, g_a, sh_m, sc_m, g_m = modulation(ctx, blk, c, index)
    if reuse_attn:
        A = cache[(index, "attn")]
    else:
        A = attn_branch(ctx, blk, x, sh_a, sc_a, tokens, heads, index)
        ctx.emit(f"blk{index}.attn_branch", A)
        if cache is not None:
            cache[(index, "attn")] = store(A, ctx.storage.cache)
    x = gated_residual(ctx, x, g_a, A, tokens)
    ctx.emit(f"blk{index}.x_mid", x)
    if reuse_mlp:
        Mo = cache[(index, "mlp")]
    else:
        Mo = mlp_branch(ctx, blk, x, sh_m, sc_m, tokens, index)
        ctx.emit(f"blk{index}.mlp_branch", Mo)
        if cache is not None:
            cache[(index, "mlp")] = store(Mo, ctx.storage.cache)
    x = gated_residual(ctx, x, g_m, Mo, tokens)
    ctx.emit(f"blk{index}.x_out", x)
    return x


def blocks_reuse(ctx: Context, blocks, x, c, tokens: int, cache: dict):
    """A fully skipped step: no LayerNorm, attention or MLP is evaluated; every block
    adds its cached branch outputs under the CURRENT step's gates,
        x_out = x + sum_b (gate_msa_b * A_b + gate_mlp_b * Mo_b),
    accumulated exactly and stored once."""
    b = np.arange(x.shape[0]) // tokens
    acc = np.asarray(x, dtype=np.float64).copy()
    for i, blk in enumerate(blocks):
        _, _, g_a, _, _, g_m = modulation(ctx, blk, c, i)
        acc += g_a[b] * cache[(i, "attn")] + g_m[b] * cache[(i, "mlp")]
    return store(acc, ctx.storage.resid)


# ----------------------------------------------------------------------------- whole network
@dataclass
class QModel:
    cfg: object            # synth.DiTConfig-like: hidden, heads, grid, patch, channels, freq_dim ...
    blocks: list
    w: dict                # float parameters of the un-quantized layers


def make_qmodel(cfg, weights: dict, weight_bits: int = 8) -> QModel:
    """weight_bits = 4 gives the W4A8 setting of Table 2 (4-bit channel-wise weights, 8-bit activations)."""
    fl = {k: np.asarray(v, dtype=np.float64) for k, v in weights.items() if k != "blocks"}
    return QModel(cfg, [make_qblock(bw, weight_bits) for bw in weights["blocks"]], fl)


def timestep_features(t, dim: int):
    """Sinusoidal features [B, dim]: cos then sin of t * 10000^(-j/(dim/2))."""
    half = dim // 2
    freqs = np.exp(-np.log(10000.0) * np.arange(half, dtype=np.float64) / half)
    a = np.asarray(t, dtype=np.float64)[:, None] * freqs[None, :]
    return np.concatenate([np.cos(a), np.sin(a)], axis=1)


def conditioning(model: QModel, t, y):
    """c = MLP(sinusoid(t)) + label_table[y]   (float layers)."""
    w = model.w
    h = timestep_features(t, model.cfg.freq_dim) @ w["w_t1"].T + w["b_t1"]
    h = silu(h) @ w["w_t2"].T + w["b_t2"]
    return h + w["y_table"][np.asarray(y, dtype=np.int64)]


def patchify(cfg, latent):
    """[B,C,Hl,Wl] -> [B*T, p*p*C]; patch vector ordered (c, py, px)."""
    B, C, Hl, Wl = latent.shape
    p, g = cfg.patch, cfg.grid
    x = np.asarray(latent, dtype=np.float64).reshape(B, C, g, p, g, p)
    x = x.transpose(0, 2, 4, 1, 3, 5)            # B, gy, gx, C, py, px
    return x.reshape(B * g * g, C * p * p)


def unpatchify(cfg, tok, B: int):
    """[B*T, p*p*Cout] -> [B,Cout,Hl,Wl]; output vector ordered (py, px, c)."""
    p, g = cfg.patch, cfg.grid
    co = tok.shape[1] // (p * p)
    x = tok.reshape(B, g, g, p, p, co).transpose(0, 5, 1, 3, 2, 4)   # B, c, gy, py, gx, px
    return x.reshape(B, co, g * p, g * p)


def embed(model: QModel, ctx: Context, latent):
    w = model.w
    B = latent.shape[0]
    x = patchify(model.cfg, latent) @ w["w_patch"].T + w["b_patch"] + np.tile(w["pos"], (B, 1))
    return store(x, ctx.storage.resid)


def final_layer(model: QModel, x, c, B: int):
    w = model.w
    mod = silu(c) @ w["w_ada_f"].T + w["b_ada_f"]
    shift, scale = np.split(mod, 2, axis=1)
    h = layer_norm_modulate(x, shift, scale, model.cfg.tokens)
    return unpatchify(model.cfg, h @ w["w_out"].T + w["b_out"], B)


def forward(model: QModel, ctx: Context, latent, t, y, cache=None, reuse: bool = False, mask=None):
    """One network evaluation -> [B, 2C, Hl, Wl] (noise prediction in the first C channels).

    reuse=False: every block is computed (and written to `cache` if given).
    reuse=True : every block is skipped and served from `cache`.
    mask       : optional [blocks, 2] booleans (attention branch, MLP branch), True = serve that branch from the
                 cache.  All True is the fully skipped step above, all False the refresh step; a mixed mask walks
                 the blocks in order, each reused branch entering the residual like a computed one.
    """
    if mask is not None:
        mask = np.asarray(mask, dtype=bool).reshape(len(model.blocks), 2)
        reuse = bool(mask.all())
        if reuse or not mask.any():
            mask = None
    cfg = model.cfg
    B = latent.shape[0]
    x = embed(model, ctx, latent)
    c = conditioning(model, t, y)
    ctx.emit("c", c)
    ctx.emit("x_embed", x)
    if reuse and ctx.reuse_walk:
        # the cache rule taken literally, block by block: the same sum as blocks_reuse, rounded after every branch
        for i, blk in enumerate(model.blocks):
            x = block_forward(ctx, blk, x, c, cfg.tokens, cfg.heads, i, cache, True, True)
    elif reuse:
        x = blocks_reuse(ctx, model.blocks, x, c, cfg.tokens, cache)
    else:
        for i, blk in enumerate(model.blocks):
            ra, rm = (bool(mask[i, 0]), bool(mask[i, 1])) if mask is not None else (False, False)
            x = block_forward(ctx, blk, x, c, cfg.tokens, cfg.heads, i, cache, ra, rm)
    ctx.emit("x_final", x)
    return final_layer(model, x, c, B)
