"""Activation-range collection on a calibration batch.  Test infrastructure.

"Using a calibration dataset and equations (2) and (3), we can derive the
statistical information for s and z" (text after Eq. 3).  How the calibration
SET is chosen (the paper's TAP clustering) is outside this package; here the
set is given.  Procedure: run the network over the calibration inputs with
every activation quantizer in "dynamic" mode (each takes the range of its own
input, so later layers see the quantization of earlier ones), record the
largest |x| seen at every quantized linear's input, and turn it into static
symmetric parameters s = absmax / 127, z = 0.
"""
from __future__ import annotations

import numpy as np

from . import dit
from .quant import qparams_symmetric


class _AbsmaxCollector:
    def __init__(self):
        self.absmax = {}

    def __call__(self, name, arr):
        if name.endswith(".absmax"):
            key = name[: -len(".absmax")]
            self.absmax[key] = max(self.absmax.get(key, 0.0), float(arr))


def _scales_from(absmax: dict, depth: int) -> dit.ActScales:
    ada = max(absmax[f"blk{i}.ada"] for i in range(depth))
    blocks = [{n: qparams_symmetric(absmax[f"blk{i}.{n}"]) for n in ("qkv", "proj", "fc1", "fc2")}
              for i in range(depth)]
    return dit.ActScales(qparams_symmetric(ada), blocks)


def calibrate_block(blk: dit.QBlock, batches, tokens: int, heads: int, storage=None) -> dit.ActScales:
    """batches: iterable of (x [M,D], c [B,D]) calibration inputs of one block."""
    col = _AbsmaxCollector()
    ctx = dit.Context(quant="dynamic", storage=storage or dit.Storage(), tap=col)
    for x, c in batches:
        dit.block_forward(ctx, blk, dit.store(x, ctx.storage.resid), c, tokens, heads, 0)
    return _scales_from(col.absmax, 1)


def calibrate_model(model: dit.QModel, batches, storage=None) -> dit.ActScales:
    """batches: iterable of (latent [B,C,Hl,Wl], t [B], y [B]) calibration inputs."""
    col = _AbsmaxCollector()
    ctx = dit.Context(quant="dynamic", storage=storage or dit.Storage(), tap=col)
    for latent, t, y in batches:
        dit.forward(model, ctx, np.asarray(latent, dtype=np.float64), t, y)
    return _scales_from(col.absmax, len(model.blocks))
