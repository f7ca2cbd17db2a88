"""CPU oracle for the fp32 glue of a decoder block and for the per-head MXInt attention matmuls.

TEST INFRASTRUCTURE ONLY (see mx_oracle.py).  The glue operators are their textbook definitions
written out in numpy float64 (the paper keeps LayerNorm, softmax and the activation in floating
point around the MX operators, Fig. 1(d)); the matmuls go through the C oracle.  Pins:
tests/test_oracle_pins.py checks these against scipy / torch float64 library routines and
against the invariants of the definitions.
"""
from __future__ import annotations

import numpy as np

from . import mx_oracle as orc


def layernorm(x, gamma, beta, eps):
    x = np.asarray(x, np.float64)
    mean = x.mean(axis=1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=1, keepdims=True)           # biased variance
    y = (x - mean) / np.sqrt(var + eps)
    if gamma is not None:
        y = y * np.asarray(gamma, np.float64)
    if beta is not None:
        y = y + np.asarray(beta, np.float64)
    return y


def softmax_causal(s, scale, rows_per_batch):
    """Row r attends to columns j <= r % rows_per_batch; masked entries are 0."""
    s = np.asarray(s, np.float64) * scale
    rows, cols = s.shape
    limit = (np.arange(rows) % rows_per_batch)[:, None]
    mask = np.arange(cols)[None, :] <= limit
    z = np.where(mask, s, -np.inf)
    z = z - z.max(axis=1, keepdims=True)
    e = np.where(mask, np.exp(z), 0.0)
    return e / e.sum(axis=1, keepdims=True)


def relu(x):
    return np.maximum(np.asarray(x, np.float64), 0.0)


def linear(x, w_q, w_e, block, wa, ww, bias=None):
    """MXInt linear on fp32 input x: quantize x, block-scaled product with quantized weights."""
    qa, ea, _ = orc.quantize(np.ascontiguousarray(x, np.float32), block, wa)
    return orc.gemm(qa, ea, wa, w_q, w_e, ww, block, bias=bias)        # (y_ref, y_seq, S)


def attention_scores(q, k, heads, d, block, w):
    """Per head h: S_h = Q_h K_h^T with both operands quantized along the head dimension."""
    out = []
    for h in range(heads):
        qa, ea, _ = orc.quantize(np.ascontiguousarray(q[:, h * d:(h + 1) * d], np.float32), block, w)
        qk, ek, _ = orc.quantize(np.ascontiguousarray(k[:, h * d:(h + 1) * d], np.float32), block, w)
        out.append(orc.gemm(qa, ea, w, qk, ek, w, block))
    return out


def attention_context(p, v, heads, d, block, w):
    """Per head h: O_h = P_h V_h with both operands quantized along the key/token axis."""
    seq = v.shape[0]
    out = []
    for h in range(heads):
        ph = np.ascontiguousarray(p[h * seq:(h + 1) * seq], np.float32)
        qa, ea, _ = orc.quantize(ph, block, w)
        qv, ev, _ = orc.quantize(np.asarray(v[:, h * d:(h + 1) * d], np.float32).T, block, w)   # strided view
        out.append(orc.gemm(qa, ea, w, qv, ev, w, block))
    return out
