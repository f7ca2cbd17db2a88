"""One pre-LayerNorm transformer decoder block with every matmul in MXInt (the block of the paper's
Fig. 1(d): linears, Q K^T and P V quantized; LayerNorm, softmax and ReLU in fp32).

This module only sequences calls of the C ABI (through ``binding``): every arithmetic step runs in
the library's kernels.  ``run`` returns the block output and, on request, every intermediate
tensor so that each stage can be checked against the oracle on identical inputs.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, Optional

import torch

from . import binding as mxb


@dataclass
class BlockConfig:
    hidden: int
    heads: int
    head_dim: int
    ffn: int
    block: int = 16
    w_act: int = 8           # activations and both attention operands
    w_wgt: int = 4           # weights of the linears
    eps: float = 1e-5


def quantize_weights(cfg: BlockConfig, weights: Dict[str, torch.Tensor]):
    """weights: fp32 CUDA tensors wq, wk, wv, wo [hidden, hidden], w1 [ffn, hidden], w2 [hidden, ffn].
    The three projections of the block input are stored as one [3 * hidden, hidden] matrix (rows of wq, then
    wk, then wv): one layer call then quantizes the input once and produces q, k and v side by side."""
    fw = mxb.MxFormat(cfg.block, cfg.w_wgt)
    out = {k: mxb.mx_quantize(v, fw) for k, v in weights.items() if k not in ("wq", "wk", "wv")}
    parts = [mxb.mx_quantize(weights[k], fw) for k in ("wq", "wk", "wv")]      # rows are quantized independently
    out["wqkv"] = (torch.cat([p[0] for p in parts]), torch.cat([p[1] for p in parts]))
    return out


def prepare_params(params: Dict[str, torch.Tensor]) -> Dict[str, torch.Tensor]:
    """Adds the concatenated bias of the fused q/k/v projection."""
    out = dict(params)
    out["bqkv"] = torch.cat([params["bq"], params["bk"], params["bv"]])
    return out


def run(cfg: BlockConfig, x: torch.Tensor, qweights, params: Dict[str, torch.Tensor],
        keep: Optional[dict] = None) -> torch.Tensor:
    """x: [seq, hidden] fp32 CUDA.  params: ln1_g, ln1_b, ln2_g, ln2_b, bq, bk, bv, bo, b1, b2."""
    seq, hid, H, d = x.shape[0], cfg.hidden, cfg.heads, cfg.head_dim
    assert hid == H * d
    fa, fw = mxb.MxFormat(cfg.block, cfg.w_act), mxb.MxFormat(cfg.block, cfg.w_wgt)

    def rec(name, t):
        if keep is not None:
            keep[name] = t
        return t
    rec.keep = keep

    def linear(inp, name, bias, n_out):
        wm, we = qweights[name]
        return mxb.mx_linear(inp, fa, wm, we, fw, n_out, bias=bias)

    if "bqkv" not in params:
        params = prepare_params(params)
    fused_path = keep is None and d in (64, 128) and seq % 32 == 0
    if fused_path:
        # LayerNorm runs inside the projection's operand pass: the normalised tensor is never stored
        wm, we = qweights["wqkv"]
        qkv = mxb.mx_linear_fused(x, fa, wm, we, fw, 3 * hid, bias=params["bqkv"],
                                  layernorm=(params["ln1_g"], params["ln1_b"], cfg.eps))
    else:
        h1 = rec("ln1", mxb.mx_layernorm(x, params["ln1_g"], params["ln1_b"], cfg.eps))
        qkv = linear(h1, "wqkv", params["bqkv"], 3 * hid)       # [seq, 3 * hidden]: q | k | v
    q, k, v = rec("q", qkv[:, :hid]), rec("k", qkv[:, hid:2 * hid]), rec("v", qkv[:, 2 * hid:])
    if fused_path:
        # q, k, v quantized straight to the operand form, then scores, causal softmax, quantized probabilities and
        # context in one kernel: nothing of size seq x seq and no packed copy of q, k, v is stored
        ctx = mxb.mx_attention_fp(q, k, v, fa, fa, H, d, 1.0 / math.sqrt(d), fa, causal=True)
        return _after_attention(cfg, x, ctx, qweights, params, linear, rec)
    # attention scores per head: both operands MXInt, blocks along the head dimension
    qm, qe = mxb.mx_quantize(q, fa)
    km, ke = mxb.mx_quantize(k, fa)
    s = torch.empty((H * seq, seq), dtype=torch.float32, device=x.device)
    mxb.mx_gemm_batched(qm, qe, fa, hid, d, km, ke, fa, hid, d, seq, seq, d, H, s, seq, seq * seq)
    rec("scores", s.clone() if keep is not None else s)
    # context per head: probabilities and values MXInt, blocks along the key/token axis
    if keep is None:
        # softmax and quantization in one pass: the fp32 probabilities are never written
        pm, pe = mxb.mx_softmax_q(s, fa, 1.0 / math.sqrt(d), causal=True, rows_per_batch=seq)
    else:
        p = rec("probs", mxb.mx_softmax(s, 1.0 / math.sqrt(d), causal=True, rows_per_batch=seq))
        pm, pe = mxb.mx_quantize(p, fa)
    vm, ve = mxb.mx_quantize(v.t(), fa)                      # [hidden, seq]: blocks along tokens
    ctx = torch.empty((seq, hid), dtype=torch.float32, device=x.device)
    mxb.mx_gemm_batched(pm, pe, fa, seq, seq * seq, vm, ve, fa, seq, d * seq, seq, d, seq, H, ctx, hid, d)
    rec("ctx", ctx)
    return _after_attention(cfg, x, ctx, qweights, params, linear, rec)


def _after_attention(cfg, x, ctx, qweights, params, linear, rec):
    """Output projection, skip connections and the feed-forward half of the block."""
    hid = cfg.hidden
    fa, fw = mxb.MxFormat(cfg.block, cfg.w_act), mxb.MxFormat(cfg.block, cfg.w_wgt)
    if rec.keep is None:
        # bias, ReLU and the skip connections run in the products' epilogues; the feed-forward activation
        # leaves its product already quantized (the next product's operand), so no fp32 tensor of width ffn exists
        wm, we = qweights["wo"]
        x1 = mxb.mx_linear_fused(ctx, fa, wm, we, fw, hid, bias=params["bo"], residual=x)
        wm, we = qweights["w1"]
        fm, fe = mxb.mx_linear_fused(x1, fa, wm, we, fw, cfg.ffn, bias=params["b1"], relu=True, fy=fa,
                                     layernorm=(params["ln2_g"], params["ln2_b"], cfg.eps))
        wm, we = qweights["w2"]
        return mxb.mx_gemm_fused(fm, fe, fa, wm, we, fw, x.shape[0], hid, cfg.ffn, bias=params["b2"], residual=x1)
    a = rec("attn_out", linear(ctx, "wo", params["bo"], hid))
    x1 = rec("x1", mxb.mx_relu_add(a, x))
    h2 = rec("ln2", mxb.mx_layernorm(x1, params["ln2_g"], params["ln2_b"], cfg.eps))
    f = rec("ffn_pre", linear(h2, "w1", params["b1"], cfg.ffn))
    f = rec("ffn_act", mxb.mx_relu_add(f, None, relu=True))
    o = rec("ffn_out", linear(f, "w2", params["b2"], hid))
    return rec("x2", mxb.mx_relu_add(o, x1))


def flops(cfg: BlockConfig, seq: int) -> float:
    """2*M*N*K of the eight MXInt matmuls of one block."""
    hid, H, d = cfg.hidden, cfg.heads, cfg.head_dim
    lin = 2.0 * seq * (4 * hid * hid + 2 * hid * cfg.ffn)
    att = 2.0 * H * (seq * seq * d) * 2
    return lin + att
