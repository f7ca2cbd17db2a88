"""GPU parity of the decoder-block composition (all matmuls in MXInt; LayerNorm, causal softmax and
ReLU in fp32).  Quantization is discontinuous, so a block cannot be compared end to end against a
CPU run (one fp32 ulp in a LayerNorm output may flip a mantissa downstream); instead every stage of
the GPU run is checked against the oracle applied to the GPU's own input of that stage:
MXInt stages within 1e-5 * S, fp32 glue within a few fp32 ulps."""
import math

import numpy as np
import pytest
import torch

from oracle import block_oracle as blk
from oracle import mx_oracle as orc
from paper_2307_15517_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-5


@pytest.fixture(scope="module")
def mods():
    from paper_2307_15517_b200 import binding, decoder_block
    return binding, decoder_block


def _mx_close(got, ref):
    y_ref, _, S = ref
    err = np.abs(got.astype(np.float64) - y_ref)
    assert (err <= TOL * S + 1e-30).all(), float((err / np.maximum(S, 1e-300)).max())


def _fp_close(got, want, rtol=2e-6, atol=2e-6):
    assert np.allclose(got.astype(np.float64), want, rtol=rtol, atol=atol), float(np.abs(got - want).max())


def test_glue_kernels(mods):
    mxb, _ = mods
    g = torch.Generator().manual_seed(3)
    for rows, cols in ((5, 96), (33, 1000), (7, 4096), (3, 8192)):
        x = torch.randn(rows, cols, generator=g) * 4 + 0.5
        ga, be = torch.randn(cols, generator=g), torch.randn(cols, generator=g)
        y = mxb.mx_layernorm(x.cuda(), ga.cuda(), be.cuda(), 1e-5).cpu().numpy()
        _fp_close(y, blk.layernorm(x.numpy(), ga.numpy(), be.numpy(), 1e-5), rtol=1e-5, atol=1e-5)
    for heads, seq in ((2, 40), (3, 257), (1, 2048)):
        s = torch.randn(heads * seq, seq, generator=g) * 5
        p = mxb.mx_softmax(s.clone().cuda(), 0.3, causal=True, rows_per_batch=seq).cpu().numpy()
        want = blk.softmax_causal(s.numpy(), 0.3, seq)
        _fp_close(p, want, rtol=1e-5, atol=1e-7)
        assert (p[want == 0] == 0).all()
    s = torch.randn(6, 100, generator=g)
    p = mxb.mx_softmax(s.clone().cuda(), 1.0).cpu().numpy()
    z = s.numpy().astype(np.float64)
    e = np.exp(z - z.max(axis=1, keepdims=True))
    _fp_close(p, e / e.sum(axis=1, keepdims=True), rtol=1e-5, atol=1e-7)
    a, b = torch.randn(1003, generator=g), torch.randn(1003, generator=g)
    a[5] = float("nan")
    y = mxb.mx_relu_add(a.cuda(), b.cuda(), relu=True).cpu()
    want = torch.relu(a) + b
    assert torch.equal(torch.isnan(y), torch.isnan(want)) and torch.equal(y[~torch.isnan(y)], want[~torch.isnan(want)])


def test_batched_product_on_head_slices(mods):
    """Q K^T per head from packed [tokens, heads*d] tensors, ragged token count."""
    mxb, _ = mods
    seq, H, d, B, w = 200, 3, 64, 16, 8
    q = synth.student_t_activations(seq, H * d, 1)
    k = synth.outlier_activations(seq, H * d, 2, 3, 30.0)
    fa = mxb.MxFormat(B, w)
    qm, qe = mxb.mx_quantize(q.cuda(), fa)
    km, ke = mxb.mx_quantize(k.cuda(), fa)
    s = torch.full((H * seq, seq), 9.0, device="cuda")
    mxb.mx_gemm_batched(qm, qe, fa, H * d, d, km, ke, fa, H * d, d, seq, seq, d, H, s, seq, seq * seq)
    assert mxb.mx_poll_status() == 0
    ref = blk.attention_scores(q.numpy(), k.numpy(), H, d, B, w)
    got = s.cpu().numpy()
    for h in range(H):
        _mx_close(got[h * seq:(h + 1) * seq], ref[h])


def test_decoder_block_stage_by_stage(mods):
    mxb, db = mods
    cfg = db.BlockConfig(hidden=256, heads=2, head_dim=128, ffn=512)
    seq = 160
    g = torch.Generator().manual_seed(11)
    x = synth.outlier_activations(seq, cfg.hidden, 5, 2, 40.0)
    W = {n: synth.gaussian_weights(o, i, 20 + j) for j, (n, o, i) in enumerate(
        [("wq", 256, 256), ("wk", 256, 256), ("wv", 256, 256), ("wo", 256, 256), ("w1", 512, 256), ("w2", 256, 512)])}
    P = {n: torch.randn(sz, generator=g) * 0.1 for n, sz in
         [("bq", 256), ("bk", 256), ("bv", 256), ("bo", 256), ("b1", 512), ("b2", 256), ("ln1_b", 256), ("ln2_b", 256)]}
    P["ln1_g"] = 1 + 0.1 * torch.randn(256, generator=g)
    P["ln2_g"] = 1 + 0.1 * torch.randn(256, generator=g)
    qw = db.quantize_weights(cfg, {k: v.cuda() for k, v in W.items()})
    keep = {}
    out = db.run(cfg, x.cuda(), qw, {k: v.cuda() for k, v in P.items()}, keep=keep)
    assert mxb.mx_poll_status() == 0
    T = {k: v.cpu().numpy() for k, v in keep.items()}
    Wq = {n: orc.quantize(w.numpy(), cfg.block, cfg.w_wgt)[:2] for n, w in W.items()}
    p = {k: v.numpy() for k, v in P.items()}
    B, wa, ww, H, d = cfg.block, cfg.w_act, cfg.w_wgt, cfg.heads, cfg.head_dim

    _fp_close(T["ln1"], blk.layernorm(x.numpy(), p["ln1_g"], p["ln1_b"], cfg.eps), rtol=1e-5, atol=1e-5)
    for name, wn, bn in (("q", "wq", "bq"), ("k", "wk", "bk"), ("v", "wv", "bv")):
        _mx_close(T[name], blk.linear(T["ln1"], *Wq[wn], B, wa, ww, bias=p[bn]))
    sc = blk.attention_scores(T["q"], T["k"], H, d, B, wa)
    for h in range(H):
        _mx_close(T["scores"][h * seq:(h + 1) * seq], sc[h])
    _fp_close(T["probs"], blk.softmax_causal(T["scores"], 1 / math.sqrt(d), seq), rtol=1e-5, atol=1e-7)
    cx = blk.attention_context(T["probs"], T["v"], H, d, B, wa)
    for h in range(H):
        _mx_close(T["ctx"][:, h * d:(h + 1) * d], cx[h])
    _mx_close(T["attn_out"], blk.linear(T["ctx"], *Wq["wo"], B, wa, ww, bias=p["bo"]))
    assert np.array_equal(T["x1"], T["attn_out"] + x.numpy())
    _fp_close(T["ln2"], blk.layernorm(T["x1"], p["ln2_g"], p["ln2_b"], cfg.eps), rtol=1e-5, atol=1e-5)
    _mx_close(T["ffn_pre"], blk.linear(T["ln2"], *Wq["w1"], B, wa, ww, bias=p["b1"]))
    assert np.array_equal(T["ffn_act"], np.maximum(T["ffn_pre"], 0))
    _mx_close(T["ffn_out"], blk.linear(T["ffn_act"], *Wq["w2"], B, wa, ww, bias=p["b2"]))
    assert np.array_equal(out.cpu().numpy(), T["ffn_out"] + T["x1"])
    assert np.isfinite(out.cpu().numpy()).all()


@pytest.mark.parametrize("fmt", [(16, 8), (32, 4), (16, 6)])
def test_softmax_with_mxint_result(mods, fmt):
    """mx_softmax_q against the oracle's softmax (fp64) quantized by the oracle: every code is a
    rounding of the exact probability up to the fp32 softmax's own error, nearly all codes and
    exponent bytes are the oracle's, and masked positions are exact zeros."""
    mxb, _ = mods
    B, w = fmt
    g = torch.Generator().manual_seed(B + w)
    for heads, seq in ((2, 160), (1, 2048), (3, 96), (1, 4096)):
        s = torch.randn(heads * seq, seq, generator=g) * 5
        want = blk.softmax_causal(s.numpy(), 0.3, seq)
        q, e, _ = orc.quantize(want.astype(np.float32), B, w)
        pm, pe = mxb.mx_softmax_q(s.cuda(), mxb.MxFormat(B, w), 0.3, causal=True, rows_per_batch=seq)
        eg = pe.cpu().numpy()
        qg = orc.unpack(pm.cpu().numpy(), seq, w)
        assert (eg == e).mean() > 0.995 and np.abs(eg.astype(int) - e.astype(int)).max() <= 1
        assert (qg == q).mean() > 0.99
        step = np.repeat(np.ldexp(1.0, eg.astype(np.int64) - 127 - (w - 2)), B, axis=1)
        qmax = 2 ** (w - 1) - 1
        tol = 2e-5 * want + 1e-9                       # fp32 exp and row sum
        free = np.abs(qg) < qmax
        assert (np.abs(qg * step - want)[free] <= (0.5 * step + tol)[free]).all()
        assert (want[~free] >= ((qmax - 0.5) * step - tol)[~free]).all()
        assert (qg[want == 0] == 0).all()
        # the two-step path of the library gives the same codes up to the last-bit differences of its row sums
        p2 = mxb.mx_softmax(s.clone().cuda(), 0.3, causal=True, rows_per_batch=seq)
        pm2, pe2 = mxb.mx_quantize(p2, mxb.MxFormat(B, w))
        assert (pm2 == pm).float().mean().item() > 0.995 and (pe2 == pe).float().mean().item() > 0.999


@pytest.mark.parametrize("heads,head_dim,seq", [(2, 128, 160), (2, 128, 256), (4, 64, 256)])
def test_decoder_block_fused_softmax_matches_staged_run(mods, heads, head_dim, seq):
    """The path the benchmark times (products with fused tails; the fused attention kernel when the sequence is
    a whole number of 128-query tiles, for head dimensions 128 and 64) against the staged run of the same block."""
    mxb, db = mods
    cfg = db.BlockConfig(hidden=256, heads=heads, head_dim=head_dim, ffn=512)
    g = torch.Generator().manual_seed(12)
    x = synth.outlier_activations(seq, cfg.hidden, 6, 2, 40.0).cuda()
    W = {n: synth.gaussian_weights(o, i, 30 + j).cuda() for j, (n, o, i) in enumerate(
        [("wq", 256, 256), ("wk", 256, 256), ("wv", 256, 256), ("wo", 256, 256), ("w1", 512, 256), ("w2", 256, 512)])}
    P = {n: (torch.randn(sz, generator=g) * 0.1).cuda() for n, sz in
         [("bq", 256), ("bk", 256), ("bv", 256), ("bo", 256), ("b1", 512), ("b2", 256), ("ln1_b", 256), ("ln2_b", 256)]}
    P["ln1_g"] = torch.ones(256, device="cuda")
    P["ln2_g"] = torch.ones(256, device="cuda")
    qw = db.quantize_weights(cfg, W)
    staged = db.run(cfg, x, qw, P, keep={}).cpu().numpy()
    fused = db.run(cfg, x, qw, P).cpu().numpy()
    assert mxb.mx_poll_status() == 0
    assert np.abs(fused - staged).max() <= 2e-3 * np.abs(staged).max()
