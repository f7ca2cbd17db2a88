"""Full-size parity of the decoder block (Fig. 1(d)) at OPT-6.7B shapes -- hidden 4096, 32 heads of
128, FFN 16384, sequence 2048 -- in the launch configuration bench.py times, and of the batched
tensor-core kernel when every CTA walks several tiles of several batch items.

A block cannot be compared end to end with a CPU run (quantization is discontinuous), so every
stage of ONE GPU run is checked against the oracle applied to the GPU's own input of that stage:
MXInt products on sampled outputs within 1e-5 * S, the transposing quantizer bit for bit on sampled
rows, the fp32 glue within a few fp32 ulps."""
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


def _close(got, ref, S, what):
    err = np.abs(np.asarray(got, np.float64) - np.asarray(ref, np.float64))
    assert (err <= TOL * S + 1e-30).all(), "%s: max |d|/S = %.3e" % (what, float((err / np.maximum(S, 1e-300)).max()))


@pytest.mark.parametrize("case", [
    # batch, M, N, K, B, w : tiles per launch
    (80, 384, 512, 64, 16, 8),      # 480 tiles of 128x256 over 148 CTAs: three to four tiles of different items per CTA
    (100, 300, 100, 96, 32, 8),     # 300 tiles of 128x128, ragged M and N, K tail
    (40, 130, 260, 256, 16, 4),     # nibble operands, 4 K steps, 160 tiles
])
def test_batched_product_many_tiles_per_cta(mods, case):
    """Every output of every item against the oracle: the persistent loop with more than one tile
    per CTA and more than one batch item (item-major tile numbering, rank-3 tensor maps).  The block
    exponents differ from row to row and from item to item but not along K inside an item, so every
    partial sum is an integer below 2^24 times one power of two: any order of accumulation gives the
    exactly summed result and the comparison is bit for bit -- a tile, item or row taken from the
    wrong place cannot hide inside a tolerance."""
    mxb, _ = mods
    batch, M, N, K, B, w = case
    qmax = 2 ** (w - 1) - 1
    nb = K // B
    assert K * qmax * qmax < 2 ** 24
    qa = synth.random_ints((M, batch * K), -qmax, qmax, 900 + batch).numpy()
    qw = synth.random_ints((N, batch * K), -qmax, qmax, 901 + batch).numpy()
    ea = np.repeat(synth.random_bytes((M, batch), 121, 133, 902 + batch).numpy(), nb, axis=1)
    ew = np.repeat(synth.random_bytes((N, batch), 115, 127, 903 + batch).numpy(), nb, axis=1)
    f = mxb.MxFormat(B, w)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    y = torch.full((batch * M, N), 5.0, device="cuda")
    mxb.mx_gemm_batched(dev(orc.pack(qa, w)), dev(ea), f, batch * K, K, dev(orc.pack(qw, w)), dev(ew), f,
                        batch * K, K, M, N, K, batch, y, N, M * N)
    assert mxb.mx_poll_status() == 0
    got = y.cpu().numpy()
    for b in range(batch):
        y_ref, y_seq, S = orc.gemm(qa[:, b * K:(b + 1) * K], ea[:, b * nb:(b + 1) * nb], w,
                                   qw[:, b * K:(b + 1) * K], ew[:, b * nb:(b + 1) * nb], w, B)
        assert np.array_equal(y_ref, y_seq)                 # order-independent by construction
        assert np.array_equal(got[b * M:(b + 1) * M], y_ref), "item %d" % b


def test_batched_product_exponents_varying_along_k(mods):
    """The same launch shape with block exponents that also change along K (within 2^+-1 per operand,
    as the rows of attention operands do): every output within 1e-5 * S."""
    mxb, _ = mods
    batch, M, N, K, B, w = 48, 300, 260, 128, 16, 8
    qmax = 2 ** (w - 1) - 1
    nb = K // B
    qa = synth.random_ints((M, batch * K), -qmax, qmax, 910).numpy()
    qw = synth.random_ints((N, batch * K), -qmax, qmax, 911).numpy()
    ea = synth.random_bytes((M, batch * nb), 126, 128, 912).numpy()
    ew = synth.random_bytes((N, batch * nb), 120, 122, 913).numpy()
    f = mxb.MxFormat(B, w)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    y = torch.full((batch * M, N), 5.0, device="cuda")
    mxb.mx_gemm_batched(dev(orc.pack(qa, w)), dev(ea), f, batch * K, K, dev(orc.pack(qw, w)), dev(ew), f,
                        batch * K, K, M, N, K, batch, y, N, M * N)
    assert mxb.mx_poll_status() == 0
    got = y.cpu().numpy()
    for b in range(batch):
        y_ref, _, S = orc.gemm(qa[:, b * K:(b + 1) * K], ea[:, b * nb:(b + 1) * nb], w,
                               qw[:, b * K:(b + 1) * K], ew[:, b * nb:(b + 1) * nb], w, B)
        _close(got[b * M:(b + 1) * M], y_ref, S, "item %d" % b)


def _sampled_linear(rng, x_gpu_np, w_cpu, bias, B, wa, ww, got, what, n=768):
    """got[i, j] against the oracle's product of the quantized rows of x (the GPU's own stage input)
    and the quantized weights, at n random positions."""
    qa, ea, _ = orc.quantize(np.ascontiguousarray(x_gpu_np, np.float32), B, wa)
    qw, ew, _ = orc.quantize(w_cpu, B, ww)
    M, N = got.shape
    si, sj = rng.integers(0, M, n), rng.integers(0, N, n)
    y_ref, _, S = orc.gemm_samples(qa, ea, wa, qw, ew, ww, B, si, sj, bias=bias)
    _close(got[si, sj], y_ref, S, what)


def test_decoder_block_opt67b_shapes_stage_by_stage(mods):
    mxb, db = mods
    sh = synth.decoder_block_shapes()
    cfg = db.BlockConfig(hidden=sh["hidden"], heads=sh["heads"], head_dim=sh["head_dim"], ffn=sh["ffn"],
                         block=sh["block"], w_act=sh["w_act"], w_wgt=sh["w_wgt"])
    seq, hid, ffn, H, d = sh["seq"], cfg.hidden, cfg.ffn, cfg.heads, cfg.head_dim
    B, wa, ww = cfg.block, cfg.w_act, cfg.w_wgt
    assert (hid, H, d, ffn, seq) == (4096, 32, 128, 16384, 2048)
    rng = np.random.default_rng(67)
    g = torch.Generator().manual_seed(67)
    x = synth.outlier_activations(seq, hid, 4, -(-hid * 5 // 1000), 40.0)
    W = {n: synth.gaussian_weights(o, i, 670 + j) for j, (n, o, i) in enumerate(
        [("wq", hid, hid), ("wk", hid, hid), ("wv", hid, hid), ("wo", hid, hid), ("w1", ffn, hid), ("w2", hid, ffn)])}
    P = {n: torch.randn(sz, generator=g) * 0.02 for n, sz in
         [("bq", hid), ("bk", hid), ("bv", hid), ("bo", hid), ("b1", ffn), ("b2", hid), ("ln1_b", hid), ("ln2_b", hid)]}
    P["ln1_g"] = 1 + 0.1 * torch.randn(hid, generator=g)
    P["ln2_g"] = 1 + 0.1 * torch.randn(hid, generator=g)
    qw = db.quantize_weights(cfg, {k: v.cuda() for k, v in W.items()})
    keep = {}
    out = db.run(cfg, x.cuda(), qw, {k: v.cuda() for k, v in P.items()}, keep=keep)
    assert mxb.mx_poll_status() == 0
    p = {k: v.numpy() for k, v in P.items()}
    T = lambda name: keep[name].cpu().numpy()

    # ---- fp32 glue on sampled rows -------------------------------------------------------------
    rows = rng.choice(seq, 48, replace=False)
    ln1 = T("ln1")
    assert np.allclose(ln1[rows], blk.layernorm(x.numpy()[rows], p["ln1_g"], p["ln1_b"], cfg.eps), rtol=1e-5, atol=1e-5)

    # ---- q, k, v: one 12288-wide layer call on row-concatenated weights ---------------------------
    for name, wn, bn in (("q", "wq", "bq"), ("k", "wk", "bk"), ("v", "wv", "bv")):
        _sampled_linear(rng, ln1, W[wn].numpy(), p[bn], B, wa, ww, T(name), name)
    q, k, v = T("q"), T("k"), T("v")

    # ---- scores: all 32 heads, 64 sampled outputs each (batched kernel, 4096 tiles) ---------------
    scores = T("scores")
    for h in range(H):
        qa, ea, _ = orc.quantize(np.ascontiguousarray(q[:, h * d:(h + 1) * d]), B, wa)
        qk, ek, _ = orc.quantize(np.ascontiguousarray(k[:, h * d:(h + 1) * d]), B, wa)
        si, sj = rng.integers(0, seq, 64), rng.integers(0, seq, 64)
        y_ref, _, S = orc.gemm_samples(qa, ea, wa, qk, ek, wa, B, si, sj)
        _close(scores[h * seq + si, sj], y_ref, S, "scores head %d" % h)

    # ---- causal softmax: three whole heads --------------------------------------------------------
    probs = T("probs")
    for h in (0, 13, H - 1):
        want = blk.softmax_causal(scores[h * seq:(h + 1) * seq], 1 / math.sqrt(d), seq)
        got = probs[h * seq:(h + 1) * seq]
        assert np.allclose(got, want, rtol=1e-5, atol=1e-7), "softmax head %d" % h
        assert (got[want == 0] == 0).all()

    # ---- V quantized along the token axis (transposing quantizer at 4096 x 2048): sampled rows ----
    fa = mxb.MxFormat(B, wa)
    vm, ve = mxb.mx_quantize(keep["v"].t(), fa)
    vrows = rng.choice(hid, 64, replace=False)
    qv, ev, _ = orc.quantize(np.ascontiguousarray(v.T[vrows]), B, wa)
    assert np.array_equal(vm.cpu().numpy()[vrows], orc.pack(qv, wa))
    assert np.array_equal(ve.cpu().numpy()[vrows], ev)

    # ---- context: per head 16 rows of P against all 128 columns of V ------------------------------
    ctx = T("ctx")
    for h in range(H):
        prow = rng.choice(seq, 16, replace=False)
        qa, ea, _ = orc.quantize(np.ascontiguousarray(probs[h * seq + prow]), B, wa)
        qv, ev, _ = orc.quantize(np.ascontiguousarray(v[:, h * d:(h + 1) * d].T), B, wa)
        y_ref, _, S = orc.gemm(qa, ea, wa, qv, ev, wa, B)
        _close(ctx[prow][:, h * d:(h + 1) * d], y_ref, S, "ctx head %d" % h)

    # ---- out projection, residual, second LayerNorm, FFN ------------------------------------------
    attn_out = T("attn_out")
    _sampled_linear(rng, ctx, W["wo"].numpy(), p["bo"], B, wa, ww, attn_out, "attn_out")
    x1 = T("x1")
    assert np.array_equal(x1, attn_out + x.numpy())
    ln2 = T("ln2")
    assert np.allclose(ln2[rows], blk.layernorm(x1[rows], p["ln2_g"], p["ln2_b"], cfg.eps), rtol=1e-5, atol=1e-5)
    ffn_pre = T("ffn_pre")
    _sampled_linear(rng, ln2, W["w1"].numpy(), p["b1"], B, wa, ww, ffn_pre, "ffn_pre")
    ffn_act = T("ffn_act")
    assert np.array_equal(ffn_act, np.maximum(ffn_pre, 0))
    ffn_out = T("ffn_out")
    _sampled_linear(rng, ffn_act, W["w2"].numpy(), p["b2"], B, wa, ww, ffn_out, "ffn_out")
    res = out.cpu().numpy()
    assert np.array_equal(res, ffn_out + x1)
    assert np.isfinite(res).all()


def test_fused_attention_opt67b_shapes(mods):
    """The fused attention kernel at 32 heads x 128, sequence 2048 (512 work items over 148 CTAs, up to 16 key
    tiles per item): on sampled query rows of every fourth head, the probabilities it quantized against the
    oracle's softmax of the oracle's scores, and the context against the oracle's product of the kernel's own
    probability codes with the oracle-quantized V."""
    mxb, _ = mods
    H, seq, d, B, w = 32, 2048, 128, 16, 8
    hid = H * d
    q = synth.student_t_activations(seq, hid, 31)
    k = synth.outlier_activations(seq, hid, 32, 20, 20.0)
    v = synth.student_t_activations(seq, hid, 33)
    fa = mxb.MxFormat(B, w)
    qm, qe = mxb.mx_quantize(q.cuda(), fa)
    km, ke = mxb.mx_quantize(k.cuda(), fa)
    vm, ve = mxb.mx_quantize(v.cuda().t(), fa)
    scale = 1.0 / math.sqrt(d)
    ctx, pm, pe = mxb.mx_attention(qm, qe, km, ke, fa, vm, ve, fa, seq, H, d, scale, fa, causal=True, return_p=True)
    assert mxb.mx_poll_status() == 0
    ctx2 = mxb.mx_attention(qm, qe, km, ke, fa, vm, ve, fa, seq, H, d, scale, fa, causal=True)
    assert torch.equal(ctx, ctx2)                                  # the optional output changes nothing
    ctx = ctx.cpu().numpy()
    rng = np.random.default_rng(3)
    qn, kn, vn = q.numpy(), k.numpy(), v.numpy()
    for h in range(0, H, 4):
        rows = np.sort(rng.choice(seq, 24, replace=False))
        rows[0], rows[-1] = 0, seq - 1
        qa, ea, _ = orc.quantize(np.ascontiguousarray(qn[rows, h * d:(h + 1) * d]), B, w)
        qk, ek, _ = orc.quantize(np.ascontiguousarray(kn[:, h * d:(h + 1) * d]), B, w)
        s_ref, _, _ = orc.gemm(qa, ea, w, qk, ek, w, B)             # [24, seq]
        z = s_ref.astype(np.float64) * scale
        mask = np.arange(seq)[None, :] <= rows[:, None]
        z = np.where(mask, z, -np.inf)
        e = np.where(mask, np.exp(z - z.max(axis=1, keepdims=True)), 0.0)
        want = e / e.sum(axis=1, keepdims=True)
        q_or, e_or, _ = orc.quantize(want.astype(np.float32), B, w)
        sel = torch.from_numpy(h * seq + rows).cuda()
        eg = pe[sel].cpu().numpy()
        qg = orc.unpack(pm[sel].cpu().numpy(), seq, w)
        assert (eg == e_or).mean() > 0.99 and np.abs(eg.astype(int) - e_or.astype(int)).max() <= 1
        assert (qg == q_or).mean() > 0.98
        step = np.repeat(np.ldexp(1.0, eg.astype(np.int64) - 127 - (w - 2)), B, axis=1)
        tol = 3e-5 * want + 1e-9
        free = np.abs(qg) < 127
        assert (np.abs(qg * step - want)[free] <= (0.5 * step + tol)[free]).all()
        assert (qg[~mask] == 0).all()
        qv, ev, _ = orc.quantize(np.ascontiguousarray(vn[:, h * d:(h + 1) * d].T), B, w)
        y_ref, _, S = orc.gemm(qg, eg, w, qv, ev, w, B)
        _close(ctx[rows][:, h * d:(h + 1) * d], y_ref, S, "ctx head %d" % h)


def test_fused_tails_opt67b_shapes(mods):
    """The three products of the block's second half as the timed path runs them -- output projection with the
    residual, FFN-up with bias, ReLU and an MXInt8 result, FFN-down from that result with bias and residual -- at
    2048 x 4096 / 16384, each on sampled outputs against the oracle fed with the GPU's own inputs of that stage."""
    mxb, _ = mods
    seq, hid, ffn, B, wa, ww = 2048, 4096, 16384, 16, 8, 4
    fa, fw = mxb.MxFormat(B, wa), mxb.MxFormat(B, ww)
    rng = np.random.default_rng(9)
    ctx = synth.student_t_activations(seq, hid, 91)
    x = synth.outlier_activations(seq, hid, 92, 20, 40.0)
    W = {n: synth.gaussian_weights(o, i, 93 + j) for j, (n, o, i) in enumerate([("wo", hid, hid), ("w1", ffn, hid), ("w2", hid, ffn)])}
    g = torch.Generator().manual_seed(94)
    bo, b1, b2 = (torch.randn(n, generator=g) * 0.05 for n in (hid, ffn, hid))
    q = {n: mxb.mx_quantize(w.cuda(), fw) for n, w in W.items()}
    qo = {n: orc.quantize(w.numpy(), B, ww)[:2] for n, w in W.items()}
    n = 640

    # output projection + bias + residual
    x1 = mxb.mx_linear_fused(ctx.cuda(), fa, q["wo"][0], q["wo"][1], fw, hid, bias=bo.cuda(), residual=x.cuda())
    qa, ea, _ = orc.quantize(ctx.numpy(), B, wa)
    si, sj = rng.integers(0, seq, n), rng.integers(0, hid, n)
    y_ref, _, S = orc.gemm_samples(qa, ea, wa, qo["wo"][0], qo["wo"][1], ww, B, si, sj, bias=bo.numpy())
    res = x.numpy()[si, sj].astype(np.float64)
    _close(x1.cpu().numpy()[si, sj], y_ref.astype(np.float64) + res, S + np.abs(res) + np.abs(bo.numpy()[sj]), "out-proj + residual")

    # FFN-up + bias + ReLU, MXInt8 result: codes must be a correct rounding of the oracle's values
    h2 = synth.student_t_activations(seq, hid, 95)
    fm, fe = mxb.mx_linear_fused(h2.cuda(), fa, q["w1"][0], q["w1"][1], fw, ffn, bias=b1.cuda(), relu=True, fy=fa)
    assert mxb.mx_poll_status() == 0
    qa, ea, _ = orc.quantize(h2.numpy(), B, wa)
    rows = np.sort(rng.choice(seq, 6, replace=False))
    cols = np.arange(0, ffn, 16)[rng.choice(ffn // 16, 96, replace=False)]
    fe_n, fm_n = fe.cpu().numpy(), fm.cpu().numpy()
    for r in rows:
        sj = (cols[:, None] + np.arange(16)[None, :]).ravel()               # whole output blocks of 16
        si = np.full_like(sj, r)
        y_ref, _, S = orc.gemm_samples(qa, ea, wa, qo["w1"][0], qo["w1"][1], ww, B, si, sj, bias=b1.numpy())
        want = np.maximum(y_ref.astype(np.float64), 0.0).reshape(-1, 16)
        tol = (TOL * (S + np.abs(b1.numpy()[sj]))).reshape(-1, 16)
        eg = fe_n[r, cols // 16].astype(np.int64)
        codes = fm_n[r].view(np.int8)[sj].reshape(-1, 16).astype(np.float64)
        e_lo = np.where(np.maximum(want - tol, 0).max(axis=1) > 0, np.frexp(np.maximum(want - tol, 0).max(axis=1))[1] - 1 + 127, 0)
        e_hi = np.maximum(np.frexp((want + tol).max(axis=1))[1] - 1 + 127, 0)
        assert ((eg >= e_lo) & (eg <= e_hi)).all()
        step = np.ldexp(1.0, eg - 127 - (wa - 2))[:, None]
        free = np.abs(codes) < 127
        assert (np.abs(codes * step - want)[free] <= (0.5 * step + tol)[free]).all()
        assert (codes >= 0).all()

    # FFN-down from the kernel's own MXInt8 result + bias + residual
    o = mxb.mx_gemm_fused(fm, fe, fa, q["w2"][0], q["w2"][1], fw, seq, hid, ffn, bias=b2.cuda(), residual=x1)
    assert mxb.mx_poll_status() == 0
    qf = fm_n.view(np.int8)
    si, sj = rng.integers(0, seq, n), rng.integers(0, hid, n)
    y_ref, _, S = orc.gemm_samples(qf, fe_n, wa, qo["w2"][0], qo["w2"][1], ww, B, si, sj, bias=b2.numpy())
    res = x1.cpu().numpy()[si, sj].astype(np.float64)
    _close(o.cpu().numpy()[si, sj], y_ref.astype(np.float64) + res, S + np.abs(res) + np.abs(b2.numpy()[sj]), "FFN-down + residual")
