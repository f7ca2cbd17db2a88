"""GPU parity of the fused attention kernel (scores, causal softmax, MXInt probabilities and context in one
launch).  Quantization is discontinuous, so the check is stage by stage on ONE run: the probabilities the
kernel quantized (optional output) against the oracle's softmax of the oracle's scores -- every code a
correct rounding of the exact probability up to the fp32 softmax's own error, nearly all codes and exponent
bytes the oracle's, masked positions exact zeros -- and the context against the oracle's product of the
kernel's OWN probability codes with the oracle-quantized V, within 1e-5 * S."""
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
def mxb():
    from paper_2307_15517_b200 import binding
    return binding


@pytest.mark.parametrize("d", [128, 64])
@pytest.mark.parametrize("case", [(2, 256, 16, 8, True), (3, 384, 32, 8, True), (1, 512, 16, 4, True), (2, 256, 16, 8, False),
                                  (1, 128, 32, 3, True), (5, 640, 16, 6, False),    # one tile only; five key tiles, no mask
                                  (2, 160, 16, 8, True), (2, 416, 32, 8, False), (3, 32, 16, 8, True)])   # ragged last tiles
def test_fused_attention_stage_by_stage(mxb, case, d):
    H, seq, B, wp, causal = case
    w = 8
    hid = H * d
    q = synth.student_t_activations(seq, hid, 21)
    k = synth.outlier_activations(seq, hid, 22, 3, 20.0)
    v = synth.student_t_activations(seq, hid, 23)
    fa, fp = mxb.MxFormat(B, w), mxb.MxFormat(B, wp)
    qm, qe = mxb.mx_quantize(q.cuda(), fa)
    km, ke = mxb.mx_quantize(k.cuda(), fa)
    vm, ve = mxb.mx_quantize(v.cuda().t(), fa)                  # [hid, seq]: blocks along the tokens
    scale = 1.0 / math.sqrt(d)
    ctx, pm, pe = mxb.mx_attention(qm, qe, km, ke, fa, vm, ve, fa, seq, H, d, scale, fp, causal=causal, return_p=True)
    assert mxb.mx_poll_status() == 0
    ctx, pm, pe = ctx.cpu().numpy(), pm.cpu().numpy(), pe.cpu().numpy()
    sc = blk.attention_scores(q.numpy(), k.numpy(), H, d, B, w)
    qmax = 2 ** (wp - 1) - 1
    for h in range(H):
        s_ref = sc[h][0].astype(np.float64)
        if causal:
            want = blk.softmax_causal(s_ref, scale, seq)
        else:
            z = s_ref * scale
            e = np.exp(z - z.max(axis=1, keepdims=True))
            want = e / e.sum(axis=1, keepdims=True)
        q_or, e_or, _ = orc.quantize(want.astype(np.float32), B, wp)
        eg = pe[h * seq:(h + 1) * seq]
        qg = orc.unpack(pm[h * seq:(h + 1) * seq], seq, wp)
        assert (eg == e_or).mean() > 0.99 and np.abs(eg.astype(int) - e_or.astype(int)).max() <= 1
        assert (qg == q_or).mean() > 0.98
        step = np.repeat(np.ldexp(1.0, eg.astype(np.int64) - 127 - (wp - 2)), B, axis=1)
        tol = 3e-5 * want + 1e-9                          # fp32 exp, row sum and the scores' own tolerance
        free = np.abs(qg) < qmax
        assert (np.abs(qg * step - want)[free] <= (0.5 * step + tol)[free]).all()
        assert (want[~free] >= ((qmax - 0.5) * step - tol)[~free]).all()
        assert (qg[want == 0] == 0).all()
        # context from the kernel's own probability codes
        qv, ev, _ = orc.quantize(np.ascontiguousarray(v.numpy()[:, h * d:(h + 1) * d].T), B, w)
        y_ref, _, S = orc.gemm(qg, eg, wp, qv, ev, w, B)
        err = np.abs(ctx[:, h * d:(h + 1) * d].astype(np.float64) - y_ref)
        assert (err <= TOL * S + 1e-30).all(), (h, float((err / np.maximum(S, 1e-300)).max()))


def test_fused_attention_refuses_what_it_cannot_tile(mxb):
    f = mxb.MxFormat(16, 8)
    z = lambda r, c: torch.zeros((r, c), dtype=torch.uint8, device="cuda")
    for seq, H, d, status in ((200, 2, 128, -2), (256, 2, 96, -2)):       # 200 % 32 != 0; head dimension 96
        with pytest.raises(mxb.MxError) as e:
            mxb.mx_attention(z(seq, H * d), z(seq, H * d // 16), z(seq, H * d), z(seq, H * d // 16), f, z(H * d, seq),
                             z(H * d, seq // 16), f, seq, H, d, 0.1, f, workspace=mxb.alloc_workspace(1 << 22))
        assert e.value.status == status


@pytest.mark.parametrize("d", [128, 64])
@pytest.mark.parametrize("case", [(2, 256, 16, torch.float32), (3, 384, 32, torch.bfloat16), (2, 224, 16, torch.float32)])
def test_attention_on_floating_point_operands_equals_quantize_then_attention(mxb, case, d):
    """mx_attention_fp quantizes q, k (along the head dimension) and v (along the tokens) on the fly; its
    context must equal, bit for bit, mx_attention on the operands quantized by mx_quantize (which the
    quantizer tests tie to the oracle), also when q, k, v are column slices of one wider tensor."""
    H, seq, B, dtype = case
    hid = H * d
    qkv = torch.cat([synth.student_t_activations(seq, hid, 41), synth.outlier_activations(seq, hid, 42, 3, 20.0),
                     synth.student_t_activations(seq, hid, 43)], dim=1).to(dtype).cuda()
    q, k, v = qkv[:, :hid], qkv[:, hid:2 * hid], qkv[:, 2 * hid:]
    fa, fp = mxb.MxFormat(B, 8), mxb.MxFormat(B, 8)
    scale = 1.0 / math.sqrt(d)
    got = mxb.mx_attention_fp(q, k, v, fa, fa, H, d, scale, fp, causal=True)
    qm, qe = mxb.mx_quantize(q, fa)
    km, ke = mxb.mx_quantize(k, fa)
    vm, ve = mxb.mx_quantize(v.t(), fa)
    want = mxb.mx_attention(qm, qe, km, ke, fa, vm, ve, fa, seq, H, d, scale, fp, causal=True)
    assert mxb.mx_poll_status() == 0
    assert torch.equal(got, want)
