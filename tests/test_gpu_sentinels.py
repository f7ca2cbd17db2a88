"""Nothing is written outside a result: every output tensor of these calls is a view into a larger buffer
filled with a sentinel value, on shapes with ragged tails, and the frame must survive the call.  (Stands in for a
bounds-checking build: a store that strays by a few elements lands in the frame.)"""
import math

import numpy as np
import pytest
import torch

from oracle import mx_oracle as orc
from paper_2307_15517_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mxb():
    from paper_2307_15517_b200 import binding
    return binding


def _framed(rows, cols, dtype, pad_rows=4, pad_cols=16, fill=0x5A):
    """(view [rows, cols], check): the view sits at the top-left of a larger buffer filled with `fill`."""
    big = torch.full((rows + pad_rows, cols + pad_cols), fill, dtype=dtype, device="cuda")
    view = big[:rows, :cols]

    def intact():
        return bool((big[rows:, :] == fill).all()) and bool((big[:, cols:] == fill).all())
    return view, intact


@pytest.mark.parametrize("case", [(37, 272, 16, 4), (130, 96, 32, 8), (64, 1040, 16, 3)])
def test_quantizer_and_decoder_outputs_stay_inside(mxb, case):
    rows, K, B, w = case
    f = mxb.MxFormat(B, w)
    x = synth.student_t_activations(rows, K, rows + K).cuda()
    mcols = K // 2 if w <= 4 else K
    # the library wants dense rows for the packed outputs: frame them with extra rows only
    mant_big = torch.full((rows + 3, mcols), 0x5A, dtype=torch.uint8, device="cuda")
    exp_big = torch.full((rows + 3, K // B), 0x5A, dtype=torch.uint8, device="cuda")
    mxb.mx_quantize(x, f, mant_out=mant_big[:rows], exp_out=exp_big[:rows])
    assert mxb.mx_poll_status() == 0
    assert (mant_big[rows:] == 0x5A).all() and (exp_big[rows:] == 0x5A).all()
    q, e, _ = orc.quantize(x.cpu().numpy(), B, w)
    assert np.array_equal(mant_big[:rows].cpu().numpy(), orc.pack(q, w)) and np.array_equal(exp_big[:rows].cpu().numpy(), e)
    # transposed view: blocks along the slow axis (rows of the result = columns of xt)
    if K % 32 == 0 and rows % B == 0:
        mt_big = torch.full((K + 3, rows // 2 if w <= 4 else rows), 0x5A, dtype=torch.uint8, device="cuda")
        et_big = torch.full((K + 3, rows // B), 0x5A, dtype=torch.uint8, device="cuda")
        mxb.mx_quantize(x.t(), f, mant_out=mt_big[:K], exp_out=et_big[:K])
        assert (mt_big[K:] == 0x5A).all() and (et_big[K:] == 0x5A).all()
    # decode into a padded fp32 view
    out, intact = _framed(rows, K, torch.float32, fill=-3.0)
    mxb.mx_dequantize(mant_big[:rows], exp_big[:rows], K, f, out=out)
    assert intact()
    assert np.array_equal(out.cpu().numpy().astype(np.float64), orc.dequantize(q, e, B, w))


@pytest.mark.parametrize("case", [(300, 528, 320, 16), (129, 48, 96, 16), (2100, 2336, 128, 16)])
def test_mxint_result_stays_inside(mxb, case):
    M, N, K, By = case
    fa, fw, fy = mxb.MxFormat(16, 8), mxb.MxFormat(16, 4), mxb.MxFormat(By, 8)
    x = synth.student_t_activations(M, K, M).cuda()
    wm, we = mxb.mx_quantize(synth.gaussian_weights(N, K, N).cuda(), fw)
    ym_big = torch.full((M + 5, N), 0x5A, dtype=torch.uint8, device="cuda")
    ye_big = torch.full((M + 5, N // By), 0x5A, dtype=torch.uint8, device="cuda")
    mxb.mx_linear_q(x, fa, wm, we, fw, N, fy, y_mant=ym_big[:M], y_exp=ye_big[:M])
    assert mxb.mx_poll_status() == 0
    assert (ym_big[M:] == 0x5A).all() and (ye_big[M:] == 0x5A).all()
    assert (ye_big[:M] != 0x5A).any()


@pytest.mark.parametrize("T", [1, 4, 16])
def test_streamed_decode_result_stays_inside(mxb, T):
    K, N = 512, 1000                                   # ragged last 16-row tile
    fa, fw = mxb.MxFormat(32, 8), mxb.MxFormat(32, 4)
    layers, checks = [], []
    for i in range(5):
        y, intact = _framed(T, N, torch.float32, pad_rows=2, pad_cols=8, fill=-3.0)
        wm, we = mxb.mx_quantize(synth.gaussian_weights(N, K, 10 + i).cuda(), fw)
        layers.append(dict(x=synth.student_t_activations(T, K, 20 + i).cuda(), fa=fa, w_mant=wm, w_exp=we, fw=fw, N=N, y=y))
        checks.append(intact)
    mxb.mx_linear_grouped(mxb.make_linear_args(layers))
    assert mxb.mx_poll_status() == 0
    assert all(c() for c in checks)
    assert all(bool((L["y"] != -3.0).any()) for L in layers)


@pytest.mark.parametrize("seq,d", [(256, 128), (160, 128), (96, 64)])      # whole and ragged query tiles
def test_attention_context_stays_inside(mxb, seq, d):
    H = 2
    hid = H * d
    fa = mxb.MxFormat(16, 8)
    q, k, v = (synth.student_t_activations(seq, hid, s).cuda() for s in (1, 2, 3))
    fill = -3.1234567                                  # not on any MXInt8 grid (row 0 of the context is a row of V as quantized)
    ctx, intact = _framed(seq, hid, torch.float32, fill=fill)
    mxb.mx_attention_fp(q, k, v, fa, fa, H, d, 1.0 / math.sqrt(d), fa, causal=True, ctx=ctx)
    assert mxb.mx_poll_status() == 0
    assert intact() and bool((ctx != fill).all())
