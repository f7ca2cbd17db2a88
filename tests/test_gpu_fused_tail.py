"""GPU parity of the product with a fused element-wise tail (mx_gemm_fused / mx_linear_fused):
out = act(A W^T + bias) + residual, stored as fp32 or quantized to MXInt in the same epilogue.

The oracle side is the oracle's product followed by the tail written out in numpy.  On operands whose
partial sums are exact in fp32 the results must match bit for bit (fp32 values, codes and exponent bytes);
on general operands the fp32 result lies within the product's tolerance."""
import numpy as np
import pytest
import torch

from oracle import mx_oracle as orc
from paper_2307_15517_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-5


@pytest.fixture(scope="module")
def mxb():
    from paper_2307_15517_b200 import binding
    return binding


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _grid_case(M, N, K, B, seed):
    qa = synth.random_ints((M, K), -7, 7, seed).numpy()
    qw = synth.random_ints((N, K), -7, 7, seed + 1).numpy()
    ea = np.full((M, K // B), 129, np.uint8)
    ew = np.full((N, K // B), 124, np.uint8)
    unit = 2.0 ** ((129 - 127 - 2) + (124 - 127 - 2))
    bias = (synth.random_ints((1, N), -1000, 1000, seed + 2).numpy()[0] * unit).astype(np.float32)
    res = (synth.random_ints((M, N), -3000, 3000, seed + 3).numpy() * unit).astype(np.float32)
    return qa, ea, qw, ew, bias, res


def _tail(y_ref_no_bias, bias, relu, res):
    t = y_ref_no_bias.astype(np.float32)
    if bias is not None:
        t = t + bias[None, :]
    if relu:
        t = np.where(t < 0, np.float32(0), t)
    if res is not None:
        t = t + res
    return t.astype(np.float32)


CASES = [
    # M, N, K, B, relu, bias, residual
    (300, 544, 512, 16, True, True, True),
    (300, 544, 512, 16, False, True, True),
    (130, 208, 256, 32, True, False, False),      # ragged last chunk, relu alone
    (2100, 2336, 128, 16, True, True, True),      # more than one wave of 256 x 256 tiles: the CTA-pair kernel
    (2048, 1024, 320, 16, False, False, True),    # wide tiles, several per CTA, residual alone
    (1, 64, 64, 32, True, True, True),
]


@pytest.mark.parametrize("case", CASES)
def test_fused_tail_bit_exact_on_grid_operands(mxb, case):
    M, N, K, B, relu, use_bias, use_res = case
    qa, ea, qw, ew, bias, res = _grid_case(M, N, K, B, seed=M + N + K)
    bias = bias if use_bias else None
    res = res if use_res else None
    y0 = orc.gemm(qa, ea, 4, qw, ew, 4, B)[0]                   # exact here, no rounding anywhere
    want = _tail(y0, bias, relu, res)
    fa = fw = mxb.MxFormat(B, 4)
    am, wm = _dev(orc.pack(qa, 4)), _dev(orc.pack(qw, 4))
    kw = dict(bias=None if bias is None else _dev(bias), relu=relu, residual=None if res is None else _dev(res))
    y = mxb.mx_gemm_fused(am, _dev(ea), fa, wm, _dev(ew), fw, M, N, K, **kw)
    assert mxb.mx_poll_status() == 0
    assert np.array_equal(y.cpu().numpy(), want)
    # MXInt result of the same tail: the quantizer's rule on the fp32 values
    for By, wy in ((16, 8), (32, 4)):
        if N % By:
            continue
        fy = mxb.MxFormat(By, wy)
        ym, ye = mxb.mx_gemm_fused(am, _dev(ea), fa, wm, _dev(ew), fw, M, N, K, fy=fy, **kw)
        assert mxb.mx_poll_status() == 0
        q_or, e_or, _ = orc.quantize(want, By, wy)
        assert np.array_equal(ye.cpu().numpy(), e_or)
        assert np.array_equal(ym.cpu().numpy(), orc.pack(q_or, wy))


def test_linear_fused_equals_unfused_sequence(mxb):
    """The layer entry point on general data: quantize-on-the-fly + product + tail in one call against
    the oracle's quantizer, product and the tail in numpy; then the chain the decoder block uses
    (ReLU + MXInt8 result feeding the next product, residual added there)."""
    M, K, N, N2, B = 384, 512, 1024, 256, 16
    x = synth.student_t_activations(M, K, 31)
    w = synth.gaussian_weights(N, K, 32)
    w2 = synth.gaussian_weights(N2, N, 33)
    bias = torch.randn(N, generator=torch.Generator().manual_seed(34))
    res = torch.randn(M, N2, generator=torch.Generator().manual_seed(35))
    fa, fw = mxb.MxFormat(B, 8), mxb.MxFormat(B, 4)
    wm, we = mxb.mx_quantize(w.cuda(), fw)
    w2m, w2e = mxb.mx_quantize(w2.cuda(), fw)
    y = mxb.mx_linear_fused(x.cuda(), fa, wm, we, fw, N, bias=bias.cuda(), relu=True)
    qa, ea, _ = orc.quantize(x.numpy(), B, 8)
    qw, ew, _ = orc.quantize(w.numpy(), B, 4)
    y_ref, _, S = orc.gemm(qa, ea, 8, qw, ew, 4, B, bias=bias.numpy())
    want = np.where(y_ref < 0, 0, y_ref)
    assert (np.abs(y.cpu().numpy().astype(np.float64) - want) <= TOL * (S + np.abs(bias.numpy())[None, :])).all()
    assert (y.cpu().numpy() >= 0).all()
    # chain: MXInt8 result of the same call, consumed as the packed operand of the next product
    fm, fe = mxb.mx_linear_fused(x.cuda(), fa, wm, we, fw, N, bias=bias.cuda(), relu=True, fy=fa)
    qf, ef, _ = orc.quantize(y.cpu().numpy(), B, 8)             # the kernel's own fp32 values, the oracle's quantizer
    assert np.array_equal(fe.cpu().numpy(), ef) and np.array_equal(fm.cpu().numpy(), orc.pack(qf, 8))
    o = mxb.mx_gemm_fused(fm, fe, fa, w2m, w2e, fw, M, N2, N, residual=res.cuda())
    assert mxb.mx_poll_status() == 0
    q2, e2, _ = orc.quantize(w2.numpy(), B, 4)
    o_ref, _, S2 = orc.gemm(qf, ef, 8, q2, e2, 4, B)
    assert (np.abs(o.cpu().numpy().astype(np.float64) - (o_ref.astype(np.float64) + res.numpy())) <= TOL * (S2 + np.abs(res.numpy()))).all()


def test_fused_tail_argument_checks(mxb):
    import ctypes as C
    M, N, K, B = 64, 64, 64, 16
    f = mxb.MxFormat(B, 4)
    am = torch.zeros((M, K // 2), dtype=torch.uint8, device="cuda")
    ae = torch.full((M, K // B), 127, dtype=torch.uint8, device="cuda")
    y = torch.empty((M, N), dtype=torch.float32, device="cuda")
    ym = torch.empty((M, N), dtype=torch.uint8, device="cuda")
    ye = torch.empty((M, N // B), dtype=torch.uint8, device="cuda")
    ws = mxb.alloc_workspace(mxb.mx_workspace_bytes_ex(M, N, K, f, f, mxb.MX_ALGO_TCGEN05), "cuda")
    call = lambda ep, yp, ymp: mxb.lib.mx_gemm_fused(am.data_ptr(), ae.data_ptr(), f, am.data_ptr(), ae.data_ptr(), f, M, N, K,
                                                     ep, yp, N, mxb.MxFormat(B, 8), ymp, ye.data_ptr(), ws.data_ptr(), ws.numel(), None)
    # status codes: 0 MX_OK, -1 MX_ERR_NULL, -2 MX_ERR_SHAPE
    assert call(None, y.data_ptr(), ym.data_ptr()) == -1        # two results
    assert call(None, None, None) == -1                         # none
    ep = mxb.MxEpilogue()
    ep.residual, ep.ldr = y.data_ptr(), N - 1
    assert call(C.byref(ep), y.data_ptr(), None) == -2
    assert call(None, y.data_ptr(), None) == 0
    assert mxb.mx_poll_status() == 0
    assert torch.count_nonzero(y).item() == 0


@pytest.mark.parametrize("case", [(300, 512, 528, 16, True), (129, 1056, 256, 32, False), (2048, 4096, 1024, 16, True)])
def test_layernorm_in_the_operand_pass_equals_the_separate_kernel(mxb, case):
    """mx_linear_fused with a LayerNorm prologue normalises each row with the arithmetic of mx_layernorm and
    quantizes it straight to the operand: the product must equal mx_layernorm followed by mx_linear bit for bit
    (the staged sequence is checked against the oracle stage by stage elsewhere), also with a poisoned row."""
    M, K, N, B, affine = case
    x = synth.outlier_activations(M, K, 51, 3, 30.0)
    x[M // 2, 5] = float("nan")                                  # one non-finite row: the poison must carry over
    g = torch.Generator().manual_seed(52)
    gamma = (1 + 0.1 * torch.randn(K, generator=g)).cuda() if affine else None
    beta = (0.1 * torch.randn(K, generator=g)).cuda() if affine else None
    bias = torch.randn(N, generator=g).cuda()
    fa, fw = mxb.MxFormat(B, 8), mxb.MxFormat(B, 4)
    wm, we = mxb.mx_quantize(synth.gaussian_weights(N, K, 53).cuda(), fw)
    xd = x.cuda()
    h = mxb.mx_layernorm(xd, gamma, beta, 1e-5)
    want = mxb.mx_linear(h, fa, wm, we, fw, N, bias=bias, algo=mxb.MX_ALGO_TCGEN05)
    got = mxb.mx_linear_fused(xd, fa, wm, we, fw, N, bias=bias, layernorm=(gamma, beta, 1e-5))
    assert mxb.mx_poll_status() == 0
    w_, g_ = want.cpu().numpy(), got.cpu().numpy()
    assert np.array_equal(np.isnan(w_), np.isnan(g_)) and np.isnan(g_[M // 2]).all() and not np.isnan(g_[0]).any()
    assert np.array_equal(w_[~np.isnan(w_)], g_[~np.isnan(g_)])
    # and with the tail and an MXInt8 result, as the decoder block's FFN-up runs it
    qm, qe = mxb.mx_linear_fused(xd, fa, wm, we, fw, N, bias=bias, relu=True, fy=fa, layernorm=(gamma, beta, 1e-5))
    qm2, qe2 = mxb.mx_linear_fused(h, fa, wm, we, fw, N, bias=bias, relu=True, fy=fa)
    assert torch.equal(qm, qm2) and torch.equal(qe, qe2)
