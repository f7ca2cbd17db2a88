"""GPU parity for two-row blocks (the paper's (16,2) block shape): quantizer bit-exact against
the oracle's ``quantize_2d``, products against the oracle's product on the per-row expansion of
the shared exponents."""
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


@pytest.mark.parametrize("B", (16, 32))
@pytest.mark.parametrize("w", (2, 4, 5, 8))
def test_quantize_two_row_blocks_bit_exact(mxb, B, w):
    F = mxb.MxFormat(B, w, 8, 2)
    rng = np.random.default_rng(10 * B + w)
    x = (rng.standard_t(3, (130, 2080)) * np.exp(rng.uniform(-6, 6, (130, 1)))).astype(np.float32)
    x[4, :B] = 0.0
    x[5, :B] = 0.0                                    # an all-zero pair block
    x[6, 40] = np.inf                                 # a non-finite pair block
    x[9, :] = np.ldexp(x[9, :], 110).astype(np.float32)   # near the top: the multiply-based rounding path
    x[10, ::3] = (rng.integers(-7, 8, x[10, ::3].shape) * 0.5).astype(np.float32)   # ties
    for data in (x, x[:2, :64].copy(), np.zeros((0, 64), np.float32)):
        q, e, bad = orc.quantize_2d(data, B, 2, w)
        cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
        mant, exps = mxb.mx_quantize(_dev(data), F, nonfinite_count=cnt)
        assert exps.shape == e.shape and np.array_equal(exps.cpu().numpy(), e)
        assert np.array_equal(mant.cpu().numpy(), orc.pack(q, w))
        assert int(cnt.item()) == bad
        if data.shape[0]:
            want = orc.dequantize(q, orc.expand_exponent_rows(e, 2), B, w)
            for dtype in (torch.float32, torch.bfloat16):
                got = mxb.mx_dequantize(mant, exps, data.shape[1], F, dtype=dtype).float().cpu().numpy()
                ok = ~np.isnan(want)
                assert np.array_equal(np.isnan(got), np.isnan(want))
                assert np.array_equal(got[ok].astype(np.float64), want[ok])
    xb = torch.from_numpy(x).to(torch.bfloat16)
    q, e, _ = orc.quantize_2d(xb.float().numpy(), B, 2, w)
    mant, exps = mxb.mx_quantize(xb.cuda(), F)
    assert np.array_equal(mant.cpu().numpy(), orc.pack(q, w)) and np.array_equal(exps.cpu().numpy(), e)


@pytest.mark.parametrize("case", [(16, 8, 4, 2, 2), (16, 8, 4, 2, 1), (32, 4, 4, 1, 2), (16, 6, 3, 2, 2)])
def test_products_with_two_row_blocks(mxb, case):
    """The paper's layer: activations MXInt((16,2),8,7), weights MXInt((16,2),8,3) -- and the mixed
    cases where only one operand has two-row blocks."""
    B, wa, ww, ra, rw = case
    M, K, N = 300, 1152, 528
    x = synth.student_t_activations(M, K, seed=wa).numpy()
    wt = synth.gaussian_weights(N, K, seed=ww).numpy()
    bias = synth.gaussian_weights(1, N, seed=5, std=1.0)[0].numpy()
    qa, ea, _ = orc.quantize_2d(x, B, ra, wa)
    qw, ew, _ = orc.quantize_2d(wt, B, rw, ww)
    y_ref, y_seq, S = orc.gemm(qa, orc.expand_exponent_rows(ea, ra), wa, qw, orc.expand_exponent_rows(ew, rw), ww, B,
                               bias=bias)
    fa, fw = mxb.MxFormat(B, wa, 8, ra), mxb.MxFormat(B, ww, 8, rw)
    w_mant, w_exp = mxb.mx_quantize(_dev(wt), fw)
    assert np.array_equal(w_exp.cpu().numpy(), ew)
    y = mxb.mx_linear(_dev(x), fa, w_mant, w_exp, fw, N, bias=_dev(bias))
    assert mxb.mx_poll_status() == 0
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
    assert (err <= TOL * S + 1e-37).all()
    a_mant, a_exp = mxb.mx_quantize(_dev(x), fa)
    y2 = mxb.mx_gemm(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias=_dev(bias), algo=mxb.MX_ALGO_TCGEN05)
    assert np.array_equal(y2.cpu().numpy(), y.cpu().numpy())
    y3 = mxb.mx_gemm(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, bias=_dev(bias), algo=mxb.MX_ALGO_SIMT)
    assert np.array_equal(y3.cpu().numpy(), y_seq)
    # the MXInt-result form accepts two-row inputs as well
    qo, eo, _, _, _ = orc.gemm_requant(qa, orc.expand_exponent_rows(ea, ra), wa, qw, orc.expand_exponent_rows(ew, rw),
                                       ww, B, 16, 8, bias=bias)
    ym, ye = mxb.mx_gemm_q(a_mant, a_exp, fa, w_mant, w_exp, fw, M, N, K, mxb.MxFormat(16, 8), bias=_dev(bias))
    assert (ye.cpu().numpy() == eo).mean() > 0.99
    assert (orc.unpack(ym.cpu().numpy(), N, 8) == qo).mean() > 0.99


def test_two_row_blocks_are_refused_where_unsupported(mxb):
    F2 = mxb.MxFormat(32, 4, 8, 2)
    F1 = mxb.MxFormat(32, 4)
    x = torch.randn(4, 256, device="cuda")
    with pytest.raises(mxb.MxError):
        mxb.mx_quantize(torch.randn(3, 64, device="cuda"), mxb.MxFormat(16, 4, 8, 2))      # odd row count
    with pytest.raises(mxb.MxError):
        mxb.mx_quantize(torch.randn(64, 4, device="cuda").t(), mxb.MxFormat(16, 4, 8, 2))  # strided axis
    wm, we = mxb.mx_quantize(torch.randn(64, 256, device="cuda"), F2)
    with pytest.raises(mxb.MxError):
        mxb.mx_linear(x, mxb.MxFormat(32, 8), wm, we, F2, 64, algo=mxb.MX_ALGO_TCGEN05_FUSED)   # in-kernel decode
    with pytest.raises(mxb.MxError):
        mxb.mx_linear(x[:3], mxb.MxFormat(32, 8, 8, 2), wm, we, F2, 64)                          # odd token count
    y = mxb.mx_linear(x, mxb.MxFormat(32, 8), wm, we, F2, 64)
    assert torch.isfinite(y).all() and mxb.mx_poll_status() == 0
    del F1


@pytest.mark.parametrize("case", [(2, 256, 2, 2), (4, 1024, 2, 1), (16, 1024, 1, 2), (16, 512, 2, 2), (1, 256, 1, 2)])
def test_streamed_decode_with_two_row_blocks_is_bit_exact(mxb, case):
    """The decode path (one launch over several layers, weights streamed once) on (32,2) blocks of the
    weights, of the tokens, or of both: integer block sums and ascending fp32 block adds, so the result is
    the oracle's sequential sum bit for bit, as for one-row blocks."""
    T, K, ra, rw = case
    N, B, wa, ww = 4096, 32, 8, 4
    fa, fw = mxb.MxFormat(B, wa, 8, ra), mxb.MxFormat(B, ww, 8, rw)
    layers, want = [], []
    for i in range(6):
        x = synth.student_t_activations(T, K, seed=11 * T + i).numpy()
        wt = synth.gaussian_weights(N, K, seed=50 + i).numpy()
        bias = synth.gaussian_weights(1, N, seed=90 + i, std=1.0)[0].numpy() if i % 2 else None
        qa, ea, _ = orc.quantize_2d(x, B, ra, wa)
        qw, ew, _ = orc.quantize_2d(wt, B, rw, ww)
        want.append(orc.gemm(qa, orc.expand_exponent_rows(ea, ra), wa, qw, orc.expand_exponent_rows(ew, rw), ww, B,
                             bias=bias)[1])
        w_mant, w_exp = mxb.mx_quantize(_dev(wt), fw)
        assert np.array_equal(w_exp.cpu().numpy(), ew)
        layers.append(dict(x=_dev(x), fa=fa, w_mant=w_mant, w_exp=w_exp, fw=fw, N=N,
                           bias=None if bias is None else _dev(bias),
                           y=torch.empty((T, N), dtype=torch.float32, device="cuda")))
    mxb.mx_linear_grouped(mxb.make_linear_args(layers))
    assert mxb.mx_poll_status() == 0
    for L, y_seq in zip(layers, want):
        assert np.array_equal(L["y"].cpu().numpy(), y_seq)
    # one layer through mx_linear: AUTO picks the streaming kernel for these shapes
    L = layers[0]
    y = mxb.mx_linear(L["x"], fa, L["w_mant"], L["w_exp"], fw, N, bias=L["bias"], algo=mxb.MX_ALGO_STREAM)
    assert np.array_equal(y.cpu().numpy(), want[0])


@pytest.mark.parametrize("case", [(300, 544, 512, 16, 16, 4), (130, 208, 256, 32, 16, 8), (2100, 2336, 128, 16, 16, 8),
                                  (2048, 1024, 320, 16, 32, 6)])
def test_result_in_two_row_blocks_bit_exact_where_fp32_is_order_independent(mxb, case):
    """mx_gemm_q with fy = (By, 2): the rows of Y pair up and share exponent bytes.  Operands whose partial
    sums are all exactly representable, so the fp32 product is the oracle's whatever the order, and the
    codes must be the oracle's two-row quantization of it, bit for bit (one-CTA and CTA-pair epilogues)."""
    M, N, K, B, By, wy = case
    qa = synth.random_ints((M, K), -7, 7, M + wy).numpy()
    qw = synth.random_ints((N, K), -7, 7, N + wy).numpy()
    ea = np.full((M, K // B), 129, np.uint8)
    ew = np.full((N, K // B), 124, np.uint8)
    scale = 2.0 ** ((129 - 127 - 2) + (124 - 127 - 2))
    bias = (synth.random_ints((1, N), -1000, 1000, 7).numpy()[0] * scale).astype(np.float32)
    y_ref, y_seq, _ = orc.gemm(qa, ea, 4, qw, ew, 4, B, bias=bias)
    assert np.array_equal(y_ref, y_seq)
    qy, ey, bad = orc.quantize_2d(y_ref, By, 2, wy)
    f4 = mxb.MxFormat(B, 4)
    ym, ye = mxb.mx_gemm_q(_dev(orc.pack(qa, 4)), _dev(ea), f4, _dev(orc.pack(qw, 4)), _dev(ew), f4, M, N, K,
                           mxb.MxFormat(By, wy, 8, 2), bias=_dev(bias),
                           y_exp=torch.empty((M // 2, N // By), dtype=torch.uint8, device="cuda"))
    assert mxb.mx_poll_status() == 0 and bad == 0
    assert np.array_equal(ye.cpu().numpy(), ey)
    assert np.array_equal(ym.cpu().numpy(), orc.pack(qy, wy))


def test_batched_product_on_two_row_blocks(mxb):
    """Per-head products on slices of packed [tokens, heads*d] tensors quantized in (16,2) blocks, and
    items stacked along the rows of the weight-side tensor: bit for bit on order-independent operands."""
    H, M, N, d, B, w = 5, 200, 136, 64, 16, 8
    qa = synth.random_ints((M, H * d), -127, 127, 70).numpy()
    ea = np.repeat(np.repeat(synth.random_bytes((M // 2, H), 121, 133, 71).numpy(), d // B, axis=1), 1, axis=0)
    qw = synth.random_ints((H * N, d), -127, 127, 72).numpy()              # items stacked along rows
    ew = np.repeat(synth.random_bytes((H * N // 2, 1), 115, 127, 73).numpy(), d // B, axis=1)
    f2 = mxb.MxFormat(B, w, 8, 2)
    y = torch.full((H * M, N), 3.0, device="cuda")
    mxb.mx_gemm_batched(_dev(orc.pack(qa, w)), _dev(ea), f2, H * d, d, _dev(orc.pack(qw, w)), _dev(ew), f2,
                        d, N * d, M, N, d, H, y, N, M * N)
    assert mxb.mx_poll_status() == 0
    got = y.cpu().numpy()
    ea_rows, ew_rows = orc.expand_exponent_rows(ea, 2), orc.expand_exponent_rows(ew, 2)
    nb = d // B
    for h in range(H):
        y_ref, y_seq, _ = orc.gemm(qa[:, h * d:(h + 1) * d], ea_rows[:, h * nb:(h + 1) * nb], w,
                                   qw[h * N:(h + 1) * N], ew_rows[h * N:(h + 1) * N], w, B)
        assert np.array_equal(y_ref, y_seq)
        assert np.array_equal(got[h * M:(h + 1) * M], y_ref), h
