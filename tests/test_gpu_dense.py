"""Dense storage of the mantissas (Eq. 1: m + 1 bits per value, so w = 2, 3, 5, 6 take no more than
that): packing and unpacking bit for bit against the oracle's byte images, the stored size equal to
Eq. 1's, and the layer computed straight from dense weights equal to the one from the container."""
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


@pytest.mark.parametrize("w", (2, 3, 4, 5, 6, 7, 8))
@pytest.mark.parametrize("B", (16, 32))
def test_dense_pack_unpack_bit_exact_and_eq1_size(mxb, w, B):
    rows, K = 37, 5 * B + 32 * 3
    K -= K % B
    x = synth.student_t_activations(rows, K, w).numpy()
    q, e, _ = orc.quantize(x, B, w)
    f = mxb.MxFormat(B, w)
    mant, exps = mxb.mx_quantize(_dev(x), f)
    dense = mxb.mx_pack_dense(mant, K, f)
    assert np.array_equal(dense.cpu().numpy(), orc.pack_dense(q, w))
    assert dense.numel() == mxb.mx_mant_bytes(rows, K, f.dense()) == rows * K * w // 8
    # stored bits per value = Eq. 1
    bits = 8.0 * (dense.numel() + exps.numel()) / (rows * K)
    assert abs(bits - mxb.mx_format_bits(f)) < 1e-12 and abs(bits - orc.format_bits(B, w)) < 1e-12
    back = mxb.mx_unpack_dense(dense, K, f)
    assert torch.equal(back, mant)
    # decode straight from the dense form, fp32 and bf16
    want = orc.dequantize(q, e, B, w)
    for dtype in (torch.float32, torch.bfloat16):
        got = mxb.mx_dequantize(dense, exps, K, f.dense(), dtype=dtype).float().cpu().numpy().astype(np.float64)
        assert np.array_equal(got, want)


@pytest.mark.parametrize("case", [(16, 8, 3, 300, 1152, 528), (32, 4, 5, 130, 256, 72), (16, 6, 2, 257, 2048, 1000),
                                  (32, 8, 6, 2048, 512, 2304)])
def test_layer_from_dense_weights(mxb, case):
    B, wa, ww, M, K, N = case
    x = synth.student_t_activations(M, K, seed=wa).numpy()
    wt = synth.gaussian_weights(N, K, seed=ww).numpy()
    qa, ea, _ = orc.quantize(x, B, wa)
    qw, ew, _ = orc.quantize(wt, B, ww)
    bias = np.random.default_rng(3).standard_normal(N).astype(np.float32)
    y_ref, y_seq, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias)
    fa, fw = mxb.MxFormat(B, wa), mxb.MxFormat(B, ww)
    w_dense = _dev(orc.pack_dense(qw, ww))
    w_cont = _dev(orc.pack(qw, ww))
    for algo in (mxb.MX_ALGO_AUTO, mxb.MX_ALGO_TCGEN05_BLOCKWISE):
        y = mxb.mx_linear(_dev(x), fa, w_dense, _dev(ew), fw.dense(), N, bias=_dev(bias), algo=algo)
        y_c = mxb.mx_linear(_dev(x), fa, w_cont, _dev(ew), fw, N, bias=_dev(bias), algo=algo)
        assert mxb.mx_poll_status() == 0
        err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
        assert (err <= TOL * S + 1e-37).all(), float((err / S).max())
        assert torch.equal(y, y_c)                              # same operand bits, same kernel
        if algo == mxb.MX_ALGO_TCGEN05_BLOCKWISE:
            assert np.array_equal(y.cpu().numpy(), y_seq)
    # both operands pre-quantized, activations dense as well
    y = mxb.mx_gemm(_dev(orc.pack_dense(qa, wa)), _dev(ea), fa.dense(), w_dense, _dev(ew), fw.dense(), M, N, K,
                    bias=_dev(bias), algo=mxb.MX_ALGO_TCGEN05)
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
    assert (err <= TOL * S + 1e-37).all()
    if N % B:
        return
    # MXInt result from dense weights
    ym, ye = mxb.mx_linear_q(_dev(x), fa, w_dense, _dev(ew), fw.dense(), N, mxb.MxFormat(B, 8), bias=_dev(bias))
    ym_c, ye_c = mxb.mx_linear_q(_dev(x), fa, w_cont, _dev(ew), fw, N, mxb.MxFormat(B, 8), bias=_dev(bias))
    assert torch.equal(ym, ym_c) and torch.equal(ye, ye_c)


def test_dense_refused_where_only_the_container_is_read(mxb):
    f = mxb.MxFormat(32, 3)
    x = torch.zeros((8, 256), device="cuda")
    with pytest.raises(mxb.MxError) as e:
        mxb.mx_quantize(x, f.dense())
    assert e.value.status == -3
    mant, exps = mxb.mx_quantize(x, f)
    dense = mxb.mx_pack_dense(mant, 256, f)
    for algo in (mxb.MX_ALGO_SIMT, mxb.MX_ALGO_STREAM, mxb.MX_ALGO_TCGEN05_FUSED):
        with pytest.raises(mxb.MxError) as e:
            mxb.mx_linear(x, mxb.MxFormat(32, 8), dense, exps, f.dense(), 8, algo=algo)
        assert e.value.status == -3, algo
    with pytest.raises(mxb.MxError) as e:
        mxb.mx_linear(x, mxb.MxFormat(32, 8).dense(), dense, exps, f.dense(), 8)
    assert e.value.status == -3
