"""GPU parity of the hardware block-scaled tensor-core path (MX_ALGO_TCGEN05_MXF8): MXInt tensors with
blocks of 32 and mantissas of at most 5 bits, held exactly as E4M3 elements with E8M0 block scales."""
import numpy as np
import pytest
import torch

from oracle import mx_oracle as orc
from paper_2307_15517_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-5
B = 32


@pytest.fixture(scope="module")
def mxb():
    from paper_2307_15517_b200 import binding
    return binding


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _gemm(mxb, qa, ea, wa, qw, ew, ww, bias=None, y=None):
    M, K = qa.shape
    N = qw.shape[0]
    return mxb.mx_gemm(_dev(orc.pack(qa, wa)), _dev(ea), mxb.MxFormat(B, wa), _dev(orc.pack(qw, ww)), _dev(ew),
                       mxb.MxFormat(B, ww), M, N, K, bias=None if bias is None else _dev(bias), y=y,
                       algo=mxb.MX_ALGO_TCGEN05_MXF8)


@pytest.mark.parametrize("ww", (2, 3, 4, 5))
def test_one_hot_rows_return_the_decoded_weights(mxb, ww):
    """A = identity-like rows: Y must be the decoded weights element for element -- operand bytes, swizzled
    tiles, the scale-chunk layout and the scale-factor ids of the four K sub-steps all have to be right."""
    K, N = 256, 384
    x = np.zeros((K, K), np.float32)
    x[np.arange(K), np.arange(K)] = 1.0
    qa, ea, _ = orc.quantize(x, B, 5)
    wt = synth.student_t_activations(N, K, 3).numpy()
    qw, ew, _ = orc.quantize(wt, B, ww)
    y = _gemm(mxb, qa, ea, 5, qw, ew, ww)
    assert mxb.mx_poll_status() == 0
    assert np.array_equal(y.cpu().numpy().astype(np.float64), orc.dequantize(qw, ew, B, ww).T)


@pytest.mark.parametrize("shape", [(128, 128, 128, 4, 4), (300, 520, 1152, 5, 3), (257, 513, 2048, 5, 2),
                                   (1536, 2560, 256, 4, 5), (2100, 2330, 384, 5, 5)])
def test_block_scaled_product_within_tolerance(mxb, shape):
    M, N, K, wa, ww = shape
    qa = synth.random_ints((M, K), -(2 ** (wa - 1) - 1), 2 ** (wa - 1) - 1, M).numpy()
    qw = synth.random_ints((N, K), -(2 ** (ww - 1) - 1), 2 ** (ww - 1) - 1, N).numpy()
    ea = synth.random_bytes((M, K // B), 124, 130, M + 1).numpy()
    ew = synth.random_bytes((N, K // B), 117, 123, N + 1).numpy()
    bias = np.random.default_rng(2).standard_normal(N).astype(np.float32)
    y_ref, _, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias)
    ypad = torch.full((M, N + 8), -77.0, device="cuda")
    _gemm(mxb, qa, ea, wa, qw, ew, ww, bias=bias, y=ypad[:, :N])
    assert mxb.mx_poll_status() == 0
    err = np.abs(ypad[:, :N].cpu().numpy().astype(np.float64) - y_ref)
    assert (err <= TOL * S + 1e-37).all(), float((err / S).max())
    assert (ypad[:, N:] == -77.0).all()


def test_block_scaled_product_exact_on_order_independent_operands_and_poisoning(mxb):
    M, N, K = 384, 640, 512
    qa = synth.random_ints((M, K), -15, 15, 5).numpy()
    qw = synth.random_ints((N, K), -7, 7, 6).numpy()
    ea = np.repeat(synth.random_bytes((M, 1), 121, 133, 7).numpy(), K // B, axis=1)
    ew = np.repeat(synth.random_bytes((N, 1), 3, 250, 8).numpy(), K // B, axis=1)      # scales across the whole range
    ew[:, :] = np.clip(ew, 60, 190)                                                      # keep products inside fp32
    y_ref, y_seq, _ = orc.gemm(qa, ea, 5, qw, ew, 4, B)
    assert np.array_equal(y_ref, y_seq)
    y = _gemm(mxb, qa, ea, 5, qw, ew, 4).cpu().numpy()
    assert np.array_equal(y, y_ref)
    ew2 = ew.copy()
    ew2[11, 3] = 255
    ea2 = ea.copy()
    ea2[5, 0] = 255
    y = _gemm(mxb, qa, ea2, 5, qw, ew2, 4).cpu().numpy()
    want = np.zeros((M, N), bool)
    want[:, 11] = True
    want[5, :] = True
    assert np.array_equal(np.isnan(y), want)
    assert np.array_equal(y[~want], y_ref[~want])


def test_linear_on_the_block_scaled_path(mxb):
    M, K, N = 1024, 1024, 768
    x = synth.student_t_activations(M, K, 4)
    w = synth.gaussian_weights(N, K, 5)
    qa, ea, _ = orc.quantize(x.numpy(), B, 5)
    qw, ew, _ = orc.quantize(w.numpy(), B, 3)
    y_ref, _, S = orc.gemm(qa, ea, 5, qw, ew, 3, B)
    fw = mxb.MxFormat(B, 3)
    wm, we = mxb.mx_quantize(w.cuda(), fw)
    y = mxb.mx_linear(x.cuda(), mxb.MxFormat(B, 5), wm, we, fw, N, algo=mxb.MX_ALGO_TCGEN05_MXF8)
    assert mxb.mx_poll_status() == 0
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
    assert (err <= TOL * S + 1e-37).all(), float((err / S).max())


def test_formats_outside_the_exact_subset_are_refused(mxb):
    x = torch.zeros((128, 256), device="cuda")
    for fa, fw, K in ((mxb.MxFormat(16, 4), mxb.MxFormat(16, 4), 256), (mxb.MxFormat(32, 8), mxb.MxFormat(32, 4), 256),
                      (mxb.MxFormat(32, 4), mxb.MxFormat(32, 6), 256), (mxb.MxFormat(32, 4), mxb.MxFormat(32, 4), 192)):
        wm, we = mxb.mx_quantize(torch.zeros((128, K), device="cuda"), fw)
        with pytest.raises(mxb.MxError) as e:
            mxb.mx_linear(x[:, :K], fa, wm, we, fw, 128, algo=mxb.MX_ALGO_TCGEN05_MXF8,
                          workspace=mxb.alloc_workspace(1 << 22))
        assert e.value.status == -3
