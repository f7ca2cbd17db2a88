"""GPU parity of the layer with an MXInt result (mx_gemm_q / mx_linear_q) against the oracle's
``gemm_requant``: the fp32 product quantized again, in blocks along the output-feature axis.

The codes are integers decided by fp32 values, and the fp32 accumulation order of the tensor pipe
is not the oracle's.  So: (1) on operands whose partial sums are all exactly representable every
order gives the same fp32 value, and the codes and exponent bytes must match bit for bit;
(2) on general operands a code may differ only where the oracle's value lies within the product's
tolerance (1e-5 * S) of a rounding or binade boundary -- everything else must be identical, and
every code must be a correct rounding of some value inside the tolerance."""
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


def _exact_operands(M, N, K, B, seed):
    """4-bit mantissas, one exponent per operand: every partial sum is an integer below 2^24
    times one power of two, exact in fp32 in any order."""
    qa = synth.random_ints((M, K), -7, 7, seed).numpy()
    qw = synth.random_ints((N, K), -7, 7, seed + 1).numpy()
    ea = np.full((M, K // B), 129, np.uint8)
    ew = np.full((N, K // B), 124, np.uint8)
    return qa, ea, qw, ew


EXACT_CASES = [
    # M, N, K, B, By, wy
    (300, 544, 512, 16, 16, 4),
    (300, 544, 512, 16, 32, 8),
    (130, 208, 256, 32, 16, 2),       # N % 32 == 16: the last 32-column chunk is half outside
    (2048, 1024, 320, 16, 32, 6),     # wide tiles, several per CTA
    (1, 64, 64, 32, 32, 5),
    (2100, 2336, 128, 16, 16, 8),     # 90 tiles of 256x256, ragged rows: the CTA-pair kernel's epilogue
]


@pytest.mark.parametrize("case", EXACT_CASES)
def test_requantized_product_bit_exact_where_fp32_is_order_independent(mxb, case):
    M, N, K, B, By, wy = case
    qa, ea, qw, ew = _exact_operands(M, N, K, B, seed=M + N + wy)
    scale = 2.0 ** ((129 - 127 - 2) + (124 - 127 - 2))                     # one unit of the product grid
    bias = (synth.random_ints((1, N), -1000, 1000, 7).numpy()[0] * scale).astype(np.float32)
    qy, ey, bad, y_ref, _ = orc.gemm_requant(qa, ea, 4, qw, ew, 4, B, By, wy, bias=bias)
    fa = fw = mxb.MxFormat(B, 4)
    fy = mxb.MxFormat(By, wy)
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    ym, ye = mxb.mx_gemm_q(_dev(orc.pack(qa, 4)), _dev(ea), fa, _dev(orc.pack(qw, 4)), _dev(ew), fw,
                           M, N, K, fy, bias=_dev(bias), nonfinite_count=cnt)
    assert mxb.mx_poll_status() == 0
    assert np.array_equal(ye.cpu().numpy(), ey)
    assert np.array_equal(ym.cpu().numpy(), orc.pack(qy, wy))
    assert int(cnt.item()) == bad == 0
    # the fp32 entry point on the same operands returns exactly the oracle's values
    y = mxb.mx_gemm(_dev(orc.pack(qa, 4)), _dev(ea), fa, _dev(orc.pack(qw, 4)), _dev(ew), fw, M, N, K,
                    bias=_dev(bias), algo=mxb.MX_ALGO_TCGEN05)
    assert np.array_equal(y.cpu().numpy(), y_ref)


def _check_valid_codes(qg, eg, qo, eo, y_ref, S, By, wy):
    M, N = y_ref.shape
    y = y_ref.astype(np.float64)
    tol = TOL * S + 1e-300
    qmax = 2 ** (wy - 1) - 1
    yb, tb = np.abs(y).reshape(M, N // By, By), tol.reshape(M, N // By, By)
    lo = np.maximum(yb - tb, 0).max(axis=2)
    hi = (yb + tb).max(axis=2)
    e_lo = np.where(lo > 0, np.frexp(lo)[1] - 1 + 127, 0)
    e_hi = np.maximum(np.frexp(hi)[1] - 1 + 127, 0)
    eg64 = eg.astype(np.int64)
    assert ((eg64 >= e_lo) & (eg64 <= e_hi)).all(), "exponent byte outside what the tolerance allows"
    step = np.repeat(np.ldexp(1.0, eg64 - 127 - (wy - 2)), By, axis=1)
    xg = qg.astype(np.float64) * step
    free = np.abs(qg) < qmax
    assert (np.abs(xg - y)[free] <= (0.5 * step + tol)[free]).all(), "a code is not a rounding of y within tolerance"
    sat = ~free
    assert (np.abs(y)[sat] >= ((qmax - 0.5) * step - tol)[sat]).all() and (np.sign(y[sat]) == np.sign(qg[sat])).all()
    # where the oracle's decision is stable under the tolerance, the codes are the oracle's
    same_e = np.repeat(eg == eo, By, axis=1)
    r = y / step
    away = np.abs((r - np.floor(r)) - 0.5) * step > tol
    stable = same_e & away
    assert np.array_equal(qg[stable], qo[stable])
    assert stable.mean() > 0.99 and (eg == eo).mean() > 0.99
    return float((qg != qo).mean())


@pytest.mark.parametrize("case", [(257, 544, 1024, 16, 8, 4, 16, 4), (384, 640, 2048, 32, 8, 4, 32, 8),
                                  (200, 320, 320, 32, 4, 4, 16, 8)])
def test_requantized_product_general_operands(mxb, case):
    M, N, K, B, wa, ww, By, wy = case
    qa = synth.random_ints((M, K), -(2 ** (wa - 1) - 1), 2 ** (wa - 1) - 1, 3 * M).numpy()
    qw = synth.random_ints((N, K), -(2 ** (ww - 1) - 1), 2 ** (ww - 1) - 1, 3 * M + 1).numpy()
    ea = synth.random_bytes((M, K // B), 124, 130, 3 * M + 2).numpy()
    ew = synth.random_bytes((N, K // B), 117, 123, 3 * M + 3).numpy()
    bias = np.random.default_rng(5).standard_normal(N).astype(np.float32)
    qo, eo, bad, y_ref, S = orc.gemm_requant(qa, ea, wa, qw, ew, ww, B, By, wy, bias=bias)
    S = S + np.abs(bias)[None, :]
    fa, fw, fy = mxb.MxFormat(B, wa), mxb.MxFormat(B, ww), mxb.MxFormat(By, wy)
    ym, ye = mxb.mx_gemm_q(_dev(orc.pack(qa, wa)), _dev(ea), fa, _dev(orc.pack(qw, ww)), _dev(ew), fw,
                           M, N, K, fy, bias=_dev(bias))
    assert mxb.mx_poll_status() == 0
    qg = orc.unpack(ym.cpu().numpy(), N, wy)
    _check_valid_codes(qg, ye.cpu().numpy(), qo, eo, y_ref, S, By, wy)


def test_linear_q_feeds_the_next_layer(mxb):
    """Two layers: the first returns MXInt8 activations straight from its epilogue, the second
    consumes them as its quantized input.  On order-independent operands the hand-over is bit
    exact, so the oracle's own chain is the reference for the second layer."""
    M, K1, N1, N2, B = 256, 256, 512, 384, 16
    x = (synth.random_ints((M, K1), -7, 7, 1).numpy() * 0.25).astype(np.float32)       # representable at w=4
    x[:, ::16] = 1.75                                                                 # every block has E = 0
    w1 = (synth.random_ints((N1, K1), -7, 7, 2).numpy() * 0.125).astype(np.float32)
    w1[:, ::16] = 0.875
    w2 = synth.gaussian_weights(N2, N1, seed=3).numpy()
    qa, ea, _ = orc.quantize(x, B, 4)
    q1, e1, _ = orc.quantize(w1, B, 4)
    q2, e2, _ = orc.quantize(w2, B, 4)
    assert np.array_equal(orc.dequantize(qa, ea, B, 4), x) and np.array_equal(orc.dequantize(q1, e1, B, 4), w1)
    qh, eh, _, _, _ = orc.gemm_requant(qa, ea, 4, q1, e1, 4, B, B, 8)
    y_ref, _, S = orc.gemm(qh, eh, 8, q2, e2, 4, B)
    f4, f8 = mxb.MxFormat(B, 4), mxb.MxFormat(B, 8)
    w1m, w1e = mxb.mx_quantize(_dev(w1), f4)
    w2m, w2e = mxb.mx_quantize(_dev(w2), f4)
    hm, he = mxb.mx_linear_q(_dev(x), f4, w1m, w1e, f4, N1, f8)
    assert np.array_equal(he.cpu().numpy(), eh) and np.array_equal(hm.cpu().numpy(), orc.pack(qh, 8))
    y = mxb.mx_gemm(hm, he, f8, w2m, w2e, f4, M, N2, N1, algo=mxb.MX_ALGO_TCGEN05)
    assert mxb.mx_poll_status() == 0
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
    assert (err <= TOL * S + 1e-37).all()


def test_requantized_product_nonfinite_blocks(mxb):
    M, N, K, B = 130, 256, 128, 16
    qa, ea, qw, ew = _exact_operands(M, N, K, B, seed=9)
    ea[3, 2] = 255                                   # row 3 of the result is NaN
    ew[200, 7] = 255                                 # column 200 of the result is NaN
    qy, ey, bad, y_ref, _ = orc.gemm_requant(qa, ea, 4, qw, ew, 4, B, 32, 4)
    assert bad == (N // 32) + (M - 1)
    f4 = mxb.MxFormat(B, 4)
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    ym, ye = mxb.mx_gemm_q(_dev(orc.pack(qa, 4)), _dev(ea), f4, _dev(orc.pack(qw, 4)), _dev(ew), f4, M, N, K,
                           mxb.MxFormat(32, 4), nonfinite_count=cnt)
    assert np.array_equal(ye.cpu().numpy(), ey) and np.array_equal(ym.cpu().numpy(), orc.pack(qy, 4))
    assert int(cnt.item()) == bad
