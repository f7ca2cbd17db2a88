"""GPU parity of the two other MX formats of the paper's Sec. 2 -- Block Minifloat and Block Logarithm:
quantizer codes and shared bytes bit for bit against the oracle, the decode exact, the product on the
tensor-core kernels within 1e-5 * S (S = sum of the magnitudes of the element products)."""
import numpy as np
import pytest
import torch

from oracle import mx_oracle as orc
from paper_2307_15517_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-5
FORMATS = [(orc.KIND_BMF, 4, 3), (orc.KIND_BMF, 2, 5), (orc.KIND_BMF, 5, 2), (orc.KIND_BMF, 3, 2),
           (orc.KIND_BL, 4, 0), (orc.KIND_BL, 3, 0), (orc.KIND_BL, 5, 0)]


@pytest.fixture(scope="module")
def mxb():
    from paper_2307_15517_b200 import binding
    return binding


def _edge_rows(K, B):
    """Rows with zeros, ties, saturation, sqrt(2) neighbours, tiny, huge, subnormal and non-finite values."""
    g = np.random.default_rng(9)
    x = (g.standard_normal((24, K)) * np.exp2(g.integers(-20, 20, (24, 1)))).astype(np.float32)
    x[0, :B] = 0.0
    x[1, 3] = np.inf
    x[2, B + 1] = np.nan
    x[3, :B] = (g.standard_normal(B) * 2.0 ** -110).astype(np.float32)           # below 2^-95: zero block
    x[4, :B] = (g.standard_normal(B) * 2.0 ** -96).astype(np.float32)            # straddles the cut
    x[5, :B] = (g.standard_normal(B) * 2.0 ** 120).astype(np.float32)
    x[6, :8] = np.array([1.0, 1.4142135, 1.4142137, 1.9999999, 0.70710677, 0.7071068, 2.0, -1.5], np.float32)
    x[7, :8] = np.array([1.0625, 1.1875, 1.3125, 1.9375, 1.96875, -1.03125, 0.53125, 0.515625], np.float32)   # ties
    x[8, :B] = np.float32(1e-41)                                                  # binary32 subnormals
    x[9, :4] = np.array([3.0e38, -1.0, 2.0 ** 100, 2.0 ** -20], np.float32)
    x[10, :B] = np.ldexp(np.float32(1.0), -np.arange(B)).astype(np.float32)        # one value per binade
    return x


@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("B", (16, 32))
def test_alt_quantize_bit_exact(mxb, fmt, B):
    kind, eb, mb = fmt
    K = 8 * B + 64
    x = np.vstack([_edge_rows(K, B), synth.student_t_activations(40, K, 3).numpy(),
                   synth.outlier_activations(40, K, 4, 3, 40.0).numpy()])
    codes, shared, bad = orc.alt_quantize(x, kind, B, eb, mb)
    f = mxb.MxAltFormat(kind, B, eb, mb)
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    cg, sg = mxb.mx_alt_quantize(torch.from_numpy(x).cuda(), f, nonfinite_count=cnt)
    assert np.array_equal(sg.cpu().numpy(), shared)
    assert np.array_equal(cg.cpu().numpy(), codes)
    assert int(cnt.item()) == bad
    # decode: exact, in fp32 and in bf16
    want = orc.alt_dequantize(codes, shared, kind, B, eb, mb)
    for dtype in (torch.float32, torch.bfloat16):
        got = mxb.mx_alt_dequantize(cg, sg, f, dtype=dtype).float().cpu().numpy().astype(np.float64)
        assert np.array_equal(np.isnan(got), np.isnan(want))
        assert np.array_equal(got[~np.isnan(want)], want[~np.isnan(want)])
    # bf16 input and a padded leading dimension
    xb = torch.from_numpy(x).to(torch.bfloat16)
    codes_b, shared_b, _ = orc.alt_quantize(xb.float().numpy(), kind, B, eb, mb)
    pad = torch.zeros((x.shape[0], K + 24), dtype=torch.bfloat16, device="cuda")
    pad[:, :K] = xb.cuda()
    cb, sb = mxb.mx_alt_quantize(pad[:, :K], f)
    assert np.array_equal(cb.cpu().numpy(), codes_b) and np.array_equal(sb.cpu().numpy(), shared_b)


@pytest.mark.parametrize("case", [
    # (a format, w format, B, M, N, K)
    ((orc.KIND_BMF, 4, 3), (orc.KIND_BMF, 4, 3), 16, 300, 520, 1152),
    ((orc.KIND_BMF, 3, 4), (orc.KIND_BL, 4, 0), 32, 130, 260, 256),
    ((orc.KIND_BL, 5, 0), (orc.KIND_BL, 3, 0), 16, 257, 513, 512),
    ((orc.KIND_BMF, 5, 2), (orc.KIND_BMF, 2, 5), 32, 1536, 2560, 256),       # multi-wave tiles
])
def test_alt_gemm_within_tolerance(mxb, case):
    afmt, wfmt, B, M, N, K = case
    a = synth.student_t_activations(M, K, 11).numpy()
    w = synth.gaussian_weights(N, K, 12).numpy()
    ac, ash, _ = orc.alt_quantize(a, afmt[0], B, afmt[1], afmt[2])
    wc, wsh, _ = orc.alt_quantize(w, wfmt[0], B, wfmt[1], wfmt[2])
    wsh[7, 1] = 255                                      # a non-finite weight block: column 7 is NaN
    bias = np.random.default_rng(2).standard_normal(N).astype(np.float32)
    y_ref, S = orc.alt_gemm(ac, ash, afmt, wc, wsh, wfmt, B, bias=bias)
    dev = lambda t: torch.from_numpy(np.ascontiguousarray(t)).cuda()
    ypad = torch.full((M, N + 8), -77.0, device="cuda")
    mxb.mx_alt_gemm(dev(ac), dev(ash), mxb.MxAltFormat(afmt[0], B, afmt[1], afmt[2]), dev(wc), dev(wsh),
                    mxb.MxAltFormat(wfmt[0], B, wfmt[1], wfmt[2]), bias=dev(bias), y=ypad[:, :N])
    assert mxb.mx_poll_status() == 0
    y = ypad[:, :N].cpu().numpy()
    assert np.array_equal(np.isnan(y), np.isnan(y_ref)) and np.isnan(y[:, 7]).all()
    ok = ~np.isnan(y_ref)
    err = np.abs(y.astype(np.float64) - y_ref.astype(np.float64))
    assert (err[ok] <= (TOL * S + 1e-37)[ok]).all(), float((err[ok] / np.maximum(S[ok], 1e-300)).max())
    assert (ypad[:, N:] == -77.0).all()


def test_alt_arguments_rejected_on_the_host(mxb):
    x = torch.zeros((4, 64), device="cuda")
    for bad in (mxb.MxAltFormat(1, 16, 6, 1), mxb.MxAltFormat(1, 16, 4, 4), mxb.MxAltFormat(2, 16, 4, 1),
                mxb.MxAltFormat(3, 16, 4, 3), mxb.MxAltFormat(1, 8, 4, 3)):
        with pytest.raises(mxb.MxError) as e:
            mxb.mx_alt_quantize(x, bad)
        assert e.value.status == -3
    with pytest.raises(mxb.MxError) as e:
        mxb.mx_alt_quantize(torch.zeros((4, 40), device="cuda"), mxb.MxAltFormat(1, 16, 4, 3))
    assert e.value.status == -2
