"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on identical seeded
inputs.  Mantissas and exponent bytes must match bit for bit; fp32 outputs of the block-scaled
product must satisfy |Y - Y_ref| <= 1e-5 * S with S = sum_b |t_b| the sum of the absolute block
terms (so <= 1e-5 relative wherever there is no cancellation); the CUDA-core kernel adds the
blocks in ascending order and must equal the oracle's sequential-fp32 result exactly."""
import numpy as np
import pytest
import torch

from oracle import mx_oracle as orc
from paper_2307_15517_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5
WIDTHS = (2, 3, 4, 5, 6, 8)


@pytest.fixture(scope="module")
def mxb():
    from paper_2307_15517_b200 import binding
    return binding


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _oracle_packed(x_np, B, w):
    q, e, bad = orc.quantize(x_np, B, w)
    return q, e, orc.pack(q, w), bad


def _check_tol(y_gpu, y_ref, S):
    y = y_gpu.cpu().numpy().astype(np.float64)
    err = np.abs(y - y_ref.astype(np.float64))
    bound = TOL * S + 1e-37
    worst = float((err / np.maximum(S, 1e-300)).max())
    assert (err <= bound).all(), "max |dY|/S = %.3e" % worst
    return worst


# ------------------------------------------------------------------------------ quantizer

def _edge_case_rows(K):
    """Rows that exercise zeros, subnormals, ties, saturation, huge and non-finite values."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal((12, K)).astype(np.float32)
    x[0] = 0.0
    x[1, :] = (rng.integers(-7, 8, K) * 0.5).astype(np.float32)          # many exact ties
    x[1, ::16] = 4.0
    x[2] = np.ldexp(x[2], -140).astype(np.float32)                         # subnormal blocks
    x[3] = np.ldexp(x[3], 120).astype(np.float32)                          # near the top
    x[3, 5] = 3.0e38
    x[4, 3] = np.inf
    x[4, 40] = -np.inf
    x[5, 17] = np.nan
    x[6, :] = 7.99                                                          # saturating maximum
    x[7, :] = np.float32(2.0 ** -126) - np.float32(2.0 ** -149)
    x[8, ::2] = -x[8, ::2] * 1000
    x[9] = np.ldexp(np.ones(K), rng.integers(-126, 127, K)).astype(np.float32)
    x[10, :] = -0.0
    x[11] = rng.standard_t(3, K).astype(np.float32) * 40
    return x


@pytest.mark.parametrize("B", (16, 32))
@pytest.mark.parametrize("w", WIDTHS)
def test_quantize_bit_exact(mxb, B, w):
    F = mxb.MxFormat(B, w)
    rng = np.random.default_rng(100 * B + w)
    cases = [
        (rng.standard_normal((37, 96)) * np.exp(rng.uniform(-8, 8, (37, 1)))).astype(np.float32),
        rng.standard_t(3, (130, 2080)).astype(np.float32),       # ragged last warp, several CTAs
        _edge_case_rows(64),
        np.zeros((0, 64), np.float32),
    ]
    for x in cases:
        q, e, packed, bad = _oracle_packed(x, B, w)
        cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
        mant, exps = mxb.mx_quantize(_dev(x), F, nonfinite_count=cnt)
        assert np.array_equal(exps.cpu().numpy(), e)
        assert np.array_equal(mant.cpu().numpy(), packed)
        assert int(cnt.item()) == bad
        if x.shape[0]:
            xhat = mxb.mx_dequantize(mant, exps, x.shape[1], F).cpu().numpy()
            want = orc.dequantize(q, e, B, w)
            assert np.array_equal(np.isnan(xhat), np.isnan(want))
            ok = ~np.isnan(want)
            assert np.array_equal(xhat[ok].astype(np.float64), want[ok])
            xhat16 = mxb.mx_dequantize(mant, exps, x.shape[1], F, dtype=torch.bfloat16)
            assert np.array_equal(xhat16.float().cpu().numpy()[ok].astype(np.float64), want[ok])


@pytest.mark.parametrize("w", (4, 8))
def test_quantize_bf16_input_and_padded_rows(mxb, w):
    F = mxb.MxFormat(32, w)
    g = torch.Generator().manual_seed(w)
    xb = (torch.randn(67, 256, generator=g) * 3).to(torch.bfloat16)
    q, e, packed, _ = _oracle_packed(xb.float().numpy(), 32, w)
    mant, exps = mxb.mx_quantize(xb.cuda(), F)
    assert np.array_equal(mant.cpu().numpy(), packed) and np.array_equal(exps.cpu().numpy(), e)
    # a view with a leading dimension larger than K
    big = torch.randn(67, 512, generator=g)
    view = big.cuda()[:, 128:384]
    q, e, packed, _ = _oracle_packed(big[:, 128:384].contiguous().numpy(), 32, w)
    mant, exps = mxb.mx_quantize(view, F)
    assert np.array_equal(mant.cpu().numpy(), packed) and np.array_equal(exps.cpu().numpy(), e)


def test_quantize_along_a_strided_axis(mxb):
    """V of attention is blocked along the token axis: x[r, k] = v[k, r]."""
    g = torch.Generator().manual_seed(9)
    v = torch.randn(192, 40, generator=g)                      # [tokens, d]
    for w, B in ((8, 16), (4, 32)):
        F = mxb.MxFormat(B, w)
        q, e, packed, _ = _oracle_packed(v.numpy().T, B, w)
        mant, exps = mxb.mx_quantize(v.cuda().t(), F)
        assert np.array_equal(mant.cpu().numpy(), packed) and np.array_equal(exps.cpu().numpy(), e)


@pytest.mark.parametrize("B,w", [(16, 4), (32, 8), (16, 6), (32, 2)])
def test_quantize_transposed_view_bit_exact(mxb, B, w):
    """Blocks along the slow axis of a row-major tensor (the transposing kernel): ragged row and k
    tiles, edge-case values, non-finite count."""
    rng = np.random.default_rng(B + w)
    base = (rng.standard_t(3, (608, 77)) * np.exp(rng.uniform(-6, 6, (1, 77)))).astype(np.float32)   # [k, r]
    edge = _edge_case_rows(608)                                                                     # [12, 608]
    base[:, :12] = edge.T
    q, e, bad = orc.quantize(np.ascontiguousarray(base.T), B, w)
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    mant, exps = mxb.mx_quantize(_dev(base).t(), mxb.MxFormat(B, w), nonfinite_count=cnt)
    assert np.array_equal(exps.cpu().numpy(), e)
    assert np.array_equal(mant.cpu().numpy(), orc.pack(q, w))
    assert int(cnt.item()) == bad and bad > 0
    xb = torch.from_numpy(base).to(torch.bfloat16)
    q, e, _ = orc.quantize(np.ascontiguousarray(xb.float().numpy().T), B, w)
    mant, exps = mxb.mx_quantize(xb.cuda().t(), mxb.MxFormat(B, w))
    assert np.array_equal(mant.cpu().numpy(), orc.pack(q, w)) and np.array_equal(exps.cpu().numpy(), e)


def test_quantize_single_layer_config(mxb):
    x, wt, spec = synth.single_layer(0)
    F = mxb.MxFormat(spec.block, spec.w_act)
    for t in (x, wt):
        q, e, packed, _ = _oracle_packed(t.numpy(), spec.block, spec.w_act)
        mant, exps = mxb.mx_quantize(t.cuda(), F)
        assert np.array_equal(mant.cpu().numpy(), packed) and np.array_equal(exps.cpu().numpy(), e)


# ------------------------------------------------------------------------------ product

def _random_operands(M, N, K, B, wa, ww, seed, spread=8):
    """Raw mantissas and exponent bytes (not produced by any quantizer): full value range
    including -2^(w-1), exponents spread over 2^spread."""
    qa = synth.random_ints((M, K), -(2 ** (wa - 1)) if wa > 2 else -1, 2 ** (wa - 1) - 1, seed).numpy()
    qw = synth.random_ints((N, K), -(2 ** (ww - 1)) if ww > 2 else -1, 2 ** (ww - 1) - 1, seed + 1).numpy()
    ea = synth.random_bytes((M, K // B), 127 - spread, 127 + spread, seed + 2).numpy()
    ew = synth.random_bytes((N, K // B), 120 - spread, 120 + spread, seed + 3).numpy()
    return qa, ea, qw, ew


GEMM_SHAPES = [
    # M, N, K, B, wa, ww
    (128, 768, 768, 16, 4, 4),        # the single-layer configuration's shape
    (200, 300, 320, 32, 8, 4),        # ragged M and N tails, K tail (320 = 5 * 64)
    (384, 640, 1024, 16, 8, 8),       # several tiles each way
    (130, 40, 96, 16, 6, 3),          # K not a multiple of 64, N below one tile
    (70, 136, 112, 16, 4, 4),         # K % 32 != 0: the tensor-core path decodes W in a pre-pass
    (1, 256, 128, 32, 8, 4),          # a single row
    (257, 513, 2048, 32, 5, 2),
    (1536, 2560, 256, 16, 8, 4),      # 120 tiles of 128x256: the wide-tile kernel, multi-wave
    (2100, 2330, 192, 32, 8, 4),      # 90 tiles of 256x256, ragged both ways: the CTA-pair kernel
]


@pytest.mark.parametrize("shape", GEMM_SHAPES)
def test_gemm_simt_matches_sequential_oracle_exactly(mxb, shape):
    M, N, K, B, wa, ww = shape
    qa, ea, qw, ew = _random_operands(M, N, K, B, wa, ww, seed=M + N)
    bias = np.random.default_rng(1).standard_normal(N).astype(np.float32)
    y_ref, y_seq, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias)
    y = mxb.mx_gemm(_dev(orc.pack(qa, wa)), _dev(ea), mxb.MxFormat(B, wa), _dev(orc.pack(qw, ww)),
                    _dev(ew), mxb.MxFormat(B, ww), M, N, K, bias=_dev(bias), algo=mxb.MX_ALGO_SIMT)
    assert np.array_equal(y.cpu().numpy(), y_seq)
    _check_tol(y, y_ref, S)


TC_ALGOS = ("MX_ALGO_TCGEN05", "MX_ALGO_TCGEN05_FUSED")
TC_ALGOS_ALL = TC_ALGOS + ("MX_ALGO_TCGEN05_BLOCKWISE",)


@pytest.mark.parametrize("shape", GEMM_SHAPES)
@pytest.mark.parametrize("with_bias", (False, True))
@pytest.mark.parametrize("algo", TC_ALGOS_ALL)
def test_gemm_tensor_core_within_tolerance(mxb, shape, with_bias, algo):
    """Block exponents spread over 2^+-3 per operand (2^+-6 per product term), wider than any of
    the paper-shaped workloads produce within one row."""
    M, N, K, B, wa, ww = shape
    qa, ea, qw, ew = _random_operands(M, N, K, B, wa, ww, seed=7 * M + N, spread=3)
    bias = np.random.default_rng(2).standard_normal(N).astype(np.float32) if with_bias else None
    y_ref, y_seq, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias)
    ypad = torch.full((M, N + 8), -77.0, device="cuda")           # canary columns, ldy > N
    y = mxb.mx_gemm(_dev(orc.pack(qa, wa)), _dev(ea), mxb.MxFormat(B, wa), _dev(orc.pack(qw, ww)),
                    _dev(ew), mxb.MxFormat(B, ww), M, N, K, bias=None if bias is None else _dev(bias),
                    y=ypad[:, :N], algo=getattr(mxb, algo))
    assert mxb.mx_poll_status() == 0
    _check_tol(y, y_ref, S)
    assert (ypad[:, N:] == -77.0).all()


def test_gemm_tensor_core_adversarial_exponent_spread(mxb):
    """Block exponents drawn uniformly over 2^+-8 per operand (terms 2^+-16 apart).  The tensor
    pipe aligns the 16 products of one MMA step and the accumulator to the largest of them and
    truncates each (measured: no rounding, no guard bit), so its worst case is 17 truncations of
    one accumulator ulp per step: |dY| < ceil(K/16) * 17 * 2^-23 * S.  The CUDA-core kernel, which
    rounds once per block, stays inside 1e-5 * S on the same operands."""
    M, N, K, B, wa, ww = 200, 300, 320, 32, 8, 4
    qa, ea, qw, ew = _random_operands(M, N, K, B, wa, ww, seed=1700, spread=8)
    y_ref, y_seq, S = orc.gemm(qa, ea, wa, qw, ew, ww, B)
    args = (_dev(orc.pack(qa, wa)), _dev(ea), mxb.MxFormat(B, wa), _dev(orc.pack(qw, ww)), _dev(ew),
            mxb.MxFormat(B, ww), M, N, K)
    bound = -(-K // 16) * 17 * 2.0 ** -23 * S
    for algo in TC_ALGOS:
        y = mxb.mx_gemm(*args, algo=getattr(mxb, algo)).cpu().numpy().astype(np.float64)
        assert mxb.mx_poll_status() == 0
        assert (np.abs(y - y_ref) <= bound).all()
    y = mxb.mx_gemm(*args, algo=mxb.MX_ALGO_SIMT)
    assert np.array_equal(y.cpu().numpy(), y_seq)
    _check_tol(y, y_ref, S)


@pytest.mark.parametrize("shape", GEMM_SHAPES)
def test_gemm_blockwise_accumulation_is_the_sequential_fp32_sum(mxb, shape):
    """Block exponents drawn uniformly over 2^+-8 per operand (terms 2^+-16 apart), where the
    single-accumulator kernels only meet their derived bound: with one tensor-memory accumulator per
    block and the block terms added in fp32 registers in ascending order, the result is the oracle's
    sequential sum bit for bit, and the stated 1e-5 * S holds on every shape."""
    M, N, K, B, wa, ww = shape
    qa, ea, qw, ew = _random_operands(M, N, K, B, wa, ww, seed=31 * M + N, spread=8)
    bias = np.random.default_rng(3).standard_normal(N).astype(np.float32) if (M + N) % 2 else None
    y_ref, y_seq, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias)
    ypad = torch.full((M, N + 8), -77.0, device="cuda")
    y = mxb.mx_gemm(_dev(orc.pack(qa, wa)), _dev(ea), mxb.MxFormat(B, wa), _dev(orc.pack(qw, ww)),
                    _dev(ew), mxb.MxFormat(B, ww), M, N, K, bias=None if bias is None else _dev(bias),
                    y=ypad[:, :N], algo=mxb.MX_ALGO_TCGEN05_BLOCKWISE)
    assert mxb.mx_poll_status() == 0
    _check_tol(y, y_ref, S)
    assert np.array_equal(y.cpu().numpy(), y_seq)
    assert (ypad[:, N:] == -77.0).all()


@pytest.mark.parametrize("K", (11008, 16384))
def test_gemm_long_reductions_with_wide_exponent_spread(mxb, K):
    """The longest reductions of the paper-shaped workloads (LLaMA-7B down projection, OPT-6.7B FFN)
    with the adversarial +-8 exponent spread: the block-wise kernel equal to the sequential fp32 sum
    and inside 1e-5 * S, the default kernel
    inside its derived bound ceil(K/16) * 17 * 2^-23 * S (asserted at these K, not only at K = 320)."""
    M, N, B, wa, ww = 160, 200, 16, 8, 4
    qa, ea, qw, ew = _random_operands(M, N, K, B, wa, ww, seed=K, spread=8)
    y_ref, y_seq, S = orc.gemm(qa, ea, wa, qw, ew, ww, B)
    args = (_dev(orc.pack(qa, wa)), _dev(ea), mxb.MxFormat(B, wa), _dev(orc.pack(qw, ww)), _dev(ew),
            mxb.MxFormat(B, ww), M, N, K)
    y = mxb.mx_gemm(*args, algo=mxb.MX_ALGO_TCGEN05_BLOCKWISE)
    assert mxb.mx_poll_status() == 0
    _check_tol(y, y_ref, S)
    assert np.array_equal(y.cpu().numpy(), y_seq)
    worst_blockwise = float((np.abs(y.cpu().numpy().astype(np.float64) - y_ref) / S).max())
    y = mxb.mx_gemm(*args, algo=mxb.MX_ALGO_TCGEN05).cpu().numpy().astype(np.float64)
    assert mxb.mx_poll_status() == 0
    assert (np.abs(y - y_ref) <= -(-K // 16) * 17 * 2.0 ** -23 * S).all()
    worst_default = float((np.abs(y - y_ref) / S).max())
    print("K=%d spread +-8: max |dY|/S block-wise %.2e, single accumulator %.2e" % (K, worst_blockwise, worst_default))
    assert worst_blockwise <= 1e-5


def test_linear_student_t_full_reduction_length_default_kernel(mxb):
    """Heavy-tailed (Student-t, nu = 3) activations over the full K = 11008 of the LLaMA-7B down
    projection through mx_linear with the default kernel: every output (not a sample) inside
    1e-5 * S, and the measured worst ratio is reported."""
    M, N, K, B, wa, ww = 256, 384, 11008, 16, 8, 4
    x = synth.student_t_activations(M, K, 5)
    w = synth.gaussian_weights(N, K, 6)
    qa, ea, _ = orc.quantize(x.numpy(), B, wa)
    qw, ew, _ = orc.quantize(w.numpy(), B, ww)
    y_ref, _, S = orc.gemm(qa, ea, wa, qw, ew, ww, B)
    fw = mxb.MxFormat(B, ww)
    wm, we = mxb.mx_quantize(w.cuda(), fw)
    worst = {}
    for name in ("MX_ALGO_AUTO", "MX_ALGO_TCGEN05_BLOCKWISE"):
        y = mxb.mx_linear(x.cuda(), mxb.MxFormat(B, wa), wm, we, fw, N, algo=getattr(mxb, name))
        assert mxb.mx_poll_status() == 0
        _check_tol(y, y_ref, S)
        worst[name] = float((np.abs(y.cpu().numpy().astype(np.float64) - y_ref) / np.maximum(S, 1e-300)).max())
    print("Student-t K=11008: max |dY|/S", worst)


@pytest.mark.parametrize("algo", TC_ALGOS_ALL)
@pytest.mark.parametrize("ww,B", [(4, 16), (4, 32), (3, 16), (8, 16), (6, 32)])
def test_gemm_one_hot_rows_expose_the_operand_layout(mxb, algo, ww, B):
    """A = identity-like rows: Y must be the decoded weights, element for element (catches any
    error in the swizzled shared-memory layout, the descriptors or the in-kernel decode)."""
    K, N = 256, 512
    x = np.zeros((K, K), np.float32)
    x[np.arange(K), np.arange(K)] = 1.0
    qa, ea, _ = orc.quantize(x, B, 8)
    wt = synth.student_t_activations(N, K, 3).numpy()
    qw, ew, _ = orc.quantize(wt, B, ww)
    y = mxb.mx_gemm(_dev(orc.pack(qa, 8)), _dev(ea), mxb.MxFormat(B, 8), _dev(orc.pack(qw, ww)),
                    _dev(ew), mxb.MxFormat(B, ww), K, N, K, algo=getattr(mxb, algo))
    assert mxb.mx_poll_status() == 0
    assert np.array_equal(y.cpu().numpy().astype(np.float64), orc.dequantize(qw, ew, B, ww).T)


@pytest.mark.parametrize("ww", (2, 4, 8))
def test_gemm_decode_is_exact_over_the_exponent_range(mxb, ww):
    """Raw weights with every mantissa value (incl. -2^(w-1)) and exponent bytes from 0 (bf16
    subnormal scale) to 253; one-hot activations of value
    2^-60 / 1 / 2^60 keep each output inside fp32, so Y must equal the decoded weight times that
    power of two exactly."""
    K, N, B = 128, 256, 16
    lo = -(2 ** (ww - 1))
    qw = synth.random_ints((N, K), lo, -lo - 1, 11).numpy()
    # byte 254 is left out: -2^(w-1) * 2^(127-(w-2)) = -2^128 is outside bf16 and fp32 (the
    # quantizer never emits -2^(w-1), so it cannot occur in quantized data)
    ew = synth.random_bytes((N, K // B), 0, 253, 12).numpy()
    ew[:, 0] = np.arange(N) % 254                      # every byte value 0..253 appears
    x = np.zeros((K, K), np.float32)
    x[np.arange(K), np.arange(K)] = 1.0
    qa, ea0, _ = orc.quantize(x, B, 8)
    want = orc.dequantize(qw, ew, B, ww).T             # [K, N]
    for shift in (-60, 0, 60):
        ea = (ea0.astype(np.int32) + shift * (ea0 > 0)).astype(np.uint8)
        ref = np.ldexp(want, shift).astype(np.float32)  # rounds only where fp32 itself must
        finite = np.isfinite(ref) & (np.abs(np.ldexp(want, shift)) >= 2.0 ** -126)
        for algo in TC_ALGOS:
            y = mxb.mx_gemm(_dev(orc.pack(qa, 8)), _dev(ea), mxb.MxFormat(B, 8), _dev(orc.pack(qw, ww)),
                            _dev(ew), mxb.MxFormat(B, ww), K, N, K, algo=getattr(mxb, algo)).cpu().numpy()
            assert mxb.mx_poll_status() == 0
            assert finite.sum() > 1000
            assert np.array_equal(y[finite], ref[finite]), (ww, shift, algo)


def test_gemm_nonfinite_blocks_poison_their_outputs(mxb):
    M, N, K, B = 130, 260, 128, 16
    qa, ea, qw, ew = _random_operands(M, N, K, B, 8, 4, seed=5)
    ea[3, 2] = 255
    ew[200, 7] = 255
    y_ref, _, _ = orc.gemm(qa, ea, 8, qw, ew, 4, B)
    for algo in (mxb.MX_ALGO_SIMT, mxb.MX_ALGO_TCGEN05_FUSED, mxb.MX_ALGO_TCGEN05):
        y = mxb.mx_gemm(_dev(orc.pack(qa, 8)), _dev(ea), mxb.MxFormat(B, 8), _dev(orc.pack(qw, 4)),
                        _dev(ew), mxb.MxFormat(B, 4), M, N, K, algo=algo).cpu().numpy()
        assert np.array_equal(np.isnan(y), np.isnan(y_ref))
        assert np.isnan(y[3]).all() and np.isnan(y[:, 200]).all() and not np.isnan(y[4, 5])


# ------------------------------------------------------------------------------ the layer

def test_linear_single_layer_config(mxb):
    """Configuration 1 end to end: quantize X on the fly, weights pre-quantized, Y = X W^T."""
    x, wt, spec = synth.single_layer(0)
    fa, fw = mxb.MxFormat(spec.block, spec.w_act), mxb.MxFormat(spec.block, spec.w_wgt)
    qa, ea, _ = orc.quantize(x.numpy(), spec.block, spec.w_act)
    qw, ew, _ = orc.quantize(wt.numpy(), spec.block, spec.w_wgt)
    y_ref, y_seq, S = orc.gemm(qa, ea, spec.w_act, qw, ew, spec.w_wgt, spec.block)
    w_mant, w_exp = mxb.mx_quantize(wt.cuda(), fw)
    y_tc = mxb.mx_linear(x.cuda(), fa, w_mant, w_exp, fw, spec.N)
    y_fused = mxb.mx_linear(x.cuda(), fa, w_mant, w_exp, fw, spec.N, algo=mxb.MX_ALGO_TCGEN05_FUSED)
    y_simt = mxb.mx_linear(x.cuda(), fa, w_mant, w_exp, fw, spec.N, algo=mxb.MX_ALGO_SIMT)
    assert mxb.mx_poll_status() == 0
    assert np.array_equal(y_simt.cpu().numpy(), y_seq)
    _check_tol(y_tc, y_ref, S)
    _check_tol(y_fused, y_ref, S)


@pytest.mark.parametrize("case", [(16, 8, 4, 300, 1152, 520), (32, 4, 2, 130, 256, 72), (16, 6, 3, 257, 2048, 1000),
                                  (32, 8, 4, 2048, 512, 2304)])
def test_linear_in_kernel_weight_decode(mxb, case):
    """mx_linear with MX_ALGO_TCGEN05_FUSED and 4-bit-container weights, K % 64 == 0: the product
    kernel decodes the packed weights itself and both operand tiles hold k in a permuted order
    inside every group of 8.  Includes all-zero weight blocks, a non-finite weight block and
    weight exponents near both ends of the range (the decode's slow path)."""
    B, wa, ww, M, K, N = case
    x = synth.student_t_activations(M, K, seed=wa + 1)
    wt = synth.gaussian_weights(N, K, seed=ww + 1).numpy()
    wt[5, :B] = 0.0                                           # a zero block
    wt[7, B:2 * B] *= np.float32(2.0 ** -120)                 # scale below the bf16 normal range
    wt[9 % N, :B] *= np.float32(2.0 ** 100)                   # scale near the top
    qa, ea, _ = orc.quantize(x.numpy(), B, wa)
    qw, ew, _ = orc.quantize(wt, B, ww)
    ew[11, 1] = 255                                           # a non-finite block: column 11 is NaN
    fa, fw = mxb.MxFormat(B, wa), mxb.MxFormat(B, ww)
    y_ref, _, S = orc.gemm(qa, ea, wa, qw, ew, ww, B)
    y = mxb.mx_linear(x.cuda(), fa, _dev(orc.pack(qw, ww)), _dev(ew), fw, N, algo=mxb.MX_ALGO_TCGEN05_FUSED)
    assert mxb.mx_poll_status() == 0
    y = y.cpu().numpy()
    assert np.array_equal(np.isnan(y), np.isnan(y_ref)) and np.isnan(y[:, 11]).all()
    ok = ~np.isnan(y_ref)
    err = np.abs(y.astype(np.float64) - y_ref.astype(np.float64))
    assert (err[ok] <= (TOL * S + 1e-37)[ok]).all()


@pytest.mark.parametrize("case", [
    # B, wa, ww, M, K, N, bf16 input
    (16, 8, 4, 700, 768, 1100, False),      # ragged M and N: partly filled panels and tiles
    (32, 4, 4, 300, 1024, 520, True),       # bf16 activations, block 32
    (32, 4, 8, 300, 1024, 520, True),       # int8 weight container
    (16, 6, 3, 1500, 256, 2600, False),     # a single K group, more tiles than CTA pairs
    (32, 8, 4, 2304, 2048, 640, False),     # more activation panels than the first wave covers
])
def test_linear_tensor_core_ragged_shapes_and_edge_blocks(mxb, case):
    """mx_linear with MX_ALGO_TCGEN05 on shapes with ragged tiles both ways (one-CTA and CTA-pair
    kernels, both weight containers, bf16 and fp32 activations): every output against the oracle, with
    zero, tiny, huge and non-finite weight blocks, a bias and canary columns."""
    B, wa, ww, M, K, N, bf16 = case
    x = synth.student_t_activations(M, K, seed=wa + 3)
    if bf16:
        x = x.to(torch.bfloat16)
    wt = synth.gaussian_weights(N, K, seed=ww + 3).numpy()
    wt[5, :B] = 0.0
    wt[7, B:2 * B] *= np.float32(2.0 ** -120)
    wt[9, :B] *= np.float32(2.0 ** 100)
    qa, ea, _ = orc.quantize(x.float().numpy(), B, wa)
    qw, ew, _ = orc.quantize(wt, B, ww)
    ew[11, 1] = 255
    bias = np.random.default_rng(4).standard_normal(N).astype(np.float32)
    fa, fw = mxb.MxFormat(B, wa), mxb.MxFormat(B, ww)
    y_ref, _, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias)
    ypad = torch.full((M, N + 8), -77.0, device="cuda")
    mxb.mx_linear(x.cuda(), fa, _dev(orc.pack(qw, ww)), _dev(ew), fw, N, bias=_dev(bias), y=ypad[:, :N],
                  algo=mxb.MX_ALGO_TCGEN05)
    assert mxb.mx_poll_status() == 0
    y = ypad[:, :N].cpu().numpy()
    assert np.array_equal(np.isnan(y), np.isnan(y_ref)) and np.isnan(y[:, 11]).all()
    ok = ~np.isnan(y_ref)
    err = np.abs(y.astype(np.float64) - y_ref.astype(np.float64))
    assert (err[ok] <= (TOL * S + 1e-37)[ok]).all(), float((err[ok] / np.maximum(S[ok], 1e-300)).max())
    assert (ypad[:, N:] == -77.0).all()
    # a second call into a caller-provided workspace gives the same bits
    ws = mxb.alloc_workspace(mxb.mx_workspace_bytes(M, N, K, fa, fw))
    wm, we = _dev(orc.pack(qw, ww)), _dev(ew)
    y1 = mxb.mx_linear(x.cuda(), fa, wm, we, fw, N, bias=_dev(bias), workspace=ws, algo=mxb.MX_ALGO_TCGEN05).clone()
    y2 = mxb.mx_linear(x.cuda(), fa, wm, we, fw, N, bias=_dev(bias), workspace=ws, algo=mxb.MX_ALGO_TCGEN05)
    assert mxb.mx_poll_status() == 0
    assert torch.equal(torch.nan_to_num(y1), torch.nan_to_num(y2)) and np.array_equal(y1.cpu().numpy()[ok], y[ok])


@pytest.mark.parametrize("case", [(16, 8, 4), (32, 4, 4), (32, 6, 3), (16, 2, 8)])
def test_linear_mixed_precision(mxb, case):
    B, wa, ww = case
    M, K, N = 300, 1152, 520
    x = synth.student_t_activations(M, K, seed=wa)
    wt = synth.gaussian_weights(N, K, seed=ww)
    bias = synth.gaussian_weights(1, N, seed=5, std=1.0)[0]
    qa, ea, _ = orc.quantize(x.numpy(), B, wa)
    qw, ew, _ = orc.quantize(wt.numpy(), B, ww)
    y_ref, _, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias.numpy())
    fa, fw = mxb.MxFormat(B, wa), mxb.MxFormat(B, ww)
    w_mant, w_exp = mxb.mx_quantize(wt.cuda(), fw)
    y = mxb.mx_linear(x.cuda(), fa, w_mant, w_exp, fw, N, bias=bias.cuda())
    assert mxb.mx_poll_status() == 0
    _check_tol(y, y_ref, S)
    yb = mxb.mx_linear(x.to(torch.bfloat16).cuda(), fa, w_mant, w_exp, fw, N, bias=bias.cuda())
    qa, ea, _ = orc.quantize(x.to(torch.bfloat16).float().numpy(), B, wa)
    y_ref, _, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias.numpy())
    _check_tol(yb, y_ref, S)


# ------------------------------------------------------------------------------ casts

@pytest.mark.parametrize("case", [(16, 8, 16, 4), (32, 4, 32, 8), (16, 6, 32, 3), (32, 8, 16, 2), (16, 3, 16, 3)])
def test_cast_between_widths_bit_exact(mxb, case):
    """mx_cast against the oracle's cast (the quantizer on the decoded values): integer work, bit for
    bit, including zero, subnormal-scale, top-of-range and non-finite blocks."""
    b_in, w_in, b_out, w_out = case
    rng = np.random.default_rng(b_in + 7 * w_in + w_out)
    x = np.concatenate([(rng.standard_t(3, (131, 2080)) * np.exp(rng.uniform(-8, 8, (131, 1)))).astype(np.float32),
                        _edge_case_rows(2080)[:12]])
    q, e, _ = orc.quantize(x, b_in, w_in)
    qo, eo, bad = orc.cast(q, e, b_in, w_in, b_out, w_out)
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    mant, exps = mxb.mx_cast(_dev(orc.pack(q, w_in)), _dev(e), 2080, mxb.MxFormat(b_in, w_in), mxb.MxFormat(b_out, w_out),
                             nonfinite_count=cnt)
    assert np.array_equal(exps.cpu().numpy(), eo)
    assert np.array_equal(mant.cpu().numpy(), orc.pack(qo, w_out))
    assert int(cnt.item()) == bad


@pytest.mark.parametrize("shape", [(2100, 2330, 192), (2048, 8000, 128), (300, 520, 320), (130, 40, 96)])
@pytest.mark.parametrize("ldy_pad", [8, 6])
def test_products_write_nothing_outside_their_result(mxb, shape, ldy_pad):
    """Ragged M and N on the CTA-pair and the one-CTA kernel, through the tiled TMA store (ldy % 4 == 0) and the
    direct stores (ldy % 4 != 0), with and without the fused tail: the result sits in a frame of sentinel values
    that must survive, and equals the oracle bit for bit (operands whose partial sums are exact in fp32)."""
    M, N, K = shape
    B = 16
    qa = synth.random_ints((M, K), -7, 7, M + N).numpy()
    qw = synth.random_ints((N, K), -7, 7, M + N + 1).numpy()
    ea = np.full((M, K // B), 129, np.uint8)
    ew = synth.random_bytes((N, 1), 120, 126, 5).numpy().repeat(K // B, axis=1)     # one scale per weight row: still exact
    unit = 2.0 ** ((129 - 127 - 2) + (120 - 127 - 2))
    bias = (synth.random_ints((1, N), -1000, 1000, 7).numpy()[0] * unit).astype(np.float32)
    res = (synth.random_ints((M, N), -3000, 3000, 8).numpy() * unit).astype(np.float32)
    y_ref, y_seq, _ = orc.gemm(qa, ea, 4, qw, ew, 4, B, bias=bias)
    assert np.array_equal(y_ref, y_seq)
    f = mxb.MxFormat(B, 4)
    am, wm = _dev(orc.pack(qa, 4)), _dev(orc.pack(qw, 4))
    for tail in (False, True):
        canvas = torch.full((M + 8, N + ldy_pad), -7.0, dtype=torch.float32, device="cuda")
        y = canvas[:M, :N]
        if tail:
            mxb.mx_gemm_fused(am, _dev(ea), f, wm, _dev(ew), f, M, N, K, bias=_dev(bias), relu=True, residual=_dev(res), y=y)
            want = np.where(y_ref < 0, np.float32(0), y_ref) + res
        else:
            mxb.mx_gemm(am, _dev(ea), f, wm, _dev(ew), f, M, N, K, bias=_dev(bias), y=y, algo=mxb.MX_ALGO_TCGEN05)
            want = y_ref
        assert mxb.mx_poll_status() == 0
        assert np.array_equal(y.cpu().numpy(), want)
        assert (canvas[M:, :] == -7.0).all() and (canvas[:, N:] == -7.0).all()
