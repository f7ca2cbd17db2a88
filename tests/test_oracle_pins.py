"""Pins for the CPU oracle: everything here checks ``oracle/`` against something other than
itself -- numbers the paper prints, blocks worked by hand (tests/golden), exact rational
arithmetic on tiny inputs, numpy's own fp64/int64 matmul on special cases, and invariants the
format definition implies (Sec. 2 "What are MX Formats?", Sec. 4.1, Eq. 1, Sec. 3.2)."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import mx_oracle as orc
from tests import golden_io

WIDTHS = (2, 3, 4, 5, 6, 8)
BLOCKS = (16, 32)


def _block_row(vals, B):
    x = np.zeros((1, B), np.float32)
    x[0, : len(vals)] = np.asarray(vals, np.float32)
    return x


# --------------------------------------------------------------------------- paper numbers

def test_average_bits_matches_paper_example():
    recs = [r for r in golden_io.load() if r["kind"] in ("paper", "closed") and "bits" in r]
    assert recs
    for r in recs:
        w = int(r["m"]) + 1
        got = orc.format_bits(int(r["block"]), w, int(r["block_rows"]), int(r["exp_bits"]))
        assert got == float(r["bits"])


def test_memory_density_matches_table1():
    rec = [r for r in golden_io.load() if "mxint8_density" in r][0]
    bits = orc.format_bits(16, 8, 2, 8)
    density = float(rec["fp32_bits"]) / bits
    assert math.floor(density * 10) / 10 == float(rec["mxint8_density"])


# --------------------------------------------------------------------------- hand-worked blocks

@pytest.mark.parametrize("B", BLOCKS)
def test_hand_worked_blocks(B):
    recs = [r for r in golden_io.load() if r["kind"] == "block"]
    assert len(recs) >= 8
    for r in recs:
        w = int(r["w"])
        xs = golden_io.floats(r["x"])
        q, e, bad = orc.quantize(_block_row(xs, B), B, w)
        assert bad == 0
        assert int(e[0, 0]) == int(r["ebyte"]), r["id"]
        assert q[0, : len(xs)].tolist() == golden_io.ints(r["q"]), r["id"]
        assert not q[0, len(xs):].any()
        xhat = orc.dequantize(q, e, B, w)
        assert xhat[0, : len(xs)].tolist() == golden_io.floats(r["xhat"]), r["id"]
        if r["packed"] != "-":
            want = [int(t, 16) for t in r["packed"].split(",")]
            got = orc.pack(q, w)
            assert got[0, : len(want)].tolist() == want, r["id"]
            assert np.array_equal(orc.unpack(got, B, w), q)


def test_hand_worked_dot_products():
    recs = golden_io.load()
    blocks = {r["id"]: r for r in recs if r["kind"] == "block"}
    dots = [r for r in recs if r["kind"] == "dot"]
    assert dots
    for d in dots:
        ra, rb = blocks[d["a"]], blocks[d["b"]]
        wa, wb = int(ra["w"]), int(rb["w"])
        qa, ea, _ = orc.quantize(_block_row(golden_io.floats(ra["x"]), 16), 16, wa)
        qb, eb, _ = orc.quantize(_block_row(golden_io.floats(rb["x"]), 16), 16, wb)
        y_ref, y_seq, S = orc.gemm(qa, ea, wa, qb, eb, wb, 16)
        assert float(y_ref[0, 0]) == float(d["y"])
        assert float(y_seq[0, 0]) == float(d["y"])
        # the integer block sum and the shared shift, separately
        P = int(np.dot(qa[0].astype(np.int64), qb[0].astype(np.int64)))
        assert P == int(d["P"])
        shift = (int(ea[0, 0]) - 127) - (wa - 2) + (int(eb[0, 0]) - 127) - (wb - 2)
        assert shift == int(d["shift"])
        assert S[0, 0] >= abs(float(d["y"]))


# --------------------------------------------------------------------------- exponent invariants

@pytest.mark.parametrize("B", BLOCKS)
@pytest.mark.parametrize("w", WIDTHS)
def test_exponent_is_the_block_maximums(B, w):
    rng = np.random.default_rng(10 * B + w)
    x = (rng.standard_normal((37, 4 * B)) * np.exp(rng.uniform(-20, 20, (37, 1)))).astype(np.float32)
    x[3, :B] = 0.0
    q, e, bad = orc.quantize(x, B, w)
    assert bad == 0
    amax = np.abs(x.reshape(37, 4, B)).max(axis=2)
    mant, ex = np.frexp(amax)               # independent library route to floor(log2)
    want = np.where(amax > 0, ex - 1 + 127, 0)
    assert np.array_equal(e.astype(np.int64), want)
    bits = amax.astype(np.float32).view(np.uint32) >> 23      # the binary32 exponent field
    assert np.array_equal(e.astype(np.uint32), bits)
    # the max element uses the top magnitude bit: 2^(w-2) <= |q|max <= 2^(w-1)-1
    qmax = np.abs(q.reshape(37, 4, B).astype(np.int32)).max(axis=2)
    nz = amax > 0
    assert (qmax[nz] >= 2 ** (w - 2)).all() and (qmax <= 2 ** (w - 1) - 1).all()
    assert (qmax[~nz] == 0).all()


@pytest.mark.parametrize("w", WIDTHS)
def test_scale_covariance(w):
    rng = np.random.default_rng(w)
    x = rng.standard_normal((8, 64)).astype(np.float32)
    q0, e0, _ = orc.quantize(x, 16, w)
    for k in (-30, -3, 1, 17):
        q1, e1, _ = orc.quantize(np.ldexp(x, k).astype(np.float32), 16, w)
        assert np.array_equal(q0, q1)
        assert np.array_equal(e0.astype(np.int32) + k, e1.astype(np.int32))


# --------------------------------------------------------------------------- round-trip invariants

@pytest.mark.parametrize("B", BLOCKS)
@pytest.mark.parametrize("w", WIDTHS)
def test_round_trip_invariants(B, w):
    rng = np.random.default_rng(100 * B + w)
    x = rng.standard_t(3, (64, 8 * B)).astype(np.float32)
    q, e, _ = orc.quantize(x, B, w)
    xhat = orc.dequantize(q, e, B, w)
    # idempotence, bit-exact
    q2, e2, _ = orc.quantize(xhat.astype(np.float32), B, w)
    assert np.array_equal(q, q2) and np.array_equal(e, e2)
    # error bound: half a step unless the element saturated (only the block maximum can)
    E = e.astype(np.int64) - 127
    s = np.repeat(np.ldexp(1.0, E - (w - 2)), B, axis=1)
    err = np.abs(x.astype(np.float64) - xhat)
    sat = np.abs(q.astype(np.int32)) == 2 ** (w - 1) - 1
    assert (err[~sat] <= s[~sat] / 2).all()
    assert (err[sat] < s[sat]).all()
    # "the shared exponent bounds the range of values in the block"
    assert (np.abs(xhat) < np.repeat(np.ldexp(1.0, E + 1), B, axis=1)).all()
    # round-half-even is monotone and sign-symmetric
    qn, en, _ = orc.quantize(-x, B, w)
    assert np.array_equal(qn, -q) and np.array_equal(en, e)


@pytest.mark.parametrize("B", BLOCKS)
@pytest.mark.parametrize("w", WIDTHS)
def test_representable_values_survive(B, w):
    rng = np.random.default_rng(1000 * B + w)
    qmax = 2 ** (w - 1) - 1
    qi = rng.integers(-qmax, qmax + 1, (50, 4 * B))
    E = rng.integers(-100, 100, (50, 4))
    x = np.ldexp(qi.astype(np.float64), np.repeat(E, B, axis=1) - (w - 2)).astype(np.float32)
    q, e, _ = orc.quantize(x, B, w)
    xhat = orc.dequantize(q, e, B, w)
    assert np.array_equal(xhat, x.astype(np.float64))   # even when the block is un-normalised


def test_ties_go_to_even_and_saturate():
    # s = 1 for w=4 when the maximum lies in [4, 8): E=2.
    x = _block_row([4.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, 7.5, 7.49, -7.6, 6.5], 16)
    q, e, _ = orc.quantize(x, 16, 4)
    assert int(e[0, 0]) == 129
    assert q[0, :12].tolist() == [4, 0, 2, 2, 0, -2, -2, 4, 7, 7, -7, 6]


def test_zero_subnormal_and_nonfinite_blocks():
    x = np.zeros((1, 64), np.float32)
    x[0, 16] = np.float32(2.0 ** -126) - np.float32(2.0 ** -149)   # largest subnormal -> byte 0
    x[0, 17] = -(2.0 ** -127)
    x[0, 18] = 2.0 ** -130
    x[0, 19] = 3 * 2.0 ** -130
    x[0, 32] = np.inf
    x[0, 33] = 5.0
    x[0, 48] = np.nan
    q, e, bad = orc.quantize(x, 16, 4)
    assert e[0].tolist() == [0, 0, 255, 255]
    assert bad == 2
    assert not q[0, :16].any() and not q[0, 32:].any()
    # grid of the lowest exponent: s = 2^(-127-2); 7.99.. saturates at 7; 0.5 -> 0, 1.5 -> 2
    assert q[0, 16:20].tolist() == [7, -4, 0, 2]
    xhat = orc.dequantize(q, e, 16, 4)
    assert np.isnan(xhat[0, 32:]).all()
    y, yseq, S = orc.gemm(q, e, 4, q, e, 4, 16)
    assert np.isnan(y).all() and np.isnan(yseq).all()


def test_largest_exponent_byte():
    x = _block_row([3.0e38, -1.0e38, 2.0 ** 127], 16)
    q, e, bad = orc.quantize(x, 16, 8)
    assert bad == 0 and int(e[0, 0]) == 254
    xhat = orc.dequantize(q, e, 16, 8)
    assert abs(xhat[0, 0] - 3.0e38) <= 2.0 ** 121 / 2 and xhat[0, 2] == 2.0 ** 127


def test_strided_axis_equals_transposed_copy():
    rng = np.random.default_rng(5)
    v = rng.standard_normal((96, 40)).astype(np.float32)        # [tokens, d]
    q1, e1, _ = orc.quantize(v.T, 32, 8)                         # blocks along tokens, strided
    q2, e2, _ = orc.quantize(np.ascontiguousarray(v.T), 32, 8)
    assert np.array_equal(q1, q2) and np.array_equal(e1, e2)


def test_pack_round_trip_all_widths():
    rng = np.random.default_rng(6)
    for w in WIDTHS:
        qmax = 2 ** (w - 1) - 1
        q = rng.integers(-qmax - 1, qmax + 1, (5, 64)).astype(np.int8)   # incl. -2^(w-1)
        if w < 4:
            q = np.clip(q, -qmax, qmax).astype(np.int8)
        p = orc.pack(q, w)
        assert p.shape == (5, 32 if w <= 4 else 64)
        assert np.array_equal(orc.unpack(p, 64, w), q)


# --------------------------------------------------------------------------- GEMM: exact brute force

def _nearest_f32(fr: Fraction) -> float:
    """Correctly rounded binary32 of an exact rational (ties to even), via integer arithmetic."""
    if fr == 0:
        return 0.0
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    e = max(e, -126)
    ulp = Fraction(2) ** (e - 23)
    n = a / ulp
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return sign * float(fl * ulp)


@pytest.mark.parametrize("B", BLOCKS)
def test_gemm_equals_exact_rational_dot_products(B):
    rng = np.random.default_rng(B)
    for wa in WIDTHS:
        for ww in (2, 4, 8):
            M, N, K = 3, 4, 2 * B
            x = (rng.standard_normal((M, K)) * np.exp(rng.uniform(-6, 6, (M, K)))).astype(np.float32)
            wt = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
            bias = rng.standard_normal(N).astype(np.float32)
            qa, ea, _ = orc.quantize(x, B, wa)
            qw, ew, _ = orc.quantize(wt, B, ww)
            y, yseq, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias)
            # emulator form (Sec. 3.2): plain dot product of the dequantized values, exactly
            xa = orc.dequantize(qa, ea, B, wa)
            xw = orc.dequantize(qw, ew, B, ww)
            for i in range(M):
                for j in range(N):
                    exact = sum(Fraction(float(xa[i, k])) * Fraction(float(xw[j, k])) for k in range(K))
                    exact += Fraction(float(bias[j]))
                    assert float(y[i, j]) == _nearest_f32(exact), (wa, ww, i, j)
                    sabs = sum(abs(Fraction(float(xa[i, k])) * Fraction(float(xw[j, k]))) for k in range(K))
                    assert abs(Fraction(float(yseq[i, j])) - exact) <= Fraction(1, 10 ** 5) * (sabs + abs(Fraction(float(bias[j])))) + Fraction(1, 2 ** 140)
                    assert S[i, j] <= float(sabs + abs(Fraction(float(bias[j])))) * (1 + 1e-12)


def test_gemm_hardware_form_equals_emulator_form():
    """Integer block sums times one shared power of two == fp matmul of dequantized values."""
    rng = np.random.default_rng(77)
    M, N, K, B = 5, 6, 128, 32
    x = rng.standard_normal((M, K)).astype(np.float32)
    wt = rng.standard_normal((N, K)).astype(np.float32)
    qa, ea, _ = orc.quantize(x, B, 8)
    qw, ew, _ = orc.quantize(wt, B, 4)
    y, _, _ = orc.gemm(qa, ea, 8, qw, ew, 4, B)
    xa, xw = orc.dequantize(qa, ea, B, 8), orc.dequantize(qw, ew, B, 4)
    # N(0,1) data: all terms within 2^-12..2^4, 128 of them -> fp64 matmul is exact here
    assert np.array_equal(y, (xa @ xw.T).astype(np.float32))


def test_gemm_equal_exponents_is_integer_matmul():
    rng = np.random.default_rng(8)
    M, N, K, B = 7, 9, 96, 16
    qa = rng.integers(-127, 128, (M, K)).astype(np.int8)
    qw = rng.integers(-7, 8, (N, K)).astype(np.int8)
    ea = np.full((M, K // B), 130, np.uint8)
    ew = np.full((N, K // B), 120, np.uint8)
    y, yseq, S = orc.gemm(qa, ea, 8, qw, ew, 4, B)
    P = qa.astype(np.int64) @ qw.astype(np.int64).T
    want = np.ldexp(P.astype(np.float64), (130 - 127 - 6) + (120 - 127 - 2))
    assert np.array_equal(y.astype(np.float64), want) and np.array_equal(yseq, y)


def test_gemm_representable_inputs_equal_fp64_matmul():
    rng = np.random.default_rng(9)
    M, N, K, B, wa, ww = 6, 5, 64, 16, 6, 4
    A = np.ldexp(rng.integers(-31, 32, (M, K)).astype(np.float64),
                 np.repeat(rng.integers(-3, 4, (M, K // B)), B, axis=1)).astype(np.float32)
    W = np.ldexp(rng.integers(-7, 8, (N, K)).astype(np.float64),
                 np.repeat(rng.integers(-3, 4, (N, K // B)), B, axis=1)).astype(np.float32)
    qa, ea, _ = orc.quantize(A, B, wa)
    qw, ew, _ = orc.quantize(W, B, ww)
    y, _, _ = orc.gemm(qa, ea, wa, qw, ew, ww, B)
    assert np.array_equal(y, (A.astype(np.float64) @ W.astype(np.float64).T).astype(np.float32))


def test_gemm_one_hot_rows_return_dequantized_weights():
    rng = np.random.default_rng(10)
    N, K, B, ww = 8, 64, 16, 4
    W = rng.standard_normal((N, K)).astype(np.float32)
    qw, ew, _ = orc.quantize(W, B, ww)
    A = np.eye(K, dtype=np.float32)
    qa, ea, _ = orc.quantize(A, B, 8)
    y, yseq, _ = orc.gemm(qa, ea, 8, qw, ew, ww, B)
    assert np.array_equal(y.astype(np.float64), orc.dequantize(qw, ew, B, ww).T)
    assert np.array_equal(y, yseq)


def test_gemm_samples_agree_with_full():
    rng = np.random.default_rng(11)
    M, N, K, B = 9, 11, 64, 32
    qa = rng.integers(-127, 128, (M, K)).astype(np.int8)
    qw = rng.integers(-7, 8, (N, K)).astype(np.int8)
    ea = rng.integers(100, 140, (M, K // B)).astype(np.uint8)
    ew = rng.integers(100, 140, (N, K // B)).astype(np.uint8)
    bias = rng.standard_normal(N).astype(np.float32)
    y, yseq, S = orc.gemm(qa, ea, 8, qw, ew, 4, B, bias=bias)
    si = rng.integers(0, M, 20)
    sj = rng.integers(0, N, 20)
    ys, yseqs, Ss = orc.gemm_samples(qa, ea, 8, qw, ew, 4, B, si, sj, bias=bias)
    assert np.array_equal(ys, y[si, sj]) and np.array_equal(yseqs, yseq[si, sj])
    assert np.array_equal(Ss, S[si, sj])


def test_sequential_fp32_sum_sits_inside_the_tolerance():
    rng = np.random.default_rng(12)
    M, N, K, B = 8, 8, 11008, 16
    x = rng.standard_t(3, (M, K)).astype(np.float32)
    wt = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    qa, ea, _ = orc.quantize(x, B, 8)
    qw, ew, _ = orc.quantize(wt, B, 4)
    y, yseq, S = orc.gemm(qa, ea, 8, qw, ew, 4, B)
    assert (np.abs(yseq.astype(np.float64) - y) <= 1e-5 * S).all()
    assert (S >= np.abs(y) * (1 - 1e-6)).all()


def test_rejects_bad_arguments():
    x = np.zeros((2, 40), np.float32)
    with pytest.raises(ValueError):
        orc.quantize(x, 16, 4)          # K not a multiple of the block
    with pytest.raises(ValueError):
        orc.quantize(np.zeros((2, 32), np.float32), 16, 9)


# --------------------------------------------------------------------------- fp32 glue of the block

def test_glue_oracle_against_library_routines():
    import scipy.special
    import torch
    from oracle import block_oracle as blk
    rng = np.random.default_rng(21)
    x = rng.standard_normal((7, 96)) * 3 + 1
    g, b = rng.standard_normal(96), rng.standard_normal(96)
    want = torch.nn.functional.layer_norm(torch.from_numpy(x), (96,), torch.from_numpy(g), torch.from_numpy(b), 1e-5)
    assert np.allclose(blk.layernorm(x, g, b, 1e-5), want.numpy(), rtol=1e-12, atol=1e-12)
    y = blk.layernorm(x, None, None, 0.0)
    assert np.allclose(y.mean(axis=1), 0, atol=1e-12) and np.allclose((y ** 2).mean(axis=1), 1, atol=1e-12)
    s = rng.standard_normal((2 * 5, 5))                       # two batches of 5 query rows
    p = blk.softmax_causal(s, 0.5, 5)
    for r in range(10):
        n = r % 5 + 1
        assert np.allclose(p[r, :n], scipy.special.softmax(0.5 * s[r, :n]), rtol=1e-13)
        assert (p[r, n:] == 0).all()
    assert np.allclose(p.sum(axis=1), 1)
    assert np.array_equal(blk.relu(np.array([-1.0, 0.0, 2.5])), np.array([0.0, 0.0, 2.5]))


def test_attention_oracle_reduces_to_plain_matmul_on_representable_inputs():
    from oracle import block_oracle as blk
    rng = np.random.default_rng(22)
    seq, H, d = 32, 2, 16
    q = rng.integers(-127, 128, (seq, H * d)).astype(np.float32)
    k = rng.integers(-127, 128, (seq, H * d)).astype(np.float32)
    q[:, ::16] = 127
    k[:, ::16] = -127                                         # every block's maximum uses the top bit
    sc = blk.attention_scores(q, k, H, d, 16, 8)
    for h in range(H):
        want = q[:, h * d:(h + 1) * d].astype(np.float64) @ k[:, h * d:(h + 1) * d].astype(np.float64).T
        assert np.array_equal(sc[h][0].astype(np.float64), want)
    p = rng.integers(0, 128, (H * seq, seq)).astype(np.float32)
    v = rng.integers(-127, 128, (seq, H * d)).astype(np.float32)
    p[:, ::16] = 127
    v[::16, :] = 127
    ctx = blk.attention_context(p, v, H, d, 16, 8)
    for h in range(H):
        want = p[h * seq:(h + 1) * seq].astype(np.float64) @ v[:, h * d:(h + 1) * d].astype(np.float64)
        assert np.array_equal(ctx[h][0].astype(np.float64), want)


# ---------------------------------------------------------------- product with an MXInt result

def _requant_fixture():
    rows = golden_io.load()
    K = N = 16
    a = [r for r in rows if r["kind"] == "rq_a"]
    w = [r for r in rows if r["kind"] == "rq_w"]
    qa = np.zeros((len(a), K), np.int8)
    ea = np.zeros((len(a), 1), np.uint8)
    for r in a:
        v = golden_io.ints(r["q"])
        qa[int(r["row"]), :len(v)] = v
        ea[int(r["row"]), 0] = int(r["ebyte"])
    qw = np.zeros((N, K), np.int8)
    ew = np.zeros((N, 1), np.uint8)
    for r in w:
        v = golden_io.ints(r["q"])
        qw[int(r["row"]), :len(v)] = v
        ew[int(r["row"]), 0] = int(r["ebyte"])
    bias = np.zeros(N, np.float32)
    for r in rows:
        if r["kind"] == "rq_bias":
            bias[int(r["col"])] = float(r["value"])
    return rows, qa, ea, int(a[0]["w"]), qw, ew, int(w[0]["w"]), bias


def test_requantized_product_hand_worked():
    """The pencil-worked layer of tests/golden: exact fp32 outputs (bias included), then one block
    of 16 along the output-feature axis per row, at two output widths."""
    rows, qa, ea, wa, qw, ew, ww, bias = _requant_fixture()
    want_y = {int(r["row"]): golden_io.floats(r["y"]) for r in rows if r["kind"] == "rq_y"}
    for wy in (4, 8):
        qy, ey, bad, y_ref, _ = orc.gemm_requant(qa, ea, wa, qw, ew, ww, 16, 16, wy, bias=bias)
        assert bad == 0
        for r in (r for r in rows if r["kind"] == "rq_q" and int(r["wy"]) == wy):
            i = int(r["row"])
            q = golden_io.ints(r["q"])
            assert y_ref[i, :len(want_y[i])].tolist() == want_y[i]
            assert (y_ref[i, len(want_y[i]):] == 0).all()
            assert ey[i, 0] == int(r["ebyte"])
            assert qy[i, :len(q)].tolist() == q and (qy[i, len(q):] == 0).all()


@pytest.mark.parametrize("By,wy", [(16, 4), (32, 8), (16, 2), (32, 5)])
def test_requantized_product_invariants(By, wy):
    """Whatever the widths: the result's exponent is that of the largest |y| of its block of the
    exact fp32 product, every code is within half a step of y (one step where it saturates), and
    an MXInt result that is fed back as an input is reproduced exactly by a second quantization."""
    rng = np.random.default_rng(By + wy)
    M, N, K, B, wa, ww = 5, 64, 96, 32, 8, 4
    qa = rng.integers(-127, 128, (M, K)).astype(np.int8)
    qw = rng.integers(-7, 8, (N, K)).astype(np.int8)
    ea = rng.integers(120, 131, (M, K // B)).astype(np.uint8)
    ew = rng.integers(115, 125, (N, K // B)).astype(np.uint8)
    bias = rng.standard_normal(N).astype(np.float32)
    qy, ey, bad, y_ref, _ = orc.gemm_requant(qa, ea, wa, qw, ew, ww, B, By, wy, bias=bias)
    assert bad == 0
    y = y_ref.astype(np.float64).reshape(M, N // By, By)
    amax = np.abs(y).max(axis=2)
    _, ex = np.frexp(amax)                                    # amax = f * 2^ex, f in [0.5, 1)
    assert np.array_equal(ey.astype(np.int64), ex - 1 + 127)
    step = np.ldexp(1.0, ey.astype(np.int64) - 127 - (wy - 2))[:, :, None]
    q = qy.astype(np.float64).reshape(M, N // By, By)
    qmax = 2 ** (wy - 1) - 1
    err = np.abs(q * step - y)
    free = np.abs(q) < qmax
    assert (err[free] <= 0.5 * step.repeat(By, 2)[free]).all()
    assert (err <= step).all()
    # the MXInt result as the next layer's input: quantizing its decoded values changes nothing
    again_q, again_e, _ = orc.quantize(orc.dequantize(qy, ey, By, wy).astype(np.float32), By, wy)
    assert np.array_equal(again_q, qy) and np.array_equal(again_e, ey)


# ---------------------------------------------------------------- two-dimensional blocks

def test_two_row_blocks_hand_worked():
    for r in (r for r in golden_io.load() if r["kind"] == "block2d"):
        w = int(r["w"])
        x = np.zeros((2, 16), np.float32)
        for i, key in enumerate(("x0", "x1")):
            v = golden_io.floats(r[key])
            x[i, :len(v)] = v
        q, e, bad = orc.quantize_2d(x, 16, 2, w)
        assert e.shape == (1, 1) and e[0, 0] == int(r["ebyte"]) and bad == 0
        for i, key in enumerate(("q0", "q1")):
            want = golden_io.ints(r[key])
            assert q[i, :len(want)].tolist() == want and (q[i, len(want):] == 0).all()


@pytest.mark.parametrize("B,w", [(16, 4), (16, 8), (32, 3)])
def test_two_row_blocks_reduce_to_known_cases(B, w):
    """(B, 1) blocks are the one-dimensional quantizer; a (B, 2) block is the one-dimensional block
    of 2B values obtained by laying the two rows side by side; the shared exponent is the larger of
    the two rows' own exponents; the paper's storage figure follows (8.25 bits at (16,2), m = 7)."""
    rng = np.random.default_rng(B + w)
    x = (rng.standard_t(3, (6, 4 * B)) * np.exp(rng.uniform(-3, 3, (6, 1)))).astype(np.float32)
    q1, e1, _ = orc.quantize(x, B, w)
    qa, ea, _ = orc.quantize_2d(x, B, 1, w)
    assert np.array_equal(qa, q1) and np.array_equal(ea, e1)
    q2, e2, _ = orc.quantize_2d(x, B, 2, w)
    assert np.array_equal(e2, np.maximum(e1[0::2], e1[1::2]))
    side = np.concatenate([x[0::2].reshape(3, 4, B), x[1::2].reshape(3, 4, B)], axis=2).reshape(3, 8 * B)
    qs, es, _ = orc.quantize(side, 2 * B, w) if 2 * B <= 32 else (None, None, None)
    if qs is not None:
        assert np.array_equal(es, e2)
        assert np.array_equal(qs.reshape(3, 4, 2, B)[:, :, 0].reshape(3, 4 * B), q2[0::2])
        assert np.array_equal(qs.reshape(3, 4, 2, B)[:, :, 1].reshape(3, 4 * B), q2[1::2])
    full = orc.expand_exponent_rows(e2, 2)
    assert np.array_equal(full[0::2], e2) and np.array_equal(full[1::2], e2)
    # decoded values obey the one-dimensional bounds with the shared exponent
    xhat = orc.dequantize(q2, full, B, w)
    step = np.repeat(np.ldexp(1.0, full.astype(np.int64) - 127 - (w - 2)), B, axis=1)
    qmax = 2 ** (w - 1) - 1
    free = np.abs(q2) < qmax
    assert (np.abs(xhat - x)[free] <= 0.5 * step[free]).all() and (np.abs(xhat - x) <= step).all()
    # nonfinite: one NaN poisons the pair of rows' block
    x[1, 3] = np.nan
    q3, e3, bad = orc.quantize_2d(x, B, 2, w)
    assert bad == 1 and e3[0, 0] == 255 and (q3[0:2, :B] == 0).all()
    assert orc.lib().mxo_format_bits(16, 2, 8, 8) == 8.25


# ---------------------------------------------------------------- casts between widths

def test_casts_hand_worked():
    rows = golden_io.load()
    blocks = {r["id"]: r for r in rows if r["kind"] == "block"}
    for r in (r for r in rows if r["kind"] == "cast"):
        src = blocks[r["from"]]
        assert int(src["w"]) == int(r["w_in"])
        q = np.zeros((1, 16), np.int8)
        v = golden_io.ints(src["q"])
        q[0, :len(v)] = v
        e = np.array([[int(src["ebyte"])]], np.uint8)
        qo, eo, bad = orc.cast(q, e, 16, int(r["w_in"]), 16, int(r["w_out"]))
        want = golden_io.ints(r["q"])
        assert bad == 0 and eo[0, 0] == int(r["ebyte"])
        assert qo[0, :len(want)].tolist() == want and (qo[0, len(want):] == 0).all()


@pytest.mark.parametrize("w_in,w_out", [(4, 8), (3, 6), (8, 8), (2, 5)])
def test_widening_casts_lose_nothing(w_in, w_out):
    rng = np.random.default_rng(w_in * 10 + w_out)
    x = (rng.standard_t(3, (9, 128)) * np.exp(rng.uniform(-5, 5, (9, 1)))).astype(np.float32)
    q, e, _ = orc.quantize(x, 32, w_in)
    for b_out in (16, 32):
        qo, eo, bad = orc.cast(q, e, 32, w_in, b_out, w_out)
        assert bad == 0
        assert np.array_equal(orc.dequantize(qo, eo, b_out, w_out), orc.dequantize(q, e, 32, w_in))
    q2, e2, _ = orc.cast(q, e, 32, w_in, 32, w_in)                 # same format: identity
    assert np.array_equal(q2, q) and np.array_equal(e2, e)


def test_narrowing_cast_error_bound_and_nonfinite():
    rng = np.random.default_rng(77)
    x = rng.standard_normal((5, 64)).astype(np.float32)
    q, e, _ = orc.quantize(x, 16, 8)
    e[2, 1] = 255
    qo, eo, bad = orc.cast(q, e, 16, 8, 32, 3)
    assert bad == 1 and eo[2, 0] == 255 and (qo[2, :32] == 0).all()
    xin = orc.dequantize(q, e, 16, 8)
    xout = orc.dequantize(qo, eo, 32, 3)
    ok = ~np.isnan(xout)
    step = np.repeat(np.ldexp(1.0, eo.astype(np.int64) - 127 - 1), 32, axis=1)
    assert (np.abs(xout - xin)[ok] <= step[ok]).all()
    free = ok & (np.abs(qo) < 3)
    assert (np.abs(xout - xin)[free] <= 0.5 * step[free]).all()


# ------------------------------------------------------------------------------ Block Minifloat / Block Logarithm

ALT_FORMATS = [(orc.KIND_BMF, 4, 3), (orc.KIND_BMF, 2, 5), (orc.KIND_BMF, 5, 2), (orc.KIND_BMF, 3, 2),
               (orc.KIND_BL, 4, 0), (orc.KIND_BL, 3, 0), (orc.KIND_BL, 5, 0)]


def test_alt_formats_hand_worked_blocks():
    """The pencil-worked BMF / BL blocks of the fixture: shared byte, code bytes and decoded values."""
    rows = [r for r in golden_io.load() if r["kind"] == "alt"]
    assert len(rows) == 4
    for r in rows:
        kind, eb, mb, B = (orc.KIND_BMF if r["fmt"] == "bmf" else orc.KIND_BL), int(r["ebits"]), int(r["mbits"]), int(r["block"])
        x = np.zeros((1, B), np.float32)
        vals = golden_io.floats(r["x"])
        x[0, :len(vals)] = vals
        codes, shared, bad = orc.alt_quantize(x, kind, B, eb, mb)
        assert bad == 0 and shared[0, 0] == int(r["shared"]), r["id"]
        want = [int(t, 16) for t in r["codes"].split(",")]
        assert list(codes[0, :len(want)]) == want, r["id"]
        assert (codes[0, len(want):] == 0).all()
        xhat = orc.alt_dequantize(codes, shared, kind, B, eb, mb)
        assert list(xhat[0, :len(want)]) == golden_io.floats(r["xhat"]), r["id"]


@pytest.mark.parametrize("fmt", ALT_FORMATS)
def test_alt_formats_invariants(fmt):
    kind, eb, mb = fmt
    B = 16
    rng = np.random.default_rng(10 * eb + mb + kind)
    x = (rng.standard_normal((40, 8 * B)) * np.exp2(rng.integers(-12, 12, (40, 1)))).astype(np.float32)
    x[3, :B] = 0.0
    x[4, 5] = np.inf
    x[5, B + 2] = np.nan
    x[6, :B] = (rng.standard_normal(B) * 2.0 ** -110).astype(np.float32)        # below 2^-95: a zero block
    codes, shared, bad = orc.alt_quantize(x, kind, B, eb, mb)
    xh = orc.alt_dequantize(codes, shared, kind, B, eb, mb)
    fmax = 2 ** eb - 1
    assert bad == 2 and shared[4, 0] == 255 and shared[5, 1] == 255 and np.isnan(xh[4, :B]).all()
    assert shared[3, 0] == 0 and shared[6, 0] == 0 and (xh[3, :B] == 0).all() and (xh[6, :B] == 0).all()
    assert (codes >> (1 + eb + mb) == 0).all()                      # unused high bits stay clear
    ok = np.ones_like(x, bool)
    ok[4, :B] = ok[5, B:2 * B] = ok[3, :B] = ok[6, :B] = False
    amax = np.abs(np.where(ok, x, 0)).reshape(40, 8, B).max(axis=2)
    live = amax > 0
    live[4, 0] = live[5, 1] = False
    # shared byte: exponent of the block maximum (BMF: frexp; BL: nearest power of two in the log domain)
    mant, ex = np.frexp(amax[live].astype(np.float64))
    if kind == orc.KIND_BMF:
        assert (shared[live] == ex - 1 + 127).all()
    else:
        up = (2 * mant) ** 2 >= 2.0
        assert (shared[live] == ex - 1 + up + 127).all()
    beta = np.repeat(shared.astype(np.int64) - 127, B, axis=1)
    a, ah = np.abs(x.astype(np.float64)), np.abs(xh)
    assert (np.sign(xh[ok]) * np.sign(x[ok]) >= 0).all()            # signs survive (zero may appear)
    assert (ah[ok] <= np.exp2(beta[ok] + 1.0)).all()                # the shared byte bounds the block's range
    top = np.exp2(beta.astype(np.float64))
    if kind == orc.KIND_BMF:
        lo = top * 2.0 ** -(fmax - 1)                               # smallest normal binade of the block
        normal = ok & (a >= lo) & (a < top * (2 - 2.0 ** -mb))      # not saturated, not subnormal
        assert (np.abs(ah - a)[normal] <= a[normal] * 2.0 ** -(mb + 1)).all()      # half an ulp of mb+1 bits
        sub = ok & (a < lo)
        assert (np.abs(ah - a)[sub] <= (lo * 2.0 ** -(mb + 1))[sub]).all()          # half a subnormal step
        # decoded values carry at most mb + 1 significant bits
        m, _ = np.frexp(ah[ok])
        assert (np.ldexp(m, mb + 1) % 1 == 0).all()
    else:
        kept = ok & (ah > 0) & (a < top)
        ratio = ah[kept] / a[kept]
        assert (ratio <= 2 ** 0.5 * (1 + 1e-12)).all() and (ratio >= 2 ** -0.5 * (1 - 1e-12)).all()
        assert (np.log2(ah[ok & (ah > 0)]) % 1 == 0).all()          # always a power of two
        flushed = ok & (ah == 0) & (a > 0)
        assert (a[flushed] < (top * 2.0 ** -(fmax - 1) * 2 ** -0.5 * (1 + 1e-12))[flushed]).all()
    # every decoded value is a bf16 number: its binary32 image has 16 zero low bits
    f32 = xh[ok].astype(np.float32)
    assert (f32.astype(np.float64) == xh[ok]).all() and (f32.view(np.uint32) & 0xFFFF == 0).all()
    # idempotence: the decoded tensor quantizes to the same codes and shared bytes
    c2, s2, _ = orc.alt_quantize(np.where(np.isnan(xh), 0, xh).astype(np.float32), kind, B, eb, mb)
    good_rows = [r for r in range(40) if r not in (4, 5)]
    assert np.array_equal(c2[good_rows], codes[good_rows]) and np.array_equal(s2[good_rows], shared[good_rows])
    # sign symmetry
    c3, s3, _ = orc.alt_quantize(np.where(np.isfinite(x), -x, x).astype(np.float32), kind, B, eb, mb)
    assert np.array_equal(s3, shared) and np.array_equal(c3 & (2 ** (eb + mb) - 1), codes & (2 ** (eb + mb) - 1))


@pytest.mark.parametrize("mb", (2, 3, 5))
def test_bmf_top_binade_is_the_mxint_grid(mb):
    """Inside the binade of the block maximum a minifloat with mb mantissa bits and MXInt of width
    mb + 2 have the same grid (step 2^(E - mb)) and the same rounding: the two quantizers, pinned
    separately, must decode to the same values there."""
    B = 16
    rng = np.random.default_rng(mb)
    x = (rng.uniform(1.0, 2.0, (30, 4 * B)) * rng.choice([-1.0, 1.0], (30, 4 * B)) *
         np.exp2(rng.integers(-6, 6, (30, 1)))).astype(np.float32)
    codes, shared, _ = orc.alt_quantize(x, orc.KIND_BMF, B, 8 - 1 - mb if mb >= 3 else 4, mb)
    eb = 8 - 1 - mb if mb >= 3 else 4
    q, e, _ = orc.quantize(x, B, mb + 2)
    assert np.array_equal(shared, e)
    assert np.array_equal(orc.alt_dequantize(codes, shared, orc.KIND_BMF, B, eb, mb), orc.dequantize(q, e, B, mb + 2))


def test_alt_gemm_is_the_fp64_matmul_of_the_decoded_values():
    """Emulator form of Sec. 3.2 on BMF / BL operands: the product of the decoded tensors, summed exactly
    (numpy float64 holds every product and every sum of these few terms exactly), rounded to fp32 once."""
    B, M, N, K = 16, 9, 11, 64
    rng = np.random.default_rng(5)
    a = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    for afmt, wfmt in (((orc.KIND_BMF, 4, 3), (orc.KIND_BMF, 4, 3)), ((orc.KIND_BMF, 3, 4), (orc.KIND_BL, 4, 0)),
                       ((orc.KIND_BL, 5, 0), (orc.KIND_BL, 3, 0))):
        ac, ash, _ = orc.alt_quantize(a, afmt[0], B, afmt[1], afmt[2])
        wc, wsh, _ = orc.alt_quantize(w, wfmt[0], B, wfmt[1], wfmt[2])
        y, S = orc.alt_gemm(ac, ash, afmt, wc, wsh, wfmt, B, bias=bias)
        ah = orc.alt_dequantize(ac, ash, afmt[0], B, afmt[1], afmt[2])
        wh = orc.alt_dequantize(wc, wsh, wfmt[0], B, wfmt[1], wfmt[2])
        # exact reference with Python fractions
        from fractions import Fraction
        for i in (0, 4, 8):
            for j in (0, 5, 10):
                exact = sum(Fraction(float(ah[i, k])) * Fraction(float(wh[j, k])) for k in range(K)) + Fraction(float(bias[j]))
                assert abs(Fraction(float(y[i, j])) - exact) <= Fraction(float(np.spacing(np.float32(abs(float(exact)))))) / 2
                assert abs(S[i, j] - float(sum(abs(Fraction(float(ah[i, k])) * Fraction(float(wh[j, k]))) for k in range(K))
                                           + abs(Fraction(float(bias[j]))))) <= 1e-12 * S[i, j]
        assert np.allclose(y, (ah @ wh.T + bias).astype(np.float32), rtol=1e-6, atol=1e-6)
    wsh2 = wsh.copy()
    wsh2[2, 1] = 255
    y, S = orc.alt_gemm(ac, ash, afmt, wc, wsh2, wfmt, B)
    assert np.isnan(y[:, 2]).all() and not np.isnan(np.delete(y, 2, axis=1)).any()


# ------------------------------------------------------------------------------ dense storage

def test_dense_packing_hand_worked_and_eq1():
    rows = [r for r in golden_io.load() if r["kind"] == "dense"]
    assert len(rows) == 4
    for r in rows:
        w, q = int(r["w"]), np.array([golden_io.ints(r["q"])], np.int8)
        img = orc.pack_dense(q, w)
        assert [int(t, 16) for t in r["bytes"].split(",")] == list(img[0]), r
        assert np.array_equal(orc.unpack_dense(img, q.shape[1], w), q)
    rng = np.random.default_rng(8)
    for w in range(2, 9):
        K, B = 96, 32
        q = rng.integers(-(2 ** (w - 1)), 2 ** (w - 1), (7, K)).astype(np.int8)
        img = orc.pack_dense(q, w)
        # Eq. 1: bits per value = exponent share + m + 1; the mantissa part is exactly w = m + 1 bits
        assert img.shape[1] * 8 == K * w
        assert abs((img.shape[1] * 8 + 8 * (K // B)) / K - orc.format_bits(B, w)) < 1e-12
        assert np.array_equal(orc.unpack_dense(img, K, w), q)
        # an independent construction: numpy bit arrays, little-endian within bytes
        bits = ((q.astype(np.int64)[:, :, None] >> np.arange(w)) & 1).reshape(7, K * w).astype(np.uint8)
        assert np.array_equal(np.packbits(bits, axis=1, bitorder="little"), img)
    # the 4- and 8-bit widths coincide with the containers
    q4 = rng.integers(-8, 8, (3, 32)).astype(np.int8)
    assert np.array_equal(orc.pack_dense(q4, 4), orc.pack(q4, 4))
    q8 = rng.integers(-128, 128, (3, 32)).astype(np.int8)
    assert np.array_equal(orc.pack_dense(q8, 8), orc.pack(q8, 8))
