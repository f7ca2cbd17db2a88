"""ctypes front for the C oracle (``mx_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  Nothing on the product path may import this module.  It holds no
arithmetic of its own -- every number comes from the C file, which states the paper
passages it follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mx_oracle.c")
_LIB = os.path.join(_HERE, "libmx_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over output rows only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i64, i32 = C.c_int64, C.c_int
        p = C.c_void_p
        L.mxo_quantize.argtypes = [p, i64, i64, i64, i64, i32, i32, p, p, p]
        L.mxo_dequantize.argtypes = [p, p, i64, i64, i32, i32, p]
        L.mxo_pack.argtypes = [p, i64, i64, i32, p]
        L.mxo_unpack.argtypes = [p, i64, i64, i32, p]
        L.mxo_pack_dense.argtypes = [p, i64, i64, i32, p]
        L.mxo_unpack_dense.argtypes = [p, i64, i64, i32, p]
        L.mxo_gemm.argtypes = [p, p, i32, p, p, i32, i64, i64, i64, i32, p, p, p, p]
        L.mxo_gemm_samples.argtypes = [p, p, i32, p, p, i32, i64, i64, i64, i32, p, p, p, i64,
                                       p, p, p]
        L.mxo_gemm_requant.argtypes = [p, p, i32, p, p, i32, i64, i64, i64, i32, p, i32, i32, p, p,
                                       p, p, p]
        L.mxo_quantize_2d.argtypes = [p, i64, i64, i64, i64, i32, i32, i32, p, p, p]
        L.mxo_expand_exponent_rows.argtypes = [p, i64, i64, i32, p]
        L.mxo_cast.argtypes = [p, p, i64, i64, i32, i32, i32, i32, p, p, p]
        L.mxo_alt_quantize.argtypes = [p, i64, i64, i64, i32, i32, i32, i32, p, p, p]
        L.mxo_alt_dequantize.argtypes = [p, p, i64, i64, i32, i32, i32, i32, p]
        L.mxo_alt_gemm.argtypes = [p, p, i32, i32, i32, p, p, i32, i32, i32, i64, i64, i64, i32, p, p, p]
        L.mxo_format_bits.argtypes = [i32, i32, i32, i32]
        L.mxo_format_bits.restype = C.c_double
        L.mxo_threads.restype = i32
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _check(rc):
    if rc != 0:
        raise ValueError("oracle rejected its arguments (rc=%d)" % rc)


def quantize(x, block: int, w: int, axis_strided: bool = False):
    """x: float32 array [rows, K].  Returns (q int8 [rows,K], ebyte uint8 [rows,K/B], nonfinite)."""
    x = np.asarray(x)
    assert x.dtype == np.float32 and x.ndim == 2
    rows, K = x.shape
    sr, sk = x.strides[0] // 4, x.strides[1] // 4
    q = np.zeros((rows, K), np.int8)
    e = np.zeros((rows, K // block if block > 0 else 0), np.uint8)
    bad = C.c_uint32(0)
    _check(lib().mxo_quantize(_ptr(x), rows, K, sr, sk, block, w, _ptr(q), _ptr(e),
                              C.addressof(bad)))
    return q, e, int(bad.value)


def quantize_2d(x, block: int, block_rows: int, w: int):
    """Blocks of `block` along K times `block_rows` adjacent rows.  Returns (q int8 [rows,K],
    ebyte uint8 [rows/block_rows, K/block], nonfinite)."""
    x = np.asarray(x)
    assert x.dtype == np.float32 and x.ndim == 2
    rows, K = x.shape
    sr, sk = x.strides[0] // 4, x.strides[1] // 4
    q = np.zeros((rows, K), np.int8)
    e = np.zeros((rows // block_rows, K // block), np.uint8)
    bad = C.c_uint32(0)
    _check(lib().mxo_quantize_2d(_ptr(x), rows, K, sr, sk, block, block_rows, w, _ptr(q), _ptr(e),
                                 C.addressof(bad)))
    return q, e, int(bad.value)


def expand_exponent_rows(e, block_rows: int):
    """Exponent bytes of a (block, block_rows) tensor written out once per row."""
    e = np.ascontiguousarray(e, np.uint8)
    out = np.zeros((e.shape[0] * block_rows, e.shape[1]), np.uint8)
    _check(lib().mxo_expand_exponent_rows(_ptr(e), out.shape[0], e.shape[1], block_rows, _ptr(out)))
    return out


def cast(q, e, block_in: int, w_in: int, block_out: int, w_out: int):
    """MXInt -> MXInt of another width (and block size).  Returns (q int8, ebyte uint8, nonfinite)."""
    q = np.ascontiguousarray(q, np.int8)
    e = np.ascontiguousarray(e, np.uint8)
    rows, K = q.shape
    qo = np.zeros((rows, K), np.int8)
    eo = np.zeros((rows, K // block_out), np.uint8)
    bad = C.c_uint32(0)
    _check(lib().mxo_cast(_ptr(q), _ptr(e), rows, K, block_in, w_in, block_out, w_out, _ptr(qo), _ptr(eo),
                          C.addressof(bad)))
    return qo, eo, int(bad.value)


def dequantize(q, e, block: int, w: int):
    q = np.ascontiguousarray(q, np.int8)
    e = np.ascontiguousarray(e, np.uint8)
    rows, K = q.shape
    out = np.zeros((rows, K), np.float64)
    _check(lib().mxo_dequantize(_ptr(q), _ptr(e), rows, K, block, w, _ptr(out)))
    return out


def pack(q, w: int):
    q = np.ascontiguousarray(q, np.int8)
    rows, K = q.shape
    out = np.zeros((rows, K // 2 if w <= 4 else K), np.uint8)
    _check(lib().mxo_pack(_ptr(q), rows, K, w, _ptr(out)))
    return out


def pack_dense(q, w: int):
    """w bits per element, K*w/8 bytes per row (the storage Eq. 1 counts)."""
    q = np.ascontiguousarray(q, np.int8)
    rows, K = q.shape
    out = np.zeros((rows, K * w // 8), np.uint8)
    _check(lib().mxo_pack_dense(_ptr(q), rows, K, w, _ptr(out)))
    return out


def unpack_dense(packed, K: int, w: int):
    packed = np.ascontiguousarray(packed, np.uint8)
    rows = packed.shape[0]
    q = np.zeros((rows, K), np.int8)
    _check(lib().mxo_unpack_dense(_ptr(packed), rows, K, w, _ptr(q)))
    return q


def unpack(packed, K: int, w: int):
    packed = np.ascontiguousarray(packed, np.uint8)
    rows = packed.shape[0]
    q = np.zeros((rows, K), np.int8)
    _check(lib().mxo_unpack(_ptr(packed), rows, K, w, _ptr(q)))
    return q


def gemm(qa, ea, wa: int, qw, ew, ww: int, block: int, bias=None):
    """Returns (y_ref fp32 [M,N], y_seq fp32 [M,N], S fp64 [M,N])."""
    qa = np.ascontiguousarray(qa, np.int8)
    qw = np.ascontiguousarray(qw, np.int8)
    ea = np.ascontiguousarray(ea, np.uint8)
    ew = np.ascontiguousarray(ew, np.uint8)
    M, K = qa.shape
    N = qw.shape[0]
    assert qw.shape[1] == K
    if bias is not None:
        bias = np.ascontiguousarray(bias, np.float32)
    y_ref = np.zeros((M, N), np.float32)
    y_seq = np.zeros((M, N), np.float32)
    S = np.zeros((M, N), np.float64)
    _check(lib().mxo_gemm(_ptr(qa), _ptr(ea), wa, _ptr(qw), _ptr(ew), ww, M, N, K, block,
                          _ptr(bias), _ptr(y_ref), _ptr(y_seq), _ptr(S)))
    return y_ref, y_seq, S


def gemm_requant(qa, ea, wa: int, qw, ew, ww: int, block: int, block_y: int, wy: int, bias=None):
    """The product with an MXInt result.  Returns (qy int8 [M,N], ey uint8 [M,N/By], nonfinite,
    y_ref fp32 [M,N], S fp64 [M,N])."""
    qa = np.ascontiguousarray(qa, np.int8)
    qw = np.ascontiguousarray(qw, np.int8)
    ea = np.ascontiguousarray(ea, np.uint8)
    ew = np.ascontiguousarray(ew, np.uint8)
    M, K = qa.shape
    N = qw.shape[0]
    assert qw.shape[1] == K
    if bias is not None:
        bias = np.ascontiguousarray(bias, np.float32)
    qy = np.zeros((M, N), np.int8)
    ey = np.zeros((M, N // block_y), np.uint8)
    y_ref = np.zeros((M, N), np.float32)
    S = np.zeros((M, N), np.float64)
    bad = C.c_uint32(0)
    _check(lib().mxo_gemm_requant(_ptr(qa), _ptr(ea), wa, _ptr(qw), _ptr(ew), ww, M, N, K, block,
                                  _ptr(bias), block_y, wy, _ptr(qy), _ptr(ey), C.addressof(bad),
                                  _ptr(y_ref), _ptr(S)))
    return qy, ey, int(bad.value), y_ref, S


def gemm_samples(qa, ea, wa: int, qw, ew, ww: int, block: int, si, sj, bias=None):
    """The same three results at the output positions (si[t], sj[t])."""
    qa = np.ascontiguousarray(qa, np.int8)
    qw = np.ascontiguousarray(qw, np.int8)
    ea = np.ascontiguousarray(ea, np.uint8)
    ew = np.ascontiguousarray(ew, np.uint8)
    si = np.ascontiguousarray(si, np.int64)
    sj = np.ascontiguousarray(sj, np.int64)
    M, K = qa.shape
    N = qw.shape[0]
    n = si.shape[0]
    if bias is not None:
        bias = np.ascontiguousarray(bias, np.float32)
    y_ref = np.zeros(n, np.float32)
    y_seq = np.zeros(n, np.float32)
    S = np.zeros(n, np.float64)
    _check(lib().mxo_gemm_samples(_ptr(qa), _ptr(ea), wa, _ptr(qw), _ptr(ew), ww, M, N, K,
                                  block, _ptr(bias), _ptr(si), _ptr(sj), n, _ptr(y_ref),
                                  _ptr(y_seq), _ptr(S)))
    return y_ref, y_seq, S


KIND_BMF, KIND_BL = 1, 2


def alt_quantize(x, kind: int, block: int, ebits: int, mbits: int = 0):
    """Block Minifloat (kind 1) / Block Logarithm (kind 2) quantizer.  x: float32 [rows, K].
    Returns (codes uint8 [rows, K], shared bytes uint8 [rows, K/B], nonfinite)."""
    x = np.ascontiguousarray(x, np.float32)
    rows, K = x.shape
    codes = np.zeros((rows, K), np.uint8)
    shared = np.zeros((rows, K // block), np.uint8)
    bad = C.c_uint32(0)
    _check(lib().mxo_alt_quantize(_ptr(x), rows, K, K, kind, block, ebits, mbits, _ptr(codes), _ptr(shared),
                                  C.addressof(bad)))
    return codes, shared, int(bad.value)


def alt_dequantize(codes, shared, kind: int, block: int, ebits: int, mbits: int = 0):
    codes = np.ascontiguousarray(codes, np.uint8)
    shared = np.ascontiguousarray(shared, np.uint8)
    rows, K = codes.shape
    out = np.zeros((rows, K), np.float64)
    _check(lib().mxo_alt_dequantize(_ptr(codes), _ptr(shared), rows, K, kind, block, ebits, mbits, _ptr(out)))
    return out


def alt_gemm(ac, ash, afmt, wc, wsh, wfmt, block: int, bias=None):
    """afmt / wfmt = (kind, ebits, mbits).  Returns (y_ref fp32 [M,N], S fp64 [M,N])."""
    ac = np.ascontiguousarray(ac, np.uint8)
    wc = np.ascontiguousarray(wc, np.uint8)
    ash = np.ascontiguousarray(ash, np.uint8)
    wsh = np.ascontiguousarray(wsh, np.uint8)
    M, K = ac.shape
    N = wc.shape[0]
    if bias is not None:
        bias = np.ascontiguousarray(bias, np.float32)
    y = np.zeros((M, N), np.float32)
    S = np.zeros((M, N), np.float64)
    _check(lib().mxo_alt_gemm(_ptr(ac), _ptr(ash), afmt[0], afmt[1], afmt[2], _ptr(wc), _ptr(wsh), wfmt[0],
                              wfmt[1], wfmt[2], M, N, K, block, _ptr(bias), _ptr(y), _ptr(S)))
    return y, S


def format_bits(block: int, w: int, block_rows: int = 1, exp_bits: int = 8) -> float:
    return float(lib().mxo_format_bits(block, block_rows, exp_bits, w))


def threads() -> int:
    return int(lib().mxo_threads())
