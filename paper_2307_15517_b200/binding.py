"""Thin ctypes binding of ``libmxint.so`` -- argument marshalling only.

Every function has the name of the C entry point it calls (see ``include/mxint.h``) and takes
torch CUDA tensors for device memory; torch is used for allocation and streams, never for
arithmetic.  There is no fallback: if the shared library is missing the import fails, and a
negative status from the library raises ``MxError``.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmxint.so")

MX_F32, MX_BF16 = 0, 1
MX_ALGO_AUTO, MX_ALGO_SIMT, MX_ALGO_TCGEN05, MX_ALGO_STREAM, MX_ALGO_TCGEN05_FUSED = 0, 1, 2, 3, 4
MX_ALGO_TCGEN05_BLOCKWISE = 5
MX_ALGO_TCGEN05_MXF8 = 6

STATUS_NAMES = {0: "MX_OK", -1: "MX_ERR_NULL", -2: "MX_ERR_SHAPE", -3: "MX_ERR_FORMAT",
                -4: "MX_ERR_ALIGN", -5: "MX_ERR_WORKSPACE", -6: "MX_ERR_CUDA",
                -7: "MX_ERR_TIMEOUT", -8: "MX_ERR_ARCH"}


class MxFormat(C.Structure):
    """The (B, e, m) tuple of the paper's Sec. 4.1 with w = m + 1 (sign included)."""
    _fields_ = [("block", C.c_int32), ("elem_bits", C.c_int32), ("exp_bits", C.c_int32),
                ("block_rows", C.c_int32), ("packing", C.c_int32)]

    def __init__(self, block: int = 16, elem_bits: int = 4, exp_bits: int = 8, block_rows: int = 1, packing: int = 0):
        super().__init__(block, elem_bits, exp_bits, block_rows, packing)

    def dense(self) -> "MxFormat":
        """The same format with dense storage of the mantissas (elem_bits bits per element)."""
        return MxFormat(self.block, self.elem_bits, self.exp_bits, self.block_rows, 1)

    def __repr__(self):
        return "MxFormat(block=%d, elem_bits=%d, block_rows=%d, packing=%d)" % (self.block, self.elem_bits,
                                                                                  self.block_rows, self.packing)


class MxEpilogue(C.Structure):
    """Mirrors ``mx_epilogue_t``: bias, activation and residual applied in the product's epilogue."""
    _fields_ = [("bias", C.c_void_p), ("relu", C.c_int32), ("residual", C.c_void_p), ("ldr", C.c_int64)]


class MxPrologue(C.Structure):
    """Mirrors ``mx_prologue_t``: LayerNorm applied to the rows of x in front of the quantizer."""
    _fields_ = [("layernorm", C.c_int32), ("ln_gamma", C.c_void_p), ("ln_beta", C.c_void_p), ("ln_eps", C.c_float)]


class MxAltFormat(C.Structure):
    """A Block Minifloat (kind 1) or Block Logarithm (kind 2) format: mirrors ``mx_alt_format_t``."""
    _fields_ = [("kind", C.c_int32), ("block", C.c_int32), ("elem_exp_bits", C.c_int32),
                ("elem_man_bits", C.c_int32)]

    def __init__(self, kind: int, block: int, elem_exp_bits: int, elem_man_bits: int = 0):
        super().__init__(kind, block, elem_exp_bits, elem_man_bits)


MX_ELEM_BMF, MX_ELEM_BL = 1, 2


class MxLinearArgs(C.Structure):
    """One layer of ``mx_linear_grouped`` (mirrors ``mx_linear_args_t``)."""
    _fields_ = [("x", C.c_void_p), ("dt", C.c_int), ("M", C.c_int64), ("K", C.c_int64),
                ("ldx", C.c_int64), ("fa", MxFormat), ("w_mant", C.c_void_p), ("w_exp", C.c_void_p),
                ("fw", MxFormat), ("N", C.c_int64), ("bias", C.c_void_p), ("y", C.c_void_p),
                ("ldy", C.c_int64)]


class MxError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__("%s failed: %s%s" % (where, STATUS_NAMES.get(status, str(status)),
                                              (" (" + detail + ")") if detail else ""))


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libmxint.so is not built (%s). Run `python -m paper_2307_15517_b200.build`; there is "
            "no CPU or PyTorch fallback for these kernels." % LIB_PATH)
    L = C.CDLL(LIB_PATH)
    vp, i64, sz, i32 = C.c_void_p, C.c_int64, C.c_size_t, C.c_int
    F = MxFormat
    L.mx_mant_bytes.argtypes = [i64, i64, F]
    L.mx_mant_bytes.restype = sz
    L.mx_exp_bytes.argtypes = [i64, i64, F]
    L.mx_exp_bytes.restype = sz
    L.mx_format_bits.argtypes = [F]
    L.mx_format_bits.restype = C.c_double
    L.mx_workspace_bytes.argtypes = [i64, i64, i64, F, F]
    L.mx_workspace_bytes.restype = sz
    L.mx_workspace_bytes_ex.argtypes = [i64, i64, i64, F, F, i32]
    L.mx_workspace_bytes_ex.restype = sz
    L.mx_status_string.argtypes = [i32]
    L.mx_status_string.restype = C.c_char_p
    L.mx_last_cuda_error.argtypes = []
    L.mx_last_cuda_error.restype = C.c_char_p
    L.mx_quantize.argtypes = [vp, i32, i64, i64, i64, i64, F, vp, vp, vp, vp]
    L.mx_dequantize.argtypes = [vp, vp, i64, i64, F, vp, i32, i64, vp]
    L.mx_pack_dense.argtypes = [vp, i64, i64, F, vp, vp]
    L.mx_unpack_dense.argtypes = [vp, i64, i64, F, vp, vp]
    L.mx_pack_dense.restype = i32
    L.mx_unpack_dense.restype = i32
    L.mx_cast.argtypes = [vp, vp, F, i64, i64, F, vp, vp, vp, vp]
    L.mx_cast.restype = i32
    L.mx_gemm.argtypes = [vp, vp, F, vp, vp, F, i64, i64, i64, vp, vp, i64, vp, sz, vp]
    L.mx_gemm_ex.argtypes = [vp, vp, F, vp, vp, F, i64, i64, i64, vp, vp, i64, vp, sz, i32, vp]
    L.mx_linear.argtypes = [vp, i32, i64, i64, i64, F, vp, vp, F, i64, vp, vp, i64, vp, sz, vp]
    L.mx_linear_ex.argtypes = [vp, i32, i64, i64, i64, F, vp, vp, F, i64, vp, vp, i64, vp, sz, i32, vp]
    L.mx_gemm_q.argtypes = [vp, vp, F, vp, vp, F, i64, i64, i64, vp, F, vp, vp, vp, vp, sz, vp]
    L.mx_linear_q.argtypes = [vp, i32, i64, i64, i64, F, vp, vp, F, i64, vp, F, vp, vp, vp, vp, sz, vp]
    L.mx_gemm_q.restype = i32
    L.mx_linear_q.restype = i32
    E = C.POINTER(MxEpilogue)
    L.mx_gemm_fused.argtypes = [vp, vp, F, vp, vp, F, i64, i64, i64, E, vp, i64, F, vp, vp, vp, sz, vp]
    L.mx_linear_fused.argtypes = [vp, i32, i64, i64, i64, F, C.POINTER(MxPrologue), vp, vp, F, i64, E, vp, i64, F, vp, vp,
                                  vp, sz, vp]
    L.mx_gemm_fused.restype = i32
    L.mx_poll_status.argtypes = [vp]
    L.mx_selftest_wait_expiry.argtypes = [C.c_uint32, vp]
    L.mx_selftest_wait_expiry.restype = i32
    L.mx_gemm_batched_workspace_bytes.argtypes = [i64, i64, i64, i64]
    L.mx_gemm_batched_workspace_bytes.restype = sz
    L.mx_gemm_batched.argtypes = [vp, vp, F, i64, i64, vp, vp, F, i64, i64, i64, i64, i64, i64, vp, i64, i64,
                                  vp, sz, vp]
    L.mx_layernorm.argtypes = [vp, i64, vp, vp, C.c_float, i64, i64, vp, i64, vp]
    L.mx_softmax.argtypes = [vp, i64, i64, i64, C.c_float, i32, i64, vp]
    L.mx_relu_add.argtypes = [vp, vp, vp, i64, i32, vp]
    L.mx_softmax_q.argtypes = [vp, i64, i64, i64, C.c_float, i32, i64, F, vp, vp, vp]
    L.mx_softmax_q.restype = i32
    for name in ("mx_gemm_batched", "mx_layernorm", "mx_softmax", "mx_relu_add"):
        getattr(L, name).restype = i32
    L.mx_linear_grouped_workspace_bytes.argtypes = [C.POINTER(MxLinearArgs), i32]
    L.mx_linear_grouped_workspace_bytes.restype = sz
    L.mx_linear_grouped.argtypes = [C.POINTER(MxLinearArgs), i32, vp, sz, vp]
    L.mx_linear_grouped.restype = i32
    L.mx_gemm_static.argtypes = [vp, vp, F, vp, vp, F, i64, i64, i64, vp, vp, i64, vp]
    L.mx_gemm_static.restype = i32
    A = MxAltFormat
    L.mx_alt_quantize.argtypes = [vp, i32, i64, i64, i64, A, vp, vp, vp, vp]
    L.mx_alt_dequantize.argtypes = [vp, vp, i64, i64, A, vp, i32, i64, vp]
    L.mx_alt_gemm_workspace_bytes.argtypes = [i64, i64, i64]
    L.mx_alt_gemm_workspace_bytes.restype = sz
    L.mx_alt_gemm.argtypes = [vp, vp, A, vp, vp, A, i64, i64, i64, vp, vp, i64, vp, sz, vp]
    for name in ("mx_alt_quantize", "mx_alt_dequantize", "mx_alt_gemm"):
        getattr(L, name).restype = i32
    L.mx_attention_workspace_bytes.argtypes = [i64, i64, i64]
    L.mx_attention_workspace_bytes.restype = sz
    L.mx_attention.argtypes = [vp, vp, vp, vp, F, vp, vp, F, i64, i64, i64, C.c_float, i32, F, vp, i64, vp, vp, vp, sz, vp]
    L.mx_attention.restype = i32
    L.mx_attention_fp.argtypes = [vp, vp, vp, i32, i64, i64, i64, F, F, i64, i64, i64, C.c_float, i32, F, vp, i64, vp, sz, vp]
    L.mx_attention_fp.restype = i32
    L.mx_profile_begin.argtypes = []
    L.mx_profile_end.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    for name in ("mx_quantize", "mx_dequantize", "mx_gemm", "mx_gemm_ex", "mx_linear",
                 "mx_linear_ex", "mx_poll_status", "mx_profile_begin", "mx_profile_end"):
        getattr(L, name).restype = i32
    return L


lib = _load()


def _check(status: int, where: str):
    if status != 0:
        raise MxError(status, where, lib.mx_last_cuda_error().decode() if status == -6 else "")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return MX_F32
    if t.dtype == torch.bfloat16:
        return MX_BF16
    raise TypeError("expected float32 or bfloat16, got %s" % t.dtype)


def _need_cuda(*tensors):
    """Every tensor must live on the CURRENT CUDA device: the library launches on the current device
    and keeps its per-device state (status word, built-in scratch) by that device's index."""
    cur = None
    for t in tensors:
        if t is None:
            continue
        if not t.is_cuda:
            raise ValueError("device tensors required (this library has no host path)")
        if cur is None:
            cur = torch.cuda.current_device()
        if t.device.index != cur:
            raise ValueError("tensor on cuda:%d but the current device is cuda:%d; select the device first "
                             "(torch.cuda.set_device / torch.cuda.device)" % (t.device.index, cur))


# ---- size helpers ---------------------------------------------------------------------------

def mx_mant_bytes(rows: int, K: int, f: MxFormat) -> int:
    return int(lib.mx_mant_bytes(rows, K, f))


def mx_exp_bytes(rows: int, K: int, f: MxFormat) -> int:
    return int(lib.mx_exp_bytes(rows, K, f))


def mx_format_bits(f: MxFormat) -> float:
    return float(lib.mx_format_bits(f))


def mx_workspace_bytes(M: int, N: int, K: int, fa: MxFormat, fw: MxFormat) -> int:
    return int(lib.mx_workspace_bytes(M, N, K, fa, fw))


def mx_workspace_bytes_ex(M: int, N: int, K: int, fa: MxFormat, fw: MxFormat, algo: int) -> int:
    return int(lib.mx_workspace_bytes_ex(M, N, K, fa, fw, algo))


def mx_status_string(status: int) -> str:
    return lib.mx_status_string(status).decode()


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned scratch buffer (torch's caching allocator aligns to 512 bytes)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


# ---- compute entry points --------------------------------------------------------------------

def mx_quantize(x: torch.Tensor, f: MxFormat, mant_out: Optional[torch.Tensor] = None,
                exp_out: Optional[torch.Tensor] = None,
                nonfinite_count: Optional[torch.Tensor] = None,
                stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """x: [rows, K] fp32/bf16 CUDA tensor (any strides).  Returns (mant uint8, exps uint8)."""
    _need_cuda(x, mant_out, exp_out, nonfinite_count)
    assert x.dim() == 2
    rows, K = x.shape
    if mant_out is None:
        mant_out = torch.empty((rows, K // 2 if f.elem_bits <= 4 else K), dtype=torch.uint8, device=x.device)
    if exp_out is None:          # two-row blocks: one row of exponent bytes per pair of rows
        exp_out = torch.empty((rows // max(f.block_rows, 1), K // f.block), dtype=torch.uint8, device=x.device)
    _check(lib.mx_quantize(_ptr(x), _dtype_code(x), rows, K, x.stride(0), x.stride(1), f,
                           _ptr(mant_out), _ptr(exp_out), _ptr(nonfinite_count), _stream(stream)),
           "mx_quantize")
    return mant_out, exp_out


def mx_pack_dense(mant: torch.Tensor, K: int, f: MxFormat, stream=None) -> torch.Tensor:
    """Container mantissas [rows, K/2 or K] -> dense storage [rows, K * elem_bits / 8]."""
    _need_cuda(mant)
    rows = mant.shape[0]
    out = torch.empty((rows, K * f.elem_bits // 8), dtype=torch.uint8, device=mant.device)
    _check(lib.mx_pack_dense(_ptr(mant), rows, K, f, _ptr(out), _stream(stream)), "mx_pack_dense")
    return out


def mx_unpack_dense(dense: torch.Tensor, K: int, f: MxFormat, stream=None) -> torch.Tensor:
    _need_cuda(dense)
    rows = dense.shape[0]
    out = torch.empty((rows, K // 2 if f.elem_bits <= 4 else K), dtype=torch.uint8, device=dense.device)
    _check(lib.mx_unpack_dense(_ptr(dense), rows, K, f, _ptr(out), _stream(stream)), "mx_unpack_dense")
    return out


def mx_cast(mant: torch.Tensor, exps: torch.Tensor, K: int, f_in: MxFormat, f_out: MxFormat,
            nonfinite_count: Optional[torch.Tensor] = None, stream=None):
    """MXInt tensor -> MXInt tensor of another width / block size.  Returns (mant, exps)."""
    _need_cuda(mant, exps, nonfinite_count)
    rows = mant.shape[0]
    mant_out = torch.empty((rows, K // 2 if f_out.elem_bits <= 4 else K), dtype=torch.uint8, device=mant.device)
    exp_out = torch.empty((rows, K // f_out.block), dtype=torch.uint8, device=mant.device)
    _check(lib.mx_cast(_ptr(mant), _ptr(exps), f_in, rows, K, f_out, _ptr(mant_out), _ptr(exp_out),
                       _ptr(nonfinite_count), _stream(stream)), "mx_cast")
    return mant_out, exp_out


def mx_dequantize(mant: torch.Tensor, exps: torch.Tensor, K: int, f: MxFormat,
                  dtype=torch.float32, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    _need_cuda(mant, exps, out)
    rows = mant.shape[0]
    if out is None:
        out = torch.empty((rows, K), dtype=dtype, device=mant.device)
    assert out.shape == (rows, K) and out.stride(1) == 1
    _check(lib.mx_dequantize(_ptr(mant), _ptr(exps), rows, K, f, _ptr(out), _dtype_code(out), out.stride(0),
                             _stream(stream)), "mx_dequantize")
    return out


def mx_gemm(a_mant, a_exp, fa: MxFormat, w_mant, w_exp, fw: MxFormat, M: int, N: int, K: int,
            bias: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None,
            workspace: Optional[torch.Tensor] = None, algo: int = MX_ALGO_AUTO, stream=None):
    _need_cuda(a_mant, a_exp, w_mant, w_exp, bias, y, workspace)
    if y is None:
        y = torch.empty((M, N), dtype=torch.float32, device=a_mant.device)
    if workspace is None and algo != MX_ALGO_SIMT:
        workspace = alloc_workspace(mx_workspace_bytes_ex(M, N, K, fa, fw, algo), a_mant.device)
    _check(lib.mx_gemm_ex(_ptr(a_mant), _ptr(a_exp), fa, _ptr(w_mant), _ptr(w_exp), fw, M, N, K,
                          _ptr(bias), _ptr(y), y.stride(0), _ptr(workspace),
                          0 if workspace is None else workspace.numel(), algo, _stream(stream)),
           "mx_gemm")
    return y


def mx_linear(x: torch.Tensor, fa: MxFormat, w_mant, w_exp, fw: MxFormat, N: int,
              bias: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None,
              workspace: Optional[torch.Tensor] = None, algo: int = MX_ALGO_AUTO, stream=None):
    _need_cuda(x, w_mant, w_exp, bias, y, workspace)
    M, K = x.shape
    assert x.stride(1) == 1
    if y is None:
        y = torch.empty((M, N), dtype=torch.float32, device=x.device)
    if workspace is None:
        workspace = alloc_workspace(mx_workspace_bytes_ex(M, N, K, fa, fw, algo), x.device)
    _check(lib.mx_linear_ex(_ptr(x), _dtype_code(x), M, K, x.stride(0), fa, _ptr(w_mant),
                            _ptr(w_exp), fw, N, _ptr(bias), _ptr(y), y.stride(0), _ptr(workspace),
                            workspace.numel(), algo, _stream(stream)), "mx_linear")
    return y


def _quantized_out(M: int, N: int, fy: MxFormat, device, y_mant, y_exp):
    if y_mant is None:
        y_mant = torch.empty((M, N // 2 if fy.elem_bits <= 4 else N), dtype=torch.uint8, device=device)
    if y_exp is None:
        y_exp = torch.empty((M // max(fy.block_rows, 1), N // fy.block), dtype=torch.uint8, device=device)
    return y_mant, y_exp


def mx_gemm_q(a_mant, a_exp, fa: MxFormat, w_mant, w_exp, fw: MxFormat, M: int, N: int, K: int,
              fy: MxFormat, bias: Optional[torch.Tensor] = None, y_mant=None, y_exp=None,
              nonfinite_count: Optional[torch.Tensor] = None,
              workspace: Optional[torch.Tensor] = None, stream=None):
    """mx_gemm with the result quantized to format ``fy`` along N.  Returns (y_mant, y_exp)."""
    _need_cuda(a_mant, a_exp, w_mant, w_exp, bias, y_mant, y_exp, nonfinite_count, workspace)
    y_mant, y_exp = _quantized_out(M, N, fy, a_mant.device, y_mant, y_exp)
    if workspace is None:
        workspace = alloc_workspace(mx_workspace_bytes_ex(M, N, K, fa, fw, MX_ALGO_TCGEN05), a_mant.device)
    _check(lib.mx_gemm_q(_ptr(a_mant), _ptr(a_exp), fa, _ptr(w_mant), _ptr(w_exp), fw, M, N, K,
                         _ptr(bias), fy, _ptr(y_mant), _ptr(y_exp), _ptr(nonfinite_count),
                         _ptr(workspace), workspace.numel(), _stream(stream)), "mx_gemm_q")
    return y_mant, y_exp


def mx_linear_q(x: torch.Tensor, fa: MxFormat, w_mant, w_exp, fw: MxFormat, N: int, fy: MxFormat,
                bias: Optional[torch.Tensor] = None, y_mant=None, y_exp=None,
                nonfinite_count: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None, stream=None):
    """mx_linear with the result quantized to format ``fy`` along N.  Returns (y_mant, y_exp)."""
    _need_cuda(x, w_mant, w_exp, bias, y_mant, y_exp, nonfinite_count, workspace)
    M, K = x.shape
    assert x.stride(1) == 1
    y_mant, y_exp = _quantized_out(M, N, fy, x.device, y_mant, y_exp)
    if workspace is None:
        workspace = alloc_workspace(mx_workspace_bytes_ex(M, N, K, fa, fw, MX_ALGO_TCGEN05), x.device)
    _check(lib.mx_linear_q(_ptr(x), _dtype_code(x), M, K, x.stride(0), fa, _ptr(w_mant), _ptr(w_exp),
                           fw, N, _ptr(bias), fy, _ptr(y_mant), _ptr(y_exp), _ptr(nonfinite_count),
                           _ptr(workspace), workspace.numel(), _stream(stream)), "mx_linear_q")
    return y_mant, y_exp


def _epilogue(bias, relu, residual):
    ep = MxEpilogue()
    ep.bias = None if bias is None else bias.data_ptr()
    ep.relu = 1 if relu else 0
    ep.residual = None if residual is None else residual.data_ptr()
    ep.ldr = 0 if residual is None else residual.stride(0)
    return ep


def mx_linear_fused(x: torch.Tensor, fa: MxFormat, w_mant, w_exp, fw: MxFormat, N: int,
                    bias: Optional[torch.Tensor] = None, relu: bool = False,
                    residual: Optional[torch.Tensor] = None, fy: Optional[MxFormat] = None, y=None,
                    y_mant=None, y_exp=None, layernorm=None, workspace: Optional[torch.Tensor] = None, stream=None):
    """mx_linear with bias, ReLU and a residual applied in the epilogue.  ``fy`` None: returns the fp32
    result; else returns (y_mant, y_exp), the result quantized to ``fy`` along N.
    ``layernorm`` = (gamma, beta, eps): the rows of x are layer-normalised in front of the quantizer."""
    _need_cuda(x, w_mant, w_exp, bias, residual, y, y_mant, y_exp, workspace)
    pro = None
    if layernorm is not None:
        gamma, beta, eps = layernorm
        _need_cuda(gamma, beta)
        pro = MxPrologue(1, None if gamma is None else gamma.data_ptr(), None if beta is None else beta.data_ptr(), eps)
    M, K = x.shape
    assert x.stride(1) == 1 and (residual is None or (residual.stride(1) == 1 and residual.dtype == torch.float32))
    if fy is None:
        if y is None:
            y = torch.empty((M, N), dtype=torch.float32, device=x.device)
        assert y.dtype == torch.float32 and y.stride(1) == 1
    else:
        y_mant, y_exp = _quantized_out(M, N, fy, x.device, y_mant, y_exp)
    if workspace is None:
        workspace = alloc_workspace(mx_workspace_bytes_ex(M, N, K, fa, fw, MX_ALGO_TCGEN05), x.device)
    ep = _epilogue(bias, relu, residual)
    _check(lib.mx_linear_fused(_ptr(x), _dtype_code(x), M, K, x.stride(0), fa, None if pro is None else C.byref(pro),
                               _ptr(w_mant), _ptr(w_exp), fw, N, C.byref(ep), _ptr(y) if fy is None else None, y.stride(0) if fy is None else N,
                               fy if fy is not None else MxFormat(), None if fy is None else _ptr(y_mant),
                               None if fy is None else _ptr(y_exp), _ptr(workspace), workspace.numel(),
                               _stream(stream)), "mx_linear_fused")
    return y if fy is None else (y_mant, y_exp)


def mx_gemm_fused(a_mant, a_exp, fa: MxFormat, w_mant, w_exp, fw: MxFormat, M: int, N: int, K: int,
                  bias: Optional[torch.Tensor] = None, relu: bool = False,
                  residual: Optional[torch.Tensor] = None, fy: Optional[MxFormat] = None, y=None,
                  y_mant=None, y_exp=None, workspace: Optional[torch.Tensor] = None, stream=None):
    """mx_gemm with bias, ReLU and a residual applied in the epilogue; result as for ``mx_linear_fused``."""
    _need_cuda(a_mant, a_exp, w_mant, w_exp, bias, residual, y, y_mant, y_exp, workspace)
    assert residual is None or (residual.stride(1) == 1 and residual.dtype == torch.float32)
    if fy is None:
        if y is None:
            y = torch.empty((M, N), dtype=torch.float32, device=a_mant.device)
        assert y.dtype == torch.float32 and y.stride(1) == 1
    else:
        y_mant, y_exp = _quantized_out(M, N, fy, a_mant.device, y_mant, y_exp)
    if workspace is None:
        workspace = alloc_workspace(mx_workspace_bytes_ex(M, N, K, fa, fw, MX_ALGO_TCGEN05), a_mant.device)
    ep = _epilogue(bias, relu, residual)
    _check(lib.mx_gemm_fused(_ptr(a_mant), _ptr(a_exp), fa, _ptr(w_mant), _ptr(w_exp), fw, M, N, K, C.byref(ep),
                             _ptr(y) if fy is None else None, y.stride(0) if fy is None else N,
                             fy if fy is not None else MxFormat(), None if fy is None else _ptr(y_mant),
                             None if fy is None else _ptr(y_exp), _ptr(workspace), workspace.numel(),
                             _stream(stream)), "mx_gemm_fused")
    return y if fy is None else (y_mant, y_exp)


def make_linear_args(layers):
    """layers: iterable of dicts with x, fa, w_mant, w_exp, fw, N, y and optionally bias.
    Returns a ctypes array of ``MxLinearArgs`` (host memory) for ``mx_linear_grouped``."""
    layers = list(layers)
    arr = (MxLinearArgs * len(layers))()
    for a, L in zip(arr, layers):
        x, y = L["x"], L["y"]
        _need_cuda(x, y, L["w_mant"], L["w_exp"], L.get("bias"))
        assert x.stride(1) == 1
        a.x, a.dt, a.M, a.K, a.ldx, a.fa = x.data_ptr(), _dtype_code(x), x.shape[0], x.shape[1], x.stride(0), L["fa"]
        a.w_mant, a.w_exp, a.fw, a.N = L["w_mant"].data_ptr(), L["w_exp"].data_ptr(), L["fw"], L["N"]
        bias = L.get("bias")
        a.bias = None if bias is None else bias.data_ptr()
        a.y, a.ldy = y.data_ptr(), y.stride(0)
    return arr


def mx_linear_grouped_workspace_bytes(args) -> int:
    return int(lib.mx_linear_grouped_workspace_bytes(args, len(args)))


def mx_linear_grouped(args, workspace: Optional[torch.Tensor] = None, stream=None):
    """args: the array made by ``make_linear_args``.  One launch over all layers (decode)."""
    if workspace is None:
        workspace = alloc_workspace(mx_linear_grouped_workspace_bytes(args))
    _check(lib.mx_linear_grouped(args, len(args), _ptr(workspace), workspace.numel(), _stream(stream)),
           "mx_linear_grouped")
    return workspace


def mx_gemm_batched(a_mant, a_exp, fa: MxFormat, lda: int, stride_a: int, w_mant, w_exp, fw: MxFormat,
                    ldw: int, stride_w: int, M: int, N: int, K: int, batch: int, y: torch.Tensor,
                    ldy: int, stride_y: int, workspace: Optional[torch.Tensor] = None, stream=None):
    """`batch` products Y_b = A_b W_b^T on slices of packed tensors (strides in elements)."""
    _need_cuda(a_mant, a_exp, w_mant, w_exp, y, workspace)
    if workspace is None:
        workspace = alloc_workspace(int(lib.mx_gemm_batched_workspace_bytes(M, N, K, batch)), y.device)
    _check(lib.mx_gemm_batched(_ptr(a_mant), _ptr(a_exp), fa, lda, stride_a, _ptr(w_mant), _ptr(w_exp), fw,
                               ldw, stride_w, M, N, K, batch, _ptr(y), ldy, stride_y, _ptr(workspace),
                               workspace.numel(), _stream(stream)), "mx_gemm_batched")
    return y


def mx_attention(q_mant, q_exp, k_mant, k_exp, fqk: MxFormat, vt_mant, vt_exp, fv: MxFormat, seq: int, heads: int,
                 head_dim: int, scale: float, fp: MxFormat, causal: bool = True, ctx: Optional[torch.Tensor] = None,
                 return_p: bool = False, workspace: Optional[torch.Tensor] = None, stream=None):
    """Scores, causal softmax, quantized probabilities and context of all heads in one kernel.
    Returns ctx [seq, heads*head_dim] fp32 (and the quantized probabilities (mant, exps) with return_p)."""
    _need_cuda(q_mant, q_exp, k_mant, k_exp, vt_mant, vt_exp, ctx, workspace)
    dev = q_mant.device
    if ctx is None:
        ctx = torch.empty((seq, heads * head_dim), dtype=torch.float32, device=dev)
    pm = pe = None
    if return_p:
        pm = torch.zeros((heads * seq, seq // 2 if fp.elem_bits <= 4 else seq), dtype=torch.uint8, device=dev)
        pe = torch.zeros((heads * seq, seq // fp.block), dtype=torch.uint8, device=dev)
    if workspace is None:
        workspace = alloc_workspace(int(lib.mx_attention_workspace_bytes(seq, heads, head_dim)), dev)
    _check(lib.mx_attention(_ptr(q_mant), _ptr(q_exp), _ptr(k_mant), _ptr(k_exp), fqk, _ptr(vt_mant), _ptr(vt_exp), fv,
                            seq, heads, head_dim, scale, 1 if causal else 0, fp, _ptr(ctx), ctx.stride(0), _ptr(pm),
                            _ptr(pe), _ptr(workspace), workspace.numel(), _stream(stream)), "mx_attention")
    return (ctx, pm, pe) if return_p else ctx


def mx_attention_fp(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, fqk: MxFormat, fv: MxFormat, heads: int,
                    head_dim: int, scale: float, fp: MxFormat, causal: bool = True,
                    ctx: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None):
    """mx_attention on floating-point q, k, v ([seq, heads*head_dim], row-major views allowed): the three
    operands are quantized on the fly (q, k along the head dimension, v along the tokens)."""
    _need_cuda(q, k, v, ctx, workspace)
    seq = q.shape[0]
    assert q.dtype == k.dtype == v.dtype and q.stride(1) == k.stride(1) == v.stride(1) == 1
    assert q.shape == k.shape == v.shape == (seq, heads * head_dim)
    if ctx is None:
        ctx = torch.empty((seq, heads * head_dim), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = alloc_workspace(int(lib.mx_attention_workspace_bytes(seq, heads, head_dim)), q.device)
    _check(lib.mx_attention_fp(_ptr(q), _ptr(k), _ptr(v), _dtype_code(q), q.stride(0), k.stride(0), v.stride(0), fqk, fv,
                               seq, heads, head_dim, scale, 1 if causal else 0, fp, _ptr(ctx), ctx.stride(0),
                               _ptr(workspace), workspace.numel(), _stream(stream)), "mx_attention_fp")
    return ctx


def mx_layernorm(x: torch.Tensor, gamma, beta, eps: float, y: Optional[torch.Tensor] = None, stream=None):
    _need_cuda(x, gamma, beta, y)
    assert x.dim() == 2 and x.stride(1) == 1 and x.dtype == torch.float32
    if y is None:
        y = torch.empty_like(x)
    _check(lib.mx_layernorm(_ptr(x), x.stride(0), _ptr(gamma), _ptr(beta), eps, x.shape[0], x.shape[1],
                            _ptr(y), y.stride(0), _stream(stream)), "mx_layernorm")
    return y


def mx_softmax(s: torch.Tensor, scale: float = 1.0, causal: bool = False, rows_per_batch: int = 0, stream=None):
    """In place over the rows of the 2-D fp32 tensor s."""
    _need_cuda(s)
    assert s.dim() == 2 and s.stride(1) == 1 and s.dtype == torch.float32
    _check(lib.mx_softmax(_ptr(s), s.stride(0), s.shape[0], s.shape[1], scale, 1 if causal else 0,
                          rows_per_batch, _stream(stream)), "mx_softmax")
    return s


def mx_softmax_q(s: torch.Tensor, fp: MxFormat, scale: float = 1.0, causal: bool = False, rows_per_batch: int = 0,
                 stream=None):
    """Softmax over the rows of the 2-D fp32 tensor s, returned quantized to format fp: (mant, exps)."""
    _need_cuda(s)
    assert s.dim() == 2 and s.stride(1) == 1 and s.dtype == torch.float32
    rows, cols = s.shape
    mant = torch.empty((rows, cols // 2 if fp.elem_bits <= 4 else cols), dtype=torch.uint8, device=s.device)
    exps = torch.empty((rows, cols // fp.block), dtype=torch.uint8, device=s.device)
    _check(lib.mx_softmax_q(_ptr(s), s.stride(0), rows, cols, scale, 1 if causal else 0, rows_per_batch, fp,
                            _ptr(mant), _ptr(exps), _stream(stream)), "mx_softmax_q")
    return mant, exps


def mx_relu_add(a: torch.Tensor, b: Optional[torch.Tensor], y: Optional[torch.Tensor] = None,
                relu: bool = False, stream=None):
    """y = (relu ? max(a, 0) : a) + b over contiguous fp32 tensors."""
    _need_cuda(a, b, y)
    assert a.is_contiguous() and (b is None or b.is_contiguous())
    if y is None:
        y = torch.empty_like(a)
    _check(lib.mx_relu_add(_ptr(a), _ptr(b), _ptr(y), a.numel(), 1 if relu else 0, _stream(stream)),
           "mx_relu_add")
    return y


def mx_alt_quantize(x: torch.Tensor, f: MxAltFormat, nonfinite_count: Optional[torch.Tensor] = None, stream=None):
    """x: [rows, K] fp32/bf16, rows contiguous.  Returns (codes uint8 [rows, K], shared uint8 [rows, K/block])."""
    _need_cuda(x, nonfinite_count)
    assert x.dim() == 2 and x.stride(1) == 1
    rows, K = x.shape
    codes = torch.empty((rows, K), dtype=torch.uint8, device=x.device)
    shared = torch.empty((rows, K // f.block), dtype=torch.uint8, device=x.device)
    _check(lib.mx_alt_quantize(_ptr(x), _dtype_code(x), rows, K, x.stride(0), f, _ptr(codes), _ptr(shared),
                               _ptr(nonfinite_count), _stream(stream)), "mx_alt_quantize")
    return codes, shared


def mx_alt_dequantize(codes: torch.Tensor, shared: torch.Tensor, f: MxAltFormat, dtype=torch.float32, stream=None):
    _need_cuda(codes, shared)
    rows, K = codes.shape
    out = torch.empty((rows, K), dtype=dtype, device=codes.device)
    _check(lib.mx_alt_dequantize(_ptr(codes), _ptr(shared), rows, K, f, _ptr(out), _dtype_code(out), K,
                                 _stream(stream)), "mx_alt_dequantize")
    return out


def mx_alt_gemm(a_codes, a_shared, fa: MxAltFormat, w_codes, w_shared, fw: MxAltFormat,
                bias: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None, stream=None):
    """Y = A W^T on Block Minifloat / Block Logarithm operands (codes [M, K] and [N, K])."""
    _need_cuda(a_codes, a_shared, w_codes, w_shared, bias, y, workspace)
    M, K = a_codes.shape
    N = w_codes.shape[0]
    if y is None:
        y = torch.empty((M, N), dtype=torch.float32, device=a_codes.device)
    if workspace is None:
        workspace = alloc_workspace(int(lib.mx_alt_gemm_workspace_bytes(M, N, K)), a_codes.device)
    _check(lib.mx_alt_gemm(_ptr(a_codes), _ptr(a_shared), fa, _ptr(w_codes), _ptr(w_shared), fw, M, N, K,
                           _ptr(bias), _ptr(y), y.stride(0), _ptr(workspace), workspace.numel(), _stream(stream)),
           "mx_alt_gemm")
    return y


MX_STATIC_SCRATCH_BYTES = 32 << 20


def mx_gemm_static(a_mant, a_exp, fa: MxFormat, w_mant, w_exp, fw: MxFormat, M: int, N: int, K: int,
                   bias: Optional[torch.Tensor] = None, y: Optional[torch.Tensor] = None, stream=None):
    """The tensor-core product for callers that must not allocate device memory: same arguments
    and result as ``mx_gemm`` minus the workspace, which is a fixed array inside the library
    (2*(M+N)*K bytes must fit in ``MX_STATIC_SCRATCH_BYTES``; ``MxError`` with
    ``MX_ERR_WORKSPACE`` otherwise).  Pass ``y`` to keep this wrapper allocation-free as well."""
    _need_cuda(a_mant, a_exp, w_mant, w_exp, bias, y)
    if y is None:
        y = torch.empty((M, N), dtype=torch.float32, device=a_mant.device)
    rc = lib.mx_gemm_static(_ptr(a_mant), _ptr(a_exp), fa, _ptr(w_mant), _ptr(w_exp), fw, M, N, K,
                            _ptr(bias), _ptr(y), y.stride(0), _stream(stream))
    if rc == -5:
        raise MxError(rc, "mx_gemm_static", lib.mx_last_cuda_error().decode())
    _check(rc, "mx_gemm_static")
    return y


def mx_poll_status(stream=None) -> int:
    """Synchronises the stream and returns the library's device status (0 = MX_OK)."""
    return int(lib.mx_poll_status(_stream(stream)))


def mx_selftest_wait_expiry(limit_us: int = 2000, stream=None) -> None:
    """Launches the library's bounded-wait self-test (a wait nobody satisfies, given up after limit_us)."""
    _check(lib.mx_selftest_wait_expiry(limit_us, _stream(stream)), "mx_selftest_wait_expiry")


KERNEL_KINDS = ("quantize", "dequantize", "gemm_tc", "gemm_simt", "gemm_stream", "prep", "glue")


def mx_profile_begin() -> None:
    _check(lib.mx_profile_begin(), "mx_profile_begin")


def mx_profile_end():
    """Returns {kind: (milliseconds, launches)} for the kernels launched since mx_profile_begin."""
    ms = (C.c_double * 8)()
    n = (C.c_int64 * 8)()
    _check(lib.mx_profile_end(ms, n), "mx_profile_end")
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_KINDS)}
