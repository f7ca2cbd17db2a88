"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, its size helpers reproduce the paper's storage accounting (Eq. 1), and
invalid arguments are rejected before any launch."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2307_15517_b200 import build as mx_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mxb():
    mx_build.build()
    from paper_2307_15517_b200 import binding
    return binding


def _declared_symbols():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names += re.findall(r"MX_API\s+[\w\s\*]+?\b(mx_\w+)\s*\(", text)
    return names


def test_every_declared_symbol_is_exported(mxb):
    names = _declared_symbols()
    assert len(names) >= 13 and "mx_quantize" in names and "mx_gemm" in names and "mx_linear" in names
    for n in names:
        assert hasattr(mxb.lib, n), n


def test_size_helpers_match_eq1(mxb):
    F = mxb.MxFormat
    assert mxb.mx_format_bits(F(16, 8, 8, 2)) == 8.25          # the paper's MXInt((16,2),8,7)
    assert mxb.mx_format_bits(F(16, 4)) == 4.5 and mxb.mx_format_bits(F(32, 4)) == 4.25
    assert mxb.mx_mant_bytes(128, 768, F(16, 4)) == 128 * 384
    assert mxb.mx_mant_bytes(128, 768, F(16, 5)) == 128 * 768
    assert mxb.mx_exp_bytes(128, 768, F(16, 4)) == 128 * 48
    assert mxb.mx_exp_bytes(4096, 11008, F(32, 4)) == 4096 * 344
    # decode weight stream of one 4096x4096 W4/B32 matrix: 0.53125 bytes per weight
    total = mxb.mx_mant_bytes(4096, 4096, F(32, 4)) + mxb.mx_exp_bytes(4096, 4096, F(32, 4))
    assert total == int(4096 * 4096 * 0.53125)
    assert mxb.mx_mant_bytes(4, 40, F(16, 4)) == 0             # K not a multiple of the block
    assert mxb.mx_mant_bytes(4, 64, F(8, 4)) == 0              # unsupported block
    assert mxb.mx_exp_bytes(128, 768, F(16, 8, 8, 2)) == 64 * 48   # (16,2) blocks: one exponent row per pair of rows
    assert mxb.mx_exp_bytes(127, 768, F(16, 8, 8, 2)) == 0
    f4 = F(16, 4)
    assert mxb.mx_workspace_bytes(128, 768, 768, f4, f4) >= 2 * (128 + 768) * 768   # both operands as bf16
    fused = mxb.mx_workspace_bytes_ex(128, 768, 768, f4, f4, mxb.MX_ALGO_TCGEN05_FUSED)
    assert 2 * 128 * 768 <= fused < 2 * (128 + 768) * 768                           # activations only
    assert mxb.mx_workspace_bytes_ex(128, 768, 112, f4, f4, mxb.MX_ALGO_TCGEN05_FUSED) >= 2 * (128 + 768) * 112
    assert mxb.mx_workspace_bytes_ex(128, 768, 768, f4, f4, 99) == 0


def test_status_strings(mxb):
    for code in range(0, -9, -1):
        assert mxb.mx_status_string(code) not in ("", "unknown status")


def test_invalid_arguments_are_rejected_on_the_host(mxb):
    F = mxb.MxFormat
    L = mxb.lib
    fake = C.c_void_p(0x10000)       # never dereferenced: validation fails first
    odd = C.c_void_p(0x10004)
    f = F(16, 4)
    assert L.mx_quantize(None, 0, 4, 64, 64, 1, f, fake, fake, None, None) == -1
    assert L.mx_quantize(fake, 0, 4, 40, 40, 1, f, fake, fake, None, None) == -2
    assert L.mx_quantize(fake, 0, 4, 64, 32, 1, f, fake, fake, None, None) == -2   # ld < K
    assert L.mx_quantize(fake, 0, 4, 64, 64, 1, F(16, 9), fake, fake, None, None) == -3
    assert L.mx_quantize(fake, 0, 4, 64, 64, 1, F(16, 4, 5), fake, fake, None, None) == -3
    assert L.mx_quantize(fake, 0, 4, 64, 64, 1, F(16, 4, 8, 3), fake, fake, None, None) == -3   # block_rows 1 or 2
    assert L.mx_quantize(fake, 0, 3, 64, 64, 1, F(16, 4, 8, 2), fake, fake, None, None) == -2   # odd rows, two-row blocks
    assert L.mx_quantize(fake, 0, 4, 64, 1, 4, F(16, 4, 8, 2), fake, fake, None, None) == -3    # two-row blocks, strided axis
    assert L.mx_quantize(fake, 7, 4, 64, 64, 1, f, fake, fake, None, None) == -3
    assert L.mx_quantize(odd, 0, 4, 64, 64, 1, f, fake, fake, None, None) == -4
    assert L.mx_quantize(fake, 0, 4, 64, 68, 1, f, fake, fake, None, None) == -4   # ld % 8
    g = lambda **kw: L.mx_gemm_ex(kw.get("a", fake), fake, kw.get("fa", f), fake, fake, kw.get("fw", f),
                                  kw.get("M", 8), kw.get("N", 8), kw.get("K", 64), None,
                                  kw.get("y", fake), kw.get("ldy", 8), kw.get("ws", None), 0,
                                  kw.get("algo", 2), None)
    assert g(a=None) == -1
    assert g(K=40) == -2 and g(M=0) == -2 and g(ldy=4) == -2
    assert g(fa=F(32, 4)) == -3                     # blocks of A and W differ
    assert g(y=odd) == -4
    assert g(algo=9) == -3
    assert L.mx_linear_ex(fake, 0, 8, 64, 60, f, fake, fake, f, 8, None, fake, 8, None, 0, 2, None) == -2
    # the calls with an MXInt result: N must hold whole output blocks, outputs must be there
    q = lambda **kw: L.mx_linear_q(fake, 0, kw.get("M", 8), 64, 64, f, fake, fake, f, kw.get("N", 32), None, kw.get("fy", f),
                                   kw.get("ym", fake), kw.get("ye", fake), None, None, 0, None)
    assert q(N=40) == -2                                     # 40 is not a multiple of the output block
    assert q(fy=mxb.MxFormat(8, 4)) == -3
    assert q(ym=None) == -1 and q(ye=None) == -1
    assert q(fy=F(16, 4, 8, 2), M=7) == -2                   # a two-row result format needs an even number of rows
    assert q(fy=F(16, 4, 8, 3)) == -3
    # the product with a fused tail: exactly one kind of result, residual rows at least N wide
    ep = mxb.MxEpilogue()
    ep.residual, ep.ldr = fake, 16
    ft = lambda ep, y, ym, pro=None, K=64, dt=0: L.mx_linear_fused(fake, dt, 8, K, K, f, pro, fake, fake, f, 32, ep, y, 32, f, ym,
                                                                 fake, fake, 1 << 20, None)
    assert ft(None, fake, fake) == -1 and ft(None, None, None) == -1
    assert ft(C.byref(ep), fake, None) == -2
    ln = mxb.MxPrologue(1, None, None, 1e-5)
    assert ft(None, fake, None, C.byref(ln), dt=1) == -3        # LayerNorm in the operand pass wants fp32 rows
    assert ft(None, fake, None, C.byref(ln), K=16384) == -2     # ... of at most 8192 values
    # casts and the softmax with an MXInt result
    c = lambda **kw: L.mx_cast(kw.get("m", fake), fake, kw.get("fi", f), kw.get("rows", 4), kw.get("K", 64),
                               kw.get("fo", F(32, 8)), kw.get("mo", fake), fake, None, None)
    assert c(K=48) == -2                                     # 48 is not a multiple of the output block 32
    assert c(fi=F(16, 4, 8, 2)) == -3 and c(fo=F(16, 9)) == -3
    assert c(m=None) == -1 and c(mo=odd) == -4
    assert c(rows=0) == 0                                    # empty tensor: nothing to do
    sq = lambda **kw: L.mx_softmax_q(kw.get("s", fake), kw.get("ld", 64), 4, kw.get("cols", 64), C.c_float(1.0),
                                     kw.get("causal", 0), kw.get("rpb", 0), kw.get("fp", F(16, 8)), fake, fake, None)
    assert sq(cols=40) == -2 and sq(cols=16384, ld=16384) == -2 and sq(ld=32) == -2
    assert sq(causal=1, rpb=0) == -2
    assert sq(fp=F(16, 8, 8, 2)) == -3
    assert sq(s=None) == -1 and sq(ld=66) == -4
    assert L.mx_selftest_wait_expiry(0, None) == -2
    # fused attention: head dimension 128, whole query tiles, one-row container formats, aligned leading dimensions
    f8 = F(16, 8)
    at = lambda **kw: L.mx_attention(kw.get("q", fake), fake, fake, fake, kw.get("fqk", f8), fake, fake, f8,
                                     kw.get("seq", 256), 2, kw.get("d", 128), C.c_float(0.1), 1, kw.get("fp", f8),
                                     fake, kw.get("ldc", 256), kw.get("pm", None), None, None, 0, None)
    assert at(q=None) == -1 and at(pm=fake) == -1            # probabilities out: both arrays or none
    assert at(d=96) == -2 and at(seq=200) == -2 and at(ldc=128) == -2
    assert L.mx_attention(fake, fake, fake, fake, f8, fake, fake, f8, 256, 2, 128, C.c_float(-0.1), 1, f8, fake, 256, None,
                          None, None, 0, None) == -2       # the softmax scale must be positive
    assert at(fqk=F(16, 8, 8, 2)) == -3 and at(fp=F(16, 9)) == -3
    assert at() == -5                                        # no workspace
    af = lambda **kw: L.mx_attention_fp(kw.get("q", fake), fake, fake, kw.get("dt", 0), kw.get("ldq", 768), 768, 768,
                                        kw.get("fqk", f8), f8, kw.get("seq", 256), 2, kw.get("d", 128), C.c_float(0.1),
                                        1, f8, fake, 256, None, 0, None)
    assert af(q=None) == -1 and af(dt=5) == -3 and af(fqk=f8.dense()) == -3
    assert af(ldq=128) == -2 and af(seq=136) == -2 and af(d=96) == -2
    assert af(ldq=772) == -4 and af() == -5


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_compute_calls_fail_loudly_without_a_gpu(mxb):
    F = mxb.MxFormat
    fake = C.c_void_p(0x10000)
    rc = mxb.lib.mx_quantize(fake, 0, 4, 64, 64, 1, F(16, 4), fake, fake, None, None)
    assert rc in (-6, -8)
    with pytest.raises(ValueError):
        mxb.mx_quantize(torch.zeros(4, 64), F(16, 4))       # host tensors are refused
