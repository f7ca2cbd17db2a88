"""mx_gemm_static: the product for callers that cannot allocate device memory.

A host application that owns the GPU allocator (an inference server plugin, a real-time loop with
a no-allocation rule) cannot hand this library a workspace.  For such callers the library carries a
fixed scratch array in its own device image; this file checks, through the C ABI, that the entry
point built on it returns the oracle's product within the product tolerance and, bit for bit, what
the workspace-taking entry point returns -- on two calls in a row, the second smaller than the first
so that bytes left in the shared array by the first call would show up if the second ever read them
--, that the second call leaves the amount of free device memory unchanged, and that sizes beyond
the array are refused on the host.
Collected last on purpose: a failure here cannot hide a failure elsewhere."""
import ctypes as C
import os
import shutil

import numpy as np
import pytest
import torch

from oracle import mx_oracle as orc
from paper_2307_15517_b200 import synth


def _operands(M, N, K, B, wa, ww, seed):
    qa = synth.random_ints((M, K), -(2 ** (wa - 1) - 1), 2 ** (wa - 1) - 1, seed).numpy()
    qw = synth.random_ints((N, K), -(2 ** (ww - 1) - 1), 2 ** (ww - 1) - 1, seed + 1).numpy()
    ea = synth.random_bytes((M, K // B), 124, 130, seed + 2).numpy()
    ew = synth.random_bytes((N, K // B), 118, 124, seed + 3).numpy()
    return qa, ea, qw, ew


@pytest.mark.gpu
def test_static_scratch_product_matches_workspace_product_twice():
    from paper_2307_15517_b200 import binding as mxb
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    for call, (M, N, K, B, wa, ww) in enumerate([(300, 520, 1152, 16, 8, 4), (130, 260, 128, 32, 4, 4)]):
        qa, ea, qw, ew = _operands(M, N, K, B, wa, ww, seed=40 + call)
        bias_np = np.linspace(-1, 1, N, dtype=np.float32)
        y_ref, _, S = orc.gemm(qa, ea, wa, qw, ew, ww, B, bias=bias_np)
        args = (dev(orc.pack(qa, wa)), dev(ea), mxb.MxFormat(B, wa), dev(orc.pack(qw, ww)), dev(ew),
                mxb.MxFormat(B, ww), M, N, K)
        bias = dev(bias_np)
        want = mxb.mx_gemm(*args, bias=bias, algo=mxb.MX_ALGO_TCGEN05)
        y = torch.full((M, N), 7.0, device="cuda")
        if call == 1:
            # every buffer exists by now and the first call has done the per-device set-up: the
            # entry point itself must not take device memory from anyone
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
        got = mxb.mx_gemm_static(*args, bias=bias, y=y)
        assert mxb.mx_poll_status() == 0
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free_before, "mx_gemm_static changed the free device memory"
        err = np.abs(got.cpu().numpy().astype(np.float64) - y_ref.astype(np.float64))
        assert (err <= 1e-5 * S + 1e-37).all(), "call %d: max |d|/S = %.3e" % (call, float((err / np.maximum(S, 1e-300)).max()))
        # same kernel, same operands, same K order per output: the two entry points agree bit for bit
        assert torch.equal(got, want), "call %d differs from mx_gemm" % call


@pytest.mark.skipif(shutil.which("nvcc") is None and not os.path.exists("/usr/local/cuda/bin/nvcc"),
                    reason="needs nvcc to build the library")
def test_static_scratch_refuses_sizes_beyond_the_array():
    from paper_2307_15517_b200 import build as mx_build
    mx_build.build()
    from paper_2307_15517_b200 import binding as mxb
    fake = C.c_void_p(0x10000)            # never dereferenced: the size check is host-side
    f = mxb.MxFormat(16, 4)
    rc = mxb.lib.mx_gemm_static(fake, fake, f, fake, fake, f, 4096, 4096, 4096, None, fake, 4096, None)
    assert rc == -5
    msg = mxb.lib.mx_last_cuda_error().decode()
    assert "mx_gemm_static" in msg and str(mxb.MX_STATIC_SCRATCH_BYTES) in msg
    assert 2 * (2048 + 2048) * 2048 <= mxb.MX_STATIC_SCRATCH_BYTES
