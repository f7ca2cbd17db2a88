"""Full-size parity: the paper-shaped workloads at the sizes the benchmark runs (OPT-1.3B prefill
linears, LLaMA-7B mixed-precision linears), in the launch configuration bench.py times
(mx_linear, default algorithm).  The oracle quantizes the full tensors (bit-exact comparison of
sampled rows of the GPU quantizer) and computes sampled outputs one by one."""
import numpy as np
import pytest
import torch

from oracle import mx_oracle as orc
from paper_2307_15517_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-5
N_SAMPLES = 768


@pytest.fixture(scope="module")
def mxb():
    from paper_2307_15517_b200 import binding
    return binding


def _check_layer(mxb, x, w, block, wa, ww, seed):
    M, K = x.shape
    N = w.shape[0]
    fa, fw = mxb.MxFormat(block, wa), mxb.MxFormat(block, ww)
    qa, ea, _ = orc.quantize(x.numpy(), block, wa)
    qw, ew, _ = orc.quantize(w.numpy(), block, ww)
    w_mant, w_exp = mxb.mx_quantize(w.cuda(), fw)
    a_mant, a_exp = mxb.mx_quantize(x.cuda(), fa)
    rng = np.random.default_rng(seed)
    rows = rng.choice(N, 64, replace=False)
    assert np.array_equal(w_mant[torch.from_numpy(rows).cuda()].cpu().numpy(), orc.pack(qw[rows], ww))
    assert np.array_equal(w_exp.cpu().numpy(), ew)
    assert np.array_equal(a_exp.cpu().numpy(), ea)
    rows = rng.choice(M, 64, replace=False)
    assert np.array_equal(a_mant[torch.from_numpy(rows).cuda()].cpu().numpy(), orc.pack(qa[rows], wa))
    y = mxb.mx_linear(x.cuda(), fa, w_mant, w_exp, fw, N)
    assert mxb.mx_poll_status() == 0
    si, sj = rng.integers(0, M, N_SAMPLES), rng.integers(0, N, N_SAMPLES)
    y_ref, _, S = orc.gemm_samples(qa, ea, wa, qw, ew, ww, block, si, sj)
    got = y.cpu().numpy()[si, sj].astype(np.float64)
    err = np.abs(got - y_ref)
    assert (err <= TOL * S + 1e-37).all(), float((err / np.maximum(S, 1e-300)).max())
    assert np.isfinite(y.cpu().numpy()).all()


@pytest.mark.parametrize("layer", range(4))
def test_opt13b_prefill_layer(mxb, layer):
    x, w, spec = synth.opt13b_inputs(layer, seed=0)
    _check_layer(mxb, x, w, spec.block, spec.w_act, spec.w_wgt, seed=layer)


@pytest.mark.parametrize("layer", (0, 3, 4, 6))
def test_llama7b_mixed_precision_layer(mxb, layer):
    """q, o, gate and down projections with the widths and block size drawn for seed 0."""
    spec = synth.llama7b_mixed_layers(0)[layer]
    x, w = synth.llama7b_inputs(spec, layer, seed=0)
    _check_layer(mxb, x, w, spec.block, spec.w_act, spec.w_wgt, seed=10 + layer)


def test_llama7b_layer_specs_average_about_four_bits():
    widths = []
    for seed in range(3):
        for s in synth.llama7b_mixed_layers(seed):
            widths += [s.w_act, s.w_wgt]
            assert s.block in (16, 32) and s.w_act in synth.WIDTH_CHOICES
    assert 3.0 <= float(np.mean(widths)) <= 5.2
