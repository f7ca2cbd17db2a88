"""GPU parity of the decode path (few tokens, weights streamed once) against the CPU oracle.
When the row tiles alone fill the GPU the kernel adds each output's blocks in ascending order with
one fp32 rounding per block and must equal the oracle's sequential-fp32 result bit for bit; when K
is cut over warps (single small layers) the result must stay within 1e-5 * S of the exact value."""
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


def _layer(mxb, T, K, N, seed, wa=8, ww=4, with_bias=False, heavy=False):
    x = synth.student_t_activations(T, K, seed) if heavy else synth.decode_activations(T, K, seed)
    w = synth.gaussian_weights(N, K, seed + 1)
    bias = synth.gaussian_weights(1, N, seed + 2, std=1.0)[0] if with_bias else None
    fa, fw = mxb.MxFormat(32, wa), mxb.MxFormat(32, ww)
    qa, ea, _ = orc.quantize(x.numpy(), 32, wa)
    qw, ew, _ = orc.quantize(w.numpy(), 32, ww)
    dev = dict(x=x.cuda(), fa=fa, fw=fw, N=N, bias=None if bias is None else bias.cuda(),
               w_mant=torch.from_numpy(orc.pack(qw, ww)).cuda(), w_exp=torch.from_numpy(ew).cuda(),
               y=torch.full((T, N), -5.0, device="cuda"))
    ref = dict(qa=qa, ea=ea, qw=qw, ew=ew, wa=wa, ww=ww, bias=None if bias is None else bias.numpy())
    return dev, ref


def _oracle(ref):
    return orc.gemm(ref["qa"], ref["ea"], ref["wa"], ref["qw"], ref["ew"], ref["ww"], 32, bias=ref["bias"])


@pytest.mark.parametrize("T", (1, 4, 8, 16))
@pytest.mark.parametrize("shape", [(1024, 512), (4096, 272), (128, 40)])
def test_stream_single_layer_within_tolerance(mxb, T, shape):
    K, N = shape
    dev, ref = _layer(mxb, T, K, N, seed=T + K, with_bias=True, heavy=True)
    y_ref, y_seq, S = _oracle(ref)
    y = mxb.mx_linear(dev["x"], dev["fa"], dev["w_mant"], dev["w_exp"], dev["fw"], N, bias=dev["bias"],
                      y=dev["y"], algo=mxb.MX_ALGO_STREAM)
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
    assert (err <= TOL * S + 1e-37).all(), float((err / np.maximum(S, 1e-300)).max())
    # AUTO picks the same kernel for these shapes
    y2 = mxb.mx_linear(dev["x"], dev["fa"], dev["w_mant"], dev["w_exp"], dev["fw"], N, bias=dev["bias"])
    assert torch.equal(y, y2)


@pytest.mark.parametrize("T,n_layers,K", [(1, 20, 256), (4, 20, 256), (16, 10, 256),
                                          (4, 20, 512), (16, 20, 1024), (1, 20, 1536)])
def test_grouped_launch_is_bit_exact_against_sequential_oracle(mxb, T, n_layers, K):
    """Enough row tiles to fill the GPU without cutting K: ascending fp32 block sums, exactly.
    K = 256 takes the register-prefetch kernel, K % 512 == 0 the bulk-copy staged one."""
    N = 4096
    layers, refs = [], []
    for i in range(n_layers):
        dev, ref = _layer(mxb, T, K, N, seed=100 * T + 3 * i, wa=(8, 6, 4)[i % 3], ww=(4, 3, 2)[i % 3],
                          with_bias=(i % 2 == 0))
        if i % 4 == 1:                          # layers sharing one activation tensor (q, k, v)
            dev["x"], dev["fa"] = layers[-1]["x"], layers[-1]["fa"]
            ref["qa"], ref["ea"], ref["wa"] = refs[-1]["qa"], refs[-1]["ea"], refs[-1]["wa"]
        layers.append(dev)
        refs.append(ref)
    args = mxb.make_linear_args(layers)
    mxb.mx_linear_grouped(args)
    assert mxb.mx_poll_status() == 0
    for dev, ref in zip(layers, refs):
        y_ref, y_seq, S = _oracle(ref)
        assert np.array_equal(dev["y"].cpu().numpy(), y_seq)


def test_stream_mixed_layer_shapes_and_nonfinite(mxb):
    """Different N and K per layer, a ragged last row tile, a poisoned weight and token block."""
    specs = [(4, 512, 1000), (4, 1024, 48), (3, 128, 4096), (4, 512, 1000)]
    layers, refs = [], []
    for i, (T, K, N) in enumerate(specs):
        dev, ref = _layer(mxb, T, K, N, seed=50 + i, with_bias=(i == 1))
        layers.append(dev)
        refs.append(ref)
    refs[2]["ew"][7, 1] = 255
    layers[2]["w_exp"] = torch.from_numpy(refs[2]["ew"]).cuda()
    x3 = layers[3]["x"].clone()
    x3[1, 40] = float("inf")
    layers[3]["x"] = x3
    refs[3]["qa"], refs[3]["ea"], _ = orc.quantize(x3.cpu().numpy(), 32, 8)
    mxb.mx_linear_grouped(mxb.make_linear_args(layers))
    for dev, ref in zip(layers, refs):
        y_ref, y_seq, S = _oracle(ref)
        y = dev["y"].cpu().numpy()
        assert np.array_equal(np.isnan(y), np.isnan(y_ref))
        ok = ~np.isnan(y_ref)
        assert (np.abs(y[ok].astype(np.float64) - y_ref[ok]) <= TOL * S[ok] + 1e-37).all()
    assert np.isnan(layers[2]["y"][:, 7].cpu().numpy()).all()
    assert np.isnan(layers[3]["y"][1].cpu().numpy()).all() and not np.isnan(layers[3]["y"][0].cpu().numpy()).any()


def test_decode_shapes_sampled(mxb):
    """The decode configuration's own shapes (4096 -> 4096 and 4096 -> 11008, 16 tokens):
    every output of 64 sampled weight rows against the oracle."""
    for N in (4096, 11008):
        dev, ref = _layer(mxb, 16, 4096, N, seed=N)
        y = mxb.mx_linear(dev["x"], dev["fa"], dev["w_mant"], dev["w_exp"], dev["fw"], N, y=dev["y"])
        rows = np.random.default_rng(N).choice(N, 64, replace=False)
        si, sj = np.meshgrid(np.arange(16), rows, indexing="ij")
        y_ref, y_seq, S = orc.gemm_samples(ref["qa"], ref["ea"], 8, ref["qw"], ref["ew"], 4, 32, si.ravel(), sj.ravel())
        got = y.cpu().numpy()[si.ravel(), sj.ravel()].astype(np.float64)
        assert (np.abs(got - y_ref) <= TOL * S + 1e-37).all()


def test_gemm_on_packed_activations_streams_too(mxb):
    """mx_gemm with already quantized tokens (M <= 16) takes the same kernel, no quantize launch."""
    dev, ref = _layer(mxb, 8, 1024, 640, seed=77, with_bias=True)
    y_ref, y_seq, S = _oracle(ref)
    a_mant = torch.from_numpy(orc.pack(ref["qa"], 8)).cuda()
    a_exp = torch.from_numpy(ref["ea"]).cuda()
    for algo in (mxb.MX_ALGO_STREAM, mxb.MX_ALGO_AUTO):
        y = mxb.mx_gemm(a_mant, a_exp, dev["fa"], dev["w_mant"], dev["w_exp"], dev["fw"], 8, 640, 1024,
                        bias=dev["bias"], algo=algo)
        err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
        assert (err <= TOL * S + 1e-37).all()
    y_tc = mxb.mx_gemm(a_mant, a_exp, dev["fa"], dev["w_mant"], dev["w_exp"], dev["fw"], 8, 640, 1024,
                       bias=dev["bias"], algo=mxb.MX_ALGO_TCGEN05)
    assert (np.abs(y_tc.cpu().numpy().astype(np.float64) - y_ref) <= TOL * S + 1e-37).all()


def test_stream_rejects_what_it_cannot_stage(mxb):
    dev, _ = _layer(mxb, 4, 256, 64, seed=1)
    with pytest.raises(mxb.MxError):                       # block 16 weights are not streamable
        mxb.mx_linear(dev["x"], mxb.MxFormat(16, 8), dev["w_mant"], dev["w_exp"], mxb.MxFormat(16, 4), 64,
                      algo=mxb.MX_ALGO_STREAM)
    x17 = torch.zeros(17, 256, device="cuda")
    with pytest.raises(mxb.MxError):                       # more than 16 tokens
        mxb.mx_linear(x17, dev["fa"], dev["w_mant"], dev["w_exp"], dev["fw"], 64, algo=mxb.MX_ALGO_STREAM)
