"""Seeded synthetic inputs with the shapes and value structure of the paper's workloads.

The paper evaluates OPT and LLaMA checkpoints on text datasets; neither is available here, so
tensors with those models' layer shapes stand in for them: Gaussian weights of small variance,
activations with a few large "outlier" channels or heavy tails (the large per-tensor variance
spread the paper shows in Fig. 1(a) is what motivates block scaling).

This module draws random numbers and nothing else: no quantization, no exponent or
rounding arithmetic lives here, so both the CUDA tests and the CPU oracle can use it.
Everything is generated on the host with a seeded ``torch.Generator`` so that both sides
see identical bits.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import torch

#: mantissa widths (sign included) a layer may take, and how often: mean 4.1 bits, shaped
#: like the per-tensor width histogram of Fig. 1(b).
WIDTH_CHOICES = (2, 3, 4, 5, 6, 8)
WIDTH_PMF = (0.10, 0.25, 0.35, 0.15, 0.10, 0.05)


@dataclass(frozen=True)
class LayerSpec:
    name: str
    K: int          # input features (reduction dimension)
    N: int          # output features
    block: int      # elements sharing one exponent along K
    w_act: int      # signed mantissa width of activations
    w_wgt: int      # signed mantissa width of weights


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def gaussian_weights(N: int, K: int, seed: int, std: float = 0.02) -> torch.Tensor:
    """W[N, K] ~ N(0, std^2), fp32, row-major (the nn.Linear layout)."""
    return torch.randn(N, K, generator=_gen(seed), dtype=torch.float32) * std


def outlier_activations(M: int, K: int, seed: int, n_outlier: int, gain: float) -> torch.Tensor:
    """X[M, K] ~ N(0,1) with ``n_outlier`` randomly chosen input channels scaled by ``gain``."""
    g = _gen(seed)
    x = torch.randn(M, K, generator=g, dtype=torch.float32)
    if n_outlier > 0:
        idx = torch.randperm(K, generator=g)[:n_outlier]
        x[:, idx] *= gain
    return x


def student_t_activations(M: int, K: int, seed: int, nu: int = 3) -> torch.Tensor:
    """Heavy-tailed activations: z / sqrt(chi2_nu / nu) with z ~ N(0,1)."""
    g = _gen(seed)
    z = torch.randn(M, K, generator=g, dtype=torch.float32)
    chi2 = torch.zeros(M, K, dtype=torch.float32)
    for _ in range(nu):
        chi2 += torch.randn(M, K, generator=g, dtype=torch.float32) ** 2
    return z / torch.sqrt(chi2 / nu)


# ---------------------------------------------------------------------------------------
# The five workloads
# ---------------------------------------------------------------------------------------

def single_layer(seed: int = 0) -> Tuple[torch.Tensor, torch.Tensor, LayerSpec]:
    """One linear layer: X 128x768, W 768x768 ~ N(0,1), 4 outlier channels x50; B=16, w=4."""
    g = _gen(seed)
    x = torch.randn(128, 768, generator=g, dtype=torch.float32)
    w = torch.randn(768, 768, generator=g, dtype=torch.float32)
    idx = torch.randperm(768, generator=g)[:4]
    x[:, idx] *= 50.0
    return x, w, LayerSpec("single", 768, 768, 16, 4, 4)


def opt13b_prefill_layers() -> List[LayerSpec]:
    """OPT-1.3B-shaped prefill linears (hidden 2048, FFN 8192); MXInt4, block 16."""
    return [
        LayerSpec("qkv", 2048, 6144, 16, 4, 4),
        LayerSpec("out_proj", 2048, 2048, 16, 4, 4),
        LayerSpec("ffn_up", 2048, 8192, 16, 4, 4),
        LayerSpec("ffn_down", 8192, 2048, 16, 4, 4),
    ]


OPT13B_TOKENS = 2048


def opt13b_inputs(layer_index: int, tokens: int = OPT13B_TOKENS, seed: int = 0):
    """(X[tokens,K], W[N,K], spec) of one OPT-1.3B-shaped layer; 0.5% outlier channels x40."""
    spec = opt13b_prefill_layers()[layer_index]
    n_out = -(-spec.K * 5 // 1000)  # ceil(0.005 K)
    x = outlier_activations(tokens, spec.K, 1000 * seed + 2 * layer_index, n_out, 40.0)
    w = gaussian_weights(spec.N, spec.K, 1000 * seed + 2 * layer_index + 1)
    return x, w, spec


LLAMA7B_TOKENS = 4096


def llama7b_mixed_layers(seed: int = 0) -> List[LayerSpec]:
    """LLaMA-7B-shaped linears with per-layer widths drawn from WIDTH_PMF and block in {16,32}."""
    g = _gen(7000 + seed)
    shapes = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
              ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096)]
    pmf = torch.tensor(WIDTH_PMF, dtype=torch.float64)
    out = []
    for name, K, N in shapes:
        wi = torch.multinomial(pmf, 2, replacement=True, generator=g)
        blk = (16, 32)[int(torch.randint(0, 2, (1,), generator=g))]
        out.append(LayerSpec(name, K, N, blk, WIDTH_CHOICES[int(wi[0])], WIDTH_CHOICES[int(wi[1])]))
    return out


def llama7b_inputs(spec: LayerSpec, layer_index: int, tokens: int = LLAMA7B_TOKENS, seed: int = 0):
    x = student_t_activations(tokens, spec.K, 3000 * (seed + 1) + 2 * layer_index)
    w = gaussian_weights(spec.N, spec.K, 3000 * (seed + 1) + 2 * layer_index + 1)
    return x, w


def decode_layer_shapes() -> List[Tuple[str, int, int]]:
    """Per decoder layer: four 4096->4096 and two 4096->11008 weight matrices."""
    return [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
            ("gate", 4096, 11008), ("up", 4096, 11008)]


DECODE_LAYERS = 32
DECODE_TOKEN_BATCHES = (1, 4, 16)
DECODE_SPEC = dict(block=32, w_act=8, w_wgt=4)


def decode_activations(tokens: int, K: int = 4096, seed: int = 0) -> torch.Tensor:
    return torch.randn(tokens, K, generator=_gen(5000 + seed), dtype=torch.float32)


def decoder_block_shapes():
    """OPT-6.7B-shaped decoder block: hidden 4096, 32 heads x 128, FFN 16384, sequence 2048."""
    return dict(hidden=4096, heads=32, head_dim=128, ffn=16384, seq=2048, block=16,
                w_act=8, w_wgt=4)


def random_ints(shape, lo: int, hi: int, seed: int) -> torch.Tensor:
    """Uniform integers in [lo, hi] (inclusive) as int8 -- raw mantissas for GEMM-only tests."""
    return torch.randint(lo, hi + 1, shape, generator=_gen(seed), dtype=torch.int32).to(torch.int8)


def random_bytes(shape, lo: int, hi: int, seed: int) -> torch.Tensor:
    """Uniform integers in [lo, hi] (inclusive) as uint8 -- raw exponent bytes."""
    return torch.randint(lo, hi + 1, shape, generator=_gen(seed), dtype=torch.int32).to(torch.uint8)
