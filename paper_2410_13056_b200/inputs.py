"""Seeded synthetic inputs shaped like the paper's LLM layers.

This module holds input generation only -- none of the method's arithmetic -- so
that the CUDA library's tests, the benchmark and the CPU checker can all be fed
the same bytes.  Real LLaMA weights and C4 calibration text (Section 4.1 of the
paper: 128 segments of 2048 tokens) are replaced by random tensors that keep the
layer shapes, the storage dtype, the heavy-tailed weight entries and the
channel-wise activation outliers shown in the paper's activation figure.

Recipe
  W [d_in][d_out] : N(0, 0.02^2); a Bernoulli(0.005) subset of the entries is
                    replaced by 0.1 * StudentT(df=3); clamped to |w| <= 8;
                    rounded to the 16-bit dtype; |w| < 2^-24 flushed to +0.
  X [n][d_in]     : X[t,j] = z * sigma_j, z ~ N(0,1), sigma_j = exp(N(0,1)),
                    multiplied by 50 on a random set of outlier channels
                    (a fixed count, or round(0.01 * d_in)); clamped to +-60000
                    for fp16; rounded to the dtype.
Generation runs on whatever device is asked for with a torch.Generator seeded
there, in fixed-size row chunks, so a (seed, device type) pair fixes the bytes.
"""
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import torch

F16 = 0
BF16 = 1

_TORCH_DTYPE = {F16: torch.float16, BF16: torch.bfloat16}
_W_CHUNK_ROWS = 1024
_X_CHUNK_ROWS = 8192


def torch_dtype(dtype_code: int) -> torch.dtype:
    return _TORCH_DTYPE[dtype_code]


def make_weight(d_in: int, d_out: int, dtype_code: int, seed: int, device="cpu") -> torch.Tensor:
    """Weight matrix in the library's layout: row i = input channel i, d_out contiguous weights."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed))
    out = torch.empty((d_in, d_out), dtype=_TORCH_DTYPE[dtype_code], device=dev)
    for r0 in range(0, d_in, _W_CHUNK_ROWS):
        r1 = min(d_in, r0 + _W_CHUNK_ROWS)
        shape = (r1 - r0, d_out)
        w = torch.randn(shape, generator=g, device=dev, dtype=torch.float32) * 0.02
        mask = torch.rand(shape, generator=g, device=dev) < 0.005
        z = torch.randn(shape, generator=g, device=dev, dtype=torch.float32)
        chi = torch.randn((3,) + shape, generator=g, device=dev, dtype=torch.float32).square().sum(0)
        t3 = z / torch.sqrt(chi / 3.0)
        w = torch.where(mask, 0.1 * t3, w).clamp_(-8.0, 8.0)
        w16 = w.to(_TORCH_DTYPE[dtype_code])
        w16 = torch.where(w16.float().abs() < 2.0 ** -24, torch.zeros_like(w16), w16)
        out[r0:r1] = w16
    return out


def make_activations(n_tokens: int, d_in: int, dtype_code: int, seed: int, device="cpu",
                     n_outlier_channels: Optional[int] = None) -> torch.Tensor:
    """Calibration activations [n_tokens][d_in] with channel-wise outliers."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(int(seed) + 7919)
    sigma = torch.exp(torch.randn(d_in, generator=g, device=dev, dtype=torch.float32))
    if n_outlier_channels is None:
        n_outlier_channels = int(round(0.01 * d_in))
    chosen = torch.randperm(d_in, generator=g, device=dev)[:n_outlier_channels]
    sigma[chosen] *= 50.0
    out = torch.empty((n_tokens, d_in), dtype=_TORCH_DTYPE[dtype_code], device=dev)
    for r0 in range(0, n_tokens, _X_CHUNK_ROWS):
        r1 = min(n_tokens, r0 + _X_CHUNK_ROWS)
        x = torch.randn((r1 - r0, d_in), generator=g, device=dev, dtype=torch.float32) * sigma
        if dtype_code == F16:
            x.clamp_(-60000.0, 60000.0)
        out[r0:r1] = x.to(_TORCH_DTYPE[dtype_code])
    return out


def as_u16(t: torch.Tensor):
    """The raw 16-bit patterns of an fp16/bf16 tensor as a numpy uint16 array (host copy)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view("uint16")


def make_quantized_layer(d_in: int, d_out: int, counts: Tuple[int, int, int], dtype_code: int, seed: int,
                         n_act: int = 0, n_q: int = 0):
    """A random ALREADY-QUANTIZED layer for the inference product, as host numpy arrays: bit widths with
    counts[0], counts[1], counts[2] channels of 2, 3, 4 bits at random positions, uniformly random byte
    codes below 2^bits, ascending N(0, 0.02^2) look-up tables (unused entries 0), an outlier list of
    n_act whole random rows plus n_q distinct random entries elsewhere (sorted by (row, col), values
    0.1 * N(0,1) in the dtype), and one input token with the channel scales of make_activations.
    Nothing here quantizes anything: the arrays only have the shapes and value ranges a quantized
    layer has."""
    import numpy as np

    assert sum(counts) == d_in
    g = np.random.default_rng(int(seed))
    bits = np.repeat(np.array([2, 3, 4], np.uint8), counts)[g.permutation(d_in)]
    codes = (g.integers(0, 16, size=(d_in, d_out), dtype=np.uint8) & ((1 << bits) - 1)[:, None]).astype(np.uint8)
    lut = np.sort(g.normal(0.0, 0.02, size=(d_in, 16)).astype(np.float32), axis=1)
    lut[np.arange(16)[None, :] >= (1 << bits.astype(np.int64))[:, None]] = 0.0
    act_rows = np.sort(g.choice(d_in, size=n_act, replace=False)) if n_act else np.zeros(0, np.int64)
    lin = [np.add.outer(act_rows * d_out, np.arange(d_out)).reshape(-1)]
    if n_q:
        free_rows = np.setdiff1d(np.arange(d_in), act_rows)
        pick = g.choice(free_rows.size * d_out, size=n_q, replace=False)
        lin.append(free_rows[pick // d_out] * d_out + pick % d_out)
    lin = np.sort(np.concatenate(lin).astype(np.int64))
    rows, cols = (lin // d_out).astype(np.int32), (lin % d_out).astype(np.int32)
    vals = as_u16(torch.from_numpy(0.1 * g.normal(size=lin.size)).to(_TORCH_DTYPE[dtype_code]))
    sigma = np.exp(g.normal(size=d_in))
    sigma[g.permutation(d_in)[: int(round(0.01 * d_in))]] *= 50.0
    x = torch.from_numpy(g.normal(size=d_in) * sigma).to(_TORCH_DTYPE[dtype_code])
    return dict(bits=bits, codes=codes, lut=lut, rows=rows, cols=cols, vals=vals, x=as_u16(x))


@dataclass(frozen=True)
class Layer:
    d_in: int
    d_out: int


@dataclass(frozen=True)
class Config:
    """One workload: layers (d_in, d_out), storage dtype, calibration tokens, budgets, Lloyd iterations."""
    name: str
    layers: Tuple[Layer, ...]
    dtype: int
    n_tokens: int
    budgets: Tuple[float, ...]
    lloyd_iters: int
    seed: int
    n_outlier_channels: Optional[int] = None  # None -> round(0.01 * d_in)
    repeat: int = 1  # how many times the layer list occurs (transformer blocks)


# Shapes are given in the paper's orientation: d_in input channels of d_out weights each.
_ATTN = Layer(4096, 4096)
_UP = Layer(4096, 11008)
_DOWN = Layer(11008, 4096)

CONFIGS = {
    "c1_small": Config("c1_small", (Layer(512, 512),), F16, 512, (3.0,), 10, 0, n_outlier_channels=8),
    "c2_attn7b": Config("c2_attn7b", (_ATTN,), BF16, 131072, (2.2,), 20, 2000),
    "c3_mlp7b": Config("c3_mlp7b", (_UP, _DOWN), BF16, 131072, (2.0, 2.5, 3.0, 3.5, 4.0), 20, 3000),
    "c4_stack7b": Config("c4_stack7b", (_ATTN, _ATTN, _ATTN, _ATTN, _UP, _UP, _DOWN), BF16, 131072,
                         (3.0,), 20, 4000, repeat=32),
    "c5_mlp70b": Config("c5_mlp70b", (Layer(8192, 28672), Layer(28672, 8192)), BF16, 65536, (2.5,),
                        20, 5000),
}


def layer_seed(cfg: Config, layer_index: int) -> int:
    return cfg.seed + layer_index


def stack_layers(cfg: Config) -> List[Tuple[int, int, Layer]]:
    """Every layer of a multi-block workload in order: (block, index inside the block, layer)."""
    return [(b, i, L) for b in range(cfg.repeat) for i, L in enumerate(cfg.layers)]


def stack_layer_seed(cfg: Config, block: int, index: int) -> int:
    """Seed of one layer's weights in a multi-block workload (distinct for every layer)."""
    return cfg.seed + len(cfg.layers) * block + index


class StackInputs:
    """Inputs of a multi-block workload, layer by layer: every layer has its own seeded weights (drawn
    when asked for, into one buffer per shape so that addresses stay fixed); the calibration activations
    are drawn once per distinct input width and shared by the layers of that width (the statistic's cost
    does not depend on the values, and a gigabyte per layer would only lengthen the preparation)."""

    def __init__(self, cfg: Config, device="cuda"):
        self.cfg, self.device = cfg, device
        self.layers = stack_layers(cfg)
        self._X, self._W = {}, {}

    def shapes(self) -> List[Tuple[int, int]]:
        return [(L.d_in, L.d_out) for _, _, L in self.layers]

    def activations(self, d_in: int) -> torch.Tensor:
        if d_in not in self._X:
            self._X[d_in] = make_activations(self.cfg.n_tokens, d_in, self.cfg.dtype, self.cfg.seed + d_in,
                                             device=self.device)
        return self._X[d_in]

    def weights(self, shape: Tuple[int, int]) -> torch.Tensor:
        """The buffer that holds the weights of the layer of this shape drawn last."""
        return self._W[shape]

    def __call__(self, k: int):
        b, i, L = self.layers[k]
        W = make_weight(L.d_in, L.d_out, self.cfg.dtype, stack_layer_seed(self.cfg, b, i), device=self.device)
        buf = self._W.setdefault((L.d_in, L.d_out), W)
        if buf is not W:
            buf.copy_(W)
        return self.activations(L.d_in), buf
