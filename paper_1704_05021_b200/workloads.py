"""Seeded synthetic gradients shaped like the paper's two workloads (Section 5).

This module only draws random inputs; it holds none of the method's arithmetic and is the one
piece shared by the CPU oracle's tests and the CUDA path's tests and benchmark.  The paper's
experiments use MNIST and a Romanian-English translation system; neither data set is used
here.  Only the tensor shapes, the batch size of 80 sentences and the skew the paper describes
(most updates near zero, embedding rows untouched by a mini-batch) are taken, and the inputs
below stand in for the real training gradients.

Five workloads, numbered as in the benchmark definition:
  1  flat 2^20, Laplace(0, 1e-3) with 0.5% entries N(0, 1e-1); drop 99%, global, 1 shard, 5 steps
  2  MNIST-shaped MLP (784-4096-4096-10, six tensors), Gaussian per-layer std 1e-2/3e-3/1e-3
     with 1% outliers at 20x std; drop 99%; global or per-layer; 4 shards; 20 steps
  3  NMT-shaped set (two 85000x500 embeddings, 500x85000 output projection + bias, four
     recurrent blocks of 1500x1000 + 1000x1000); embedding gradients row-sparse (rows = the
     tokens of 80 sentences x 50 tokens drawn Zipf(1.1) over 85000 words, values N(0, 1e-3)),
     dense tensors N(0, 1e-4); drop 99% per layer; 4 shards; 20 steps
  4  workload 3 with two-value quantisation after dropping; parameter shards N(0, 0.01)
  5  flat 2^30, Laplace(0, 1e-3) with 0.1% entries N(0, 1e-1); drop 99.9%, global, 8 shards, 10 steps
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import torch

SCOPE_GLOBAL = 0
SCOPE_PER_LAYER = 1
VALUES_FP32 = 0
VALUES_TWO_MEANS = 1
VALUES_THRESHOLD = 2
VALUES_COLUMN_MEANS = 3

_CHUNK = 1 << 24  # elements generated per call of the random generator (bounds temporaries)


@dataclass
class Workload:
    name: str
    config: int
    layer_names: List[str]
    layer_shapes: List[Tuple[int, ...]]
    drop_ppm: int
    scope_mode: int
    value_mode: int
    n_shards: int
    steps: int
    layer_off: List[int] = field(default_factory=list)
    shard_off: List[int] = field(default_factory=list)

    def __post_init__(self):
        off = [0]
        for shp in self.layer_shapes:
            cnt = 1
            for d in shp:
                cnt *= d
            off.append(off[-1] + cnt)
        self.layer_off = off
        n = off[-1]
        chunk = -(-n // self.n_shards)
        self.shard_off = [min(j * chunk, n) for j in range(self.n_shards + 1)]

    @property
    def n(self) -> int:
        return self.layer_off[-1]

    @property
    def layer_cols(self) -> List[int]:
        """Columns of each layer seen as a row-major matrix (1 for vectors): the last dimension of its shape."""
        return [int(shp[-1]) if len(shp) > 1 else 1 for shp in self.layer_shapes]

    def seed(self, step: int) -> int:
        return step if self.config == 1 else 1000 * self.config + step


_MNIST_SHAPES = [(784, 4096), (4096,), (4096, 4096), (4096,), (4096, 10), (10,)]
_MNIST_NAMES = ["W1", "b1", "W2", "b2", "W3", "b3"]
_MNIST_STD = [1e-2, 1e-2, 3e-3, 3e-3, 1e-3, 1e-3]

_NMT_VOCAB, _NMT_EMB = 85000, 500
_NMT_SHAPES = ([(_NMT_VOCAB, _NMT_EMB), (_NMT_VOCAB, _NMT_EMB), (_NMT_EMB, _NMT_VOCAB), (_NMT_VOCAB,)]
               + [(1500, 1000), (1000, 1000)] * 4)
_NMT_NAMES = (["src_emb", "tgt_emb", "out_W", "out_b"]
              + [f"gru{b}_{w}" for b in range(4) for w in ("Wx", "Wh")])


def workload(config: int, *, scope_mode: int | None = None, scale_log2: int | None = None) -> Workload:
    """The description of workload `config` (1..5).

    scope_mode overrides the threshold scope (workload 2 is run both ways); scale_log2 replaces
    the length of the flat workloads 1 and 5 (used by tests that need a smaller or ragged size).
    """
    if config == 1:
        n = 1 << (20 if scale_log2 is None else scale_log2)
        return Workload("flat-2^20-laplace", 1, ["flat"], [(n,)], 990_000,
                        SCOPE_GLOBAL if scope_mode is None else scope_mode, VALUES_FP32, 1, 5)
    if config == 2:
        return Workload("mnist-mlp", 2, list(_MNIST_NAMES), list(_MNIST_SHAPES), 990_000,
                        SCOPE_GLOBAL if scope_mode is None else scope_mode, VALUES_FP32, 4, 20)
    if config in (3, 4):
        return Workload("nmt" if config == 3 else "nmt-two-means", config, list(_NMT_NAMES),
                        list(_NMT_SHAPES), 990_000,
                        SCOPE_PER_LAYER if scope_mode is None else scope_mode,
                        VALUES_FP32 if config == 3 else VALUES_TWO_MEANS, 4, 20)
    if config == 5:
        n = 1 << (30 if scale_log2 is None else scale_log2)
        return Workload("flat-2^30-laplace", 5, ["flat"], [(n,)], 999_000,
                        SCOPE_GLOBAL if scope_mode is None else scope_mode, VALUES_FP32, 8, 10)
    raise ValueError("config must be 1..5")


def _generator(device, seed: int) -> torch.Generator:
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    return gen


def _fill_laplace_with_outliers(out: torch.Tensor, gen, scale: float, p_out: float, std_out: float):
    n = out.numel()
    for lo in range(0, n, _CHUNK):
        hi = min(lo + _CHUNK, n)
        part = out[lo:hi]
        u = torch.rand(hi - lo, generator=gen, device=out.device, dtype=torch.float32) - 0.5
        # inverse CDF of Laplace(0, scale); the clamp keeps rand() == 0 finite (|x| <= ~17.3 * scale)
        lap = -scale * torch.sign(u) * torch.log((1.0 - 2.0 * u.abs()).clamp_min(2.0 ** -25))
        pick = torch.rand(hi - lo, generator=gen, device=out.device, dtype=torch.float32) < p_out
        big = torch.randn(hi - lo, generator=gen, device=out.device, dtype=torch.float32) * std_out
        part.copy_(torch.where(pick, big, lap))
        del u, lap, pick, big


def _fill_gauss_with_outliers(out: torch.Tensor, gen, std: float, p_out: float, factor: float):
    n = out.numel()
    for lo in range(0, n, _CHUNK):
        hi = min(lo + _CHUNK, n)
        z = torch.randn(hi - lo, generator=gen, device=out.device, dtype=torch.float32)
        pick = torch.rand(hi - lo, generator=gen, device=out.device, dtype=torch.float32) < p_out
        out[lo:hi].copy_(z * torch.where(pick, std * factor, std))
        del z, pick


def _fill_row_sparse(out2d: torch.Tensor, gen, tokens: int, zipf_s: float, std: float):
    rows, width = out2d.shape
    out2d.zero_()
    ranks = torch.arange(1, rows + 1, device=out2d.device, dtype=torch.float64)
    prob = ranks.pow(-zipf_s)
    prob = (prob / prob.sum()).to(torch.float32)
    tok = torch.multinomial(prob, tokens, replacement=True, generator=gen)
    hit = torch.unique(tok)
    vals = torch.randn(hit.numel(), width, generator=gen, device=out2d.device, dtype=torch.float32) * std
    out2d[hit] = vals


def make_gradient(w: Workload, step: int, device="cpu", out: torch.Tensor | None = None) -> torch.Tensor:
    """The flat fp32 gradient of workload `w` at `step` (seeded; same call, same bytes)."""
    device = torch.device(device)
    if out is None:
        out = torch.empty(w.n, dtype=torch.float32, device=device)
    assert out.numel() == w.n and out.dtype == torch.float32 and out.is_contiguous()
    gen = _generator(out.device, w.seed(step))
    if w.config == 1:
        _fill_laplace_with_outliers(out, gen, 1e-3, 0.005, 1e-1)
    elif w.config == 5:
        _fill_laplace_with_outliers(out, gen, 1e-3, 0.001, 1e-1)
    elif w.config == 2:
        for li, std in enumerate(_MNIST_STD):
            _fill_gauss_with_outliers(out[w.layer_off[li]:w.layer_off[li + 1]], gen, std, 0.01, 20.0)
    else:
        for li, shp in enumerate(w.layer_shapes):
            part = out[w.layer_off[li]:w.layer_off[li + 1]]
            if li < 2:
                _fill_row_sparse(part.view(*shp), gen, 80 * 50, 1.1, 1e-3)
            else:
                _fill_gauss_with_outliers(part, gen, 1e-4, 0.0, 1.0)
    return out


def make_params(w: Workload, device="cpu") -> torch.Tensor:
    """The flat fp32 parameters the shards start from: N(0, 0.01) for workload 4, zeros otherwise."""
    device = torch.device(device)
    p = torch.zeros(w.n, dtype=torch.float32, device=device)
    if w.config == 4:
        gen = _generator(device, 4999)
        for lo in range(0, w.n, _CHUNK):
            hi = min(lo + _CHUNK, w.n)
            p[lo:hi].copy_(torch.randn(hi - lo, generator=gen, device=device, dtype=torch.float32) * 0.01)
    return p


def small_layered(n_layers: int, sizes: List[int], drop_ppm: int, scope_mode: int, value_mode: int,
                  n_shards: int) -> Workload:
    """A free-form layered workload for tests (ragged sizes, tiny layers, empty layers)."""
    assert len(sizes) == n_layers
    w = Workload("custom", 2, [f"L{i}" for i in range(n_layers)], [(s,) for s in sizes], drop_ppm,
                 scope_mode, value_mode, n_shards, 1)
    return w
