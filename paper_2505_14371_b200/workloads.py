"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle harness.

This module holds no arithmetic of the quantizer or of QODA: it only describes layer
shapes and draws random values.  Both the CUDA path and the CPU oracle are fed from
the tensors made here, so the two sides always see the same bits.

The paper trains a WGAN on CIFAR and a Transformer-XL on WikiText-103 (Section 7);
those datasets are not available, so the gradient sets below only take the *shapes*
of those models and draw heavy-tailed values per layer.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import torch

SEED_BASE = 20250514
PHILOX_SEED = 0x5EED0DA


@dataclass
class Workload:
    """A ragged list of layers plus the recipe for the values of each layer."""
    name: str
    layer_sizes: List[int]
    bits: int
    q: int                    # 0 means the infinity norm
    num_workers: int
    dist: str                 # "normal" | "laplace" | "student3"
    scales: List[float] = field(default_factory=list)
    zero_row_layers: dict = field(default_factory=dict)   # layer -> (row_len, p_zero)
    config_id: int = 0

    @property
    def num_layers(self) -> int:
        return len(self.layer_sizes)

    @property
    def num_coords(self) -> int:
        return int(sum(self.layer_sizes))


def _log_uniform_scales(n: int, lo_exp: float, hi_exp: float, seed: int) -> List[float]:
    g = torch.Generator(device="cpu").manual_seed(seed)
    e = torch.rand(n, generator=g, dtype=torch.float64) * (hi_exp - lo_exp) + lo_exp
    return [float(10.0 ** x) for x in e.tolist()]


def mlp_workload() -> Workload:
    """Config 1: gradients of a 784-256-10 MLP, K=4, 3-bit uniform levels."""
    return Workload("mlp", [784 * 256, 256, 256 * 10, 10], bits=3, q=2, num_workers=4,
                    dist="normal", scales=[1e-2, 1e-3, 1e-1, 1e-4], config_id=1)


def bilinear_workload() -> Workload:
    """Config 2: the joint 8192-vector of a bilinear game split into 8 layers of 1024."""
    return Workload("bilinear", [1024] * 8, bits=4, q=2, num_workers=8,
                    dist="normal", scales=[1.0] * 8, config_id=2)


def wgan_workload() -> Workload:
    """Config 3: DCGAN-style WGAN generator + discriminator tensors (Section 7.1 shapes)."""
    g = [128 * 8192, 8192, 512 * 256 * 16, 256 * 128 * 16, 128 * 3 * 16]
    d = [3 * 128 * 16, 128 * 256 * 16, 256 * 512 * 16, 8192]
    sizes = g + d
    return Workload("wgan", sizes, bits=3, q=2, num_workers=8, dist="laplace",
                    scales=_log_uniform_scales(len(sizes), -4.0, -1.0, SEED_BASE + 3),
                    config_id=3)


def transformer_xl_workload(num_blocks: int = 16, vocab: int = 267735) -> Workload:
    """Config 4: Transformer-XL-base shaped tensors (Section 7.2 model), embedding first."""
    dm, nh, dh, dff = 410, 10, 41, 2100
    sizes = [vocab * dm]
    for _ in range(num_blocks):
        sizes += [dm * 3 * nh * dh, 3 * nh * dh,      # QKV weight, bias
                  dm * dm, dm,                        # attention output
                  dm * dm, dm,                        # relative-position projection
                  dm * dff, dff,                      # FFN in
                  dff * dm, dm,                       # FFN out
                  dm, dm, dm, dm]                     # two LayerNorms (weight, bias)
    return Workload("transformer_xl", sizes, bits=4, q=2, num_workers=8, dist="student3",
                    scales=_log_uniform_scales(len(sizes), -5.0, -2.0, SEED_BASE + 4),
                    zero_row_layers={0: (dm, 0.9)}, config_id=4)


def powersgd_factor_workload(rank: int = 32, num_blocks: int = 16, vocab: int = 267735) -> Workload:
    """Low-rank factor shapes of the Transformer-XL experiment (Section 7.2): every weight matrix (n x m) of the
    model is replaced by its two rank-`rank` factors (n x rank and m x rank), which is what gets quantized
    there; vectors (biases, LayerNorm) stay as they are.  A factor row is zero where the matrix row is, so
    the embedding's first factor keeps 90 % zero rows, now `rank` values long."""
    dm, nh, dh, dff = 410, 10, 41, 2100
    mats = [(vocab, dm)]
    vecs: List[int] = []
    for _ in range(num_blocks):
        mats += [(dm, 3 * nh * dh), (dm, dm), (dm, dm), (dm, dff), (dff, dm)]
        vecs += [3 * nh * dh, dm, dm, dff, dm, dm, dm, dm, dm]
    sizes: List[int] = []
    for n, m in mats:
        sizes += [n * rank, m * rank]
    sizes += vecs
    return Workload(f"powersgd_rank{rank}", sizes, bits=4, q=2, num_workers=8, dist="normal",
                    scales=_log_uniform_scales(len(sizes), -4.0, -1.0, SEED_BASE + 6),
                    zero_row_layers={0: (rank, 0.9)}, config_id=6)


def flat_workload(log2_n: int, bits: int, num_workers: int, q: int) -> Workload:
    """Config 5a: one flat N(0,1) layer of 2**log2_n coordinates."""
    return Workload(f"flat_2^{log2_n}", [1 << log2_n], bits=bits, q=q,
                    num_workers=num_workers, dist="normal", scales=[1.0], config_id=5)


def ragged_workload(bits: int, num_workers: int, q: int, num_layers: int = 2048,
                    lo: int = 64, hi: int = 4 << 20) -> Workload:
    """Config 5b: `num_layers` layers with sizes log-uniform in [lo, hi]."""
    g = torch.Generator(device="cpu").manual_seed(SEED_BASE + 5)
    e = torch.rand(num_layers, generator=g, dtype=torch.float64)
    sizes = [int(math.floor(math.exp(math.log(lo) + x * (math.log(hi) - math.log(lo)))))
             for x in e.tolist()]
    return Workload(f"ragged_{num_layers}", sizes, bits=bits, q=q, num_workers=num_workers,
                    dist="normal", scales=[1.0] * num_layers, config_id=5)


def _draw(dist: str, n: int, gen: torch.Generator, device) -> torch.Tensor:
    if dist == "normal":
        return torch.randn(n, generator=gen, device=device, dtype=torch.float32)
    if dist == "laplace":
        u = torch.rand(n, generator=gen, device=device, dtype=torch.float32) - 0.5
        return -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.4999999))
    if dist == "student3":
        z = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
        c = torch.zeros(n, device=device, dtype=torch.float32)
        for _ in range(3):
            r = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
            c.addcmul_(r, r)
        return z / torch.sqrt(c / 3.0).clamp_(min=1e-12)
    raise ValueError(dist)


def fill_layer(w: Workload, worker: int, layer: int, out: torch.Tensor,
               gen: torch.Generator) -> None:
    """Write the values of (worker, layer) into `out` (a 1-D fp32 view of the layer)."""
    n = w.layer_sizes[layer]
    chunk = 1 << 26
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        out[s:e] = _draw(w.dist, e - s, gen, out.device) * w.scales[layer]
    if layer in w.zero_row_layers:
        row, p = w.zero_row_layers[layer]
        rows = n // row
        keep = (torch.rand(rows, generator=gen, device=out.device) >= p).to(torch.float32)
        out[: rows * row].view(rows, row).mul_(keep[:, None])


def make_gradients(w: Workload, elem_offsets: List[int], padded_elems: int, device,
                   workers: Optional[int] = None) -> torch.Tensor:
    """Return grads[K][padded_elems] fp32 with layer m of worker k at elem_offsets[m].

    Worker k draws from a generator seeded SEED_BASE + 1000*config + k, layer after
    layer in plan order.  Padding between layers is left at zero.
    """
    K = w.num_workers if workers is None else workers
    grads = torch.zeros((K, padded_elems), dtype=torch.float32, device=device)
    for k in range(K):
        gen = torch.Generator(device=device).manual_seed(SEED_BASE + 1000 * w.config_id + k)
        for m, n in enumerate(w.layer_sizes):
            if n:
                fill_layer(w, k, m, grads[k, elem_offsets[m]: elem_offsets[m] + n], gen)
    return grads


def bilinear_game(n: int = 4096, seed: int = SEED_BASE + 2000):
    """A (n x n, fp32, entries N(0,1/n)) and the start point z1 of the game min_x max_y x'Ay."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    A = torch.randn((n, n), generator=g, dtype=torch.float32) / math.sqrt(n)
    z1 = torch.randn(2 * n, generator=g, dtype=torch.float32) / math.sqrt(2 * n)
    return A, z1


def bilinear_noise(step: int, num_workers: int, dim: int, sigma: float = 0.1,
                   seed: int = SEED_BASE + 2001) -> torch.Tensor:
    """Per-worker absolute noise N(0, sigma^2) for one iteration, drawn on the host."""
    g = torch.Generator(device="cpu").manual_seed(seed + 7919 * step)
    return torch.randn((num_workers, dim), generator=g, dtype=torch.float32) * sigma
