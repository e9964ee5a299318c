"""Seeded synthetic gradients shaped like the paper's workloads.

This module only *makes inputs*: it contains none of the codec's arithmetic and
imports neither the CUDA binding nor the CPU oracle, so both can be fed from it.
The paper's own datasets (Syn-*, YearPredictionMSD, gisette, CIFAR-10,
ILSVRC-12) and trained models are not reproduced; the generators below take
only their shapes, sizes and value distributions (Section 6 of the paper names
linear models, ResNet-style CNNs and a 512-GPU ResNet-50 projection).

Every tensor is a deterministic function of (workload, worker, step, device
type).  A tensor made on the GPU is copied to the host bit for bit when a CPU
check needs the same values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Tuple

import torch

CODEC_SEED = 1234  # Philox seed of the codec itself, separate from the input seeds


@dataclass(frozen=True)
class Workload:
    """One benchmark/parity configuration of the codec."""
    name: str
    index: int            # 1-based, used in the input seeds
    W: int                # simulated workers (the paper's P)
    d: int                # flat gradient length
    bucket: int
    s: int                # non-zero quantisation levels
    alpha: float
    beta: float
    steps: int            # iterations the parity run follows
    kind: str             # value recipe, see gradient()
    layers: Tuple[int, ...] = field(default=(), repr=False)

    def input_seed(self, worker: int, step: int) -> int:
        return 10_000 * self.index + 100 * step + worker


def _resnet50_layers() -> List[int]:
    """Parameter tensors of the standard ResNet-50 in definition order (161)."""
    sizes: List[int] = [64 * 3 * 7 * 7, 64, 64]
    inplanes = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for blk in range(blocks):
            sizes += [planes * inplanes, planes, planes]           # 1x1 + BN
            sizes += [planes * planes * 9, planes, planes]         # 3x3 + BN
            sizes += [planes * 4 * planes, planes * 4, planes * 4]  # 1x1 + BN
            if blk == 0:                                           # projection + BN
                sizes += [planes * 4 * inplanes, planes * 4, planes * 4]
            inplanes = planes * 4
    sizes += [1000 * 2048, 1000]
    return sizes


def _alexnet_layers() -> List[int]:
    """Parameter tensors of single-tower AlexNet (8 weights + 8 biases)."""
    return [64 * 3 * 11 * 11, 64, 192 * 64 * 5 * 5, 192, 384 * 192 * 3 * 3, 384,
            256 * 384 * 3 * 3, 256, 256 * 256 * 3 * 3, 256,
            4096 * 9216, 4096, 4096 * 4096, 4096, 1000 * 4096, 1000]


def _lm_layers() -> List[int]:
    """24 transformer blocks of four matrices each plus a token embedding."""
    per = [1024 * 4096, 4096 * 1024, 1024 * 3072, 1024 * 1024]
    return per * 24 + [50257 * 1024]


_R50 = tuple(_resnet50_layers())
_ALEX = tuple(_alexnet_layers())
_LM = tuple(_lm_layers())
assert len(_R50) == 161 and sum(_R50) == 25_557_032
assert len(_ALEX) == 16 and sum(_ALEX) == 61_100_840
assert sum(_LM) == 353_453_056

WORKLOADS = {
    "gauss_1m": Workload("gauss_1m", 1, 4, 1 << 20, 512, 4, 1.0, 0.9, 10, "gauss"),
    "lsq_4m": Workload("lsq_4m", 2, 8, 4_194_304, 1024, 2, 1.0, 0.95, 20, "lsq"),
    "resnet50": Workload("resnet50", 3, 8, sum(_R50), 512, 8, 1.0, 0.9, 5, "layers", _R50),
    "alexnet": Workload("alexnet", 4, 16, sum(_ALEX), 2048, 1, 1.0, 0.99, 5, "student", _ALEX),
    "lm_350m": Workload("lm_350m", 5, 32, sum(_LM), 512, 4, 1.0, 0.9, 2, "outliers", _LM),
}
LM_SWEEP_BUCKETS = (128, 512, 4096)
LM_SWEEP_LEVELS = (1, 4, 8, 128)


def with_codec(w: Workload, bucket: int, s: int) -> Workload:
    """Same inputs, different bucket size / level count (the lm_350m sweep)."""
    return Workload(w.name, w.index, w.W, w.d, bucket, s, w.alpha, w.beta, w.steps,
                    w.kind, w.layers)


def scaled(w: Workload, d: int, W: int | None = None) -> Workload:
    """A shorter vector with the same value recipe (small parity cases)."""
    return Workload(w.name, w.index, W or w.W, d, w.bucket, w.s, w.alpha, w.beta,
                    w.steps, w.kind, ())


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _layer_sigmas(w: Workload, device) -> torch.Tensor:
    """Per-element standard deviation: one log-uniform sigma per layer."""
    gen = _gen(10_000 * w.index + 9_999, "cpu")
    if w.layers:
        n_layers, sizes = len(w.layers), torch.tensor(w.layers, dtype=torch.int64)
    else:  # shortened vector: layers of 4096 entries
        n_layers = (w.d + 4095) // 4096
        sizes = torch.full((n_layers,), 4096, dtype=torch.int64)
        sizes[-1] = w.d - 4096 * (n_layers - 1)
    u = torch.rand(n_layers, generator=gen, dtype=torch.float64)
    sig = torch.exp(math.log(1e-5) + u * (math.log(1e-2) - math.log(1e-5))).float()
    return torch.repeat_interleave(sig.to(device), sizes.to(device))


class _LeastSquares:
    """Sparse least-squares problem of the lsq_4m workload (one per worker)."""
    rows = 256
    density = 1e-3

    def __init__(self, w: Workload, worker: int, device):
        d = w.d
        base = 10_000 * w.index
        gs = _gen(base + 9_000, device)
        self.w_star = torch.randn(d, generator=gs, device=device)
        self.w0 = 0.1 * torch.randn(d, generator=gs, device=device)
        gp = _gen(base + 9_100 + worker, device)
        nnz = int(round(self.rows * d * self.density))
        self.r = torch.randint(0, self.rows, (nnz,), generator=gp, device=device)
        self.c = torch.randint(0, d, (nnz,), generator=gp, device=device)
        self.x = torch.randn(nnz, generator=gp, device=device)
        self.y = self.matvec(self.w_star) + 0.01 * torch.randn(self.rows, generator=gp, device=device)
        self.d = d

    def matvec(self, v: torch.Tensor) -> torch.Tensor:
        out = torch.zeros(self.rows, device=v.device, dtype=torch.float32)
        return out.index_add_(0, self.r, self.x * v[self.c])

    def grad(self, step: int) -> torch.Tensor:
        # The iterate follows a fixed geometric path towards the optimum, so the
        # inputs do not depend on any codec's output.
        wt = self.w_star + (0.98 ** step) * (self.w0 - self.w_star)
        res = self.matvec(wt) - self.y
        g = torch.zeros(self.d, device=wt.device, dtype=torch.float32)
        g.index_add_(0, self.c, self.x * res[self.r])
        return g / self.rows


_lsq_cache: dict = {}


def gradient(w: Workload, worker: int, step: int, device="cpu") -> torch.Tensor:
    """Local gradient g_p^(t) of ``worker`` at iteration ``step`` (fp32, [d])."""
    device = torch.device(device)
    gen = _gen(w.input_seed(worker, step), device)
    d = w.d
    if w.kind == "gauss":
        return 0.01 * torch.randn(d, generator=gen, device=device)
    if w.kind == "lsq":
        key = (w.index, w.d, worker, str(device))
        if key not in _lsq_cache:
            _lsq_cache[key] = _LeastSquares(w, worker, device)
        return _lsq_cache[key].grad(step)
    if w.kind == "layers":
        g = torch.randn(d, generator=gen, device=device)
        return g.mul_(_layer_sigmas(w, device))
    if w.kind == "student":
        z = torch.randn(d, generator=gen, device=device)
        chi = torch.zeros(d, device=device)
        for _ in range(3):
            chi.add_(torch.randn(d, generator=gen, device=device).square_())
        g = z.div_(chi.div_(3.0).sqrt_()).mul_(1e-3)
        mask = torch.rand(d, generator=gen, device=device) < 0.01
        g[mask] = 0.0
        return g
    if w.kind == "outliers":
        g = torch.randn(d, generator=gen, device=device).mul_(1e-3)
        u = torch.rand(d, generator=gen, device=device)
        g = torch.where(u < 5e-4, torch.full_like(g, 0.1), g)
        g = torch.where(u > 1.0 - 5e-4, torch.full_like(g, -0.1), g)
        return g
    raise ValueError("unknown workload kind %r" % w.kind)


def clear_cache() -> None:
    _lsq_cache.clear()


class SynLinReg:
    """Synthetic linear regression in the style of the paper's Syn-256/512/1024 runs
    (Section 6.1): N samples x ~ N(0, I_d), y = <w*, x> + noise, split evenly over W workers.
    The paper does not state the noise level; 0.1 is used here.  Only data and mini-batch
    sampling live here; the optimiser loop belongs to whoever uses it."""

    def __init__(self, d: int, W: int, seed: int, n_samples: int = 10_000, noise: float = 0.1,
                 device="cuda"):
        self.d, self.W = d, W
        self.gen = _gen(770_000 + seed, torch.device(device))
        self.X = torch.randn(n_samples, d, generator=self.gen, device=device)
        self.w_star = torch.randn(d, generator=self.gen, device=device)
        self.y = self.X @ self.w_star + noise * torch.randn(n_samples, generator=self.gen, device=device)
        self.shards = torch.chunk(torch.arange(n_samples, device=device), W)

    def minibatch_gradient(self, worker: int, w: torch.Tensor, batch: int = 64) -> torch.Tensor:
        """Gradient of the mean squared error over a random mini-batch of the worker's shard."""
        shard = self.shards[worker]
        idx = shard[torch.randint(0, len(shard), (batch,), generator=self.gen, device=w.device)]
        xb = self.X[idx]
        return (xb.T @ (xb @ w - self.y[idx]) / batch).contiguous()
