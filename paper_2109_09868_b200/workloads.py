"""Seeded synthetic inputs for the five ApproxIFER workloads.

This module only draws inputs: queries, availability masks, stand-in hosted
models, adversary sets and their noise.  It contains none of the method's
arithmetic (no nodes, no interpolation weights, no locator), so both the CUDA
library's tests and the CPU checker can consume exactly the same tensors.

The paper evaluates on MNIST / Fashion-MNIST (1x28x28) and CIFAR-10 (3x32x32,
10 classes) with pretrained networks (Section 4.1).  Those are replaced here by
uniform[0,1) tensors of the same shapes, seeded linear (+softmax) stand-ins for
the hosted model f, Gaussian logits, and Gaussian Byzantine noise as in
Section 4.2 ("Byzantine-Robustness").

Payloads come from a ``torch.Generator`` on the requested device (a CUDA
generator and a CPU generator give different streams; a test always hands the
same tensor to both sides).  Masks and adversary sets come from
``numpy.random.Generator(PCG64(seed))`` on the host.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, Optional

import numpy as np
import torch

SEED_BASE = 210909868


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape of one workload.  W is the number of workers (the paper's N+1)."""

    cfg: int
    K: int
    W: int
    S: int  # stragglers tolerated / drawn at most
    E: int  # Byzantine workers
    G: int  # groups
    D: int  # payload elements per query
    C: int  # payload elements per prediction
    note: str

    @property
    def seed(self) -> int:
        return SEED_BASE + self.cfg

    def with_groups(self, G: int) -> "Workload":
        return dataclasses.replace(self, G=int(G))


WORKLOADS = {
    1: Workload(1, 4, 5, 1, 0, 256, 784, 10, "1x28x28 queries, linear 784->10 + softmax, one straggler"),
    2: Workload(2, 8, 12, 4, 0, 65536, 3072, 10, "3x32x32 queries, N(0,1) logits, 0-4 stragglers"),
    3: Workload(3, 12, 20, 8, 0, 4096, 150528, 1000, "3x224x224 queries, N(0,2) logits, Bernoulli(0.3) stragglers <= 8"),
    4: Workload(4, 16, 24, 8, 0, 262144, 32, 1000, "decode-heavy: 1000-class predictions, 16-24 workers present"),
    5: Workload(5, 8, 24, 2, 2, 65536, 64, 10, "Byzantine: 2 stragglers, 2 adversaries with N(0,10^2) noise"),
}


def workload(cfg: int, G: Optional[int] = None) -> Workload:
    wl = WORKLOADS[int(cfg)]
    return wl if G is None else wl.with_groups(G)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def queries(wl: Workload, device="cpu", seed_offset: int = 0) -> torch.Tensor:
    """float32 [G][K][D], uniform on [0,1)."""
    g = _gen(device, wl.seed * 16 + 1 + seed_offset)
    return torch.rand((wl.G, wl.K, wl.D), generator=g, device=device, dtype=torch.float32)


def gaussian_predictions(wl: Workload, device="cpu", std: Optional[float] = None) -> torch.Tensor:
    """float32 [G][W][C] iid Gaussian coded predictions (workloads 2 and 3).
    "N(0,2)" is read as variance 2, i.e. std sqrt(2)."""
    if std is None:
        std = math.sqrt(2.0) if wl.cfg == 3 else 1.0
    g = _gen(device, wl.seed * 16 + 2)
    out = torch.randn((wl.G, wl.W, wl.C), generator=g, device=device, dtype=torch.float32)
    return out.mul_(std)


def model_matrix(wl: Workload, device="cpu") -> torch.Tensor:
    """Weights [D][C] of the seeded linear stand-in for the hosted model f."""
    g = _gen("cpu", wl.seed * 16 + 3)
    if wl.cfg == 4:
        var = 12.0 / wl.D  # unit-variance logits for centred uniform inputs
    else:
        var = 1.0 / wl.D
    m = torch.randn((wl.D, wl.C), generator=g, dtype=torch.float32) * math.sqrt(var)
    return m.to(device)


def apply_model(wl: Workload, Xt: torch.Tensor, softmax: Optional[bool] = None) -> torch.Tensor:
    """Stand-in hosted model on coded queries: float32 [G][W][D] -> [G][W][C].

    workload 1: linear + softmax; 4: linear on centred inputs; others: linear.
    """
    M = model_matrix(wl, Xt.device)
    if softmax is None:
        softmax = wl.cfg == 1
    x = Xt - 0.5 if wl.cfg == 4 else Xt
    y = torch.matmul(x.to(torch.float32), M)
    if softmax:
        y = torch.softmax(y, dim=-1)
    return y.contiguous()


def _bits(sel: np.ndarray) -> np.ndarray:
    """bool [G][W] -> uint32 [G], bit i = column i."""
    W = sel.shape[1]
    weights = (np.uint64(1) << np.arange(W, dtype=np.uint64))
    return (sel.astype(np.uint64) * weights).sum(axis=1).astype(np.uint32)


def masks(wl: Workload, seed_offset: int = 0) -> np.ndarray:
    """uint32 [G] availability masks, bit i set = worker i answered."""
    rng = np.random.Generator(np.random.PCG64(wl.seed * 16 + 4 + seed_offset))
    G, W = wl.G, wl.W
    order = rng.random((G, W)).argsort(axis=1)  # a uniform random order of the workers
    rank = np.empty_like(order)
    np.put_along_axis(rank, order, np.broadcast_to(np.arange(W), (G, W)), axis=1)
    if wl.cfg == 1:
        n_s = np.ones(G, dtype=np.int64)
    elif wl.cfg == 2:
        n_s = rng.integers(0, wl.S + 1, size=G)
    elif wl.cfg == 3:
        slow = rng.random((G, W)) < 0.3
        # keep at most S stragglers: the first S of them in the random order
        pos = np.where(slow, rank, W + 1)
        kth = np.sort(pos, axis=1)[:, wl.S - 1 : wl.S]  # S-th smallest position among stragglers
        slow &= pos <= kth
        return _bits(~slow)
    elif wl.cfg == 4:
        n_s = W - rng.integers(wl.K, W + 1, size=G)
    else:
        n_s = np.full(G, wl.S, dtype=np.int64)
    absent = rank < n_s[:, None]
    return _bits(~absent)


def adversaries(wl: Workload, mask: np.ndarray, seed_offset: int = 0) -> np.ndarray:
    """int32 [G][E]: E distinct workers drawn uniformly among those present, ascending."""
    rng = np.random.Generator(np.random.PCG64(wl.seed * 16 + 5 + seed_offset))
    G, W, E = len(mask), wl.W, wl.E
    present = ((mask[:, None] >> np.arange(W, dtype=np.uint32)) & 1).astype(bool)
    key = rng.random((G, W))
    key[~present] = 2.0
    adv = np.sort(np.argsort(key, axis=1)[:, :E], axis=1)
    return adv.astype(np.int32)


def corrupt(wl: Workload, Yt: torch.Tensor, adv: np.ndarray, sigma: float = 10.0) -> torch.Tensor:
    """Add N(0, sigma^2) noise to every class of the adversaries' predictions (in place)."""
    G, E = adv.shape
    g = _gen(Yt.device, wl.seed * 16 + 6)
    noise = torch.randn((G, E, Yt.shape[2]), generator=g, device=Yt.device, dtype=torch.float32) * sigma
    idx = torch.as_tensor(adv.astype(np.int64), device=Yt.device)
    rows = torch.arange(G, device=Yt.device)[:, None].expand(G, E)
    Yt[rows, idx] += noise
    return Yt


def coded_predictions(wl: Workload, encode_fn: Callable[[torch.Tensor], torch.Tensor], device="cpu",
                      softmax: Optional[bool] = None) -> torch.Tensor:
    """Workloads 1, 4, 5: hidden queries -> coded queries (by the caller's
    ``encode_fn``: float32 [G][K][D] -> float32 [G][W][D]) -> stand-in model."""
    X = queries(wl, device)
    Xt = encode_fn(X)
    return apply_model(wl, Xt, softmax)
