"""Seeded synthetic micro-gradient workloads.

This module only draws inputs; it contains none of the method's arithmetic (no
dot product, norm, distance or filtering).  The same tensors are handed to the
CUDA library and, as numpy views of the same bits, to the CPU oracle used by the
tests.

Model for every workload: one shared direction ``s`` and one private direction
``n_i`` per micro-gradient, all iid N(0, sigma_d^2) per element, mixed as

    g_i = sign(rho_i) * sqrt(|rho_i|) * s + sqrt(1 - |rho_i|) * n_i

so that the expected cosine between g_i and g_j is sign * sqrt(|rho_i rho_j|).
A negative rho flips the sign of the shared part.  This stands in for the
ResNet18 / ViT micro-gradients of the paper's experiments (Section 4), whose
datasets and weights are not available: late in training their pairwise cosine
distances sit near 1 and reach 1.1-1.6 (Figure 1), which the rho ranges below
reproduce.

The five named configurations:

  1  K=4  D=1,000,000     fp32  rho=(0.9, 0.5, 0.0, -0.3)  tau=0.97   seed 0
  2  K=4  D=11,227,812    fp32  ResNet18 (100 classes) tensor layout, per-tensor
                                sigma ~ lognormal(log 1e-3, 1), rho ~ U(-0.2, 0.6),
                                tau in {0.95, 0.97, 1.0}
  3  K=32 D=11,227,812    bf16  pairwise matrix, rho ~ U(-0.5, 0.9)
  4  K=8  D=124,439,808   fp32  rho ~ N(0.02, 0.05^2), tau=0.97
  5  K=8  D=1,000,000,000 bf16  rho ~ 50% U(0.3, 0.8) / 50% U(-0.3, 0.1), tau=0.97

Configuration n uses seed n-1.  rho values are drawn first, from a CPU generator,
so they do not depend on the device; the vectors are drawn on the requested
device (CPU and GPU streams differ, which is fine: both consumers see the same
bits of one draw).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

RESNET18_100_NUMEL = 11_227_812
GPT2_SMALL_NUMEL = 124_439_808


def resnet18_tensor_sizes(num_classes: int = 100) -> List[int]:
    """Element counts of ResNet18's parameter tensors in network order.

    Convolutions carry no bias; every batch-norm contributes a weight and a
    bias vector; the 128/256/512-channel stages open with a block that has a
    1x1 shortcut convolution plus batch-norm.
    """
    sizes: List[int] = [64 * 3 * 7 * 7, 64, 64]
    in_ch = 64
    for out_ch in (64, 128, 256, 512):
        for block in range(2):
            cin = in_ch if block == 0 else out_ch
            sizes += [out_ch * cin * 9, out_ch, out_ch]
            sizes += [out_ch * out_ch * 9, out_ch, out_ch]
            if block == 0 and cin != out_ch:
                sizes += [out_ch * cin, out_ch, out_ch]
        in_ch = out_ch
    sizes += [num_classes * 512, num_classes]
    return sizes


@dataclass
class Workload:
    name: str
    K: int
    D: int
    dtype: str                    # "f32" or "bf16"
    taus: List[float]
    rho: List[float]
    seed: int
    grads: List[torch.Tensor] = field(default_factory=list)
    order: Optional[List[int]] = None

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


def as_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """Host numpy view of a gradient: float32 as is, bfloat16 as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def _draw(K: int, D: int, dtype: str, rho: Sequence[float], seed: int,
          device: str, sigma, chunk: int = 1 << 24, stacked: bool = False) -> List[torch.Tensor]:
    """Draw K micro-gradients of D elements.  ``sigma`` is a float or a
    per-element float32 tensor on ``device``.  ``stacked``: the gradients are the
    rows of one matrix whose row stride is D rounded up to 128 elements (what an
    all-gather of padded flat gradients leaves); the values are the same either way."""
    tdtype = torch.float32 if dtype == "f32" else torch.bfloat16
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    if stacked:
        matrix = torch.zeros(K, (D + 127) // 128 * 128, dtype=tdtype, device=device)
        grads = [matrix[i, :D] for i in range(K)]
    else:
        grads = [torch.empty(D, dtype=tdtype, device=device) for _ in range(K)]
    alpha = [math.copysign(math.sqrt(abs(r)), r) for r in rho]
    beta = [math.sqrt(1.0 - abs(r)) for r in rho]
    for lo in range(0, D, chunk):
        hi = min(D, lo + chunk)
        sig = sigma[lo:hi] if torch.is_tensor(sigma) else float(sigma)
        s = torch.randn(hi - lo, generator=gen, device=device, dtype=torch.float32) * sig
        for i in range(K):
            n = torch.randn(hi - lo, generator=gen, device=device, dtype=torch.float32) * sig
            grads[i][lo:hi] = (alpha[i] * s + beta[i] * n).to(tdtype)
    return grads


def _clip_rho(r: Sequence[float]) -> List[float]:
    return [float(min(0.999, max(-0.999, x))) for x in r]


def mixture(K: int, D: int, dtype: str, rho: Sequence[float], seed: int,
            device: str = "cpu", sigma=1e-3, taus: Sequence[float] = (0.97,),
            name: str = "custom", stacked: bool = False) -> Workload:
    """A workload with explicit rho values (used by the tests for small and
    ragged shapes)."""
    rho = _clip_rho(rho)
    assert len(rho) == K
    w = Workload(name, K, D, dtype, [float(t) for t in taus], rho, seed)
    w.grads = _draw(K, D, dtype, rho, seed, device, sigma, stacked=stacked)
    return w


def config(n: int, device: str = "cpu", D: Optional[int] = None,
           K: Optional[int] = None, seed: Optional[int] = None, stacked: bool = False) -> Workload:
    """Named configuration ``n`` (1..5).  ``D``/``K`` override the size for
    scaled-down copies of the same recipe (the tensor layout of configuration 2
    is kept only at its native D); ``seed`` draws another instance of it."""
    seed = n - 1 if seed is None else seed
    rgen = np.random.RandomState(seed)
    if n == 1:
        K_, D_, dtype, taus = 4, 1_000_000, "f32", [0.97]
        rho = [0.9, 0.5, 0.0, -0.3]
        if K is not None and K != K_:
            rho = (rho * ((K + 3) // 4))[:K]
    elif n == 2:
        K_, D_, dtype, taus = 4, RESNET18_100_NUMEL, "f32", [0.95, 0.97, 1.0]
        rho = rgen.uniform(-0.2, 0.6, size=K or K_).tolist()
    elif n == 3:
        K_, D_, dtype, taus = 32, RESNET18_100_NUMEL, "bf16", []
        rho = rgen.uniform(-0.5, 0.9, size=K or K_).tolist()
    elif n == 4:
        K_, D_, dtype, taus = 8, GPT2_SMALL_NUMEL, "f32", [0.97]
        rho = rgen.normal(0.02, 0.05, size=K or K_).tolist()
    elif n == 5:
        K_, D_, dtype, taus = 8, 1_000_000_000, "bf16", [0.97]
        kk = K or K_
        pick = rgen.uniform(size=kk) < 0.5
        hi = rgen.uniform(0.3, 0.8, size=kk)
        lo = rgen.uniform(-0.3, 0.1, size=kk)
        rho = np.where(pick, hi, lo).tolist()
    else:
        raise ValueError("configurations are numbered 1..5")
    K_ = K or K_
    native = D is None or D == D_
    D_ = D or D_
    rho = _clip_rho(rho)

    sigma = 1e-3
    if n == 2 and native:
        sizes = resnet18_tensor_sizes(100)
        assert sum(sizes) == RESNET18_100_NUMEL
        per_tensor = np.exp(rgen.normal(math.log(1e-3), 1.0, size=len(sizes))).astype(np.float32)
        sigma = torch.repeat_interleave(torch.from_numpy(per_tensor),
                                        torch.tensor(sizes)).to(device)
    w = Workload(f"config{n}", K_, D_, dtype, taus, rho, seed)
    w.grads = _draw(K_, D_, dtype, rho, seed, device, sigma, stacked=stacked)
    return w
