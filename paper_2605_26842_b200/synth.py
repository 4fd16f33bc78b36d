"""Seeded synthetic inputs: parameter-set shapes, initial weights and the gradient process.

This module only draws random numbers and lists shapes.  It holds none of the optimizer's
arithmetic, so both the CUDA path and the CPU oracle may be fed from it.

Parameter sets (the five benchmark configurations):
  0  one 256x512 weight
  1  dense transformer blocks: 12 layers x {Wq,Wk,Wv,Wo 1024x1024; W1,W3 2816x1024; W2 1024x2816}
  2  ~1B MoE: 16 layers, hidden 1024, 32 experts {W1,W3 512x1024; W2 1024x512}, 4 attention
     1024x1024, router 32x1024
  3  ~7B MoE: 24 layers, hidden 2048, 64 experts {W1,W3 768x2048; W2 2048x768}, 4 attention
     2048x2048, one shared expert 1536x2048; Student-t(4) gradients
  4  large-MoE shard: hidden 4096, 128 experts {W1,W3 1024x4096; W2 4096x1024}, 4 attention
     4096x4096, bf16 gradients; the layer count is a parameter because the nominal 8 layers
     need more memory than one GPU has.

  5-7  expert matrices of the paper's own models (section "Pretraining"; only the expert shapes are stated,
     so attention and router weights are left out): 5 = MOE-1B-A0d2B (10 layers, hidden 768, 128 experts of
     FFN width 256), 6 = MOE-6B-A0d5B (10 layers, hidden 1536, 128 experts of width 1024), 7 = MOE-68B-A3B
     (14 layers, hidden 3072, 256 experts of width 1024; layer count is a parameter, the full set exceeds
     one GPU).  Each expert has W1, W3 (width x hidden) and W2 (hidden x width), as in configurations 2-4.

Gradient process per element (stationary AR(1), variance sigma^2, lag-1 correlation rho):
  g_1 = sigma xi_1,   g_k = rho g_{k-1} + sqrt(1 - rho^2) sigma xi_k,
with xi standard normal, or Student-t with 4 degrees of freedom divided by sqrt(2) (unit variance).
Initial weights are N(0, 0.02^2).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List

import torch


@dataclass
class MatrixSpec:
    """`batch` same-shape row-major matrices stacked contiguously (experts of one layer)."""
    name: str
    rows: int
    cols: int
    batch: int = 1

    @property
    def numel(self) -> int:
        return self.rows * self.cols * self.batch


@dataclass
class Workload:
    name: str
    specs: List[MatrixSpec]
    steps: int
    rho: float = 0.9
    sigma: float = 1e-3
    dist: str = "normal"            # "normal" | "student_t4"
    grad_dtype: torch.dtype = torch.float32
    accel_beta: float = 0.99        # beta_a; alpha follows alpha = -1 / (2 (1 - beta_a))
    seed: int = 1234
    notes: str = ""

    @property
    def accel_alpha(self) -> float:
        return -1.0 / (2.0 * (1.0 - self.accel_beta))

    @property
    def n_params(self) -> int:
        return sum(s.numel for s in self.specs)

    @property
    def n_matrices(self) -> int:
        return sum(s.batch for s in self.specs)


def workload(index: int, layers: int | None = None) -> Workload:
    """The benchmark configuration `index` (0..7).  `layers` overrides the layer count."""
    if index == 0:
        return Workload("single_256x512", [MatrixSpec("W", 256, 512)], steps=5, seed=1234)
    if index == 1:
        L = layers or 12
        specs = []
        for l in range(L):
            specs += [MatrixSpec(f"l{l}.w{q}", 1024, 1024) for q in "qkvo"]
            specs += [MatrixSpec(f"l{l}.w1", 2816, 1024), MatrixSpec(f"l{l}.w3", 2816, 1024),
                      MatrixSpec(f"l{l}.w2", 1024, 2816)]
        return Workload(f"dense_blocks_{L}L", specs, steps=20, seed=1235)
    if index == 2:
        L = layers or 16
        specs = []
        for l in range(L):
            specs += [MatrixSpec(f"l{l}.experts.w1", 512, 1024, 32), MatrixSpec(f"l{l}.experts.w3", 512, 1024, 32),
                      MatrixSpec(f"l{l}.experts.w2", 1024, 512, 32)]
            specs += [MatrixSpec(f"l{l}.w{q}", 1024, 1024) for q in "qkvo"]
            specs += [MatrixSpec(f"l{l}.router", 32, 1024)]
        return Workload(f"moe_1b_{L}L", specs, steps=20, seed=1236)
    if index == 3:
        L = layers or 24
        specs = []
        for l in range(L):
            specs += [MatrixSpec(f"l{l}.experts.w1", 768, 2048, 64), MatrixSpec(f"l{l}.experts.w3", 768, 2048, 64),
                      MatrixSpec(f"l{l}.experts.w2", 2048, 768, 64)]
            specs += [MatrixSpec(f"l{l}.w{q}", 2048, 2048) for q in "qkvo"]
            specs += [MatrixSpec(f"l{l}.shared", 1536, 2048)]
        return Workload(f"moe_7b_{L}L", specs, steps=10, rho=0.8, dist="student_t4", accel_beta=0.98, seed=1237)
    if index == 4:
        L = layers or 8
        specs = []
        for l in range(L):
            specs += [MatrixSpec(f"l{l}.experts.w1", 1024, 4096, 128), MatrixSpec(f"l{l}.experts.w3", 1024, 4096, 128),
                      MatrixSpec(f"l{l}.experts.w2", 4096, 1024, 128)]
            specs += [MatrixSpec(f"l{l}.w{q}", 4096, 4096) for q in "qkvo"]
        return Workload(f"moe_shard_{L}L", specs, steps=5, grad_dtype=torch.bfloat16, accel_beta=0.975, seed=1238)
    if index in (5, 6, 7):
        nominal, hidden, width, experts, beta = {5: (10, 768, 256, 128, 0.99), 6: (10, 1536, 1024, 128, 0.98),
                                                  7: (14, 3072, 1024, 256, 0.975)}[index]
        L = layers or nominal
        specs = []
        for l in range(L):
            specs += [MatrixSpec(f"l{l}.experts.w1", width, hidden, experts), MatrixSpec(f"l{l}.experts.w3", width, hidden, experts),
                      MatrixSpec(f"l{l}.experts.w2", hidden, width, experts)]
        name = {5: "paper_moe_1b_experts", 6: "paper_moe_6b_experts", 7: "paper_moe_68b_experts"}[index]
        return Workload(f"{name}_{L}L", specs, steps=10, accel_beta=beta, seed=1234 + index)
    raise ValueError(f"no such configuration: {index}")


def resident_bytes(wl: Workload) -> int:
    """Bytes held on the device for W, M, A, G_prev (fp32) and G."""
    g = 2 if wl.grad_dtype == torch.bfloat16 else 4
    return wl.n_params * (16 + g)


def init_params(wl: Workload, device, seed_offset: int = 0) -> List[torch.Tensor]:
    """One fp32 tensor of shape (batch, rows, cols) per spec, N(0, 0.02^2)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(wl.seed * 1000 + 17 + seed_offset)
    out = []
    for s in wl.specs:
        w = torch.empty((s.batch, s.rows, s.cols), dtype=torch.float32, device=device)
        w.normal_(0.0, 0.02, generator=gen)
        out.append(w)
    return out


class GradientProcess:
    """Holds one gradient tensor per spec and advances all of them by one step of the AR(1)
    process in place.  The recursion itself is carried in fp32 (`_g32`) only when the visible
    gradient dtype is narrower; otherwise the visible tensor is the state."""

    SLICE = 1 << 26

    def __init__(self, wl: Workload, device, keep_fp32_shadow: bool | None = None):
        self.wl = wl
        self.device = torch.device(device)
        self.gen = torch.Generator(device=device)
        self.gen.manual_seed(wl.seed * 1000 + 91)
        self.k = 0
        self.grads = [torch.zeros((s.batch, s.rows, s.cols), dtype=wl.grad_dtype, device=device) for s in wl.specs]
        narrow = wl.grad_dtype != torch.float32
        self.shadow = narrow if keep_fp32_shadow is None else (keep_fp32_shadow and narrow)
        self._g32 = [torch.zeros_like(g, dtype=torch.float32) for g in self.grads] if self.shadow else None

    def _noise(self, shape) -> torch.Tensor:
        z = torch.empty(shape, dtype=torch.float32, device=self.device)
        z.normal_(0.0, 1.0, generator=self.gen)
        if self.wl.dist == "student_t4":
            chi = torch.zeros(shape, dtype=torch.float32, device=self.device)
            t = torch.empty(shape, dtype=torch.float32, device=self.device)
            for _ in range(4):
                t.normal_(0.0, 1.0, generator=self.gen)
                chi.addcmul_(t, t)
            z.div_(chi.mul_(0.25).sqrt_()).mul_(1.0 / math.sqrt(2.0))
        return z

    def next(self) -> List[torch.Tensor]:
        """Advance to g_{k+1}; returns the (in-place updated) gradient tensors."""
        wl = self.wl
        first = self.k == 0
        c_old = 0.0 if first else wl.rho
        c_new = wl.sigma if first else math.sqrt(1.0 - wl.rho * wl.rho) * wl.sigma
        for i, g in enumerate(self.grads):
            flat = g.view(-1)
            flat32 = self._g32[i].view(-1) if self.shadow else None
            # bounded slices keep the temporaries small next to a nearly full device
            for lo in range(0, flat.numel(), self.SLICE):
                hi = min(lo + self.SLICE, flat.numel())
                z = self._noise((hi - lo,))
                if flat.dtype == torch.float32:
                    flat[lo:hi].mul_(c_old).add_(z, alpha=c_new)
                elif self.shadow:
                    flat32[lo:hi].mul_(c_old).add_(z, alpha=c_new)
                    flat[lo:hi].copy_(flat32[lo:hi])
                else:
                    flat[lo:hi].copy_(flat[lo:hi].float().mul_(c_old).add_(z, alpha=c_new))
        self.k += 1
        return self.grads
