"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the sparsifier: it only produces gradients (and, for the
least-squares problem, the loss whose gradients they are).  Both the CUDA library and the CPU oracle
consume the bytes produced here; a batch is generated once and copied, never generated twice.

Recipe shared by the model-shaped workloads (stand-ins for the paper's ResNet-18/CIFAR-10 and
fine-tuning experiments, whose data and weights are not available): every parameter tensor l gets a
scale sigma_l drawn log-uniformly from a range; a component shared by all workers follows an AR(1)
process over rounds, c^0 = sigma z^0, c^t = rho c^{t-1} + sqrt(1 - rho^2) sigma z^t; worker n's
gradient is g_n^t = c^t + 0.5 sigma z_n^t, with z i.i.d. from the workload's base distribution.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch


# ---- parameter-tensor tables -----------------------------------------------------------------------
def resnet18_cifar_shapes() -> List[int]:
    """CIFAR-style ResNet-18: 62 tensors, 11,173,962 parameters."""
    s = [64 * 3 * 3 * 3, 64, 64]
    inp = 64
    for width, first_stride in ((64, 1), (128, 2), (256, 2), (512, 2)):
        for b in range(2):
            cin = inp if b == 0 else width
            s += [width * cin * 9, width, width, width * width * 9, width, width]
            if b == 0 and (first_stride != 1 or cin != width):
                s += [width * cin, width, width]
        inp = width
    s += [512 * 10, 10]
    return s


def resnet50_shapes() -> List[int]:
    """ImageNet ResNet-50: 161 tensors, 25,557,032 parameters."""
    s = [64 * 3 * 7 * 7, 64, 64]
    inp = 64
    for width, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        out = width * 4
        for b in range(blocks):
            cin = inp if b == 0 else out
            s += [width * cin, width, width, width * width * 9, width, width, out * width, out, out]
            if b == 0:
                s += [out * cin, out, out]
        inp = out
    s += [2048 * 1000, 1000]
    return s


def gpt2_small_shapes() -> List[int]:
    """GPT-2 small: 148 tensors, 124,439,808 parameters; tensor 0 is the 50257 x 768 token embedding."""
    s = [50257 * 768, 1024 * 768]
    for _ in range(12):
        s += [768, 768, 768 * 2304, 2304, 768 * 768, 768, 768, 768, 768 * 3072, 3072, 3072 * 768, 768]
    s += [768, 768]
    return s


def scaled_shapes(shapes: List[int], target_total: int) -> List[int]:
    """The same table shrunk to about target_total parameters (at least one per tensor)."""
    tot = sum(shapes)
    return [max(1, int(round(x * target_total / tot))) for x in shapes]


# ---- workloads -------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    shapes: List[int]
    N: int
    sparsity: List[float]
    base: str  # "gauss" | "student3" | "laplace"
    sigma_range: Optional[tuple]  # log-uniform per tensor; None = constant scale `const_sigma`
    rho: float
    steps: int
    grad_dtype: str = "f32"  # "f32" | "bf16"
    zero_fraction: float = 0.0  # share of coordinates in tensors whose gradient is exactly zero
    embedding_rows: Optional[tuple] = None  # (rows, cols, share of rows that are non-zero)
    boost: Optional[tuple] = None  # (share of coordinates, factor) at fixed random positions
    const_sigma: float = 1.0
    mu: float = 4.0

    @property
    def d(self) -> int:
        return int(sum(self.shapes))

    def k_values(self) -> List[int]:
        return [int(math.floor(s * self.d + 0.5)) for s in self.sparsity]


def workload(name: str, scale_to: Optional[int] = None) -> Workload:
    """The model-shaped benchmark workloads; scale_to shrinks the tensor table for parity tests."""
    if name == "resnet18":
        w = Workload("resnet18", resnet18_cifar_shapes(), 8, [1e-3, 1e-2], "gauss", (1e-4, 1e-1), 0.9, 20)
    elif name == "resnet50":
        w = Workload("resnet50", resnet50_shapes(), 16, [1e-3], "student3", (1e-5, 1e-2), 0.8, 20,
                     zero_fraction=0.3)
    elif name == "gpt2":
        w = Workload("gpt2", gpt2_small_shapes(), 8, [1e-4, 1e-3], "gauss", (1e-4, 1e-1), 0.9, 10,
                     grad_dtype="bf16", embedding_rows=(50257, 768, 0.1))
    elif name == "flat1p3b":
        w = Workload("flat1p3b", [1_300_000_000], 4, [1e-4, 1e-3, 1e-2], "laplace", None, 0.95, 5,
                     boost=(0.01, 100.0), const_sigma=1e-3)
    else:
        raise KeyError(name)
    if scale_to is not None:
        if w.embedding_rows is not None:
            rows, cols, share = w.embedding_rows
            cols_s = max(8, int(round(cols * math.sqrt(scale_to / w.d))))
            rows_s = max(16, int(round(rows * cols * scale_to / w.d / cols_s)))
            rest = scaled_shapes(w.shapes[1:], max(1, scale_to - rows_s * cols_s))
            w.shapes = [rows_s * cols_s] + rest
            w.embedding_rows = (rows_s, cols_s, share)
        else:
            w.shapes = scaled_shapes(w.shapes, scale_to)
    return w


class GradientStream:
    """Seeded generator of the rounds of one workload: next() returns grads [N, ld] on `device`
    (float32, or bfloat16 for bf16 workloads), ld = d rounded up to `pad_to`; the padding is zero."""

    def __init__(self, w: Workload, device="cpu", seed=0, pad_to=1, chunk=1 << 24):
        self.w, self.device, self.chunk = w, torch.device(device), chunk
        self.d = w.d
        self.ld = (self.d + pad_to - 1) // pad_to * pad_to
        self.gen = torch.Generator(device=self.device)
        self.gen.manual_seed(seed)
        host = np.random.default_rng(seed)
        L = len(w.shapes)
        if w.sigma_range is None:
            sig = np.full(L, w.const_sigma)
        else:
            lo, hi = w.sigma_range
            sig = np.exp(host.uniform(math.log(lo), math.log(hi), size=L))
        frozen = np.zeros(L, bool)
        self.partial_frozen = None
        if w.zero_fraction > 0:
            want = int(w.zero_fraction * self.d)
            got = 0
            starts = np.concatenate([[0], np.cumsum(w.shapes)])
            for l in host.permutation(L):
                if got >= want:
                    break
                if got + w.shapes[l] <= want:
                    frozen[l] = True
                    got += w.shapes[l]
                else:  # the last one only partially
                    self.partial_frozen = (int(starts[l]), int(starts[l] + (want - got)))
                    got = want
        sig = np.where(frozen, 0.0, sig)
        sizes = torch.tensor(w.shapes, dtype=torch.int64)
        self.sigma = torch.repeat_interleave(torch.tensor(sig, dtype=torch.float32), sizes).to(self.device)
        if self.partial_frozen is not None:
            self.sigma[self.partial_frozen[0]:self.partial_frozen[1]] = 0.0
        if w.boost is not None:
            share, factor = w.boost
            nb = int(share * self.d)
            pos = torch.randint(0, self.d, (nb,), generator=self.gen, device=self.device)
            self.sigma[pos] *= factor
        self.c = None
        self.t = 0

    def _base(self, n):
        b = self.w.base
        if b == "gauss":
            return torch.randn(n, generator=self.gen, device=self.device)
        if b == "student3":
            z = torch.randn(n, generator=self.gen, device=self.device)
            q = torch.zeros(n, device=self.device)
            for _ in range(3):
                q += torch.randn(n, generator=self.gen, device=self.device) ** 2
            return z / torch.sqrt(q / 3.0)
        if b == "laplace":
            u = torch.rand(n, generator=self.gen, device=self.device) - 0.5
            return -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.4999999))
        raise ValueError(b)

    def next(self) -> torch.Tensor:
        w, d = self.w, self.d
        if self.c is None:
            self.c = torch.empty(d, device=self.device)
        out_dtype = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
        grads = torch.zeros((w.N, self.ld), dtype=out_dtype, device=self.device)
        a = math.sqrt(1.0 - w.rho * w.rho)
        for s in range(0, d, self.chunk):
            e = min(d, s + self.chunk)
            sg = self.sigma[s:e]
            z = self._base(e - s) * sg
            if self.t == 0:
                self.c[s:e] = z
            else:
                self.c[s:e] = w.rho * self.c[s:e] + a * z
            for n in range(w.N):
                grads[n, s:e] = (self.c[s:e] + 0.5 * sg * self._base(e - s)).to(out_dtype)
        if w.embedding_rows is not None:
            rows, cols, share = w.embedding_rows
            for n in range(w.N):
                keep = torch.rand(rows, generator=self.gen, device=self.device) < share
                block = grads[n, : rows * cols].view(rows, cols)
                block.mul_(keep.to(out_dtype).unsqueeze(1))
        self.t += 1
        return grads


# ---- distributed least squares (the small end-to-end problem) ---------------------------------------
@dataclass
class LeastSquares:
    """N workers, each with A_n (rows x d) ~ N(0, 1/d) and y_n = A_n x* + noise * N(0,1), x* ~ N(0,1).
    Loss 0.5 * mean_n ||A_n theta - y_n||^2; worker gradient g_n = A_n^T (A_n theta - y_n)."""
    N: int = 8
    rows: int = 512
    d: int = 4096
    noise: float = 0.01
    seed: int = 0
    A: np.ndarray = field(init=False, repr=False)
    y: np.ndarray = field(init=False, repr=False)
    x_star: np.ndarray = field(init=False, repr=False)

    def __post_init__(self):
        rng = np.random.default_rng(self.seed)
        self.x_star = rng.standard_normal(self.d)
        self.A = rng.standard_normal((self.N, self.rows, self.d)) / math.sqrt(self.d)
        self.y = np.einsum("nrd,d->nr", self.A, self.x_star) + self.noise * rng.standard_normal((self.N, self.rows))

    def gradients(self, theta: np.ndarray) -> np.ndarray:
        r = np.einsum("nrd,d->nr", self.A, theta) - self.y
        return np.einsum("nrd,nr->nd", self.A, r).astype(np.float32)

    def loss(self, theta: np.ndarray) -> float:
        r = np.einsum("nrd,d->nr", self.A, theta) - self.y
        return float(0.5 * np.mean(np.sum(r * r, axis=1)))
