"""Seeded synthetic inputs for the plasticity-evaluation path.

This module only *draws inputs*: activation pairs (A_T, A_R) in bfloat16 and raw
loss histories in float32.  It holds none of the method's arithmetic (no Gram,
no normalisation, no loss, no smoothing, no fit) and imports neither the CUDA
binding nor the CPU oracle, so both can be fed from it.

The five named workloads stand in for the activations of the paper's vision and
language tasks (Sec. 6.1, Table 1: ResNet-56/CIFAR-10, ResNet-50/ImageNet,
BERT-base/SQuAD, Transformer language models); only their shapes and value
structure are reproduced -- the datasets and weights are not needed.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

SEED_BASE = 20220106


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                  # 1-based position in the list of named workloads
    b: int                      # batch size (rows of every activation matrix)
    d: Tuple[int, ...]          # flattened per-sample size of every monitored module
    kind: str                   # "relu" | "ln_outlier" | "normal"
    sigma: Tuple[float, float]  # reference perturbation, first .. last module
    H: int                      # length of the raw-loss history for the slope stage
    W: int                      # window (smoothing span, fit window, stale count)
    T: float                    # tolerance on |slope|
    hist_noise: float = 0.0     # std-dev of the noise added to the synthetic history
    shape_note: str = ""

    @property
    def M(self) -> int:
        return len(self.d)

    @property
    def sum_d(self) -> int:
        return int(sum(self.d))

    @property
    def input_bytes(self) -> int:
        """Bytes of both bf16 matrices of every module: 4 * b * sum(d)."""
        return 4 * self.b * self.sum_d

    def sigma_of(self, l: int) -> float:
        if self.M == 1:
            return self.sigma[0]
        return self.sigma[0] + (self.sigma[1] - self.sigma[0]) * l / (self.M - 1)

    def seed_of(self, l: int) -> int:
        return SEED_BASE + 1000 * self.index + l


WORKLOADS = {
    "tiny": Workload("tiny", 1, 8, (4096,), "relu", (0.1, 0.1), 20, 5, 1e-3,
                     shape_note="single module, b=8, d=4096"),
    "resnet56": Workload("resnet56", 2, 128, (16384,) * 9 + (8192,) * 9 + (4096,) * 9, "relu",
                         (0.02, 0.5), 40, 10, 1e-4,
                         shape_note="27 residual-block outputs, CIFAR-sized feature maps"),
    "resnet50": Workload("resnet50", 3, 64,
                         (802816,) * 3 + (401408,) * 4 + (200704,) * 6 + (100352,) * 3, "relu",
                         (0.01, 0.3), 200, 20, 1e-4,
                         shape_note="16 bottleneck outputs, ImageNet-sized feature maps"),
    "bert_base": Workload("bert_base", 4, 32, (128 * 768,) * 12, "ln_outlier", (0.05, 0.4),
                          40, 10, 1e-4, shape_note="12 encoder layers, seq 128 x hidden 768"),
    "gpt2_medium": Workload("gpt2_medium", 5, 256, (256 * 1024,) * 24, "normal", (0.02, 0.3),
                            1000, 50, 5e-5, hist_noise=1e-5,
                            shape_note="24 decoder layers, seq 256 x hidden 1024"),
}
ORDER = ["tiny", "resnet56", "resnet50", "bert_base", "gpt2_medium"]


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_pair(b: int, d: int, kind: str, sigma: float, seed: int, device="cpu",
              hidden: int = 768) -> Tuple[torch.Tensor, torch.Tensor]:
    """One (A_T, A_R) pair, bfloat16 [b, d], from one seed.

    relu       : pre ~ N(0,1); A_T = relu(pre); A_R = relu(pre + sigma*N(0,1))
                 (half-normal values, about half of them exactly zero)
    normal     : x ~ N(0,1); A_T = x; A_R = x + sigma*N(0,1)
    ln_outlier : as normal, but 1% of the `hidden` feature indices (seeded choice,
                 same at every position) are scaled by 8 before the noise is added
    """
    g = _gen(device, seed)
    x = torch.randn((b, d), generator=g, device=device, dtype=torch.float32)
    if kind == "ln_outlier":
        n_out = max(1, round(0.01 * hidden))
        gi = torch.Generator(device="cpu")
        gi.manual_seed(int(seed) ^ 0x5EED)
        idx = torch.randperm(hidden, generator=gi)[:n_out].to(device)
        scale = torch.ones(hidden, device=device, dtype=torch.float32)
        scale[idx] = 8.0
        reps = (d + hidden - 1) // hidden
        x = x * scale.repeat(reps)[:d].unsqueeze(0)
    noise = torch.randn((b, d), generator=g, device=device, dtype=torch.float32)
    y = x + float(sigma) * noise
    del noise
    if kind == "relu":
        x = torch.relu_(x)
        y = torch.relu_(y)
    elif kind not in ("normal", "ln_outlier"):
        raise ValueError(f"unknown activation kind {kind!r}")
    return x.to(torch.bfloat16).contiguous(), y.to(torch.bfloat16).contiguous()


def make_module(w: Workload, l: int, device="cpu", sigma: Optional[float] = None,
                seed_offset: int = 0) -> Tuple[torch.Tensor, torch.Tensor]:
    """Activation pair of module l of a named workload."""
    s = w.sigma_of(l) if sigma is None else sigma
    return make_pair(w.b, w.d[l], w.kind, s, w.seed_of(l) + 100000 * seed_offset, device)


def make_activations(w: Workload, device="cpu", modules: Optional[Sequence[int]] = None
                     ) -> Tuple[List[torch.Tensor], List[torch.Tensor]]:
    """Activation pairs of every (or the listed) module of a named workload."""
    ms = range(w.M) if modules is None else modules
    at, ar = [], []
    for l in ms:
        t, r = make_module(w, l, device)
        at.append(t)
        ar.append(r)
    return at, ar


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The bfloat16 bit patterns of a tensor as a host uint16 array (same shape)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def from_bits(bits: np.ndarray, device="cpu") -> torch.Tensor:
    """Inverse of bf16_bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def tiny_history_sigmas(w: Workload) -> List[float]:
    """Perturbation per evaluation of the tiny workload's real 20-step history."""
    if w.H == 1:
        return [0.5]
    return [0.5 + (0.01 - 0.5) * k / (w.H - 1) for k in range(w.H)]


def make_history(w: Workload, levels: Sequence[float], H: Optional[int] = None,
                 tau_scale: float = 1.0) -> np.ndarray:
    """Synthetic raw-loss histories, float32 [M, H].

    Module l decays towards its level L_l: h_l[k] = L_l * (1 + 4*exp(-k/tau_l)) (+ noise),
    tau_l = tau_scale * H * (0.05 + 0.5*l/(M-1)), so front modules flatten inside the history
    and deep ones do not (a small tau_scale makes every module flatten quickly).  Noise (if
    any) is N(0, hist_noise), seeded."""
    H = w.H if H is None else H
    M = len(levels)
    k = np.arange(H, dtype=np.float64)
    out = np.empty((M, H), dtype=np.float64)
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + 1000 * w.index + 999))
    for l in range(M):
        tau = tau_scale * H * (0.05 + 0.5 * (l / (M - 1) if M > 1 else 0.0))
        out[l] = float(levels[l]) * (1.0 + 4.0 * np.exp(-k / tau))
        if w.hist_noise > 0.0:
            out[l] += rng.normal(0.0, w.hist_noise, size=H)
    return out.astype(np.float32)
