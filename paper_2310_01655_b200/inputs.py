"""Seeded synthetic inputs for causal Polysketch attention.

This module only draws random tensors and applies the per-row normalisation
that stands in for the LayerNorm the paper applies to queries and keys before
attention (Section 2.1).  It holds none of the attention arithmetic, so both
the CUDA library's tests and the CPU oracle's tests can take their inputs from
it without sharing any of the method's code.

Layout: Q, K, V, dO are [B, H, n, h] contiguous; G1, G2 are [H, h, r] (one pair
per head, shared across the batch and between Q and K).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, asdict

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    n: int
    h: int
    r: int
    p: int
    b: int
    dtype: str          # "f32" | "bf16"  (storage type of Q, K, V, G, O, gradients)
    backward: bool
    data_seed: int
    g_seed: int
    correlated: bool = False

    @property
    def head_tokens(self) -> int:
        return self.B * self.H * self.n

    @property
    def model_tokens(self) -> int:
        return self.B * self.n

    def asdict(self):
        return asdict(self)


# The five benchmark configurations.  c0's seeds are fixed by the configuration
# text; the others follow "1000 + index" (data) and "2000 + index" (sketch).
WORKLOADS = {
    "c0": Workload("c0", 1, 1, 1024, 64, 16, 4, 128, "f32", False, 0, 1),
    "c1": Workload("c1", 128, 12, 8192, 64, 32, 4, 256, "bf16", False, 1001, 2001),
    "c2": Workload("c2", 32, 12, 32768, 64, 32, 4, 256, "bf16", True, 1002, 2002),
    "c3": Workload("c3", 32, 12, 32768, 64, 64, 4, 512, "bf16", True, 1003, 2003),
    "c4": Workload("c4", 8, 16, 131072, 64, 32, 4, 256, "bf16", True, 1004, 2004, True),
    # profiling-sized slices of c2 / c3 (same n, r, b; 2 batch elements): a few GB on the device
    "c2s": Workload("c2s", 2, 12, 32768, 64, 32, 4, 256, "bf16", True, 1002, 2002),
    "c3s": Workload("c3s", 2, 12, 32768, 64, 64, 4, 512, "bf16", True, 1003, 2003),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _normalise_rows(x: torch.Tensor) -> torch.Tensor:
    """L2-normalise each row and scale by sqrt(h) (fp32)."""
    h = x.shape[-1]
    return x * (math.sqrt(h) / x.norm(dim=-1, keepdim=True).clamp_min(1e-30))


def make_inputs(w: Workload, device="cpu", with_dO=None):
    """Draw Q, K, V (and dO), G1, G2 for a workload.

    Values are drawn in fp32 from a generator seeded with the workload's seeds
    on `device` (the CPU and CUDA generators give different streams; whoever
    checks a result copies the stored tensors, never re-draws them).  Q and K
    rows are normalised in fp32, then everything is rounded to the storage type.
    Drawn one batch element at a time so the fp32 temporaries stay small.
    """
    dev = torch.device(device)
    dt = torch_dtype(w.dtype)
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.data_seed)
    want_dO = w.backward if with_dO is None else with_dO
    shape = (w.B, w.H, w.n, w.h)
    names = ["Q", "K", "V"] + (["dO"] if want_dO else [])
    out = {k: torch.empty(shape, dtype=dt, device=dev) for k in names}
    if w.correlated:
        u = torch.randn((w.H, 1, w.h), generator=gen, device=dev, dtype=torch.float32)
        u = u / u.norm(dim=-1, keepdim=True)
        shift = math.sqrt(w.h) * u
    for bi in range(w.B):
        for k in names:
            x = torch.randn((w.H, w.n, w.h), generator=gen, device=dev, dtype=torch.float32)
            if w.correlated and k != "dO":
                x = x + shift
            if k in ("Q", "K"):
                x = _normalise_rows(x)
            out[k][bi].copy_(x)
    ggen = torch.Generator(device=dev)
    ggen.manual_seed(w.g_seed)
    out["G1"] = torch.randn((w.H, w.h, w.r), generator=ggen, device=dev, dtype=torch.float32).to(dt)
    out["G2"] = torch.randn((w.H, w.h, w.r), generator=ggen, device=dev, dtype=torch.float32).to(dt)
    return out


def small_workload(name="tiny", B=1, H=2, n=384, h=64, r=16, b=128, dtype="f32",
                   backward=True, seed=7, correlated=False) -> Workload:
    """A test-sized workload with the same recipe as the benchmark configurations."""
    return Workload(name, B, H, n, h, r, 4, b, dtype, backward, seed, seed + 1000, correlated)


def head_slice_f64(t: torch.Tensor, bi: int, hi: int):
    """One (batch, head) slice of a stored tensor, widened to float64 on the host."""
    return t[bi, hi].detach().to("cpu").to(torch.float64).numpy()


def learned_network_params(h: int, r: int, seed: int):
    """Seeded parameters of the learnable sketch's two dense networks (Algorithm 2 of the appendix) as two
    dicts of float64 numpy arrays: gains near one, small biases, weights scaled so that every layer
    keeps its input's scale.  Draws only; none of the method's arithmetic."""
    import numpy as np
    g = np.random.default_rng(seed)
    m = 8 * r

    def net():
        return {"g0": 1.0 + 0.1 * g.standard_normal(h), "c0": 0.1 * g.standard_normal(h),
                "W1": g.standard_normal((h, m)) / np.sqrt(h), "b1": 0.1 * g.standard_normal(m),
                "g1": 1.0 + 0.1 * g.standard_normal(m), "c1": 0.1 * g.standard_normal(m),
                "W2": g.standard_normal((m, r)) / np.sqrt(m), "b2": 0.1 * g.standard_normal(r),
                "W3": g.standard_normal((r, m)) / np.sqrt(r), "b3": 0.1 * g.standard_normal(m),
                "W4": 1.5 * g.standard_normal((m, r)) / np.sqrt(m), "b4": 0.1 * g.standard_normal(r)}

    return net(), net()
