"""Seeded synthetic inputs and the named workload shapes.

This module holds NO arithmetic of the method: it only draws Q/K/V/dY/gate logits
from a seeded generator, rounds them once to the run dtype, and names the shapes.
Both the CUDA path and the CPU checker are fed the same rounded values from here,
so a comparison measures the kernels and not the input rounding.

Shapes follow the attention geometry of the paper's settings (pre-training model:
16 heads of 64, w = 256, App. B; Qwen3-8B / Qwen3-30B-A3B prefill: 32 query heads
over 8 / 4 KV heads of 128, Sec. 4.2).  They stand in for those models' activations:
no dataset, weight or benchmark item is used anywhere.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

CAUSAL = 1
LINEAR_WINDOW = 2
SWA_ONE_SIDED = 4
SAVE_FOR_BWD = 8
VALIDATE_PERM = 16


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str          # "f32" | "bf16"
    B: int
    Hq: int
    Hkv: int
    n: int
    d: int
    w: int
    layers: int = 1
    seed: int = 0
    flags: int = CAUSAL | SWA_ONE_SIDED
    qkv_scale: float = 1.0   # multiplies the N(0,1) draws of Q, K, V
    ops: str = "sa_fwd"      # "sa_fwd" | "gated_fwd" | "gated_fwd_bwd"

    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations the library is measured and checked on.
C1 = Workload("C1_tiny_f32", "f32", 1, 1, 1, 256, 64, 32, seed=0, ops="sa_fwd")
C2 = Workload("C2_layer_bf16", "bf16", 2, 16, 16, 4096, 128, 256, seed=1,
              qkv_scale=128 ** -0.5, ops="sa_fwd")
C3 = Workload("C3_qwen3_8b_gated", "bf16", 1, 32, 8, 32768, 128, 1024, seed=2, ops="gated_fwd")
C4 = Workload("C4_qwen3_30b_a3b_prefill", "bf16", 1, 32, 4, 131072, 128, 2048, layers=48,
              seed=3, ops="gated_fwd")
C5 = Workload("C5_pretrain_fwd_bwd", "bf16", 8, 12, 12, 4096, 64, 128, layers=12, seed=4,
              ops="gated_fwd_bwd")
CONFIGS = {c.name: c for c in (C1, C2, C3, C4, C5)}


def draw(wl: Workload, device="cpu", pin=False):
    """Q, K, V, dY ~ N(0,1)*qkv_scale (dY unscaled), gate logits ~ N(0,1) fp32.

    Drawn on the host in float32 from torch's seeded CPU generator, rounded once
    to the run dtype.  Returns a dict of tensors (contiguous [B,H,n,d])."""
    g = torch.Generator(device="cpu")
    g.manual_seed(wl.seed)
    dt = wl.torch_dtype()

    def normal(*shape, scale=1.0):
        t = torch.randn(*shape, generator=g, dtype=torch.float32)
        if scale != 1.0:
            t = t * scale
        t = t.to(dt)
        if pin and device == "cpu":
            t = t.pin_memory()
        return t.to(device)

    out = {
        "q": normal(wl.B, wl.Hq, wl.n, wl.d, scale=wl.qkv_scale),
        "k": normal(wl.B, wl.Hkv, wl.n, wl.d, scale=wl.qkv_scale),
        "v": normal(wl.B, wl.Hkv, wl.n, wl.d, scale=wl.qkv_scale),
    }
    if wl.ops == "gated_fwd_bwd":
        out["dy"] = normal(wl.B, wl.Hq, wl.n, wl.d)
    logits = torch.randn(2, wl.Hq, generator=g, dtype=torch.float32)
    out["gate_logits"] = logits.to(device)
    return out


def as_f64(t: torch.Tensor):
    """Widen a (possibly bf16, possibly CUDA) tensor to a float64 numpy array."""
    return t.detach().to("cpu").to(torch.float64).numpy()
