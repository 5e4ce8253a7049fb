"""Gated SA + SWA forward for tensors that live in host memory.

A thin holder of the device workspace around the C entry point ``sa_swa_gated_forward_host``,
which owns the pipeline: the KV heads (and the query heads that share them) travel through the
GPU in pieces on three streams (copy in, compute, copy out), the permutation of Section 3.1 is
drawn once per call and shared by all pieces.  Nothing of the path runs here.
"""
from typing import Optional

import torch

from . import binding as sa


class HostForward:
    """Preallocated device workspace for repeated host-to-host forwards of one shape."""

    def __init__(self, B: int, Hq: int, Hkv: int, n: int, d: int, w: int,
                 flags: int = sa.CAUSAL | sa.SWA_ONE_SIDED, dtype=torch.bfloat16,
                 n_groups: int = 8, q_parts: int = 2, device: Optional[torch.device] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("HostForward needs a CUDA device")
        self.device = device or torch.device("cuda", torch.cuda.current_device())
        self.shape = (B, Hq, Hkv, n, d)
        self.w, self.flags, self.dtype = w, flags, dtype
        self.n_groups, self.q_parts = n_groups, q_parts
        self.pieces = sa.host_forward_plan(Hq, Hkv, n_groups, q_parts)
        code = sa.BF16 if dtype == torch.bfloat16 else sa.F32
        self.ws = torch.empty(sa.host_forward_ws_bytes(B, Hq, Hkv, n, d, code), dtype=torch.uint8,
                              device=self.device)

    def _elt(self) -> int:
        return 2 if self.dtype == torch.bfloat16 else 4

    def h2d_bytes(self) -> int:
        B, Hq, Hkv, n, d = self.shape
        return (B * Hq + 2 * B * Hkv) * n * d * self._elt() + 2 * Hq * 4

    def d2h_bytes(self) -> int:
        B, Hq, _, n, d = self.shape
        return B * Hq * n * d * self._elt()

    def forward(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, gate_logits: torch.Tensor,
                y: torch.Tensor, seed: int, layer: int) -> torch.Tensor:
        """q, k, v, gate_logits: host tensors (pinned for the copies to overlap); y: host output,
        complete once the current stream has been synchronised."""
        return sa.sa_swa_gated_forward_host(q, k, v, gate_logits, y, self.w, self.flags, seed,
                                            layer, self.ws, self.n_groups, self.q_parts)
