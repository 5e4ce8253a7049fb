"""Gated SA + SWA forward for tensors that live in host memory.

The attention of one KV head (and of the query heads that share it) reads nothing of the other
heads, so the heads travel through the GPU in groups: while one group is being computed, the
next one is on its way in over PCIe and the previous result is on its way out.  Three streams
(copy in, compute, copy out) and one event pair per group do the ordering; every kernel is the
same C-ABI call the device-resident path makes, on strided views of whole-size device buffers.
The permutation of Section 3.1 is drawn once per call and shared by all groups.
"""
from typing import List, Optional, Tuple

import torch

from . import binding as sa


def head_groups(Hq: int, Hkv: int, n_groups: int) -> List[Tuple[int, int, int, int]]:
    """Splits the KV heads into at most ``n_groups`` contiguous ranges.

    Returns (kv_begin, kv_end, q_begin, q_end) per range; the query heads of a KV head h are
    h*G .. (h+1)*G - 1 with G = Hq / Hkv (the grouped-query layout of the library)."""
    if Hq < 1 or Hkv < 1 or Hq % Hkv:
        raise ValueError("Hq must be a positive multiple of Hkv")
    n_groups = max(1, min(int(n_groups), Hkv))
    G = Hq // Hkv
    out = []
    for i in range(n_groups):
        a = i * Hkv // n_groups
        b = (i + 1) * Hkv // n_groups
        if b > a:
            out.append((a, b, a * G, b * G))
    return out


def split_query_heads(groups: List[Tuple[int, int, int, int]], parts: int
                      ) -> List[Tuple[int, int, int, int, bool]]:
    """Cuts every single-KV-head range of ``head_groups`` into ``parts`` ranges of query heads
    (kv_begin, kv_end, q_begin, q_end, carries_kv); only the first range of a KV head carries
    its K/V copy.  Ranges with several KV heads, or whose query heads do not divide, stay whole.
    Smaller first and last pieces shorten the parts of the pipeline that cannot overlap."""
    out = []
    for ka, kb, qa, qb in groups:
        G = qb - qa
        if kb - ka == 1 and parts > 1 and G % parts == 0:
            step = G // parts
            for i in range(parts):
                out.append((ka, kb, qa + i * step, qa + (i + 1) * step, i == 0))
        else:
            out.append((ka, kb, qa, qb, True))
    return out


class HostForward:
    """Preallocated device buffers, streams and events for repeated host-to-host forwards."""

    def __init__(self, B: int, Hq: int, Hkv: int, n: int, d: int, w: int,
                 flags: int = sa.CAUSAL | sa.SWA_ONE_SIDED, dtype=torch.bfloat16,
                 n_groups: int = 8, q_parts: int = 2, device: Optional[torch.device] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("HostForward needs a CUDA device")
        self.device = device or torch.device("cuda", torch.cuda.current_device())
        self.shape = (B, Hq, Hkv, n, d)
        self.w, self.flags = w, flags
        self.groups = split_query_heads(head_groups(Hq, Hkv, n_groups), q_parts)
        dev = self.device
        self.q = torch.empty(B, Hq, n, d, dtype=dtype, device=dev)
        self.k = torch.empty(B, Hkv, n, d, dtype=dtype, device=dev)
        self.v = torch.empty(B, Hkv, n, d, dtype=dtype, device=dev)
        self.y = torch.empty(B, Hq, n, d, dtype=dtype, device=dev)
        self.gate = torch.empty(2, Hq, dtype=torch.float32, device=dev)
        # the library wants each group's logits as a contiguous [2, heads] block
        self.gate_g = [torch.empty(2, qe - qb, dtype=torch.float32, device=dev)
                       for (_, _, qb, qe, _) in self.groups]
        self.perm = torch.empty(B, n, dtype=torch.int32, device=dev)
        self.inv = torch.empty(B, n, dtype=torch.int32, device=dev)
        nbytes = sa.sa_workspace_bytes(sa.SaProblem(B=B, n=n), sa.OP_MAKE_PERM)
        self.ws = torch.empty(max(nbytes, 1), dtype=torch.uint8, device=dev)
        # scratch for the local branch's rows of one head group (in the layout of y)
        self.scratch = torch.empty(self.y.numel() * self.y.element_size(), dtype=torch.uint8,
                                   device=dev)
        self.s_in = torch.cuda.Stream(dev)
        self.s_run = torch.cuda.Stream(dev)
        self.s_out = torch.cuda.Stream(dev)
        self.ev_in = [torch.cuda.Event() for _ in self.groups]
        self.ev_done = [torch.cuda.Event() for _ in self.groups]

    def h2d_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in (self.q, self.k, self.v, self.gate))

    def d2h_bytes(self) -> int:
        return self.y.numel() * self.y.element_size()

    def forward(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, gate_logits: torch.Tensor,
                y: torch.Tensor, seed: int, layer: int) -> torch.Tensor:
        """q, k, v, gate_logits: host tensors (pinned for the copies to overlap); y: host output.

        Work is ordered after what the current stream has queued, and the current stream waits
        for the last copy out, so the caller synchronises (or times) on the current stream."""
        cur = torch.cuda.current_stream(self.device)
        for s in (self.s_in, self.s_run, self.s_out):
            s.wait_stream(cur)
        with torch.cuda.stream(self.s_in):
            self.gate.copy_(gate_logits, non_blocking=True)
            B = self.shape[0]
            for i, (ka, kb, qa, qb, with_kv) in enumerate(self.groups):
                for bi in range(B):          # one contiguous block per sequence and tensor
                    if with_kv:
                        self.k[bi, ka:kb].copy_(k[bi, ka:kb], non_blocking=True)
                        self.v[bi, ka:kb].copy_(v[bi, ka:kb], non_blocking=True)
                    self.q[bi, qa:qb].copy_(q[bi, qa:qb], non_blocking=True)
                self.ev_in[i].record(self.s_in)
        with torch.cuda.stream(self.s_run):
            B, _, _, n, _ = self.shape
            sa.sa_make_perm(seed, layer, B, n, perm=self.perm, inv=self.inv, ws=self.ws)
            for i, (ka, kb, qa, qb, _) in enumerate(self.groups):
                self.s_run.wait_event(self.ev_in[i])
                self.gate_g[i].copy_(self.gate[:, qa:qb])
                sa.sa_swa_gated_forward(self.q[:, qa:qb], self.k[:, ka:kb], self.v[:, ka:kb],
                                        self.perm, self.inv, self.gate_g[i], self.w, self.flags,
                                        out={"y": self.y[:, qa:qb]}, ws=self.scratch)
                self.ev_done[i].record(self.s_run)
        with torch.cuda.stream(self.s_out):
            for i, (_, _, qa, qb, _) in enumerate(self.groups):
                self.s_out.wait_event(self.ev_done[i])
                for bi in range(self.shape[0]):
                    y[bi, qa:qb].copy_(self.y[bi, qa:qb], non_blocking=True)
        cur.wait_stream(self.s_out)
        return y
