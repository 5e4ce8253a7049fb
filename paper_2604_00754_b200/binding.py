"""Python binding of the C ABI declared in ``include/sa.h``: argument marshalling only.

Every step of the path runs in the CUDA library; torch is used here for device memory
and the current stream.  There is no fallback of any kind: if the shared library is
missing and cannot be built, or a call returns an error status, an exception is raised.

The functions carry the C names (``sa_make_perm``, ``sa_forward``, ``sa_swa_forward``,
``sa_swa_gated_forward``, ``sa_backward``, ``sa_coverage``) and take torch CUDA tensors
where the C functions take device pointers.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

SA_OK = 0
CAUSAL, LINEAR_WINDOW, SWA_ONE_SIDED, SAVE_FOR_BWD, VALIDATE_PERM = 1, 2, 4, 8, 16
OP_MAKE_PERM, OP_FORWARD, OP_SWA_FORWARD, OP_GATED_FORWARD, OP_BACKWARD, OP_COVERAGE = range(6)
OP_GATED_FORWARD_SCRATCH = 6
F32, BF16 = 0, 1

EXPORTS = [
    "sa_problem_set_contiguous", "sa_workspace_bytes", "sa_make_perm", "sa_forward",
    "sa_swa_forward", "sa_swa_gated_forward", "sa_backward", "sa_coverage", "sa_read_status",
    "sa_status_string", "sa_launch_count", "sa_set_profile_events", "sa_make_perm_static",
    "sa_gate_projection_forward", "sa_gate_projection_backward",
    "sa_gate_projection_backward_ws_bytes", "sa_debug_set", "sa_debug_wait_timeout",
    "sa_swa_gated_forward_host", "sa_host_forward_ws_bytes", "sa_host_forward_plan",
    "sa_rope_table", "sa_rope_apply", "sa_forward_rope", "sa_swa_gated_forward_rope",
]
OP_FORWARD_ROPE = 7
DEBUG_SCORE_BLOCK, DEBUG_SWA_TILE_LOADS, DEBUG_TENSOR_CORES, DEBUG_GATE_WIDE_TILES = range(4)


class SaProblem(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32),
        ("n", ctypes.c_int32), ("d", ctypes.c_int32), ("w", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("flags", ctypes.c_uint32),
        ("softmax_scale", ctypes.c_float), ("L", ctypes.c_int32),
        ("q_stride", ctypes.c_int64 * 3), ("kv_stride", ctypes.c_int64 * 3),
    ]


class SaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (where, status_string(status), status))


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads (building first if the sources are newer) the CUDA library; raises if it cannot."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    if path is None:
        path = _build.LIB
        if _build.stale():
            try:
                _build.build_library()
            except Exception as e:  # no nvcc, compile error
                # never run a library older than its sources: that would test stale kernels
                what = "is older than its sources" if os.path.exists(path) else "is missing"
                raise RuntimeError("CUDA library %s %s and could not be built: %s"
                                   % (path, what, e)) from e
    lib = ctypes.CDLL(path)
    vp, i32, u32, u64, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32, ctypes.c_uint64,
                             ctypes.c_size_t)
    pp = ctypes.POINTER(SaProblem)
    lib.sa_problem_set_contiguous.argtypes = [pp]
    lib.sa_problem_set_contiguous.restype = None
    lib.sa_workspace_bytes.argtypes = [pp, ctypes.c_int]
    lib.sa_workspace_bytes.restype = sz
    lib.sa_make_perm.argtypes = [u64, u32, i32, i32, vp, vp, vp, sz, vp]
    lib.sa_make_perm_static.argtypes = [u64, u32, i32, i32, vp, vp, vp]
    lib.sa_make_perm_static.restype = ctypes.c_int
    lib.sa_forward.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sa_swa_forward.argtypes = [pp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sa_swa_gated_forward.argtypes = [pp] + [vp] * 12 + [sz, vp]
    lib.sa_backward.argtypes = [pp] + [vp] * 16 + [sz, vp]
    lib.sa_coverage.argtypes = [i32, i32, i32, u32, vp, vp, i32, vp, vp, vp, vp, sz, vp]
    lib.sa_gate_projection_forward.argtypes = [ctypes.c_int64, i32, i32, vp, vp, ctypes.c_int64,
                                               vp, vp, vp, ctypes.c_int64, vp]
    lib.sa_gate_projection_forward.restype = ctypes.c_int
    i64 = ctypes.c_int64
    lib.sa_gate_projection_backward_ws_bytes.argtypes = [i64, i32]
    lib.sa_gate_projection_backward_ws_bytes.restype = sz
    lib.sa_gate_projection_backward.argtypes = [i64, i32, i32, vp, i64, vp, vp, i64, vp, vp, vp, vp,
                                                i64, vp, vp, vp, sz, vp]
    lib.sa_gate_projection_backward.restype = ctypes.c_int
    lib.sa_read_status.argtypes = [vp]
    for f in ("sa_make_perm", "sa_forward", "sa_swa_forward", "sa_swa_gated_forward",
              "sa_backward", "sa_coverage", "sa_read_status"):
        getattr(lib, f).restype = ctypes.c_int
    lib.sa_status_string.argtypes = [ctypes.c_int]
    lib.sa_status_string.restype = ctypes.c_char_p
    lib.sa_set_profile_events.argtypes = [vp, vp]
    lib.sa_set_profile_events.restype = None
    lib.sa_launch_count.argtypes = []
    lib.sa_launch_count.restype = u64
    lib.sa_host_forward_ws_bytes.argtypes = [pp]
    lib.sa_host_forward_ws_bytes.restype = sz
    lib.sa_host_forward_plan.argtypes = [i32, i32, i32, i32, vp, i32]
    lib.sa_host_forward_plan.restype = i32
    lib.sa_swa_gated_forward_host.argtypes = [pp, vp, vp, vp, vp, vp, u64, u32, i32, i32, vp, sz, vp]
    lib.sa_swa_gated_forward_host.restype = ctypes.c_int
    lib.sa_rope_table.argtypes = [i32, i32, ctypes.c_double, vp, vp, vp]
    lib.sa_rope_table.restype = ctypes.c_int
    lib.sa_rope_apply.argtypes = [pp, i32, vp, vp, vp, i32, vp, vp]
    lib.sa_rope_apply.restype = ctypes.c_int
    lib.sa_forward_rope.argtypes = [pp] + [vp] * 9 + [vp, sz, vp]
    lib.sa_forward_rope.restype = ctypes.c_int
    lib.sa_swa_gated_forward_rope.argtypes = [pp] + [vp] * 13 + [vp, sz, vp]
    lib.sa_swa_gated_forward_rope.restype = ctypes.c_int
    lib.sa_debug_set.argtypes = [ctypes.c_int, ctypes.c_int]
    lib.sa_debug_set.restype = ctypes.c_int
    lib.sa_debug_wait_timeout.argtypes = [i64, vp]
    lib.sa_debug_wait_timeout.restype = ctypes.c_int
    if path == _build.LIB:
        _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().sa_status_string(int(status)).decode()


def launch_count() -> int:
    return int(load_library().sa_launch_count())


def set_profile_events(start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]):
    """Brackets the SA-branch attention kernel of later forward calls with these events."""
    lib = load_library()
    if start is None or stop is None:
        lib.sa_set_profile_events(None, None)
        return
    # torch creates the underlying cudaEvent lazily, at the first record
    if not start.cuda_event:
        start.record()
    if not stop.cuda_event:
        stop.record()
    lib.sa_set_profile_events(ctypes.c_void_p(start.cuda_event), ctypes.c_void_p(stop.cuda_event))


def debug_set(key: int, value: int):
    """Test hook: selects a kernel variant for later calls (see sa_debug_set in sa.h)."""
    _check(load_library().sa_debug_set(int(key), int(value)), "sa_debug_set")


def debug_wait_timeout(limit_cycles: int):
    """Test hook: one small kernel whose bounded wait runs out after limit_cycles."""
    _check(load_library().sa_debug_wait_timeout(int(limit_cycles), _stream()),
           "sa_debug_wait_timeout")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str):
    if status != SA_OK:
        raise SaError(status, where)


def make_problem(q: torch.Tensor, k: torch.Tensor, w: int, flags: int, scale: float = 0.0,
                 L: int = 0) -> SaProblem:
    """Describes [B,H,n,d] tensors (any strides with d contiguous) to the library."""
    if q.dtype == torch.float32:
        dt = F32
    elif q.dtype == torch.bfloat16:
        dt = BF16
    else:
        raise TypeError("q/k/v must be float32 or bfloat16")
    B, Hq, n, d = q.shape
    p = SaProblem(B=B, Hq=Hq, Hkv=k.shape[1], n=n, d=d, w=int(w), dtype=dt, flags=int(flags),
                  softmax_scale=float(scale), L=int(L))
    if q.stride(3) != 1 or k.stride(3) != 1:
        raise ValueError("the head dimension must be contiguous")
    p.q_stride[:] = [q.stride(0), q.stride(1), q.stride(2)]
    p.kv_stride[:] = [k.stride(0), k.stride(1), k.stride(2)]
    return p


def sa_workspace_bytes(p: SaProblem, op: int) -> int:
    r = int(load_library().sa_workspace_bytes(ctypes.byref(p), int(op)))
    if r == ctypes.c_size_t(-1).value:
        raise SaError(1, "sa_workspace_bytes")
    return r


def _workspace(nbytes: int, device, ws: Optional[torch.Tensor]):
    if ws is not None:
        return ws
    return torch.empty(max(nbytes, 16), dtype=torch.uint8, device=device)


def _same_layout(ref: torch.Tensor, *others):
    for t in others:
        if t is not None and (t.shape != ref.shape or t.stride() != ref.stride()
                              or t.dtype != ref.dtype):
            raise ValueError("tensor does not share the layout of its reference tensor")


def sa_make_perm(seed: int, layer: int, B: int, n: int, device="cuda", perm=None, inv=None,
                 ws=None):
    """One uniform permutation per sequence and its inverse (int32 [B,n] each)."""
    lib = load_library()
    perm = torch.empty(B, n, dtype=torch.int32, device=device) if perm is None else perm
    inv = torch.empty(B, n, dtype=torch.int32, device=device) if inv is None else inv
    p = SaProblem(B=B, n=n)
    nbytes = sa_workspace_bytes(p, OP_MAKE_PERM)
    ws = _workspace(nbytes, perm.device, ws)
    _check(lib.sa_make_perm(int(seed) & (2 ** 64 - 1), int(layer), B, n, _ptr(perm), _ptr(inv),
                            _ptr(ws), ws.numel(), _stream()), "sa_make_perm")
    return perm, inv


STATIC_SCRATCH_BYTES = 4 << 20


def sa_make_perm_static(seed: int, layer: int, B: int, n: int, perm: torch.Tensor,
                        inv: torch.Tensor):
    """sa_make_perm without a workspace, for callers that must not allocate.

    Same permutations as sa_make_perm, bit for bit.  The sort's scratch is a fixed array
    inside the library (STATIC_SCRATCH_BYTES per GPU), so this wrapper creates no tensor: the
    caller hands in both outputs (int32 [B,n], CUDA).  Raises SaError (status 7) when B*n
    needs more scratch than is built in (roughly B*n > 200,000).  Calls that may overlap on
    one GPU race on the shared array: keep them on one stream."""
    lib = load_library()
    for t in (perm, inv):
        if t.dtype != torch.int32 or tuple(t.shape) != (B, n) or not t.is_contiguous():
            raise ValueError("perm and inv must be contiguous int32 [B,n]")
    _check(lib.sa_make_perm_static(int(seed) & (2 ** 64 - 1), int(layer), B, n, _ptr(perm),
                                   _ptr(inv), _stream()), "sa_make_perm_static")
    return perm, inv


def sa_forward(q, k, v, perm, inv, w, flags=CAUSAL, scale=0.0, y=None, want_lse=False,
               lse=None):
    """SA forward; returns y (and lse when asked)."""
    lib = load_library()
    _same_layout(k, v)
    p = make_problem(q, k, w, flags, scale)
    y = torch.empty_like(q) if y is None else y
    _same_layout(q, y)
    if want_lse and lse is None:
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
    _check(lib.sa_forward(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(perm), _ptr(inv),
                          _ptr(y), _ptr(lse), None, 0, _stream()), "sa_forward")
    return (y, lse) if (want_lse or lse is not None) else y


def sa_swa_forward(q, k, v, w, flags=CAUSAL | SWA_ONE_SIDED, scale=0.0, y=None, want_lse=False,
                   lse=None):
    """Plain sliding-window attention forward in the original order."""
    lib = load_library()
    _same_layout(k, v)
    p = make_problem(q, k, w, flags, scale)
    y = torch.empty_like(q) if y is None else y
    _same_layout(q, y)
    if want_lse and lse is None:
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
    _check(lib.sa_swa_forward(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(y), _ptr(lse),
                              None, 0, _stream()), "sa_swa_forward")
    return (y, lse) if (want_lse or lse is not None) else y


def sa_rope_table(n: int, d: int, base: float = 10000.0, device="cuda"):
    """cos and sin of the rotary angles t * base^(-2c/d): fp32 [n, d/2] each."""
    cs = torch.empty(n, d // 2, dtype=torch.float32, device=device)
    sn = torch.empty_like(cs)
    _check(load_library().sa_rope_table(n, d, float(base), _ptr(cs), _ptr(sn), _stream()),
           "sa_rope_table")
    return cs, sn


def sa_rope_apply(x, k_like, rope_cos, rope_sin, w=1, inverse=False, out=None, kv=False):
    """Rotates x ([B,H,n,d]) by its tokens' original positions; ``k_like`` is any tensor with the
    KV layout (only needed to describe the problem when x is a query-side tensor)."""
    q_like = k_like if kv else x
    kv_like = x if kv else k_like
    p = make_problem(q_like, kv_like, w, CAUSAL)
    out = torch.empty_like(x) if out is None else out
    _same_layout(x, out)
    _check(load_library().sa_rope_apply(ctypes.byref(p), 1 if kv else 0, _ptr(x), _ptr(rope_cos),
                                        _ptr(rope_sin), 1 if inverse else 0, _ptr(out), _stream()),
           "sa_rope_apply")
    return out


def sa_forward_rope(q, k, v, perm, inv, rope_cos, rope_sin, w, flags=CAUSAL, scale=0.0, y=None,
                    want_lse=False):
    """SA forward on Q and K rotated by their original positions (rotation inside the gather
    where the tensor-core kernels apply, a rotated copy in a workspace otherwise)."""
    lib = load_library()
    _same_layout(k, v)
    p = make_problem(q, k, w, flags, scale)
    y = torch.empty_like(q) if y is None else y
    _same_layout(q, y)
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device) if want_lse else None
    ws = _workspace(sa_workspace_bytes(p, OP_FORWARD_ROPE), q.device, None)
    _check(lib.sa_forward_rope(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(perm), _ptr(inv),
                               _ptr(rope_cos), _ptr(rope_sin), _ptr(y), _ptr(lse), _ptr(ws),
                               ws.numel(), _stream()), "sa_forward_rope")
    return (y, lse) if want_lse else y


def sa_swa_gated_forward_rope(q, k, v, perm, inv, rope_cos, rope_sin, gate_logits, w,
                              flags=CAUSAL | SWA_ONE_SIDED, scale=0.0, save_for_bwd=False):
    """Gated SA + SWA forward on rotated Q and K.  Returns y, or the five saved tensors."""
    lib = load_library()
    _same_layout(k, v)
    out = {}
    if save_for_bwd:
        flags |= SAVE_FOR_BWD
        for name in ("y_sa", "y_swa"):
            out[name] = torch.empty_like(q)
        for name in ("lse_sa", "lse_swa"):
            out[name] = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
    y = torch.empty_like(q)
    p = make_problem(q, k, w, flags, scale)
    ws = _workspace(sa_workspace_bytes(p, OP_FORWARD_ROPE), q.device, None)
    _check(lib.sa_swa_gated_forward_rope(
        ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(perm), _ptr(inv), _ptr(rope_cos),
        _ptr(rope_sin), _ptr(gate_logits), _ptr(y), _ptr(out.get("y_sa")), _ptr(out.get("y_swa")),
        _ptr(out.get("lse_sa")), _ptr(out.get("lse_swa")), _ptr(ws), ws.numel(), _stream()),
        "sa_swa_gated_forward_rope")
    if save_for_bwd:
        return y, out["y_sa"], out["y_swa"], out["lse_sa"], out["lse_swa"]
    return y


def sa_swa_gated_forward(q, k, v, perm, inv, gate_logits, w, flags=CAUSAL | SWA_ONE_SIDED,
                         scale=0.0, save_for_bwd=False, out=None, ws=None, fused_epilogue=False):
    """Gated SA + SWA forward.  Returns y, or (y, y_sa, y_swa, lse_sa, lse_swa) when saving.

    ``out`` may hold preallocated tensors under the keys y, y_sa, y_swa, lse_sa, lse_swa.
    ``ws``: optional scratch (uint8, OP_GATED_FORWARD_SCRATCH bytes) for the SA branch's rows
    when neither branch output is kept: the local branch's launch then combines with its idle
    warps instead of in the row threads' epilogue.  ``fused_epilogue=True`` drops a given
    ``ws``.  Two launches either way."""
    lib = load_library()
    _same_layout(k, v)
    out = dict(out or {})
    if save_for_bwd:
        flags |= SAVE_FOR_BWD
        for name in ("y_sa", "y_swa"):
            out.setdefault(name, torch.empty_like(q))
        for name in ("lse_sa", "lse_swa"):
            out.setdefault(name, torch.empty(q.shape[:3], dtype=torch.float32, device=q.device))
    y = out.setdefault("y", torch.empty_like(q))
    _same_layout(q, y, out.get("y_sa"), out.get("y_swa"))
    p = make_problem(q, k, w, flags, scale)
    if fused_epilogue:
        ws = None
    _check(lib.sa_swa_gated_forward(
        ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(perm), _ptr(inv), _ptr(gate_logits),
        _ptr(y), _ptr(out.get("y_sa")), _ptr(out.get("y_swa")), _ptr(out.get("lse_sa")),
        _ptr(out.get("lse_swa")), _ptr(ws), 0 if ws is None else ws.numel(), _stream()),
        "sa_swa_gated_forward")
    if save_for_bwd:
        return y, out["y_sa"], out["y_swa"], out["lse_sa"], out["lse_swa"]
    return y


def sa_backward(q, k, v, perm, inv, gate_logits, y_sa, y_swa, lse_sa, lse_swa, dy, w,
                flags=CAUSAL | SWA_ONE_SIDED, scale=0.0, ws=None, out=None):
    """Backward of the (gated) forward.  Returns (dq, dk, dv, dgate_logits or None)."""
    lib = load_library()
    _same_layout(k, v)
    _same_layout(q, dy, y_sa, y_swa)
    out = dict(out or {})
    dq = out.setdefault("dq", torch.empty_like(q))
    dk = out.setdefault("dk", torch.empty_like(k))
    dv = out.setdefault("dv", torch.empty_like(v))
    _same_layout(q, dq)
    _same_layout(k, dk, dv)
    dgate = None
    if gate_logits is not None:
        dgate = out.setdefault("dgate", torch.empty(2, q.shape[1], dtype=torch.float32,
                                                    device=q.device))
    p = make_problem(q, k, w, flags, scale)
    ws = _workspace(sa_workspace_bytes(p, OP_BACKWARD), q.device, ws)
    _check(lib.sa_backward(
        ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(perm), _ptr(inv), _ptr(gate_logits),
        _ptr(y_sa), _ptr(y_swa), _ptr(lse_sa), _ptr(lse_swa), _ptr(dy), _ptr(dq), _ptr(dk),
        _ptr(dv), _ptr(dgate), _ptr(ws), ws.numel(), _stream()), "sa_backward")
    return dq, dk, dv, dgate


def sa_coverage(perm, inv, w, flags, src, want_row_count=True, ws=None):
    """Mask row counts, their totals, and reachable-set sizes over the L layers of perm [L,n]."""
    lib = load_library()
    L, n = perm.shape
    dev = perm.device
    nnz = torch.empty(L, dtype=torch.int64, device=dev)
    reach = torch.empty(L, dtype=torch.int32, device=dev)
    rc = torch.empty(L, n, dtype=torch.int32, device=dev) if want_row_count else None
    p = SaProblem(n=n, L=L)
    ws = _workspace(sa_workspace_bytes(p, OP_COVERAGE), dev, ws)
    _check(lib.sa_coverage(L, n, int(w), int(flags), _ptr(perm), _ptr(inv), int(src), _ptr(nnz),
                           _ptr(rc), _ptr(reach), _ptr(ws), ws.numel(), _stream()),
           "sa_coverage")
    return nnz, rc, reach


def sa_gate_projection_forward(y_sa, w_sa, y_swa=None, w_swa=None, out=None):
    """out = sigmoid(y_sa w_sa^T) * y_sa (+ sigmoid(y_swa w_swa^T) * y_swa): Eq. 5-6.

    y_*: [rows, dm] with unit stride along dm (any row pitch, e.g. a [B*n, Hq*d] view of a
    [B,n,Hq,d] attention output); w_*: contiguous [dm, dm] (out_features x in_features)."""
    lib = load_library()
    rows, dm = y_sa.shape
    if y_sa.dtype == torch.float32:
        dt = 0
    elif y_sa.dtype == torch.bfloat16:
        dt = 1
    else:
        raise ValueError("dtype must be float32 or bfloat16")
    for t in (y_sa, y_swa):
        if t is not None and (t.dim() != 2 or t.stride(1) != 1 or t.shape != y_sa.shape
                              or t.stride(0) != y_sa.stride(0) or t.dtype != y_sa.dtype):
            raise ValueError("y tensors must be [rows, dm] with unit inner stride and one pitch")
    for t in (w_sa, w_swa):
        if t is not None and (tuple(t.shape) != (dm, dm) or not t.is_contiguous()
                              or t.dtype != y_sa.dtype):
            raise ValueError("w tensors must be contiguous [dm, dm] of the run dtype")
    if out is None:
        out = torch.empty(rows, dm, dtype=y_sa.dtype, device=y_sa.device)
    if out.stride(1) != 1 or tuple(out.shape) != (rows, dm) or out.dtype != y_sa.dtype:
        raise ValueError("out must be [rows, dm] with unit inner stride")
    _check(lib.sa_gate_projection_forward(rows, dm, dt, _ptr(y_sa), _ptr(y_swa), y_sa.stride(0),
                                          _ptr(w_sa), _ptr(w_swa), _ptr(out), out.stride(0),
                                          _stream()), "sa_gate_projection_forward")
    return out


def sa_gate_projection_backward(dout, y_sa, w_sa, y_swa=None, w_swa=None, ws=None):
    """Gradients of sa_gate_projection_forward: (dy_sa, dw_sa) or, for the dual path,
    (dy_sa, dw_sa, dy_swa, dw_swa).  Tensors as in the forward; dout: [rows, dm]."""
    lib = load_library()
    rows, dm = y_sa.shape
    dt = {torch.float32: 0, torch.bfloat16: 1}.get(y_sa.dtype)
    if dt is None:
        raise ValueError("dtype must be float32 or bfloat16")
    for t in (dout, y_sa, y_swa):
        if t is not None and (t.dim() != 2 or t.stride(1) != 1 or t.shape != y_sa.shape
                              or t.dtype != y_sa.dtype):
            raise ValueError("dout and y tensors must be [rows, dm] with unit inner stride")
    if y_swa is not None and y_swa.stride(0) != y_sa.stride(0):
        raise ValueError("y_sa and y_swa must share one row pitch")
    for t in (w_sa, w_swa):
        if t is not None and (tuple(t.shape) != (dm, dm) or not t.is_contiguous()
                              or t.dtype != y_sa.dtype):
            raise ValueError("w tensors must be contiguous [dm, dm] of the run dtype")
    dual = y_swa is not None
    dy_sa, dw_sa = torch.empty_like(y_sa, memory_format=torch.contiguous_format), torch.empty_like(w_sa)
    dy_swa = torch.empty_like(dy_sa) if dual else None
    dw_swa = torch.empty_like(w_sa) if dual else None
    ws = _workspace(int(lib.sa_gate_projection_backward_ws_bytes(rows, dm)), y_sa.device, ws)
    _check(lib.sa_gate_projection_backward(
        rows, dm, dt, _ptr(dout), dout.stride(0), _ptr(y_sa), _ptr(y_swa), y_sa.stride(0),
        _ptr(w_sa), _ptr(w_swa), _ptr(dy_sa), _ptr(dy_swa), dy_sa.stride(0), _ptr(dw_sa),
        _ptr(dw_swa), _ptr(ws), ws.numel(), _stream()), "sa_gate_projection_backward")
    return (dy_sa, dw_sa, dy_swa, dw_swa) if dual else (dy_sa, dw_sa)


def host_forward_plan(Hq: int, Hkv: int, n_groups: int, q_parts: int):
    """Head ranges of the host-memory forward: (kv_begin, kv_end, q_begin, q_end, carries_kv)."""
    buf = (ctypes.c_int32 * (5 * 256))()
    cnt = int(load_library().sa_host_forward_plan(Hq, Hkv, n_groups, q_parts, buf, 256))
    if cnt < 0:
        raise ValueError("Hq must be a positive multiple of Hkv")
    return [tuple(buf[5 * i + j] for j in range(4)) + (bool(buf[5 * i + 4]),) for i in range(cnt)]


def host_forward_ws_bytes(B, Hq, Hkv, n, d, dtype=BF16) -> int:
    p = SaProblem(B=B, Hq=Hq, Hkv=Hkv, n=n, d=d, w=1, dtype=dtype)
    r = int(load_library().sa_host_forward_ws_bytes(ctypes.byref(p)))
    if r == ctypes.c_size_t(-1).value:
        raise SaError(1, "sa_host_forward_ws_bytes")
    return r


def sa_swa_gated_forward_host(q, k, v, gate_logits, y, w, flags, seed, layer, ws, n_groups=8,
                              q_parts=2, scale=0.0):
    """Fresh permutation + gated SA+SWA forward on HOST tensors (contiguous [B,H,n,d], pinned
    for overlap); ws: CUDA uint8 tensor of host_forward_ws_bytes(...).  y (host) is complete
    once the current stream has been synchronised."""
    for t in (q, k, v, y, gate_logits):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("host tensors must be contiguous CPU tensors")
    dt = {torch.float32: F32, torch.bfloat16: BF16}[q.dtype]
    B, Hq, n, d = q.shape
    p = SaProblem(B=B, Hq=Hq, Hkv=k.shape[1], n=n, d=d, w=int(w), dtype=dt, flags=int(flags),
                  softmax_scale=float(scale))
    _check(load_library().sa_swa_gated_forward_host(
        ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(gate_logits), _ptr(y),
        int(seed) & (2 ** 64 - 1), int(layer), int(n_groups), int(q_parts), _ptr(ws), ws.numel(),
        _stream()), "sa_swa_gated_forward_host")
    return y


def sa_read_status() -> int:
    """Synchronises the current stream and returns (and clears) the device status word."""
    return int(load_library().sa_read_status(_stream()))
