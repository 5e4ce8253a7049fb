"""Float64 CPU oracle for Stochastic Attention -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end of ``sa_oracle.c`` (plain C, float64, OpenMP over rows).
Nothing in the CUDA library imports this package and this package imports nothing
of the CUDA library; only the tests, the smoke check and the benchmark's CPU
baseline leg may use it.  Each wrapper names the passage of the paper its C
function follows; the arithmetic itself lives in the C file.

Conventions: every tensor is a contiguous float64 numpy array, q/y/dq of shape
[B,Hq,n,d], k/v/dk/dv [B,Hkv,n,d], perm/inv int32 [B,n], lse [B,Hq,n], all in
ORIGINAL token order.  perm[b,p] is the token in slot p, inv[b,i] the slot of
token i (the paper's sigma(i) of Eq. 3).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

CAUSAL = 1
LINEAR_WINDOW = 2
SWA_ONE_SIDED = 4

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sa_oracle.c")
_LIB = os.path.join(_HERE, "libsa_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile sa_oracle.c with gcc (no fast-math: sums run in the written order)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_sort_key.restype = ctypes.c_uint64
        lib.oracle_sort_key.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32,
                                        ctypes.c_uint32]
        lib.oracle_visible.restype = ctypes.c_int
        lib.oracle_swa_visible.restype = ctypes.c_int
        _lib = lib
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops will use (what the CPU-baseline timing reports)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


def _f64(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(ctypes.c_void_p)


def _i32(a):
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(ctypes.c_void_p)


def _scale(d, scale):
    return float(scale) if scale else 1.0 / float(np.sqrt(d))


def philox4x32_10(ctr, key):
    """Philox4x32 with 10 rounds (Salmon et al., SC'11): 4-word counter, 2-word key."""
    c = (ctypes.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    out = (ctypes.c_uint32 * 4)()
    _load().oracle_philox4x32_10(c, k, out)
    return [int(x) for x in out]


def sort_key(seed, layer, b, i) -> int:
    """64-bit sort key of token i in sequence b at a layer (permutation recipe)."""
    return int(_load().oracle_sort_key(int(seed), int(layer), int(b), int(i)))


def make_perm(seed, layer, B, n):
    """Alg. 1 line 1: one uniform permutation per sequence; returns (perm, inv)."""
    perm = np.empty((B, n), np.int32)
    inv = np.empty((B, n), np.int32)
    _load().oracle_make_perm(ctypes.c_uint64(int(seed)), ctypes.c_uint32(int(layer)),
                             ctypes.c_int32(B), ctypes.c_int32(n),
                             perm.ctypes.data_as(ctypes.c_void_p),
                             inv.ctypes.data_as(ctypes.c_void_p))
    return perm, inv


def visible(n, w, flags, inv, i, j) -> bool:
    """Eq. 3 window in shuffled space (+ App. B causal rule); inv = one sequence or None."""
    a, p = _i32(inv)
    return bool(_load().oracle_visible(ctypes.c_int32(n), ctypes.c_int32(w),
                                       ctypes.c_uint32(flags), p, ctypes.c_int32(i),
                                       ctypes.c_int32(j)))


def swa_visible(n, w, flags, i, j) -> bool:
    """Plain-SWA predicate (Sec. 3.1 and its footnote)."""
    return bool(_load().oracle_swa_visible(ctypes.c_int32(n), ctypes.c_int32(w),
                                           ctypes.c_uint32(flags), ctypes.c_int32(i),
                                           ctypes.c_int32(j)))


def _forward(fn, swa, q, k, v, perm, inv, w, flags, scale):
    q, qp = _f64(q)
    k, kp = _f64(k)
    v, vp = _f64(v)
    B, Hq, n, d = q.shape
    Hkv = k.shape[1]
    assert k.shape == (B, Hkv, n, d) and v.shape == k.shape and Hq % Hkv == 0
    perm, pp = _i32(perm)
    inv, ip = _i32(inv)
    y = np.empty_like(q)
    lse = np.empty((B, Hq, n), np.float64)
    fn(ctypes.c_int32(int(swa)), ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(Hkv),
       ctypes.c_int32(n), ctypes.c_int32(d), ctypes.c_int32(w), ctypes.c_uint32(flags),
       ctypes.c_double(_scale(d, scale)), qp, kp, vp, pp, ip,
       y.ctypes.data_as(ctypes.c_void_p), lse.ctypes.data_as(ctypes.c_void_p))
    return y, lse


def sa_forward(q, k, v, perm, inv, w, flags=CAUSAL, scale=0.0):
    """SA forward: Eq. 1 on the neighbourhood of Eq. 3 (== Alg. 1 == Eq. 4)."""
    return _forward(_load().oracle_forward, 0, q, k, v, perm, inv, w, flags, scale)


def swa_forward(q, k, v, w, flags=CAUSAL, scale=0.0):
    """Plain SWA forward (Eq. 1) in the original order."""
    return _forward(_load().oracle_forward, 1, q, k, v, None, None, w, flags, scale)


def sa_forward_dense(q, k, v, perm, inv, w, flags=CAUSAL, scale=0.0):
    """Eq. 4 literally: all n*n pairs tested against the mask (small n only)."""
    return _forward(_load().oracle_forward_dense, 0, q, k, v, perm, inv, w, flags, scale)


def swa_forward_dense(q, k, v, w, flags=CAUSAL, scale=0.0):
    return _forward(_load().oracle_forward_dense, 1, q, k, v, None, None, w, flags, scale)


def gated_forward(q, k, v, perm, inv, gate_logits, w, flags=CAUSAL | SWA_ONE_SIDED, scale=0.0):
    """Eq. 5 with per-head scalar gate logits [2,Hq] (row 0 SA, row 1 SWA).

    Returns (y, y_sa, y_swa, lse_sa, lse_swa)."""
    q, qp = _f64(q)
    k, kp = _f64(k)
    v, vp = _f64(v)
    B, Hq, n, d = q.shape
    Hkv = k.shape[1]
    perm, pp = _i32(perm)
    inv, ip = _i32(inv)
    g, gp = _f64(gate_logits)
    assert g.shape == (2, Hq)
    y, y_sa, y_swa = np.empty_like(q), np.empty_like(q), np.empty_like(q)
    lse_sa = np.empty((B, Hq, n), np.float64)
    lse_swa = np.empty((B, Hq, n), np.float64)
    _load().oracle_gated_forward(
        ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(n),
        ctypes.c_int32(d), ctypes.c_int32(w), ctypes.c_uint32(flags),
        ctypes.c_double(_scale(d, scale)), qp, kp, vp, pp, ip, gp,
        *[a.ctypes.data_as(ctypes.c_void_p) for a in (y, y_sa, y_swa, lse_sa, lse_swa)])
    return y, y_sa, y_swa, lse_sa, lse_swa


def backward(q, k, v, perm, inv, gate_logits, dy, w, flags=CAUSAL | SWA_ONE_SIDED, scale=0.0):
    """Gradients of sum(dy*y): (dq, dk, dv, dgate_logits or None).

    gate_logits None => ungated SA only.  Textbook softmax-attention derivative;
    the forward is recomputed in float64 inside."""
    q, qp = _f64(q)
    k, kp = _f64(k)
    v, vp = _f64(v)
    dy, dyp = _f64(dy)
    B, Hq, n, d = q.shape
    Hkv = k.shape[1]
    perm, pp = _i32(perm)
    inv, ip = _i32(inv)
    if gate_logits is None:
        g, gp, dg, dgp = None, None, None, None
    else:
        g, gp = _f64(gate_logits)
        dg = np.zeros((2, Hq), np.float64)
        dgp = dg.ctypes.data_as(ctypes.c_void_p)
    dq = np.empty_like(q)
    dk = np.empty_like(k)
    dv = np.empty_like(v)
    _load().oracle_backward(
        ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(n),
        ctypes.c_int32(d), ctypes.c_int32(w), ctypes.c_uint32(flags),
        ctypes.c_double(_scale(d, scale)), qp, kp, vp, pp, ip, gp, dyp,
        dq.ctypes.data_as(ctypes.c_void_p), dk.ctypes.data_as(ctypes.c_void_p),
        dv.ctypes.data_as(ctypes.c_void_p), dgp)
    return dq, dk, dv, dg


def coverage(perm, inv, w, flags, src):
    """Mask row counts and the reachable-set sizes of Prop. 2 over L layers.

    perm/inv int32 [L,n] (inv None => identity at every layer, needs n via perm shape).
    Returns (nnz int64 [L], row_count int32 [L,n], reach int32 [L])."""
    perm, pp = _i32(perm)
    L, n = perm.shape
    inv, ip = _i32(inv)
    nnz = np.zeros(L, np.int64)
    row_count = np.zeros((L, n), np.int32)
    reach = np.zeros(L, np.int32)
    _load().oracle_coverage(ctypes.c_int32(L), ctypes.c_int32(n), ctypes.c_int32(w),
                            ctypes.c_uint32(flags), pp, ip, ctypes.c_int32(src),
                            nnz.ctypes.data_as(ctypes.c_void_p),
                            row_count.ctypes.data_as(ctypes.c_void_p),
                            reach.ctypes.data_as(ctypes.c_void_p))
    return nnz, row_count, reach


def forward_rows(swa, q, k, v, perm, inv, w, flags, rows, scale=0.0):
    """Eq. 1 for selected rows only; rows = flat (b*Hq+hq)*n+i indices.  Returns (y_rows, lse_rows)."""
    q, qp = _f64(q)
    k, kp = _f64(k)
    v, vp = _f64(v)
    B, Hq, n, d = q.shape
    Hkv = k.shape[1]
    perm, pp = _i32(None if swa else perm)
    inv, ip = _i32(None if swa else inv)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    y = np.empty((rows.size, d), np.float64)
    lse = np.empty(rows.size, np.float64)
    _load().oracle_forward_rows(
        ctypes.c_int32(int(swa)), ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(Hkv),
        ctypes.c_int32(n), ctypes.c_int32(d), ctypes.c_int32(w), ctypes.c_uint32(flags),
        ctypes.c_double(_scale(d, scale)), qp, kp, vp, pp, ip, ctypes.c_int64(rows.size),
        rows.ctypes.data_as(ctypes.c_void_p), y.ctypes.data_as(ctypes.c_void_p),
        lse.ctypes.data_as(ctypes.c_void_p))
    return y, lse


def backward_rows(q, k, v, perm, inv, gate_logits, dy, w, flags, q_rows, kv_rows, scale=0.0):
    """Selected rows of the gradients of sum(dy*y) (same derivative as ``backward``).

    q_rows: flat (b*Hq+hq)*n+i indices -> dq rows; kv_rows: flat (b*Hkv+hk)*n+j indices ->
    dk and dv rows (summed over the group's query heads, the branches and every query that
    sees the key).  gate_logits None => ungated SA only.  Returns (dq_rows, dk_rows, dv_rows)."""
    q, qp = _f64(q)
    k, kp = _f64(k)
    v, vp = _f64(v)
    dy, dyp = _f64(dy)
    B, Hq, n, d = q.shape
    Hkv = k.shape[1]
    perm, pp = _i32(perm)
    inv, ip = _i32(inv)
    g, gp = (None, None) if gate_logits is None else _f64(gate_logits)
    q_rows = np.ascontiguousarray(q_rows, dtype=np.int64)
    kv_rows = np.ascontiguousarray(kv_rows, dtype=np.int64)
    dq = np.empty((q_rows.size, d), np.float64)
    dk = np.empty((kv_rows.size, d), np.float64)
    dv = np.empty((kv_rows.size, d), np.float64)
    _load().oracle_backward_rows(
        ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(n),
        ctypes.c_int32(d), ctypes.c_int32(w), ctypes.c_uint32(flags),
        ctypes.c_double(_scale(d, scale)), qp, kp, vp, pp, ip, gp, dyp,
        ctypes.c_int64(q_rows.size), q_rows.ctypes.data_as(ctypes.c_void_p),
        dq.ctypes.data_as(ctypes.c_void_p),
        ctypes.c_int64(kv_rows.size), kv_rows.ctypes.data_as(ctypes.c_void_p),
        dk.ctypes.data_as(ctypes.c_void_p), dv.ctypes.data_as(ctypes.c_void_p))
    return dq, dk, dv


def rope(x, positions, base=10000.0, inverse=False):
    """Rotary position embedding (Su et al.) of the last dimension of x, as the paper applies it
    to Q and K BEFORE the shuffle, i.e. with each token's ORIGINAL position (Sec. 4.2 and the
    attention paragraph of App. B).

    x: [..., n, d] with d even; positions: [n] (the original token indices).  Dimension c of
    the first half is paired with dimension c + d/2 (the half-split layout of the Qwen3 /
    Llama family the paper retrofits; the adjacent-pair layout of the original formulation
    differs only by a fixed permutation of the head dimensions).  The pair (x1, x2) of token
    t is rotated by the angle positions[t] * base**(-2c/d):
        out1 = x1 cos - x2 sin,   out2 = x2 cos + x1 sin.
    inverse=True rotates by the opposite angle (the transpose: what maps a gradient with respect
    to the rotated tensor back to the unrotated one).  Plain float64 numpy."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    if d % 2:
        raise ValueError("the head dimension must be even")
    half = d // 2
    pos = np.asarray(positions, dtype=np.float64)
    if pos.shape != (x.shape[-2],):
        raise ValueError("one position per token")
    inv_freq = np.asarray(base, dtype=np.float64) ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = pos[:, None] * inv_freq[None, :]
    c, s = np.cos(ang), np.sin(ang)
    if inverse:
        s = -s
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def gate_projection(y_sa, w_sa, y_swa=None, w_swa=None):
    """Projection gates of Eq. 5-6 (App. B, dual-path and single-path attention gate).

    y_*: [rows, dm] attention outputs with the heads concatenated per token; w_*: [dm, dm]
    weights of a bias-free linear layer (out_features x in_features), so the gate of a path is
    g = sigmoid(y w^T), per token and per dimension, and the result is
    g_sa * y_sa (+ g_swa * y_swa for the dual path).  Plain float64 numpy: one matmul, one
    logistic and one product per path, nothing blocked or fused."""
    def one(y, w):
        y = np.asarray(y, dtype=np.float64)
        w = np.asarray(w, dtype=np.float64)
        if y.ndim != 2 or w.shape != (y.shape[1], y.shape[1]):
            raise ValueError("y must be [rows, dm] and w [dm, dm]")
        g = 1.0 / (1.0 + np.exp(-(y @ w.T)))
        return g * y
    out = one(y_sa, w_sa)
    if y_swa is not None:
        out = out + one(y_swa, w_swa)
    return out


def gate_projection_backward(dout, y_sa, w_sa, y_swa=None, w_swa=None):
    """Derivative of gate_projection (Eq. 5-6) with respect to its inputs and weights.

    With z = y w^T and g = sigmoid(z), out = g * y per path, so for an upstream gradient dout
        dz = dout * y * g * (1 - g),   dw = dz^T y,   dy = dout * g + dz w.
    Returns (dy_sa, dw_sa) for the single path, (dy_sa, dw_sa, dy_swa, dw_swa) for the dual
    path (the paths only share dout).  Plain float64 numpy."""
    dout = np.asarray(dout, dtype=np.float64)

    def one(y, w):
        y = np.asarray(y, dtype=np.float64)
        w = np.asarray(w, dtype=np.float64)
        if y.ndim != 2 or w.shape != (y.shape[1], y.shape[1]) or dout.shape != y.shape:
            raise ValueError("y and dout must be [rows, dm] and w [dm, dm]")
        g = 1.0 / (1.0 + np.exp(-(y @ w.T)))
        dz = dout * y * g * (1.0 - g)
        return dout * g + dz @ w, dz.T @ y
    res = one(y_sa, w_sa)
    if y_swa is not None:
        res = res + one(y_swa, w_swa)
    return res
