"""GPU parity: every entry point of the C ABI against the float64 CPU oracle on the
same seeded inputs.  Integers bit-exact; fp32 outputs within 1e-4 max-abs; bf16 outputs
within 2e-2 of the reference tensor's largest magnitude (max|y-ref| / max|ref|)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_00754_b200 import binding as sa
from paper_2604_00754_b200 import workloads as wl
from paper_2604_00754_b200.workloads import CAUSAL, LINEAR_WINDOW, SWA_ONE_SIDED, as_f64

pytestmark = pytest.mark.gpu

F32_ATOL = 1e-4
BF16_REL = 2e-2


def close(got: torch.Tensor, ref: np.ndarray, dtype, what=""):
    g = as_f64(got)
    err = np.abs(g - ref).max()
    if dtype == torch.float32:
        assert err <= F32_ATOL, "%s max-abs %.3e" % (what, err)
    else:
        # 1e-5 floor: a reference that is identically zero (w = 1 gives dq = dk = 0) still
        # meets bf16 roundings of cancelling terms
        assert err <= BF16_REL * np.abs(ref).max() + 1e-5, \
            "%s rel %.3e" % (what, err / max(np.abs(ref).max(), 1e-30))
    return err


def draw(shape_q, shape_k, dtype, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    mk = lambda s: (torch.randn(*s, generator=g) * scale).to(dtype)
    return mk(shape_q), mk(shape_k), mk(shape_k)


def perms(seed, layer, B, n):
    perm, inv = sa.sa_make_perm(seed, layer, B, n)
    return perm, inv, perm.cpu().numpy(), inv.cpu().numpy()


# ------------------------------------------------------------------ permutation

@pytest.mark.parametrize("B,n", [(1, 1), (3, 2), (2, 27), (1, 255), (2, 256), (3, 2049),
                                 (8, 4096), (1, 32768), (2, 100000), (1, 131072)])
def test_make_perm_bit_exact(B, n):
    for seed, layer in [(0, 0), (0xDEADBEEFCAFEF00D, 47)]:
        perm, inv = sa.sa_make_perm(seed, layer, B, n)
        operm, oinv = oracle.make_perm(seed, layer, B, n)
        assert np.array_equal(perm.cpu().numpy(), operm)
        assert np.array_equal(inv.cpu().numpy(), oinv)
    assert sa.sa_read_status() == 0


def test_make_perm_is_deterministic_run_to_run():
    # equal 64-bit Philox keys cannot be forced through the public call, so the tie-break of
    # the ranking step is not reachable here; what is checked is run-to-run determinism
    a, _ = sa.sa_make_perm(5, 1, 4, 5000)
    b, _ = sa.sa_make_perm(5, 1, 4, 5000)
    assert torch.equal(a, b)


# ---------------------------------------------------------------------- forward

SMALL = [
    # B, Hq, Hkv, n, d, w, flags
    (1, 1, 1, 1, 8, 1, CAUSAL),
    (1, 1, 1, 27, 64, 8, CAUSAL),                       # Fig. 3 shape
    (2, 4, 2, 300, 64, 33, CAUSAL),
    (2, 4, 2, 300, 64, 33, 0),
    (1, 2, 1, 257, 128, 64, CAUSAL | LINEAR_WINDOW),
    (1, 2, 2, 130, 32, 1, CAUSAL),
    (1, 2, 2, 96, 128, 500, CAUSAL),                    # w > n: every causal key
    (1, 2, 2, 96, 128, 96, 0),                          # w == n even: antipode excluded
    (1, 6, 2, 511, 128, 129, CAUSAL),
    (1, 1, 1, 700, 256, 40, 0),
    (1, 3, 3, 64, 8, 5, LINEAR_WINDOW),
    (2, 3, 3, 1000, 64, 300, CAUSAL),                   # odd group size: two slot tiles per item
    (1, 8, 2, 1153, 64, 128, CAUSAL),                   # w = tile width, ragged tail, GQA
    (1, 4, 4, 640, 128, 1, 0),                          # w = 1 on the tensor-core path
    (1, 2, 1, 900, 128, 257, LINEAR_WINDOW),
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B,Hq,Hkv,n,d,w,flags", SMALL)
def test_sa_forward_small(B, Hq, Hkv, n, d, w, flags, dtype):
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), dtype, seed=n + w)
    perm, inv, permc, invc = perms(n, w, B, n)
    y, lse = sa.sa_forward(q.cuda(), k.cuda(), v.cuda(), perm, inv, w, flags, want_lse=True)
    ry, rlse = oracle.sa_forward(as_f64(q), as_f64(k), as_f64(v), permc, invc, w, flags)
    close(y, ry, dtype, "y")
    assert np.abs(as_f64(lse) - rlse).max() <= (1e-4 if dtype == torch.float32 else 2e-2)
    assert sa.sa_read_status() == 0


SWA_SMALL = [
    (2, 4, 2, 300, 64, 33, CAUSAL | SWA_ONE_SIDED),
    (1, 2, 1, 257, 128, 64, CAUSAL | SWA_ONE_SIDED),
    (1, 2, 2, 96, 128, 500, CAUSAL | SWA_ONE_SIDED),
    (1, 2, 2, 130, 64, 1, CAUSAL | SWA_ONE_SIDED),
    (2, 4, 2, 300, 64, 33, CAUSAL),
    (2, 4, 2, 300, 64, 33, 0),
    (1, 1, 1, 200, 128, 31, LINEAR_WINDOW),
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B,Hq,Hkv,n,d,w,flags", SWA_SMALL)
def test_swa_forward_small(B, Hq, Hkv, n, d, w, flags, dtype):
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), dtype, seed=3 * n + w)
    y, lse = sa.sa_swa_forward(q.cuda(), k.cuda(), v.cuda(), w, flags, want_lse=True)
    ry, rlse = oracle.swa_forward(as_f64(q), as_f64(k), as_f64(v), w, flags)
    close(y, ry, dtype, "y")
    assert np.abs(as_f64(lse) - rlse).max() <= (1e-4 if dtype == torch.float32 else 2e-2)


@pytest.fixture
def debug_option():
    """Sets a test hook of the library for one test and restores the default afterwards."""
    defaults = {sa.DEBUG_SCORE_BLOCK: 0, sa.DEBUG_SWA_TILE_LOADS: 1, sa.DEBUG_TENSOR_CORES: 1,
                sa.DEBUG_GATE_WIDE_TILES: 1}
    touched = []

    def set_(key, value):
        touched.append(key)
        sa.debug_set(key, value)
    yield set_
    for key in touched:
        sa.debug_set(key, defaults[key])


@pytest.mark.parametrize("block", [64, 128])
def test_both_score_block_widths(block, debug_option):
    # the tensor-core kernels have a 64-key and a 128-key score block; the library picks by w,
    # the test hook forces each in turn on the same cases (bf16 only: fp32 never runs them)
    debug_option(sa.DEBUG_SCORE_BLOCK, block)
    bf = torch.bfloat16
    for case in SMALL:
        test_sa_forward_small(*case, bf)
    for case in SWA_SMALL:
        test_swa_forward_small(*case, bf)
    for save in (False, True):
        test_gated_forward_small(bf, save)
    for case in BWD_SMALL:
        for gated in (False, True):
            test_backward_small(*case, gated, bf)


def test_swa_branch_without_tma_tile_loads(debug_option):
    # the one-sided SWA branch loads whole tiles by TMA when its tensors are plain row
    # matrices; with the hook off it gathers rows with cp.async like the SA branch
    debug_option(sa.DEBUG_SWA_TILE_LOADS, 0)
    bf = torch.bfloat16
    for case in SWA_SMALL:
        test_swa_forward_small(*case, bf)
    for save in (False, True):
        test_gated_forward_small(bf, save)
    for fused in (False, True):
        for token_major in (False, True):
            test_gated_forward_both_combine_paths(bf, fused, token_major)
    # the backward of the local branch loads its tiles the same two ways
    for case in BWD_SMALL:
        if case[6] & SWA_ONE_SIDED:
            test_backward_small(*case, True, bf)


def test_backward_swa_tiles_past_the_sequence_read_zeros():
    """Gated backward on views of longer buffers whose tails hold NaN: the local branch's tile
    loads must fill rows past token n - 1 with zeros (a NaN row would poison dK and dV of every
    key of the tile through 0 * NaN)."""
    B, Hq, Hkv, n, d, w, pad = 1, 4, 2, 389, 128, 200, 640
    flags = CAUSAL | SWA_ONE_SIDED
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), torch.bfloat16, seed=61)
    g = torch.Generator().manual_seed(62)
    dy = torch.randn(B, Hq, n, d, generator=g).to(torch.bfloat16)
    lg = torch.randn(2, Hq, generator=g)
    perm, inv, permc, invc = perms(61, 0, B, n)

    def padded(t):
        buf = torch.full((B, t.shape[1], pad, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        buf[:, :, :n] = t.cuda()
        return buf[:, :, :n]
    qd, kd, vd, dyd = padded(q), padded(k), padded(v), padded(dy)
    mk = lambda like: torch.zeros((B, like.shape[1], pad, d), dtype=torch.bfloat16, device="cuda")[:, :, :n]
    y, y_sa, y_swa, lse_sa, lse_swa = sa.sa_swa_gated_forward(
        qd, kd, vd, perm, inv, lg.cuda(), w, flags, save_for_bwd=True,
        out={"y": mk(q), "y_sa": mk(q), "y_swa": mk(q)})
    dq, dk, dv, dg = sa.sa_backward(qd, kd, vd, perm, inv, lg.cuda(), y_sa, y_swa, lse_sa, lse_swa,
                                    dyd, w, flags, out={"dq": mk(q), "dk": mk(k), "dv": mk(k)})
    assert sa.sa_read_status() == 0
    rdq, rdk, rdv, rdg = oracle.backward(as_f64(q), as_f64(k), as_f64(v), permc, invc,
                                         lg.double().numpy(), as_f64(dy), w, flags)
    for got, r, name in ((dq, rdq, "dq"), (dk, rdk, "dk"), (dv, rdv, "dv")):
        assert torch.isfinite(got.float()).all(), name
        close(got, r, torch.bfloat16, name)


def test_cuda_core_kernels_on_tensor_core_shapes(debug_option):
    # with the tensor cores switched off the general kernels serve the bf16 d = 64 / 128 cases
    debug_option(sa.DEBUG_TENSOR_CORES, 0)
    bf = torch.bfloat16
    for case in SMALL[:9]:
        test_sa_forward_small(*case, bf)
    for case in BWD_SMALL[:4]:
        test_backward_small(*case, True, bf)


def test_swa_tma_path_ragged_tail_and_strides():
    """One-sided SWA on the tensor-core path with n not a multiple of 128 (the last tile reads
    rows of the next head, or past the matrix), several heads and batches, both layouts."""
    B, Hq, Hkv, n, w = 2, 4, 2, 389, 200
    flags = CAUSAL | SWA_ONE_SIDED
    for d in (64, 128):
        q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), torch.bfloat16, seed=40 + d)
        ry, _ = oracle.swa_forward(as_f64(q), as_f64(k), as_f64(v), w, flags)
        for token_major in (False, True):
            if token_major:
                dev = [t.permute(0, 2, 1, 3).contiguous().cuda().permute(0, 2, 1, 3) for t in (q, k, v)]
            else:
                dev = [t.cuda() for t in (q, k, v)]
            y = sa.sa_swa_forward(dev[0], dev[1], dev[2], w, flags, y=torch.empty_like(dev[0]))
            close(y, ry, torch.bfloat16, "d=%d token_major=%s" % (d, token_major))
        # views of longer buffers whose tails hold NaN (an unwritten KV-cache tail, say): the
        # last tile must read zeros past token n - 1, not those rows (0 * NaN would poison
        # every valid query of the tile through P V)
        pad = 700
        dev = []
        for t in (q, k, v):
            buf = torch.full((B, t.shape[1], pad, d), float("nan"), dtype=torch.bfloat16,
                             device="cuda")
            buf[:, :, :n] = t.cuda()
            dev.append(buf[:, :, :n])
        assert not dev[0].is_contiguous()
        ybuf = torch.zeros((B, Hq, pad, d), dtype=torch.bfloat16, device="cuda")
        y = sa.sa_swa_forward(dev[0], dev[1], dev[2], w, flags, y=ybuf[:, :, :n])
        assert torch.isfinite(y.float()).all()
        close(y, ry, torch.bfloat16, "d=%d NaN tail" % d)
    assert sa.sa_read_status() == 0


def crafted_perms(n, rng):
    """Permutations that stress the masked online softmax: (a) slots hold the tokens in
    decreasing order, so the first half of every query's band is masked out entirely and the
    running maximum stays at minus infinity for whole score blocks; (b) a random permutation
    with token 0 moved to the last slot, whose only visible key (itself) is then the last
    element of the last block of its band under the linear window."""
    rev = np.arange(n - 1, -1, -1, dtype=np.int32)
    rnd = rng.permutation(n).astype(np.int32)
    at0 = int(np.nonzero(rnd == 0)[0][0])
    rnd[at0], rnd[n - 1] = rnd[n - 1], rnd[at0]
    out = []
    for pm in (rev, rnd):
        iv = np.empty_like(pm)
        iv[pm] = np.arange(n, dtype=np.int32)
        out.append((pm[None].copy(), iv[None].copy()))
    return out


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n,d,w,flags", [
    (700, 128, 300, CAUSAL | LINEAR_WINDOW),    # 128-key score blocks, ragged tail
    (700, 128, 300, CAUSAL),                    # the same with the circular window
    (900, 64, 100, CAUSAL | LINEAR_WINDOW),     # 64-key score blocks
    (515, 128, 2000, CAUSAL),                   # window covers the sequence
])
def test_forward_large_scores_and_late_first_visible_key(n, d, w, flags, dtype):
    """Scaled scores of magnitude ~50 (Q, K ~ 4 N(0,1)), so that exp2 arguments span far more
    than the lazy-rescaling threshold and a missed rescale or a stale maximum would overflow
    or flush a row to zero; on permutations whose rows meet their first visible key late."""
    B, Hq, Hkv = 1, 2, 1
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), dtype, seed=n + d, scale=1.0)
    q, k = (q.float() * 4).to(dtype), (k.float() * 4).to(dtype)
    s_abs = (as_f64(q)[0, 0] @ as_f64(k)[0, 0].T / np.sqrt(d))
    assert np.abs(s_abs).max() > 40
    for permc, invc in crafted_perms(n, np.random.default_rng(n)):
        perm, inv = torch.from_numpy(permc).cuda(), torch.from_numpy(invc).cuda()
        y, lse = sa.sa_forward(q.cuda(), k.cuda(), v.cuda(), perm, inv, w, flags, want_lse=True)
        assert sa.sa_read_status() == 0
        assert torch.isfinite(y.float()).all() and torch.isfinite(lse).all()
        ry, rlse = oracle.sa_forward(as_f64(q), as_f64(k), as_f64(v), permc, invc, w, flags)
        close(y, ry, dtype, "y")
        # lse is of the order of the largest score here: compare relative to its size
        tol = (1e-4 if dtype == torch.float32 else 2e-2) * max(1.0, np.abs(rlse).max() / 8)
        assert np.abs(as_f64(lse) - rlse).max() <= tol
    # the plain-SWA kernels on the same scores (one-sided window: first blocks fully visible)
    y = sa.sa_swa_forward(q.cuda(), k.cuda(), v.cuda(), w, CAUSAL | SWA_ONE_SIDED)
    ry, _ = oracle.swa_forward(as_f64(q), as_f64(k), as_f64(v), w, CAUSAL | SWA_ONE_SIDED)
    close(y, ry, dtype, "y_swa")


def test_identity_permutation_equals_swa_on_device():
    B, Hq, Hkv, n, d, w = 1, 2, 1, 333, 64, 17
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), torch.float32, seed=1)
    ident = torch.arange(n, dtype=torch.int32, device="cuda")[None].contiguous()
    y1 = sa.sa_forward(q.cuda(), k.cuda(), v.cuda(), ident, ident, w, CAUSAL)
    y2 = sa.sa_swa_forward(q.cuda(), k.cuda(), v.cuda(), w, CAUSAL)
    assert torch.equal(y1, y2)


def test_token_major_strides():
    # [B,n,H,d] storage viewed as [B,H,n,d]
    B, Hq, Hkv, n, d, w = 2, 4, 2, 200, 64, 21
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), torch.bfloat16, seed=9)
    tm = lambda t: t.cuda().permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    perm, inv, permc, invc = perms(9, 0, B, n)
    qd, kd, vd = tm(q), tm(k), tm(v)
    assert not qd.is_contiguous()
    y = sa.sa_forward(qd, kd, vd, perm, inv, w, CAUSAL, y=torch.empty_like(qd))
    ry, _ = oracle.sa_forward(as_f64(q), as_f64(k), as_f64(v), permc, invc, w, CAUSAL)
    close(y, ry, torch.bfloat16)


def test_softmax_scale():
    B, Hq, Hkv, n, d, w = 1, 1, 1, 100, 64, 9
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), torch.float32, seed=2)
    perm, inv, permc, invc = perms(2, 0, B, n)
    y = sa.sa_forward(q.cuda(), k.cuda(), v.cuda(), perm, inv, w, 0, scale=0.05)
    ry, _ = oracle.sa_forward(as_f64(q), as_f64(k), as_f64(v), permc, invc, w, 0, scale=0.05)
    close(y, ry, torch.float32)


def test_config_c1_full():
    c = wl.C1
    t = wl.draw(c)
    perm, inv, permc, invc = perms(c.seed, 0, c.B, c.n)
    y = sa.sa_forward(t["q"].cuda(), t["k"].cuda(), t["v"].cuda(), perm, inv, c.w, c.flags)
    ry, _ = oracle.sa_forward(as_f64(t["q"]), as_f64(t["k"]), as_f64(t["v"]), permc, invc, c.w,
                              c.flags)
    close(y, ry, torch.float32, "C1")
    assert np.array_equal(permc, oracle.make_perm(c.seed, 0, c.B, c.n)[0])


def test_config_c2_full():
    c = wl.C2
    t = wl.draw(c)
    perm, inv, permc, invc = perms(c.seed, 0, c.B, c.n)
    operm, oinv = oracle.make_perm(c.seed, 0, c.B, c.n)
    assert np.array_equal(permc, operm) and np.array_equal(invc, oinv)
    y = sa.sa_forward(t["q"].cuda(), t["k"].cuda(), t["v"].cuda(), perm, inv, c.w, c.flags)
    ry, _ = oracle.sa_forward(as_f64(t["q"]), as_f64(t["k"]), as_f64(t["v"]), operm, oinv, c.w,
                              c.flags)
    close(y, ry, torch.bfloat16, "C2")


def sample_rows(c, rng, count):
    """Random rows plus every row of the first / last 128 slots' worth of tokens."""
    total = c.B * c.Hq * c.n
    rows = rng.choice(total, size=count, replace=False)
    edge = np.concatenate([np.arange(0, 128), np.arange(c.n - 128, c.n)])
    return np.unique(np.concatenate([rows, edge, (c.Hq - 1) * c.n + edge])).astype(np.int64)


def gated_rows_reference(c, t, permc, invc, rows):
    q, k, v = as_f64(t["q"]), as_f64(t["k"]), as_f64(t["v"])
    ysa, lsa = oracle.forward_rows(0, q, k, v, permc, invc, c.w, c.flags, rows)
    ysw, lsw = oracle.forward_rows(1, q, k, v, None, None, c.w, c.flags, rows)
    lg = t["gate_logits"].double().numpy()
    hq = (rows // c.n) % c.Hq
    g = 1 / (1 + np.exp(-lg))
    return g[0, hq][:, None] * ysa + g[1, hq][:, None] * ysw, ysa, ysw, lsa, lsw


def test_config_c3_sampled_rows():
    c = wl.C3
    t = wl.draw(c)
    perm, inv, permc, invc = perms(c.seed, 0, c.B, c.n)
    operm, oinv = oracle.make_perm(c.seed, 0, c.B, c.n)
    assert np.array_equal(permc, operm) and np.array_equal(invc, oinv)
    d = {k_: v_.cuda() for k_, v_ in t.items()}
    y, y_sa, y_swa, lse_sa, lse_swa = sa.sa_swa_gated_forward(
        d["q"], d["k"], d["v"], perm, inv, d["gate_logits"], c.w, c.flags, save_for_bwd=True)
    y_only_sa = sa.sa_forward(d["q"], d["k"], d["v"], perm, inv, c.w, c.flags)
    assert torch.equal(y_only_sa, y_sa)
    rows = sample_rows(c, np.random.default_rng(0), 4096)
    ry, rysa, rysw, rlsa, rlsw = gated_rows_reference(c, t, operm, oinv, rows)
    flat = lambda x: x.reshape(-1, c.d)[torch.from_numpy(rows).cuda()]
    close(flat(y), ry, torch.bfloat16, "y")
    close(flat(y_sa), rysa, torch.bfloat16, "y_sa")
    close(flat(y_swa), rysw, torch.bfloat16, "y_swa")
    assert np.abs(as_f64(lse_sa.reshape(-1)[torch.from_numpy(rows).cuda()]) - rlsa).max() < 2e-2
    assert np.abs(as_f64(lse_swa.reshape(-1)[torch.from_numpy(rows).cuda()]) - rlsw).max() < 2e-2
    # a property that holds at any size: each output row is a convex combination of V rows
    vmax = d["v"].float().norm(dim=-1).max()
    assert y_sa.float().norm(dim=-1).max() <= vmax * 1.01
    assert sa.sa_read_status() == 0


def test_config_c4_two_layers_sampled_rows():
    c = wl.C4
    t = wl.draw(c)
    d = {k_: v_.cuda() for k_, v_ in t.items()}
    rng = np.random.default_rng(1)
    for layer in (0, c.layers - 1):
        perm, inv, permc, invc = perms(c.seed, layer, c.B, c.n)
        operm, oinv = oracle.make_perm(c.seed, layer, c.B, c.n)
        assert np.array_equal(permc, operm) and np.array_equal(invc, oinv)
        y = sa.sa_swa_gated_forward(d["q"], d["k"], d["v"], perm, inv, d["gate_logits"], c.w,
                                    c.flags)
        rows = sample_rows(c, rng, 1024)
        ry = gated_rows_reference(c, t, operm, oinv, rows)[0]
        close(y.reshape(-1, c.d)[torch.from_numpy(rows).cuda()], ry, torch.bfloat16, "C4 y")
    assert sa.sa_read_status() == 0


# ------------------------------------------------------------------------ gated

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("save", [False, True])
def test_gated_forward_small(dtype, save):
    B, Hq, Hkv, n, d, w = 2, 4, 2, 391, 64, 50
    flags = CAUSAL | SWA_ONE_SIDED
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), dtype, seed=77)
    lg = torch.randn(2, Hq, generator=torch.Generator().manual_seed(5))
    perm, inv, permc, invc = perms(77, 2, B, n)
    out = sa.sa_swa_gated_forward(q.cuda(), k.cuda(), v.cuda(), perm, inv, lg.cuda(), w, flags,
                                  save_for_bwd=save)
    ref = oracle.gated_forward(as_f64(q), as_f64(k), as_f64(v), permc, invc, lg.double().numpy(),
                               w, flags)
    if save:
        for got, r, name in zip(out[:3], ref[:3], ("y", "y_sa", "y_swa")):
            close(got, r, dtype, name)
        for got, r in zip(out[3:], ref[3:]):
            assert np.abs(as_f64(got) - r).max() <= (1e-4 if dtype == torch.float32 else 2e-2)
    else:
        close(out, ref[0], dtype, "y")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("token_major", [False, True])
def test_gated_forward_both_combine_paths(dtype, fused, token_major):
    """The gates are applied inside the local branch's launch, either by its two idle warps
    over stored rows (scratch given: the SA rows go there) or in the row threads' epilogue (no
    scratch: the SA rows sit in y itself); d = 128 and w = 300 put the bf16 case on the
    tensor-core kernels with 128-key blocks.  Also on token-major tensors.  Two launches
    either way."""
    B, Hq, Hkv, n, d, w = 1, 4, 2, 521, 128, 300
    flags = CAUSAL | SWA_ONE_SIDED
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), dtype, seed=31)
    lg = torch.randn(2, Hq, generator=torch.Generator().manual_seed(6))
    perm, inv, permc, invc = perms(31, 1, B, n)
    if token_major:   # memory order [B,n,H,d], seen as [B,H,n,d]
        dev = [t.permute(0, 2, 1, 3).contiguous().cuda().permute(0, 2, 1, 3) for t in (q, k, v)]
    else:
        dev = [t.cuda() for t in (q, k, v)]
    y = torch.empty_like(dev[0])
    ws = None
    if not fused:
        nbytes = sa.sa_workspace_bytes(sa.make_problem(dev[0], dev[1], w, flags),
                                       sa.OP_GATED_FORWARD_SCRATCH)
        assert nbytes >= y.numel() * y.element_size()
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    launches = sa.launch_count()
    sa.sa_swa_gated_forward(dev[0], dev[1], dev[2], perm, inv, lg.cuda(), w, flags,
                            out={"y": y}, ws=ws, fused_epilogue=fused)
    assert sa.launch_count() - launches == 2
    assert sa.sa_read_status() == 0
    ref = oracle.gated_forward(as_f64(q), as_f64(k), as_f64(v), permc, invc, lg.double().numpy(),
                               w, flags)
    close(y, ref[0], dtype, "y")


# --------------------------------------------------------------------- backward

def run_backward(q, k, v, dy, lg, perm, inv, w, flags):
    qd, kd, vd, dyd = q.cuda(), k.cuda(), v.cuda(), dy.cuda()
    if lg is None:
        y, lse = sa.sa_forward(qd, kd, vd, perm, inv, w, flags, want_lse=True)
        return sa.sa_backward(qd, kd, vd, perm, inv, None, y, None, lse, None, dyd, w, flags)
    y, y_sa, y_swa, lse_sa, lse_swa = sa.sa_swa_gated_forward(qd, kd, vd, perm, inv, lg.cuda(), w,
                                                              flags, save_for_bwd=True)
    return sa.sa_backward(qd, kd, vd, perm, inv, lg.cuda(), y_sa, y_swa, lse_sa, lse_swa, dyd, w,
                          flags)


BWD_SMALL = [
    (2, 4, 2, 200, 64, 21, CAUSAL | SWA_ONE_SIDED),
    (1, 2, 2, 130, 128, 40, 0),
    (1, 2, 1, 77, 32, 300, CAUSAL),
    (1, 1, 1, 260, 64, 1, CAUSAL | SWA_ONE_SIDED),
    (1, 8, 2, 700, 128, 200, CAUSAL | SWA_ONE_SIDED),   # GQA group of 4, several tiles, wrap-around
    (2, 2, 1, 515, 64, 129, CAUSAL | LINEAR_WINDOW),    # no wrap, ragged last tile
    (1, 2, 2, 384, 128, 96, 0),                         # non-causal, n a tile multiple
    (1, 2, 1, 200, 64, 1000, CAUSAL | SWA_ONE_SIDED),   # w > n: every causal key, two tiles
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("B,Hq,Hkv,n,d,w,flags", BWD_SMALL)
def test_backward_small(B, Hq, Hkv, n, d, w, flags, gated, dtype):
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), dtype, seed=n)
    g = torch.Generator().manual_seed(n + 1)
    dy = torch.randn(B, Hq, n, d, generator=g).to(dtype)
    lg = torch.randn(2, Hq, generator=g) if gated else None
    perm, inv, permc, invc = perms(n, 1, B, n)
    dq, dk, dv, dg = run_backward(q, k, v, dy, lg, perm, inv, w, flags)
    rdq, rdk, rdv, rdg = oracle.backward(as_f64(q), as_f64(k), as_f64(v), permc, invc,
                                         None if lg is None else lg.double().numpy(),
                                         as_f64(dy), w, flags)
    if dtype == torch.float32:
        # gradients are sums of up to band*G terms of size O(1): scale the fp32 bound
        for got, r, name in ((dq, rdq, "dq"), (dk, rdk, "dk"), (dv, rdv, "dv")):
            assert np.abs(as_f64(got) - r).max() <= 1e-4 * max(1.0, np.abs(r).max()), name
        if gated:
            assert np.abs(as_f64(dg) - rdg).max() <= 1e-4 * max(1.0, np.abs(rdg).max())
    else:
        close(dq, rdq, dtype, "dq")
        close(dk, rdk, dtype, "dk")
        close(dv, rdv, dtype, "dv")
        if gated:
            close(dg, rdg, dtype, "dgate")
    assert sa.sa_read_status() == 0


def test_config_c5_one_layer_full():
    c = wl.C5
    t = wl.draw(c)
    perm, inv, permc, invc = perms(c.seed, 0, c.B, c.n)
    dq, dk, dv, dg = run_backward(t["q"], t["k"], t["v"], t["dy"], t["gate_logits"], perm, inv,
                                  c.w, c.flags)
    rdq, rdk, rdv, rdg = oracle.backward(as_f64(t["q"]), as_f64(t["k"]), as_f64(t["v"]), permc,
                                         invc, t["gate_logits"].double().numpy(),
                                         as_f64(t["dy"]), c.w, c.flags)
    close(dq, rdq, torch.bfloat16, "dq")
    close(dk, rdk, torch.bfloat16, "dk")
    close(dv, rdv, torch.bfloat16, "dv")
    close(dg, rdg, torch.bfloat16, "dgate")
    y = sa.sa_swa_gated_forward(t["q"].cuda(), t["k"].cuda(), t["v"].cuda(), perm, inv,
                                t["gate_logits"].cuda(), c.w, c.flags)
    ry = oracle.gated_forward(as_f64(t["q"]), as_f64(t["k"]), as_f64(t["v"]), permc, invc,
                              t["gate_logits"].double().numpy(), c.w, c.flags)[0]
    close(y, ry, torch.bfloat16, "y")


def test_config_c3_backward_sampled_rows():
    """Gated backward at the Qwen3-8B-shaped size, where the whole-tensor oracle would take
    days: >= 1024 rows of dq and >= 1024 rows of dk / dv (random rows plus the first and the
    last 128 tokens, whose windows wrap around in slot order), and the full dgate."""
    c = wl.C3
    t = wl.draw(c)
    g = torch.Generator().manual_seed(c.seed + 100)
    dy = torch.randn(c.B, c.Hq, c.n, c.d, generator=g).to(torch.bfloat16)
    perm, inv, permc, invc = perms(c.seed, 0, c.B, c.n)
    lg = t["gate_logits"]
    dq, dk, dv, dg = run_backward(t["q"], t["k"], t["v"], dy, lg, perm, inv, c.w, c.flags)
    assert sa.sa_read_status() == 0
    rng = np.random.default_rng(7)
    edge = np.concatenate([np.arange(0, 128), np.arange(c.n - 128, c.n)])
    q_rows = np.unique(np.concatenate([rng.choice(c.B * c.Hq * c.n, size=1024, replace=False),
                                       edge, (c.Hq - 1) * c.n + edge])).astype(np.int64)
    kv_rows = np.unique(np.concatenate([rng.choice(c.B * c.Hkv * c.n, size=768, replace=False),
                                        edge, (c.Hkv - 1) * c.n + edge[::2]])).astype(np.int64)
    assert q_rows.size >= 1024 and kv_rows.size >= 1024
    f = as_f64
    rdq, rdk, rdv = oracle.backward_rows(f(t["q"]), f(t["k"]), f(t["v"]), permc, invc,
                                         lg.double().numpy(), f(dy), c.w, c.flags, q_rows, kv_rows)
    pick = lambda x, rows: x.reshape(-1, c.d)[torch.from_numpy(rows).cuda()]
    close(pick(dq, q_rows), rdq, torch.bfloat16, "dq rows")
    close(pick(dk, kv_rows), rdk, torch.bfloat16, "dk rows")
    close(pick(dv, kv_rows), rdv, torch.bfloat16, "dv rows")
    # dgate[x, hq] = g(1-g) sum(dY o Y_x): Y_x rows from the row oracle would need every row, so
    # use what holds at any size instead: the sum over a head of dY o (oracle rows of Y_x) on
    # the sampled rows agrees with the device branch outputs the full reduction is taken over
    d = {k_: v_.cuda() for k_, v_ in t.items()}
    _, y_sa, y_swa, _, _ = sa.sa_swa_gated_forward(d["q"], d["k"], d["v"], perm, inv,
                                                   d["gate_logits"], c.w, c.flags, save_for_bwd=True)
    sg = torch.sigmoid(lg.double())
    dyd = dy.cuda().double()
    for x, yx in enumerate((y_sa, y_swa)):
        want = (sg[x] * (1 - sg[x])).cuda() * (dyd * yx.double()).sum(dim=(0, 2, 3))
        assert torch.allclose(dg[x].double(), want, rtol=2e-2, atol=2e-2 * want.abs().max().item())


def test_backward_is_deterministic():
    B, Hq, Hkv, n, d, w = 1, 4, 2, 500, 64, 33
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), torch.bfloat16, seed=4)
    g = torch.Generator().manual_seed(8)
    dy = torch.randn(B, Hq, n, d, generator=g).to(torch.bfloat16)
    lg = torch.randn(2, Hq, generator=g)
    perm, inv, _, _ = perms(4, 0, B, n)
    a = run_backward(q, k, v, dy, lg, perm, inv, w, CAUSAL | SWA_ONE_SIDED)
    b = run_backward(q, k, v, dy, lg, perm, inv, w, CAUSAL | SWA_ONE_SIDED)
    for x, y in zip(a, b):
        assert torch.equal(x, y)


# --------------------------------------------------------------------- coverage

@pytest.mark.parametrize("n,w,flags,L", [(2048, 32, 0, 6), (2048, 32, CAUSAL, 6), (27, 8, CAUSAL, 3),
                                         (1000, 9, LINEAR_WINDOW, 5), (64, 200, 0, 2),
                                         (50, 50, 0, 2)])
def test_coverage_bit_exact(n, w, flags, L):
    pl = [sa.sa_make_perm(31, l, 1, n) for l in range(L)]
    perm = torch.cat([a for a, _ in pl]).contiguous()
    inv = torch.cat([b for _, b in pl]).contiguous()
    for src in (0, n - 1, n // 3):
        nnz, rc, reach = sa.sa_coverage(perm, inv, w, flags, src)
        onnz, orc, oreach = oracle.coverage(perm.cpu().numpy(), inv.cpu().numpy(), w, flags, src)
        assert np.array_equal(nnz.cpu().numpy(), onnz)
        assert np.array_equal(rc.cpu().numpy(), orc)
        assert np.array_equal(reach.cpu().numpy(), oreach)


def test_coverage_study_sa_against_swa_and_prop2_bound():
    # Fig. 2 (left) setting: n = 2048, w = 32.  Seed-averaged reach of SA per layer against the
    # expansion bound of Prop. 2, and against plain SWA, whose reach grows by 2h per layer.
    n, w, L, seeds, src = 2048, 32, 6, 24, 5
    h = (w + 1) // 2 - 1
    band = 2 * h + 1
    pr = (band - 1) / (n - 1)
    sizes = np.zeros((seeds, L))
    for s_ in range(seeds):
        pl = [sa.sa_make_perm(7000 + s_, l, 1, n) for l in range(L)]
        perm = torch.cat([a_ for a_, _ in pl]).contiguous()
        inv = torch.cat([b_ for _, b_ in pl]).contiguous()
        nnz, rc, reach = sa.sa_coverage(perm, inv, w, 0, src)
        sizes[s_] = reach.cpu().numpy()
        assert int(rc.min()) == band and int(rc.max()) == band
    assert np.all(sizes[:, 0] == band) and np.all(np.diff(sizes, axis=1) >= 0)
    mean = sizes.mean(axis=0)
    for l in range(L - 1):
        r = sizes[:, l]
        assert mean[l + 1] >= 0.97 * (r + (n - r) * (1 - (1 - pr) ** r)).mean()
    assert mean[3] > 0.99 * n                       # full coverage in O(log_w n) layers
    ident = torch.arange(n, dtype=torch.int32, device="cuda").repeat(L, 1).contiguous()
    _, _, swa_reach = sa.sa_coverage(ident, ident, w, 0, src)
    assert swa_reach.cpu().tolist() == [min(n, 2 * (l + 1) * h + 1) for l in range(L)]
    assert mean[2] > 10 * swa_reach[2].item()       # SA has spread far beyond the local window


@pytest.mark.parametrize("n,w,L,seeds", [(2048, 32, 6, 4), (4096, 128, 4, 2), (32768, 1024, 3, 1)])
def test_coverage_fixed_sigma_against_independent_sigma(n, w, L, seeds):
    """The paper's two inference modes at the benchmark shapes: one fixed permutation reused at
    every layer gives the linear growth min(n, 2lh+1) of plain SWA (closed form, any size);
    an independent permutation per layer respects Prop. 2's expansion bound and covers the
    sequence within a few layers.  Bit-exact against the oracle where it finishes in seconds."""
    h = (w + 1) // 2 - 1
    band = min(n, 2 * h + 1)
    pr = (band - 1) / (n - 1)
    src = n // 3
    for s_ in range(seeds):
        pl = [sa.sa_make_perm(500 + s_, l, 1, n) for l in range(L)]
        perm = torch.cat([a for a, _ in pl]).contiguous()
        inv = torch.cat([b for _, b in pl]).contiguous()
        nnz, _, reach = sa.sa_coverage(perm, inv, w, 0, src, want_row_count=False)
        reach = reach.cpu().numpy()
        assert np.all(nnz.cpu().numpy() == n * band)          # closed form, every permutation
        assert reach[0] == band and np.all(np.diff(reach) >= 0)
        # one layer of Prop. 2's bound from the measured set size, with slack for one draw
        for l in range(L - 1):
            r = float(reach[l])
            assert reach[l + 1] >= 0.9 * (r + (n - r) * (1 - (1 - pr) ** r))
        assert reach[-1] == n
        fixed_p = pl[0][0].repeat(L, 1).contiguous()
        fixed_i = pl[0][1].repeat(L, 1).contiguous()
        _, _, fr = sa.sa_coverage(fixed_p, fixed_i, w, 0, src, want_row_count=False)
        assert fr.cpu().tolist() == [min(n, 2 * (l + 1) * h + 1) for l in range(L)]
        if n <= 4096:
            _, _, oreach = oracle.coverage(perm.cpu().numpy(), inv.cpu().numpy(), w, 0, src)
            assert np.array_equal(reach, oreach)
            _, _, ofr = oracle.coverage(fixed_p.cpu().numpy(), fixed_i.cpu().numpy(), w, 0, src)
            assert np.array_equal(fr.cpu().numpy(), ofr)


# ----------------------------------------------------------------------- status

def test_bounded_wait_runs_out_and_reports_timeout():
    """The failure path of the kernels' bounded waits, provoked without breaking anything: a
    hook kernel waits with the library's wait routine on a barrier nothing completes, with a
    limit of about a millisecond; it must return on its own, the status word must read
    SA_ERR_TIMEOUT (6), tensor-core launches are skipped while it is set, and reading clears
    it so that the next call works again."""
    B, Hq, Hkv, n, d, w = 1, 2, 1, 300, 64, 40
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), torch.bfloat16, seed=12)
    perm, inv, _, _ = perms(12, 0, B, n)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    good = sa.sa_forward(qd, kd, vd, perm, inv, w, CAUSAL)
    assert sa.sa_read_status() == 0
    sa.debug_wait_timeout(2_000_000)
    torch.cuda.synchronize()                       # the kernel came back by itself
    sentinel = torch.full_like(good, 7.0)
    sa.sa_forward(qd, kd, vd, perm, inv, w, CAUSAL, y=sentinel)   # skipped: status is sticky
    assert sa.sa_read_status() == 6
    assert torch.equal(sentinel, torch.full_like(good, 7.0))
    assert sa.sa_read_status() == 0                # reading cleared it
    again = sa.sa_forward(qd, kd, vd, perm, inv, w, CAUSAL)
    assert sa.sa_read_status() == 0 and torch.equal(again, good)
    with pytest.raises(sa.SaError):
        sa.debug_wait_timeout(0)


def test_validate_perm_reports_a_non_bijection():
    B, Hq, Hkv, n, d, w = 1, 1, 1, 64, 64, 9
    q, k, v = draw((B, Hq, n, d), (B, Hkv, n, d), torch.float32, seed=6)
    perm, inv, _, _ = perms(6, 0, B, n)
    y = sa.sa_forward(q.cuda(), k.cuda(), v.cuda(), perm, inv, w, CAUSAL | wl.VALIDATE_PERM)
    assert sa.sa_read_status() == 0
    bad = perm.clone()
    bad[0, 5] = bad[0, 6]                 # in range, but token repeated: not a bijection
    sa.sa_forward(q.cuda(), k.cuda(), v.cuda(), bad, inv, w, CAUSAL | wl.VALIDATE_PERM)
    assert sa.sa_read_status() == 5       # SA_ERR_BAD_PERM
    assert sa.sa_read_status() == 0       # reading clears it
    y2 = sa.sa_forward(q.cuda(), k.cuda(), v.cuda(), perm, inv, w, CAUSAL | wl.VALIDATE_PERM)
    assert torch.equal(y, y2)
