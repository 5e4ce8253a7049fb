"""Projection gates of Eq. 5-6 through the C ABI against the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def _draw(rows, dm, seed, dtype, pitch=None):
    g = torch.Generator().manual_seed(seed)
    pitch = pitch or dm
    def y():
        t = torch.randn(rows, pitch, generator=g).to(dtype)
        return t
    ws = (dm ** -0.5)
    return y(), y(), (torch.randn(dm, dm, generator=g) * ws).to(dtype), (torch.randn(dm, dm, generator=g) * ws).to(dtype)


def _check(out, ya, wa, yb, wb, dm, tol):
    want = oracle.gate_projection(ya[:, :dm].double().numpy(), wa.double().numpy(),
                                  None if yb is None else yb[:, :dm].double().numpy(),
                                  None if wb is None else wb.double().numpy())
    got = out.double().cpu().numpy()
    err = np.abs(got - want)
    bound = tol * np.maximum(np.abs(want), 1.0)
    assert (err <= bound).all(), float((err / np.maximum(np.abs(want), 1.0)).max())


# bf16 result: one rounding of the output (2^-9 relative) plus fp32 accumulation of bf16 products
@pytest.mark.parametrize("rows,dm,pitch", [(300, 192, None), (1000, 256, None), (129, 64, 128),
                                           (128, 128, None), (517, 320, 512)])
@pytest.mark.parametrize("dual", [True, False])
def test_tensor_core_path_bf16(rows, dm, pitch, dual):
    from paper_2604_00754_b200 import binding as sa
    ya, yb, wa, wb = _draw(rows, dm, 3 + rows, torch.bfloat16, pitch)
    args = [ya.cuda()[:, :dm], wa.cuda()]
    if dual:
        args += [yb.cuda()[:, :dm], wb.cuda()]
    out = sa.sa_gate_projection_forward(*args)
    assert sa.sa_read_status() == 0
    _check(out, ya, wa, yb if dual else None, wb if dual else None, dm, 2e-2)


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-4), (torch.bfloat16, 2e-2)])
def test_plain_path_odd_sizes(dtype, tol):
    from paper_2604_00754_b200 import binding as sa
    rows, dm = 37, 50           # dm not a multiple of 64: the plain kernel
    ya, yb, wa, wb = _draw(rows, dm, 5, dtype)
    out = sa.sa_gate_projection_forward(ya.cuda(), wa.cuda(), yb.cuda(), wb.cuda())
    assert sa.sa_read_status() == 0
    _check(out, ya, wa, yb, wb, dm, tol)


def _model_width_rows(rows, rng):
    """>= 512 random rows plus every row of the first and of the last 128-row tile."""
    idx = np.unique(np.concatenate([rng.choice(rows, size=512, replace=False),
                                    np.arange(0, 128), np.arange(rows - 128, rows)]))
    return torch.from_numpy(idx)


@pytest.mark.parametrize("wide", [True, False])
@pytest.mark.parametrize("dual", [True, False])
def test_model_width_sampled_rows(wide, dual):
    """Qwen3-8B width (Hq*d = 4096) on the attention output layout [B,n,Hq,d] viewed as
    [B*n, Hq*d].  wide: the 128 x 256-tile kernel the library picks at this size (dual path:
    second launch accumulates into the rounded result of the first); not wide: the fused
    128 x 128 kernel forced at the same size through the test hook."""
    from paper_2604_00754_b200 import binding as sa
    rows, dm = 4096, 4096
    ya, yb, wa, wb = _draw(rows, dm, 9, torch.bfloat16)
    sa.debug_set(sa.DEBUG_GATE_WIDE_TILES, 1 if wide else 0)
    try:
        launches = sa.launch_count()
        if dual:
            out = sa.sa_gate_projection_forward(ya.cuda(), wa.cuda(), yb.cuda(), wb.cuda())
        else:
            out = sa.sa_gate_projection_forward(ya.cuda(), wa.cuda())
        # the two kernels differ in their launch count on the dual path (one per path / one)
        if dual:
            assert sa.launch_count() - launches == (2 if wide else 1)
    finally:
        sa.debug_set(sa.DEBUG_GATE_WIDE_TILES, 1)
    assert sa.sa_read_status() == 0
    idx = _model_width_rows(rows, np.random.default_rng(3))
    _check(out[idx.cuda()], ya[idx], wa, yb[idx] if dual else None, wb if dual else None, dm, 2e-2)


def test_rejects_bad_arguments():
    from paper_2604_00754_b200 import binding as sa
    y = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(64, 32, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ValueError):
        sa.sa_gate_projection_forward(y, w)


def test_dual_path_block_on_token_major_layout():
    """Alg. 2 with the projection gates of Eq. 6 end to end: Q/K/V stored token-major
    ([B,n,H,d], as a QKV projection writes them), both attention branches write their outputs
    in the same layout, and the gate product reads them as [B*n, Hq*d] without any copy."""
    from paper_2604_00754_b200 import binding as sa
    B, Hq, Hkv, n, d, w = 2, 4, 2, 700, 64, 256
    dm = Hq * d
    g = torch.Generator().manual_seed(21)
    q = torch.randn(B, n, Hq, d, generator=g).bfloat16()
    k = torch.randn(B, n, Hkv, d, generator=g).bfloat16()
    v = torch.randn(B, n, Hkv, d, generator=g).bfloat16()
    wa = (torch.randn(dm, dm, generator=g) * dm ** -0.5).bfloat16()
    wb = (torch.randn(dm, dm, generator=g) * dm ** -0.5).bfloat16()
    qd, kd, vd = (t.cuda().permute(0, 2, 1, 3) for t in (q, k, v))      # [B,H,n,d] views
    perm, inv = sa.sa_make_perm(4, 0, B, n)
    flags = sa.CAUSAL | sa.SWA_ONE_SIDED
    y_sa = torch.empty(B, n, Hq, d, dtype=torch.bfloat16, device="cuda")
    y_swa = torch.empty_like(y_sa)
    sa.sa_forward(qd, kd, vd, perm, inv, w, flags, y=y_sa.permute(0, 2, 1, 3))
    sa.sa_swa_forward(qd, kd, vd, w, flags, y=y_swa.permute(0, 2, 1, 3))
    out = sa.sa_gate_projection_forward(y_sa.view(B * n, dm), wa.cuda(), y_swa.view(B * n, dm), wb.cuda())
    assert sa.sa_read_status() == 0

    f64 = lambda t: np.ascontiguousarray(t.permute(0, 2, 1, 3).double().numpy())
    p_np, i_np = perm.cpu().numpy(), inv.cpu().numpy()
    o_sa = oracle.sa_forward(f64(q), f64(k), f64(v), p_np, i_np, w, flags)[0]
    o_swa = oracle.swa_forward(f64(q), f64(k), f64(v), w, flags)[0]
    tok_major = lambda a: np.ascontiguousarray(a.transpose(0, 2, 1, 3)).reshape(B * n, dm)
    want = oracle.gate_projection(tok_major(o_sa), wa.double().numpy(), tok_major(o_swa), wb.double().numpy())
    got = out.double().cpu().numpy()
    # two bf16 roundings in a row (branch outputs, then the gated sum) and a dm-long product
    # of the rounded outputs: 3e-2 of max(|want|, 1)
    err = np.abs(got - want) / np.maximum(np.abs(want), 1.0)
    assert err.max() <= 3e-2, float(err.max())


def _check_grads(got, want, tol):
    for g, w_, name in zip(got, want, ("dy_sa", "dw_sa", "dy_swa", "dw_swa")):
        g = g.double().cpu().numpy()
        # gradients are sums of many signed terms: the bound is relative to the tensor's scale
        scale = max(np.abs(w_).max(), 1e-6)
        err = np.abs(g - w_).max() / scale
        assert err <= tol, (name, float(err))


@pytest.mark.parametrize("rows,dm,pitch", [(300, 192, None), (1000, 256, None), (129, 64, 128),
                                           (128, 128, None), (517, 320, 512)])
@pytest.mark.parametrize("dual", [True, False])
def test_backward_tensor_core_path_bf16(rows, dm, pitch, dual):
    from paper_2604_00754_b200 import binding as sa
    ya, yb, wa, wb = _draw(rows, dm, 13 + rows, torch.bfloat16, pitch)
    dout = torch.randn(rows, dm, generator=torch.Generator().manual_seed(rows)).bfloat16()
    args = [dout.cuda(), ya.cuda()[:, :dm], wa.cuda()]
    if dual:
        args += [yb.cuda()[:, :dm], wb.cuda()]
    got = sa.sa_gate_projection_backward(*args)
    assert sa.sa_read_status() == 0
    want = oracle.gate_projection_backward(
        dout.double().numpy(), ya[:, :dm].double().numpy(), wa.double().numpy(),
        yb[:, :dm].double().numpy() if dual else None, wb.double().numpy() if dual else None)
    # bf16 intermediates (dz, dout * g) and bf16 results, fp32 accumulation: 2e-2 of the scale
    _check_grads(got, want, 2e-2)


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-4), (torch.bfloat16, 2e-2)])
def test_backward_plain_path_odd_sizes(dtype, tol):
    from paper_2604_00754_b200 import binding as sa
    rows, dm = 37, 50
    ya, yb, wa, wb = _draw(rows, dm, 15, dtype)
    dout = torch.randn(rows, dm, generator=torch.Generator().manual_seed(2)).to(dtype)
    got = sa.sa_gate_projection_backward(dout.cuda(), ya.cuda(), wa.cuda(), yb.cuda(), wb.cuda())
    assert sa.sa_read_status() == 0
    want = oracle.gate_projection_backward(dout.double().numpy(), ya.double().numpy(), wa.double().numpy(),
                                           yb.double().numpy(), wb.double().numpy())
    _check_grads(got, want, tol)


def test_backward_model_width_single_path():
    """Qwen3-8B width (dm = 4096), 4096 tokens, single path, whole result against the oracle."""
    from paper_2604_00754_b200 import binding as sa
    rows, dm = 4096, 4096
    ya, _, wa, _ = _draw(rows, dm, 19, torch.bfloat16)
    dout = torch.randn(rows, dm, generator=torch.Generator().manual_seed(3)).bfloat16()
    got = sa.sa_gate_projection_backward(dout.cuda(), ya.cuda(), wa.cuda())
    assert sa.sa_read_status() == 0
    want = oracle.gate_projection_backward(dout.double().numpy(), ya.double().numpy(), wa.double().numpy())
    _check_grads(got, want, 2e-2)


@pytest.mark.parametrize("rows,dm", [(1, 64), (127, 64), (130, 448)])
def test_gate_edge_shapes_forward_and_backward(rows, dm):
    """A single row, one row short of a tile, a ragged last row tile with a half column tile."""
    from paper_2604_00754_b200 import binding as sa
    ya, yb, wa, wb = _draw(rows, dm, 100 + rows, torch.bfloat16)
    dout = torch.randn(rows, dm, generator=torch.Generator().manual_seed(rows)).bfloat16()
    out = sa.sa_gate_projection_forward(ya.cuda(), wa.cuda(), yb.cuda(), wb.cuda())
    got = sa.sa_gate_projection_backward(dout.cuda(), ya.cuda(), wa.cuda(), yb.cuda(), wb.cuda())
    assert sa.sa_read_status() == 0
    _check(out, ya, wa, yb, wb, dm, 2e-2)
    want = oracle.gate_projection_backward(dout.double().numpy(), ya.double().numpy(), wa.double().numpy(),
                                           yb.double().numpy(), wb.double().numpy())
    _check_grads(got, want, 2e-2)


def test_gate_backward_rejects_small_workspace():
    from paper_2604_00754_b200 import binding as sa
    y = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sa.SaError):
        sa.sa_gate_projection_backward(y, y, w, ws=torch.empty(16, dtype=torch.uint8, device="cuda"))
