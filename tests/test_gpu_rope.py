"""Rotary position embedding with original positions (Sec. 4.2, App. B) through the C ABI
against the float64 oracle: the table, the stand-alone rotation, and the forward calls that
rotate Q and K rows inside the gather."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_00754_b200 import binding as sa
from paper_2604_00754_b200.workloads import CAUSAL, LINEAR_WINDOW, SWA_ONE_SIDED, as_f64

pytestmark = pytest.mark.gpu


def draw(B, Hq, Hkv, n, d, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    mk = lambda h: torch.randn(B, h, n, d, generator=g).to(dtype)
    return mk(Hq), mk(Hkv), mk(Hkv)


def close(got, ref, dtype, what):
    err = np.abs(as_f64(got) - ref).max()
    bound = 1e-4 if dtype == torch.float32 else 2e-2 * np.abs(ref).max() + 1e-5
    assert err <= bound, "%s: %.3e > %.3e" % (what, err, bound)


@pytest.mark.parametrize("n,d,base", [(1, 2, 10000.0), (300, 64, 10000.0), (40000, 128, 1e6)])
def test_rope_table(n, d, base):
    cs, sn = sa.sa_rope_table(n, d, base)
    ang = np.arange(n, dtype=np.float64)[:, None] * base ** (-2.0 * np.arange(d // 2) / d)
    assert np.abs(as_f64(cs) - np.cos(ang)).max() < 2e-7
    assert np.abs(as_f64(sn) - np.sin(ang)).max() < 2e-7


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [8, 64, 128, 40])
def test_rope_apply_and_its_inverse(d, dtype):
    B, Hq, Hkv, n = 2, 4, 2, 333
    q, k, _ = draw(B, Hq, Hkv, n, d, dtype, seed=d)
    cs, sn = sa.sa_rope_table(n, d, 10000.0)
    pos = np.arange(n)
    qd, kd = q.cuda(), k.cuda()
    qr = sa.sa_rope_apply(qd, kd, cs, sn)
    kr = sa.sa_rope_apply(kd, qd, cs, sn, kv=True)
    close(qr, oracle.rope(as_f64(q), pos), dtype, "q")
    close(kr, oracle.rope(as_f64(k), pos), dtype, "k")
    back = sa.sa_rope_apply(qr, kd, cs, sn, inverse=True)
    close(back, as_f64(q), dtype, "inverse")


ROPE_CASES = [
    # B, Hq, Hkv, n, d, w, flags
    (1, 2, 1, 300, 64, 33, CAUSAL),
    (2, 4, 2, 389, 128, 200, CAUSAL),                  # 128-key score blocks, ragged tail, GQA
    (1, 8, 2, 1153, 64, 128, CAUSAL),                  # group of 4: two heads share a stream
    (1, 3, 3, 700, 128, 96, 0),                        # odd group: two slot tiles per item
    (1, 2, 2, 515, 128, 300, CAUSAL | LINEAR_WINDOW),
    (2, 8, 2, 6000, 64, 96, CAUSAL),                   # several items per CTA: both Q buffers turn over
]


@pytest.mark.parametrize("B,Hq,Hkv,n,d,w,flags", ROPE_CASES)
def test_forward_rope_in_the_gather(B, Hq, Hkv, n, d, w, flags):
    dtype = torch.bfloat16
    q, k, v = draw(B, Hq, Hkv, n, d, dtype, seed=n + d)
    perm, inv = sa.sa_make_perm(n, 1, B, n)
    cs, sn = sa.sa_rope_table(n, d, 10000.0)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    launches = sa.launch_count()
    y, lse = sa.sa_forward_rope(qd, kd, vd, perm, inv, cs, sn, w, flags, want_lse=True)
    assert sa.launch_count() - launches == 1           # one kernel: no rotation pass
    assert sa.sa_read_status() == 0
    pos = np.arange(n)
    ry, rlse = oracle.sa_forward(oracle.rope(as_f64(q), pos), oracle.rope(as_f64(k), pos),
                                 as_f64(v), perm.cpu().numpy(), inv.cpu().numpy(), w, flags)
    close(y, ry, dtype, "y")
    assert np.abs(as_f64(lse) - rlse).max() <= 2e-2 * max(1.0, np.abs(rlse).max() / 8)
    # the same arithmetic as the stand-alone rotation followed by the plain call
    y2 = sa.sa_forward(sa.sa_rope_apply(qd, kd, cs, sn), sa.sa_rope_apply(kd, qd, cs, sn, kv=True),
                       vd, perm, inv, w, flags)
    assert torch.equal(y, y2)
    # rotating by slot instead of by original position is a different function
    assert not torch.equal(y, sa.sa_forward(qd, kd, vd, perm, inv, w, flags))


@pytest.mark.parametrize("block", [64, 128])
def test_forward_rope_both_score_block_widths(block):
    sa.debug_set(sa.DEBUG_SCORE_BLOCK, block)
    try:
        for case in ROPE_CASES[:3]:
            test_forward_rope_in_the_gather(*case)
    finally:
        sa.debug_set(sa.DEBUG_SCORE_BLOCK, 0)


@pytest.mark.parametrize("dtype,d", [(torch.float32, 64), (torch.bfloat16, 32), (torch.float32, 8)])
def test_forward_rope_general_path(dtype, d):
    # fp32 and other head sizes: rotated copies in the workspace, then the general kernel
    B, Hq, Hkv, n, w = 1, 2, 1, 257, 40
    q, k, v = draw(B, Hq, Hkv, n, d, dtype, seed=d)
    perm, inv = sa.sa_make_perm(3, 0, B, n)
    cs, sn = sa.sa_rope_table(n, d, 500.0)
    y = sa.sa_forward_rope(q.cuda(), k.cuda(), v.cuda(), perm, inv, cs, sn, w, CAUSAL)
    pos = np.arange(n)
    ry, _ = oracle.sa_forward(oracle.rope(as_f64(q), pos, 500.0), oracle.rope(as_f64(k), pos, 500.0),
                              as_f64(v), perm.cpu().numpy(), inv.cpu().numpy(), w, CAUSAL)
    close(y, ry, dtype, "y")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_gated_forward_rope(dtype):
    B, Hq, Hkv, n, d, w = 2, 4, 2, 391, 64, 150
    flags = CAUSAL | SWA_ONE_SIDED
    q, k, v = draw(B, Hq, Hkv, n, d, dtype, seed=5)
    lg = torch.randn(2, Hq, generator=torch.Generator().manual_seed(6))
    perm, inv = sa.sa_make_perm(8, 0, B, n)
    cs, sn = sa.sa_rope_table(n, d, 10000.0)
    out = sa.sa_swa_gated_forward_rope(q.cuda(), k.cuda(), v.cuda(), perm, inv, cs, sn, lg.cuda(),
                                       w, flags, save_for_bwd=True)
    pos = np.arange(n)
    ref = oracle.gated_forward(oracle.rope(as_f64(q), pos), oracle.rope(as_f64(k), pos), as_f64(v),
                               perm.cpu().numpy(), inv.cpu().numpy(), lg.double().numpy(), w, flags)
    for got, r, name in zip(out[:3], ref[:3], ("y", "y_sa", "y_swa")):
        close(got, r, dtype, name)
    assert sa.sa_read_status() == 0


def test_backward_through_the_rotation():
    """Gradients with respect to the UNROTATED q and k: rotate, sa_backward, rotate back with the
    inverse (the transpose of the rotation), against the oracle's chain of the same steps."""
    dtype = torch.bfloat16
    B, Hq, Hkv, n, d, w = 1, 4, 2, 300, 64, 65
    flags = CAUSAL
    q, k, v = draw(B, Hq, Hkv, n, d, dtype, seed=21)
    dy = torch.randn(B, Hq, n, d, generator=torch.Generator().manual_seed(22)).to(dtype)
    perm, inv = sa.sa_make_perm(9, 0, B, n)
    cs, sn = sa.sa_rope_table(n, d, 10000.0)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    qr, kr = sa.sa_rope_apply(qd, kd, cs, sn), sa.sa_rope_apply(kd, qd, cs, sn, kv=True)
    y, lse = sa.sa_forward(qr, kr, vd, perm, inv, w, flags, want_lse=True)
    dq_r, dk_r, dv, _ = sa.sa_backward(qr, kr, vd, perm, inv, None, y, None, lse, None, dy.cuda(),
                                       w, flags)
    dq = sa.sa_rope_apply(dq_r, kd, cs, sn, inverse=True)
    dk = sa.sa_rope_apply(dk_r, qd, cs, sn, inverse=True, kv=True)
    pos = np.arange(n)
    rdq, rdk, rdv, _ = oracle.backward(oracle.rope(as_f64(q), pos), oracle.rope(as_f64(k), pos),
                                       as_f64(v), perm.cpu().numpy(), inv.cpu().numpy(), None,
                                       as_f64(dy), w, flags)
    close(dq, oracle.rope(rdq, pos, inverse=True), dtype, "dq")
    close(dk, oracle.rope(rdk, pos, inverse=True), dtype, "dk")
    close(dv, rdv, dtype, "dv")
