"""Host-to-host forward: the head grouping (CPU) and, on a GPU, that the pipelined path gives
the bits of the single device-resident call."""
import pytest
import torch

from paper_2604_00754_b200 import binding as sab
from paper_2604_00754_b200 import host


def test_head_groups_cover_every_head_once():
    for Hq, Hkv, ng in [(32, 8, 8), (32, 8, 3), (12, 12, 5), (4, 1, 8), (16, 4, 1)]:
        groups = sab.host_forward_plan(Hq, Hkv, ng, 1)
        assert len(groups) <= max(1, min(ng, Hkv))
        G = Hq // Hkv
        kv_seen, q_seen = [], []
        for ka, kb, qa, qb, with_kv in groups:
            assert kb > ka and (qa, qb) == (ka * G, kb * G) and with_kv
            kv_seen += list(range(ka, kb))
            q_seen += list(range(qa, qb))
        assert kv_seen == list(range(Hkv)) and q_seen == list(range(Hq))


def test_split_query_heads_keeps_coverage_and_kv_ownership():
    # the first and the last KV head are cut by query heads, the ones in between stay whole
    g = sab.host_forward_plan(32, 8, 8, 2)
    assert [x[2:4] for x in g] == [(0, 2), (2, 4)] + [(4 * i, 4 * i + 4) for i in range(1, 7)] + \
        [(28, 30), (30, 32)]
    assert [x[4] for x in g] == [True, False] + [True] * 6 + [True, False]   # K/V with the first part
    assert all(kb - ka == 1 for ka, kb, *_ in g)
    g = sab.host_forward_plan(32, 8, 8, 4)
    assert len(g) == 14 and [x[2:4] for x in g][-4:] == [(28, 29), (29, 30), (30, 31), (31, 32)]
    assert sab.host_forward_plan(4, 1, 1, 2) == [(0, 1, 0, 2, True), (0, 1, 2, 4, False)]
    # ranges with several KV heads, or an odd number of query heads per KV head, stay whole
    assert sab.host_forward_plan(8, 4, 2, 2) == [(0, 2, 0, 4, True), (2, 4, 4, 8, True)]
    assert sab.host_forward_plan(3, 1, 1, 2) == [(0, 1, 0, 3, True)]


def test_head_groups_rejects_bad_head_counts():
    with pytest.raises(ValueError):
        sab.host_forward_plan(10, 4, 2, 1)
    with pytest.raises(ValueError):
        sab.host_forward_plan(0, 1, 1, 1)


def test_host_forward_rejects_bad_arguments_before_any_cuda_call():
    import ctypes
    lib = sab.load_library()
    p = sab.SaProblem(B=1, Hq=4, Hkv=2, n=64, d=64, w=8, dtype=sab.BF16, flags=sab.CAUSAL)
    need = sab.host_forward_ws_bytes(1, 4, 2, 64, 64)
    assert need >= (3 * 4 + 2 * 2) * 64 * 64 * 2       # q, y, scratch + k, v
    fake = ctypes.c_void_p(0x10000)
    args = lambda ws, nbytes: (ctypes.byref(p), fake, fake, fake, fake, fake, 1, 0, 2, 1, ws,
                               nbytes, None)
    assert lib.sa_swa_gated_forward_host(*args(None, need)) == 1
    assert lib.sa_swa_gated_forward_host(*args(ctypes.c_void_p(0x10010), need)) == 1   # alignment
    assert lib.sa_swa_gated_forward_host(*args(fake, need - 1)) == 3


@pytest.mark.gpu
@pytest.mark.parametrize("n_groups,q_parts", [(1, 1), (3, 2), (4, 2), (4, 1)])
def test_pipelined_forward_equals_single_call(n_groups, q_parts):
    from paper_2604_00754_b200 import binding as sa
    B, Hq, Hkv, n, d, w = 2, 8, 4, 1000, 64, 256
    g = torch.Generator().manual_seed(11)
    q = torch.randn(B, Hq, n, d, generator=g).bfloat16().pin_memory()
    k = torch.randn(B, Hkv, n, d, generator=g).bfloat16().pin_memory()
    v = torch.randn(B, Hkv, n, d, generator=g).bfloat16().pin_memory()
    lg = torch.randn(2, Hq, generator=g).pin_memory()
    hy = torch.empty_like(q).pin_memory()
    hf = host.HostForward(B, Hq, Hkv, n, d, w, n_groups=n_groups, q_parts=q_parts)
    hf.forward(q, k, v, lg, hy, seed=5, layer=2)
    torch.cuda.synchronize()
    perm, inv = sa.sa_make_perm(5, 2, B, n)
    # the pipeline hands the library scratch, so its gates are applied by the idle-warp
    # kernel: the single call does the same (the fused epilogue rounds differently)
    scratch = torch.empty(hy.numel() * hy.element_size(), dtype=torch.uint8, device="cuda")
    ref = sa.sa_swa_gated_forward(q.cuda(), k.cuda(), v.cuda(), perm, inv, lg.cuda(), w, ws=scratch)
    assert sa.sa_read_status() == 0
    assert torch.equal(hy, ref.cpu())
    # a second call with another layer index draws another permutation
    hf.forward(q, k, v, lg, hy, seed=5, layer=3)
    torch.cuda.synchronize()
    perm, inv = sa.sa_make_perm(5, 3, B, n)
    ref = sa.sa_swa_gated_forward(q.cuda(), k.cuda(), v.cuda(), perm, inv, lg.cuda(), w, ws=scratch)
    assert torch.equal(hy, ref.cpu())
