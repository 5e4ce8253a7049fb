"""The no-allocation variant of the permutation call against the ordinary one.

sa_make_perm_static exists for callers that are not allowed to allocate device memory (code
running while someone else owns the allocator, or inside a loop that must stay clear of the
driver's memory manager): its sort scratch is a fixed array inside the library instead of a
caller-supplied workspace.  Its result has to be identical to sa_make_perm's, and because
every call reuses the same array with whatever the previous call left in it, the check runs
on two calls in a row with different sizes, seeds and layers.  This file sorts last on
purpose so that a run that stops at the first failure has already run everything else.
"""
import pytest
import torch

from paper_2604_00754_b200 import binding as sa

pytestmark = pytest.mark.gpu


def both(seed, layer, B, n):
    want_perm, want_inv = sa.sa_make_perm(seed, layer, B, n)
    perm = torch.full((B, n), -1, dtype=torch.int32, device="cuda")
    inv = torch.full((B, n), -1, dtype=torch.int32, device="cuda")
    sa.sa_make_perm_static(seed, layer, B, n, perm, inv)
    return perm, inv, want_perm, want_inv


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    # second call is smaller and differently shaped, so it runs over the first call's leftovers
    for seed, layer, B, n in [(7, 3, 2, 50000), (0xDEADBEEFCAFEF00D, 47, 3, 2049)]:
        perm, inv, want_perm, want_inv = both(seed, layer, B, n)
        assert torch.equal(perm, want_perm)       # integer work: bit-exact
        assert torch.equal(inv, want_inv)
    assert sa.sa_read_status() == 0


def test_static_scratch_largest_and_too_large():
    perm, inv, want_perm, want_inv = both(11, 0, 1, 131072)
    assert torch.equal(perm, want_perm) and torch.equal(inv, want_inv)
    B, n = 2, 131072                               # needs more than the 4 MiB built in: refused
    out = torch.empty(B, n, dtype=torch.int32, device="cuda")
    with pytest.raises(sa.SaError) as e:
        sa.sa_make_perm_static(1, 0, B, n, out, torch.empty_like(out))
    assert e.value.status == 7
    assert "built in" in str(e.value)
