"""Host-side checks that need no GPU: the library loads, exports what include/sa.h
declares, sizes workspaces, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

from paper_2604_00754_b200 import binding as sa

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_functions():
    text = open(os.path.join(ROOT, "include", "sa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sa_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = sa.load_library()
    names = header_functions()
    assert set(sa.EXPORTS) == set(names)
    for name in names:
        assert getattr(lib, name) is not None


def problem(**kw):
    base = dict(B=2, Hq=4, Hkv=2, n=100, d=64, w=9, dtype=sa.BF16, flags=sa.CAUSAL)
    base.update(kw)
    p = sa.SaProblem(**base)
    sa.load_library().sa_problem_set_contiguous(ctypes.byref(p))
    return p


def test_contiguous_strides_and_workspace_sizes():
    p = problem()
    assert list(p.q_stride) == [4 * 100 * 64, 100 * 64, 64]
    assert list(p.kv_stride) == [2 * 100 * 64, 100 * 64, 64]
    assert sa.sa_workspace_bytes(p, sa.OP_FORWARD) == 0
    assert sa.sa_workspace_bytes(p, sa.OP_MAKE_PERM) >= 2 * 100 * (8 + 4) * 2
    assert sa.sa_workspace_bytes(p, sa.OP_BACKWARD) >= 2 * 2 * 4 * 100 * 4
    with pytest.raises(sa.SaError):
        sa.sa_workspace_bytes(problem(Hq=5), sa.OP_FORWARD)
    with pytest.raises(sa.SaError):
        sa.sa_workspace_bytes(p, 99)


FAKE = ctypes.c_void_p(0x1000)      # aligned, never dereferenced: every case fails before a launch
ODD = ctypes.c_void_p(0x1004)


@pytest.mark.parametrize("kw,expect", [
    (dict(Hq=5), 1), (dict(n=0), 1), (dict(w=0), 1), (dict(dtype=7), 1), (dict(flags=1024), 1),
    (dict(flags=sa.SWA_ONE_SIDED), 1), (dict(d=20), 2), (dict(d=512), 2),
    (dict(softmax_scale=-1.0), 1),
])
def test_forward_rejects_bad_problem(kw, expect):
    lib = sa.load_library()
    p = problem(**kw)
    st = lib.sa_forward(ctypes.byref(p), FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, None, 0, None)
    assert st == expect


def test_null_and_misaligned_pointers_are_rejected():
    lib = sa.load_library()
    p = problem()
    assert lib.sa_forward(ctypes.byref(p), None, FAKE, FAKE, FAKE, FAKE, FAKE, None, None, 0, None) == 1
    assert lib.sa_forward(ctypes.byref(p), FAKE, FAKE, ODD, FAKE, FAKE, FAKE, None, None, 0, None) == 1
    assert lib.sa_forward(None, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, None, 0, None) == 1
    assert lib.sa_swa_forward(ctypes.byref(p), FAKE, FAKE, FAKE, None, None, None, 0, None) == 1
    args = [FAKE] * 12
    args[5] = None      # gate logits
    assert lib.sa_swa_gated_forward(ctypes.byref(p), *args, 0, None) == 1
    p2 = problem(flags=sa.CAUSAL | sa.SAVE_FOR_BWD)
    args = [FAKE] * 12
    args[8] = None      # y_swa missing although saving was asked for
    assert lib.sa_swa_gated_forward(ctypes.byref(p2), *args, 0, None) == 1
    assert lib.sa_make_perm(1, 0, 0, 16, FAKE, FAKE, FAKE, 1 << 20, None) == 1
    assert lib.sa_make_perm(1, 0, 1, 16, FAKE, None, FAKE, 1 << 20, None) == 1
    assert lib.sa_coverage(1, 16, 0, 0, FAKE, FAKE, 0, FAKE, None, FAKE, FAKE, 1 << 20, None) == 1
    assert lib.sa_coverage(1, 16, 4, 0, FAKE, FAKE, 16, FAKE, None, FAKE, FAKE, 1 << 20, None) == 1


def test_short_workspace_is_rejected():
    lib = sa.load_library()
    assert lib.sa_make_perm(1, 0, 2, 1000, FAKE, FAKE, FAKE, 16, None) == 3
    p = problem()
    args = [FAKE] * 16
    assert lib.sa_backward(ctypes.byref(p), *args, 16, None) == 3
    assert lib.sa_coverage(2, 1000, 4, 0, FAKE, FAKE, 0, FAKE, None, FAKE, FAKE, 16, None) == 3


def test_status_strings():
    assert sa.status_string(0) == "ok"
    assert "workspace" in sa.status_string(3)
    assert "permutation" in sa.status_string(5)


def test_debug_hooks_validate_their_arguments():
    lib = sa.load_library()
    assert lib.sa_debug_set(99, 0) == 1
    assert lib.sa_debug_set(sa.DEBUG_SCORE_BLOCK, 96) == 1
    assert lib.sa_debug_set(sa.DEBUG_TENSOR_CORES, 2) == 1
    for key, default in ((sa.DEBUG_SCORE_BLOCK, 0), (sa.DEBUG_SWA_TILE_LOADS, 1),
                         (sa.DEBUG_TENSOR_CORES, 1), (sa.DEBUG_GATE_WIDE_TILES, 1)):
        assert lib.sa_debug_set(key, default) == 0
    assert lib.sa_debug_wait_timeout(0, None) == 1          # rejected before any launch
    assert lib.sa_debug_wait_timeout(1 << 40, None) == 1


def test_library_reads_no_environment_variable():
    # kernel choice must not depend on the environment: no getenv in the sources
    csrc = os.path.join(ROOT, "paper_2604_00754_b200", "csrc")
    for name in os.listdir(csrc):
        assert "getenv" not in open(os.path.join(csrc, name)).read(), name


def test_stale_library_is_not_loaded_when_the_rebuild_fails(tmp_path, monkeypatch):
    from paper_2604_00754_b200 import build as b
    monkeypatch.setattr(sa, "_lib", None)
    monkeypatch.setattr(b, "stale", lambda: True)

    def fail(*a, **k):
        raise OSError("no compiler")
    monkeypatch.setattr(b, "build_library", fail)
    with pytest.raises(RuntimeError, match="older than its sources"):
        sa.load_library()
