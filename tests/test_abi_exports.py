"""CPU-only checks of the boundary: the library builds, loads, exports every symbol the header
declares, and its host-side queries and argument checks behave (no kernel runs here)."""
import ctypes
import os
import re

import pytest

from paper_2510_11062_b200 import atgrpo as A
from paper_2510_11062_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return A.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "atgrpo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(atgrpo_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert len(names) >= 9
    for n in names:
        assert hasattr(lib, n), n
    assert set(A.EXPORTS) == set(names)


def test_status_strings(lib):
    texts = {A.status_string(c) for c in range(8)}
    assert len(texts) == 8 and A.status_string(99) == "unknown status"


def test_workspace_queries_are_monotone_and_aligned(lib):
    a = A.atgrpo_group_advantages_workspace_bytes(1000, 64)
    b = A.atgrpo_group_advantages_workspace_bytes(2_230_914, 262_144)
    assert 0 < a < b and a % 256 == 0 and b % 256 == 0
    f = A.atgrpo_policy_loss_workspace_bytes(16157, 2048, 151936, 1, False)
    g = A.atgrpo_policy_loss_workspace_bytes(16157, 2048, 151936, 1, True)
    assert 0 < f < g < (3 << 29)                       # two bounded chunk buffers, not T x V
    assert g < 16157 * 151936 * 2 / 3                  # a fraction of the full [T, V] dlogits
    assert A.atgrpo_policy_loss_launch_count(16157, 2048, 151936, 1, True) > \
        A.atgrpo_policy_loss_launch_count(16157, 2048, 151936, 1, False) > 0
    assert A.atgrpo_clipped_loss_workspace_bytes(4_194_304) > 0
    for bwd in (False, True):                          # degenerate sizes must not trip the planners
        assert A.atgrpo_policy_loss_workspace_bytes(0, 64, 512, 1, bwd) > 0
        assert A.atgrpo_policy_loss_workspace_bytes(1, 64, 1, 8, bwd) > 0
    assert A.atgrpo_group_advantages_workspace_bytes(0, 1) >= 0
    # the workspace-free entry point's built-in 4 MiB array holds the plan of its documented maxima
    assert A.atgrpo_group_advantages_workspace_bytes(A.NOALLOC_MAX_CAND, A.NOALLOC_MAX_GROUPS) <= 4 << 20


def test_host_side_argument_checks_need_no_gpu(lib):
    p = A.Params().c()
    rc = lib.atgrpo_group_advantages(None, None, None, None, 4, 1, 1, 1, ctypes.byref(p), None, None, None,
                                     None, None, None, None, None, 0, None)
    assert rc == A.ERR_INVALID_ARG
    rc = lib.atgrpo_group_advantages(None, None, None, None, -1, 1, 1, 1, ctypes.byref(p), None, None, None,
                                     None, None, None, None, None, 0, None)
    assert rc == A.ERR_INVALID_ARG
    rc = lib.atgrpo_clipped_loss(None, None, None, None, 0, 0, ctypes.byref(p), None, None, None, None, None, 0, None)
    assert rc == A.ERR_INVALID_ARG                     # loss pointer is required
    W = (ctypes.c_void_p * 1)(256)
    rc = lib.atgrpo_policy_loss_fwd(None, 2048, W, 9, None, None, None, 0, None, None, 0, None, 0, 2048, 1000,
                                    ctypes.byref(p), None, None, None, None, None, None, None, None, 0, None)
    assert rc == A.ERR_UNSUPPORTED                     # more heads than ATGRPO_MAX_HEADS
    rc = lib.atgrpo_policy_loss_fwd(None, 2044, W, 1, None, None, None, 0, None, None, 0, None, 0, 2044, 1000,
                                    ctypes.byref(p), None, None, None, None, None, None, None, None, 0, None)
    assert rc == A.ERR_UNSUPPORTED                     # d not a multiple of 8


def test_binding_refuses_cpu_tensors(lib):
    import torch
    t = torch.zeros(4)
    with pytest.raises(A.AtgrpoError):
        A.atgrpo_clipped_loss(t, t, t.int(), t, A.Params(), t[:1], workspace=torch.zeros(256, dtype=torch.uint8))


def test_parameter_structs_have_the_same_layout_in_c_and_in_the_binding(tmp_path):
    # compile a tiny C program against include/atgrpo.h and compare sizes and offsets with ctypes
    import subprocess
    fields_p = [f[0] for f in A._Params._fields_]
    fields_a = [f[0] for f in A._AdamWParams._fields_]
    src = tmp_path / "layout.c"
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "atgrpo.h"', 'int main(void) {',
             '  printf("%zu\\n", sizeof(atgrpo_params));']
    lines += ['  printf("%%zu\\n", offsetof(atgrpo_params, %s));' % f for f in fields_p]
    lines += ['  printf("%zu\\n", sizeof(atgrpo_adamw_params));']
    lines += ['  printf("%%zu\\n", offsetof(atgrpo_adamw_params, %s));' % f for f in fields_a]
    lines += ['  return 0;', '}']
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    got = [int(x) for x in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()]
    want = [ctypes.sizeof(A._Params)] + [getattr(A._Params, f).offset for f in fields_p] + \
           [ctypes.sizeof(A._AdamWParams)] + [getattr(A._AdamWParams, f).offset for f in fields_a]
    assert got == want
