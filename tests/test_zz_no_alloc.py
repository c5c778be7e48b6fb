"""The allocation-free prefix sum `acc_scanl_add_i32_static` against the regular path.

Some users of the library call it from places where device memory cannot be allocated
(a serving loop that must not hit cudaMalloc's device-wide synchronisation, a plug-in that
only receives raw pointers).  For them the scan's tile states live in a fixed array inside
the library.  That array is shared by all calls and keeps its old contents, so the test
calls the entry point twice in a row, with different data and lengths, and requires each
result to equal what `acc_run` computes for the same input with a caller-provided
workspace: bit for bit, as for every integer result in this suite.

This file sorts last on purpose: a run that stops at the first failure has then already
exercised every other test.
"""
import pytest

import workloads as W
from workloads import Node

pytestmark = pytest.mark.gpu


def regular_scan(x):
    """Inclusive int32 prefix sum through acc_run (one scan node, workspace from torch)."""
    import torch
    from paper_2407_13585_b200 import binding as B
    n = x.numel()
    nodes = [Node("input", "i32", (n,), name="x"), Node("scanl", "i32", (n,), (0,), 1, fn="add", name="out")]
    g = B.Graph(nodes, [1])
    out = torch.empty(n, dtype=torch.int32, device="cuda")
    g.bind(0, x)
    g.bind(1, out)
    g.run(B.UNFUSED)
    return out


def test_static_scan_matches_regular_scan_twice_in_a_row():
    import torch
    from paper_2407_13585_b200 import binding as B
    # first call: many tiles, vector path; second call: fewer tiles, ragged length, scalar path.
    # The second call would see the first call's tile states if the entry point did not clear them.
    for seed, n in ((1, (1 << 20) + 4096), (2, 300001), (3, 8)):
        x = W.uniform_int(seed, 0, n, 1 << 31, device="cuda")
        got = torch.full((n,), -7, dtype=torch.int32, device="cuda")
        B.scanl_add_i32_static(x, got)
        want = regular_scan(x)
        assert torch.equal(got, want), (seed, n)
    # and the same input again gives the same answer
    B.scanl_add_i32_static(x, got)
    assert torch.equal(got, want)


def test_static_scan_refuses_what_its_array_cannot_hold():
    import ctypes
    from paper_2407_13585_b200 import binding as B
    too_many = (1 << 26) + 1
    rc = B.lib().acc_scanl_add_i32_static(ctypes.c_void_p(256), ctypes.c_void_p(512), too_many, None)
    assert B.STATUS_NAME[rc] == "ACC_ERR_TOO_LARGE"
    assert "at most" in B.lib().acc_last_error().decode()
    assert B.lib().acc_scanl_add_i32_static(None, None, 0, None) == 0          # nothing to do, nothing touched
