"""The allocation-free prefix sum `acc_scanl_add_i32_static` against the regular path.

Some users of the library call it from places where device memory cannot be allocated
(a plug-in that only receives raw pointers, a process whose device memory is handed out
completely up front).  For them the scan's tile states live in a fixed array inside
the library.  That array is shared by all calls and keeps its old contents, so the test
calls the entry point several times in a row, with different data and lengths, and requires
each result to equal what `acc_run` computes for the same input with a caller-provided
workspace, and what the CPU oracle computes for it (both paths share a kernel, so their
agreement alone would prove little): bit for bit, as for every integer result in this suite.

This file sorts last on purpose: a run that stops at the first failure has then already
exercised every other test.
"""
import numpy as np
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


def oracle_scan(x):
    """The same prefix sum by the oracle's interpreter (wrapping int32 adds, Section 2's scanl)."""
    from oracle import interp
    n = x.numel()
    nodes = [Node("input", "i32", (n,), name="x"), Node("scanl", "i32", (n,), (0,), 1, fn="add", name="out")]
    return interp.to_external(interp.run(nodes, {0: x.cpu().numpy()}).values[1], "i32")


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
        assert np.array_equal(got.cpu().numpy(), oracle_scan(x)), (seed, n)
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
