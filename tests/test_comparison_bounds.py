"""The comparison rules of the GPU parity tests, checked on the CPU: which arrays must match bit for
bit, and how the stated tolerance of an fp32 fold / scan / scatter travels to arrays computed from it."""
import numpy as np
import pytest

from workloads import Node, Program
from helpers import TOL, compare, error_bounds, oracle_run

F32, I32 = np.float32, np.int32


def _prog():
    nodes = [Node("input", "f32", (4,), name="x"), Node("input", "i32", (3,), name="is"),
             Node("scanl", "f32", (4,), (0,), 1, fn="add", name="run"),
             Node("backpermute", "f32", (4,), (2,), 1, idx_fn="reverse", name="rev"),
             Node("gather", "f32", (3,), (1, 2), 2, name="picked"),
             Node("map", "f32", (4,), (3,), 1, fn="affine", fparam=(2.0, 1.0), name="twice")]
    return Program("bounds", nodes, [3, 4, 5])


def test_bounds_follow_index_maps():
    p = _prog()
    x, idx = np.array([1, -2, 4, 8], F32), np.array([3, 0, 0], I32)
    ref = oracle_run(p, {0: x, 1: idx})
    b = error_bounds(p, ref)
    scan_bound = TOL * np.array([1, 3, 7, 15.0]) + np.abs([1, -1, 3, 11.0]) * 2.0 ** -24    # sum|x| and the sums, by hand
    assert np.allclose(b[2], scan_bound, rtol=1e-12, atol=1e-29)
    assert np.allclose(b[3], scan_bound[::-1], rtol=1e-12, atol=1e-29)                       # reversed with the values
    assert np.allclose(b[4], scan_bound[[3, 0, 0]], rtol=1e-12, atol=1e-29)                  # picked with the values
    assert np.all(b[5] >= 2.0 * scan_bound[::-1])                                            # carried through 2x+1


def test_compare_accepts_within_and_rejects_beyond():
    p = _prog()
    x, idx = np.array([1, -2, 4, 8], F32), np.array([3, 0, 0], I32)
    ref = oracle_run(p, {0: x, 1: idx})
    good = {i: ref.values[i].copy() for i in (2, 3, 4, 5)}
    compare(p, ref, good)
    off = {i: a.copy() for i, a in good.items()}
    off[3][0] += F32(1e-3)                                # 1e-3 on a sum whose bound is 15e-5 + an ulp
    with pytest.raises(AssertionError):
        compare(p, ref, off)
    near = {i: a.copy() for i, a in good.items()}
    near[3][0] = np.nextafter(near[3][0], F32(np.inf))    # one ulp of 11: within 1e-5 * 15
    compare(p, ref, near)
