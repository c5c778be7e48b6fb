"""Pins for the node-at-a-time oracle: hand-worked examples, closed forms and
the equivalences the paper states (Section 2).  None of these re-types the
oracle's own formulas: expected values are literals, closed forms, or loops
written out here from the paper's definitions."""
import numpy as np
import pytest

import workloads as W
from workloads import Node, Program
from oracle import interp

F32, I32, U32 = np.float32, np.int32, np.uint32


def _inp(name, dtype, shape):
    return Node("input", dtype, tuple(shape), name=name)


def run(nodes, inputs):
    return interp.run(nodes, inputs).values


def test_map_worked():
    # map(\x -> 2x+1) [1,2,3] = [3,5,7]
    nodes = [_inp("x", "f32", (3,)), Node("map", "f32", (3,), (0,), 1, fn="affine", fparam=(2.0, 1.0))]
    out = run(nodes, {0: np.array([1, 2, 3], F32)})[1]
    assert out.tolist() == [3.0, 5.0, 7.0]


def test_generate_and_fold_closed_form():
    # generate(n, \i -> i) = [0..n-1]; its sum is n(n-1)/2
    nodes = [Node("generate", "i32", (4,), (), 0, fn="iota"), Node("fold", "i32", (), (0,), 1, fn="add")]
    v = run(nodes, {})
    assert v[0].tolist() == [0, 1, 2, 3] and int(v[1]) == 6
    n = 1 << 16
    nodes = [Node("generate", "i32", (n,), (), 0, fn="iota"), Node("fold", "i32", (), (0,), 1, fn="add"),
             Node("generate", "f32", (n,), (), 0, fn="iota"), Node("fold", "f32", (), (2,), 1, fn="add")]
    r = interp.run(nodes, {})
    assert int(r.values[1]) == n * (n - 1) // 2 == 2147450880
    assert r.exact[3] == float(n * (n - 1) // 2)
    assert r.abs_sum[3] == float(n * (n - 1) // 2)


def test_backpermute_reverse_and_involution():
    nodes = [_inp("x", "f32", (3,)), Node("backpermute", "f32", (3,), (0,), 1, idx_fn="reverse")]
    assert run(nodes, {0: np.array([10, 20, 30], F32)})[1].tolist() == [30.0, 20.0, 10.0]
    n = 1 << 16
    x = W.uniform_f32(0, 0, n).numpy()
    nodes = [_inp("x", "f32", (n,)), Node("backpermute", "f32", (n,), (0,), 1, idx_fn="reverse"),
             Node("backpermute", "f32", (n,), (1,), 1, idx_fn="reverse")]
    v = run(nodes, {0: x})
    assert np.array_equal(v[2], x) and np.array_equal(v[1], x[::-1])


def test_gather_worked_and_as_indexing_map():
    # gather([2,0,0,1], [10,20,30]) = [30,10,10,20]  ==  map(\i -> as!i, is)
    nodes = [_inp("is", "i32", (4,)), _inp("as", "f32", (3,)), Node("gather", "f32", (4,), (0, 1), 2)]
    is_, as_ = np.array([2, 0, 0, 1], I32), np.array([10, 20, 30], F32)
    out = run(nodes, {0: is_, 1: as_})[2]
    assert out.tolist() == [30.0, 10.0, 10.0, 20.0]
    assert out.tolist() == [float(as_[i]) for i in is_]


def test_gather_out_of_range_is_an_error():
    nodes = [_inp("is", "i32", (2,)), _inp("as", "f32", (3,)), Node("gather", "f32", (2,), (0, 1), 2)]
    with pytest.raises(IndexError):
        run(nodes, {0: np.array([0, 3], I32), 1: np.zeros(3, F32)})


def test_fold_2d_rows():
    # fold(+) [[1,2,3],[4,5,6]] = [6,15]
    nodes = [_inp("x", "f32", (2, 3)), Node("fold", "f32", (2,), (0,), 1, fn="add")]
    assert run(nodes, {0: np.array([[1, 2, 3], [4, 5, 6]], F32)})[1].tolist() == [6.0, 15.0]


def test_fold_empty_extent_rejected():
    nodes = [_inp("x", "f32", (2, 0)), Node("fold", "f32", (2,), (0,), 1, fn="add")]
    with pytest.raises(ValueError):
        run(nodes, {0: np.zeros((2, 0), F32)})


def test_scans_worked():
    # inclusive: scanl(+) [1,2,3,4] = [1,3,6,10]; scanr = [10,9,7,4]; per row in 2-D; last = fold
    x = np.array([1, 2, 3, 4], I32)
    nodes = [_inp("x", "i32", (4,)), Node("scanl", "i32", (4,), (0,), 1, fn="add"),
             Node("scanr", "i32", (4,), (0,), 1, fn="add"), Node("fold", "i32", (), (0,), 1, fn="add")]
    v = run(nodes, {0: x})
    assert v[1].tolist() == [1, 3, 6, 10] and v[2].tolist() == [10, 9, 7, 4]
    assert int(v[1][-1]) == int(v[3]) == int(v[2][0])
    nodes = [_inp("x", "f32", (2, 3)), Node("scanl", "f32", (2, 3), (0,), 1, fn="add"),
             Node("scanr", "f32", (2, 3), (0,), 1, fn="add")]
    v = run(nodes, {0: np.array([[1, 2, 3], [4, 5, 6]], F32)})
    assert v[1].tolist() == [[1, 3, 6], [4, 9, 15]] and v[2].tolist() == [[6, 5, 3], [15, 11, 6]]


def test_exclusive_seeded_scans_worked():
    # exclusive, seeded: scanl(+, seed 0) [1,2,3,4] = [0,1,3,6]; seed 10 -> [10,11,13,16]; from the right
    # [9,7,4,0]; element k is the seed combined with the inclusive scan's element before it, and the
    # inclusive scan's last element is the exclusive one's last element combined with the last input
    x = np.array([1, 2, 3, 4], I32)
    nodes = [_inp("x", "i32", (4,)),
             Node("scanl", "i32", (4,), (0,), 1, fn="add", iparam=(0,), exclusive=True),
             Node("scanl", "i32", (4,), (0,), 1, fn="add", iparam=(10,), exclusive=True),
             Node("scanr", "i32", (4,), (0,), 1, fn="add", iparam=(0,), exclusive=True),
             Node("scanl", "i32", (4,), (0,), 1, fn="add")]
    v = run(nodes, {0: x})
    assert v[1].tolist() == [0, 1, 3, 6] and v[2].tolist() == [10, 11, 13, 16] and v[3].tolist() == [9, 7, 4, 0]
    assert (v[1][1:] == v[4][:-1]).all() and int(v[1][-1]) + int(x[-1]) == int(v[4][-1])
    # per row, another operator: the running maximum of what lies to the left, seeded with -1
    nodes = [_inp("x", "f32", (2, 3)), Node("scanl", "f32", (2, 3), (0,), 1, fn="max", fparam=(-1.0,), exclusive=True)]
    v = run(nodes, {0: np.array([[1, 5, 3], [-4, -5, 6]], F32)})
    assert v[1].tolist() == [[-1, 1, 5], [-1, -1, -1]]
    # a wrapping int32 sum, seeded at the top of the range
    nodes = [_inp("x", "i32", (3,)), Node("scanl", "i32", (3,), (0,), 1, fn="add", iparam=(2**31 - 1,), exclusive=True)]
    out = interp.to_external(run(nodes, {0: np.array([1, 1, 7], I32)})[1], "i32")
    assert out.tolist() == [2**31 - 1, -2**31, -2**31 + 1]
    # the loop a cluster denotes gives the same arrays, alone and with the map fused in
    from oracle import cluster_loop, legality
    p = W.exclusive_scans(50)
    inputs = {k: t.numpy() for k, t in W.make_inputs(p).items()}
    want = interp.run(p.nodes, inputs)
    parts = legality.enumerate_partitions(p.nodes, p.outputs)
    assert len(parts) == 2
    for pi in parts:
        got = cluster_loop.run(p.nodes, p.outputs, pi, inputs)
        assert np.array_equal(got[3], want.values[3])
        assert np.allclose(got[4], want.values[4], rtol=0, atol=1e-5 * np.abs(inputs[1]).sum())


def test_scan_wraps_int32():
    nodes = [_inp("x", "i32", (2,)), Node("scanl", "i32", (2,), (0,), 1, fn="add")]
    out = interp.to_external(run(nodes, {0: np.array([2**31 - 1, 1], I32)})[1], "i32")
    assert out.tolist() == [2**31 - 1, -2**31]


def test_permute_worked_and_count_total():
    # permute(+, zeros(3), idx=[0,2,2,0,1], ones(5)) = [2,1,2]
    nodes = [_inp("d", "f32", (3,)), _inp("i", "i32", (5,)), _inp("v", "f32", (5,)),
             Node("permute", "f32", (3,), (0, 1, 2), 3, fn="add")]
    out = run(nodes, {0: np.zeros(3, F32), 1: np.array([0, 2, 2, 0, 1], I32), 2: np.ones(5, F32)})[3]
    assert out.tolist() == [2.0, 1.0, 2.0]
    # defaults are kept: dest[i] = op(dest[i], x)
    out = run(nodes, {0: np.array([5, 6, 7], F32), 1: np.array([0, 2, 2, 0, 1], I32), 2: np.ones(5, F32)})[3]
    assert out.tolist() == [7.0, 7.0, 9.0]
    n, bins = 1 << 20, 1 << 10
    idx = W.uniform_int(0, 4, n, bins).numpy()
    nodes = [_inp("d", "f32", (bins,)), _inp("i", "i32", (n,)), _inp("v", "f32", (n,)),
             Node("permute", "f32", (bins,), (0, 1, 2), 3, fn="add")]
    r = interp.run(nodes, {0: np.zeros(bins, F32), 1: idx, 2: np.ones(n, F32)})
    assert r.exact[3].sum() == n
    assert np.array_equal(r.values[3], np.bincount(idx, minlength=bins).astype(F32))
    # integer flavour, with repeated indices
    nodes = [_inp("d", "i32", (3,)), _inp("i", "i32", (4,)), _inp("v", "i32", (4,)),
             Node("permute", "i32", (3,), (0, 1, 2), 3, fn="add")]
    out = run(nodes, {0: np.array([1, 1, 1], I32), 1: np.array([1, 1, 2, 1], I32), 2: np.array([5, 6, 7, 8], I32)})[3]
    assert out.tolist() == [1, 20, 8]


def test_transpose_involution_ragged():
    R, C = 33, 65
    x = W.uniform_f32(0, 0, R * C).numpy().reshape(R, C)
    nodes = [_inp("x", "f32", (R, C)), Node("backpermute", "f32", (C, R), (0,), 1, idx_fn="transpose"),
             Node("backpermute", "f32", (R, C), (1,), 1, idx_fn="transpose")]
    v = run(nodes, {0: x})
    assert np.array_equal(v[1], x.T) and np.array_equal(v[2], x)
    assert v[1][5, 7] == x[7, 5]


def test_backpermute_is_generate_then_gather():
    n = 100
    x = W.uniform_f32(0, 0, n).numpy()
    nodes = [_inp("x", "f32", (n,)), Node("backpermute", "f32", (n,), (0,), 1, idx_fn="reverse"),
             _inp("inds", "i32", (n,)), Node("gather", "f32", (n,), (2, 0), 2)]
    inds = np.array([n - i - 1 for i in range(n)], I32)      # generate(n, \i -> n-i-1), Section 2 `reverse`
    v = run(nodes, {0: x, 2: inds})
    assert np.array_equal(v[1], v[3])


def test_map_fusion_law():
    # map f (map g xs) == map (f . g) xs, element by element
    n = 1000
    x = W.uniform_f32(0, 0, n).numpy()
    nodes = [_inp("x", "f32", (n,)), Node("map", "f32", (n,), (0,), 1, fn="affine", fparam=(2.0, 1.0)),
             Node("map", "f32", (n,), (1,), 1, fn="affine", fparam=(-0.5, 3.0))]
    out = run(nodes, {0: x})[2]
    expect = [F32(F32(F32(-0.5) * F32(F32(F32(2.0) * xi) + F32(1.0))) + F32(3.0)) for xi in x]
    assert out.tolist() == [float(e) for e in expect]


def test_fp32_chain_not_contracted():
    # a*x+b must round after the multiply; pick inputs on which a fused multiply-add would differ
    a, b = F32(1.7), F32(-1.3)
    x = W.uniform_f32(0, 0, 4096).numpy()
    nodes = [_inp("x", "f32", (4096,)), Node("map", "f32", (4096,), (0,), 1, fn="affine", fparam=(float(a), float(b)))]
    out = run(nodes, {0: x})[1]
    two_step = np.array([F32(F32(a * xi) + b) for xi in x], F32)
    fused = (np.float64(a) * x.astype(np.float64) + np.float64(b)).astype(F32)
    assert (two_step != fused).sum() > 100, "inputs must separate the two roundings"
    assert np.array_equal(out, two_step)


def test_integer_functions_worked():
    # (v*2654435761) xor (v>>13) on the uint32 view, wrap-around multiply
    v = np.array([1, 0x7FFFFFFF, 123456789], I32)
    nodes = [_inp("x", "i32", (3,)),
             Node("map", "i32", (3,), (0,), 1, fn="hash_mul_xorshift", iparam=(2654435761, 13)),
             Node("map", "i32", (3,), (1,), 1, fn="and_mask", iparam=(0xFFFF,)),
             Node("map", "u32", (3,), (0,), 1, fn="mul_mod", iparam=(40503, 65536))]
    r = run(nodes, {0: v})
    expect = [((int(t) * 2654435761) % 2**32) ^ (int(t) >> 13) for t in v]
    assert [int(t) for t in r[1]] == expect
    assert [int(t) for t in r[2]] == [e & 0xFFFF for e in expect]
    assert [int(t) for t in r[3]] == [(int(t) * 40503 % 2**32) % 65536 for t in v]
    assert expect[0] == 2654435761


def test_shift_clamp_neighbours():
    x = np.arange(12, dtype=F32).reshape(3, 4)
    mk = lambda dr, dc: Node("backpermute", "f32", (3, 4), (0,), 1, idx_fn="shift_clamp", iparam=(dr, dc))
    nodes = [_inp("x", "f32", (3, 4)), mk(-1, 0), mk(1, 0), mk(0, 1), mk(0, -1), mk(0, 0)]
    v = run(nodes, {0: x})
    assert v[1].tolist() == [[0, 1, 2, 3], [0, 1, 2, 3], [4, 5, 6, 7]]          # row above, clamped at the top
    assert v[2].tolist() == [[4, 5, 6, 7], [8, 9, 10, 11], [8, 9, 10, 11]]
    assert v[3].tolist() == [[1, 2, 3, 3], [5, 6, 7, 7], [9, 10, 11, 11]]
    assert v[4].tolist() == [[0, 0, 1, 2], [4, 4, 5, 6], [8, 8, 9, 10]]
    assert np.array_equal(v[5], x)


def test_jacobi_constant_and_impulse():
    # a constant field stays constant up to the rounding of 0.2f; a unit impulse spreads to the 5-point star
    p = W.config4(8, 8, iters=1)
    c = F32(3.0)
    out = run(p.nodes, {0: np.full((8, 8), c, F32)})[p.outputs[0]]
    expect = F32(0.2) * F32(F32(F32(F32(c + c) + c) + c) + c)
    assert np.all(out == expect)
    x = np.zeros((8, 8), F32)
    x[4, 3] = 1.0
    out = run(p.nodes, {0: x})[p.outputs[0]]
    star = {(4, 3), (3, 3), (5, 3), (4, 2), (4, 4)}
    for r in range(8):
        for cc in range(8):
            assert out[r, cc] == (F32(0.2) if (r, cc) in star else F32(0.0))
    # four chained iterations keep the total mass of an interior impulse (weights sum to one)
    p4 = W.config4(16, 16, iters=4)
    x = np.zeros((16, 16), F32)
    x[8, 8] = 1.0
    out = run(p4.nodes, {0: x})[p4.outputs[0]]
    assert abs(float(out.astype(np.float64).sum()) - 1.0) < 1e-6


def test_config2_closed_form_and_symmetry():
    n = 96
    p = W.config2(n)
    A = W.make_inputs(p)[0].numpy()
    r = interp.run(p.nodes, {0: A})
    rows = r.exact[3]
    A64 = A.astype(np.float64)
    assert abs(rows.sum() - ((A64 * A64.T).sum() + 0.5 * n * n)) < 1e-3
    C = r.values[2]
    assert np.array_equal(C, C.T)                     # a*b == b*a in fp32: C is symmetric
    assert np.allclose(rows, C.astype(np.float64).sum(axis=0), rtol=0, atol=1e-9)


def test_config5_totals():
    n, bins = 1 << 14, 1 << 8
    p = W.config5(n, bins)
    r = interp.run(p.nodes, {k: v.numpy() for k, v in W.make_inputs(p).items()})
    hist, total, frac = r.exact[4], r.exact[5], r.values[6]
    full, rem = divmod(n, 7)
    assert total == full * 21 + sum(range(rem))       # sum of i mod 7 in closed form
    assert abs(hist.sum() - total) < 1e-6
    assert abs(float(frac.astype(np.float64).sum()) - 1.0) < 1e-4
    assert r.values[2].max() < bins


def test_config3_last_scan_element_is_wrapping_fold():
    n = 1 << 12
    p = W.config3(n)
    inp = {k: v.numpy() for k, v in W.make_inputs(p).items()}
    v = run(p.nodes, inp)
    o = v[4].astype(np.uint64)
    assert int(v[5][-1]) == int(o.sum() % 2**32)
    assert int(v[4].max()) <= 0xFFFF
    # element 17 by hand, from the definitions
    x, idx = inp[0].view(U32), inp[1]
    t = int(x[idx[17]])
    assert int(v[4][17]) == ((((t * 2654435761) % 2**32) ^ (t >> 13)) & 0xFFFF)


def test_zipf_generator_range_and_head():
    keys = W.zipf_keys(0, 0, 1 << 18).numpy()
    assert keys.min() >= 0 and keys.max() < (1 << 20)
    h = sum(r ** -1.1 for r in range(1, (1 << 20) + 1))
    assert abs((keys == 0).mean() - 1.0 / h) < 0.01


def test_shape_mismatch_rejected():
    nodes = [_inp("a", "f32", (3,)), _inp("b", "f32", (4,)), Node("zipwith", "f32", (3,), (0, 1), 2, fn="add")]
    with pytest.raises(ValueError):
        run(nodes, {0: np.zeros(3, F32), 1: np.zeros(4, F32)})


def test_foldseg_worked_and_reductions_to_fold():
    # foldSeg(+) [1,2,3,4,5] with offsets [0,2,5] = [1+2, 3+4+5]; elements outside [off[0], off[-1]) are ignored
    nodes = [_inp("x", "f32", (5,)), _inp("off", "i32", (3,)),
             Node("foldseg", "f32", (2,), (0, 1), 1, fn="add"), Node("foldseg", "f32", (2,), (0, 1), 1, fn="max")]
    v = run(nodes, {0: np.array([1, 2, 3, 4, 5], F32), 1: np.array([0, 2, 5], I32)})
    assert v[2].tolist() == [3.0, 12.0] and v[3].tolist() == [2.0, 5.0]
    v = run(nodes, {0: np.array([1, 2, 3, 4, 5], F32), 1: np.array([1, 2, 4], I32)})
    assert v[2].tolist() == [2.0, 7.0]
    # one segment over everything is fold; equal segments are the row fold of the reshaped array
    n, m = 12, 7
    x = W.uniform_f32(0, 0, n * m).numpy()
    nodes = [_inp("x", "f32", (n * m,)), _inp("off", "i32", (n + 1,)), Node("foldseg", "f32", (n,), (0, 1), 1, fn="add"),
             _inp("x2", "f32", (n, m)), Node("fold", "f32", (n,), (3,), 1, fn="add"),
             _inp("one", "i32", (2,)), Node("foldseg", "f32", (1,), (0, 5), 1, fn="add"),
             Node("fold", "f32", (), (0,), 1, fn="add")]
    r = interp.run(nodes, {0: x, 1: np.arange(0, n * m + 1, m, dtype=I32), 3: x.reshape(n, m), 5: np.array([0, n * m], I32)})
    assert np.array_equal(r.exact[2], r.exact[4])
    assert abs(r.exact[6][0] - r.exact[7]) < 1e-12 and abs(r.exact[2].sum() - r.exact[7]) < 1e-9
    # integers wrap like every other integer fold
    nodes = [_inp("x", "i32", (3,)), _inp("off", "i32", (2,)), Node("foldseg", "i32", (1,), (0, 1), 1, fn="add")]
    out = interp.to_external(run(nodes, {0: np.array([2**31 - 1, 1, 5], I32), 1: np.array([0, 3], I32)})[2], "i32")
    assert out.tolist() == [-2**31 + 5]


def test_foldseg_rejects_empty_and_stray_segments():
    nodes = [_inp("x", "f32", (5,)), _inp("off", "i32", (3,)), Node("foldseg", "f32", (2,), (0, 1), 1, fn="add")]
    with pytest.raises(ValueError):
        run(nodes, {0: np.zeros(5, F32), 1: np.array([0, 2, 2], I32)})       # no seed: an empty segment has no value
    with pytest.raises(IndexError):
        run(nodes, {0: np.zeros(5, F32), 1: np.array([0, 2, 6], I32)})


def test_diagonal_of_a_product_against_matmul():
    # d[i] = sum_j A[i][j] * B[j][i] is the diagonal of the matrix product; the products are rounded to fp32
    # (one rounding of at most 2^-24 relative each), the sums carried in fp64
    p = W.diagonal_of_product(37)
    inp = {k: v.numpy() for k, v in W.make_inputs(p).items()}
    res = interp.run(p.nodes, inp)
    a, b = inp[0].astype(np.float64), inp[1].astype(np.float64)
    want = np.diag(a @ b)
    bound = 2.0 ** -24 * np.einsum("ij,ji->i", np.abs(a), np.abs(b)) + 1e-12
    assert (np.abs(res.exact[4] - want) <= bound).all()
    assert (np.abs(res.values[4] - want) <= bound + 2.0 ** -24 * np.abs(want)).all()


# ---- element functions and operators that no benchmark configuration pins -------------------------
# Expected values below are worked by hand from Section 2's definitions (generate: ys[i] = f(i);
# map: ys[i] = f(xs[i]); fold / scan / scatter with an operator other than +).  Integer cases mix
# signs so that an unsigned comparison where a signed one is meant (or the reverse) gives another answer.

def test_generate_functions_worked():
    # row_index on a 2 x 3 array: the row of every element; iota on rank 2 counts row-major
    nodes = [Node("generate", "i32", (2, 3), (), 0, fn="row_index"), Node("generate", "i32", (2, 3), (), 0, fn="iota"),
             Node("generate", "f32", (2, 3), (), 0, fn="iota")]
    v = run(nodes, {})
    assert v[0].tolist() == [[0, 0, 0], [1, 1, 1]]
    assert v[1].tolist() == [[0, 1, 2], [3, 4, 5]] and v[2].tolist() == [[0.0, 1.0, 2.0], [3.0, 4.0, 5.0]]
    # iota_plus_free: float(i) + the scalar read from a free-variable slot (element 0 of that array)
    nodes = [_inp("t", "f32", ()), Node("generate", "f32", (4,), (0,), 0, fn="iota_plus_free")]
    assert run(nodes, {0: np.array(2.5, F32)})[1].tolist() == [2.5, 3.5, 4.5, 5.5]
    assert run(nodes, {0: np.array(-1.0, F32)})[1].tolist() == [-1.0, 0.0, 1.0, 2.0]
    # imod_to_f32: float(i mod m)
    nodes = [Node("generate", "f32", (9,), (), 0, fn="imod_to_f32", iparam=(7,))]
    assert run(nodes, {})[0].tolist() == [0, 1, 2, 3, 4, 5, 6, 0, 1]


def test_unary_and_free_variable_functions_worked():
    x = np.array([1.0, 2.0, -4.0], F32)
    nodes = [_inp("x", "f32", (3,)), _inp("t", "f32", ()),
             Node("map", "f32", (3,), (0, 1), 1, fn="add_free"), Node("map", "f32", (3,), (0, 1), 1, fn="div_free"),
             Node("map", "f32", (3,), (0,), 1, fn="identity"),
             Node("zipwith", "f32", (3,), (0, 0, 2), 3, fn="add3"),
             Node("zipwith", "f32", (3,), (0, 2), 2, fn="add_scale", fparam=(0.5,))]
    v = run(nodes, {0: x, 1: np.array(0.5, F32)})
    assert v[2].tolist() == [1.5, 2.5, -3.5]                   # x + t
    assert v[3].tolist() == [2.0, 4.0, -8.0]                   # x / t
    assert v[4].tolist() == [1.0, 2.0, -4.0]
    assert v[5].tolist() == [3.5, 6.5, -11.5]                  # (x + x) + (x + t)
    assert v[6].tolist() == [1.25, 2.25, -3.75]                # 0.5 * (x + (x + t))
    # integer constants act on the 32-bit pattern and wrap
    xi = np.array([3, -2, 2**31 - 1], I32)
    nodes = [_inp("x", "i32", (3,)), Node("map", "i32", (3,), (0,), 1, fn="mul_const", iparam=(5,)),
             Node("map", "i32", (3,), (0,), 1, fn="add_const", iparam=(1,)),
             Node("map", "i32", (3,), (0,), 1, fn="add_const", iparam=(-7,)),
             Node("map", "i32", (3,), (0,), 1, fn="mul_const", iparam=(-1,))]
    v = {k: interp.to_external(a, "i32") for k, a in run(nodes, {0: xi}).items()}
    assert v[1].tolist() == [15, -10, 2147483643]              # (2^31 - 1) * 5 = 2 * 2^32 + 2147483643
    assert v[2].tolist() == [4, -1, -2**31]
    assert v[3].tolist() == [-4, -9, 2**31 - 8]
    assert v[4].tolist() == [-3, 2, -(2**31 - 1)]


def test_folds_with_other_operators_worked():
    x = np.array([[1, -2, 3], [0.5, 4, -1]], F32)
    mk = lambda op: Node("fold", "f32", (2,), (0,), 1, fn=op)
    v = run([_inp("x", "f32", (2, 3)), mk("mul"), mk("min"), mk("max")], {0: x})
    assert v[1].tolist() == [-6.0, -2.0] and v[2].tolist() == [-2.0, -1.0] and v[3].tolist() == [3.0, 4.0]
    xi = np.array([[-3, 2, 7], [5, -1, -8]], I32)
    mk = lambda op: Node("fold", "i32", (2,), (0,), 1, fn=op)
    v = {k: interp.to_external(a, "i32") for k, a in run([_inp("x", "i32", (2, 3)), mk("mul"), mk("min"), mk("max")], {0: xi}).items()}
    assert v[1].tolist() == [-42, 40]
    assert v[2].tolist() == [-3, -8]                           # compared as unsigned patterns these would be 2 and 5
    assert v[3].tolist() == [7, 5]                             # ... and these -3 and -1
    # the same bit patterns declared unsigned compare the other way round
    mk = lambda op: Node("fold", "u32", (2,), (0,), 1, fn=op)
    v = run([_inp("x", "u32", (2, 3)), mk("min"), mk("max")], {0: xi.view(U32)})
    assert v[1].tolist() == [2, 5] and v[2].tolist() == [2**32 - 3, 2**32 - 1]
    # products wrap: 65536 * 65536 = 2^32 -> 0; 65536 * 32768 = 2^31 -> the most negative int32
    v = run([_inp("x", "i32", (2, 2)), Node("fold", "i32", (2,), (0,), 1, fn="mul")],
            {0: np.array([[65536, 65536], [65536, 32768]], I32)})
    assert interp.to_external(v[1], "i32").tolist() == [0, -2**31]
    # a whole-array fold of a rank-1 array gives a scalar
    v = run([_inp("x", "i32", (4,)), Node("fold", "i32", (), (0,), 1, fn="min")], {0: np.array([4, -9, 0, 3], I32)})
    assert int(interp.to_external(v[1], "i32")) == -9


def test_scans_with_other_operators_worked():
    xi = np.array([3, -1, 2, -5, 0], I32)
    mk = lambda kind, op, dt="i32": Node(kind, dt, (5,), (0,), 1, fn=op)
    v = {k: interp.to_external(a, "i32") for k, a in
         run([_inp("x", "i32", (5,)), mk("scanl", "min"), mk("scanl", "max"), mk("scanr", "min"), mk("scanr", "max"),
              mk("scanl", "mul")], {0: xi}).items()}
    assert v[1].tolist() == [3, -1, -1, -5, -5]
    assert v[2].tolist() == [3, 3, 3, 3, 3]
    assert v[3].tolist() == [-5, -5, -5, -5, 0]
    assert v[4].tolist() == [3, 2, 2, 0, 0]
    assert v[5].tolist() == [3, -3, -6, 30, 0]
    # running maximum that starts negative (an unsigned comparison would keep -4 forever)
    v = run([_inp("x", "i32", (4,)), Node("scanl", "i32", (4,), (0,), 1, fn="max")], {0: np.array([-4, -2, -3, 1], I32)})
    assert interp.to_external(v[1], "i32").tolist() == [-4, -2, -2, 1]
    # unsigned: 2^31 is large, not negative
    xu = np.array([1, 2**31, 5], U32)
    v = run([_inp("x", "u32", (3,)), Node("scanl", "u32", (3,), (0,), 1, fn="max"), Node("scanl", "u32", (3,), (0,), 1, fn="min")], {0: xu})
    assert v[1].tolist() == [1, 2**31, 2**31] and v[2].tolist() == [1, 1, 1]
    v = run([_inp("x", "i32", (3,)), Node("scanl", "i32", (3,), (0,), 1, fn="max")], {0: xu.view(I32)})
    assert interp.to_external(v[1], "i32").tolist() == [1, 1, 5]
    # fp32: product, minimum and maximum, per row, both directions
    xf = np.array([[0.5, 4, -1], [2, -3, 0.25]], F32)
    mk = lambda kind, op: Node(kind, "f32", (2, 3), (0,), 1, fn=op)
    v = run([_inp("x", "f32", (2, 3)), mk("scanl", "mul"), mk("scanl", "min"), mk("scanr", "max"), mk("scanr", "mul")], {0: xf})
    assert v[1].tolist() == [[0.5, 2.0, -2.0], [2.0, -6.0, -1.5]]
    assert v[2].tolist() == [[0.5, 0.5, -1.0], [2.0, -3.0, -3.0]]
    assert v[3].tolist() == [[4.0, 4.0, -1.0], [2.0, 0.25, 0.25]]
    assert v[4].tolist() == [[-2.0, -4.0, -1.0], [-1.5, -0.75, 0.25]]


def test_scatters_with_other_operators_worked():
    def scatter(dt, op, dest, idx, vals):
        np_dt = F32 if dt == "f32" else (I32 if dt == "i32" else U32)
        nodes = [_inp("d", dt, (len(dest),)), _inp("i", "i32", (len(idx),)), _inp("v", dt, (len(vals),)),
                 Node("permute", dt, (len(dest),), (0, 1, 2), 3, fn=op)]
        out = run(nodes, {0: np.array(dest, np_dt), 1: np.array(idx, I32), 2: np.array(vals, np_dt)})[3]
        return interp.to_external(out, dt).tolist()
    # dest[i] = op(dest[i], x) for every (i, x); untouched bins keep their defaults
    assert scatter("i32", "min", [10, 10, 10], [0, 0, 2, 2], [-3, 4, 11, 12]) == [-3, 10, 10]
    assert scatter("i32", "max", [10, 10, 10], [0, 0, 2, 2], [-3, 4, 11, 12]) == [10, 10, 12]
    assert scatter("i32", "max", [-1, -1], [0, 1], [-2, 3]) == [-1, 3]        # unsigned: -1 would beat 3
    assert scatter("i32", "min", [-1, -1], [0, 1], [-2, 3]) == [-2, -1]
    assert scatter("u32", "max", [1, 1], [0, 1, 1], [2**31, 0, 7]) == [2**31, 7]
    assert scatter("u32", "min", [2**32 - 1, 9], [0, 1, 1], [2**31, 12, 7]) == [2**31, 7]
    assert scatter("i32", "mul", [2, 3], [0, 0, 1], [5, -1, 4]) == [-10, 12]
    assert scatter("f32", "min", [1.0, 1.0], [0, 1, 1], [0.5, 2.0, -3.0]) == [0.5, -3.0]
    assert scatter("f32", "max", [1.0, 1.0], [0, 1, 1], [0.5, 2.0, -3.0]) == [1.0, 2.0]
    assert scatter("f32", "mul", [1.0, 1.0], [0, 1, 1], [0.5, 2.0, -3.0]) == [0.5, -6.0]
    with pytest.raises(IndexError):
        scatter("i32", "min", [0, 0], [0, 2], [1, 1])
