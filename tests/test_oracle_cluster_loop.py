"""The oracle's two evaluators against each other and against the loops the
paper prints: for every legal clustering of the small programs, the loop that
the clusters denote must produce the arrays of the node-at-a-time interpreter
(bit for bit on integers and fp32 element chains)."""
import numpy as np
import pytest

import workloads as W
from oracle import interp, legality, cluster_loop

F32 = np.float32


def npin(p):
    return {k: v.numpy() for k, v in W.make_inputs(p).items()}


def downstream_of_fp_accumulation(nodes):
    acc = set()
    for i, nd in enumerate(nodes):
        if (nd.kind in ("fold", "foldseg", "scanl", "scanr", "permute") and nd.dtype == "f32") or any(s in acc for s in nd.inputs):
            acc.add(i)
    return acc


def agree_everywhere(p, max_partitions=None):
    inp = npin(p)
    ref = interp.run(p.nodes, inp)
    loose = downstream_of_fp_accumulation(p.nodes)
    legal = legality.enumerate_partitions(p.nodes, p.outputs)
    assert legal
    for pi in legal[:max_partitions]:
        mem = cluster_loop.run(p.nodes, p.outputs, pi, inp)
        man = legality.manifest_set(p.nodes, p.outputs, pi, legality.edges_of(p.nodes))
        assert set(mem) == man
        for k, v in mem.items():
            a = ref.values[k].reshape(-1)
            if k in loose:
                assert np.allclose(a, v.reshape(-1), rtol=2e-7, atol=0), (p.name, pi, k)
            else:
                assert np.array_equal(a, v.reshape(-1)), (p.name, pi, k)
    return len(legal)


@pytest.mark.parametrize("prog,count", [
    (W.config1(200), 8), (W.config2(9), 4), (W.config3(128), 8), (W.config5(300, 16), 10),
    (W.scatter_example(24), None), (W.single_loop(33), None), (W.simple1(), 2), (W.simple2(), 2),
    (W.simple3(), 1), (W.simple4(), 2), (W.simple5(), None), (W.greedy_bottom_up_bad(3, 5), None),
    (W.greedy_top_down_bad(17), None), (W.config4(5, 6, iters=1), None), (W.segmented_sums(200, 9), None),
    (W.scan_consumers(41), None), (W.scan_consumers(7, 3), None), (W.offsets_then_gather(64), 20), (W.histogram_2d(4, 16, 8), 10), (W.fold_of_scan(33), None)])
def test_both_evaluators_agree_on_every_legal_clustering(prog, count):
    n = agree_everywhere(prog, max_partitions=40)
    if count is not None:
        assert n == count


@pytest.mark.parametrize("seed", range(14))
def test_both_evaluators_agree_on_random_programs(seed):
    # seeded random DAGs of element-wise nodes, reversals, gathers, folds, scans and scatters, rank 1 and rank 2
    agree_everywhere(W.random_program(seed, 37), max_partitions=60)
    agree_everywhere(W.random_program(seed, 9, 4), max_partitions=30)
    agree_everywhere(W.random_int_program(seed, 37), max_partitions=40)
    agree_everywhere(W.random_int_program(seed, 9, 4), max_partitions=30)
    agree_everywhere(W.random_int_program(seed + 10, 6, 6), max_partitions=30)      # square: with transposes
    agree_everywhere(W.random_scan_program(seed, 37), max_partitions=40)            # a scan in the middle, with readers
    agree_everywhere(W.random_scan_program(seed, 9, 4), max_partitions=30)


def test_config1_full_size_all_clusterings():
    assert agree_everywhere(W.config1(1 << 16)) == 8


def test_paper_loop_simple1():
    p = W.simple1()
    inp = npin(p)
    is_, xs = inp[0], inp[1]
    bs = np.empty(len(is_), F32)
    for j in range(len(is_)):
        i = is_[j]
        x = xs[i]
        a = F32(F32(F32(2.0) * x) + F32(1.0))
        bs[j] = a
    assert np.array_equal(interp.run(p.nodes, inp).values[3], bs)


def test_paper_loop_simple2():
    p = W.simple2()
    inp = npin(p)
    is1, is2, xs = inp[0], inp[1], inp[2]
    bs = np.empty(len(is2), F32)
    for i in range(len(is2)):
        i2 = is2[i]
        i1 = is1[i2]
        bs[i] = xs[i1]
    assert np.array_equal(interp.run(p.nodes, inp).values[4], bs)


def test_paper_loop_simple4():
    p = W.simple4()
    inp = npin(p)
    is_, xs = inp[0], inp[1]
    m, n = xs.shape
    flat = xs.reshape(-1)
    bs = np.empty(len(is_), np.float64)
    for i in range(len(is_)):
        i3 = int(is_[i]) * n
        a = float(flat[i3])
        for j in range(1, n):
            a = a + float(flat[i3 + j])
        bs[i] = a
    got = interp.run(p.nodes, inp).values[3]
    assert np.allclose(got, bs.astype(F32), rtol=2e-7, atol=0)


def test_paper_loop_simple5():
    p = W.simple5()
    inp = npin(p)
    is_, xs = inp[0], inp[1]
    cs = np.empty(len(xs), F32)
    for i in range(min(len(is_), len(xs))):
        x = xs[i]
        a = F32(F32(F32(-1.5) * x) + F32(0.25))
        b = xs[is_[i]]
        cs[i] = a * b
    assert np.array_equal(interp.run(p.nodes, inp).values[4], cs)


def test_single_loop_is_one_traversal():
    # Section 1: reverse, two maps and a zipWith3 in one loop that reads `as` in two orders
    p = W.single_loop(33)
    inp = npin(p)
    a = inp[0]
    n = len(a)
    res = np.empty(n, F32)
    for i in range(n):
        b = a[n - 1 - i]
        c = F32(F32(F32(3.0) * a[i]) + F32(-1.0))
        d = F32(F32(F32(0.5) * c) + F32(2.0))
        res[i] = F32(F32(b + c) + d)
    mem = cluster_loop.run(p.nodes, p.outputs, [-1, 0, 0, 0, 0], inp)
    assert np.array_equal(mem[4], res)
    assert set(mem) == {0, 4}                          # no intermediate array is written
