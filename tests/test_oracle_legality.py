"""Pins for the oracle's legality model: the graph and clusterings the paper
prints for `scatterExample`, the legal/illegal examples of Section 3.3, the
consequences of Figure 3 that can be derived by hand, and hand-counted numbers
of legal clusterings for the small programs."""
import os

import pytest

import workloads as W
from workloads import Node
from oracle import legality as L

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "scatter_example_graph.txt")


def _inp(name, dtype="f32", shape=(8,)):
    return Node("input", dtype, tuple(shape), name=name)


def _parse_golden():
    names, F, I, clusterings = [], set(), set(), []
    for line in open(GOLDEN):
        t = line.split()
        if not t or t[0] == "#":
            continue
        if t[0] == "N":
            names = t[1:]
        elif t[0] in "FI":
            (F if t[0] == "F" else I).update(tuple(e.split(">")) for e in t[1:])
        elif t[0] == "clustering":
            blocks = " ".join(t[1:]).split("|")
            clusterings.append([sorted(b.strip().split(",")) for b in blocks])
    return names, F, I, clusterings


def test_scatter_example_graph_matches_paper():
    names, F, I, clusterings = _parse_golden()
    p = W.scatter_example_paper_graph()
    gF, gI = L.graph_sets(p.nodes)
    nm = lambda s: {(p.nodes[a].name, p.nodes[b].name) for a, b in s}
    assert [nd.name for nd in p.nodes] == names and len(p.nodes) == 4
    assert nm(gF) == F and nm(gI) == I
    legal = L.enumerate_partitions(p.nodes, p.outputs)
    as_blocks = []
    for pi in legal:
        blocks = {}
        for i, c in enumerate(pi):
            if c >= 0:
                blocks.setdefault(c, []).append(p.nodes[i].name)
        as_blocks.append([sorted(blocks[c]) for c in sorted(blocks)])
    # exactly the two drawn clusterings plus "nothing fused"
    for cl in clusterings:
        assert cl in as_blocks
    assert len(legal) == 3
    assert [["as"], ["bs"], ["result"]] in as_blocks


def test_scatter_dest_and_result_edges_are_infusible():
    p = W.scatter_example_paper_graph()
    # bs (the destination) in the scatter's cluster is illegal, so is everything in one cluster
    assert not L.check(p.nodes, p.outputs, [-1, 0, 1, 1])[0]
    assert not L.check(p.nodes, p.outputs, [-1, 0, 0, 0])[0]
    # bs must come before the scatter, not after
    assert not L.check(p.nodes, p.outputs, [-1, 0, 2, 1])[0]
    # a consumer of the scatter result cannot share its cluster
    nodes = p.nodes + [Node("map", "i32", (8,), (3,), 1, fn="identity", name="after")]
    assert L.check(nodes, [4], [-1, 0, 0, 1, 2])[0]
    assert not L.check(nodes, [4], [-1, 0, 0, 1, 1])[0]


def test_scatter_temporal_uniqueness():
    # another reader of the destination must run strictly before the scatter
    nodes = [_inp("xs", "i32"),
             Node("map", "i32", (8,), (0,), 1, fn="identity", name="as"),
             Node("map", "i32", (8,), (0,), 1, fn="add_const", iparam=(1,), name="bs"),
             Node("map", "i32", (8,), (2,), 1, fn="identity", name="peek"),
             Node("permute", "i32", (8,), (2, 1, 1), 3, fn="add", name="result")]
    assert L.check(nodes, [3, 4], [-1, 0, 0, 1, 2])[0]
    assert not L.check(nodes, [3, 4], [-1, 0, 0, 2, 1])[0]      # peek after the scatter
    assert not L.check(nodes, [3, 4], [-1, 0, 0, 1, 1])[0]      # peek beside the scatter


def test_simple1_2_4_5_fuse_into_one_cluster():
    for prog in (W.simple1(), W.simple2(), W.simple4(), W.simple5(), W.single_loop()):
        pi = [-1 if nd.kind == "input" else 0 for nd in prog.nodes]
        ok, why = L.check(prog.nodes, prog.outputs, pi)
        assert ok, (prog.name, why)


def test_simple3_cannot_be_one_cluster():
    # `as` is a program output and the source of the gather: its order would be the gather's label
    p = W.simple3()
    assert not L.check(p.nodes, p.outputs, [-1, -1, 0, 0])[0]
    assert L.check(p.nodes, p.outputs, [-1, -1, 0, 1])[0]
    assert len(L.enumerate_partitions(p.nodes, p.outputs)) == 1


def test_scan_never_fuses_into_a_gather_source():
    nodes = [_inp("is", "i32"), _inp("xs"),
             Node("scanl", "f32", (8,), (1,), 1, fn="add", name="sc"),
             Node("gather", "f32", (8,), (0, 2), 2, name="g")]
    assert not L.check(nodes, [3], [-1, -1, 0, 0])[0]
    assert L.check(nodes, [3], [-1, -1, 0, 1])[0]
    # but a scan may be fed by a gather, and may feed a map, in one cluster
    nodes = [_inp("is", "i32"), _inp("xs"),
             Node("gather", "f32", (8,), (0, 1), 2, name="g"),
             Node("scanl", "f32", (8,), (2,), 1, fn="add", name="sc"),
             Node("map", "f32", (8,), (3,), 1, fn="identity", name="m")]
    assert L.check(nodes, [4], [-1, -1, 0, 0, 0])[0]


def test_scanl_and_scanr_do_not_share_a_read():
    nodes = [_inp("x"), Node("scanl", "f32", (8,), (0,), 1, fn="add"), Node("scanr", "f32", (8,), (0,), 1, fn="add")]
    assert not L.check(nodes, [1, 2], [-1, 0, 0])[0]
    assert L.check(nodes, [1, 2], [-1, 0, 1])[0]
    # a map can join either of them: its free order follows the scan it shares the read with
    nodes.append(Node("map", "f32", (8,), (0,), 1, fn="identity"))
    assert L.check(nodes, [1, 2, 3], [-1, 0, 1, 1])[0]
    assert L.check(nodes, [1, 2, 3], [-1, 0, 1, 0])[0]
    assert not L.check(nodes, [1, 2, 3], [-1, 0, 0, 0])[0]
    # a scanr fused after a scanl would need order 0 == 1
    nodes = [_inp("x"), Node("scanl", "f32", (8,), (0,), 1, fn="add"), Node("scanr", "f32", (8,), (1,), 1, fn="add")]
    assert not L.check(nodes, [2], [-1, 0, 0])[0]


def test_two_gather_like_consumers_force_a_manifest_array():
    # an array read by two backpermutes can be fused with neither, unless it has a single consumer
    nodes = [_inp("x"), Node("map", "f32", (8,), (0,), 1, fn="identity", name="y"),
             Node("backpermute", "f32", (8,), (1,), 1, idx_fn="reverse", name="b1"),
             Node("backpermute", "f32", (8,), (1,), 1, idx_fn="identity", name="b2")]
    assert not L.check(nodes, [2, 3], [-1, 0, 0, 0])[0]
    assert not L.check(nodes, [2, 3], [-1, 0, 0, 1])[0]
    # b1 and b2 read y in two different labels: no shared read, so they do not hang together either
    assert not L.check(nodes, [2, 3], [-1, 0, 1, 1])[0]
    assert L.check(nodes, [2, 3], [-1, 0, 1, 2])[0]


def test_independent_loops_do_not_share_a_cluster():
    nodes = [_inp("a"), _inp("b"), Node("map", "f32", (8,), (0,), 1, fn="identity"),
             Node("map", "f32", (8,), (1,), 1, fn="identity")]
    assert not L.check(nodes, [2, 3], [-1, -1, 0, 0])[0]
    nodes[3] = Node("map", "f32", (8,), (0,), 1, fn="identity")
    assert L.check(nodes, [2, 3], [-1, -1, 0, 0])[0]       # horizontal fusion over input a


def test_free_variable_and_force_edges():
    nodes = [_inp("x"), Node("fold", "f32", (), (0,), 1, fn="add", name="t"),
             Node("map", "f32", (8,), (0, 1), 1, fn="div_free", name="m")]
    assert not L.check(nodes, [2], [-1, 0, 0])[0]
    assert L.check(nodes, [2], [-1, 0, 1])[0]
    nodes = [_inp("x"), Node("map", "f32", (8,), (0,), 1, fn="identity"),
             Node("map", "f32", (8,), (1,), 1, fn="identity", force=(0,))]
    assert not L.check(nodes, [2], [-1, 0, 0])[0]
    assert L.check(nodes, [2], [-1, 0, 1])[0]


def test_counts_of_legal_clusterings():
    # hand-derived: a chain of k fusible edges has 2^k; config 5 has ten (see the case list in the test body)
    assert len(L.enumerate_partitions(W.config1(8).nodes, [4])) == 8
    assert len(L.enumerate_partitions(W.config2(4).nodes, [3])) == 4
    assert len(L.enumerate_partitions(W.config3(8).nodes, [5])) == 8
    p = W.config5(16, 4)
    legal = L.enumerate_partitions(p.nodes, p.outputs)
    k, vals, hist, total, frac = 2, 3, 4, 5, 6
    groups = set()
    for pi in legal:
        blocks = {}
        for i in (k, vals, hist, total, frac):
            blocks.setdefault(pi[i], set()).add(i)
        assert blocks[pi[frac]] == {frac}                 # two infusible in-edges keep frac alone
        groups.add(frozenset(frozenset(b) for b in blocks.values() if len(b) > 1))
    fs = lambda *bs: frozenset(frozenset(b) for b in bs)
    assert groups == {
        fs(), fs({k, hist}), fs({vals, hist}), fs({vals, total}), fs({hist, total}),
        fs({k, hist}, {vals, total}), fs({k, hist, vals}), fs({k, hist, total}),
        fs({vals, hist, total}), fs({k, vals, hist, total})}
    assert len(legal) == 10


def test_config4_needs_one_cluster_per_iteration():
    p = W.config4(8, 8, iters=2)
    per_iter = [-1] + [0] * 9 + [1] * 9
    assert L.check(p.nodes, p.outputs, per_iter)[0]
    assert not L.check(p.nodes, p.outputs, [-1] + [0] * 18)[0]
    # pulling the second iteration's centre read into the first cluster pins Y0 to that label
    bad = list(per_iter)
    bad[10] = 0
    assert not L.check(p.nodes, p.outputs, bad)[0]
    unfused = [-1] + list(range(18))
    assert L.check(p.nodes, p.outputs, unfused)[0]


def test_greedy_trap_programs_optima_are_legal():
    p = W.greedy_bottom_up_bad(4, 5)
    # is, large and both folds in one cluster; result afterwards (it indexes zs)
    assert L.check(p.nodes, p.outputs, [-1, 0, 0, 0, 0, 1])[0]
    # once ys sits with result, zs must precede them and `large` cannot be contracted
    assert L.check(p.nodes, p.outputs, [-1, 0, 0, 1, 0, 1])[0]
    assert not L.check(p.nodes, p.outputs, [-1, 0, 0, 0, 0, 0])[0]
    q = W.greedy_top_down_bad(16)
    assert L.check(q.nodes, q.outputs, [-1, 0, 1, 1, 1, 1])[0]       # cs fused vertically into es
    assert L.check(q.nodes, q.outputs, [-1, 0, 0, 1, 1, 1])[0]       # cs fused diagonally with bs
    assert not L.check(q.nodes, q.outputs, [-1, 0, 0, 0, 0, 0])[0]   # ds indexes bs


def test_traffic_counts_shared_and_separate_reads():
    p = W.config1(8)
    assert L.traffic(p.nodes, p.outputs, [-1, 0, 1, 2, 3]) == (5, 4)   # x, y, z+x, w read; 4 arrays written
    assert L.traffic(p.nodes, p.outputs, [-1, 0, 0, 0, 0]) == (2, 1)   # x in two orders; only s written
    q = W.simple5()
    assert L.traffic(q.nodes, q.outputs, [-1, -1, 0, 0, 0]) == (3, 1)  # is, xs in order 0, xs in the label


# ---- clusterings that recompute (an extension: Section 6 leaves duplicated work to future work) ----

def _two_orders():
    # ys is read as it lies (by zs) and reversed (by bp): the pattern of Section 3.3's `simple5`
    return [_inp("xs"),
            Node("map", "f32", (8,), (0,), 1, fn="affine", fparam=(2.0, 1.0), name="ys"),
            Node("backpermute", "f32", (8,), (1,), 1, idx_fn="reverse", name="bp"),
            Node("zipwith", "f32", (8,), (2, 1), 2, fn="add", name="zs")]


def test_recompute_lets_one_array_be_read_in_two_orders():
    nodes = _two_orders()
    # the paper's model: ys must be stored before bp reads it, so only {bp, zs} can fuse
    assert L.enumerate_partitions(nodes, [3]) == [[-1, 0, 1, 1], [-1, 0, 1, 2]]
    # with one copy of ys per order, ys fuses into bp (its stored copy still serves zs), and all
    # three share a cluster; {ys, zs} without bp stays impossible (bp lies between them)
    assert L.enumerate_partitions(nodes, [3], recompute=1) == [[-1, 0, 0, 0], [-1, 0, 0, 1], [-1, 0, 1, 1], [-1, 0, 1, 2]]
    assert not L.check(nodes, [3], [-1, 0, 1, 0], recompute=1)[0]


def test_recompute_does_not_change_what_is_not_about_orders():
    # a scan can still not be produced in a gather's order
    nodes = [_inp("is", "i32"), _inp("xs"),
             Node("scanl", "f32", (8,), (1,), 1, fn="add", name="sc"),
             Node("gather", "f32", (8,), (0, 2), 2, name="g")]
    assert not L.check(nodes, [3], [-1, -1, 0, 0], recompute=2)[0]
    # nor a stored array in both scan orders at once
    nodes = [_inp("x"), Node("scanl", "f32", (8,), (0,), 1, fn="add"), Node("scanr", "f32", (8,), (0,), 1, fn="add"),
             Node("zipwith", "f32", (8,), (1, 2), 2, fn="add")]
    assert not L.check(nodes, [3], [-1, 0, 0, 0], recompute=2)[0]
    # infusible edges, the execution order and the scatter rule are as before
    p = W.scatter_example(16)
    strict = L.enumerate_partitions(p.nodes, p.outputs)
    assert L.enumerate_partitions(p.nodes, p.outputs, recompute=2) == strict
    for prog in (W.config1(64), W.config3(64), W.config5(256, 16)):
        assert L.enumerate_partitions(prog.nodes, prog.outputs, recompute=2) == L.enumerate_partitions(prog.nodes, prog.outputs)


def test_recompute_copies_a_shared_producer_for_each_scan_direction():
    # m feeds a scanl and a scanr: one order for m is impossible, one copy per scan is fine
    nodes = [_inp("x"), Node("map", "f32", (8,), (0,), 1, fn="identity", name="m"),
             Node("scanl", "f32", (8,), (1,), 1, fn="add"), Node("scanr", "f32", (8,), (1,), 1, fn="add")]
    assert not L.check(nodes, [2, 3], [-1, 0, 0, 0])[0]
    assert L.check(nodes, [2, 3], [-1, 0, 0, 0], recompute=1)[0]


def test_recompute_depth_bounds_stacked_stencil_iterations():
    p = W.config4(4, 4, iters=3)
    one = [-1] + [0] * 27
    two_one = [-1] + [0] * 18 + [1] * 9
    assert not L.check(p.nodes, p.outputs, two_one)[0]                      # the paper's model: one iteration each
    assert not L.check(p.nodes, p.outputs, two_one, recompute=1)[0]        # two shifts stacked
    assert L.check(p.nodes, p.outputs, two_one, recompute=2)[0]
    assert not L.check(p.nodes, p.outputs, one, recompute=2)[0]
    assert L.check(p.nodes, p.outputs, one, recompute=3)[0]
    # a cut inside an iteration ({c, n, s, t1, t2} | {e, w, t3, Y}) is as legal as before
    cut = [-1, 0, 0, 0, 1, 1, 0, 0, 1, 1] + [2] * 18
    assert not L.check(p.nodes, p.outputs, cut)[0] and L.check(p.nodes, p.outputs, cut, recompute=2)[0]
    cut = [-1, 0, 0, 0, 1, 1, 0, 0, 1, 1] + [2] * 9 + [3] * 9
    assert L.check(p.nodes, p.outputs, cut)[0] and L.check(p.nodes, p.outputs, cut, recompute=1)[0]


def test_recomputing_clusters_compute_the_same_arrays():
    import numpy as np
    from oracle import cluster_loop, interp
    nodes = _two_orders()
    x = np.linspace(-1, 1, 8).astype(np.float32)
    want = interp.run(nodes, {0: x}).values[3]
    np.testing.assert_array_equal(want, (2 * x + 1)[::-1] + (2 * x + 1))     # worked by hand
    for pi in L.enumerate_partitions(nodes, [3], recompute=1):
        got = cluster_loop.run(nodes, [3], pi, {0: x})
        assert np.array_equal(got[3].view(np.uint32), want.view(np.uint32)), pi
    p = W.config4(5, 6, iters=2)
    x = W.make_inputs(p)[0].numpy()
    want = interp.run(p.nodes, {0: x}).values[p.outputs[0]]
    got = cluster_loop.run(p.nodes, p.outputs, [-1] + [0] * 18, {0: x})
    assert np.array_equal(got[p.outputs[0]].view(np.uint32), want.view(np.uint32))


# ---- nodes copied into further clusters ----

def test_a_copy_lets_the_total_regenerate_its_values():
    import numpy as np
    from oracle import cluster_loop, interp
    p = W.config5(64, 8)                                    # keys, zeros, k, vals, hist, total, frac
    pi = [-1, -1, 0, 0, 0, 1, 2]
    # without the copy, `vals` (3) is stored for `total`; with a copy of it in cluster 1 nothing reads the stored one
    nodes2, outputs2, pi2, home, copy_ids = L.unfold_copies(p.nodes, p.outputs, pi, [(3, 1)])
    assert len(nodes2) == len(p.nodes) + 1 and pi2[copy_ids[(3, 1)]] == 1
    assert nodes2[home[5]].inputs == (copy_ids[(3, 1)],) and nodes2[home[4]].inputs[2] == home[3]
    assert L.check_with_copies(p.nodes, p.outputs, pi, [(3, 1)])[0]
    edges = L.edges_of(nodes2)
    assert home[3] not in L.manifest_set(nodes2, outputs2, pi2, edges)
    assert 3 in L.manifest_set(p.nodes, p.outputs, pi, L.edges_of(p.nodes))
    # the arrays are those of the program itself
    inputs = {k: t.numpy() for k, t in W.make_inputs(p).items()}
    want = interp.run(p.nodes, inputs)
    got = cluster_loop.run(nodes2, outputs2, pi2, {home[k]: v for k, v in inputs.items()})
    for o in p.outputs:
        assert np.allclose(got[home[o]], want.values[o], rtol=1e-6, atol=0)
    # what a copy cannot be: of an input, in the node's own cluster, without a reader, or a scatter's result
    assert not L.check_with_copies(p.nodes, p.outputs, pi, [(0, 1)])[0]
    assert not L.check_with_copies(p.nodes, p.outputs, pi, [(3, 0)])[0]
    assert not L.check_with_copies(p.nodes, p.outputs, pi, [(3, 2)])[0]          # nobody in cluster 2 reads vals
    assert not L.check_with_copies(p.nodes, p.outputs, pi, [(4, 2)])[0]          # frac reads hist through an infusible edge: not inside one cluster
