"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the
same seeded inputs, element by element, under every legal clustering of the small
programs and under the unfused executor.  Sizes span several tiles and a ragged tail."""
import numpy as np
import pytest

import workloads as W
from helpers import all_partitions, compare, gpu_run, oracle_run

pytestmark = pytest.mark.gpu


def np_inputs(inputs_t):
    return {k: v.cpu().numpy() for k, v in inputs_t.items()}


def check_program(prog, partitions="all", runs=1, passes=False, inputs_t=None):
    from paper_2407_13585_b200 import binding as B
    inputs_t = W.make_inputs(prog) if inputs_t is None else inputs_t
    ref = oracle_run(prog, np_inputs(inputs_t))
    got, g = gpu_run(prog, inputs_t, None, B.UNFUSED)
    # one launch per combinator; a segmented fold takes a second, small one for the segments that cross its blocks
    assert g.launch_count() == sum((nd.kind != "input") + (nd.kind == "foldseg") for nd in prog.nodes)
    passes = passes or any(nd.kind == "foldseg" for nd in prog.nodes)
    compare(prog, ref, got, f"{prog.name} unfused")
    pis = all_partitions(prog) if partitions == "all" else partitions
    for pi in pis:
        got, g = gpu_run(prog, inputs_t, pi, B.FUSED, runs=runs)
        # passes: a cluster with roots that no one kernel walks together takes one launch per group of them
        clusters = len({c for c in pi if c >= 0})
        assert g.launch_count() >= clusters if passes else g.launch_count() == clusters
        compare(prog, ref, got, f"{prog.name} pi={pi}")
    return len(pis)


# several tiles plus a ragged tail; multiples of four (128-bit path) and not (scalar path)
@pytest.mark.parametrize("n", [1, 3, 4, 31, 1024, 4099, 70000, 1 << 16])
def test_config1_all_partitions(n):
    assert check_program(W.config1(n)) == 8


# below one 64 x 64 tile: generic kernels; from 64 rows on: shared-memory tile pairs, with ragged
# edge tiles (100, 130), without 128-bit accesses (130, 67: the threads stage the tiles; otherwise
# tensor copies do) and on whole tiles (64, 256); 1600 and 2052 give every persistent block
# several tile pairs, 2052 with an edge tile that lies almost wholly outside the array
@pytest.mark.parametrize("rows", [1, 4, 33, 64, 67, 100, 130, 256, 1600, 2052])
def test_config2_all_partitions(rows):
    assert check_program(W.config2(rows)) == 4


@pytest.mark.parametrize("n", [1, 4, 64, 4096, 8192, 1 << 17])
def test_config3_all_partitions(n):
    assert check_program(W.config3(n)) == 8


# one gather stored with a map of it and a map of its indices beside it: lengths the 128-bit paths take and not
@pytest.mark.parametrize("n", [1, 1000, 4099, 1 << 16])
def test_gather_with_three_roots_all_partitions(n):
    assert check_program(W.gather_three_roots(5000, n)) == 4


def test_config3_ragged_lengths():
    # lengths that are not powers of two: the scan's last tile is partial, the scalar path runs
    for n in (5, 4097, 12289 + 3):
        prog = W.config3(n)
        prog.name = "fixture"                     # generic index inputs bounded by n
        prog.index_bound = {"idx": n, "x": 1 << 30}
        check_program(prog)


# small domains run the streaming kernel; from about 600k cells on, clusters of clamped shifts run on
# halo tiles copied by the tensor-copy engine: whole tiles (1024^2) and ragged ones (1000 x 1028)
@pytest.mark.parametrize("rows,cols", [(1, 4), (3, 5), (8, 8), (33, 64), (64, 33), (130, 260), (1024, 1024), (1000, 1028)])
def test_config4_iteration_cuts(rows, cols):
    prog = W.config4(rows, cols, iters=2)
    per_iter = [-1] + [0] * 9 + [1] * 9
    cuts = [per_iter]
    # {c,n,t1}, the other shifts alone, {t2,t3,Y}
    cuts.append([-1, 0, 0, 1, 2, 3, 0, 4, 4, 4] + [c + 5 for c in (0, 0, 1, 2, 3, 0, 4, 4, 4)])
    # shifts alone, the four sums fused
    cuts.append([-1, 0, 1, 2, 3, 4, 5, 5, 5, 5] + [c + 6 for c in (0, 1, 2, 3, 4, 5, 5, 5, 5)])
    check_program(prog, cuts)


# Several Jacobi iterations per kernel (a clustering that recomputes: the iterate in between is
# read in five orders).  Small domains are pulled through per read by the streaming kernel, from
# 64 tiles on the iterates in between stay in shared memory; ragged edges in both directions,
# tiles that lie on two array edges at once, depth 2 to 4.  Bit-exact like every element chain.
@pytest.mark.parametrize("rows,cols,iters,depth", [
    (8, 8, 2, 2), (40, 64, 4, 2), (33, 36, 3, 3),
    (512, 1024, 4, 2), (520, 1028, 4, 2), (4100, 132, 2, 2), (64, 8192, 2, 2),
    (515, 1028, 3, 3), (512, 1024, 4, 3), (520, 1036, 4, 4),
])
def test_config4_recomputing_clusters(rows, cols, iters, depth):
    from paper_2407_13585_b200 import binding as B
    prog = W.config4(rows, cols, iters=iters)
    g = B.Graph(prog.nodes, prog.outputs)
    assert g.plan("greedy_topdown", "bytes") == [-1] + [t for t in range(iters) for _ in range(9)]
    pi = g.plan_recompute("greedy_topdown", "bytes", depth)
    n_clusters = len({c for c in pi if c >= 0})
    assert n_clusters == -(-iters // depth)
    assert g.check_partition(pi) == "ACC_ERR_ILLEGAL_TRAVERSAL"        # not a clustering of the paper's model
    inputs_t = W.make_inputs(prog)
    ref = oracle_run(prog, np_inputs(inputs_t))
    got, g2 = gpu_run(prog, inputs_t, pi, B.FUSED, recompute=depth, runs=2)
    assert g2.launch_count() == n_clusters
    compare(prog, ref, got, f"config4 {rows}x{cols} depth {depth}")


def test_config4_four_iterations_planned():
    from paper_2407_13585_b200 import binding as B
    prog = W.config4(96, 128, iters=4)
    g = B.Graph(prog.nodes, prog.outputs)
    for mode in ("greedy_topdown", "greedy_bottomup"):
        pi = g.plan(mode)
        assert len({c for c in pi if c >= 0}) == 4        # one cluster per iteration is the legal minimum
        check_program(prog, [pi])


# few elements per bin: atomics on global accumulators; many: bins in one CTA's shared memory
# (up to 56 Ki), with a private overflow slice in global memory (2^16 bins), or split over a
# group of two (100000 bins) or four (3 * 2^16 bins) CTAs
@pytest.mark.parametrize("n,bins", [(1, 1), (7, 4), (1000, 16), (4096, 256), (100003, 1 << 10), (1 << 18, 1 << 16),
                                    (1 << 20, 1 << 16), (3 << 19, 50000), (1 << 20, 100000), (3 << 20, 3 << 16)])
def test_config5_all_partitions(n, bins):
    assert check_program(W.config5(n, bins)) == 10


# seeded random DAGs (element-wise nodes, reversals, gathers; folds, scans, a scatter and a map of a fold's
# result at the leaves) under every legal clustering: one element, a ragged length over several tiles, a
# length the 128-bit paths take
@pytest.mark.parametrize("n", [1, 4099, 70000])
@pytest.mark.parametrize("seed", [0, 2, 3, 5, 7, 8])
def test_random_programs_all_partitions(seed, n):
    check_program(W.random_program(seed, n), passes=True)


@pytest.mark.parametrize("rows,n", [(3, 5), (37, 300), (64, 1024)])
@pytest.mark.parametrize("seed", [0, 3, 5, 8])
def test_random_rank2_programs_all_partitions(seed, rows, n):
    check_program(W.random_program(seed, n, rows), passes=True)


# the integer counterparts (wrapping arithmetic, generated arrays, clamped shifts by up to three cells, folds,
# scans and scatters with +, min and max): every array bit for bit
@pytest.mark.parametrize("n", [1, 4099, 70000])
@pytest.mark.parametrize("seed", [1, 3, 4, 5, 8, 10, 11])
def test_random_integer_programs_all_partitions(seed, n):
    check_program(W.random_int_program(seed, n), passes=True)


@pytest.mark.parametrize("rows,n", [(3, 5), (37, 300), (64, 1024), (520, 1284)])
@pytest.mark.parametrize("seed", [2, 3, 4, 5, 7, 10])
def test_random_integer_rank2_programs_all_partitions(seed, rows, n):
    check_program(W.random_int_program(seed, n, rows), passes=True)


# square arrays, so that transposes join in: below one 64 x 64 tile, ragged tiles without 128-bit rows, whole tiles
@pytest.mark.parametrize("rows", [5, 70, 256])
@pytest.mark.parametrize("seed", [3, 7, 14, 23, 39])
def test_random_integer_square_programs_all_partitions(seed, rows):
    check_program(W.random_int_program(seed, rows, rows), passes=True)


# scans consumed element for element inside their cluster (a map of a running sum, offsets used as indices):
# the consumers are evaluated where the scanned values are final; several scans per cluster take a pass each
@pytest.mark.parametrize("n", [1, 5, 4099, 4096 * 3, 70000])
def test_scans_consumed_inside_their_cluster(n):
    assert check_program(W.scan_consumers(n), passes=True) == 152


@pytest.mark.parametrize("rows,n", [(3, 5), (37, 300), (16, 8192)])
def test_row_scans_consumed_inside_their_cluster(rows, n):
    assert check_program(W.scan_consumers(n, rows), passes=True) == 152


@pytest.mark.parametrize("n", [1, 4, 4096, 1 << 17])
def test_offsets_used_as_indices_in_the_same_cluster(n):
    assert check_program(W.offsets_then_gather(n), passes=True) == 20


def test_a_plan_without_kernels_is_refined_and_runs():
    from paper_2407_13585_b200 import binding as B
    for n in (1, 4099, 70000):
        prog = W.fold_of_scan(n)
        g = B.Graph(prog.nodes, prog.outputs)
        g.plan("enumerate", "bytes")
        splits, pi = g.refine_to_kernels()
        assert (splits, pi) == (1, [-1, 0, 1])
        check_program(prog, [pi])


def test_equal_addends_stay_within_tolerance():
    # rounding errors of a running fp32 sum cancel on random data and pile up when every addend is the same
    # number: the per-thread sums are compensated, so long folds, row folds, segmented folds and scans of a
    # constant still meet 1e-5 * sum|x|; so is a scan's chain of tile prefixes (4096 tiles here), carried as two floats
    import torch
    from paper_2407_13585_b200 import binding as B

    def constant(prog, value=0.1):
        inputs = W.make_inputs(prog)
        return {i: (torch.full_like(t, value) if t.dtype == torch.float32 else t) for i, t in inputs.items()}

    for prog in (W.config1(1 << 22), W.greedy_bottom_up_bad(4, 1 << 20), W.segmented_sums(1 << 20, 16),
                 W.scan_consumers(1 << 24), W.scan_consumers(1 << 20, 4)):
        g = B.Graph(prog.nodes, prog.outputs)
        pi = g.plan("enumerate", "bytes")
        check_program(prog, [pi], passes=True, inputs_t=constant(prog))
    # a whole-array fold beside a scatter with on-chip bins (the kernel config 5's diamond runs in), fed from memory:
    # hist = permute(+) zeros (hash keys) vals and total = fold(+) vals share a kernel through their common input
    from workloads import Node, Program
    n, bins = 1 << 24, 1 << 10
    nodes = [Node("input", "u32", (n,), name="keys"), Node("input", "f32", (bins,), name="zeros"), Node("input", "f32", (n,), name="vals"),
             Node("map", "u32", (n,), (0,), 1, fn="mul_mod", iparam=(40503, bins), name="k"),
             Node("permute", "f32", (bins,), (1, 3, 2), 3, fn="add", name="hist"),
             Node("fold", "f32", (), (2,), 1, fn="add", name="total")]
    prog = Program("weighted_histogram_with_total", nodes, [4, 5])
    inputs = {0: W.zipf_keys(0, 0, n), 1: torch.zeros(bins), 2: torch.full((n,), 0.1)}
    check_program(prog, [[-1, -1, -1, 0, 1, 1]], inputs_t=inputs)


# random DAGs around a scan in the middle.  Clusterings in which something other than an element-wise chain reads
# the scan inside its cluster (a reversal, a fold, a second scan) have no kernel: the run must say so, not guess
def around_a_scan(prog):
    from paper_2407_13585_b200 import binding as B
    from paper_2407_13585_b200 import instantiate
    built, missing = [], []
    for pi in all_partitions(prog):
        blocks = {}
        for i, c in enumerate(pi):
            if c >= 0:
                blocks.setdefault(c, set()).add(i)
        (built if all(instantiate.expressible(prog, b) for b in blocks.values()) else missing).append(pi)
    assert built
    check_program(prog, built, passes=True)
    inputs_t = W.make_inputs(prog)
    for pi in missing:
        with pytest.raises(B.AccError) as err:
            gpu_run(prog, inputs_t, pi, B.FUSED)
        assert err.value.status == "ACC_ERR_NO_KERNEL"
    return len(missing)


@pytest.mark.parametrize("n", [1, 4099, 70000])
@pytest.mark.parametrize("seed", [1, 3, 4, 7, 10, 13, 14])
def test_random_programs_around_a_scan(seed, n):
    assert (around_a_scan(W.random_scan_program(seed, n)) > 0) == (seed in (4, 7, 10, 14))


@pytest.mark.parametrize("rows,n", [(3, 5), (37, 1024)])
@pytest.mark.parametrize("seed", [4, 7, 12])
def test_random_rank2_programs_around_a_scan(seed, rows, n):
    around_a_scan(W.random_scan_program(seed, n, rows))


# a scatter histogram over rank-2 keys beside per-row totals: few elements per bin (atomics on global accumulators)
# and many (bins in shared memory, also with the private overflow slice); fused with the row folds, the scatter
# and the folds take a pass each
@pytest.mark.parametrize("rows,n,bins", [(1, 1, 1), (3, 5, 4), (37, 300, 16), (64, 4096, 256), (256, 4096, 1 << 16)])
def test_rank2_histogram_beside_row_totals(rows, n, bins):
    assert check_program(W.histogram_2d(rows, n, bins), passes=True) == 10


def test_launches_count_the_passes_of_a_cluster():
    from paper_2407_13585_b200 import binding as B
    # {s, m, z, e, t}: two scans, a pass each; {r, q}: one kernel
    prog = W.scan_consumers(4099)
    _, g = gpu_run(prog, W.make_inputs(prog), [-1, -1, 0, 0, 0, 1, 1, 0, 0], B.FUSED)
    assert g.launch_count() == 3
    # everything in one cluster on a rank-2 domain: the row folds, then the scatter
    prog = W.histogram_2d(37, 300, 16)
    _, g = gpu_run(prog, W.make_inputs(prog), [-1, -1, 0, 0, 0, 0], B.FUSED)
    assert g.launch_count() == 2
    # whole-array folds and a scatter share the streaming kernel: config 5 fused stays one launch (+ the map of the total)
    prog = W.config5(1 << 15, 256)
    g0 = B.Graph(prog.nodes, prog.outputs)
    pi = g0.plan("enumerate", "bytes")
    _, g = gpu_run(prog, W.make_inputs(prog), pi, B.FUSED)
    assert g.launch_count() == len({c for c in pi if c >= 0})


def test_runs_are_repeatable():
    # a racy fold, scan or scatter would differ between runs; integer outputs must be identical
    check_program(W.config3(1 << 16), runs=3)
    check_program(W.config5(1 << 16, 256), runs=3)


def test_end_to_end_with_host_buffers():
    # acc_run_e2e: pinned host inputs in, program, host outputs out; then two programs enqueued on two
    # streams with acc_run_e2e_async and waited for afterwards (their copies may overlap)
    import torch
    from paper_2407_13585_b200 import binding as B

    def prepare(prog):
        g = B.Graph(prog.nodes, prog.outputs)
        g.plan("enumerate", "bytes")
        inputs = W.make_inputs(prog)
        host = {}
        for i, t in inputs.items():
            g.bind(i, torch.empty_like(t, device="cuda"))          # device copy filled by the call
            host[i] = t.contiguous().pin_memory()
            g.bind_host(i, host[i])
        for o in prog.outputs:
            nd = prog.nodes[o]
            n = max(int(np.prod(nd.shape, dtype=np.int64)) if nd.shape else 1, 4)
            g.bind(o, torch.empty(n, dtype=torch.int32, device="cuda"))
            host[o] = torch.full((n,), -7, dtype=torch.int32).pin_memory()
            g.bind_host(o, host[o])
        return g, inputs, host

    def check(prog, inputs, host, what):
        ref = oracle_run(prog, np_inputs(inputs))
        got = {}
        for o in prog.outputs:
            nd = prog.nodes[o]
            n = int(np.prod(nd.shape, dtype=np.int64)) if nd.shape else 1
            a = host[o][:n].numpy()
            got[o] = (a.view(np.float32) if nd.dtype == "f32" else a.view(np.uint32)).reshape(tuple(nd.shape))
        compare(prog, ref, got, what)

    p3, p5 = W.config3(1 << 18), W.config5(1 << 18, 1 << 10)
    g3, in3, h3 = prepare(p3)
    up, down = g3.run_e2e(B.FUSED)
    assert up == 2 * 4 * (1 << 18) and down == 4 * (1 << 18)
    check(p3, in3, h3, "config3 end to end")
    g5, in5, h5 = prepare(p5)
    h3[p3.outputs[0]].fill_(-7)
    lanes = [torch.cuda.Stream(), torch.cuda.Stream()]
    for lane, g in zip(lanes, (g3, g5)):
        with torch.cuda.stream(lane):
            g.run_e2e(B.FUSED, finish=False)
    for lane, g in zip(lanes, (g3, g5)):
        with torch.cuda.stream(lane):
            g.finish()
    check(p3, in3, h3, "config3 end to end, enqueued")
    check(p5, in5, h5, "config5 end to end, enqueued")


PAPER_EXAMPLES = [W.scatter_example(64), W.single_loop(100), W.simple1(), W.simple2(), W.simple4(), W.simple5(),
                  W.greedy_bottom_up_bad(16, 100), W.greedy_top_down_bad(1000)]


@pytest.mark.parametrize("prog", PAPER_EXAMPLES, ids=lambda p: p.name)
def test_paper_examples_all_partitions(prog):
    # the programs the paper prints (Sections 1, 3.3, 3.4, 5), under every legal clustering:
    # gathers pushed through maps, gathers and a fold; a scatter fed by fused maps; two folds sharing a gather
    assert check_program(prog) >= 2


def test_empty_arrays_run():
    # element-wise clusters over zero elements are legal no-ops (a fold over nothing is rejected when built)
    prog = W.config4(0, 8, iters=1)
    check_program(prog, [[-1] + [0] * 9])


def test_scatter_out_of_range_is_reported():
    import torch
    from paper_2407_13585_b200 import binding as B
    prog = W.config5(1024, 16)
    g = B.Graph(prog.nodes, prog.outputs)
    g.plan("enumerate")
    # break the hash's modulus so that indices leave the 16 bins: the kernel must skip and report, not write
    bad = W.config5(1024, 16)
    bad.nodes[2].iparam = (40503, 64)
    g = B.Graph(bad.nodes, bad.outputs)
    g.plan("enumerate")
    inputs = W.make_inputs(bad)
    bufs = [inputs[0].cuda(), inputs[1].cuda(), torch.zeros(16, device="cuda"), torch.zeros(1, device="cuda"),
            torch.zeros(16, device="cuda")]
    g.bind(0, bufs[0]); g.bind(1, bufs[1]); g.bind(4, bufs[2]); g.bind(5, bufs[3]); g.bind(6, bufs[4])
    with pytest.raises(B.AccError) as e:
        g.run()
    assert e.value.status == "ACC_ERR_INDEX_RANGE"


def _weighted_histogram(n, bins):
    """keys, zeros, vals as inputs; k = hash keys; hist = permute(+) zeros k vals."""
    from workloads import Node, Program
    nodes = [Node("input", "u32", (n,), name="keys"), Node("input", "f32", (bins,), name="zeros"),
             Node("input", "f32", (n,), name="vals"),
             Node("map", "u32", (n,), (0,), 1, fn="mul_mod", iparam=(40503, bins), name="k"),
             Node("permute", "f32", (bins,), (1, 3, 2), 3, fn="add", name="hist")]
    return Program("weighted_histogram", nodes, [4])


@pytest.mark.parametrize("flavour", ["floats", "dyadic", "outliers", "one_hot_bin"])
def test_scatter_add_of_arbitrary_fp32_values(flavour):
    # the on-chip histogram adds multiples of its quantum as integers and everything else in fp64:
    # random floats (mostly the fp64 route), signed multiples of 1/8 (integer route), a few huge,
    # tiny, infinite values among them, and one bin hit by every element (bins spill into fp64)
    import torch
    from paper_2407_13585_b200 import binding as B
    n, bins = 1 << 20, 4096
    prog = _weighted_histogram(n, bins)
    keys = W.zipf_keys(3, 0, n)
    defaults = W.uniform_f32(3, 2, bins)
    if flavour == "floats":
        vals = W.uniform_f32(3, 4, n)
    elif flavour == "dyadic":
        vals = torch.round(W.uniform_f32(3, 4, n) * 64) / 8
    elif flavour == "outliers":
        vals = torch.round(W.uniform_f32(3, 4, n) * 64) / 8
        vals[5] = 3.0e20
        vals[77] = 1.0e-30
        vals[1000] = float("inf")
        vals[2000:2100] = 7.0e5
    else:
        keys = torch.zeros(n, dtype=torch.int32)
        vals = torch.full((n,), 262143.0)
    inputs = {0: keys, 1: defaults, 2: vals}
    ref = oracle_run(prog, np_inputs(inputs))
    for pi in ([-1, -1, -1, 0, 1], [-1, -1, -1, 0, 0]):
        got, _ = gpu_run(prog, inputs, pi, B.FUSED)
        with np.errstate(invalid="ignore"):
            compare_hist(prog, ref, got, flavour)


def compare_hist(prog, ref, got, what):
    exact, scale, a = ref.exact[4], ref.abs_sum[4], got[4].astype(np.float64)
    finite = np.isfinite(exact)
    assert np.array_equal(np.isfinite(a), finite), what
    assert np.array_equal(a[~finite], exact[~finite]) or np.all(np.isnan(exact[~finite]) == np.isnan(a[~finite])), what
    bound = 1e-5 * scale[finite] + np.abs(exact[finite]) * 2.0 ** -24 + 1e-30
    assert np.all(np.abs(a[finite] - exact[finite]) <= bound), what
    assert 3 not in got or np.array_equal(got[3], ref.values[3]), what


@pytest.mark.parametrize("n,segments", [(5, 1), (64, 5), (1000, 16), (100000, 300), (1 << 20, 1 << 12), (1 << 20, 6), (1 << 22, 1 << 18),
                                        ((1 << 21) + 3, 1 << 10)])
def test_segmented_fold(n, segments):
    # the source is walked in tiles of 4096 elements; pieces of segments by a thread, a warp or the block according to
    # their length; segments that cross tiles and blocks; a sum fed by a fused map and a maximum sharing the same walk;
    # a source without 128-bit rows (the last shape)
    from paper_2407_13585_b200 import binding as B
    prog = W.segmented_sums(n, segments)
    runnable = [pi for pi in all_partitions(prog) if pi != [-1, -1, 0, 1, 0]]
    assert check_program(prog, runnable) == 3
    # {m, maxes} is legal (they share the read of xs) but mixes an element-wise store with a segmented fold
    g = B.Graph(prog.nodes, prog.outputs)
    g.set_partition([-1, -1, 0, 1, 0])
    inputs = W.make_inputs(prog)
    with pytest.raises(B.AccError) as e:
        gpu_run(prog, inputs, [-1, -1, 0, 1, 0], B.FUSED)
    assert e.value.status == "ACC_ERR_NO_KERNEL"


def test_segmented_fold_with_skewed_and_awkward_segments():
    """One segment with 90 % of 2^22 elements among short ones; segments that begin or end exactly on tile and block
    boundaries, single elements on either side of a boundary, and offsets that leave the ends of the source out."""
    import torch
    from paper_2407_13585_b200 import binding as B
    n = 1 << 22
    T = 4096
    cuts = {100, 101, 117, 130, T - 1, T, T + 1, 2 * T, 2 * T + 16, 2 * T + 17, 5 * T + 2000}      # short pieces around tile ends
    big_lo = 6 * T + 123
    big_hi = big_lo + (n * 9) // 10                                                             # 90 % of the elements in one segment
    cuts |= {big_lo, big_hi}
    x = big_hi
    k = 0
    while x < n - 40000:                                                                           # lengths 1, 2, 3, ... 1500 after it
        k = k % 1500 + 1
        x += k
        cuts.add(x)
    cuts |= {n - 40000 + 3 * T, n - 9}                                                             # a last long piece; the source's end is left out
    offsets = torch.tensor(sorted(cuts), dtype=torch.int32)
    segments = offsets.numel() - 1
    prog = W.segmented_sums(n, segments)
    inputs = W.make_inputs(prog)
    inputs[1] = offsets
    check_program(prog, [[-1, -1, 0, 0, 0], [-1, -1, 0, 1, 2]], inputs_t=inputs)
    # the same walk on equal addends: the long segment's sum crosses hundreds of tiles and dozens of blocks
    inputs[0] = torch.full((n,), 0.1)
    ref = oracle_run(prog, np_inputs(inputs))
    got, _ = gpu_run(prog, inputs, [-1, -1, 0, 0, 0], B.FUSED)
    compare(prog, ref, got, "skewed segments, equal addends")


def test_segmented_fold_reports_bad_offsets():
    import torch
    from paper_2407_13585_b200 import binding as B
    prog = W.segmented_sums(1000, 4)
    for offsets, status in (([0, 10, 10, 500, 1000], "ACC_ERR_SHAPE"), ([0, 10, 20, 500, 1001], "ACC_ERR_INDEX_RANGE")):
        inputs = W.make_inputs(prog)
        inputs[1] = torch.tensor(offsets, dtype=torch.int32)
        with pytest.raises(B.AccError) as e:
            gpu_run(prog, inputs, [-1, -1, 0, 0, 0], B.FUSED)
        assert e.value.status == status


@pytest.mark.parametrize("rows,cols", [(1, 5), (7, 100), (64, 300), (3, 5000), (2, 4096 * 3 + 8), (200, 4096)])
def test_row_scans_both_directions(rows, cols):
    # rank-2 arrays are scanned row by row (look-back stops at the row start); scanr walks from the far end;
    # rows of several tiles and of a fraction of one, widths that allow 128-bit accesses and widths that do not
    check_program(W.row_scans(rows, cols))


@pytest.mark.parametrize("n", [1, 6, 4096, 100001, 1 << 18])
def test_right_to_left_scan_int32(n):
    check_program(W.suffix_sums(n))


# seeded exclusive scans: an int32 running sum fed by a fused map (bit-exact), an fp32 sum from the right
# and a per-row running maximum; one element, a fraction of a tile, tile boundaries, ragged tails
@pytest.mark.parametrize("n", [1, 3, 4096, 4097, 70001, 1 << 18])
def test_exclusive_seeded_scans(n):
    assert check_program(W.exclusive_scans(n)) == 2


@pytest.mark.parametrize("rows,cols", [(3, 10), (5, 4096), (2, 9000), (64, 301)])
def test_exclusive_row_scans(rows, cols):
    check_program(W.exclusive_row_scans(rows, cols))


def test_gather_indices_are_checked_on_request_and_clusters_are_timed():
    import torch
    from paper_2407_13585_b200 import binding as B
    prog = W.config3(1 << 16)
    inputs = W.make_inputs(prog)
    g = B.Graph(prog.nodes, prog.outputs)
    g.set_partition([-1, -1, 0, 1, 1, 1])
    dev = {i: t.cuda() for i, t in inputs.items()}
    for i, t in dev.items():
        g.bind(i, t)
    out = torch.empty(1 << 16, dtype=torch.int32, device="cuda")
    g.bind(prog.outputs[0], out)
    g.check_gather_indices()                               # every index below 2^16
    ms = g.run_timed(B.FUSED)
    assert len(ms) == 2 and all(0.0 < t < 50.0 for t in ms) and g.launch_count() == 2
    ref = oracle_run(prog, np_inputs(inputs))
    assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.values[prog.outputs[0]])
    # one index just past the end, one negative: reported by the check (the program is not run on them)
    idx = [i for i in prog.input_ids() if prog.nodes[i].name == "idx"][0]
    for bad in (1 << 16, -1):
        dev[idx][12345] = bad
        with pytest.raises(B.AccError) as err:
            g.check_gather_indices()
        assert err.value.status == "ACC_ERR_INDEX_RANGE"
    dev[idx][12345] = 7
    g.check_gather_indices()


@pytest.mark.parametrize("n,bins", [(1 << 12, 64), (100003, 1000), (1 << 20, 1 << 12)])
def test_histogram_total_regenerates_vals_in_its_own_kernel(n, bins):
    # a clustering with a copy: {k, vals, hist} | {vals', total} | {frac}: three kernels, vals never stored
    import torch
    from paper_2407_13585_b200 import binding as B
    prog = W.config5(n, bins)
    inputs_t = W.make_inputs(prog)
    ref = oracle_run(prog, np_inputs(inputs_t))
    g = B.Graph(prog.nodes, prog.outputs)
    g.set_partition_copies([-1, -1, 0, 0, 0, 1, 2], [(3, 1)])
    assert not g.manifest()[3]
    bufs = {}
    for i, nd in enumerate(prog.nodes):
        if nd.kind == "input":
            bufs[i] = inputs_t[i].cuda()
            g.bind(i, bufs[i])
        elif i in prog.outputs:
            cnt = int(np.prod(nd.shape, dtype=np.int64)) if nd.shape else 1
            bufs[i] = torch.full((max(cnt, 4),), -1, dtype=torch.int32, device="cuda")
            g.bind(i, bufs[i])
    g.run(B.FUSED)
    g.run(B.FUSED)
    assert g.launch_count() == 3
    got = {}
    for o in prog.outputs:
        nd = prog.nodes[o]
        cnt = int(np.prod(nd.shape, dtype=np.int64)) if nd.shape else 1
        got[o] = bufs[o][:cnt].cpu().numpy().view(np.float32).reshape(tuple(nd.shape))
    compare(prog, ref, got, "config5 with a copy of vals")


# row folds consumed by a map of the same cluster (the clustering the bottom-up greedy finds for the paper's
# trap program, and every other clustering of it): rows reduced by a block, the map applied to the reduced
# values; rows of several block strides, ragged, with and without 128-bit accesses, and short rows (pulled)
@pytest.mark.parametrize("n,m", [(64, 1000), (7, 4099), (3, 40), (300, 256)])
def test_maps_of_row_folds(n, m):
    assert check_program(W.greedy_bottom_up_bad(n, m)) >= 8


# two arrays staged as tile pairs, one read as it lies and one transposed; sizes as for config 2
@pytest.mark.parametrize("rows", [4, 64, 100, 130, 256, 1600])
def test_diagonal_of_a_product(rows):
    assert check_program(W.diagonal_of_product(rows)) == 4


def test_lookback_wait_that_runs_out_is_reported():
    """The one device-side wait that polls plain memory (a scan tile looking back at its predecessors) is given
    no patience at all: tiles that find a predecessor unfinished give up at once, the kernel ends normally, and
    the run reports ACC_ERR_DEVICE_TIMEOUT; with the default bound the same graph then gives the oracle's result."""
    import torch
    from oracle import interp
    from paper_2407_13585_b200 import binding as B
    from workloads import Node
    n = 1 << 22
    nodes = [Node("input", "i32", (n,), name="x"), Node("scanl", "i32", (n,), (0,), 1, fn="add", name="out")]
    x = W.uniform_int(5, 0, n, 1 << 31, device="cuda")
    out = torch.zeros(n, dtype=torch.int32, device="cuda")
    g = B.Graph(nodes, [1])
    g.bind(0, x)
    g.bind(1, out)
    g.set_spin_limit(0)
    with pytest.raises(B.AccError) as e:
        g.run(B.UNFUSED)
    assert e.value.status == "ACC_ERR_DEVICE_TIMEOUT"
    g.set_spin_limit(1 << 22)
    g.run(B.UNFUSED)
    want = np.cumsum(x.cpu().numpy().view(np.uint32), dtype=np.uint32).view(np.int32)       # wrapping adds, as Section 2's scanl(+)
    ref = interp.run(nodes, {0: x.cpu().numpy()}).values[1]
    assert np.array_equal(interp.to_external(ref, "i32"), want)
    assert np.array_equal(out.cpu().numpy(), want)


def test_lookback_wait_that_runs_out_where_a_warp_of_its_own_looks_back():
    """The same wait in the scan that parks a tile's values and leaves the look-back to a ninth warp (scans with a
    gather in their cluster): that warp gives up at once, still hands the other warps a prefix at their barrier, the
    kernel ends normally and the run reports the time-out; with the default bound the graph gives the oracle's result."""
    import torch
    from paper_2407_13585_b200 import binding as B
    prog = W.config3(1 << 22)
    inputs = W.make_inputs(prog, device="cuda")
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    g = B.Graph(prog.nodes, prog.outputs)
    g.set_partition([-1, -1, 0, 0, 0, 0])
    for i, t in inputs.items():
        g.bind(i, t)
    out = torch.zeros(1 << 22, dtype=torch.int32, device="cuda")
    g.bind(5, out)
    g.set_spin_limit(0)
    with pytest.raises(B.AccError) as e:
        g.run(B.FUSED)
    assert e.value.status == "ACC_ERR_DEVICE_TIMEOUT"
    g.set_spin_limit(1 << 22)
    g.run(B.FUSED)
    assert g.launch_count() == 1
    compare(prog, ref, {5: out.cpu().numpy().view(np.uint32)}, "config3 after a look-back that ran out")


def test_runs_do_not_depend_on_what_the_workspace_held():
    """A run clears the status word and the part of every cluster's scratch that must start at zero, nothing else
    (partial sums per tile, records, staged operands are written before they are read): a workspace full of 0xFF
    bytes, or left as the previous run of another clustering had it, gives the same arrays."""
    import torch
    from paper_2407_13585_b200 import binding as B
    for prog in (W.config2(1600), W.config5(1 << 18, 1 << 10), W.segmented_sums(1 << 18, 1 << 9), W.scan_consumers(70000),
                 W.config3(1 << 16), W.config1(1 << 14)):
        inputs = W.make_inputs(prog)
        ref = oracle_run(prog, np_inputs(inputs))
        g = B.Graph(prog.nodes, prog.outputs)
        g.plan("enumerate", "bytes")
        g.refine_to_kernels()
        bufs = {}
        for i, nd in enumerate(prog.nodes):
            if nd.kind == "input":
                bufs[i] = inputs[i].cuda().contiguous()
                g.bind(i, bufs[i])
            elif i in prog.outputs:
                cnt = int(np.prod(nd.shape, dtype=np.int64)) if nd.shape else 1
                bufs[i] = torch.full((max(cnt, 4),), -12345, dtype=torch.int32, device="cuda")
                g.bind(i, bufs[i])
        for executor in (B.FUSED, B.UNFUSED, B.FUSED):
            g.workspace = None
            ws = g.ensure_workspace(executor)
            ws.fill_(255)
            g.run(executor)
            g.run(executor)
            torch.cuda.synchronize()
            got = {}
            for o in prog.outputs:
                nd = prog.nodes[o]
                cnt = int(np.prod(nd.shape, dtype=np.int64)) if nd.shape else 1
                a = bufs[o][:cnt].cpu().numpy()
                got[o] = (a.view(np.float32) if nd.dtype == "f32" else a.view(np.uint32)).reshape(tuple(nd.shape))
            compare(prog, ref, got, "%s after a workspace of 0xFF bytes, executor %d" % (prog.name, executor))
