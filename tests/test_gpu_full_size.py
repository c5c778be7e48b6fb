"""GPU parity at the benchmark's full sizes, in the configuration bench.py times: the
planner's clustering, the fused executor, inputs drawn on the device.  Configs 2, 3 and 5
are compared with the oracle on every output element; config 4 on row bands (top edge,
middle, bottom edge) that the oracle recomputes from the same input rows."""
import numpy as np
import pytest

import workloads as W
from helpers import compare, oracle_run

pytestmark = pytest.mark.gpu


def run_full(prog, mode):
    import torch
    from paper_2407_13585_b200 import binding as B
    g = B.Graph(prog.nodes, prog.outputs)
    pi = g.plan(mode, "bytes")
    inputs = W.make_inputs(prog, device="cuda")
    for i, t in inputs.items():
        g.bind(i, t)
    outs = {}
    for o in prog.outputs:
        nd = prog.nodes[o]
        cnt = int(np.prod(nd.shape, dtype=np.int64)) if nd.shape else 1
        outs[o] = torch.full((max(cnt, 4),), -1, dtype=torch.int32, device="cuda")
        g.bind(o, outs[o])
    g.run(B.FUSED)
    g.run(B.FUSED)                     # a second run over the same workspace must give the same arrays
    torch.cuda.synchronize()
    got = {}
    for o, t in outs.items():
        nd = prog.nodes[o]
        cnt = int(np.prod(nd.shape, dtype=np.int64)) if nd.shape else 1
        a = t[:cnt].cpu().numpy()
        got[o] = (a.view(np.float32) if nd.dtype == "f32" else a.view(np.uint32)).reshape(tuple(nd.shape))
    return got, inputs, pi, g


def test_config2_full():
    prog = W.config2(8192)
    got, inputs, pi, g = run_full(prog, "enumerate")
    assert pi == [-1, 0, 0, 0] and g.launch_count() == 1
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    compare(prog, ref, got, "config2 full")


def test_config3_full():
    prog = W.config3(1 << 26)
    got, inputs, pi, g = run_full(prog, "enumerate")
    # one cluster; its gather reads a 256 MB source, twice the L2, so it runs as slab passes: the indices are
    # probed (random or local?), partitioned once, four launches gather a quarter of the source each, and the scan
    # merges (seven launches)
    assert pi == [-1, -1, 0, 0, 0, 0] and g.launch_count() == 7
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    compare(prog, ref, got, "config3 full")


def test_gather_scan_in_slab_passes_ragged():
    """The slab passes on shapes of their own: a 128 MB source, fewer indices than source elements, a last warp tile
    of 260 elements (left to the last kernel's direct gather), under both clusterings that keep the gather with the
    scan, under one that ends the gather's cluster at the masked values, and with every combinator alone."""
    import torch
    from workloads import Node, Program
    from paper_2407_13585_b200 import binding as B
    n_src, n = 1 << 25, (1 << 22) + (1 << 20) + 260
    nodes = [Node("input", "i32", (n_src,), name="x"), Node("input", "i32", (n,), name="idx"),
             Node("map", "i32", (n_src,), (0,), 1, fn="hash_mul_xorshift", iparam=(2654435761, 13), name="g"),
             Node("gather", "i32", (n,), (1, 2), 2, name="h"),
             Node("map", "i32", (n,), (3,), 1, fn="and_mask", iparam=(0xFFFF,), name="o"),
             Node("scanl", "i32", (n,), (4,), 1, fn="add", name="out")]
    prog = Program("gather_scan_ragged", nodes, [5])
    inputs = {0: W.uniform_int(0, 0, n_src, 1 << 31, device="cuda"), 1: W.uniform_int(0, 1, n, n_src, device="cuda")}
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    # ... and under one that stores the masked values and scans them in a cluster of its own: the element-wise
    # cluster takes the same passes, with a kernel that only merges and stores in place of the merging scan
    for pi, launches in (([-1, -1, 0, 0, 0, 0], 7), ([-1, -1, 0, 1, 1, 1], 8), ([-1, -1, 0, 0, 0, 1], 8), ([-1, -1, 0, 1, 2, 3], 10)):
        g = B.Graph(prog.nodes, prog.outputs)
        g.set_partition(pi)
        for i, t in inputs.items():
            g.bind(i, t)
        out = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        g.bind(5, out)
        g.ensure_workspace(B.FUSED).fill_(255)          # the slab codes and group sizes are not cleared by a run: they must not need it
        g.run(B.FUSED)
        g.run(B.FUSED)
        assert g.launch_count() == launches, (pi, g.launch_count())
        got = {5: out.cpu().numpy().view(np.uint32)}
        compare(prog, ref, got, "gather + scan in slab passes, pi=%s" % pi)


def test_slab_passes_with_several_element_wise_roots():
    """A cluster without a scan in slab passes, with three arrays to store: the gathered values themselves (their array
    is the staging area), a map of them, and a map of the indices that does not touch the gather."""
    import torch
    from paper_2407_13585_b200 import binding as B
    n = (1 << 22) + 260
    prog = W.gather_three_roots(1 << 25, n)
    inputs = W.make_inputs(prog, device="cuda")
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    g = B.Graph(prog.nodes, prog.outputs)
    g.set_partition([-1, -1, 0, 0, 0])
    for i, t in inputs.items():
        g.bind(i, t)
    outs = {o: torch.full((n,), -1, dtype=torch.int32, device="cuda") for o in prog.outputs}
    for o, t in outs.items():
        g.bind(o, t)
    g.run(B.FUSED)
    g.run(B.FUSED)
    assert g.launch_count() == 7
    compare(prog, ref, {o: t.cpu().numpy().view(np.uint32) for o, t in outs.items()}, "gather with three roots in slab passes")


def test_slab_passes_stand_back_for_local_indices():
    """Indices that run through a 128 MB source in order (steps of 0..3 elements) are served by the plain gather: the
    probe finds every sampled warp tile local, the partition and the four gather launches return at once, and the
    last kernel gathers for itself.  Same launches, same results as the oracle, with the scan in the gather's cluster
    and without; a source that is read at random between two runs of the same graph takes the passes again."""
    import torch
    from workloads import Node, Program
    from paper_2407_13585_b200 import binding as B
    n_src, n = 1 << 25, (1 << 22) + 516
    nodes = [Node("input", "i32", (n_src,), name="x"), Node("input", "i32", (n,), name="idx"),
             Node("gather", "i32", (n,), (1, 0), 2, name="h"),
             Node("map", "i32", (n,), (2,), 1, fn="and_mask", iparam=(0xFFFF,), name="o"),
             Node("scanl", "i32", (n,), (3,), 1, fn="add", name="out")]
    prog = Program("gather_scan_local", nodes, [4])
    x = W.uniform_int(0, 0, n_src, 1 << 31, device="cuda")
    steps = W.uniform_int(0, 1, n, 4, device="cuda")
    local = torch.cumsum(steps, 0, dtype=torch.int64).to(torch.int32)              # below 3 * n < n_src
    scattered = W.uniform_int(0, 2, n, n_src, device="cuda")
    for pi, launches in (([-1, -1, 0, 0, 0], 7), ([-1, -1, 0, 0, 1], 8)):
        g = B.Graph(prog.nodes, prog.outputs)
        g.set_partition(pi)
        g.bind(0, x)
        out = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        g.bind(4, out)
        for idx, what in ((local, "local"), (scattered, "scattered"), (local, "local again")):
            g.bind(1, idx)
            ref = oracle_run(prog, {0: x.cpu().numpy(), 1: idx.cpu().numpy()})
            g.run(B.FUSED)
            assert g.launch_count() == launches, (pi, g.launch_count())
            compare(prog, ref, {4: out.cpu().numpy().view(np.uint32)}, "gather + scan, %s indices, pi=%s" % (what, pi))


def test_gathering_scans_over_several_rounds_of_a_resident_grid():
    """Scans with a gather in their cluster walk tiles of 4096 elements with a warp that only looks back; here a block
    takes several tiles in turn (2^23 elements are 2048 tiles, more than the blocks one launch holds), and the last
    tile of the second program is ragged."""
    prog = W.offsets_then_gather(1 << 23)
    got, inputs, pi, g = run_full(prog, "enumerate")
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    compare(prog, ref, got, "offsets_then_gather, 2^23")
    # gather + scan with a 32 MB source (no slab passes) and an odd count of indices: element by element, ragged last tile
    import torch
    from workloads import Node, Program
    from paper_2407_13585_b200 import binding as B
    n_src, n = 1 << 23, (1 << 23) - 1029
    nodes = [Node("input", "i32", (n_src,), name="x"), Node("input", "i32", (n,), name="idx"),
             Node("map", "i32", (n_src,), (0,), 1, fn="hash_mul_xorshift", iparam=(2654435761, 13), name="g"),
             Node("gather", "i32", (n,), (1, 2), 2, name="h"),
             Node("map", "i32", (n,), (3,), 1, fn="and_mask", iparam=(0xFFFF,), name="o"),
             Node("scanl", "i32", (n,), (4,), 1, fn="add", name="out")]
    prog = Program("gather_scan_odd", nodes, [5])
    inputs = {0: W.uniform_int(0, 0, n_src, 1 << 31, device="cuda"), 1: W.uniform_int(0, 1, n, n_src, device="cuda")}
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    g = B.Graph(prog.nodes, prog.outputs)
    g.set_partition([-1, -1, 0, 0, 0, 0])
    for i, t in inputs.items():
        g.bind(i, t)
    out = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    g.bind(5, out)
    g.run(B.FUSED)
    g.run(B.FUSED)
    assert g.launch_count() == 1
    compare(prog, ref, {5: out.cpu().numpy().view(np.uint32)}, "gather + scan, 2^23 - 1029 indices")


def test_config5_full():
    prog = W.config5(1 << 27, 1 << 16)
    got, inputs, pi, g = run_full(prog, "enumerate")
    assert pi == [-1, -1, 0, 0, 0, 0, 1] and g.launch_count() == 2
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    compare(prog, ref, got, "config5 full")
    # the hottest bin holds far more than 2^24: plain fp32 accumulation would have lost its small addends
    assert ref.exact[4].max() > 2 ** 24


def test_config1_full():
    prog = W.config1(1 << 16)
    got, inputs, pi, g = run_full(prog, "enumerate")
    assert g.launch_count() == 1
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    compare(prog, ref, got, "config1 full")


def test_config4_full_on_row_bands():
    rows = cols = 8192
    iters = 4
    prog = W.config4(rows, cols, iters)
    got, inputs, pi, g = run_full(prog, "greedy_topdown")
    assert g.launch_count() == iters
    X = inputs[0]
    Y = got[prog.outputs[0]]
    for lo, hi in ((0, 48), (4000, 4040), (rows - 48, rows)):
        # the band plus `iters` halo rows on each open side determines the band's output exactly
        a, b = max(0, lo - iters), min(rows, hi + iters)
        sub = W.config4(b - a, cols, iters)
        ref = oracle_run(sub, {0: X[a:b].cpu().numpy()})
        want = ref.values[sub.outputs[0]][lo - a: hi - a]
        assert np.array_equal(Y[lo:hi].view(np.uint32), want.view(np.uint32)), (lo, hi)


def test_greedy_bottom_up_bad_at_paper_scale():
    # Section 5's program on which the bottom-up greedy goes wrong, at the size the paper names
    # (m = 10^6 columns): under the best clustering the gathered n x m array and both folds share a
    # kernel and the large array never exists; the bottom-up greedy clustering stores it (64 MB).
    from paper_2407_13585_b200 import binding as B
    prog = W.greedy_bottom_up_bad(16, 1000000)
    got, inputs, pi, g = run_full(prog, "branch_bound")
    assert pi == [-1, 0, 0, 0, 0, 1] and g.launch_count() == 2 and g.plan_info()[1]
    assert g.partition_cost(pi, "bytes") < g.partition_cost(g.plan("greedy_bottomup", "bytes"), "bytes") / 1000
    ref = oracle_run(prog, {k: v.cpu().numpy() for k, v in inputs.items()})
    compare(prog, ref, got, "greedy_bottom_up_bad, m = 10^6")
    # the bottom-up greedy clustering itself: a map of a row fold in one kernel
    got, inputs, pi, g = run_full(prog, "greedy_bottomup")
    assert pi == [-1, 0, 0, 1, 0, 1] and g.launch_count() == 2
    compare(prog, ref, got, "greedy_bottom_up_bad, m = 10^6, bottom-up greedy")
