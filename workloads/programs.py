"""Combinator programs as plain records.

A program is an ordered list of nodes; a node may only name earlier nodes as
inputs, so every list is a DAG in topological order.  Slot layout by kind:

  input        no slots (bound by the caller)
  generate     [free...]                       n_array = 0
  map          [xs, free...]                   n_array = 1
  zipwith      [xs1..xsk, free...]             n_array = k (2..5)
  backpermute  [src]                           index map named by idx_fn
  gather       [idx, src]                      idx holds row-major linear indices
  permute      [defaults, idx, vals]           combine op named by fn
  fold         [src]                           reduces the innermost extent
  scanl/scanr  [src]                           inclusive, per innermost row (exclusive=True: seeded, exclusive)
  foldseg      [src, offsets]                  n_array = 1; ys[s] = fold of src[offsets[s] .. offsets[s+1])

Slots at positions >= n_array are "free variable" reads (element-level
indexing: element 0, except the offsets of a foldseg, which are read at s and s+1).  Function names are interpreted by each
executor's own table; this file only spells them.
"""
from dataclasses import dataclass, field
from typing import List, Tuple


@dataclass
class Node:
    kind: str
    dtype: str                      # 'f32' | 'i32' | 'u32'
    shape: Tuple[int, ...]          # () for the scalar result of a rank-1 fold
    inputs: Tuple[int, ...] = ()
    n_array: int = 0
    fn: str = ""
    idx_fn: str = ""
    iparam: Tuple[int, ...] = ()
    fparam: Tuple[float, ...] = ()
    force: Tuple[int, ...] = ()     # slots whose read is wrapped in force()
    exclusive: bool = False         # scans: ys[i] combines the seed (fparam[0] / iparam[0]) and the elements before i
    name: str = ""


@dataclass
class Program:
    name: str
    nodes: List[Node]
    outputs: List[int]
    names: dict = field(default_factory=dict)
    index_bound: dict = field(default_factory=dict)   # exclusive bound of index-valued inputs

    def __post_init__(self):
        self.names = {nd.name: i for i, nd in enumerate(self.nodes) if nd.name}

    def id(self, name):
        return self.names[name]

    def input_ids(self):
        return [i for i, nd in enumerate(self.nodes) if nd.kind == "input"]


def _inp(name, dtype, shape):
    return Node("input", dtype, tuple(shape), name=name)


# --------------------------------------------------------------------------
# The five benchmark configurations
# --------------------------------------------------------------------------

def config1(n=1 << 16):
    """1-D chain: y=map(2x+1) x; z=backpermute(reverse) y; w=zipWith(*) z x; s=fold(+) w."""
    nodes = [
        _inp("x", "f32", (n,)),
        Node("map", "f32", (n,), (0,), 1, fn="affine", fparam=(2.0, 1.0), name="y"),
        Node("backpermute", "f32", (n,), (1,), 1, idx_fn="reverse", name="z"),
        Node("zipwith", "f32", (n,), (2, 0), 2, fn="mul", name="w"),
        Node("fold", "f32", (), (3,), 1, fn="add", name="s"),
    ]
    return Program("config1", nodes, [4])


def config2(rows=8192):
    """2-D transpose-fuse-reduce: B=transpose A; C=A*B+0.5; rowsum=fold(+) C."""
    sh = (rows, rows)
    nodes = [
        _inp("A", "f32", sh),
        Node("backpermute", "f32", sh, (0,), 1, idx_fn="transpose", name="B"),
        Node("zipwith", "f32", sh, (0, 1), 2, fn="mul_add_const", fparam=(0.5,), name="C"),
        Node("fold", "f32", (rows,), (2,), 1, fn="add", name="rowsum"),
    ]
    return Program("config2", nodes, [3])


def config3(n=1 << 26):
    """Random gather + scan on int32: g=hash x; h=gather idx g; o=h&0xFFFF; out=scanl(+) o."""
    nodes = [
        _inp("x", "i32", (n,)),
        _inp("idx", "i32", (n,)),
        Node("map", "i32", (n,), (0,), 1, fn="hash_mul_xorshift", iparam=(2654435761, 13), name="g"),
        Node("gather", "i32", (n,), (1, 2), 2, name="h"),
        Node("map", "i32", (n,), (3,), 1, fn="and_mask", iparam=(0xFFFF,), name="o"),
        Node("scanl", "i32", (n,), (4,), 1, fn="add", name="out"),
    ]
    return Program("config3", nodes, [5])


def config4(rows=8192, cols=None, iters=4):
    """Jacobi by horizontal fusion: per iteration five clamped shifts and four zipWiths."""
    cols = rows if cols is None else cols
    sh = (rows, cols)
    nodes = [_inp("X", "f32", sh)]
    prev = 0
    for t in range(iters):
        base = len(nodes)
        shifts = [("c", 0, 0), ("n", -1, 0), ("s", 1, 0), ("e", 0, 1), ("w", 0, -1)]
        for tag, dr, dc in shifts:
            nodes.append(Node("backpermute", "f32", sh, (prev,), 1, idx_fn="shift_clamp",
                              iparam=(dr, dc), name=f"{tag}{t}"))
        c, n_, s, e, w = range(base, base + 5)
        nodes.append(Node("zipwith", "f32", sh, (c, n_), 2, fn="add", name=f"t1_{t}"))
        nodes.append(Node("zipwith", "f32", sh, (base + 5, s), 2, fn="add", name=f"t2_{t}"))
        nodes.append(Node("zipwith", "f32", sh, (base + 6, e), 2, fn="add", name=f"t3_{t}"))
        nodes.append(Node("zipwith", "f32", sh, (base + 7, w), 2, fn="add_scale",
                          fparam=(0.2,), name=f"Y{t}"))
        prev = base + 8
    return Program("config4", nodes, [prev])


def config5(n=1 << 27, bins=1 << 16):
    """Scatter histogram + diamond: k=hash16 keys; vals=generate; hist=permute(+); total=fold; frac."""
    nodes = [
        _inp("keys", "u32", (n,)),
        _inp("zeros", "f32", (bins,)),
        Node("map", "u32", (n,), (0,), 1, fn="mul_mod", iparam=(40503, bins), name="k"),
        Node("generate", "f32", (n,), (), 0, fn="imod_to_f32", iparam=(7,), name="vals"),
        Node("permute", "f32", (bins,), (1, 2, 3), 3, fn="add", name="hist"),
        Node("fold", "f32", (), (3,), 1, fn="add", name="total"),
        Node("map", "f32", (bins,), (4, 5), 1, fn="div_free", name="frac"),
    ]
    return Program("config5", nodes, [6, 4, 5])


# --------------------------------------------------------------------------
# Programs the paper prints (Sections 1, 3.3, 3.4 and 5), as fixtures
# --------------------------------------------------------------------------

def single_loop(n=64):
    """Section 1 `singleLoop`: reverse + two maps + zipWith3, fusible into one loop."""
    nodes = [
        _inp("as", "f32", (n,)),
        Node("backpermute", "f32", (n,), (0,), 1, idx_fn="reverse", name="bs"),
        Node("map", "f32", (n,), (0,), 1, fn="affine", fparam=(3.0, -1.0), name="cs"),
        Node("map", "f32", (n,), (2,), 1, fn="affine", fparam=(0.5, 2.0), name="ds"),
        Node("zipwith", "f32", (n,), (1, 2, 3), 3, fn="add3", name="result"),
    ]
    return Program("single_loop", nodes, [4])


def simple1(n_is=40, n_xs=24):
    nodes = [
        _inp("is", "i32", (n_is,)), _inp("xs", "f32", (n_xs,)),
        Node("map", "f32", (n_xs,), (1,), 1, fn="affine", fparam=(2.0, 1.0), name="as"),
        Node("gather", "f32", (n_is,), (0, 2), 2, name="bs"),
    ]
    return Program("simple1", nodes, [3], index_bound={"is": n_xs})


def simple2(n_is2=50, n_is1=30, n_xs=20):
    nodes = [
        _inp("is1", "i32", (n_is1,)), _inp("is2", "i32", (n_is2,)), _inp("xs", "f32", (n_xs,)),
        Node("gather", "f32", (n_is1,), (0, 2), 2, name="as"),
        Node("gather", "f32", (n_is2,), (1, 3), 2, name="bs"),
    ]
    return Program("simple2", nodes, [4], index_bound={"is1": n_xs, "is2": n_is1})


def simple3(n_is=40, n_xs=24):
    p = simple1(n_is, n_xs)
    return Program("simple3", p.nodes, [2, 3], index_bound=p.index_bound)


def simple4(n_is=20, m=12, n=7):
    nodes = [
        _inp("is", "i32", (n_is,)), _inp("xs", "f32", (m, n)),
        Node("fold", "f32", (m,), (1,), 1, fn="add", name="as"),
        Node("gather", "f32", (n_is,), (0, 2), 2, name="bs"),
    ]
    return Program("simple4", nodes, [3], index_bound={"is": m})


def simple5(n=32):
    nodes = [
        _inp("is", "i32", (n,)), _inp("xs", "f32", (n,)),
        Node("map", "f32", (n,), (1,), 1, fn="affine", fparam=(-1.5, 0.25), name="as"),
        Node("gather", "f32", (n,), (0, 1), 2, name="bs"),
        Node("zipwith", "f32", (n,), (2, 3), 2, fn="mul", name="cs"),
    ]
    return Program("simple5", nodes, [4], index_bound={"is": n})


def scatter_example(n=48):
    """Section 3.4 `scatterExample` after the structure-of-arrays split of `as`.

    xs holds integers in [0, n/2) so that every index 2*x lands inside bs.
    """
    nodes = [
        _inp("xs", "i32", (n,)),
        Node("map", "i32", (n,), (0,), 1, fn="mul_const", iparam=(2,), name="as_i"),
        Node("map", "i32", (n,), (0,), 1, fn="identity", name="as_v"),
        Node("map", "i32", (n,), (0,), 1, fn="add_const", iparam=(1,), name="bs"),
        Node("permute", "i32", (n,), (3, 1, 2), 3, fn="add", name="result"),
    ]
    return Program("scatter_example", nodes, [4], index_bound={"xs": n // 2})


def scatter_example_paper_graph():
    """The literal four-node graph of Section 4.1: `as` is one node feeding both
    element slots of the scatter.  Only its structure is meaningful."""
    nodes = [
        _inp("xs", "i32", (8,)),
        Node("map", "i32", (8,), (0,), 1, fn="identity", name="as"),
        Node("map", "i32", (8,), (0,), 1, fn="add_const", iparam=(1,), name="bs"),
        Node("permute", "i32", (8,), (2, 1, 1), 3, fn="add", name="result"),
    ]
    return Program("scatter_example_paper_graph", nodes, [3])


def greedy_bottom_up_bad(n=16, m=1000):
    """Section 5: a gathered rank-2 array that contracts only if both folds share its cluster."""
    nodes = [
        _inp("xs", "f32", (n,)),
        Node("generate", "i32", (n, m), (), 0, fn="row_index", name="is"),
        Node("gather", "f32", (n, m), (1, 0), 2, name="large"),
        Node("fold", "f32", (n,), (2,), 1, fn="add", name="ys"),
        Node("fold", "f32", (n,), (2,), 1, fn="mul", name="zs"),
        Node("map", "f32", (n,), (3, 4), 1, fn="add_free", name="result"),
    ]
    return Program("greedy_bottom_up_bad", nodes, [5])


def greedy_top_down_bad(n=4096):
    """Section 5: greedy top-down fuses cs diagonally with bs; the optimum fuses cs into es."""
    nodes = [
        _inp("as", "f32", (n,)),
        Node("map", "f32", (n,), (0,), 1, fn="affine", fparam=(2.0, 0.0), name="bs"),
        Node("map", "f32", (n,), (1,), 1, fn="affine", fparam=(1.0, 1.0), name="cs"),
        Node("generate", "f32", (n,), (1,), 0, fn="iota_plus_free", name="ds"),
        Node("zipwith", "f32", (n,), (2, 3), 2, fn="add", name="es"),
        Node("fold", "f32", (), (4,), 1, fn="add", name="result"),
    ]
    return Program("greedy_top_down_bad", nodes, [5])


def segmented_sums(n=1 << 20, segments=1 << 12):
    """Segmented fold fed by a fused map: m = map(a*x+b) xs; sums = foldSeg(+) m offsets; maxes = foldSeg(max) xs offsets."""
    nodes = [
        _inp("xs", "f32", (n,)),
        _inp("offsets", "i32", (segments + 1,)),
        Node("map", "f32", (n,), (0,), 1, fn="affine", fparam=(0.5, 0.25), name="m"),
        Node("foldseg", "f32", (segments,), (2, 1), 1, fn="add", name="sums"),
        Node("foldseg", "f32", (segments,), (0, 1), 1, fn="max", name="maxes"),
    ]
    return Program("segmented_sums", nodes, [3, 4])


def row_scans(rows=64, cols=300):
    """Per-row scans of a rank-2 array: a left-to-right running sum, and a right-to-left running maximum of a fused map."""
    sh = (rows, cols)
    nodes = [
        _inp("x", "f32", sh),
        Node("scanl", "f32", sh, (0,), 1, fn="add", name="prefix"),
        Node("map", "f32", sh, (0,), 1, fn="affine", fparam=(-2.0, 0.5), name="m"),
        Node("scanr", "f32", sh, (2,), 1, fn="max", name="suffix_max"),
    ]
    return Program("row_scans", nodes, [1, 3])


def suffix_sums(n=1 << 16):
    """Right-to-left wrapping running sum of a masked int32 array."""
    nodes = [
        _inp("x", "i32", (n,)),
        Node("map", "i32", (n,), (0,), 1, fn="and_mask", iparam=(0xFFFFF,), name="g"),
        Node("scanr", "i32", (n,), (1,), 1, fn="add", name="suffix"),
    ]
    return Program("suffix_sums", nodes, [2])


def exclusive_scans(n=1 << 16):
    """Seeded exclusive scans: offsets from counts (wrapping int32 sum from the left of a masked array) and a
    right-to-left exclusive fp32 sum."""
    nodes = [
        _inp("x", "i32", (n,)),
        _inp("w", "f32", (n,)),
        Node("map", "i32", (n,), (0,), 1, fn="and_mask", iparam=(0xFF,), name="counts"),
        Node("scanl", "i32", (n,), (2,), 1, fn="add", iparam=(1000,), exclusive=True, name="offsets"),
        Node("scanr", "f32", (n,), (1,), 1, fn="add", fparam=(0.5,), exclusive=True, name="after"),
    ]
    return Program("exclusive_scans", nodes, [3, 4])


def exclusive_row_scans(rows=64, cols=300):
    """Per row of a rank-2 array: the running maximum of everything to the left, seeded with -1."""
    sh = (rows, cols)
    nodes = [
        _inp("x", "f32", sh),
        Node("scanl", "f32", sh, (0,), 1, fn="max", fparam=(-1.0,), exclusive=True, name="best_before"),
    ]
    return Program("exclusive_row_scans", nodes, [1])


def diagonal_of_product(rows=256):
    """d[i] = sum_j A[i][j] * B[j][i], the diagonal of A B: two square arrays, one of them read transposed."""
    sh = (rows, rows)
    nodes = [
        _inp("A", "f32", sh),
        _inp("B", "f32", sh),
        Node("backpermute", "f32", sh, (1,), 1, idx_fn="transpose", name="Bt"),
        Node("zipwith", "f32", sh, (0, 2), 2, fn="mul", name="P"),
        Node("fold", "f32", (rows,), (3,), 1, fn="add", name="d"),
    ]
    return Program("diagonal_of_product", nodes, [4])


def random_scan_program(seed, n=4099, rows=0):
    """A seeded random DAG around a scan in the middle: element-wise nodes and reversals before it, then nodes
    that may read the scan (directly, or through a reversal, which no kernel follows inside a cluster), then
    possibly a fold or a second scan of any of them.  rows = 0: rank 1."""
    from .inputs import counter_bits
    shape = (n,) if not rows else (rows, n)
    draws = iter(counter_bits(seed, 61, 96).tolist())

    def pick(k):
        return ((next(draws) & ((1 << 63) - 1)) >> 20) % k

    nodes = [_inp("x", "f32", shape), _inp("v", "f32", shape)]
    arrays = [0, 1]
    affine = [(2.0, 1.0), (-0.5, 0.25), (1.0, -3.0), (0.125, 0.0)]

    def add(node):
        nodes.append(node)
        node.name = "%s%d" % (node.kind[0], len(nodes) - 1)
        arrays.append(len(nodes) - 1)
        return len(nodes) - 1

    def some():
        return arrays[pick(len(arrays))]

    def element_wise():
        k = pick(4)
        if k == 0:
            add(Node("map", "f32", shape, (some(),), 1, fn="affine", fparam=affine[pick(4)]))
        elif k in (1, 2):
            add(Node("zipwith", "f32", shape, (some(), some()), 2, fn=("add", "mul")[pick(2)]))
        else:
            add(Node("backpermute", "f32", shape, (some(),), 1, idx_fn="reverse"))

    for _ in range(1 + pick(2)):
        element_wise()
    kind, fn = ("scanl", "scanr")[pick(2)], ("add", "max")[pick(2)]
    if pick(3) == 0:
        scan = add(Node(kind, "f32", shape, (some(),), 1, fn=fn, fparam=(0.5,), exclusive=True))
    else:
        scan = add(Node(kind, "f32", shape, (some(),), 1, fn=fn))
    add(Node("map", "f32", shape, (scan,), 1, fn="affine", fparam=affine[pick(4)]))      # at least one reader
    for _ in range(1 + pick(2)):
        element_wise()
    k = pick(3)
    if k == 1:
        add(Node("fold", "f32", shape[:-1], (some(),), 1, fn="add"))
    elif k == 2:
        add(Node("scanl", "f32", shape, (some(),), 1, fn="add"))
    used = {s for nd in nodes for s in nd.inputs}
    outputs = [i for i, nd in enumerate(nodes) if nd.kind != "input" and i not in used]
    return Program("random_scan%s_%d" % ("2d" if rows else "", seed), nodes, outputs)


def scan_consumers(n=4099, rows=None):
    """Scans whose values feed element-wise nodes: a running sum that is only consumed (never an output), a
    right-to-left running maximum that is both written and consumed, and a seeded exclusive sum."""
    sh = (n,) if rows is None else (rows, n)
    nodes = [
        _inp("x", "f32", sh),
        _inp("w", "f32", sh),
        Node("scanl", "f32", sh, (0,), 1, fn="add", name="s"),
        Node("map", "f32", sh, (2,), 1, fn="affine", fparam=(0.5, 1.0), name="m"),
        Node("zipwith", "f32", sh, (3, 1), 2, fn="mul", name="z"),
        Node("scanr", "f32", sh, (1,), 1, fn="max", name="r"),
        Node("zipwith", "f32", sh, (5, 0), 2, fn="add", name="q"),
        Node("scanl", "f32", sh, (1,), 1, fn="add", fparam=(0.25,), exclusive=True, name="e"),
        Node("zipwith", "f32", sh, (7, 0, 1), 3, fn="add3", name="t"),
    ]
    return Program("scan_consumers" + ("" if rows is None else "_2d"), nodes, [4, 5, 6, 8])


def offsets_then_gather(n=1 << 12):
    """Offsets from counts, used as indices in the same cluster: c = x & 3; o = exclusive running sum of c;
    y = src[o & (n-1)] (n a power of two); total = fold(+) c."""
    assert n & (n - 1) == 0
    nodes = [
        _inp("x", "i32", (n,)),
        _inp("src", "i32", (n,)),
        Node("map", "i32", (n,), (0,), 1, fn="and_mask", iparam=(3,), name="c"),
        Node("scanl", "i32", (n,), (2,), 1, fn="add", iparam=(0,), exclusive=True, name="o"),
        Node("map", "i32", (n,), (3,), 1, fn="and_mask", iparam=(n - 1,), name="k"),
        Node("gather", "i32", (n,), (4, 1), 2, name="y"),
        Node("fold", "i32", (), (2,), 1, fn="add", name="total"),
    ]
    return Program("offsets_then_gather", nodes, [5, 6], index_bound={"x": 1 << 30, "src": 1 << 30})


def gather_three_roots(n_src=1 << 12, n=1 << 10):
    """One gather with three arrays to store: h = src[idx]; m = h & 0xFFFF; r = idx & 0xFF (which does not touch the
    gather)."""
    nodes = [
        _inp("x", "i32", (n_src,)),
        _inp("idx", "i32", (n,)),
        Node("gather", "i32", (n,), (1, 0), 2, name="h"),
        Node("map", "i32", (n,), (2,), 1, fn="and_mask", iparam=(0xFFFF,), name="m"),
        Node("map", "i32", (n,), (1,), 1, fn="and_mask", iparam=(0xFF,), name="r"),
    ]
    return Program("gather_three_roots", nodes, [2, 3, 4], index_bound={"idx": n_src, "x": 1 << 30})


def histogram_2d(rows=64, n=4096, bins=256):
    """The scatter histogram of config 5 over a rank-2 array of keys, with per-row totals beside it: the
    scatter and the row folds share producers but no kernel walk."""
    sh = (rows, n)
    nodes = [
        _inp("keys", "u32", sh),
        _inp("zeros", "f32", (bins,)),
        Node("map", "u32", sh, (0,), 1, fn="mul_mod", iparam=(40503, bins), name="k"),
        Node("generate", "f32", sh, (), 0, fn="imod_to_f32", iparam=(7,), name="vals"),
        Node("permute", "f32", (bins,), (1, 2, 3), 3, fn="add", name="hist"),
        Node("fold", "f32", (rows,), (3,), 1, fn="add", name="row_totals"),
    ]
    return Program("histogram_2d", nodes, [4, 5], index_bound={"keys": 1 << 20})


def fold_of_scan(n=4099):
    """The largest prefix sum: a fold that consumes a scan.  Legal as one cluster; no kernel walks it so."""
    nodes = [
        _inp("x", "f32", (n,)),
        Node("scanl", "f32", (n,), (0,), 1, fn="add", name="s"),
        Node("fold", "f32", (), (1,), 1, fn="max", name="f"),
    ]
    return Program("fold_of_scan", nodes, [2])


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}


# --------------------------------------------------------------------------
# Seeded random DAGs (test programs nobody drew by hand)
# --------------------------------------------------------------------------

def random_program(seed, n=4099, rows=None, steps=None):
    """A seeded random DAG: a body of element-wise nodes, reversals and gathers over arrays of one shape
    ((n,) or (rows, n)), then accumulating nodes (folds, scans, a scatter) at the leaves and possibly a map
    that reads a fold's result.  Every node without a consumer is an output.  The draws come from the
    counter-based generator of the input arrays, so the same seed names the same program everywhere."""
    from .inputs import counter_bits
    shape = (n,) if rows is None else (rows, n)
    count = n if rows is None else rows * n
    draws = iter(counter_bits(seed, 63, 96).tolist())

    def pick(k):
        return ((next(draws) & ((1 << 63) - 1)) >> 20) % k

    nodes = [_inp("x", "f32", shape), _inp("v", "f32", shape), _inp("idx", "i32", shape)]
    arrays = [0, 1]
    affine = [(2.0, 1.0), (-0.5, 0.25), (1.0, -3.0), (0.125, 0.0)]

    def add(node):
        nodes.append(node)
        node.name = "%s%d" % (node.kind[0], len(nodes) - 1)
        return len(nodes) - 1

    def some():
        return arrays[pick(len(arrays))]

    for _ in range(3 + pick(3) if steps is None else steps):
        k = pick(6)
        if k == 0:
            i = add(Node("map", "f32", shape, (some(),), 1, fn="affine", fparam=affine[pick(4)]))
        elif k in (1, 2):
            i = add(Node("zipwith", "f32", shape, (some(), some()), 2, fn=("add", "mul", "mul_add_const", "add_scale")[pick(4)],
                         fparam=(0.75,)))
        elif k == 3:
            i = add(Node("backpermute", "f32", shape, (some(),), 1, idx_fn="reverse"))
        elif k == 4:
            i = add(Node("gather", "f32", shape, (2, some()), 2))
        else:
            i = add(Node("zipwith", "f32", shape, (some(), some(), some()), 3, fn="add3"))
        arrays.append(i)
    folded = shape[:-1]
    fold = None
    for _ in range(1 + pick(2)):
        k = pick(6)
        if k == 0:
            fold = add(Node("fold", "f32", folded, (some(),), 1, fn="add"))
        elif k == 1:
            fold = add(Node("fold", "f32", folded, (some(),), 1, fn="max"))
        elif k == 2:
            add(Node("scanl", "f32", shape, (some(),), 1, fn="add"))
        elif k == 3:
            add(Node("scanr", "f32", shape, (some(),), 1, fn="max"))
        elif k == 4:
            add(Node("scanl", "f32", shape, (some(),), 1, fn="add", fparam=(0.5,), exclusive=True))
        else:
            add(Node("permute", "f32", shape, (some(), 2, some()), 3, fn="add"))
    if fold is not None and pick(2):
        add(Node("map", "f32", shape, (some(), fold), 1, fn="add_free"))
    used = {s for nd in nodes for s in nd.inputs}
    outputs = [i for i, nd in enumerate(nodes) if nd.kind != "input" and i not in used]
    return Program("random%s_%d" % ("" if rows is None else "2d", seed), nodes, outputs, index_bound={"idx": count})


def random_int_program(seed, n=4099, rows=None):
    """The integer counterpart of `random_program`: wrapping int32 arithmetic, hashes and masks, generated
    arrays, reversals, gathers, (rank 2) clamped shifts by up to three cells and (square) transposes; folds, scans and scatters with
    +, min and max at the leaves.  Every result is exact, so every array compares bit for bit."""
    from .inputs import counter_bits
    shape = (n,) if rows is None else (rows, n)
    count = n if rows is None else rows * n
    draws = iter(counter_bits(seed, 62, 96).tolist())

    def pick(k):
        return ((next(draws) & ((1 << 63) - 1)) >> 20) % k

    nodes = [_inp("x", "i32", shape), _inp("v", "i32", shape), _inp("idx", "i32", shape)]
    arrays = [0, 1]
    unary = [("hash_mul_xorshift", (2654435761, 13)), ("and_mask", (0xFFFF,)), ("mul_const", (3,)), ("add_const", (-7,)),
             ("identity", ())]

    def add(node):
        nodes.append(node)
        node.name = "%s%d" % (node.kind[0], len(nodes) - 1)
        return len(nodes) - 1

    def some():
        return arrays[pick(len(arrays))]

    for _ in range(3 + pick(3)):
        k = pick(7)
        if k == 0:
            fn, ip = unary[pick(len(unary))]
            i = add(Node("map", "i32", shape, (some(),), 1, fn=fn, iparam=ip))
        elif k in (1, 2):
            i = add(Node("zipwith", "i32", shape, (some(), some()), 2, fn=("add", "mul")[pick(2)]))
        elif k == 3:
            i = add(Node("backpermute", "i32", shape, (some(),), 1, idx_fn="reverse"))
        elif k == 4:
            i = add(Node("gather", "i32", shape, (2, some()), 2))
        elif k == 5:
            i = add(Node("generate", "i32", shape, (), 0, fn="iota"))
        elif rows is None:
            i = add(Node("map", "i32", shape, (some(),), 1, fn="and_mask", iparam=(0xFF,)))
        elif rows == n and pick(2):                      # square arrays only: read across the diagonal
            i = add(Node("backpermute", "i32", shape, (some(),), 1, idx_fn="transpose"))
        else:
            i = add(Node("backpermute", "i32", shape, (some(),), 1, idx_fn="shift_clamp", iparam=(pick(7) - 3, pick(7) - 3)))
        arrays.append(i)
    folded = shape[:-1]
    ops = ("add", "min", "max")
    for _ in range(1 + pick(3)):
        k = pick(5)
        if k == 0:
            add(Node("fold", "i32", folded, (some(),), 1, fn=ops[pick(3)]))
        elif k == 1:
            add(Node("scanl", "i32", shape, (some(),), 1, fn=ops[pick(3)]))
        elif k == 2:
            add(Node("scanr", "i32", shape, (some(),), 1, fn=ops[pick(3)]))
        elif k == 3:
            add(Node("scanr", "i32", shape, (some(),), 1, fn="add", iparam=(1000,), exclusive=True))
        else:
            add(Node("permute", "i32", shape, (some(), 2, some()), 3, fn=ops[pick(3)]))
    used = {s for nd in nodes for s in nd.inputs}
    outputs = [i for i, nd in enumerate(nodes) if nd.kind != "input" and i not in used]
    return Program("random_int%s_%d" % ("" if rows is None else "sq" if rows == n else "2d", seed), nodes, outputs,
                   index_bound={"idx": count})
