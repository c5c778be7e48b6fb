"""Second, independent evaluator: the loop that a legal cluster denotes
(test infrastructure, CPU only; pure Python loops, small sizes).

Section 3.3 of the paper shows by example (simple1, simple2, simple4, simple5)
what one fused cluster means: a single loop over the *output* index space in
which indices are first pushed backwards through every gather-like node and
the element functions are then applied in their normal order.  A map pulls the
same index from its inputs, a gather pulls `is[j]` and then pulls its source at
that index, a fold opens an inner loop over the innermost extent of its source,
and anything produced outside the cluster is read from memory.  Clusters run
in ascending cluster number and only manifest arrays are written.

For a legal clustering this must give the arrays of the node-at-a-time
interpreter; the tests check that over every legal clustering of the small
programs.  fp32 accumulations are carried in fp64 as in the interpreter.
"""
import numpy as np

from . import functions as fns
from .interp import to_internal, _np_dtype, _count, F32, F64, U32
from .legality import edges_of, manifest_set


def run(nodes, outputs, pi, inputs):
    """Returns {node id: array} for every manifest node (inputs included)."""
    edges = edges_of(nodes)
    man = manifest_set(nodes, outputs, pi, edges)
    mem = {}
    for i, nd in enumerate(nodes):
        if nd.kind == "input":
            mem[i] = to_internal(inputs[i], nd.dtype).reshape(tuple(nd.shape))
    numbers = sorted({pi[i] for i, nd in enumerate(nodes) if nd.kind != "input"})
    with np.errstate(over="ignore"):
        for c in numbers:
            members = [i for i, nd in enumerate(nodes) if nd.kind != "input" and pi[i] == c]
            ev = _Cluster(nodes, set(members), mem)
            done = {}
            for r in members:
                if r in man:
                    done[r] = ev.materialise(r)
            mem.update(done)           # visible to later clusters only
    return mem


class _Cluster:
    def __init__(self, nodes, members, mem):
        self.nodes, self.members, self.mem = nodes, members, mem
        self.scan_cache = {}

    def free(self, nd):
        return [self.mem[s].reshape(-1)[0] for s in nd.inputs[nd.n_array:]]

    def pull(self, a, j):
        """Element j (row-major linear index) of array a."""
        nd = self.nodes[a]
        if a not in self.members:
            return self.mem[a].reshape(-1)[j]
        k = nd.kind
        if k == "generate":
            v = fns.GENERATE_FNS[nd.fn](np.int64(j), tuple(nd.shape), *self.free(nd),
                                        nd.iparam, nd.fparam, nd.dtype)
            return _np_dtype(nd.dtype)(v)
        if k in ("map", "zipwith"):
            xs = [self.pull(s, j) for s in nd.inputs[:nd.n_array]]
            return _np_dtype(nd.dtype)(fns.SCALAR_FNS[nd.fn](*xs, *self.free(nd), nd.iparam, nd.fparam))
        if k == "backpermute":
            src = nd.inputs[0]
            sj = fns.INDEX_FNS[nd.idx_fn](int(j), tuple(nd.shape), tuple(self.nodes[src].shape), nd.iparam)
            return self.pull(src, int(sj))
        if k == "gather":
            i = int(self.pull(nd.inputs[0], j))
            return self.pull(nd.inputs[1], i)
        if k == "fold":
            return self.fold_at(a, j)[0]
        if k == "foldseg":
            off = self.mem[nd.inputs[1]].reshape(-1)
            return self.reduce_range(a, nd.inputs[0], int(off[j]), int(off[j + 1]))
        if k in ("scanl", "scanr"):
            return self.scan_row(a, j)
        raise ValueError(f"{k} cannot be pulled through")

    def fold_at(self, a, o):
        nd = self.nodes[a]
        src = nd.inputs[0]
        inner = tuple(self.nodes[src].shape)[-1]
        base = o * inner
        if nd.dtype == "f32":
            acc = float(self.pull(src, base))
            for t in range(1, inner):
                acc = float(fns.combine(nd.fn, F64(acc), F64(self.pull(src, base + t))))
            return F32(acc), acc
        acc = self.pull(src, base)
        for t in range(1, inner):
            acc = self._icombine(nd, acc, self.pull(src, base + t))
        return U32(acc), None

    def reduce_range(self, a, src, lo, hi):
        """fold(op) of src[lo:hi], left to right, fp32 data carried in fp64."""
        nd = self.nodes[a]
        if hi <= lo:
            raise ValueError("an empty segment has no value")
        if nd.dtype == "f32":
            acc = float(self.pull(src, lo))
            for t in range(lo + 1, hi):
                acc = float(fns.combine(nd.fn, F64(acc), F64(self.pull(src, t))))
            return F32(acc)
        acc = self.pull(src, lo)
        for t in range(lo + 1, hi):
            acc = self._icombine(nd, acc, self.pull(src, t))
        return U32(acc)

    def _icombine(self, nd, a, b):
        if nd.fn in ("min", "max") and nd.dtype == "i32":
            r = fns.combine(nd.fn, np.int32(np.uint32(a).view(np.int32)), np.int32(np.uint32(b).view(np.int32)))
            return np.int32(r).view(U32)
        return U32(fns.combine(nd.fn, U32(a), U32(b)))

    def scan_row(self, a, j):
        """Inclusive scan value at linear index j, by walking the row from its start."""
        nd = self.nodes[a]
        src = nd.inputs[0]
        inner = tuple(nd.shape)[-1]
        row, col = divmod(j, inner)
        key = (a, row)
        if key not in self.scan_cache:
            order = range(inner) if nd.kind == "scanl" else range(inner - 1, -1, -1)
            vals = {}
            acc = None
            excl = getattr(nd, "exclusive", False)
            if excl:                                   # seeded: position t gets what was combined before it
                acc = float(F32(nd.fparam[0])) if nd.dtype == "f32" else U32(int(nd.iparam[0]) & 0xFFFFFFFF)
            for t in order:
                x = self.pull(src, row * inner + t)
                if excl:
                    vals[t] = F32(acc) if nd.dtype == "f32" else U32(acc)
                if nd.dtype == "f32":
                    acc = float(x) if acc is None else float(fns.combine(nd.fn, F64(acc), F64(x)))
                else:
                    acc = x if acc is None else self._icombine(nd, acc, x)
                if not excl:
                    vals[t] = F32(acc) if nd.dtype == "f32" else U32(acc)
            self.scan_cache[key] = vals
        return self.scan_cache[key][col]

    def materialise(self, r):
        nd = self.nodes[r]
        shape = tuple(nd.shape)
        n = _count(shape)
        dt = _np_dtype(nd.dtype)
        out = np.empty(n, dtype=dt)
        if nd.kind == "permute":
            dest, ind, vals = nd.inputs[:3]
            acc = [float(v) if nd.dtype == "f32" else v for v in self.mem[dest].reshape(-1)]
            m = _count(tuple(self.nodes[ind].shape))
            for j in range(m):
                i = int(self.pull(ind, j))
                x = self.pull(vals, j)
                if nd.dtype == "f32":
                    acc[i] = float(fns.combine(nd.fn, F64(acc[i]), F64(x)))
                else:
                    acc[i] = self._icombine(nd, acc[i], x)
            out[:] = acc
        else:
            for j in range(n):
                out[j] = self.pull(r, j)
        return out.reshape(shape)
