"""Shared pieces of the GPU parity tests: run a program through the C ABI, run the
oracle on the same inputs, compare array by array."""
import numpy as np

from oracle import interp, legality

TOL = 1e-5          # |gpu - oracle_fp64| <= TOL * sum|x_i| for fp32 folds, scans and scatters


def oracle_run(prog, inputs_np):
    return interp.run(prog.nodes, inputs_np)


def accumulating(nd):
    return nd.kind in ("fold", "foldseg", "scanl", "scanr", "permute") and nd.dtype == "f32"


def count_of(nd):
    return int(np.prod(nd.shape, dtype=np.int64)) if len(nd.shape) else 1


def gpu_run(prog, inputs_t, pi=None, executor=None, bind_all=True, runs=1, recompute=0):
    """Runs `prog` on the GPU.  pi=None with executor=UNFUSED runs one kernel per node.
    recompute > 0: pi is checked under the recomputing rules with that depth.
    Returns ({node: numpy array} for every manifest non-input node, Graph)."""
    import torch
    from paper_2407_13585_b200 import binding as B

    executor = B.FUSED if executor is None else executor
    g = B.Graph(prog.nodes, prog.outputs)
    if pi is not None:
        if recompute:
            g.set_partition_recompute(pi, recompute)
        else:
            g.set_partition(pi)
    bufs = {}
    for i, nd in enumerate(prog.nodes):
        if nd.kind == "input":
            bufs[i] = inputs_t[i].cuda().contiguous()
            g.bind(i, bufs[i])
        elif bind_all or i in prog.outputs:
            bufs[i] = torch.full((max(count_of(nd), 4),), -12345, dtype=torch.int32, device="cuda")
            g.bind(i, bufs[i])
    for _ in range(runs):
        g.run(executor)
    torch.cuda.synchronize()
    man = [True] * len(prog.nodes) if executor == B.UNFUSED else g.manifest()
    out = {}
    for i, nd in enumerate(prog.nodes):
        if nd.kind == "input" or not man[i] or i not in bufs:
            continue
        a = bufs[i][:count_of(nd)].cpu().numpy()
        a = a.view(np.float32) if nd.dtype == "f32" else a.view(np.uint32)
        out[i] = a.reshape(tuple(nd.shape))
    return out, g


def error_bounds(prog, ref):
    """Per element, how far an fp32 array may lie from the oracle's: for a fold, scan or scatter the stated
    tolerance; for maps and zipWiths of such arrays that tolerance carried through the function to first
    order (plus the second-order term of a product) and two roundings of the result; for backpermutes and
    gathers of such arrays the bound of the element each output element reads."""
    nodes, b = prog.nodes, {}
    for i, nd in enumerate(nodes):
        if nd.dtype != "f32":
            continue
        if accumulating(nd):
            b[i] = TOL * ref.abs_sum[i] + np.abs(ref.exact[i]) * 2.0 ** -24 + 1e-30
            continue
        ins = nd.inputs[:nd.n_array]
        if nd.kind in ("backpermute", "gather"):
            # an index map moves values, it computes nothing: each element inherits the bound of the
            # source element it reads (Section 2: ys[j] = xs[f(j)], ys[j] = as[is[j]])
            src = nd.inputs[0] if nd.kind == "backpermute" else nd.inputs[1]
            if src not in b:
                continue
            count = count_of(nd)
            if nd.kind == "backpermute":
                from oracle import functions as fns
                at = fns.INDEX_FNS[nd.idx_fn](np.arange(count, dtype=np.int64), tuple(nd.shape), ref.values[src].shape, nd.iparam)
            else:
                at = ref.values[nd.inputs[0]].astype(np.int64).reshape(-1)
            whole = np.broadcast_to(np.asarray(b[src], dtype=np.float64), ref.values[src].shape).reshape(-1)
            b[i] = whole[at].reshape(tuple(nd.shape))
            continue
        if nd.kind not in ("map", "zipwith") or not any(j in b for j in nd.inputs):
            continue
        mag = lambda j: np.abs(ref.values[j].astype(np.float64))
        eb = lambda j: b.get(j, 0.0)
        if nd.fn == "affine":
            e = abs(nd.fparam[0]) * eb(ins[0])
        elif nd.fn == "identity":
            e = eb(ins[0])
        elif nd.fn in ("add", "add3"):
            e = sum(eb(j) for j in ins)
        elif nd.fn in ("mul", "mul_add_const"):
            e = mag(ins[0]) * eb(ins[1]) + mag(ins[1]) * eb(ins[0]) + eb(ins[0]) * eb(ins[1])
        elif nd.fn == "add_scale":
            e = abs(nd.fparam[0]) * (eb(ins[0]) + eb(ins[1]))
        elif nd.fn == "add_free":
            e = eb(ins[0]) + np.max(eb(nd.inputs[1]))
        else:
            continue
        b[i] = e * (1 + 2.0 ** -20) + np.abs(ref.values[i].astype(np.float64)) * 2.0 ** -22 + 1e-30
    return b


def compare(prog, ref, got, what=""):
    """Element-by-element comparison of every array in `got` with the oracle result `ref`.

    Integer arrays and fp32 element chains: bit-exact.  fp32 fold/scan/scatter outputs:
    |gpu - fp64 reference| <= 1e-5 * sum|x_i| (+ half an ulp of the result for the final
    rounding).  A map that divides such an output by such a total inherits both bounds, and so do other
    maps and zipWiths of such outputs (error_bounds).
    """
    nodes = prog.nodes
    loose = set()
    for i, nd in enumerate(nodes):
        if accumulating(nd) or any(s in loose for s in nd.inputs):
            loose.add(i)
    bounds = error_bounds(prog, ref)
    for i, a in got.items():
        nd = nodes[i]
        r = ref.values[i]
        assert a.shape == r.shape, (what, i, a.shape, r.shape)
        if i not in loose:
            au, ru = a.view(np.uint32).reshape(-1), r.view(np.uint32).reshape(-1)
            if not np.array_equal(au, ru):
                bad = np.flatnonzero(au != ru)
                raise AssertionError(f"{what} node {i} ({nd.name}): {bad.size} of {a.size} elements differ, first at "
                                     f"{bad[0]}: gpu {a.reshape(-1)[bad[0]]!r} oracle {r.reshape(-1)[bad[0]]!r}")
            continue
        if accumulating(nd):
            exact, scale = ref.exact[i], ref.abs_sum[i]
            bound = TOL * scale + np.abs(exact) * 2.0 ** -24 + 1e-30
            err = np.abs(a.astype(np.float64) - exact)
            assert np.all(err <= bound), (what, i, nd.name, float((err / bound).max()))
        elif nd.fn == "div_free":
            h, t = nd.inputs[0], nd.inputs[1]
            he, te = ref.exact[h], float(ref.exact[t])
            frac = he / te
            bound = ((TOL * ref.abs_sum[h] + np.abs(frac) * TOL * float(ref.abs_sum[t])) / abs(te)
                     + np.abs(frac) * 2.0 ** -22 + 1e-30)
            err = np.abs(a.astype(np.float64) - frac)
            undefined = np.isnan(frac)             # 0/0 when the total is zero: both sides must say so
            assert np.array_equal(np.isnan(a), undefined), (what, i, nd.name)
            assert np.all((err <= bound) | undefined), (what, i, nd.name, float(np.nanmax(err / bound)))
        elif i in bounds:
            err = np.abs(a.astype(np.float64) - r.astype(np.float64))
            assert np.all(err <= bounds[i]), (what, i, nd.name, float((err / bounds[i]).max()))
        else:
            raise AssertionError(f"{what} node {i} ({nd.name}, {nd.kind} {nd.fn}): an fp32 array downstream of a fold, scan or "
                                 "scatter with no error bound derived for it")


def all_partitions(prog):
    return legality.enumerate_partitions(prog.nodes, prog.outputs)
