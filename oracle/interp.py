"""Node-at-a-time interpreter of a combinator program (test infrastructure, CPU only).

Every node is evaluated in program order and its whole result is materialised
as a row-major numpy array, exactly as the paper's Section 2 defines each
combinator:

  generate     ys[i] = f(i)
  map/zipWith  ys[i] = f(xs1[i], ..., xsk[i])      (zipWith is a map over several arrays)
  gather       ys[j] = as[is[j]]                   (== map(lambda i: as!i, is))
  backpermute  ys[j] = xs[f(j)]                    (== gather(generate(sz, f), xs))
  fold         reduce the innermost extent, no seed, rank one lower
  scanl/scanr  inclusive running combine along each innermost row, left/right
               (exclusive=True: seeded with fparam[0] / iparam[0], element k leaves itself out)
  scatter      copy dest, then dest[i] = op(dest[i], x) for every (i, x) of src
               (Section 2's text has `f (src!i, x)`; the destructive-update
               sentence that follows fixes the reading dest[i] = f(dest[i], x))

fp32 element functions round after every operation.  Accumulating nodes
(fold, scan, scatter) on fp32 data are summed in fp64 and then rounded once:
that fp64 value is the reference against which the tolerance
1e-5 * sum|x_i| is taken, and `abs_sum` returns that sum per output element.
Integers are uint32 bit patterns with wrap-around.
"""
import numpy as np

from . import functions as fns

F32, F64, U32 = np.float32, np.float64, np.uint32


def _np_dtype(dt):
    return F32 if dt == "f32" else U32


def _count(shape):
    c = 1
    for e in shape:
        c *= int(e)
    return c


def to_internal(arr, dtype):
    """Caller array (fp32 / int32 / uint32 bits) -> oracle array (fp32 / uint32)."""
    a = np.ascontiguousarray(np.asarray(arr))
    if dtype == "f32":
        assert a.dtype == F32
        return a
    assert a.dtype.itemsize == 4
    return a.view(U32)


def to_external(arr, dtype):
    """Oracle array -> fp32, int32 (for 'i32') or uint32 array."""
    if dtype == "i32":
        return arr.view(np.int32)
    return arr


def _signed_view(a, dtype):
    return a.view(np.int32) if dtype == "i32" else a


class Result:
    """values[i]: the array of node i; exact[i]: fp64 result of an fp32
    accumulating node before the final rounding; abs_sum[i]: sum of |x| that
    entered each output of such a node (the tolerance scale)."""

    def __init__(self):
        self.values, self.exact, self.abs_sum = {}, {}, {}


def run(nodes, inputs, stop_after=None):
    """Evaluate nodes in order.  inputs: {node id: array}.  Returns a Result."""
    res = Result()
    val = res.values
    for i, nd in enumerate(nodes):
        shape = tuple(nd.shape)
        n = _count(shape)
        k = nd.kind
        free = [val[s].reshape(-1)[0] for s in nd.inputs[nd.n_array:]]
        if k == "input":
            out = to_internal(inputs[i], nd.dtype).reshape(shape)
            assert out.shape == shape, (nd.name, out.shape, shape)
        elif k == "generate":
            idx = np.arange(n, dtype=np.int64)
            out = fns.GENERATE_FNS[nd.fn](idx, shape, *free, nd.iparam, nd.fparam, nd.dtype)
            out = out.astype(_np_dtype(nd.dtype)).reshape(shape)
        elif k in ("map", "zipwith"):
            xs = [val[s] for s in nd.inputs[:nd.n_array]]
            for x in xs:
                if x.shape != shape:
                    raise ValueError(f"node {i}: input shape {x.shape} != {shape}")
            with np.errstate(over="ignore"):
                out = fns.SCALAR_FNS[nd.fn](*xs, *free, nd.iparam, nd.fparam)
            out = out.astype(_np_dtype(nd.dtype), copy=False)
        elif k == "backpermute":
            src = val[nd.inputs[0]]
            j = np.arange(n, dtype=np.int64)
            sidx = fns.INDEX_FNS[nd.idx_fn](j, shape, src.shape, nd.iparam)
            out = src.reshape(-1)[sidx].reshape(shape)
        elif k == "gather":
            ind = val[nd.inputs[0]].astype(np.int64)
            src = val[nd.inputs[1]].reshape(-1)
            if ind.size and (ind.min() < 0 or ind.max() >= src.size):
                raise IndexError(f"node {i}: gather index out of range")
            out = src[ind.reshape(-1)].reshape(shape)
        elif k == "fold":
            src = val[nd.inputs[0]]
            if src.ndim < 1 or src.shape[-1] == 0:
                raise ValueError(f"node {i}: fold over an empty extent has no value")
            out = _fold(res, i, nd, src).reshape(shape)
        elif k == "foldseg":
            out = _foldseg(res, i, nd, val[nd.inputs[0]], val[nd.inputs[1]])
        elif k in ("scanl", "scanr"):
            src = val[nd.inputs[0]]
            out = _scan(res, i, nd, src, k == "scanr")
        elif k == "permute":
            dest, ind, vals = (val[s] for s in nd.inputs[:3])
            out = _permute(res, i, nd, dest, ind, vals).reshape(shape)
        else:
            raise KeyError(k)
        val[i] = np.ascontiguousarray(out).reshape(shape)
        if stop_after is not None and i == stop_after:
            break
    return res


def _fold(res, i, nd, src):
    op = nd.fn
    if nd.dtype == "f32":
        s64 = src.astype(F64)
        if op == "add":
            ex = s64.sum(axis=-1)
        elif op == "mul":
            ex = s64.prod(axis=-1)
        else:
            ex = s64.min(axis=-1) if op == "min" else s64.max(axis=-1)
        res.exact[i] = ex
        res.abs_sum[i] = np.abs(s64).sum(axis=-1)
        return ex.astype(F32)
    s = _signed_view(src, nd.dtype)
    with np.errstate(over="ignore"):
        if op == "add":
            out = np.add.reduce(src, axis=-1, dtype=U32)
        elif op == "mul":
            out = np.multiply.reduce(src, axis=-1, dtype=U32)
        else:
            out = (s.min(axis=-1) if op == "min" else s.max(axis=-1)).view(U32)
    return np.asarray(out, dtype=U32)


def _foldseg(res, i, nd, src, offsets):
    """ys[s] = fold(op) of src[offsets[s] : offsets[s+1]] (rank-1 source, no seed: segments must be non-empty).
    The paper only names foldSeg; this is the reading the library documents."""
    off = offsets.reshape(-1).astype(np.int64)
    flat = src.reshape(-1)
    S = off.size - 1
    if S != int(np.prod(nd.shape, dtype=np.int64)):
        raise ValueError(f"node {i}: {S} segments for a result of shape {tuple(nd.shape)}")
    if off[0] < 0 or off[-1] > flat.size:
        raise IndexError(f"node {i}: segment offsets leave the source")
    if np.any(off[1:] <= off[:-1]):
        raise ValueError(f"node {i}: an empty segment has no value (offsets must increase)")
    op = nd.fn
    if nd.dtype == "f32":
        ex, ab = np.empty(S, F64), np.empty(S, F64)
        red = {"add": np.sum, "mul": np.prod, "min": np.min, "max": np.max}[op]
        for s in range(S):
            seg = flat[off[s]:off[s + 1]].astype(F64)
            ex[s], ab[s] = red(seg), np.abs(seg).sum()
        res.exact[i], res.abs_sum[i] = ex, ab
        return ex.astype(F32)
    out = np.empty(S, U32)
    view = _signed_view(flat, nd.dtype)
    with np.errstate(over="ignore"):
        for s in range(S):
            if op == "add":
                out[s] = np.add.reduce(flat[off[s]:off[s + 1]], dtype=U32)
            elif op == "mul":
                out[s] = np.multiply.reduce(flat[off[s]:off[s + 1]], dtype=U32)
            else:
                seg = view[off[s]:off[s + 1]]
                out[s] = np.asarray(seg.min() if op == "min" else seg.max()).astype(view.dtype).view(U32)
    return out


def _scan(res, i, nd, src, right):
    op = nd.fn
    a = src[..., ::-1] if right else src
    if getattr(nd, "exclusive", False):
        # seeded and exclusive: element k combines the seed and the k elements before it, which is
        # the inclusive scan of the row with the seed put in front and the last element dropped
        seed = np.asarray(nd.fparam[0] if nd.dtype == "f32" else nd.iparam[0]).astype(F32 if nd.dtype == "f32" else np.int64)
        seed = seed.astype(F32) if nd.dtype == "f32" else np.asarray(int(seed) & 0xFFFFFFFF, dtype=U32)
        front = np.broadcast_to(seed, a.shape[:-1] + (1,)).astype(a.dtype)
        a = np.concatenate([front, a[..., :-1]], axis=-1)
    if nd.dtype == "f32":
        a64 = a.astype(F64)
        ufunc = {"add": np.add, "mul": np.multiply, "min": np.minimum, "max": np.maximum}[op]
        ex = ufunc.accumulate(a64, axis=-1)
        ab = np.add.accumulate(np.abs(a64), axis=-1)
        if right:
            ex, ab = ex[..., ::-1], ab[..., ::-1]
        res.exact[i], res.abs_sum[i] = np.ascontiguousarray(ex), np.ascontiguousarray(ab)
        return ex.astype(F32)
    with np.errstate(over="ignore"):
        if op == "add":
            out = np.add.accumulate(a, axis=-1, dtype=U32)
        elif op == "mul":
            out = np.multiply.accumulate(a, axis=-1, dtype=U32)
        else:
            s = _signed_view(np.ascontiguousarray(a), nd.dtype)
            out = (np.minimum if op == "min" else np.maximum).accumulate(s, axis=-1).view(U32)
    return out[..., ::-1] if right else out


def _permute(res, i, nd, dest, ind, vals):
    op = nd.fn
    ind = ind.reshape(-1).astype(np.int64)
    vals = vals.reshape(-1)
    bins = dest.size
    if ind.size != vals.size:
        raise ValueError(f"node {i}: scatter indices and values differ in size")
    if ind.size and (ind.min() < 0 or ind.max() >= bins):
        raise IndexError(f"node {i}: scatter index out of range")
    if nd.dtype == "f32":
        if op != "add":
            out = dest.reshape(-1).astype(F64).copy()
            uf = {"mul": np.multiply, "min": np.minimum, "max": np.maximum}[op]
            uf.at(out, ind, vals.astype(F64))
            res.exact[i] = out.reshape(dest.shape)
            res.abs_sum[i] = np.abs(out).reshape(dest.shape)
            return out.astype(F32)
        d64 = dest.reshape(-1).astype(F64)
        ex = d64 + np.bincount(ind, weights=vals.astype(F64), minlength=bins)
        ab = np.abs(d64) + np.bincount(ind, weights=np.abs(vals.astype(F64)), minlength=bins)
        res.exact[i], res.abs_sum[i] = ex.reshape(dest.shape), ab.reshape(dest.shape)
        return ex.astype(F32)
    out = dest.reshape(-1).copy()
    with np.errstate(over="ignore"):
        if op == "add":
            np.add.at(out, ind, vals)
        elif op == "mul":
            np.multiply.at(out, ind, vals)
        else:
            s = out.view(np.int32) if nd.dtype == "i32" else out
            v = vals.view(np.int32) if nd.dtype == "i32" else vals
            (np.minimum if op == "min" else np.maximum).at(s, ind, v)
    return out
