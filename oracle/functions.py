"""Element-level functions of the oracle (test infrastructure, CPU only).

Each entry works alike on numpy scalars and numpy arrays, one IEEE operation
per numpy call, so fp32 chains are rounded after every operation and never
contracted into a fused multiply-add.  Integer functions act on the uint32
bit pattern with wrap-around (the paper leaves element functions abstract;
these are the ones the benchmark configurations name).
"""
import numpy as np

F32 = np.float32
U32 = np.uint32


def _f(p):
    return F32(p)


# scalar functions: fn(args..., free..., iparam, fparam)
def affine(x, ip, fp):
    return (_f(fp[0]) * x) + _f(fp[1])


def mul(a, b, ip, fp):
    return a * b


def add(a, b, ip, fp):
    return a + b


def add3(a, b, c, ip, fp):
    return (a + b) + c


def mul_add_const(a, b, ip, fp):
    return (a * b) + _f(fp[0])


def add_scale(a, b, ip, fp):
    return _f(fp[0]) * (a + b)


def div_free(x, free0, ip, fp):
    return x / free0


def add_free(x, free0, ip, fp):
    return x + free0


def identity(x, ip, fp):
    return x


def hash_mul_xorshift(v, ip, fp):
    return (v * U32(ip[0] & 0xFFFFFFFF)) ^ (v >> U32(ip[1]))


def and_mask(v, ip, fp):
    return v & U32(ip[0] & 0xFFFFFFFF)


def mul_mod(v, ip, fp):
    return (v * U32(ip[0] & 0xFFFFFFFF)) % U32(ip[1])


def mul_const(v, ip, fp):
    return v * U32(ip[0] & 0xFFFFFFFF)


def add_const(v, ip, fp):
    return v + U32(ip[0] & 0xFFFFFFFF)


SCALAR_FNS = {f.__name__: f for f in (
    affine, mul, add, add3, mul_add_const, add_scale, div_free, add_free, identity,
    hash_mul_xorshift, and_mask, mul_mod, mul_const, add_const)}


# generate functions: fn(linear_index, shape, free..., iparam, fparam) -> value of the node dtype
def iota(i, shape, ip, fp, dtype):
    return np.asarray(i).astype(F32 if dtype == "f32" else U32)


def imod_to_f32(i, shape, ip, fp, dtype):
    return (np.asarray(i) % ip[0]).astype(F32)


def row_index(i, shape, ip, fp, dtype):
    return (np.asarray(i) // shape[-1]).astype(U32)


def iota_plus_free(i, shape, free0, ip, fp, dtype):
    return np.asarray(i).astype(F32) + free0


GENERATE_FNS = {f.__name__: f for f in (iota, imod_to_f32, row_index, iota_plus_free)}


# index maps of backpermute: out linear index, out shape, src shape -> src linear index
def idx_identity(j, out_shape, src_shape, ip):
    return j


def idx_reverse(j, out_shape, src_shape, ip):
    total = int(np.prod(src_shape, dtype=np.int64))
    return total - 1 - j


def idx_transpose(j, out_shape, src_shape, ip):
    r, c = j // out_shape[1], j % out_shape[1]
    return c * src_shape[1] + r


def idx_shift_clamp(j, out_shape, src_shape, ip):
    r, c = j // out_shape[1], j % out_shape[1]
    rr = np.clip(r + ip[0], 0, src_shape[0] - 1)
    cc = np.clip(c + ip[1], 0, src_shape[1] - 1)
    return rr * src_shape[1] + cc


INDEX_FNS = {"identity": idx_identity, "reverse": idx_reverse,
             "transpose": idx_transpose, "shift_clamp": idx_shift_clamp}


# combine operators of fold / scan / permute
def combine(op, a, b):
    if op == "add":
        return a + b
    if op == "mul":
        return a * b
    if op == "min":
        return np.minimum(a, b)
    if op == "max":
        return np.maximum(a, b)
    raise KeyError(op)
