"""Seeded input arrays for the benchmark programs.

Every array is a pure function of (seed, stream, element index): element i of
stream s is derived from the 64-bit SplitMix64 output function applied to the
counter  seed * 2**40 + s * 2**34 + i  (Steele, Lea & Flood 2014).  The arrays
can therefore be drawn on any device, in any chunking, with identical bits,
and the same tensor is handed to the oracle and to the CUDA library.

Distributions (as the benchmark configurations state them):
  uniform_f32   U[-1, 1) rounded to fp32
  normal_f32    N(0, 1) by Box-Muller in fp64, rounded to fp32
  uniform_int   U{0 .. hi-1}, hi a power of two
  zipf_keys     rank r in 1..ids with P(r) ~ r**-s, key = r-1, by inverse CDF
"""
import math

import torch

_GOLDEN = -7046029254386353131          # 0x9E3779B97F4A7C15 as int64
_MIX1 = -4658895280553007687            # 0xBF58476D1CE4E5B9
_MIX2 = -7723592293110705685            # 0x94D049BB133111EB


def _lsr(z, s):
    """Logical shift right of an int64 tensor."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def counter_bits(seed, stream, n, device="cpu", offset=0):
    """n 64-bit words (as int64 bit patterns) for counters offset .. offset+n-1."""
    ctr = torch.arange(offset, offset + n, dtype=torch.int64, device=device)
    ctr = ctr + (seed << 40) + (stream << 34)
    z = (ctr + 1) * _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MIX1
    z = (z ^ _lsr(z, 27)) * _MIX2
    return z ^ _lsr(z, 31)


def _unit_f64(bits):
    """53-bit uniform in [0, 1) as fp64."""
    return _lsr(bits, 11).to(torch.float64) * (1.0 / (1 << 53))


def _chunks(n, chunk=1 << 24):
    off = 0
    while off < n:
        m = min(chunk, n - off)
        yield off, m
        off += m


def uniform_f32(seed, stream, n, device="cpu"):
    out = torch.empty(n, dtype=torch.float32, device=device)
    for off, m in _chunks(n):
        u = _unit_f64(counter_bits(seed, stream, m, device, off))
        v = (u * 2.0 - 1.0).to(torch.float32)
        out[off:off + m] = torch.clamp(v, max=math.nextafter(1.0, 0.0))
    return out


def normal_f32(seed, stream, n, device="cpu"):
    out = torch.empty(n, dtype=torch.float32, device=device)
    for off, m in _chunks(n):
        u1 = _unit_f64(counter_bits(seed, stream, m, device, off))
        u2 = _unit_f64(counter_bits(seed, stream + 1, m, device, off))
        r = torch.sqrt(-2.0 * torch.log1p(-u1))          # 1-u1 in (0, 1]
        out[off:off + m] = (r * torch.cos(2.0 * math.pi * u2)).to(torch.float32)
    return out


def uniform_int(seed, stream, n, hi, dtype=torch.int32, device="cpu"):
    assert hi > 0 and hi & (hi - 1) == 0 and hi <= 1 << 31, "hi must be a power of two <= 2**31"
    out = torch.empty(n, dtype=dtype, device=device)
    for off, m in _chunks(n):
        b = _lsr(counter_bits(seed, stream, m, device, off), 33)   # 31 high bits
        out[off:off + m] = (b & (hi - 1)).to(dtype)
    return out


def zipf_keys(seed, stream, n, ids=1 << 20, s=1.1, device="cpu"):
    """Keys in [0, ids) with P(key = r-1) proportional to r**-s, as int32 bit patterns of uint32."""
    ranks = torch.arange(1, ids + 1, dtype=torch.float64, device=device)
    cdf = torch.cumsum(ranks.pow(-s), 0)
    cdf = cdf / cdf[-1].clone()
    out = torch.empty(n, dtype=torch.int32, device=device)
    for off, m in _chunks(n):
        u = _unit_f64(counter_bits(seed, stream, m, device, off))
        key = torch.searchsorted(cdf, u, right=True)
        out[off:off + m] = torch.clamp(key, max=ids - 1).to(torch.int32)
    return out


def segment_offsets(seed, stream, n, segments, s=1.1, device="cpu"):
    """segments+1 int32 offsets over n elements: every segment non-empty, the lengths beyond one
    element shared out in proportion to r**-s over a seeded shuffle of the ranks r = 1..segments."""
    assert 1 <= segments <= n
    order = torch.argsort(counter_bits(seed, stream, segments, device))       # a seeded permutation
    w = torch.empty(segments, dtype=torch.float64, device=device)
    w[order] = torch.arange(1, segments + 1, dtype=torch.float64, device=device).pow(-s)
    extra = torch.floor(w / w.sum() * (n - segments)).to(torch.int64)
    lengths = extra + 1
    lengths[order[0]] += n - int(lengths.sum())                                # the remainder goes to the longest
    off = torch.zeros(segments + 1, dtype=torch.int64, device=device)
    off[1:] = torch.cumsum(lengths, 0)
    return off.to(torch.int32)


def make_inputs(program, seed=0, device="cpu"):
    """Input tensors of a benchmark or fixture program, keyed by node id.

    uint32 arrays are stored as int32 tensors holding the same bits.
    """
    name = program.name
    nodes = program.nodes
    out = {}
    for stream, i in enumerate(program.input_ids()):
        nd = nodes[i]
        cnt = 1
        for e in nd.shape:
            cnt *= e
        st = 2 * stream
        if name == "config3" and nd.name == "x":
            t = uniform_int(seed, st, cnt, 1 << 31, device=device)
        elif name == "config3" and nd.name == "idx":
            assert cnt & (cnt - 1) == 0, "config 3 sizes are powers of two"
            t = uniform_int(seed, st, cnt, cnt, device=device)
        elif name == "segmented_sums" and nd.name == "offsets":
            t = segment_offsets(seed, st, nodes[program.id("xs")].shape[0], cnt - 1, device=device)
        elif name == "config4":
            t = normal_f32(seed, st, cnt, device=device)
        elif name == "config5" and nd.name == "keys":
            t = zipf_keys(seed, st, cnt, device=device)
        elif name == "histogram_2d" and nd.name == "zeros":
            t = torch.zeros(cnt, dtype=torch.float32, device=device)
        elif name == "config5" and nd.name == "zeros":
            t = torch.zeros(cnt, dtype=torch.float32, device=device)
        elif nd.dtype == "f32":
            t = uniform_f32(seed, st, cnt, device=device)
        else:
            # index-like fixture inputs: the caller passes the exclusive bound in `index_bound`
            bound = getattr(program, "index_bound", {}).get(nd.name, cnt)
            p2 = 1 << max(0, (bound - 1).bit_length())
            t = uniform_int(seed, st, cnt, max(p2, 1), device=device) % bound
            t = t.to(torch.int32)
        out[i] = t.reshape(nd.shape)
    return out
