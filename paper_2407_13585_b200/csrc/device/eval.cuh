// Per-element pull evaluation of a fused cluster (the loop a cluster denotes, Section 3.3):
// the value of a member at an index is obtained by pushing the index backwards through
// gather-like members and applying element functions on the way back; externals are read
// from memory.  Everything here is resolved at compile time from the cluster description,
// so a cluster compiles to straight-line register code.
//
// Values travel as raw 32-bit patterns (fp32 / int32 / uint32 all are 4 bytes); indices as
// small structs that remember whether four consecutive elements can be moved with one
// 128-bit access.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>
#include <type_traits>

#include "../cluster.h"

namespace acc {
namespace dev {

struct NodeArg {
  const void* ptr;   // external: its array; manifest member: where to write; else unused
  int32_t ip0, ip1;  // iparam[0..1] (uint32 constants keep their bit pattern)
  float fp0, fp1;    // fparam[0..1]
  int32_t R, C;      // shape as (rows, innermost extent); rank 1 -> R = 1; rank 0 -> 1 x 1
  // division by a run-time constant d without a divider and without a branch, filled by the
  // host (d = iparam[1] for ACC_FN_MUL_MOD, iparam[0] otherwise, 1 <= d < 2^32): for every 32-bit
  // v, with t = umulhi(v, div_mul):  v / d == (t + ((v - t) >> div_sh1)) >> div_sh2
  uint32_t div_mul, div_sh1, div_sh2;
  uint32_t div_mask;   // d - 1 when d is a power of two, else 0 (kernels built for such divisors use it)
};

// v / d and v mod d with the host's multiplier for d (see NodeArg).
__device__ __forceinline__ uint32_t div_by(uint32_t v, const NodeArg& p) {
  const uint32_t t = __umulhi(v, p.div_mul);
  return (t + ((v - t) >> p.div_sh1)) >> p.div_sh2;
}
// POW2: the kernel was built for divisors that are powers of two (cluster.h, kPow2): one AND.  Otherwise
// the multiplier sequence, which is right for every divisor (for d = 2^l its multiplier is 1 and the
// shifts do the work), with no test of the divisor per call.
template <bool POW2 = false>
__device__ __forceinline__ uint32_t mod_by(uint32_t v, uint32_t d, const NodeArg& p) {
  if constexpr (POW2) return v & p.div_mask;
  else return v - div_by(v, p) * d;
}

template <int N>
struct Args {
  NodeArg n[N];
  int32_t R, C;        // iteration domain of the cluster
  uint32_t* scratch;   // zeroed control/partials region of this cluster
  uint32_t* status;    // device status word of the run
  uint32_t spin_limit;
  int32_t grid;        // stride of the per-block partials of a fold
};

struct V4 { uint32_t v[4]; };

// ---- index kinds -------------------------------------------------------------------
struct Ix   { int r, c; };            // one element
struct Ix4  { int r, c; };            // c, c+1, c+2, c+3  (c % 4 == 0)
struct IxR4 { int r, c; };            // c, c-1, c-2, c-3  ((c-3) % 4 == 0)
struct IxS4 { int r, c, dc; };        // clamp(c+dc+i, 0, C-1) for i = 0..3, row r (c % 4 == 0)
struct IxG4 { Ix e[4]; };             // four unrelated positions

// Two kinds that move no data: IxPF4 asks L2 to fetch the lines of a chunk that will be read a
// few trips later, IxNone is what becomes of it behind an index map it cannot follow.  Evaluating
// a member at either one touches no array (values come back as zeros and are dropped).
struct IxPF4 { int r, c; };
struct IxNone { int r, c; };
template <class IX> struct is_prefetch { static constexpr bool value = false; };
template <> struct is_prefetch<IxPF4> { static constexpr bool value = true; };
template <> struct is_prefetch<IxNone> { static constexpr bool value = true; };

template <class IX> struct width_of { static constexpr int value = 4; };
template <> struct width_of<Ix> { static constexpr int value = 1; };
template <class IX> using val_of = std::conditional_t<width_of<IX>::value == 1, uint32_t, V4>;

__device__ __forceinline__ Ix lane(const Ix& i, int) { return i; }
__device__ __forceinline__ Ix lane(const Ix4& i, int j) { return Ix{i.r, i.c + j}; }
__device__ __forceinline__ Ix lane(const IxR4& i, int j) { return Ix{i.r, i.c - j}; }
__device__ __forceinline__ Ix lane(const IxG4& i, int j) { return i.e[j]; }
__device__ __forceinline__ Ix lane(const IxPF4& i, int j) { return Ix{i.r, i.c + j}; }
__device__ __forceinline__ Ix lane(const IxNone& i, int j) { return Ix{i.r, i.c + j}; }
__device__ __forceinline__ Ix lane_clamped(const IxS4& i, int j, int C) {
  return Ix{i.r, min(max(i.c + i.dc + j, 0), C - 1)};
}

// ---- loads -------------------------------------------------------------------------
__device__ __forceinline__ uint32_t ld1(const uint32_t* p, int C, const Ix& i) { return __ldg(p + (i.r * C + i.c)); }

__device__ __forceinline__ uint32_t ld(const uint32_t* p, int C, const Ix& i) { return ld1(p, C, i); }
__device__ __forceinline__ V4 ld(const uint32_t* p, int C, const Ix4& i) {
  const uint4 t = __ldg(reinterpret_cast<const uint4*>(p + (i.r * C + i.c)));
  return V4{{t.x, t.y, t.z, t.w}};
}
__device__ __forceinline__ V4 ld(const uint32_t* p, int C, const IxR4& i) {
  const uint4 t = __ldg(reinterpret_cast<const uint4*>(p + (i.r * C + i.c - 3)));
  return V4{{t.w, t.z, t.y, t.x}};
}
__device__ __forceinline__ V4 ld(const uint32_t* p, int C, const IxG4& i) {
  return V4{{ld1(p, C, i.e[0]), ld1(p, C, i.e[1]), ld1(p, C, i.e[2]), ld1(p, C, i.e[3])}};
}
__device__ __forceinline__ V4 ld(const uint32_t* p, int C, const IxPF4& i) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p + (i.r * C + i.c)));
  return V4{{0u, 0u, 0u, 0u}};
}
__device__ __forceinline__ V4 ld(const uint32_t*, int, const IxNone&) { return V4{{0u, 0u, 0u, 0u}}; }
// A row chunk shifted by dc columns: the aligned chunk itself plus the one element that
// slides in from the neighbouring chunk (|dc| = 1), clamped at the row ends.
__device__ __forceinline__ V4 ld(const uint32_t* p, int C, const IxS4& i) {
  if (i.dc == 0) return ld(p, C, Ix4{i.r, i.c});
  if (i.dc == 1) {
    const V4 t = ld(p, C, Ix4{i.r, i.c});
    return V4{{t.v[1], t.v[2], t.v[3], ld1(p, C, Ix{i.r, min(i.c + 4, C - 1)})}};
  }
  if (i.dc == -1) {
    const V4 t = ld(p, C, Ix4{i.r, i.c});
    return V4{{ld1(p, C, Ix{i.r, max(i.c - 1, 0)}), t.v[0], t.v[1], t.v[2]}};
  }
  return V4{{ld1(p, C, lane_clamped(i, 0, C)), ld1(p, C, lane_clamped(i, 1, C)),
             ld1(p, C, lane_clamped(i, 2, C)), ld1(p, C, lane_clamped(i, 3, C))}};
}

// ---- stores (only ever at the cluster's own iteration index) ------------------------
__device__ __forceinline__ void st(uint32_t* p, int C, const Ix& i, uint32_t v) { p[i.r * C + i.c] = v; }
__device__ __forceinline__ void st(uint32_t* p, int C, const Ix4& i, const V4& v) {
  *reinterpret_cast<uint4*>(p + (i.r * C + i.c)) = make_uint4(v.v[0], v.v[1], v.v[2], v.v[3]);
}

// ---- index maps of backpermute ------------------------------------------------------
// `self` carries the output shape and the map's constants, `src` the source shape.
template <int F> __device__ __forceinline__ Ix map1(const Ix& i, const NodeArg& self, const NodeArg& src) {
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else if constexpr (F == ACC_IDX_REVERSE) return Ix{src.R - 1 - i.r, src.C - 1 - i.c};
  else if constexpr (F == ACC_IDX_TRANSPOSE) return Ix{i.c, i.r};
  else return Ix{min(max(i.r + self.ip0, 0), src.R - 1), min(max(i.c + self.ip1, 0), src.C - 1)};
}

template <int F, class IX> __device__ __forceinline__ IxG4 map_lanes(const IX& i, const NodeArg& self, const NodeArg& src) {
  return IxG4{{map1<F>(lane(i, 0), self, src), map1<F>(lane(i, 1), self, src),
               map1<F>(lane(i, 2), self, src), map1<F>(lane(i, 3), self, src)}};
}
__device__ __forceinline__ IxG4 expand(const IxS4& i, int C) {
  return IxG4{{lane_clamped(i, 0, C), lane_clamped(i, 1, C), lane_clamped(i, 2, C), lane_clamped(i, 3, C)}};
}

template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const Ix& i, const NodeArg& self, const NodeArg& src) {
  return map1<F>(i, self, src);
}
template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const Ix4& i, const NodeArg& self, const NodeArg& src) {
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else if constexpr (F == ACC_IDX_REVERSE) return IxR4{src.R - 1 - i.r, src.C - 1 - i.c};
  else if constexpr (F == ACC_IDX_SHIFT_CLAMP) return IxS4{min(max(i.r + self.ip0, 0), src.R - 1), i.c, self.ip1};
  else return map_lanes<F>(i, self, src);
}
template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const IxR4& i, const NodeArg& self, const NodeArg& src) {
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else if constexpr (F == ACC_IDX_REVERSE) return Ix4{src.R - 1 - i.r, src.C - 1 - i.c};
  else return map_lanes<F>(i, self, src);
}
template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const IxG4& i, const NodeArg& self, const NodeArg& src) {
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else return map_lanes<F>(i, self, src);
}
template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const IxPF4& i, const NodeArg&, const NodeArg& src) {
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else if constexpr (F == ACC_IDX_REVERSE) return IxPF4{src.R - 1 - i.r, src.C - 4 - i.c};
  else return IxNone{0, 0};
}
template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const IxNone& i, const NodeArg&, const NodeArg&) { return i; }
// A shifted chunk names positions in the array it is applied to, which has the shape of
// the node that receives it (`self`); a further map acts on its four clamped lanes.
template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const IxS4& i, const NodeArg& self, const NodeArg& src) {
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else return map_lanes<F>(expand(i, self.C), self, src);
}

// ---- element functions ---------------------------------------------------------------
__device__ __forceinline__ float f_(uint32_t b) { return __uint_as_float(b); }
__device__ __forceinline__ uint32_t u_(float f) { return __float_as_uint(f); }

template <int FN, int P0 = kRunTime>
__device__ __forceinline__ uint32_t apply1(const NodeArg& p, uint32_t a, uint32_t free0) {
  if constexpr (FN == ACC_FN_IDENTITY) return a;
  else if constexpr (FN == ACC_FN_AFFINE) return u_(__fadd_rn(__fmul_rn(p.fp0, f_(a)), p.fp1));
  else if constexpr (FN == ACC_FN_DIV_FREE) return u_(__fdiv_rn(f_(a), f_(free0)));
  else if constexpr (FN == ACC_FN_ADD_FREE) return u_(__fadd_rn(f_(a), f_(free0)));
  else if constexpr (FN == ACC_FN_HASH_MUL_XORSHIFT) return (a * (uint32_t)p.ip0) ^ (a >> (uint32_t)p.ip1);
  else if constexpr (FN == ACC_FN_AND_MASK) return a & (uint32_t)p.ip0;
  else if constexpr (FN == ACC_FN_MUL_MOD) {
    const uint32_t t = a * (uint32_t)p.ip0;
    return mod_by<P0 == kPow2>(t, (uint32_t)p.ip1, p);
  }
  else if constexpr (FN == ACC_FN_MUL_CONST) return a * (uint32_t)p.ip0;
  else if constexpr (FN == ACC_FN_ADD_CONST) return a + (uint32_t)p.ip0;
  else { static_assert(FN < 0, "not a unary element function"); return 0; }
}

template <int FN, int DT>
__device__ __forceinline__ uint32_t apply2(const NodeArg& p, uint32_t a, uint32_t b) {
  if constexpr (FN == ACC_FN_MUL) { if constexpr (DT == ACC_F32) return u_(__fmul_rn(f_(a), f_(b))); else return a * b; }
  else if constexpr (FN == ACC_FN_ADD) { if constexpr (DT == ACC_F32) return u_(__fadd_rn(f_(a), f_(b))); else return a + b; }
  else if constexpr (FN == ACC_FN_MUL_ADD_CONST) return u_(__fadd_rn(__fmul_rn(f_(a), f_(b)), p.fp0));
  else if constexpr (FN == ACC_FN_ADD_SCALE) return u_(__fmul_rn(p.fp0, __fadd_rn(f_(a), f_(b))));
  else { static_assert(FN < 0, "not a binary element function"); return 0; }
}

template <int FN>
__device__ __forceinline__ uint32_t apply3(const NodeArg& p, uint32_t a, uint32_t b, uint32_t c) {
  static_assert(FN == ACC_FN_ADD3, "not a ternary element function");
  return u_(__fadd_rn(__fadd_rn(f_(a), f_(b)), f_(c)));
}

template <int FN, int DT>
__device__ __forceinline__ uint32_t generate1(const NodeArg& p, const Ix& i, uint32_t free0) {
  const uint32_t lin = (uint32_t)(i.r * p.C + i.c);
  if constexpr (FN == ACC_FN_IOTA) { if constexpr (DT == ACC_F32) return u_((float)lin); else return lin; }
  else if constexpr (FN == ACC_FN_IMOD_TO_F32) return u_((float)mod_by(lin, (uint32_t)p.ip0, p));
  else if constexpr (FN == ACC_FN_ROW_INDEX) return (uint32_t)i.r;
  else if constexpr (FN == ACC_FN_IOTA_PLUS_FREE) return u_(__fadd_rn((float)lin, f_(free0)));
  else { static_assert(FN < 0, "not a generate function"); return 0; }
}

// combine operators of fold / scan / permute
template <int FN, int DT>
__device__ __forceinline__ uint32_t combine(uint32_t a, uint32_t b) {
  if constexpr (DT == ACC_F32) {
    if constexpr (FN == ACC_FN_ADD) return u_(__fadd_rn(f_(a), f_(b)));
    else if constexpr (FN == ACC_FN_MUL) return u_(__fmul_rn(f_(a), f_(b)));
    else if constexpr (FN == ACC_FN_MIN) return u_(fminf(f_(a), f_(b)));
    else return u_(fmaxf(f_(a), f_(b)));
  } else if constexpr (DT == ACC_I32) {
    if constexpr (FN == ACC_FN_ADD) return a + b;
    else if constexpr (FN == ACC_FN_MUL) return a * b;
    else if constexpr (FN == ACC_FN_MIN) return (uint32_t)min((int)a, (int)b);
    else return (uint32_t)max((int)a, (int)b);
  } else {
    if constexpr (FN == ACC_FN_ADD) return a + b;
    else if constexpr (FN == ACC_FN_MUL) return a * b;
    else if constexpr (FN == ACC_FN_MIN) return min(a, b);
    else return max(a, b);
  }
}
template <int FN, int DT>
__device__ __forceinline__ uint32_t identity_of() {
  if constexpr (FN == ACC_FN_ADD) return DT == ACC_F32 ? u_(0.0f) : 0u;
  else if constexpr (FN == ACC_FN_MUL) return DT == ACC_F32 ? u_(1.0f) : 1u;
  else if constexpr (FN == ACC_FN_MIN) return DT == ACC_F32 ? 0x7F800000u : (DT == ACC_I32 ? 0x7FFFFFFFu : 0xFFFFFFFFu);
  else return DT == ACC_F32 ? 0xFF800000u : (DT == ACC_I32 ? 0x80000000u : 0u);
}

// ---- source index of a gather: the gathered value is a row-major linear index ----------
template <int SRC_RANK>
__device__ __forceinline__ Ix gather1(uint32_t k, const NodeArg& src) {
  if constexpr (SRC_RANK <= 1) return Ix{0, (int)k};
  else return Ix{(int)(k / (uint32_t)src.C), (int)(k % (uint32_t)src.C)};
}

// One step of a thread's running fold.  An fp32 sum carries a compensation term (Kahan's summation): one
// thread may add thousands of elements, and where their rounding errors do not cancel (equal addends) a
// plain running sum drifts beyond 1e-5 of the sum of magnitudes; with the term it stays within a few ulp.
template <int FN, int DT>
__device__ __forceinline__ void fold_step(uint32_t& acc, float& comp, uint32_t x) {
  if constexpr (FN == ACC_FN_ADD && DT == ACC_F32) {
    const float y = __fsub_rn(f_(x), comp);
    const float t = __fadd_rn(f_(acc), y);
    comp = __fsub_rn(__fsub_rn(t, f_(acc)), y);
    acc = u_(t);
  } else {
    acc = combine<FN, DT>(acc, x);
  }
}

// ---- the evaluator ----------------------------------------------------------------------
template <class CL, int I, class A, class IX>
__device__ __forceinline__ val_of<IX> eval(const A& a, const IX& ix);

// Read of external I at an index.  Skeletons that stage externals on chip overload this for
// their own index kinds.
template <class CL, int I, class A, class IX>
__device__ __forceinline__ val_of<IX> ld_ext(const A& a, const IX& ix) {
  return ld(reinterpret_cast<const uint32_t*>(a.n[I].ptr), a.n[I].C, ix);
}

// Skeletons that keep a MEMBER's values on chip (computed once over a tile, then read at
// several indices) say so per index kind, and supply the read.
template <class CL, int I, class IX> struct reads_staged { static constexpr bool value = false; };
template <class CL, int I, class A, class IX>
__device__ __forceinline__ val_of<IX> ld_staged(const A& a, const IX& ix);

template <class CL, int I, class A>
__device__ __forceinline__ uint32_t free_of(const A& a) {
  constexpr CNode nd = CL::c.nodes[I];
  if constexpr (nd.nin > nd.narr) return __ldg(reinterpret_cast<const uint32_t*>(a.n[nd.in[nd.narr]].ptr));
  else return 0u;
}

template <class CL, int I, class A, class IX>
__device__ __forceinline__ uint32_t eval_member1(const A& a, const IX& ix) {     // IX: any one-element index kind
  constexpr CNode nd = CL::c.nodes[I];
  if constexpr (nd.kind == ACC_GENERATE) {
    return generate1<nd.fn, nd.dtype>(a.n[I], lane(ix, 0), free_of<CL, I>(a));
  } else if constexpr (nd.kind == ACC_MAP) {
    return apply1<nd.fn, nd.p0>(a.n[I], eval<CL, nd.in[0]>(a, ix), free_of<CL, I>(a));
  } else if constexpr (nd.kind == ACC_ZIPWITH && nd.narr == 2) {
    return apply2<nd.fn, nd.dtype>(a.n[I], eval<CL, nd.in[0]>(a, ix), eval<CL, nd.in[1]>(a, ix));
  } else if constexpr (nd.kind == ACC_ZIPWITH && nd.narr == 3) {
    return apply3<nd.fn>(a.n[I], eval<CL, nd.in[0]>(a, ix), eval<CL, nd.in[1]>(a, ix), eval<CL, nd.in[2]>(a, ix));
  } else {
    static_assert(nd.kind < 0, "this combinator cannot be evaluated per element inside a cluster");
    return 0;
  }
}

template <class CL, int I, class A, class IX>
__device__ __forceinline__ val_of<IX> eval_here(const A& a, const IX& ix);

template <class CL, int I, class A, class IX>
__device__ __forceinline__ val_of<IX> eval(const A& a, const IX& ix) {
  if constexpr (reads_staged<CL, I, IX>::value) return ld_staged<CL, I>(a, ix);
  else return eval_here<CL, I>(a, ix);
}

// The value of node I at an index, computed here (even where a skeleton keeps it on chip:
// this is what fills that copy).
template <class CL, int I, class A, class IX>
__device__ __forceinline__ val_of<IX> eval_here(const A& a, const IX& ix) {
  constexpr CNode nd = CL::c.nodes[I];
  constexpr int W = width_of<IX>::value;
  if constexpr (!nd.member) {
    return ld_ext<CL, I>(a, ix);
  } else if constexpr (nd.kind == ACC_BACKPERMUTE) {
    return eval<CL, nd.in[0]>(a, map_index<nd.idxfn, nd.p0, nd.p1>(ix, a.n[I], a.n[nd.in[0]]));
  } else if constexpr (is_prefetch<IX>::value && (nd.kind == ACC_GATHER || nd.kind == ACC_FOLD || nd.kind == ACC_FOLDSEG)) {
    // where the data will be read from is not known before the data: only a gather's index
    // operand, read in the cluster's own order, can be fetched ahead
    if constexpr (nd.kind == ACC_GATHER) eval<CL, nd.in[0]>(a, ix);
    return V4{{0u, 0u, 0u, 0u}};
  } else if constexpr (nd.kind == ACC_GATHER) {
    constexpr int src_rank = CL::c.nodes[nd.in[1]].rank;
    const auto k = eval<CL, nd.in[0]>(a, ix);
    if constexpr (W == 1) {
      return eval<CL, nd.in[1]>(a, gather1<src_rank>(k, a.n[nd.in[1]]));
    } else {
      const NodeArg& s = a.n[nd.in[1]];
      return eval<CL, nd.in[1]>(a, IxG4{{gather1<src_rank>(k.v[0], s), gather1<src_rank>(k.v[1], s),
                                         gather1<src_rank>(k.v[2], s), gather1<src_rank>(k.v[3], s)}});
    }
  } else if constexpr (nd.kind == ACC_FOLD) {
    // a fold pulled through (Section 3.3, `simple4`): the requested output element selects a
    // row of the source, and an inner loop walks that row
    const NodeArg& s = a.n[nd.in[0]];
    auto row_value = [&](const Ix& o) {
      const int row = o.r * a.n[I].C + o.c;
      uint32_t acc = identity_of<nd.fn, nd.dtype>();
      float comp = 0.0f;
      for (int j = 0; j < s.C; ++j) fold_step<nd.fn, nd.dtype>(acc, comp, eval<CL, nd.in[0]>(a, Ix{row, j}));
      return acc;
    };
    if constexpr (W == 1) {
      return row_value(ix);
    } else if constexpr (std::is_same<IX, IxS4>::value) {
      return V4{{row_value(lane_clamped(ix, 0, a.n[I].C)), row_value(lane_clamped(ix, 1, a.n[I].C)),
                 row_value(lane_clamped(ix, 2, a.n[I].C)), row_value(lane_clamped(ix, 3, a.n[I].C))}};
    } else {
      return V4{{row_value(lane(ix, 0)), row_value(lane(ix, 1)), row_value(lane(ix, 2)), row_value(lane(ix, 3))}};
    }
  } else if constexpr (nd.kind == ACC_FOLDSEG) {
    // a segmented fold pulled through: the requested element names a segment, an inner loop
    // walks it (offsets are clamped to the source so that a bad offset cannot leave it)
    const NodeArg& s = a.n[nd.in[0]];
    const int32_t* off = reinterpret_cast<const int32_t*>(a.n[nd.in[1]].ptr);
    auto seg_value = [&](const Ix& o) {
      const int lo = max(__ldg(off + o.c), 0), hi = min(__ldg(off + o.c + 1), s.R * s.C);
      uint32_t acc = identity_of<nd.fn, nd.dtype>();
      float comp = 0.0f;
      for (int j = lo; j < hi; ++j) fold_step<nd.fn, nd.dtype>(acc, comp, eval<CL, nd.in[0]>(a, Ix{0, j}));
      return acc;
    };
    if constexpr (W == 1) {
      return seg_value(ix);
    } else if constexpr (std::is_same<IX, IxS4>::value) {
      return V4{{seg_value(lane_clamped(ix, 0, a.n[I].C)), seg_value(lane_clamped(ix, 1, a.n[I].C)),
                 seg_value(lane_clamped(ix, 2, a.n[I].C)), seg_value(lane_clamped(ix, 3, a.n[I].C))}};
    } else {
      return V4{{seg_value(lane(ix, 0)), seg_value(lane(ix, 1)), seg_value(lane(ix, 2)), seg_value(lane(ix, 3))}};
    }
  } else if constexpr (W == 1) {
    return eval_member1<CL, I>(a, ix);
  } else if constexpr (nd.kind == ACC_GENERATE) {
    const uint32_t f0 = free_of<CL, I>(a);
    V4 out;
    if constexpr (std::is_same<IX, IxS4>::value) {
#pragma unroll
      for (int j = 0; j < 4; ++j) out.v[j] = generate1<nd.fn, nd.dtype>(a.n[I], lane_clamped(ix, j, a.n[I].C), f0);
    } else if constexpr (std::is_same<IX, Ix4>::value && nd.fn == ACC_FN_IMOD_TO_F32) {
      // one division for four consecutive indices: the remainders follow by stepping
      const uint32_t m = (uint32_t)a.n[I].ip0;
      uint32_t r[4];
      r[0] = mod_by((uint32_t)(ix.r * a.n[I].C + ix.c), m, a.n[I]);
#pragma unroll
      for (int j = 1; j < 4; ++j) r[j] = r[j - 1] + 1 == m ? 0u : r[j - 1] + 1;
      if (m <= (1u << 23)) {                   // then float(r) = bits(2^23 + r) - 2^23, no conversion unit
#pragma unroll
        for (int j = 0; j < 4; ++j) out.v[j] = u_(__fadd_rn(__uint_as_float(0x4B000000u | r[j]), -8388608.0f));
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) out.v[j] = u_((float)r[j]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) out.v[j] = generate1<nd.fn, nd.dtype>(a.n[I], lane(ix, j), f0);
    }
    return out;
  } else if constexpr (nd.kind == ACC_MAP) {
    const uint32_t f0 = free_of<CL, I>(a);
    const V4 x = eval<CL, nd.in[0]>(a, ix);
    V4 out;
#pragma unroll
    for (int j = 0; j < 4; ++j) out.v[j] = apply1<nd.fn, nd.p0>(a.n[I], x.v[j], f0);
    return out;
  } else if constexpr (nd.kind == ACC_ZIPWITH && nd.narr == 2) {
    const V4 x = eval<CL, nd.in[0]>(a, ix), y = eval<CL, nd.in[1]>(a, ix);
    V4 out;
#pragma unroll
    for (int j = 0; j < 4; ++j) out.v[j] = apply2<nd.fn, nd.dtype>(a.n[I], x.v[j], y.v[j]);
    return out;
  } else if constexpr (nd.kind == ACC_ZIPWITH && nd.narr == 3) {
    const V4 x = eval<CL, nd.in[0]>(a, ix), y = eval<CL, nd.in[1]>(a, ix), z = eval<CL, nd.in[2]>(a, ix);
    V4 out;
#pragma unroll
    for (int j = 0; j < 4; ++j) out.v[j] = apply3<nd.fn>(a.n[I], x.v[j], y.v[j], z.v[j]);
    return out;
  } else {
    static_assert(nd.kind < 0, "this combinator cannot be evaluated per element inside a cluster");
    return V4{};
  }
}

// ---- compile-time queries on the cluster --------------------------------------------------
constexpr bool is_elementwise(int kind) {
  return kind == ACC_GENERATE || kind == ACC_MAP || kind == ACC_ZIPWITH || kind == ACC_BACKPERMUTE || kind == ACC_GATHER;
}
constexpr bool is_store_root(const CNode& n) { return n.member && n.manifest && is_elementwise(n.kind); }
constexpr bool is_fold_root(const CNode& n) { return n.member && n.manifest && n.kind == ACC_FOLD; }
constexpr bool is_segfold_root(const CNode& n) { return n.member && n.manifest && n.kind == ACC_FOLDSEG; }
constexpr bool is_scan_root(const CNode& n) { return n.member && (n.kind == ACC_SCANL || n.kind == ACC_SCANR); }
constexpr bool is_permute_root(const CNode& n) { return n.member && n.kind == ACC_PERMUTE; }

template <int B, int E, class F>
__device__ __forceinline__ void static_for(F&& f) {
  if constexpr (B < E) {
    f(std::integral_constant<int, B>{});
    static_for<B + 1, E>(static_cast<F&&>(f));
  }
}

}  // namespace dev
}  // namespace acc
