// Graph construction: node validation and edge classification (Sections 3.4 and 4.1).
#include "graph.h"

#include <cstdio>
#include <cstring>

namespace acc {

static thread_local char g_err[512] = "";

int set_error(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof g_err, fmt, ap);
  va_end(ap);
  return code;
}
const char* last_error() { return g_err; }
void clear_error() { g_err[0] = 0; }

static bool same_shape(const acc_node_desc& a, const acc_node_desc& b) {
  if (a.rank != b.rank) return false;
  for (int i = 0; i < a.rank; ++i)
    if (a.shape[i] != b.shape[i]) return false;
  return true;
}

static bool is_combine(int fn) { return fn == ACC_FN_ADD || fn == ACC_FN_MUL || fn == ACC_FN_MIN || fn == ACC_FN_MAX; }
static bool is_int(int dt) { return dt == ACC_I32 || dt == ACC_U32; }

// Number of array slots an element function takes, -1 if it is not a map/zipWith function;
// free_slots receives the number of free-variable slots it reads.
static int fn_arity(int fn, int* free_slots) {
  *free_slots = 0;
  switch (fn) {
    case ACC_FN_IDENTITY: case ACC_FN_AFFINE: case ACC_FN_HASH_MUL_XORSHIFT: case ACC_FN_AND_MASK:
    case ACC_FN_MUL_MOD: case ACC_FN_MUL_CONST: case ACC_FN_ADD_CONST:
      return 1;
    case ACC_FN_DIV_FREE: case ACC_FN_ADD_FREE:
      *free_slots = 1;
      return 1;
    case ACC_FN_MUL: case ACC_FN_ADD: case ACC_FN_MUL_ADD_CONST: case ACC_FN_ADD_SCALE:
      return 2;
    case ACC_FN_ADD3:
      return 3;
    default:
      return -1;
  }
}

// What an element function computes on: 1 = fp32 arithmetic, 2 = integer (bit-pattern) arithmetic,
// 0 = defined for both (identity, +, *).
static int fn_domain(int fn) {
  switch (fn) {
    case ACC_FN_AFFINE: case ACC_FN_DIV_FREE: case ACC_FN_ADD_FREE: case ACC_FN_MUL_ADD_CONST: case ACC_FN_ADD_SCALE:
    case ACC_FN_ADD3:
      return 1;
    case ACC_FN_HASH_MUL_XORSHIFT: case ACC_FN_AND_MASK: case ACC_FN_MUL_MOD: case ACC_FN_MUL_CONST: case ACC_FN_ADD_CONST:
      return 2;
    default:
      return 0;
  }
}

int add_node(Graph& g, const acc_node_desc& d) {
  const int id = (int)g.nodes.size();
  if (d.kind < ACC_INPUT || d.kind > ACC_SCANR) return set_error(ACC_ERR_ARG, "node %d: unknown kind %d", id, d.kind);
  if (d.dtype < ACC_F32 || d.dtype > ACC_U32) return set_error(ACC_ERR_DTYPE, "node %d: unknown dtype %d", id, d.dtype);
  if (d.rank < 0 || d.rank > 2) return set_error(ACC_ERR_SHAPE, "node %d: rank %d outside 0..2", id, d.rank);
  int64_t count = 1;
  for (int i = 0; i < d.rank; ++i) {
    if (d.shape[i] < 0) return set_error(ACC_ERR_SHAPE, "node %d: negative extent", id);
    count *= d.shape[i];
    // kernels index with signed 32-bit arithmetic and step past the end of a row by up to one tile
    // (2^14 elements) before they compare: leave that room
    if (count > ACC_MAX_ELEMENTS || d.shape[i] > ACC_MAX_ELEMENTS)
      return set_error(ACC_ERR_SHAPE, "node %d: more than 2^31 - 2^16 elements", id);
  }
  if (d.n_inputs < 0 || d.n_inputs > ACC_MAX_INPUTS || d.n_array_inputs < 0 || d.n_array_inputs > d.n_inputs)
    return set_error(ACC_ERR_ARG, "node %d: bad slot counts %d/%d", id, d.n_array_inputs, d.n_inputs);
  for (int s = 0; s < d.n_inputs; ++s)
    if (d.inputs[s] < 0 || d.inputs[s] >= id) return set_error(ACC_ERR_ARG, "node %d: slot %d names node %d", id, s, d.inputs[s]);
  auto in = [&](int s) -> const acc_node_desc& { return g.nodes[d.inputs[s]].d; };
  const int n_free = d.n_inputs - d.n_array_inputs;

  switch (d.kind) {
    case ACC_INPUT:
      if (d.n_inputs) return set_error(ACC_ERR_ARG, "node %d: an input has no slots", id);
      break;
    case ACC_GENERATE: {
      if (d.n_array_inputs) return set_error(ACC_ERR_ARG, "node %d: generate takes no array slot", id);
      const int fn = d.fn_id;
      if (fn != ACC_FN_IOTA && fn != ACC_FN_IMOD_TO_F32 && fn != ACC_FN_ROW_INDEX && fn != ACC_FN_IOTA_PLUS_FREE)
        return set_error(ACC_ERR_ARG, "node %d: %d is not a generate function", id, fn);
      if (n_free != (fn == ACC_FN_IOTA_PLUS_FREE ? 1 : 0)) return set_error(ACC_ERR_ARG, "node %d: wrong number of free slots", id);
      if ((fn == ACC_FN_IMOD_TO_F32 || fn == ACC_FN_IOTA_PLUS_FREE) && d.dtype != ACC_F32)
        return set_error(ACC_ERR_DTYPE, "node %d: function yields fp32", id);
      if (fn == ACC_FN_ROW_INDEX && !is_int(d.dtype)) return set_error(ACC_ERR_DTYPE, "node %d: function yields an integer", id);
      if (fn == ACC_FN_IMOD_TO_F32 && d.iparam[0] <= 0) return set_error(ACC_ERR_ARG, "node %d: modulus must be positive", id);
      if (d.rank == 0) return set_error(ACC_ERR_SHAPE, "node %d: generate of rank 0", id);
      break;
    }
    case ACC_MAP:
    case ACC_ZIPWITH: {
      int want_free = 0;
      const int ar = fn_arity(d.fn_id, &want_free);
      if (ar < 0) return set_error(ACC_ERR_ARG, "node %d: %d is not an element function", id, d.fn_id);
      if (d.n_array_inputs != ar || n_free != want_free)
        return set_error(ACC_ERR_ARG, "node %d: function %d takes %d array and %d free slots", id, d.fn_id, ar, want_free);
      if ((d.kind == ACC_MAP) != (ar == 1)) return set_error(ACC_ERR_ARG, "node %d: map takes one array, zipWith two or three", id);
      for (int s = 0; s < ar; ++s)
        if (!same_shape(in(s), d)) return set_error(ACC_ERR_SHAPE, "node %d: slot %d differs in shape", id, s);
      // element functions are typed: fp32 arithmetic on fp32 arrays, bit arithmetic on integer ones;
      // the generic ones (identity, +, *) keep the class of their operands
      const int domain = fn_domain(d.fn_id);               // 1 fp32, 2 integer, 0 either
      const bool want_int = domain == 2 || (domain == 0 && is_int(d.dtype));
      if (domain == 1 && d.dtype != ACC_F32) return set_error(ACC_ERR_DTYPE, "node %d: function %d yields fp32", id, d.fn_id);
      if (domain == 2 && !is_int(d.dtype)) return set_error(ACC_ERR_DTYPE, "node %d: function %d yields an integer", id, d.fn_id);
      for (int s = 0; s < d.n_inputs; ++s)
        if (is_int(in(s).dtype) != want_int)
          return set_error(ACC_ERR_DTYPE, "node %d: slot %d is %s, function %d works on %s", id, s, is_int(in(s).dtype) ? "integer" : "fp32",
                           d.fn_id, want_int ? "integers" : "fp32");
      if (d.fn_id == ACC_FN_MUL_MOD && d.iparam[1] <= 0) return set_error(ACC_ERR_ARG, "node %d: modulus must be positive", id);
      if (d.fn_id == ACC_FN_HASH_MUL_XORSHIFT && (d.iparam[1] < 0 || d.iparam[1] > 31))
        return set_error(ACC_ERR_ARG, "node %d: shift outside 0..31", id);
      break;
    }
    case ACC_BACKPERMUTE: {
      if (d.n_inputs != 1 || d.n_array_inputs != 1) return set_error(ACC_ERR_ARG, "node %d: backpermute takes one slot", id);
      const acc_node_desc& s = in(0);
      if (s.dtype != d.dtype) return set_error(ACC_ERR_DTYPE, "node %d: dtype differs from its source", id);
      switch (d.idx_fn_id) {
        case ACC_IDX_IDENTITY: case ACC_IDX_REVERSE:
          if (!same_shape(s, d)) return set_error(ACC_ERR_SHAPE, "node %d: shape differs from its source", id);
          break;
        case ACC_IDX_SHIFT_CLAMP:
          if (d.rank != 2 || !same_shape(s, d)) return set_error(ACC_ERR_SHAPE, "node %d: shift needs equal rank-2 shapes", id);
          break;
        case ACC_IDX_TRANSPOSE:
          if (d.rank != 2 || s.rank != 2 || s.shape[0] != d.shape[1] || s.shape[1] != d.shape[0])
            return set_error(ACC_ERR_SHAPE, "node %d: transpose needs an (R,C) result over a (C,R) source", id);
          break;
        default:
          return set_error(ACC_ERR_ARG, "node %d: unknown index map %d", id, d.idx_fn_id);
      }
      if (d.rank == 0) return set_error(ACC_ERR_SHAPE, "node %d: backpermute of rank 0", id);
      break;
    }
    case ACC_GATHER: {
      if (d.n_inputs != 2 || d.n_array_inputs != 2) return set_error(ACC_ERR_ARG, "node %d: gather takes {idx, src}", id);
      if (!is_int(in(0).dtype)) return set_error(ACC_ERR_DTYPE, "node %d: index array must be integer", id);
      if (!same_shape(in(0), d)) return set_error(ACC_ERR_SHAPE, "node %d: result must have the shape of idx", id);
      if (in(1).dtype != d.dtype) return set_error(ACC_ERR_DTYPE, "node %d: dtype differs from its source", id);
      if (d.rank == 0 || in(1).rank == 0) return set_error(ACC_ERR_SHAPE, "node %d: gather of rank 0", id);
      break;
    }
    case ACC_PERMUTE: {
      if (d.n_inputs != 3 || d.n_array_inputs != 3) return set_error(ACC_ERR_ARG, "node %d: permute takes {defaults, idx, vals}", id);
      if (!is_combine(d.fn_id)) return set_error(ACC_ERR_ARG, "node %d: %d is not a combine operator", id, d.fn_id);
      if (d.fn_id == ACC_FN_MUL || (d.fn_id != ACC_FN_ADD && d.dtype == ACC_F32))
        return set_error(ACC_ERR_UNSUPPORTED, "node %d: permute is built for + (all dtypes) and integer min/max", id);
      if (!same_shape(in(0), d) || in(0).dtype != d.dtype) return set_error(ACC_ERR_SHAPE, "node %d: result must match defaults", id);
      if (!is_int(in(1).dtype)) return set_error(ACC_ERR_DTYPE, "node %d: index array must be integer", id);
      if (!same_shape(in(1), in(2))) return set_error(ACC_ERR_SHAPE, "node %d: idx and vals differ in shape", id);
      if (in(2).dtype != d.dtype) return set_error(ACC_ERR_DTYPE, "node %d: vals differ in dtype", id);
      if (d.rank == 0) return set_error(ACC_ERR_SHAPE, "node %d: permute of rank 0", id);
      break;
    }
    case ACC_FOLD: {
      if (d.n_inputs != 1 || d.n_array_inputs != 1) return set_error(ACC_ERR_ARG, "node %d: fold takes one slot", id);
      if (!is_combine(d.fn_id)) return set_error(ACC_ERR_ARG, "node %d: %d is not a combine operator", id, d.fn_id);
      const acc_node_desc& s = in(0);
      if (s.rank < 1 || d.rank != s.rank - 1) return set_error(ACC_ERR_SHAPE, "node %d: fold lowers the rank by one", id);
      for (int i = 0; i < d.rank; ++i)
        if (d.shape[i] != s.shape[i]) return set_error(ACC_ERR_SHAPE, "node %d: outer extents differ from the source", id);
      if (s.shape[s.rank - 1] <= 0) return set_error(ACC_ERR_SHAPE, "node %d: fold over an empty extent has no value", id);
      if (s.dtype != d.dtype) return set_error(ACC_ERR_DTYPE, "node %d: dtype differs from its source", id);
      break;
    }
    case ACC_FOLDSEG: {
      if (d.n_inputs != 2 || d.n_array_inputs != 1) return set_error(ACC_ERR_ARG, "node %d: foldSeg takes {xs, offsets} with one array slot", id);
      if (!is_combine(d.fn_id)) return set_error(ACC_ERR_ARG, "node %d: %d is not a combine operator", id, d.fn_id);
      const acc_node_desc& s = in(0);
      const acc_node_desc& o = in(1);
      if (s.rank != 1 || d.rank != 1) return set_error(ACC_ERR_SHAPE, "node %d: foldSeg reduces a rank-1 array to a rank-1 array", id);
      if (o.rank != 1 || o.shape[0] != d.shape[0] + 1) return set_error(ACC_ERR_SHAPE, "node %d: S segments need S+1 offsets", id);
      if (!is_int(o.dtype)) return set_error(ACC_ERR_DTYPE, "node %d: offsets must be integer", id);
      if (s.dtype != d.dtype) return set_error(ACC_ERR_DTYPE, "node %d: dtype differs from its source", id);
      break;
    }
    case ACC_SCANL:
    case ACC_SCANR: {
      if (d.n_inputs != 1 || d.n_array_inputs != 1) return set_error(ACC_ERR_ARG, "node %d: scan takes one slot", id);
      if (!is_combine(d.fn_id)) return set_error(ACC_ERR_ARG, "node %d: %d is not a combine operator", id, d.fn_id);
      if (d.rank < 1 || !same_shape(in(0), d)) return set_error(ACC_ERR_SHAPE, "node %d: scan keeps the shape of its source", id);
      if (in(0).dtype != d.dtype) return set_error(ACC_ERR_DTYPE, "node %d: dtype differs from its source", id);
      break;
    }
  }
  for (int s = d.n_array_inputs; s < d.n_inputs; ++s)
    if (g.nodes[d.inputs[s]].count < 1) return set_error(ACC_ERR_SHAPE, "node %d: free variable %d is empty", id, s);

  Node n;
  n.d = d;
  n.count = count;
  g.nodes.push_back(n);
  for (int s = 0; s < d.n_inputs; ++s) {
    const Node& p = g.nodes[d.inputs[s]];
    const bool free_slot = s >= d.n_array_inputs;
    const bool dest = d.kind == ACC_PERMUTE && s == 0;
    const bool forced = (d.flags & ACC_FLAG_FORCE_SLOT(s)) != 0;
    const bool from_scatter = p.d.kind == ACC_PERMUTE;
    Edge e;
    e.a = d.inputs[s];
    e.b = id;
    e.slot = s;
    e.ordered = !(free_slot || dest || forced || from_scatter);
    e.fusible = e.ordered && !is_input(p);
    g.edges.push_back(e);
  }
  g.has_pi = false;
  return id;
}

}  // namespace acc
