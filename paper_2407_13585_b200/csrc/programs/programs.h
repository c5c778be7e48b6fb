// Build-time descriptions of the programs whose clusters are instantiated as kernels.
// Node ids follow the order in which the benchmark programs are built through the C ABI;
// only the structure matters here (kinds, functions, wiring): shapes and constants are
// run-time arguments.
#pragma once
#include "../cluster.h"

namespace acc {
namespace programs {

constexpr PNode input(int dtype, int rank) { return pnode(ACC_INPUT, dtype, rank, 0, 0, 0); }

// 1-D chain: y = map(a*x+b) x; z = backpermute(reverse) y; w = zipWith(*) z x; s = fold(+) w
constexpr CProgram chain1d() {
  CProgram p{5, 1ull << 4, {}};
  p.nodes[0] = input(ACC_F32, 1);
  p.nodes[1] = pnode(ACC_MAP, ACC_F32, 1, ACC_FN_AFFINE, 0, 1, 0);
  p.nodes[2] = pnode(ACC_BACKPERMUTE, ACC_F32, 1, 0, ACC_IDX_REVERSE, 1, 1);
  p.nodes[3] = pnode(ACC_ZIPWITH, ACC_F32, 1, ACC_FN_MUL, 0, 2, 2, 0);
  p.nodes[4] = pnode(ACC_FOLD, ACC_F32, 0, ACC_FN_ADD, 0, 1, 3);
  return p;
}

// 2-D: B = backpermute(transpose) A; C = zipWith(a*b+k) A B; rowsum = fold(+) C
constexpr CProgram transpose_reduce() {
  CProgram p{4, 1ull << 3, {}};
  p.nodes[0] = input(ACC_F32, 2);
  p.nodes[1] = pnode(ACC_BACKPERMUTE, ACC_F32, 2, 0, ACC_IDX_TRANSPOSE, 1, 0);
  p.nodes[2] = pnode(ACC_ZIPWITH, ACC_F32, 2, ACC_FN_MUL_ADD_CONST, 0, 2, 0, 1);
  p.nodes[3] = pnode(ACC_FOLD, ACC_F32, 1, ACC_FN_ADD, 0, 1, 2);
  return p;
}

// int32: g = map(hash) x; h = gather idx g; o = map(and mask) h; out = scanl(+) o
constexpr CProgram gather_scan() {
  CProgram p{6, 1ull << 5, {}};
  p.nodes[0] = input(ACC_I32, 1);
  p.nodes[1] = input(ACC_I32, 1);
  p.nodes[2] = pnode(ACC_MAP, ACC_I32, 1, ACC_FN_HASH_MUL_XORSHIFT, 0, 1, 0);
  p.nodes[3] = pnode(ACC_GATHER, ACC_I32, 1, 0, 0, 2, 1, 2);
  p.nodes[4] = pnode(ACC_MAP, ACC_I32, 1, ACC_FN_AND_MASK, 0, 1, 3);
  p.nodes[5] = pnode(ACC_SCANL, ACC_I32, 1, ACC_FN_ADD, 0, 1, 4);
  return p;
}

// One Jacobi iteration: five clamped shifts of X, t1 = c+n, t2 = t1+s, t3 = t2+e, Y = k*(t3+w)
constexpr CProgram jacobi_iteration() {
  CProgram p{10, 1ull << 9, {}};
  p.nodes[0] = input(ACC_F32, 2);
  for (int i = 1; i <= 5; ++i) p.nodes[i] = pnode(ACC_BACKPERMUTE, ACC_F32, 2, 0, ACC_IDX_SHIFT_CLAMP, 1, 0);
  p.nodes[6] = pnode(ACC_ZIPWITH, ACC_F32, 2, ACC_FN_ADD, 0, 2, 1, 2);
  p.nodes[7] = pnode(ACC_ZIPWITH, ACC_F32, 2, ACC_FN_ADD, 0, 2, 6, 3);
  p.nodes[8] = pnode(ACC_ZIPWITH, ACC_F32, 2, ACC_FN_ADD, 0, 2, 7, 4);
  p.nodes[9] = pnode(ACC_ZIPWITH, ACC_F32, 2, ACC_FN_ADD_SCALE, 0, 2, 8, 5);
  return p;
}

// A chain of Jacobi iterations (at most four): iteration t reads the result of iteration t - 1.
// The shifts are the five-point pattern, fixed at build time: centre, row above, row below, column
// to the right, column to the left.
constexpr CProgram jacobi_chain(int iters) {
  CProgram p{1 + 9 * iters, 1ull << (9 * iters), {}};
  p.nodes[0] = input(ACC_F32, 2);
  int prev = 0;
  constexpr int dr[5] = {0, -1, 1, 0, 0}, dc[5] = {0, 0, 0, 1, -1};
  for (int t = 0; t < iters; ++t) {
    const int base = 1 + 9 * t;
    for (int i = 0; i < 5; ++i)
      p.nodes[base + i] = fixed(pnode(ACC_BACKPERMUTE, ACC_F32, 2, 0, ACC_IDX_SHIFT_CLAMP, 1, prev), dr[i], dc[i]);
    p.nodes[base + 5] = pnode(ACC_ZIPWITH, ACC_F32, 2, ACC_FN_ADD, 0, 2, base + 0, base + 1);
    p.nodes[base + 6] = pnode(ACC_ZIPWITH, ACC_F32, 2, ACC_FN_ADD, 0, 2, base + 5, base + 2);
    p.nodes[base + 7] = pnode(ACC_ZIPWITH, ACC_F32, 2, ACC_FN_ADD, 0, 2, base + 6, base + 3);
    p.nodes[base + 8] = pnode(ACC_ZIPWITH, ACC_F32, 2, ACC_FN_ADD_SCALE, 0, 2, base + 7, base + 4);
    prev = base + 8;
  }
  return p;
}

// k = map(mul mod) keys; vals = generate(float(i mod m)); hist = permute(+) zeros k vals;
// total = fold(+) vals; frac = map(/ total!0) hist
constexpr CProgram histogram_diamond() {
  CProgram p{7, (1ull << 6) | (1ull << 4) | (1ull << 5), {}};
  p.nodes[0] = input(ACC_U32, 1);
  p.nodes[1] = input(ACC_F32, 1);
  p.nodes[2] = pnode(ACC_MAP, ACC_U32, 1, ACC_FN_MUL_MOD, 0, 1, 0);
  p.nodes[3] = pnode(ACC_GENERATE, ACC_F32, 1, ACC_FN_IMOD_TO_F32, 0, 0);
  p.nodes[4] = pnode(ACC_PERMUTE, ACC_F32, 1, ACC_FN_ADD, 0, 3, 1, 2, 3);
  p.nodes[5] = pnode(ACC_FOLD, ACC_F32, 0, ACC_FN_ADD, 0, 1, 3);
  p.nodes[6] = pnode(ACC_MAP, ACC_F32, 1, ACC_FN_DIV_FREE, 0, 1, 4, 5);
  return p;
}

// The histogram program when `total` regenerates `vals` in a kernel of its own (a clustering with a
// copy of `vals`): the scatter's cluster, in which `vals` now has no outside reader, and the copy
// with the fold.
constexpr CProgram histogram_scatter_only() {
  CProgram p{5, 1ull << 4, {}};
  p.nodes[0] = input(ACC_U32, 1);
  p.nodes[1] = input(ACC_F32, 1);
  p.nodes[2] = pnode(ACC_MAP, ACC_U32, 1, ACC_FN_MUL_MOD, 0, 1, 0);
  p.nodes[3] = pnode(ACC_GENERATE, ACC_F32, 1, ACC_FN_IMOD_TO_F32, 0, 0);
  p.nodes[4] = pnode(ACC_PERMUTE, ACC_F32, 1, ACC_FN_ADD, 0, 3, 1, 2, 3);
  return p;
}
constexpr CProgram generated_total() {
  CProgram p{2, 1ull << 1, {}};
  p.nodes[0] = pnode(ACC_GENERATE, ACC_F32, 1, ACC_FN_IMOD_TO_F32, 0, 0);
  p.nodes[1] = pnode(ACC_FOLD, ACC_F32, 0, ACC_FN_ADD, 0, 1, 0);
  return p;
}

inline constexpr CProgram kChain1d = chain1d();
inline constexpr CProgram kTransposeReduce = transpose_reduce();
inline constexpr CProgram kGatherScan = gather_scan();
inline constexpr CProgram kJacobi = jacobi_iteration();
inline constexpr CProgram kJacobiChain = jacobi_chain(4);
// The same programs for a hash whose modulus is a power of two (as many bins as a power of two).
constexpr CProgram with_pow2_hash(CProgram p) {
  p.nodes[2] = fixed(p.nodes[2], kPow2, kRunTime);
  return p;
}

inline constexpr CProgram kHistogram = histogram_diamond();
inline constexpr CProgram kHistogramScatterOnly = histogram_scatter_only();
inline constexpr CProgram kHistogramPow2 = with_pow2_hash(histogram_diamond());
inline constexpr CProgram kHistogramScatterOnlyPow2 = with_pow2_hash(histogram_scatter_only());
inline constexpr CProgram kGeneratedTotal = generated_total();

}  // namespace programs
}  // namespace acc
