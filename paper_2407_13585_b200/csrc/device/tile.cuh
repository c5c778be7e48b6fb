// k_tile_pair: the skeleton for rank-2 clusters that read an array both as it lies and
// transposed (a transposing backpermute fused into an element-wise producer).
//
// Evaluating `xs[c][r]` per output element straight from global memory reads a 32-byte sector
// for every 4 bytes.  Here one CTA owns the pair of output tiles (I,J) and (J,I) of a square
// domain.  It stages, for every rank-2 external, the two source tiles [I,J] and [J,I] in
// shared memory with coalesced 128-bit loads and stores, once; tile [I,J] then serves the
// direct reads of output tile (I,J) and the transposed reads of output tile (J,I), and tile
// [J,I] the other two.  Every external is read from HBM exactly once whatever mix of orders
// the cluster uses.
//
// A thread evaluates four consecutive ROWS of one output column.  Its transposed operand is
// then four consecutive words of one staged row (one 128-bit shared-memory load) and its
// direct operand four words one staged row apart; with a row stride of 68 words and a warp
// laid out as 16 columns x 2 row groups both accesses are free of bank conflicts.
//
// Row folds of the cluster end per tile in a half-warp shuffle tree; the per-tile partial of
// each row goes to scratch, and the CTA that delivers the last partial of a block of rows adds
// them up in a fixed order (so the result does not depend on arrival order) and writes them.
#pragma once
#include "skeletons.cuh"

namespace acc {
namespace dev {

constexpr int kTile = 64;                  // output tile edge
constexpr int kTileStride = kTile + 4;     // padded row of a staged tile, in words (16-byte aligned rows)
constexpr int kTileWords = kTile * kTileStride;

struct TileCtx {
  const uint32_t* smem;   // staged tiles: [external slot][2][kTileWords]
  int r0, c0;             // origin of the output tile being computed
  int direct;             // which of the two staged tiles lies like the output tile (0 or 1)
  int trans;              // which one holds the transposed positions (the same one on the diagonal)
};

// rows r..r+3 of output column c, read as they lie / read transposed
struct IxP4 { int r, c; const TileCtx* t; };
struct IxQ4 { int r, c; const TileCtx* t; };     // positions (c, r+j) of the source

__device__ __forceinline__ Ix lane(const IxP4& i, int j) { return Ix{i.r + j, i.c}; }
__device__ __forceinline__ Ix lane(const IxQ4& i, int j) { return Ix{i.c, i.r + j}; }

template <int F> __device__ __forceinline__ auto map_index(const IxP4& i, const NodeArg&, const NodeArg&) {
  static_assert(F == ACC_IDX_IDENTITY || F == ACC_IDX_TRANSPOSE, "only transposes are staged in tiles");
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else return IxQ4{i.r, i.c, i.t};
}
template <int F> __device__ __forceinline__ auto map_index(const IxQ4& i, const NodeArg&, const NodeArg&) {
  static_assert(F == ACC_IDX_IDENTITY || F == ACC_IDX_TRANSPOSE, "only transposes are staged in tiles");
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else return IxP4{i.r, i.c, i.t};
}

// Ordinal of external I among the staged externals (rank-2 externals read through array slots).
template <class CL> constexpr bool is_staged_external(int i) {
  const CNode& n = CL::c.nodes[i];
  if (n.member || n.rank != 2) return false;
  for (int j = 0; j < CL::c.n; ++j)
    for (int s = 0; s < CL::c.nodes[j].narr; ++s)
      if (CL::c.nodes[j].member && CL::c.nodes[j].in[s] == i) return true;
  return false;
}
template <class CL> constexpr int tile_slot(int i) {
  int k = 0;
  for (int j = 0; j < i; ++j) k += is_staged_external<CL>(j) ? 1 : 0;
  return k;
}
template <class CL> constexpr int staged_externals() { return tile_slot<CL>(CL::c.n); }

// A cluster can use this skeleton if transposes are its only index maps and every array it
// reads is a rank-2 external; its roots are rank-2 stores and row folds.
template <class CL> constexpr bool tile_eligible() {
  bool has_transpose = false;
  for (int i = 0; i < CL::c.n; ++i) {
    const CNode& n = CL::c.nodes[i];
    if (!n.member) {
      bool as_array = false;
      for (int j = 0; j < CL::c.n; ++j)
        for (int s = 0; s < CL::c.nodes[j].narr; ++s)
          if (CL::c.nodes[j].member && CL::c.nodes[j].in[s] == i) as_array = true;
      if (as_array && n.rank != 2) return false;
      continue;
    }
    switch (n.kind) {
      case ACC_MAP: case ACC_ZIPWITH: case ACC_GENERATE:
        if (n.rank != 2) return false;
        break;
      case ACC_BACKPERMUTE:
        if (n.idxfn == ACC_IDX_TRANSPOSE) has_transpose = true;
        else if (n.idxfn != ACC_IDX_IDENTITY) return false;
        break;
      case ACC_FOLD:
        if (!n.manifest || n.rank != 1) return false;     // a row fold that is a root
        for (int j = 0; j < CL::c.n; ++j)
          for (int s = 0; s < CL::c.nodes[j].nin; ++s)
            if (CL::c.nodes[j].member && CL::c.nodes[j].in[s] == i) return false;   // and only a root
        break;
      default:
        return false;
    }
  }
  return has_transpose && staged_externals<CL>() >= 1 && staged_externals<CL>() <= 3;
}

// loads from the staged tiles; `slot` is the external's ordinal
__device__ __forceinline__ V4 ld_tile(int slot, const IxP4& i) {
  const TileCtx& t = *i.t;
  const uint32_t* p = t.smem + (slot * 2 + t.direct) * kTileWords + (i.r - t.r0) * kTileStride + (i.c - t.c0);
  return V4{{p[0], p[kTileStride], p[2 * kTileStride], p[3 * kTileStride]}};
}
__device__ __forceinline__ V4 ld_tile(int slot, const IxQ4& i) {
  const TileCtx& t = *i.t;
  const uint32_t* p = t.smem + (slot * 2 + t.trans) * kTileWords + (i.c - t.c0) * kTileStride + (i.r - t.r0);
  const uint4 v = *reinterpret_cast<const uint4*>(p);     // r - r0 is a multiple of 4, rows are 16-byte aligned
  return V4{{v.x, v.y, v.z, v.w}};
}

template <class CL, int I, class A>
__device__ __forceinline__ V4 ld_ext(const A&, const IxP4& ix) { return ld_tile(tile_slot<CL>(I), ix); }
template <class CL, int I, class A>
__device__ __forceinline__ V4 ld_ext(const A&, const IxQ4& ix) { return ld_tile(tile_slot<CL>(I), ix); }

// Scratch layout (words): [0, row_blocks): arrival counters; from word align4(row_blocks):
// one partial per (row fold, column tile, row).
__host__ __device__ inline int64_t tile_partials_off(int row_blocks) { return (row_blocks + 3) & ~3; }

// Pair number p -> (I, J) with I <= J, rows of the upper triangle one after the other.
__device__ __forceinline__ void pair_of(uint32_t p, int T, int& I, int& J) {
  auto first = [T](int k) { return (uint32_t)k * (uint32_t)T - (uint32_t)(k * (k - 1) / 2); };   // first pair of row k
  const float w = (float)(2 * T + 1);
  int i = (int)((w - sqrtf(fmaxf(w * w - 8.0f * (float)p, 0.0f))) * 0.5f);
  i = max(0, min(i, T - 1));
  for (int guard = 0; guard < 4 && i > 0 && first(i) > p; ++guard) --i;
  for (int guard = 0; guard < 4 && i + 1 < T && first(i + 1) <= p; ++guard) ++i;
  I = i;
  J = min(i + (int)(p - first(i)), T - 1);
}

template <class CL, bool VEC>
__global__ void __launch_bounds__(kBlock) k_tile_pair(const __grid_constant__ Args<CL::c.n> a) {
  constexpr int N = CL::c.n;
  constexpr int NRF = count_if<CL>(is_row_fold);
  extern __shared__ __align__(16) uint32_t tiles[];
  __shared__ bool finishing[2];
  const int n = a.R;                                        // square domain: n x n
  const int blocks = (n + kTile - 1) / kTile;
  int I, J;
  pair_of(blockIdx.x, blocks, I, J);                        // one CTA per pair {(I,J),(J,I)}, I <= J

  // ---- stage source tiles [I,J] (buffer 0) and [J,I] (buffer 1) of every external ----------
  // 16 threads x 128 bits per row, 16 rows per pass
  {
    const int sx = threadIdx.x & 15, sy = threadIdx.x >> 4;
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      if constexpr (is_staged_external<CL>(i)) {
        constexpr int slot = tile_slot<CL>(i);
        const uint32_t* src = reinterpret_cast<const uint32_t*>(a.n[i].ptr);
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          if (b == 1 && I == J) break;
          const int row0 = (b == 0 ? I : J) * kTile, col0 = (b == 0 ? J : I) * kTile;
          uint32_t* dst = tiles + (slot * 2 + b) * kTileWords;
#pragma unroll
          for (int p = 0; p < kTile / 16; ++p) {
            const int r = sy + 16 * p, gr = row0 + r, gc = col0 + 4 * sx;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (gr < n) {
              if constexpr (VEC) {
                if (gc < n) v = __ldg(reinterpret_cast<const uint4*>(src + ((size_t)gr * n + gc)));
              } else {
                if (gc + 0 < n) v.x = __ldg(src + ((size_t)gr * n + gc + 0));
                if (gc + 1 < n) v.y = __ldg(src + ((size_t)gr * n + gc + 1));
                if (gc + 2 < n) v.z = __ldg(src + ((size_t)gr * n + gc + 2));
                if (gc + 3 < n) v.w = __ldg(src + ((size_t)gr * n + gc + 3));
              }
            }
            *reinterpret_cast<uint4*>(dst + r * kTileStride + 4 * sx) = v;
          }
        }
      }
    });
  }
  __syncthreads();

  uint32_t* counters = a.scratch;
  uint32_t* partials = a.scratch + tile_partials_off(blocks);
  const int cx = threadIdx.x & 15, rg = threadIdx.x >> 4;   // column within 16, group of four rows (0..15)

  // ---- output tile (I,J), then (J,I) with the roles of the two staged tiles swapped --------
  for (int o = 0; o < (I == J ? 1 : 2); ++o) {
    TileCtx ctx;
    ctx.smem = tiles;
    ctx.r0 = (o == 0 ? I : J) * kTile;
    ctx.c0 = (o == 0 ? J : I) * kTile;
    ctx.direct = (I == J) ? 0 : o;
    ctx.trans = (I == J) ? 0 : 1 - o;
    const int col_tile = o == 0 ? J : I;
    const int r = ctx.r0 + 4 * rg;
    uint32_t row_part[N][4];
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_row_fold(nd)) {
#pragma unroll
        for (int j = 0; j < 4; ++j) row_part[i][j] = identity_of<nd.fn, nd.dtype>();
      }
    });
#pragma unroll
    for (int k = 0; k < kTile / 16; ++k) {
      const int c = ctx.c0 + cx + 16 * k;
      if (r < n && c < n) {
        const IxP4 ix{r, c, &ctx};
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          constexpr CNode nd = CL::c.nodes[i];
          if constexpr (is_store_root(nd)) {
            const V4 v = eval<CL, i>(a, ix);
            uint32_t* out = reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr));
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (r + j < n) out[(size_t)(r + j) * n + c] = v.v[j];
          } else if constexpr (is_row_fold(nd)) {
            const V4 v = eval<CL, nd.in[0]>(a, ix);
#pragma unroll
            for (int j = 0; j < 4; ++j) row_part[i][j] = combine<nd.fn, nd.dtype>(row_part[i][j], v.v[j]);
          }
        });
      }
    }
    if constexpr (NRF > 0) {
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_row_fold(nd)) {
          constexpr int ord = count_if<CL>(is_row_fold, i);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t s = row_part[i][j];
#pragma unroll
            for (int w = 8; w > 0; w >>= 1) s = combine<nd.fn, nd.dtype>(s, __shfl_xor_sync(0xFFFFFFFFu, s, w));
            if (cx == 0 && r + j < n) partials[((size_t)ord * blocks + col_tile) * n + r + j] = s;
          }
        }
      });
    }
  }
  if constexpr (NRF > 0) {
    // One thread publishes the block's partials (the barrier makes them visible to it, its
    // fence orders them before the counters) and learns which blocks of rows are now complete.
    __syncthreads();
    if (threadIdx.x == 0) {
      __threadfence();
      finishing[0] = atomicAdd(counters + I, 1u) == (uint32_t)blocks - 1;
      finishing[1] = I != J && atomicAdd(counters + J, 1u) == (uint32_t)blocks - 1;
    }
    __syncthreads();
    for (int o = 0; o < 2; ++o) {
      const int row_block = o == 0 ? I : J;
      if (finishing[o]) {
        __threadfence();
        // the last contributor of this block of rows adds the column tiles up in order
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          constexpr CNode nd = CL::c.nodes[i];
          if constexpr (is_row_fold(nd)) {
            constexpr int ord = count_if<CL>(is_row_fold, i);
            const int row = row_block * kTile + (threadIdx.x >> 2), quarter = threadIdx.x & 3;
            uint32_t s = identity_of<nd.fn, nd.dtype>();
            if (row < n) {
              const volatile uint32_t* part = partials + (size_t)ord * blocks * n + row;
              for (int t = quarter; t < blocks; t += 4) s = combine<nd.fn, nd.dtype>(s, part[(size_t)t * n]);
            }
            s = combine<nd.fn, nd.dtype>(s, __shfl_xor_sync(0xFFFFFFFFu, s, 1));
            s = combine<nd.fn, nd.dtype>(s, __shfl_xor_sync(0xFFFFFFFFu, s, 2));
            if (quarter == 0 && row < n) reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[row] = s;
          }
        });
      }
    }
  }
}

}  // namespace dev
}  // namespace acc
