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
#include <cuda.h>

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

template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const IxP4& i, const NodeArg&, const NodeArg&) {
  static_assert(F == ACC_IDX_IDENTITY || F == ACC_IDX_TRANSPOSE, "only transposes are staged in tiles");
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else return IxQ4{i.r, i.c, i.t};
}
template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const IxQ4& i, const NodeArg&, const NodeArg&) {
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

// =========================================================================================
// k_tile_pair_tma: the same pairing of tiles for clusters whose roots are row folds, with the
// source tiles brought in by tensor copies (cp.async.bulk.tensor, no multicast) and the fold
// bookkeeping taken off the critical path.
//
// A persistent CTA of eight consumer warps and a copy warp walks pairs p = blockIdx.x,
// blockIdx.x + gridDim.x, ...  One lane of the copy warp issues the copies of a pair against
// the stage's `full` mbarrier as soon as the consumers have released that stage (`empty`), so
// up to kStages pairs are in flight.  A 64 x 64 tile arrives as one box, rows of 256 bytes, as it
// lies.  Parts of a box outside the array arrive as zeros and are never used.
//
// A consumer thread owns a 4 x 4 block of the output tile: four 128-bit reads give its block of
// the tile that lies like the output, four more its block of the tile read transposed (whose
// rows are the output's columns, so the transpose happens in registers).  The eight lanes that
// share a 128-bit shared-memory access sit on a diagonal of blocks (block column l, block row
// (l + d) mod 8): a row is 16 chunks of 16 bytes, so the bank group of a chunk is its column mod
// 8, and on the diagonal the eight block columns (direct read) and the eight block rows (which
// are the columns of the transposed read) are all different: no bank conflicts, no padding, no
// swizzle (the 128-byte swizzle with two boxes per tile measured 0.0604 against 0.0577 ms).  A
// consumer warp releases the stage as soon as its blocks are in registers.  Row sums of the
// blocks are combined through a small shared array (fixed order) and one partial per row and
// tile goes to scratch.
//
// The kernel is launched cooperatively (all blocks resident).  After its walk a block
// arrives at a grid-wide counter; once every block has arrived, each block adds up, in
// column-tile order, the partials of its own slice of rows.  Publishing per pair instead
// (fence + counter per block of rows, last arriver sums) was measured: the sum of 128 partials
// for 64 rows by whichever block arrived last took 0.36 ms of tail at 8192 x 8192.
//
// Every wait is bounded (wait_phase; kCopySpinLimit polls of the counter); a wait that runs out
// sets the time-out bit of the status word and the block's `abort` word, which ends the walk of
// every warp; the copy warp then still waits, with the same bound, for copies in flight before
// it leaves, and the block still arrives at the counter so that no other block waits for it.
constexpr int kTpTileWords = kTile * kTile;          // 4096 words = 16 KB per copy
constexpr int kTpSlotWords = 2 * kTpTileWords;       // tiles [I,J] and [J,I] of one external
constexpr int kTpMaxExternals = 3;
constexpr int kTpConsumers = 256;                    // eight warps of 4 x 4 blocks = one 64 x 64 tile
constexpr int kTpThreads = kTpConsumers + 32;                // + the copy warp
constexpr int kTpRedStride = 20;                     // words per row of the row-sum exchange (16 used)
constexpr uint32_t kCopySpinLimit = 1u << 20;
template <int E> constexpr int tp_stages() { return E <= 2 ? 3 : 2; }

struct TileMaps { CUtensorMap m[kTpMaxExternals]; };

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Polls an mbarrier phase; false if it did not complete within the limit.
__device__ __forceinline__ bool wait_phase(uint64_t* bar, uint32_t parity) {
  const uint32_t addr = smem_addr(bar);
  for (uint32_t spins = 0; spins < kCopySpinLimit; ++spins) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(addr), "r"(parity), "r"(2000u) : "memory");   // the thread may sleep up to 2 us per poll
    if (done) return true;
  }
  return false;
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
// Barrier 1 over the consumer threads only, returning the OR of their predicates.
__device__ __forceinline__ bool consumers_or(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, 1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"((uint32_t)pred), "n"(kTpConsumers) : "memory");
  return r != 0;
}

// The thread's blocks of every staged external, in registers.
struct BlkCtx {
  uint4 D[kTpMaxExternals][4];   // row j of the block of the tile that lies like the output
  uint4 T[kTpMaxExternals][4];   // row i of the block of the other tile = column i of the output block
};
// row r = r0 + 4*by + j of the output, columns c..c+3, as it lies / transposed
struct IxB4  { int r, c, j; const BlkCtx* b; };
struct IxBT4 { int r, c, j; const BlkCtx* b; };     // positions (c..c+3, r) of the source

__device__ __forceinline__ Ix lane(const IxB4& i, int k) { return Ix{i.r, i.c + k}; }
__device__ __forceinline__ Ix lane(const IxBT4& i, int k) { return Ix{i.c + k, i.r}; }

template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const IxB4& i, const NodeArg&, const NodeArg&) {
  static_assert(F == ACC_IDX_IDENTITY || F == ACC_IDX_TRANSPOSE, "only transposes are staged in tiles");
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else return IxBT4{i.r, i.c, i.j, i.b};
}
template <int F, int P0 = kRunTime, int P1 = kRunTime> __device__ __forceinline__ auto map_index(const IxBT4& i, const NodeArg&, const NodeArg&) {
  static_assert(F == ACC_IDX_IDENTITY || F == ACC_IDX_TRANSPOSE, "only transposes are staged in tiles");
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else return IxB4{i.r, i.c, i.j, i.b};
}

__device__ __forceinline__ uint32_t word_of(const uint4& v, int j) { return j == 0 ? v.x : j == 1 ? v.y : j == 2 ? v.z : v.w; }

template <class CL, int I, class A>
__device__ __forceinline__ V4 ld_ext(const A&, const IxB4& ix) {
  const uint4 v = ix.b->D[tile_slot<CL>(I)][ix.j];
  return V4{{v.x, v.y, v.z, v.w}};
}
template <class CL, int I, class A>
__device__ __forceinline__ V4 ld_ext(const A&, const IxBT4& ix) {
  const uint4* t = ix.b->T[tile_slot<CL>(I)];
  return V4{{word_of(t[0], ix.j), word_of(t[1], ix.j), word_of(t[2], ix.j), word_of(t[3], ix.j)}};
}

// Clusters this skeleton takes: tile-eligible, every root a row fold.
template <class CL> constexpr bool tile_tma_eligible() {
  if (!tile_eligible<CL>()) return false;
  for (int i = 0; i < CL::c.n; ++i)
    if (is_store_root(CL::c.nodes[i])) return false;
  return count_if<CL>(is_row_fold) >= 1 && count_if<CL>(is_row_fold) <= 2;
}

template <class CL>
__global__ void __launch_bounds__(kTpThreads) k_tile_pair_tma(const __grid_constant__ Args<CL::c.n> a,
                                                              const __grid_constant__ TileMaps maps) {
  constexpr int N = CL::c.n;
  constexpr int NRF = count_if<CL>(is_row_fold);
  constexpr int E = staged_externals<CL>();
  constexpr int S = tp_stages<E>();
  constexpr int kStageWords = E * kTpSlotWords;
  extern __shared__ uint32_t tp_raw[];
  __shared__ __align__(8) uint64_t full[S], empty[S];
  __shared__ uint32_t abort_walk;        // set by whoever ran out of patience
  __shared__ __align__(16) uint32_t red[2][NRF][kTile][kTpRedStride];
  // copies land on 128-byte boundaries
  uint32_t* const tiles = tp_raw + ((128u - (smem_addr(tp_raw) & 127u)) & 127u) / 4;
  const int n = a.R;                                        // square domain: n x n
  const int blocks = (n + kTile - 1) / kTile;
  const uint32_t n_pairs = (uint32_t)blocks * (uint32_t)(blocks + 1) / 2;
  uint32_t* const arrivals = a.scratch;                     // blocks that have finished their walk
  uint32_t* partials = a.scratch + tile_partials_off(blocks);
  const int lane_id = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], kTpConsumers / 32);
    }
    abort_walk = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile uint32_t* const v_abort = &abort_walk;

  if (threadIdx.x >= kTpConsumers) {
    // ---------------- copy warp: one lane keeps up to kStages pairs in flight -------------------
    if (lane_id != 0) return;
    auto issue = [&](uint32_t pair, int stage) {
      int I, J;
      pair_of(pair, blocks, I, J);
      const int n_tiles = I == J ? 1 : 2;
      const uint32_t b = smem_addr(&full[stage]);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"((uint32_t)(E * n_tiles * kTpTileWords * 4)) : "memory");
#pragma unroll
      for (int slot = 0; slot < E; ++slot) {
        for (int t = 0; t < n_tiles; ++t) {
          const int y = (t == 0 ? I : J) * kTile, x = (t == 0 ? J : I) * kTile;   // x: a multiple of 64 words
          const uint32_t dst = smem_addr(tiles + stage * kStageWords + slot * kTpSlotWords + t * kTpTileWords);
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
              ::"r"(dst), "l"(&maps.m[slot]), "r"(x), "r"(y), "r"(b) : "memory");
        }
      }
    };
    uint32_t trip = 0;                                      // trips whose copies have been started
    bool ok = true;
    for (uint32_t pair = blockIdx.x; pair < n_pairs; pair += gridDim.x, ++trip) {
      // its stage held trip - S: every consumer warp must have let go of that
      if (trip >= (uint32_t)S) ok = wait_phase(&empty[trip % S], (trip / S - 1) & 1u) && !*v_abort;
      if (!ok) break;
      issue(pair, (int)(trip % S));
    }
    if (!ok) {
      if (!*v_abort) { *v_abort = 1; atomicOr(a.status, kStatusTimeout); }
      // copies still in flight must not land in the shared memory of a block that has gone
      for (uint32_t q = 1; q <= (uint32_t)S && q <= trip; ++q) wait_phase(&full[(trip - q) % S], ((trip - q) / S) & 1u);
    }
    return;
  }

  // ---------------- consumer warps ------------------------------------------------------------
  const int l = threadIdx.x & 7, dg = (threadIdx.x >> 3) & 7, quad = threadIdx.x >> 6;
  const int bx = (quad & 1) * 8 + l, by = (quad >> 1) * 8 + ((l + dg) & 7);   // the thread's 4 x 4 block
  int dofs[4], tofs[4];                                     // word offsets of the block's rows in a tile
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int dr = 4 * by + i, tr = 4 * bx + i;
    dofs[i] = dr * kTile + 4 * bx;
    tofs[i] = tr * kTile + 4 * by;
  }
  const int red_row = threadIdx.x >> 2, red_q = threadIdx.x & 3;
  int tp = 0;                                               // which half of `red` this tile uses
  uint32_t it = 0;
  for (uint32_t pair = blockIdx.x; pair < n_pairs; pair += gridDim.x, ++it) {
    const int stage = (int)(it % S);
    const bool arrived = wait_phase(&full[stage], (it / S) & 1u) && !*v_abort;
    if (!arrived && !*v_abort) { *v_abort = 1; atomicOr(a.status, kStatusTimeout); }
    int I, J;
    pair_of(pair, blocks, I, J);
    const int n_tiles = I == J ? 1 : 2;
    bool stop = false;
    // ---- output tile (I,J), then (J,I) with the roles of the two staged tiles swapped --------
    for (int o = 0; o < n_tiles; ++o) {
      const int r0 = (o == 0 ? I : J) * kTile, c0 = (o == 0 ? J : I) * kTile;
      const int direct = (I == J) ? 0 : o, trans = (I == J) ? 0 : 1 - o;
      const int col_tile = o == 0 ? J : I;
      BlkCtx ctx;
#pragma unroll
      for (int slot = 0; slot < E; ++slot) {
        const uint32_t* sb = tiles + stage * kStageWords + slot * kTpSlotWords;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          ctx.D[slot][i] = *reinterpret_cast<const uint4*>(sb + direct * kTpTileWords + dofs[i]);
          ctx.T[slot][i] = *reinterpret_cast<const uint4*>(sb + trans * kTpTileWords + tofs[i]);
        }
      }
      if (o == n_tiles - 1) {                               // the stage is in registers: let it be refilled
        __syncwarp();
        if (lane_id == 0) mbar_arrive(&empty[stage]);
      }
      const int r = r0 + 4 * by, c = c0 + 4 * bx;           // n is a multiple of 4: a block is inside or outside
      const bool inside = r < n && c < n;
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_row_fold(nd)) {
          constexpr int ord = count_if<CL>(is_row_fold, i);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t s = identity_of<nd.fn, nd.dtype>();
            if (inside) {
              const V4 v = eval<CL, nd.in[0]>(a, IxB4{r + j, c, j, &ctx});
              s = combine<nd.fn, nd.dtype>(combine<nd.fn, nd.dtype>(v.v[0], v.v[1]), combine<nd.fn, nd.dtype>(v.v[2], v.v[3]));
            }
            red[tp][ord][4 * by + j][bx] = s;
          }
        }
      });
      stop = consumers_or(!arrived);
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_row_fold(nd)) {
          constexpr int ord = count_if<CL>(is_row_fold, i);
          const uint4 v = *reinterpret_cast<const uint4*>(&red[tp][ord][red_row][4 * red_q]);
          uint32_t s = combine<nd.fn, nd.dtype>(combine<nd.fn, nd.dtype>(v.x, v.y), combine<nd.fn, nd.dtype>(v.z, v.w));
          s = combine<nd.fn, nd.dtype>(s, __shfl_xor_sync(0xFFFFFFFFu, s, 1));
          s = combine<nd.fn, nd.dtype>(s, __shfl_xor_sync(0xFFFFFFFFu, s, 2));
          if (red_q == 0 && r0 + red_row < n) partials[((size_t)ord * blocks + col_tile) * n + r0 + red_row] = s;
        }
      });
      tp ^= 1;            // the next tile writes the other half: this one is still being read
      if (stop) break;
    }
    if (stop) break;      // agreed on by all consumers at the barrier above
  }

  // ---- every block has walked: add up this block's slice of rows --------------------------------
  // (barrier 1 makes the consumers' partials visible to thread 0, whose fence orders them before
  // its arrival; the fence after the wait orders the other blocks' partials before the reads)
  consumers_or(false);
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(arrivals, 1u);
    uint32_t spins = 0;
    while (*reinterpret_cast<volatile uint32_t*>(arrivals) < gridDim.x) {
      if (++spins > kCopySpinLimit) { atomicOr(a.status, kStatusTimeout); break; }
      __nanosleep(200);
    }
    __threadfence();
  }
  consumers_or(false);
  const int per_block = (n + (int)gridDim.x - 1) / (int)gridDim.x;
  const int slice0 = (int)blockIdx.x * per_block, slice1 = min(n, slice0 + per_block);
  for (int base = slice0; base < slice1; base += kTpConsumers / 4) {
    const int row = base + red_row;
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_row_fold(nd)) {
        constexpr int ord = count_if<CL>(is_row_fold, i);
        const uint32_t* part = partials + (size_t)ord * blocks * n + min(row, n - 1);
        uint32_t s = identity_of<nd.fn, nd.dtype>();
        for (int t = red_q; t < blocks; t += 128) {          // this thread's column tiles: t, t + 4, ...
          uint32_t v[32];                                     // all in flight together (128 tiles = 8192 columns per trip)
#pragma unroll
          for (int u = 0; u < 32; ++u) v[u] = __ldcg(part + (size_t)min(t + 4 * u, blocks - 1) * n);
#pragma unroll
          for (int u = 0; u < 32; ++u)
            if (t + 4 * u < blocks) s = combine<nd.fn, nd.dtype>(s, v[u]);
        }
        s = combine<nd.fn, nd.dtype>(s, __shfl_xor_sync(0xFFFFFFFFu, s, 1));
        s = combine<nd.fn, nd.dtype>(s, __shfl_xor_sync(0xFFFFFFFFu, s, 2));
        if (red_q == 0 && row < slice1) reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[row] = s;
      }
    });
  }
}

}  // namespace dev
}  // namespace acc
