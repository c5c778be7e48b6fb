// k_stencil: the skeleton for rank-2 clusters whose only index maps are clamped shifts by at
// most one row and one column (a stencil by horizontal fusion: several backpermutes of one
// array feeding zipWiths).
//
// A persistent CTA walks output tiles of kStRows x kStCols.  For each tile the tile plus its
// halo (one row above and below, four columns left and right so that the copy starts on a
// 16-byte boundary) of every external is brought into shared memory by ONE tensor copy
// (cp.async.bulk.tensor, no multicast), issued by one thread and tracked by an mbarrier; the
// copy of the next tile runs while the current one is computed (two stages).  Parts of the
// box outside the array arrive as zeros and are never read: shifted positions are clamped to
// the array first, and a clamped position always lies inside the tile or its halo.  All five
// reads of a Jacobi iteration are then shared-memory reads.
//
// Every wait on an mbarrier is bounded: after kCopySpinLimit polls the thread records
// ACC_ERR_DEVICE_TIMEOUT in the status word and goes on, so a lost copy cannot hang the GPU.
#pragma once
#include <cuda.h>

#include "skeletons.cuh"
#include "tile.cuh"

namespace acc {
namespace dev {

constexpr int kStRows = 64, kStCols = 128;            // output tile
constexpr int kStBoxRows = kStRows + 2;               // + halo rows
constexpr int kStBoxCols = kStCols + 8;               // + halo columns (4 each side: 16-byte alignment)
constexpr int kStBoxWords = kStBoxRows * kStBoxCols;  // 4624 words = 18496 bytes per copy
constexpr int kStBoxStride = (kStBoxWords + 31) / 32 * 32;   // boxes start on 128-byte boundaries
constexpr int kStStages = 2;
constexpr int kStMaxExternals = 2;

struct StencilMaps { CUtensorMap m[kStMaxExternals]; };

// four consecutive columns inside the staged tile / the same after one clamped shift.
// `at` points to element (r, c) in the box of external slot 0 of the current stage; the boxes
// of the other slots lie kStBoxStride words further each.
struct IxH4  { int r, c; const uint32_t* at; };
struct IxHS4 { int r, c, dc; const uint32_t* at; };    // row r (already clamped), columns clamp(c+dc+j)

__device__ __forceinline__ Ix lane(const IxH4& i, int j) { return Ix{i.r, i.c + j}; }

template <int F> __device__ __forceinline__ auto map_index(const IxH4& i, const NodeArg& self, const NodeArg& src) {
  static_assert(F == ACC_IDX_IDENTITY || F == ACC_IDX_SHIFT_CLAMP, "only clamped shifts are staged with a halo");
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else {
    const int rr = min(max(i.r + self.ip0, 0), src.R - 1);
    return IxHS4{rr, i.c, self.ip1, i.at + (rr - i.r) * kStBoxCols};
  }
}
template <int F> __device__ __forceinline__ auto map_index(const IxHS4& i, const NodeArg&, const NodeArg&) {
  static_assert(F == ACC_IDX_IDENTITY, "a halo of one serves one shift, not a shift of a shift");
  return i;
}

// A cluster can use this skeleton if its members are element-wise, its only index maps are
// shifts, no external is reached through more than one shift, every array it reads is a
// rank-2 external, and its roots are rank-2 stores.
template <class CL> constexpr int shift_depth(int i) {
  const CNode& n = CL::c.nodes[i];
  if (!n.member) return 0;
  int d = 0;
  for (int s = 0; s < n.narr; ++s) {
    const int k = shift_depth<CL>(n.in[s]);
    d = k > d ? k : d;
  }
  return d + ((n.kind == ACC_BACKPERMUTE && n.idxfn == ACC_IDX_SHIFT_CLAMP) ? 1 : 0);
}
template <class CL> constexpr bool stencil_eligible() {
  bool has_shift = false;
  int externals = 0;
  for (int i = 0; i < CL::c.n; ++i) {
    const CNode& n = CL::c.nodes[i];
    if (!n.member) {
      bool as_array = false;
      for (int j = 0; j < CL::c.n; ++j)
        for (int s = 0; s < CL::c.nodes[j].narr; ++s)
          if (CL::c.nodes[j].member && CL::c.nodes[j].in[s] == i) as_array = true;
      if (as_array) {
        if (n.rank != 2) return false;
        ++externals;
      }
      continue;
    }
    if (n.rank != 2) return false;
    if (n.kind == ACC_BACKPERMUTE) {
      if (n.idxfn == ACC_IDX_SHIFT_CLAMP) has_shift = true;
      else if (n.idxfn != ACC_IDX_IDENTITY) return false;
    } else if (n.kind != ACC_MAP && n.kind != ACC_ZIPWITH) {
      return false;
    }
    if (shift_depth<CL>(i) > 1) return false;
  }
  return has_shift && externals >= 1 && externals <= kStMaxExternals;
}

// reads from the staged boxes (a tile's box starts at row r0-1, column c0-4, so the element
// left of a chunk and the one right of it are always inside the box)
__device__ __forceinline__ V4 ld_box(int slot, const IxH4& i) {
  const uint4 v = *reinterpret_cast<const uint4*>(i.at + slot * kStBoxStride);
  return V4{{v.x, v.y, v.z, v.w}};
}
__device__ __forceinline__ V4 ld_box(int slot, const IxHS4& i, int C) {
  const uint32_t* p = i.at + slot * kStBoxStride;
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  if (i.dc == 1) return V4{{v.y, v.z, v.w, p[min(4, C - 1 - i.c)]}};      // clamped at the last column
  if (i.dc == -1) return V4{{p[max(-1, -i.c)], v.x, v.y, v.z}};           // clamped at the first column
  return V4{{v.x, v.y, v.z, v.w}};                                         // dc == 0 (larger shifts never get here)
}

template <class CL, int I, class A>
__device__ __forceinline__ V4 ld_ext(const A&, const IxH4& ix) { return ld_box(tile_slot<CL>(I), ix); }
template <class CL, int I, class A>
__device__ __forceinline__ V4 ld_ext(const A& a, const IxHS4& ix) { return ld_box(tile_slot<CL>(I), ix, a.n[I].C); }

template <class CL>
__global__ void __launch_bounds__(kBlock)
k_stencil(const __grid_constant__ Args<CL::c.n> a, const __grid_constant__ StencilMaps maps) {
  constexpr int N = CL::c.n;
  constexpr int E = staged_externals<CL>();
  extern __shared__ __align__(128) uint32_t boxes[];          // [stage][external slot][kStBoxStride]
  __shared__ __align__(8) uint64_t bar[kStStages];
  const int R = a.R, C = a.C;
  const uint32_t tiles_x = (uint32_t)(C + kStCols - 1) / kStCols;
  const uint32_t n_tiles = tiles_x * ((uint32_t)(R + kStRows - 1) / kStRows);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStStages; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bar[s])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // one thread starts the copies of a tile into a stage; the stage's barrier counts their bytes
  auto issue = [&](uint32_t tile, int stage) {
    const uint32_t ty = tile / tiles_x, tx = tile - ty * tiles_x;
    const int x = (int)(tx * kStCols) - 4, y = (int)(ty * kStRows) - 1;   // x stays a multiple of 4: 16-byte aligned
    const uint32_t b = smem_addr(&bar[stage]);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"((uint32_t)(E * kStBoxWords * 4)) : "memory");
#pragma unroll
    for (int slot = 0; slot < E; ++slot) {
      const uint32_t dst = smem_addr(boxes + (stage * E + slot) * kStBoxStride);
      asm volatile(
          "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
          ::"r"(dst), "l"(&maps.m[slot]), "r"(x), "r"(y), "r"(b) : "memory");
    }
  };

  uint32_t parity[kStStages] = {0u, 0u};
  int stage = 0;
  if (threadIdx.x == 0 && blockIdx.x < n_tiles) issue(blockIdx.x, 0);
  for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    // the other stage was last read before the barrier that ended the previous trip
    if (threadIdx.x == 0 && tile + gridDim.x < n_tiles) issue(tile + gridDim.x, stage ^ 1);
    const bool arrived = wait_phase(&bar[stage], parity[stage]);
    if (!arrived) atomicOr(a.status, kStatusTimeout);

    const uint32_t ty = tile / tiles_x, tx = tile - ty * tiles_x;
    const uint32_t* box = boxes + stage * E * kStBoxStride;
    const int r0 = (int)(ty * kStRows), c0 = (int)(tx * kStCols);
#pragma unroll
    for (int p = 0; p < kStRows / (kBlock / 32); ++p) {
      const int r = r0 + warp + (kBlock / 32) * p, c = c0 + 4 * lane;
      if (r < R && c < C) {
        const IxH4 ix{r, c, box + (r - r0 + 1) * kStBoxCols + (c - c0 + 4)};
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          if constexpr (is_store_root(CL::c.nodes[i]))
            st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), C, Ix4{r, c}, eval<CL, i>(a, ix));
        });
      }
    }
    // a stage that never arrived ends the walk: the block waits once more, again with a limit, for
    // the copies it still has in flight (they must not land in the shared memory of a block that
    // has gone) and returns; the host reports the status bit
    if (__syncthreads_or(!arrived)) {
      if (threadIdx.x == 0) {
        if (!arrived) wait_phase(&bar[stage], parity[stage]);
        if (tile + gridDim.x < n_tiles) wait_phase(&bar[stage ^ 1], parity[stage ^ 1]);
      }
      break;
    }
    parity[stage] ^= 1u;
    stage ^= 1;
  }
}

}  // namespace dev
}  // namespace acc
