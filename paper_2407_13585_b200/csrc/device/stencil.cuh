// k_stencil: the skeleton for rank-2 clusters whose only index maps are clamped shifts by at
// most one row and one column (a stencil by horizontal fusion: several backpermutes of one
// array feeding zipWiths), stacked up to kStMaxDepth deep (several iterations of such a stencil
// in one cluster, which needs the recomputing kind of clustering: the intermediate iterate is
// read in five orders).
//
// A persistent CTA walks output tiles of kStRows x kStCols.  With D = the largest number of
// shifts between an external and a root, the tile plus a halo of D rows above and below and
// four columns left and right (so that the copy starts on a 16-byte boundary; D <= 4) of every
// external is brought into shared memory by ONE tensor copy (cp.async.bulk.tensor, no
// multicast), issued by one thread and tracked by an mbarrier; the copy of the next tile runs
// while the current one is computed (two stages).  Parts of the box outside the array arrive
// as zeros and are never read: shifted positions are clamped to the array first, and a clamped
// position always lies inside the tile or its halo.
//
// A member that is itself the source of a shift (the previous iterate of a stacked stencil) is
// computed ONCE per tile, over the tile plus the halo its readers still need, into a box of the
// same geometry in shared memory, depth by depth; its readers then read that box.  So k
// iterations cost one read and one write of the array and (1 + 2(D-k)/kStRows) of the
// arithmetic per level instead of the 5^k-fold recomputation that pulling each read through
// would do.  The values are those of the plain evaluation, bit for bit: every element is
// computed by the same expression, at positions clamped in the same way.
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
constexpr int kStBoxCols = kStCols + 8;               // + halo columns (4 each side: 16-byte alignment)
constexpr int kStChunks = kStBoxCols / 4;             // 128-bit chunks per box row
constexpr int kStStages = 2;
constexpr int kStMaxExternals = 2;
constexpr int kStMaxDepth = 4;                        // the column halo is four wide
constexpr int kStMaxStagedMembers = 3;

constexpr int st_box_rows(int depth) { return kStRows + 2 * depth; }
constexpr int st_box_words(int depth) { return st_box_rows(depth) * kStBoxCols; }
constexpr int st_box_stride(int depth) { return (st_box_words(depth) + 31) / 32 * 32; }   // boxes start on 128-byte boundaries

struct StencilMaps { CUtensorMap m[kStMaxExternals]; };

// Where the boxes of the current tile are: externals of this stage, members kept on chip.
struct StCtx { const uint32_t* ext; const uint32_t* mem; };

// four consecutive columns inside a box / the same after one clamped shift.  `off` is the word
// offset of element (r, c) in a box; the box of slot k lies k box strides further.  The lanes of
// a warp hold consecutive chunks of one box row, so the word right (left) of a chunk is the first
// (last) word of the next (previous) lane's chunk and comes by shuffle; `solo` says where that
// does not hold (bit 0: no right neighbour in lane + 1, bit 1: no left neighbour in lane - 1) and
// the word is read from the box instead.  Every lane of the warp must take part in every read,
// unless bit 2 is set in all of them: then nobody shuffles and everybody reads the box.
struct IxH4  { int r, c, off, solo; StCtx t; };
// row r (already clamped), columns clamp(c+dc+j); DC is the column offset when the cluster was
// built for it, else kRunTime and `dc` holds it
template <int DC> struct IxHS4 { int r, c, dc, off, solo; StCtx t; };

__device__ __forceinline__ Ix lane(const IxH4& i, int j) { return Ix{i.r, i.c + j}; }

template <int F, int P0 = kRunTime, int P1 = kRunTime>
__device__ __forceinline__ auto map_index(const IxH4& i, const NodeArg& self, const NodeArg& src) {
  static_assert(F == ACC_IDX_IDENTITY || F == ACC_IDX_SHIFT_CLAMP, "only clamped shifts are staged with a halo");
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else if constexpr (P0 == 0) return IxHS4<P1>{i.r, i.c, self.ip1, i.off, i.solo, i.t};
  else {
    const int rr = min(max(i.r + (P0 != kRunTime ? P0 : self.ip0), 0), src.R - 1);
    return IxHS4<P1>{rr, i.c, self.ip1, i.off + (rr - i.r) * kStBoxCols, i.solo, i.t};
  }
}
template <int F, int P0 = kRunTime, int P1 = kRunTime, int DC>
__device__ __forceinline__ auto map_index(const IxHS4<DC>& i, const NodeArg&, const NodeArg&) {
  static_assert(F == ACC_IDX_IDENTITY, "the source of a shift is read from a box, never pulled through");
  return i;
}

// ---- compile-time layout of a stencil cluster -----------------------------------------------
// shifts between the externals and node i (longest path)
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
template <class CL> constexpr int max_shift_depth() {
  int d = 0;
  for (int i = 0; i < CL::c.n; ++i) {
    const int k = shift_depth<CL>(i);
    d = k > d ? k : d;
  }
  return d;
}
// a member that some shift reads: kept on chip
template <class CL> constexpr bool is_staged_member(int i) {
  if (!CL::c.nodes[i].member) return false;
  for (int j = 0; j < CL::c.n; ++j) {
    const CNode& n = CL::c.nodes[j];
    if (n.member && n.kind == ACC_BACKPERMUTE && n.idxfn == ACC_IDX_SHIFT_CLAMP && n.in[0] == i) return true;
  }
  return false;
}
template <class CL> constexpr int member_slot(int i) {
  int k = 0;
  for (int j = 0; j < i; ++j) k += is_staged_member<CL>(j) ? 1 : 0;
  return k;
}
template <class CL> constexpr int staged_members() { return member_slot<CL>(CL::c.n); }

// A cluster can use this skeleton if its members are element-wise, its only index maps are
// shifts stacked at most kStMaxDepth deep, every array it reads is a rank-2 external, and its
// roots are rank-2 stores.
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
  }
  return has_shift && externals >= 1 && externals <= kStMaxExternals && max_shift_depth<CL>() <= kStMaxDepth &&
         staged_members<CL>() <= kStMaxStagedMembers;
}

// ---- reads from the boxes ----------------------------------------------------------------------
// (a tile's box starts D rows above and four columns left of the tile, so the element left of a
// chunk and the one right of it are always words of the box)
__device__ __forceinline__ V4 ld_box(const uint32_t* p) {
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  return V4{{v.x, v.y, v.z, v.w}};
}
template <int DC>
__device__ __forceinline__ V4 ld_box(const uint32_t* p, const IxHS4<DC>& i, int C) {
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  const int dc = DC != kRunTime ? DC : i.dc;                               // the same in every lane
  if (dc == 1) {
    uint32_t right = 0;                                                    // (a single-word read per lane is a 4-way bank conflict)
    if (!(i.solo & 4)) right = __shfl_down_sync(0xFFFFFFFFu, v.x, 1);
    if (i.solo & 1) right = p[4];
    if (C - 1 - i.c < 4) right = v.w;                                      // clamped at the last column
    return V4{{v.y, v.z, v.w, right}};
  }
  if (dc == -1) {
    uint32_t left = 0;
    if (!(i.solo & 4)) left = __shfl_up_sync(0xFFFFFFFFu, v.w, 1);
    if (i.solo & 2) left = p[-1];
    if (i.c <= 0) left = v.x;                                              // clamped at the first column
    return V4{{left, v.x, v.y, v.z}};
  }
  return V4{{v.x, v.y, v.z, v.w}};                                         // dc == 0 (larger shifts never get here)
}

template <class CL, int I, class A>
__device__ __forceinline__ V4 ld_ext(const A&, const IxH4& ix) {
  return ld_box(ix.t.ext + tile_slot<CL>(I) * st_box_stride(max_shift_depth<CL>()) + ix.off);
}
template <class CL, int I, class A, int DC>
__device__ __forceinline__ V4 ld_ext(const A& a, const IxHS4<DC>& ix) {
  return ld_box(ix.t.ext + tile_slot<CL>(I) * st_box_stride(max_shift_depth<CL>()) + ix.off, ix, a.n[I].C);
}

// members kept on chip are read from their box at a shifted index, computed anywhere else
template <class CL, int I, int DC> struct reads_staged<CL, I, IxHS4<DC>> { static constexpr bool value = is_staged_member<CL>(I); };
template <class CL, int I, class A, int DC>
__device__ __forceinline__ V4 ld_staged(const A& a, const IxHS4<DC>& ix) {
  return ld_box(ix.t.mem + member_slot<CL>(I) * st_box_stride(max_shift_depth<CL>()) + ix.off, ix, a.n[I].C);
}

template <class CL>
__global__ void __launch_bounds__(kBlock)
k_stencil(const __grid_constant__ Args<CL::c.n> a, const __grid_constant__ StencilMaps maps) {
  constexpr int N = CL::c.n;
  constexpr int E = staged_externals<CL>();
  constexpr int D = max_shift_depth<CL>();
  constexpr int BR = st_box_rows(D), BS = st_box_stride(D);
  extern __shared__ __align__(128) uint32_t boxes[];          // [stage][external slot][BS], then [member slot][BS]
  __shared__ __align__(8) uint64_t bar[kStStages];
  uint32_t* const members = boxes + kStStages * E * BS;
  const int R = a.R, C = a.C;
  const uint32_t tiles_x = (uint32_t)(C + kStCols - 1) / kStCols;
  const uint32_t n_tiles = tiles_x * ((uint32_t)(R + kStRows - 1) / kStRows);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStStages; ++s) mbar_init(&bar[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // one thread starts the copies of a tile into a stage; the stage's barrier counts their bytes
  auto issue = [&](uint32_t tile, int stage) {
    const uint32_t ty = tile / tiles_x, tx = tile - ty * tiles_x;
    const int x = (int)(tx * kStCols) - 4, y = (int)(ty * kStRows) - D;   // x stays a multiple of 4: 16-byte aligned
    const uint32_t b = smem_addr(&bar[stage]);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"((uint32_t)(E * st_box_words(D) * 4)) : "memory");
#pragma unroll
    for (int slot = 0; slot < E; ++slot) {
      const uint32_t dst = smem_addr(boxes + (stage * E + slot) * BS);
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
    const int r0 = (int)(ty * kStRows), c0 = (int)(tx * kStCols);
    StCtx ctx;
    ctx.ext = boxes + stage * E * BS;
    ctx.mem = members;

    // members kept on chip, shallowest first: a member k shifts away from the externals is needed
    // (and computable) on the box rows k .. BR-1-k; whole box rows are computed, of which the
    // readers use the columns k away from the box edges at most
    static_for<1, D>([&](auto kc) {
      constexpr int k = decltype(kc)::value;
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        if constexpr (is_staged_member<CL>(i) && shift_depth<CL>(i) == k) {
          uint32_t* out = members + member_slot<CL>(i) * BS;
          constexpr int kTotal = (BR - 2 * k) * kStChunks;
          // whole warps walk the chunks (the reads shuffle between lanes); a lane past the end repeats
          // the last chunk, and chunks outside the array are computed from whatever the box holds:
          // neither is stored
          for (int q0 = (int)threadIdx.x - lane; q0 < kTotal; q0 += kBlock) {
            const int q = min(q0 + lane, kTotal - 1);
            const int ch = q % kStChunks;
            const int br = k + q / kStChunks, bc = 4 * ch;
            const int r = r0 - D + br, c = c0 - 4 + bc;
            const int off = br * kStBoxCols + bc;
            const int solo = ((lane == 31 || ch == kStChunks - 1) ? 1 : 0) | ((lane == 0 || ch == 0) ? 2 : 0);
            const V4 v = eval_here<CL, i>(a, IxH4{r, c, off, solo, ctx});
            if (q0 + lane < kTotal && r >= 0 && r < R && c >= 0 && c < C)
              *reinterpret_cast<uint4*>(out + off) = make_uint4(v.v[0], v.v[1], v.v[2], v.v[3]);
          }
          __syncthreads();
        }
      });
    });

#pragma unroll
    for (int p = 0; p < kStRows / (kBlock / 32); ++p) {
      // a warp per tile row, a lane per chunk
      const int r = r0 + warp + (kBlock / 32) * p, c = c0 + 4 * lane;
      if constexpr (D == 1) {
        // A single iteration reads its neighbour words from the box, row by row under the bounds
        // check.  Measured back to back on 8192 x 8192: 91 us per launch; with all rows computed
        // first and stored afterwards (which is what the compiler makes of the form below) 104 us,
        // with or without the shuffles, although that form is the faster one from a cold cache.
        if (r < R && c < C) {
          const IxH4 ix{r, c, (r - r0 + D) * kStBoxCols + (c - c0 + 4), 7, ctx};
          static_for<0, N>([&](auto ic) {
            constexpr int i = decltype(ic)::value;
            if constexpr (is_store_root(CL::c.nodes[i]))
              st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), C, Ix4{r, c}, eval<CL, i>(a, ix));
          });
        }
      } else {
        // computed by all lanes (the reads shuffle), stored where the chunk lies inside the array
        const IxH4 ix{r, c, (r - r0 + D) * kStBoxCols + (c - c0 + 4), (lane == 31 ? 1 : 0) | (lane == 0 ? 2 : 0), ctx};
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          if constexpr (is_store_root(CL::c.nodes[i])) {
            const V4 v = eval<CL, i>(a, ix);
            if (r < R && c < C) st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), C, Ix4{r, c}, v);
          }
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
