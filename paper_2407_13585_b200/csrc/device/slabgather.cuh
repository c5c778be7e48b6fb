// A scan whose operand gathers from an array that does not fit the L2 cache, run as slab passes (and, further down,
// the same for element-wise roots without a scan).
//
// A random 4-byte read of an array much larger than L2 costs a whole DRAM access (about 89 bytes of
// traffic on B200), and a cluster such as  out = scanl(+) (f (gather idx (g x)))  runs at the rate of
// those accesses.  The same reads served from L2 run four times faster, so the gather is cut into
// passes, each over a quarter (a slab) of the source, small enough to stay in L2 while it is being read:
//
//   k_slab_partition  walks the gather's index operand once.  Per warp tile of 512 elements it writes the
//                     index values grouped by slab (a stable counting sort in shared memory) into the
//                     scan's own output array, which serves as the staging area, the slab of every
//                     element (2 bits, one word per lane) into `codes`, and the group sizes into `counts`.
//   k_slab_gather     once per slab k: replaces the indices of group k, where they lie, by the gathered
//                     values (the gather's source, with the members fused into it, evaluated at the index).
//                     It streams a quarter of the staging area per pass and reads one slab of the source.
//   k_scan_merge      the look-back scan of skeletons.cuh, which first puts a warp tile's gathered values back
//                     into element order (the counting sort undone with the codes and the counts) and reads
//                     the gather member as those values; everything after the gather is evaluated as usual.
//
// Gather semantics (Section 2: ys[j] = as[is[j]]) and results are unchanged, bit for bit.  A last warp tile
// of fewer than 512 elements is left to the scan, which gathers for it directly.
#pragma once
#include "skeletons.cuh"

namespace acc {
namespace dev {

constexpr int kSlabs = 4;
constexpr int64_t kSlabMinSourceBytes = 96ll << 20;     // below this the source mostly stays in L2 anyway
constexpr int64_t kSlabMaxSourceBytes = 320ll << 20;    // beyond this a quarter of it no longer fits
constexpr int64_t kSlabMinElements = 1ll << 22;
constexpr uint32_t kSlabLocalSpan = 8192;               // a warp tile whose 512 indices span fewer source elements than this is local

constexpr bool depends_on(const CCluster& c, int i, int g) {
  if (i == g) return true;
  const CNode& n = c.nodes[i];
  if (!n.member) return false;
  for (int k = 0; k < n.nin; ++k)
    if (depends_on(c, n.in[k], g)) return true;
  return false;
}
// Whether every path from i down to g runs through array operands of maps and zipWiths only (so that the
// element index is the same all the way, and g's value at that index is all that is needed of it).
constexpr bool index_preserving_to(const CCluster& c, int i, int g) {
  if (i == g) return true;
  const CNode& n = c.nodes[i];
  if (!depends_on(c, i, g)) return true;
  if (n.kind != ACC_MAP && n.kind != ACC_ZIPWITH) return false;
  for (int k = 0; k < n.nin; ++k) {
    if (!depends_on(c, n.in[k], g)) continue;
    if (k >= n.narr || !index_preserving_to(c, n.in[k], g)) return false;
  }
  return true;
}

// depends_on with node `stop` taken as a leaf
constexpr bool depends_on_avoiding(const CCluster& c, int i, int g, int stop) {
  if (i == g) return true;
  if (i == stop) return false;
  const CNode& n = c.nodes[i];
  if (!n.member) return false;
  for (int k = 0; k < n.nin; ++k)
    if (depends_on_avoiding(c, n.in[k], g, stop)) return true;
  return false;
}

// One left-to-right scan of a rank-1 array as the only accumulating root, one gather (fused away) below its
// operand on index-preserving paths, and no element-wise root that would need the gather outside the scan's pass.
template <class CL> constexpr bool slab_gather_eligible() {
  const int S = first_scan<CL>();
  const int G = the_gather<CL>();
  if (S < 0 || G < 0) return false;
  const CCluster& c = CL::c;
  if (c.nodes[S].kind != ACC_SCANL || c.nodes[S].rank != 1 || !c.nodes[S].manifest || c.nodes[G].manifest || c.nodes[G].rank != 1) return false;
  for (int i = 0; i < c.n; ++i) {
    const CNode& n = c.nodes[i];
    if (i != S && (is_scan_root(n) || is_fold_root(n) || is_permute_root(n) || is_segfold_root(n))) return false;
    if (is_store_root(n) && depends_on_avoiding(c, i, G, S)) return false;     // it would gather on its own, outside the passes
  }
  if (depends_on(c, G, S)) return false;
  return depends_on(c, c.nodes[S].in[0], G) && index_preserving_to(c, c.nodes[S].in[0], G);
}

// The same passes for a cluster without a scan: element-wise roots over a rank-1 domain, one gather, nothing that
// accumulates.  The array of the first root that the gather's values reach on index-preserving paths is the staging
// area, and k_stream_merge takes the place of the merging scan.  -1: no such root.
template <class CL> constexpr int stream_staging_root() {
  const int G = the_gather<CL>();
  if (G < 0) return -1;
  const CCluster& c = CL::c;
  for (int i = 0; i < c.n; ++i)
    if (is_store_root(c.nodes[i]) && c.nodes[i].rank == 1 && depends_on(c, i, G) && index_preserving_to(c, i, G)) return i;
  return -1;
}
template <class CL> constexpr bool slab_stream_eligible() {
  const int G = the_gather<CL>();
  if (G < 0 || first_scan<CL>() >= 0 || stream_staging_root<CL>() < 0) return false;
  const CCluster& c = CL::c;
  if (c.nodes[G].rank != 1) return false;
  for (int i = 0; i < c.n; ++i) {
    const CNode& n = c.nodes[i];
    if (is_scan_root(n) || is_fold_root(n) || is_permute_root(n) || is_segfold_root(n)) return false;
    if (is_store_root(n) && (n.rank != 1 || (depends_on(c, i, G) && !index_preserving_to(c, i, G)))) return false;
  }
  return true;
}
// whose array the staged indices and values live in
template <class CL> constexpr int slab_staging() { return slab_gather_eligible<CL>() ? first_scan<CL>() : stream_staging_root<CL>(); }

// slab of a source index: the source is cut into kSlabs nearly equal ranges (mul = floor(2^32 * kSlabs / elements))
__device__ __forceinline__ uint32_t slab_of(uint32_t k, uint32_t mul) { return min(__umulhi(k, mul), (uint32_t)(kSlabs - 1)); }

// Looks at one warp tile in every (full_tiles / warps launched): the span of its 512 index values.  Indices that
// run through the source in order, or stay within a few KB per warp tile, are served well by the plain gather (a
// monotone index array reads every sector once); random ones are what the passes are for.
template <class CL>
__global__ void __launch_bounds__(kBlock) k_slab_probe(const __grid_constant__ Args<CL::c.n> a, int full_tiles, uint32_t* __restrict__ local) {
  constexpr int G = the_gather<CL>();
  constexpr int KEY = CL::c.nodes[G].in[0];
  constexpr int ROWS = kSlabWarpTile / 128;
  const int lane = threadIdx.x & 31;
  const int warps = gridDim.x * (kBlock / 32);
  const int w = blockIdx.x * (kBlock / 32) + ((int)threadIdx.x >> 5);
  const int wt = (int)(((int64_t)w * full_tiles) / warps);
  uint32_t lo = 0xFFFFFFFFu, hi = 0u;
#pragma unroll
  for (int j = 0; j < ROWS; ++j) {
    const V4 key = eval<CL, KEY>(a, Ix4{0, wt * kSlabWarpTile + (j * 32 + lane) * 4});
#pragma unroll
    for (int e = 0; e < 4; ++e) { lo = min(lo, key.v[e]); hi = max(hi, key.v[e]); }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = min(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
    hi = max(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
  }
  if (lane == 0 && hi - lo < kSlabLocalSpan) atomicAdd(local, 1u);
}

template <class CL>
__global__ void __launch_bounds__(kBlock, 4) k_slab_partition(const __grid_constant__ Args<CL::c.n> a, uint32_t* __restrict__ codes,
                                                               uint32_t* __restrict__ counts, int full_tiles, uint32_t mul, const SlabIn probe) {
  if (slab_passes_stand_back(probe)) return;
  constexpr int G = the_gather<CL>();
  constexpr int S = slab_staging<CL>();
  constexpr int KEY = CL::c.nodes[G].in[0];
  constexpr int ROWS = kSlabWarpTile / 128;
  __shared__ __align__(16) uint32_t stage[kBlock / 32][kSlabWarpTile];       // read 128 bits at a time
  const int lane = threadIdx.x & 31;
  const int stride = gridDim.x * (kBlock / 32);
  uint32_t* staging = reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[S].ptr));
  uint32_t* mine = stage[threadIdx.x >> 5];
  for (int wt = blockIdx.x * (kBlock / 32) + ((int)threadIdx.x >> 5); wt < full_tiles; wt += stride) {
    V4 key[ROWS];
#pragma unroll
    for (int j = 0; j < ROWS; ++j) key[j] = eval<CL, KEY>(a, Ix4{0, wt * kSlabWarpTile + (j * 32 + lane) * 4});
    uint32_t code = 0, c01 = 0, c23 = 0;                           // slabs of this lane's 16 elements; how many in slabs 0 | 1, 2 | 3
#pragma unroll
    for (int j = 0; j < ROWS; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t sl = slab_of(key[j].v[e], mul);
        code |= sl << (2 * (4 * j + e));
        if (sl < 2) c01 += 1u << (16 * (sl & 1)); else c23 += 1u << (16 * (sl & 1));
      }
    uint32_t i01 = c01, i23 = c23;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t u0 = __shfl_up_sync(0xFFFFFFFFu, i01, o), u1 = __shfl_up_sync(0xFFFFFFFFu, i23, o);
      if (lane >= o) { i01 += u0; i23 += u1; }
    }
    const uint32_t T01 = __shfl_sync(0xFFFFFFFFu, i01, 31), T23 = __shfl_sync(0xFFFFFFFFu, i23, 31);
    const uint32_t t0 = T01 & 0xFFFFu, t1 = T01 >> 16, t2 = T23 & 0xFFFFu;
    uint32_t a01 = (i01 - c01) + (t0 << 16);                          // next position in the lists of slabs 0 | 1
    uint32_t a23 = (i23 - c23) + (t0 + t1) + ((t0 + t1 + t2) << 16);  // ... of slabs 2 | 3
    __syncwarp();
#pragma unroll
    for (int j = 0; j < ROWS; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t sl = (code >> (2 * (4 * j + e))) & 3u;
        const uint32_t sh = 16 * (sl & 1);
        mine[((sl < 2 ? a01 : a23) >> sh) & (kSlabWarpTile - 1)] = key[j].v[e];
        if (sl < 2) a01 += 1u << sh; else a23 += 1u << sh;
      }
    __syncwarp();
#pragma unroll
    for (int j = 0; j < ROWS; ++j) {
      const int q = (j * 32 + lane) * 4;
      *reinterpret_cast<uint4*>(staging + (size_t)wt * kSlabWarpTile + q) = *reinterpret_cast<const uint4*>(mine + q);
    }
    codes[(size_t)wt * 32 + lane] = code;
    if (lane == 0) counts[wt] = t0 | (t1 << 10) | (t2 << 20);
  }
}

template <class CL>
__global__ void __launch_bounds__(kBlock) k_slab_gather(const __grid_constant__ Args<CL::c.n> a, const uint32_t* __restrict__ counts,
                                                         int full_tiles, uint32_t slab, const SlabIn probe) {
  if (slab_passes_stand_back(probe)) return;
  constexpr int G = the_gather<CL>();
  constexpr int S = slab_staging<CL>();
  constexpr int SRC = CL::c.nodes[G].in[1];
  constexpr int src_rank = CL::c.nodes[SRC].rank;
  const int lane = threadIdx.x & 31;
  const int stride = gridDim.x * (kBlock / 32);
  uint32_t* staging = reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[S].ptr));
  const uint32_t n_src = (uint32_t)(a.n[SRC].R * a.n[SRC].C);
  for (int wt = blockIdx.x * (kBlock / 32) + ((int)threadIdx.x >> 5); wt < full_tiles; wt += stride) {
    const uint32_t c = __ldg(counts + wt);
    const uint32_t t0 = c & 1023u, t1 = (c >> 10) & 1023u, t2 = (c >> 20) & 1023u;
    const uint32_t lo = slab == 0 ? 0u : slab == 1 ? t0 : slab == 2 ? t0 + t1 : t0 + t1 + t2;
    const uint32_t len = slab == 0 ? t0 : slab == 1 ? t1 : slab == 2 ? t2 : (uint32_t)kSlabWarpTile - (t0 + t1 + t2);
    uint32_t* p = staging + (size_t)wt * kSlabWarpTile + lo;
    for (uint32_t q = lane; q < len; q += 128) {                   // four reads in flight per lane
      uint32_t k[4], v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (q + 32 * u < len) k[u] = min(p[q + 32 * u], n_src - 1);   // (an index outside the source is the caller's error; it reads no foreign memory here)
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (q + 32 * u < len) v[u] = eval<CL, SRC>(a, gather1<src_rank>(k[u], a.n[SRC]));
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (q + 32 * u < len) p[q + 32 * u] = v[u];
    }
  }
}

// (five blocks per SM: the merge is issue bound, and a quarter more warps pay for a few spilled words)
template <class CL, bool STATIC = false>
__global__ void __launch_bounds__(scan_block<CL>(), 5) k_scan_merge(const __grid_constant__ Args<CL::c.n> a, int tiles_per_row, int n_tiles,
                                                                  const SlabIn slab_in) {
  SlabIn slab = slab_in;
  if (slab_passes_stand_back(slab)) slab.full_tiles = 0;     // every warp tile gathers for itself
  scan_tiles<CL, true, true, STATIC>(a, tiles_per_row, n_tiles, slab);
}

// Every root of a scan-less cluster stored from the gathered values of the earlier launches: a warp puts a warp tile
// back into element order and evaluates the roots there (the gather member reads as those values).  The staging
// area is one of the roots' own arrays: a warp has read its whole tile of it before it stores any of it.  Elements
// beyond the last full warp tile are evaluated as usual by the first block.
template <class CL>
__global__ void __launch_bounds__(kBlock, 4) k_stream_merge(const __grid_constant__ Args<CL::c.n> a, const SlabIn slab) {
  constexpr int N = CL::c.n;
  constexpr int Z = stream_staging_root<CL>();
  constexpr int ROWS = kSlabWarpTile / 128;
  __shared__ __align__(16) uint32_t stage[kBlock / 32][kSlabWarpTile];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int stride = gridDim.x * (kBlock / 32);
  if (slab_passes_stand_back(slab)) {
    // nothing was staged: every warp tile is evaluated as it stands
    for (int wt = blockIdx.x * (kBlock / 32) + warp; wt < slab.full_tiles; wt += stride) {
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        const Ix4 ix{0, wt * kSlabWarpTile + (j * 32 + lane) * 4};
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          if constexpr (is_store_root(CL::c.nodes[i]))
            st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), a.n[i].C, ix, eval<CL, i>(a, ix));
        });
      }
    }
  } else {
    for (int wt = blockIdx.x * (kBlock / 32) + warp; wt < slab.full_tiles; wt += stride) {
      V4 gathered[ROWS];
      unpermute_warp_tile<ROWS>(reinterpret_cast<const uint32_t*>(a.n[Z].ptr), slab, wt, stage[warp], gathered);
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        IxGv<Ix4> with;
        with.r = 0;
        with.c = wt * kSlabWarpTile + (j * 32 + lane) * 4;
        with.gv = gathered[j];
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          if constexpr (is_store_root(CL::c.nodes[i])) {
            const Ix4& ix = with;
            uint32_t* out = reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr));
            if constexpr (depends_on(CL::c, i, the_gather<CL>())) st(out, a.n[i].C, ix, eval<CL, i>(a, with));
            else st(out, a.n[i].C, ix, eval<CL, i>(a, ix));
          }
        });
      }
    }
  }
  if (blockIdx.x == 0) {
    for (int c = slab.full_tiles * kSlabWarpTile + (int)threadIdx.x; c < a.C; c += kBlock) {
      const Ix ix{0, c};
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        if constexpr (is_store_root(CL::c.nodes[i]))
          st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), a.n[i].C, ix, eval<CL, i>(a, ix));
      });
    }
  }
}

template <class CL>
__global__ void __launch_bounds__(scan_block<CL>() + 32, 5) k_scan_merge_pipelined(const __grid_constant__ Args<CL::c.n> a, int tiles_per_row, int n_tiles,
                                                                                  const SlabIn slab_in) {
  SlabIn slab = slab_in;
  if (slab_passes_stand_back(slab)) slab.full_tiles = 0;     // every warp tile gathers for itself
  scan_tiles_pipelined<CL, true, true>(a, tiles_per_row, n_tiles, slab);
}

}  // namespace dev
}  // namespace acc
