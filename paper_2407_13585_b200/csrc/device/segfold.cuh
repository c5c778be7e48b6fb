// k_segfold: the skeleton for clusters whose roots are segmented folds over one offsets
// array:  ys[s] = fold(op) of xs[off[s] .. off[s+1]),  xs evaluated in registers from the
// fused producers.
//
// The work is cut by elements, not by segments, so that a few very long segments among many
// short ones (skewed lengths) cost what their elements cost:
//
//  * the source range is cut into tiles of kSegTile elements; a block owns a contiguous run of
//    tiles and walks it in order.  A run of tiles that lies inside one segment is streamed;
//  * any other tile, where the arrays have 128-bit rows: its operands stay in registers, a bit per
//    element marks where segments begin, and a segmented scan (inside a chunk, across a warp by
//    shuffles, across the tile through 32 partial values) gives every element the sum of its
//    segment so far; the elements that end a segment write it.  Uniform work whatever the lengths;
//  * without 128-bit rows the tile's operands are staged in shared memory and the pieces of
//    segments are reduced from there: a thread per piece up to kSegShort elements, a warp per
//    piece up to kSegMedium, the whole block beyond;
//  * a piece that is a whole segment is written at once.  A segment that crosses tiles is carried
//    by the block from tile to tile (a compensated running value in one thread); one that crosses
//    blocks leaves a record per block (the part after its start: `tail`; a part that continues
//    one begun earlier: `head`), and a second, small launch (k_segfold_across) combines the
//    records in block order.
//
// Several segmented folds of one cluster (say a sum and a maximum over the same segments) share
// the walk.  Results do not depend on timing: every order of combination is fixed by the layout.
//
// Offsets are data, so they are checked here, every one of them: a segment that leaves the
// source is reported as ACC_ERR_INDEX_RANGE, an empty or descending one as ACC_ERR_SHAPE (a fold
// has no seed, so an empty segment has no value); pieces are clamped to their tile, so bad
// offsets cannot make the kernel read or write outside its arrays.
#pragma once
#include "skeletons.cuh"

namespace acc {
namespace dev {

constexpr int kSegTile = 4096;                 // elements per tile
constexpr int kSegShort = 32;                  // pieces up to here: one thread
constexpr int kSegMedium = 1024;               // pieces up to here: one warp; longer ones: the block
constexpr int kSegListCap = kSegTile / (kSegShort + 1) + 2;
constexpr int kSegBigCap = kSegTile / (kSegMedium + 1) + 2;    // pieces of a tile the whole block reduces
constexpr int kSegResident = 4;                // blocks per SM the kernel is built for
constexpr int kSegTilesPerBlock = 8;           // a block's run of tiles: short enough for the block scheduler to even out slow and fast runs
constexpr int kSegWindow = 1024;               // offsets kept in shared memory at a time
constexpr uint32_t kStatusEmptySegment = 4u;

template <class CL> constexpr int first_segfold() {
  for (int i = 0; i < CL::c.n; ++i)
    if (is_segfold_root(CL::c.nodes[i])) return i;
  return -1;
}

// All segmented folds of the cluster must read one offsets array, and nothing else may be a root.
template <class CL> constexpr bool segfold_eligible() {
  const int f = first_segfold<CL>();
  if (f < 0) return false;
  for (int i = 0; i < CL::c.n; ++i) {
    const CNode& n = CL::c.nodes[i];
    if (is_store_root(n) || is_fold_root(n) || is_scan_root(n) || is_permute_root(n)) return false;
    if (is_segfold_root(n) && n.in[1] != CL::c.nodes[f].in[1]) return false;
  }
  return true;
}

// Scratch of k_segfold (32-bit words): from word 4 two records per block, `head`
// then `tail`, of 2 + NF words each: segment id + 1 (0: no record), unused, one value per fold.
__host__ __device__ inline int seg_record_words(int n_folds) { return 2 + n_folds; }
__host__ __device__ inline int64_t seg_scratch_words(int n_folds, int grid) { return 4 + (int64_t)grid * 2 * seg_record_words(n_folds); }

// Largest s in [0, S) with off[s] <= x, for off[0] <= x < off[S] (any s for other x): a 32-way search by one warp.
__device__ __forceinline__ int seg_containing(const int32_t* off, int S, int x, int lane) {
  int lo = 0, hi = S;                                          // off[lo] <= x < off[hi]
  while (hi - lo > 1) {
    const int step = (hi - lo + 31) / 32;
    const int p = lo + (lane + 1) * step;
    const bool ok = p < hi && __ldg(off + p) <= x;             // true for a prefix of the lanes
    const int k = __popc(__ballot_sync(0xFFFFFFFFu, ok));
    const int nlo = lo + k * step;
    hi = min(hi, nlo + step);
    lo = nlo;
  }
  return lo;
}

template <class CL, bool VEC>
__global__ void __launch_bounds__(kBlock, kSegResident) k_segfold(const __grid_constant__ Args<CL::c.n> a, int tiles_per_block) {
  constexpr int N = CL::c.n;
  constexpr int F = first_segfold<CL>();
  constexpr int NF = count_if<CL>(is_segfold_root);
  constexpr int WARPS = kBlock / 32;
  constexpr int REC = 2 + NF;
  extern __shared__ __align__(16) uint32_t seg_vals[];                         // NF arrays of kSegTile operand values
  __shared__ uint32_t red[WARPS];
  __shared__ int off_win[kSegWindow + 1];                        // offsets of segments win_base .. win_base + kSegWindow
  __shared__ int long_seg[kSegListCap], long_lo[kSegListCap], long_hi[kSegListCap], long_kind[kSegListCap];
  __shared__ int big_seg[kSegBigCap], big_lo[kSegBigCap], big_hi[kSegBigCap], big_kind[kSegBigCap];
  __shared__ uint32_t seg_bits[VEC ? kSegTile / 32 + 2 : 1];      // bit p: element p of the tile begins a segment
  __shared__ int seg_before[VEC ? kSegTile / 32 : 1];            // starts before each 32-element word
  __shared__ uint32_t seg_unit_flag[VEC ? 32 : 1], seg_unit_val[VEC ? NF : 1][VEC ? 32 : 1];
  __shared__ int tile_open;
  __shared__ int n_long, n_big, next_s, first_open, have_first, have_last, last_seg;
  __shared__ uint32_t first_val[NF], last_val[NF];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int S = a.C;                                             // segments
  constexpr int OFF = CL::c.nodes[F].in[1], SRC = CL::c.nodes[F].in[0];
  const int32_t* off = reinterpret_cast<const int32_t*>(a.n[OFF].ptr);
  const int n_src = a.n[SRC].R * a.n[SRC].C;
  uint32_t* rec = a.scratch + 4;

  // every offset is looked at once, whatever the walk below does with it
  for (int s = blockIdx.x * kBlock + threadIdx.x; s < S; s += gridDim.x * kBlock) {
    const int lo = __ldg(off + s), hi = __ldg(off + s + 1);
    if (lo < 0 || hi > n_src) atomicOr(a.status, kStatusIndex);
    else if (hi <= lo) atomicOr(a.status, kStatusEmptySegment);
  }

  auto fold_slot_of = [](int i) { return count_if<CL>(is_segfold_root, i); };
  // kind of a piece: bit 0 = it continues a segment begun before the tile, bit 1 = its segment goes on after the tile
  auto store_piece = [&](int s, int kind, const uint32_t (&v)[N]) {
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      if constexpr (is_segfold_root(CL::c.nodes[i])) {
        const int f = fold_slot_of(i);
        if (kind & 1) first_val[f] = v[i];
        else if (kind & 2) last_val[f] = v[i];
        else reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[s] = v[i];
      }
    });
    if (kind & 1) { have_first = 1; first_open = kind >> 1; }
    else if (kind & 2) { have_last = 1; last_seg = s; }
  };
  // Inside a tile sums are plain: a thread adds at most 32 staged values and trees do the rest, which
  // stays far inside the tolerance; what is compensated is the running value a segment keeps from
  // tile to tile (thousands of steps for a long one).
  auto reduce_strided = [&](int plo, int phi, int first, int stride, int tile_lo, uint32_t (&v)[N]) {
    uint32_t w[4][N];
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_segfold_root(nd)) {
#pragma unroll
        for (int u = 0; u < 4; ++u) w[u][i] = identity_of<nd.fn, nd.dtype>();
      }
    });
    int j = plo + first;
    for (; j + 3 * stride < phi; j += 4 * stride) {              // four independent running values per fold
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) {
          const uint32_t* src = seg_vals + fold_slot_of(i) * kSegTile - tile_lo;
#pragma unroll
          for (int u = 0; u < 4; ++u) w[u][i] = combine<nd.fn, nd.dtype>(w[u][i], src[j + u * stride]);
        }
      });
    }
    for (; j < phi; j += stride) {
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) w[0][i] = combine<nd.fn, nd.dtype>(w[0][i], (seg_vals + fold_slot_of(i) * kSegTile - tile_lo)[j]);
      });
    }
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_segfold_root(nd))
        v[i] = combine<nd.fn, nd.dtype>(combine<nd.fn, nd.dtype>(w[0][i], w[1][i]), combine<nd.fn, nd.dtype>(w[2][i], w[3][i]));
    });
  };

  const int e_lo = max(__ldg(off), 0), e_hi = min(__ldg(off + S), n_src);   // elements that belong to segments
  const int first_tile = blockIdx.x * tiles_per_block;
  int s_cur = 0;                                                 // the segment that holds the next element to process (uniform)
  int win_base = -1;                                             // first segment of the offsets window, -1: not filled (uniform)
  // the block's carry: the running value of the segment that is open at the end of the last tile (thread 0)
  int carry_seg = -1;
  bool carry_from_here = false;
  uint32_t carry[N];
  float carry_comp[N] = {};

  for (int t = 0; t < tiles_per_block; ++t) {                    // (a run of tiles inside one segment advances t by its length)
    const int64_t tile_lo64 = (int64_t)(first_tile + t) * kSegTile;
    if (tile_lo64 >= e_hi) break;
    const int tile_lo = (int)tile_lo64;
    const int tile_hi = (int)(tile_lo64 + kSegTile < (int64_t)e_hi ? tile_lo64 + kSegTile : (int64_t)e_hi);
    const int lo0 = max(tile_lo, e_lo);
    if (lo0 >= tile_hi) continue;
    __syncthreads();                                             // the previous tile's values and flags have been read
    if (win_base < 0) {                                          // the block's first tile: which segment holds its first element
      if (warp == 0) {
        const int s0 = seg_containing(off, S, lo0, lane);
        if (lane == 0) next_s = s0;
      }
      __syncthreads();
      s_cur = next_s;
      __syncthreads();
    }
    if (win_base < 0 || s_cur + kBlock > win_base + kSegWindow) {  // uniform: the window of offsets moves up to s_cur
      win_base = s_cur;
      for (int k = threadIdx.x; k <= kSegWindow; k += kBlock) off_win[k] = s_cur + k <= S ? __ldg(off + s_cur + k) : 0x7FFFFFFF;
      __syncthreads();
    }
    if (threadIdx.x == 0) { n_long = 0; n_big = 0; have_first = 0; have_last = 0; first_open = 0; next_s = s_cur; }
    // Tiles that lie inside one segment need no staging: the block streams through all of them that are
    // its own, every thread keeping a compensated running value per fold, and reduces once at the end.
    const int lo_c = off_win[s_cur - win_base], hi_c = off_win[s_cur - win_base + 1];
    const bool whole = s_cur < S && lo_c <= lo0 && hi_c >= tile_hi && lo0 == tile_lo && tile_hi - tile_lo == kSegTile;
    if (whole) {                                                 // uniform
      const int own_end = first_tile + tiles_per_block;          // first tile that is not this block's
      const int inside_end = min(hi_c, e_hi) / kSegTile;         // first tile that is not wholly inside the segment
      const int run = max(1, min(own_end, inside_end) - (first_tile + t));
      const int run_hi = tile_lo + run * kSegTile;               // (no overflow: run_hi <= e_hi)
      uint32_t acc[N];
      float comp[N] = {};
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) acc[i] = identity_of<nd.fn, nd.dtype>();
      });
      if constexpr (VEC) {
        // a tile is four trips of the block, so the run is a whole number of these steps: four chunks in flight per fold
        for (int c = tile_lo + (int)threadIdx.x * 4; c < run_hi; c += kSegTile) {
          static_for<0, N>([&](auto ic) {
            constexpr int i = decltype(ic)::value;
            constexpr CNode nd = CL::c.nodes[i];
            if constexpr (is_segfold_root(nd)) {
              V4 x[kSegTile / (4 * kBlock)];
#pragma unroll
              for (int u = 0; u < kSegTile / (4 * kBlock); ++u) x[u] = eval<CL, nd.in[0]>(a, Ix4{0, c + u * kBlock * 4});
#pragma unroll
              for (int u = 0; u < kSegTile / (4 * kBlock); ++u)
                fold_step<nd.fn, nd.dtype>(acc[i], comp[i], combine<nd.fn, nd.dtype>(combine<nd.fn, nd.dtype>(x[u].v[0], x[u].v[1]),
                                                                                     combine<nd.fn, nd.dtype>(x[u].v[2], x[u].v[3])));
            }
          });
        }
      } else {
        for (int q = tile_lo + (int)threadIdx.x; q < run_hi; q += kBlock) {
          static_for<0, N>([&](auto ic) {
            constexpr int i = decltype(ic)::value;
            constexpr CNode nd = CL::c.nodes[i];
            if constexpr (is_segfold_root(nd)) fold_step<nd.fn, nd.dtype>(acc[i], comp[i], eval<CL, nd.in[0]>(a, Ix{0, q}));
          });
        }
      }
      uint32_t v[N];
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) v[i] = block_reduce<nd.fn, nd.dtype>(acc[i], red);
      });
      if (threadIdx.x == 0) {
        store_piece(s_cur, (lo_c < lo0 ? 1 : 0) | (hi_c > run_hi ? 2 : 0), v);
        next_s = hi_c > run_hi ? s_cur : s_cur + 1;
      }
      t += run - 1;
    } else if constexpr (VEC) {
      // ---- a tile with pieces of several segments, 128-bit rows: a segmented scan over the tile in registers ----
      // Thread t holds chunks (j * kBlock + t) * 4, j = 0..3, of the tile; in the order (j, warp, lane, element) the
      // values form one sequence.  `bits` marks the elements that begin a segment.  Every element gets the sum of
      // its segment up to itself: inside a chunk, across the lanes of a warp (a shuffle scan that stops at lanes
      // holding a start), across the 32 (row, warp) units through shared memory; elements that end a segment
      // (the next one begins one, or the tile ends) then hold that segment's sum over the tile and write it.
      constexpr int ROWS = kSegTile / (4 * kBlock);
      static_assert(ROWS * WARPS == 32, "the (row, warp) units of a tile are scanned by the lanes of one warp");
      uint32_t xv[N][ROWS][4];
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) {
#pragma unroll
          for (int j = 0; j < ROWS; ++j) {
            const int c = tile_lo + (j * kBlock + (int)threadIdx.x) * 4;
            V4 v = V4{{identity_of<nd.fn, nd.dtype>(), identity_of<nd.fn, nd.dtype>(), identity_of<nd.fn, nd.dtype>(), identity_of<nd.fn, nd.dtype>()}};
            if (c < tile_hi) v = eval<CL, nd.in[0]>(a, Ix4{0, c});
#pragma unroll
            for (int e = 0; e < 4; ++e) xv[i][j][e] = c + e < tile_hi ? v.v[e] : identity_of<nd.fn, nd.dtype>();
          }
        }
      });
      for (int k = threadIdx.x; k < kSegTile / 32 + 2; k += kBlock) seg_bits[k] = 0;
      if (threadIdx.x == 0) tile_open = 0;
      __syncthreads();
      for (int base = s_cur;; base += kBlock) {                  // a thread per segment: where it begins, if that is in the tile
        if (base + kBlock > win_base + kSegWindow) {             // uniform: the window moves up to `base`
          __syncthreads();
          win_base = base;
          for (int k = threadIdx.x; k <= kSegWindow; k += kBlock) off_win[k] = base + k <= S ? __ldg(off + base + k) : 0x7FFFFFFF;
          __syncthreads();
        }
        const int s = base + (int)threadIdx.x;
        const int lo_s = off_win[s - win_base], hi_s = off_win[s - win_base + 1];
        const bool beyond = s >= S || lo_s >= tile_hi;
        if (!beyond) {
          if (lo_s >= lo0) atomicOr(&seg_bits[(lo_s - tile_lo) >> 5], 1u << ((lo_s - tile_lo) & 31));
          if (hi_s >= tile_hi) { next_s = hi_s > tile_hi ? s : s + 1; tile_open = hi_s > tile_hi ? 1 : 0; }
        }
        if (__syncthreads_or(beyond)) break;
      }
      if (warp == 0) {                                           // starts before each 32-element word of the tile
        int cnt[4], sum = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) { cnt[k] = sum; sum += __popc(seg_bits[4 * lane + k]); }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int u = __shfl_up_sync(0xFFFFFFFFu, incl, o);
          if (lane >= o) incl += u;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) seg_before[4 * lane + k] = incl - sum + cnt[k];
      }
      __syncthreads();
      const bool cont = lo_c < lo0, open = tile_open != 0;
      const int lo_rel = lo0 - tile_lo, hi_rel = tile_hi - tile_lo;
      uint32_t cin[N][ROWS];                                     // what precedes the chunk in its run, within the warp's row
      uint32_t marks[ROWS];                                      // bits 0-3: starts in the chunk, 4: start right after it, 5: no start in earlier lanes
      int before[ROWS];                                          // starts before the chunk, in the tile
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        const int p = (j * kBlock + (int)threadIdx.x) * 4, w = p >> 5, sh = p & 31;
        const uint32_t word = seg_bits[w];
        const uint32_t b5 = __funnelshift_r(word, seg_bits[w + 1], sh) & 31u, b = b5 & 15u;
        before[j] = seg_before[w] + __popc(word & ((1u << sh) - 1u));
        const unsigned H = __ballot_sync(0xFFFFFFFFu, b != 0);
        const unsigned upto = H & (0xFFFFFFFFu >> (31 - lane));  // lanes up to this one that hold a start
        const int lower = upto ? 31 - __clz(upto) : 0;            // the run this chunk's end belongs to begins in that lane
        marks[j] = b5 | ((H & ((1u << lane) - 1u)) == 0 ? 32u : 0u);
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          constexpr CNode nd = CL::c.nodes[i];
          if constexpr (is_segfold_root(nd)) {
#pragma unroll
            for (int e = 1; e < 4; ++e)
              if (!((b >> e) & 1u)) xv[i][j][e] = combine<nd.fn, nd.dtype>(xv[i][j][e - 1], xv[i][j][e]);
            uint32_t run = xv[i][j][3];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
              const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, run, o);
              if (lane - o >= lower) run = combine<nd.fn, nd.dtype>(u, run);
            }
            const uint32_t prev = __shfl_up_sync(0xFFFFFFFFu, run, 1);
            cin[i][j] = lane == 0 ? identity_of<nd.fn, nd.dtype>() : prev;
            if (lane == 31) seg_unit_val[fold_slot_of(i)][j * WARPS + warp] = run;
          }
        });
        if (lane == 31) seg_unit_flag[j * WARPS + warp] = H != 0 ? 1u : 0u;
      }
      __syncthreads();
      // the 32 (row, warp) units in sequence: what runs into each of them from the units before
      const unsigned UH = __ballot_sync(0xFFFFFFFFu, seg_unit_flag[lane] != 0);
      const unsigned uupto = UH & (0xFFFFFFFFu >> (31 - lane));
      const int ulower = uupto ? 31 - __clz(uupto) : 0;
#pragma unroll
      for (int j = 0; j < ROWS; ++j) before[j] -= cont ? 0 : 1;  // now: the chunk's first element lies in segment s_cur + before (+ starts up to it)
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) {
          uint32_t run = seg_unit_val[fold_slot_of(i)][lane];
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, run, o);
            if (lane - o >= ulower) run = combine<nd.fn, nd.dtype>(u, run);
          }
#pragma unroll
          for (int j = 0; j < ROWS; ++j) {
            const int unit = j * WARPS + warp;
            const uint32_t into = __shfl_sync(0xFFFFFFFFu, run, max(unit - 1, 0));
            if ((marks[j] & 32u) && unit > 0) cin[i][j] = combine<nd.fn, nd.dtype>(into, cin[i][j]);
          }
        }
      });
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        const int p = (j * kBlock + (int)threadIdx.x) * 4;
        const uint32_t b = marks[j] & 15u;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int pos = p + e;
          const bool ends = pos >= lo_rel && pos < hi_rel && (pos == hi_rel - 1 || ((marks[j] >> (e + 1)) & 1u));
          if (ends) {
            const bool led = (b & ((2u << e) - 1u)) == 0;          // no start in the chunk up to here: the run comes in from before
            const int seg = s_cur + before[j] + __popc(b & ((2u << e) - 1u));
            uint32_t v[N];
            static_for<0, N>([&](auto ic) {
              constexpr int i = decltype(ic)::value;
              constexpr CNode nd = CL::c.nodes[i];
              if constexpr (is_segfold_root(nd)) v[i] = led ? combine<nd.fn, nd.dtype>(cin[i][j], xv[i][j][e]) : xv[i][j][e];
            });
            if ((uint32_t)seg < (uint32_t)S)
              store_piece(seg, ((seg == s_cur && cont) ? 1 : 0) | ((pos == hi_rel - 1 && open) ? 2 : 0), v);
          }
        }
      }
    } else {
    // stage the operands of the tile
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_segfold_root(nd)) {
        uint32_t* dst = seg_vals + fold_slot_of(i) * kSegTile;
        if constexpr (VEC) {
          V4 v[kSegTile / (4 * kBlock)];
#pragma unroll
          for (int j = 0; j < kSegTile / (4 * kBlock); ++j) {
            const int c = tile_lo + (j * kBlock + (int)threadIdx.x) * 4;
            if (c < tile_hi) v[j] = eval<CL, nd.in[0]>(a, Ix4{0, c});
          }
#pragma unroll
          for (int j = 0; j < kSegTile / (4 * kBlock); ++j) {
            const int q = (j * kBlock + (int)threadIdx.x) * 4;
            if (tile_lo + q < tile_hi) *reinterpret_cast<uint4*>(dst + q) = make_uint4(v[j].v[0], v[j].v[1], v[j].v[2], v[j].v[3]);
          }
        } else {
          for (int q = threadIdx.x; q < tile_hi - tile_lo; q += kBlock) dst[q] = eval<CL, nd.in[0]>(a, Ix{0, tile_lo + q});
        }
      }
    });

    // the pieces of the tile, a thread per segment; those beyond kSegShort elements are set aside
    for (int base = s_cur;; base += kBlock) {
      if (win_base < 0 || base + kBlock > win_base + kSegWindow) {     // uniform: the window moves up to `base`
        __syncthreads();
        win_base = base;
        for (int k = threadIdx.x; k <= kSegWindow; k += kBlock) off_win[k] = base + k <= S ? __ldg(off + base + k) : 0x7FFFFFFF;
      }
      __syncthreads();
      const int s = base + (int)threadIdx.x;
      const int lo_s = off_win[s - win_base], hi_s = off_win[s - win_base + 1];
      const bool beyond = s >= S || lo_s >= tile_hi;
      if (!beyond) {
        const int plo = max(lo_s, lo0), phi = min(hi_s, tile_hi);
        if (hi_s >= tile_hi) next_s = hi_s > tile_hi ? s : s + 1;      // the segment that holds the tile's last element
        if (phi > plo) {
          const int kind = (lo_s < lo0 ? 1 : 0) | (hi_s > tile_hi ? 2 : 0);
          if (phi - plo <= kSegShort) {
            uint32_t v[N];
            reduce_strided(plo, phi, 0, 1, tile_lo, v);
            store_piece(s, kind, v);
          } else if (phi - plo <= kSegMedium) {
            const int at = atomicAdd(&n_long, 1);
            if (at < kSegListCap) { long_seg[at] = s; long_lo[at] = plo; long_hi[at] = phi; long_kind[at] = kind; }
          } else {
            const int at = atomicAdd(&n_big, 1);
            if (at < kSegBigCap) { big_seg[at] = s; big_lo[at] = plo; big_hi[at] = phi; big_kind[at] = kind; }
          }
        }
      }
      if (__syncthreads_or(beyond)) break;
    }
    const int todo = min(n_long, kSegListCap);
    // a warp per piece of medium length
    for (int k = warp; k < todo; k += WARPS) {
      const int plo = long_lo[k], phi = long_hi[k];
      uint32_t v[N];
      reduce_strided(plo, phi, lane, 32, tile_lo, v);
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) v[i] = warp_reduce<nd.fn, nd.dtype>(v[i]);
      });
      if (lane == 0) store_piece(long_seg[k], long_kind[k], v);
    }
    // the whole block per piece beyond that (at most three of them in a tile)
    const int todo_big = min(n_big, kSegBigCap);
    for (int k = 0; k < todo_big; ++k) {
      const int plo = big_lo[k], phi = big_hi[k];
      uint32_t v[N];
      reduce_strided(plo, phi, (int)threadIdx.x, kBlock, tile_lo, v);
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) v[i] = block_reduce<nd.fn, nd.dtype>(v[i], red);
      });
      if (threadIdx.x == 0) store_piece(big_seg[k], big_kind[k], v);
    }
    }
    __syncthreads();

    // segments that cross the tile's ends: the block's running value
    if (threadIdx.x == 0) {
      if (have_first) {
        if (carry_seg != s_cur) {                              // begun before this block: nothing carried yet
          carry_seg = s_cur;
          carry_from_here = false;
          static_for<0, N>([&](auto ic) {
            constexpr int i = decltype(ic)::value;
            if constexpr (is_segfold_root(CL::c.nodes[i])) { carry[i] = first_val[fold_slot_of(i)]; carry_comp[i] = 0.0f; }
          });
        } else {
          static_for<0, N>([&](auto ic) {
            constexpr int i = decltype(ic)::value;
            constexpr CNode nd = CL::c.nodes[i];
            if constexpr (is_segfold_root(nd)) fold_step<nd.fn, nd.dtype>(carry[i], carry_comp[i], first_val[fold_slot_of(i)]);
          });
        }
        if (!first_open) {                                     // the segment ends in this tile
          uint32_t* head = rec + (size_t)blockIdx.x * 2 * REC;
          if (!carry_from_here) head[0] = (uint32_t)carry_seg + 1u;
          static_for<0, N>([&](auto ic) {
            constexpr int i = decltype(ic)::value;
            if constexpr (is_segfold_root(CL::c.nodes[i])) {
              if (carry_from_here) reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[carry_seg] = carry[i];
              else head[2 + fold_slot_of(i)] = carry[i];
            }
          });
          carry_seg = -1;
        }
      }
      if (have_last) {
        carry_seg = last_seg;
        carry_from_here = true;
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          if constexpr (is_segfold_root(CL::c.nodes[i])) { carry[i] = last_val[fold_slot_of(i)]; carry_comp[i] = 0.0f; }
        });
      }
    }
    s_cur = next_s;                                              // written before the barrier above, by the one thread that saw it
  }

  // what is still open where the block's run of tiles ends
  if (threadIdx.x == 0 && carry_seg >= 0) {
    uint32_t* r = rec + ((size_t)blockIdx.x * 2 + (carry_from_here ? 1 : 0)) * REC;
    r[0] = (uint32_t)carry_seg + 1u;
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      if constexpr (is_segfold_root(CL::c.nodes[i])) r[2 + fold_slot_of(i)] = carry[i];
    });
  }
}

// Second launch of a segmented-fold cluster: segments that cross the blocks of k_segfold.  A warp per block
// that left a `tail` (the part of a segment after its start): its lanes look at the blocks that follow, 32 at a
// time, take the `head` records that continue the segment, and combine them in a fixed order.
template <class CL>
__global__ void __launch_bounds__(kBlock) k_segfold_across(const __grid_constant__ Args<CL::c.n> a, int n_blocks) {
  constexpr int N = CL::c.n;
  constexpr int NF = count_if<CL>(is_segfold_root);
  constexpr int REC = 2 + NF;
  auto fold_slot_of = [](int i) { return count_if<CL>(is_segfold_root, i); };
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (kBlock / 32) + ((int)threadIdx.x >> 5);
  if (b >= n_blocks) return;
  const uint32_t* rec = a.scratch + 4;
  const uint32_t* tail = rec + ((size_t)b * 2 + 1) * REC;
  const uint32_t key = tail[0];
  if (key == 0) return;                                          // the same for the whole warp
  uint32_t v[N];
  static_for<0, N>([&](auto ic) {
    constexpr int i = decltype(ic)::value;
    if constexpr (is_segfold_root(CL::c.nodes[i])) v[i] = tail[2 + fold_slot_of(i)];
  });
  for (int base = b + 1; base < n_blocks; base += 32) {
    const int b2 = base + lane;
    const uint32_t* head = rec + (size_t)min(b2, n_blocks - 1) * 2 * REC;
    const bool same = b2 < n_blocks && head[0] == key;
    const unsigned others = ~__ballot_sync(0xFFFFFFFFu, same);
    const int n = others ? __ffs(others) - 1 : 32;               // blocks of this round that continue the segment
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_segfold_root(nd)) {
        const uint32_t x = lane < n ? head[2 + fold_slot_of(i)] : identity_of<nd.fn, nd.dtype>();
        v[i] = combine<nd.fn, nd.dtype>(v[i], warp_reduce<nd.fn, nd.dtype>(x));
      }
    });
    if (n < 32) break;
  }
  if (lane == 0) {
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      if constexpr (is_segfold_root(CL::c.nodes[i])) reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[key - 1] = v[i];
    });
  }
}

}  // namespace dev
}  // namespace acc
