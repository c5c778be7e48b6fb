// k_segfold: the skeleton for clusters whose roots are segmented folds over one offsets
// array:  ys[s] = fold(op) of xs[off[s] .. off[s+1]),  xs evaluated in registers from the
// fused producers.
//
// A warp takes a segment and walks it with coalesced reads, ending in a shuffle tree; eight
// consecutive segments go to the eight warps of a block.  A segment longer than kSegLong
// elements is set aside and reduced by the whole block afterwards, so that one long segment
// does not hold a single warp for its whole length.  Several segmented folds of one cluster
// (say a sum and a maximum over the same segments) share the walk and every load their
// producers have in common.  Results do not depend on timing: the order of combination is
// fixed by the thread layout.
//
// Offsets are data, so they are checked here: a segment that leaves the source is skipped
// and reported as ACC_ERR_INDEX_RANGE, an empty or descending one as ACC_ERR_SHAPE (a fold
// has no seed, so an empty segment has no value).
#pragma once
#include "skeletons.cuh"

namespace acc {
namespace dev {

constexpr int kSegLong = 1 << 14;
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

template <class CL>
__global__ void __launch_bounds__(kBlock) k_segfold(const __grid_constant__ Args<CL::c.n> a) {
  constexpr int N = CL::c.n;
  constexpr int F = first_segfold<CL>();
  constexpr int WARPS = kBlock / 32;
  __shared__ uint32_t red[WARPS];
  __shared__ int long_list[WARPS];
  __shared__ int n_long;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int S = a.C;                                               // segments
  constexpr int OFF = CL::c.nodes[F].in[1], SRC = CL::c.nodes[F].in[0];
  const int32_t* off = reinterpret_cast<const int32_t*>(a.n[OFF].ptr);
  const int n_src = a.n[SRC].R * a.n[SRC].C;

  for (int base = blockIdx.x * WARPS; base < S; base += gridDim.x * WARPS) {
    __syncthreads();
    if (threadIdx.x == 0) n_long = 0;
    __syncthreads();
    const int s = base + warp;
    if (s < S) {
      const int lo = __ldg(off + s), hi = __ldg(off + s + 1);
      if (lo < 0 || hi > n_src) {
        if (lane == 0) atomicOr(a.status, kStatusIndex);
      } else if (hi <= lo) {
        if (lane == 0) atomicOr(a.status, kStatusEmptySegment);
      } else if (hi - lo > kSegLong) {
        if (lane == 0) long_list[atomicAdd(&n_long, 1)] = s;
      } else {
        uint32_t acc[N];
        float comp[N] = {};                              // see fold_step
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          constexpr CNode nd = CL::c.nodes[i];
          if constexpr (is_segfold_root(nd)) acc[i] = identity_of<nd.fn, nd.dtype>();
        });
        for (int j = lo + lane; j < hi; j += 32) {
          static_for<0, N>([&](auto ic) {
            constexpr int i = decltype(ic)::value;
            constexpr CNode nd = CL::c.nodes[i];
            if constexpr (is_segfold_root(nd)) fold_step<nd.fn, nd.dtype>(acc[i], comp[i], eval<CL, nd.in[0]>(a, Ix{0, j}));
          });
        }
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          constexpr CNode nd = CL::c.nodes[i];
          if constexpr (is_segfold_root(nd)) {
            const uint32_t v = warp_reduce<nd.fn, nd.dtype>(acc[i]);
            if (lane == 0) reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[s] = v;
          }
        });
      }
    }
    __syncthreads();
    const int todo = n_long;
    for (int k = 0; k < todo; ++k) {                              // long segments: the whole block each
      const int t = long_list[k];
      const int lo = __ldg(off + t), hi = __ldg(off + t + 1);
      uint32_t acc[N];
      float comp[N] = {};
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) acc[i] = identity_of<nd.fn, nd.dtype>();
      });
      for (int j = lo + (int)threadIdx.x; j < hi; j += kBlock) {
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          constexpr CNode nd = CL::c.nodes[i];
          if constexpr (is_segfold_root(nd)) fold_step<nd.fn, nd.dtype>(acc[i], comp[i], eval<CL, nd.in[0]>(a, Ix{0, j}));
        });
      }
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_segfold_root(nd)) {
          const uint32_t v = block_reduce<nd.fn, nd.dtype>(acc[i], red);
          if (threadIdx.x == 0) reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[t] = v;
        }
      });
    }
  }
}

}  // namespace dev
}  // namespace acc
