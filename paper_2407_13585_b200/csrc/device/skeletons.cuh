// The three kernel skeletons a fused cluster is instantiated into.
//
//   k_stream   grid-stride pass over the cluster's iteration domain; stores every manifest
//              element-wise member, accumulates whole-array folds (warp shuffles, block
//              tree, ordered cross-block combine by the last block) and applies permutes
//              with atomics.
//   k_rowfold  one block per row of a rank-2 domain; folds of the innermost extent end in a
//              block reduction, no atomics.
//   k_scan     single-pass scan with decoupled look-back; the scanned operand is evaluated in
//              registers.  A tile's predecessors are always running or done: the grid is
//              cooperative and block b takes tiles b, b + G, ..., or tiles are claimed from an
//              atomic ticket.  k_scan_pipelined is the same scan with a warp that only looks
//              back, for small tiles.
//
// Each is templated on the cluster description (what to evaluate) and on VEC (whether four
// consecutive elements move as one 128-bit access).
#pragma once
#include "eval.cuh"

namespace acc {
namespace dev {

constexpr int kBlock = 256;
constexpr int kStreamTileRows = kBlock / 32;   // rows of a rank-2 tile of k_stream (one warp each)
constexpr uint32_t kStatusTimeout = 1u;
constexpr uint32_t kStatusIndex = 2u;

template <int FN, int DT>
__device__ __forceinline__ uint32_t warp_reduce(uint32_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = combine<FN, DT>(v, __shfl_down_sync(0xFFFFFFFFu, v, o));
  return v;
}

// Reduces over a block of THREADS threads; the result is valid in thread 0.  `red` holds
// THREADS/32 words.
template <int FN, int DT, int THREADS>
__device__ __forceinline__ uint32_t block_reduce_n(uint32_t v, uint32_t* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_reduce<FN, DT>(v);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  if (warp == 0) {
    v = lane < THREADS / 32 ? red[lane] : identity_of<FN, DT>();
    v = warp_reduce<FN, DT>(v);
  }
  return v;
}
template <int FN, int DT>
__device__ __forceinline__ uint32_t block_reduce(uint32_t v, uint32_t* red) {
  return block_reduce_n<FN, DT, kBlock>(v, red);
}

// ---- compile-time layout of a cluster's roots ------------------------------------------
template <class CL> constexpr int count_if(bool (*pred)(const CNode&), int upto = CL::c.n) {
  int k = 0;
  for (int i = 0; i < upto; ++i) k += pred(CL::c.nodes[i]) ? 1 : 0;
  return k;
}
constexpr bool is_f32_add_permute(const CNode& n) { return is_permute_root(n) && n.dtype == ACC_F32 && n.fn == ACC_FN_ADD; }
constexpr bool is_scalar_fold(const CNode& n) { return is_fold_root(n) && n.rank == 0; }
constexpr bool is_row_fold(const CNode& n) { return is_fold_root(n) && n.rank > 0; }

template <class CL> constexpr int first_scan() {
  for (int i = 0; i < CL::c.n; ++i)
    if (is_scan_root(CL::c.nodes[i])) return i;
  return -1;
}

// Rank of the iteration domain: taken from the first root.
template <class CL> constexpr int domain_rank() {
  for (int i = 0; i < CL::c.n; ++i) {
    const CNode& n = CL::c.nodes[i];
    if (is_store_root(n) || is_scan_root(n)) return n.rank;
    if (is_fold_root(n)) return CL::c.nodes[n.in[0]].rank;
    if (is_permute_root(n)) return CL::c.nodes[n.in[1]].rank;
  }
  return 1;
}

template <class CL> constexpr bool has_reversal() {
  for (int i = 0; i < CL::c.n; ++i)
    if (CL::c.nodes[i].member && CL::c.nodes[i].kind == ACC_BACKPERMUTE && CL::c.nodes[i].idxfn == ACC_IDX_REVERSE) return true;
  return false;
}

// Scratch layout of k_stream (32-bit words): [0] ticket, [4 ..) one partial per block per
// scalar fold, then (8-byte aligned) one fp64 accumulator per bin per fp32 '+' permute.
__host__ __device__ inline uint32_t stream_partials_off() { return 4; }
__host__ __device__ inline uint32_t stream_acc64_off(int n_scalar_folds, int grid) {
  return (4u + (uint32_t)(n_scalar_folds * grid) + 1u) & ~1u;
}

template <int FN, int DT>
__device__ __forceinline__ void permute_update(uint32_t* out, double* acc64, uint32_t bins, uint32_t k, uint32_t x,
                                               uint32_t* status) {
  if (k >= bins) { atomicOr(status, kStatusIndex); return; }
  if constexpr (DT == ACC_F32 && FN == ACC_FN_ADD) {
    // lanes of the warp that hit the same bin are summed first; one fp64 atomic per bin and warp
    const unsigned peers = __match_any_sync(__activemask(), k);
    double sum = 0.0;
    for (unsigned t = peers; t; t &= t - 1) sum += (double)__shfl_sync(peers, f_(x), __ffs(t) - 1);
    if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(acc64 + k, sum);
  } else if constexpr (FN == ACC_FN_ADD) {
    atomicAdd(out + k, x);
  } else if constexpr (FN == ACC_FN_MIN) {
    if constexpr (DT == ACC_I32) atomicMin(reinterpret_cast<int*>(out) + k, (int)x); else atomicMin(out + k, x);
  } else {
    if constexpr (DT == ACC_I32) atomicMax(reinterpret_cast<int*>(out) + k, (int)x); else atomicMax(out + k, x);
  }
}

// fp64 accumulators of the I-th member (an fp32 '+' permute): after those of earlier ones.
template <class CL, int I, class A>
__device__ __forceinline__ double* acc64_of(const A& a, double* base) {
  static_for<0, I>([&](auto jc) {
    constexpr int j = decltype(jc)::value;
    if constexpr (is_f32_add_permute(CL::c.nodes[j])) base += a.n[j].R * a.n[j].C;
  });
  return base;
}

// =========================================================================================
template <class CL, bool VEC>
__global__ void __launch_bounds__(kBlock) k_stream(const __grid_constant__ Args<CL::c.n> a) {
  constexpr int N = CL::c.n;
  constexpr int W = VEC ? 4 : 1;
  constexpr int DR = domain_rank<CL>();
  constexpr int NF = count_if<CL>(is_scalar_fold);
  constexpr int NP64 = count_if<CL>(is_f32_add_permute);
  using IX = std::conditional_t<VEC, Ix4, Ix>;
  __shared__ uint32_t red[kBlock / 32];
  __shared__ bool last_block;

  uint32_t acc[N];
  float comp[N] = {};                                    // see fold_step
  static_for<0, N>([&](auto ic) {
    constexpr int i = decltype(ic)::value;
    constexpr CNode nd = CL::c.nodes[i];
    if constexpr (is_scalar_fold(nd)) acc[i] = identity_of<nd.fn, nd.dtype>();
  });
  double* acc64_base = reinterpret_cast<double*>(a.scratch + stream_acc64_off(NF, a.grid));

  // Rank 1: a grid-stride walk over chunks.  Rank 2: a grid-stride walk over tiles of
  // kStreamTileRows rows x 32 chunks, one warp per row segment (512 contiguous bytes), so that
  // the rows a stencil reads above and below its own are rows the same block touches anyway.
  // (Measured on the 8192^2 Jacobi iteration this walk and a plain row-major walk run at the
  // same speed, 0.103 ms: the kernel is held by the load/store unit, not by L2.)
  const uint32_t per_row = (uint32_t)a.C / W;
  const uint32_t tiles_x = (per_row + 31) / 32;
  // A rank-1 cluster with a reversal reads arrays at i and at n-1-i.  Walked in mirrored pairs (a thread takes
  // chunk q and then chunk per_row-1-q) both positions need the same two chunks of such an array, and the second
  // evaluation finds them in L1: an array longer than the L2 crosses DRAM once instead of twice.
  constexpr bool MIRROR = DR <= 1 && has_reversal<CL>();
  const uint32_t half = (per_row + 1) / 2;
  const uint32_t trips = DR <= 1 ? ((MIRROR ? half : per_row) + kBlock - 1) / kBlock
                                 : tiles_x * (((uint32_t)a.R + kStreamTileRows - 1) / kStreamTileRows);
  for (uint32_t t = blockIdx.x; t < trips; t += gridDim.x) {
   for (int side = 0; side < (MIRROR ? 2 : 1); ++side) {
    IX ix;
    bool live;
    if constexpr (DR <= 1) {
      uint32_t q = t * kBlock + threadIdx.x;
      live = q < (MIRROR ? half : per_row);
      if (MIRROR && side == 1) {
        live = live && per_row - 1 - q != q;               // the middle chunk of an odd count has no partner
        q = per_row - 1 - q;
      }
      ix.r = 0;
      ix.c = (int)(q * W);
    } else {
      const uint32_t ty = t / tiles_x, tx = t - ty * tiles_x;
      const uint32_t r = ty * kStreamTileRows + (threadIdx.x >> 5), q = tx * 32 + (threadIdx.x & 31);
      live = r < (uint32_t)a.R && q < per_row;
      ix.r = (int)r;
      ix.c = (int)(q * W);
    }
    if (!live) continue;
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_store_root(nd)) {
        st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), a.n[i].C, ix, eval<CL, i>(a, ix));
      } else if constexpr (is_scalar_fold(nd)) {
        const auto v = eval<CL, nd.in[0]>(a, ix);
        if constexpr (VEC) {
#pragma unroll
          for (int j = 0; j < 4; ++j) fold_step<nd.fn, nd.dtype>(acc[i], comp[i], v.v[j]);
        } else {
          fold_step<nd.fn, nd.dtype>(acc[i], comp[i], v);
        }
      } else if constexpr (is_permute_root(nd)) {
        const auto k = eval<CL, nd.in[1]>(a, ix);
        const auto x = eval<CL, nd.in[2]>(a, ix);
        uint32_t* out = reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr));
        const uint32_t bins = (uint32_t)(a.n[i].R * a.n[i].C);
        double* acc64 = acc64_of<CL, i>(a, acc64_base);
        if constexpr (VEC) {
#pragma unroll
          for (int j = 0; j < 4; ++j) permute_update<nd.fn, nd.dtype>(out, acc64, bins, k.v[j], x.v[j], a.status);
        } else {
          permute_update<nd.fn, nd.dtype>(out, acc64, bins, k, x, a.status);
        }
      }
    });
   }
  }

  if constexpr (NF > 0 || NP64 > 0) {
    // partial of every scalar fold, then the block that arrives last finishes the job
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_scalar_fold(nd)) {
        constexpr int ord = count_if<CL>(is_scalar_fold, i);
        const uint32_t v = block_reduce<nd.fn, nd.dtype>(acc[i], red);
        if (threadIdx.x == 0) a.scratch[stream_partials_off() + ord * a.grid + blockIdx.x] = v;
      }
    });
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last_block = atomicAdd(a.scratch, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!last_block) return;
    __threadfence();
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_scalar_fold(nd)) {
        constexpr int ord = count_if<CL>(is_scalar_fold, i);
        const volatile uint32_t* part = a.scratch + stream_partials_off() + ord * a.grid;
        uint32_t v = identity_of<nd.fn, nd.dtype>();
        for (int b = threadIdx.x; b < (int)gridDim.x; b += kBlock) v = combine<nd.fn, nd.dtype>(v, part[b]);
        v = block_reduce<nd.fn, nd.dtype>(v, red);
        if (threadIdx.x == 0) *reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)) = v;
      } else if constexpr (is_f32_add_permute(nd)) {
        const volatile double* acc64 = acc64_of<CL, i>(a, acc64_base);
        const float* defaults = reinterpret_cast<const float*>(a.n[nd.in[0]].ptr);
        float* out = reinterpret_cast<float*>(const_cast<void*>(a.n[i].ptr));
        const int bins = a.n[i].R * a.n[i].C;
        for (int b = threadIdx.x; b < bins; b += kBlock) out[b] = (float)((double)defaults[b] + acc64[b]);
      }
    });
  }
}

// =========================================================================================
template <class CL, bool VEC>
__global__ void __launch_bounds__(kBlock) k_rowfold(const __grid_constant__ Args<CL::c.n> a) {
  constexpr int N = CL::c.n;
  constexpr int W = VEC ? 4 : 1;
  using IX = std::conditional_t<VEC, Ix4, Ix>;
  __shared__ uint32_t red[kBlock / 32];
  for (int r = blockIdx.x; r < a.R; r += gridDim.x) {
    uint32_t acc[N];
    float comp[N] = {};                                  // see fold_step
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_row_fold(nd)) acc[i] = identity_of<nd.fn, nd.dtype>();
    });
    for (int c = threadIdx.x * W; c < a.C; c += kBlock * W) {
      const IX ix{r, c};
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_store_root(nd)) {
          st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), a.n[i].C, ix, eval<CL, i>(a, ix));
        } else if constexpr (is_row_fold(nd)) {
          const auto v = eval<CL, nd.in[0]>(a, ix);
          if constexpr (VEC) {
#pragma unroll
            for (int j = 0; j < 4; ++j) fold_step<nd.fn, nd.dtype>(acc[i], comp[i], v.v[j]);
          } else {
            fold_step<nd.fn, nd.dtype>(acc[i], comp[i], v);
          }
        }
      });
    }
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_row_fold(nd)) {
        const uint32_t v = block_reduce<nd.fn, nd.dtype>(acc[i], red);
        if (threadIdx.x == 0) reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[r] = v;
      }
    });
  }
}

// =========================================================================================
// k_rowfold_then: row folds whose results are consumed, row for row, by element-wise members of
// the same cluster (a map of a fold: normalisations, the paper's greedyBottomUpBad).  Pulled
// through, each output element would walk its whole row in one thread; here a block reduces
// the rows of all such folds together, one thread then evaluates the consumers of that row with
// the reduced values in place of the folds (IxAfter), and folds that are manifest are stored on
// the way.
struct IxAfter { int r, c; const uint32_t* folded; };    // element c of a rank-1 result; folded[k]: value of the k-th fold at c
template <> struct width_of<IxAfter> { static constexpr int value = 1; };
__device__ __forceinline__ Ix lane(const IxAfter& i, int) { return Ix{i.r, i.c}; }
__device__ __forceinline__ uint32_t ld(const uint32_t* p, int C, const IxAfter& i) { return ld1(p, C, Ix{i.r, i.c}); }
template <int F, int P0 = kRunTime, int P1 = kRunTime>
__device__ __forceinline__ auto map_index(const IxAfter& i, const NodeArg& self, const NodeArg& src) {
  if constexpr (F == ACC_IDX_IDENTITY) return i;
  else return map1<F>(Ix{i.r, i.c}, self, src);            // behind any other map the folds are pulled through again
}

constexpr bool is_inner_row_fold(const CNode& n) { return n.member && n.kind == ACC_FOLD && n.rank == 1; }
template <class CL> constexpr int fold_slot(int i) {
  int k = 0;
  for (int j = 0; j < i; ++j) k += is_inner_row_fold(CL::c.nodes[j]) ? 1 : 0;
  return k;
}
template <class CL, int I> struct reads_staged<CL, I, IxAfter> { static constexpr bool value = is_inner_row_fold(CL::c.nodes[I]); };
template <class CL, int I, class A>
__device__ __forceinline__ uint32_t ld_staged(const A&, const IxAfter& ix) { return ix.folded[fold_slot<CL>(I)]; }

// does node i depend on a fold member (through members)?
template <class CL> constexpr bool below_fold(int i) {
  const CNode& n = CL::c.nodes[i];
  if (!n.member) return false;
  if (n.kind == ACC_FOLD) return true;
  for (int s = 0; s < n.nin; ++s)
    if (below_fold<CL>(n.in[s])) return true;
  return false;
}
// element-wise members on top of row folds: rank-1 maps / zipWiths / generates of rank-1 arrays and folds
template <class CL> constexpr bool only_elementwise_above_folds(int i) {
  const CNode& n = CL::c.nodes[i];
  if (!n.member) return n.rank <= 1;
  if (n.kind == ACC_FOLD) return true;
  if (n.rank != 1 || (n.kind != ACC_MAP && n.kind != ACC_ZIPWITH && n.kind != ACC_GENERATE)) return false;
  for (int s = 0; s < n.narr; ++s)
    if (!only_elementwise_above_folds<CL>(n.in[s])) return false;
  return true;
}
template <class CL> constexpr bool rowfold_then_eligible() {
  int inner = 0, consumers = 0;
  for (int i = 0; i < CL::c.n; ++i) {
    const CNode& n = CL::c.nodes[i];
    if (!n.member) continue;
    if (n.kind == ACC_FOLD) {
      if (n.rank != 1 || CL::c.nodes[n.in[0]].rank != 2 || below_fold<CL>(n.in[0])) return false;
      ++inner;
    } else if (n.kind == ACC_SCANL || n.kind == ACC_SCANR || n.kind == ACC_PERMUTE || n.kind == ACC_FOLDSEG) {
      return false;
    } else if (is_store_root(n)) {
      if (below_fold<CL>(i)) {
        if (!only_elementwise_above_folds<CL>(i)) return false;
        ++consumers;
      } else {
        return false;                                      // a root beside the folds: another skeleton's job
      }
    }
  }
  return inner >= 1 && inner <= 4 && consumers >= 1;
}

template <class CL, bool VEC>
__global__ void __launch_bounds__(kBlock) k_rowfold_then(const __grid_constant__ Args<CL::c.n> a) {
  constexpr int N = CL::c.n;
  constexpr int W = VEC ? 4 : 1;
  constexpr int NFOLD = count_if<CL>(is_inner_row_fold);
  using IX = std::conditional_t<VEC, Ix4, Ix>;
  __shared__ uint32_t red[kBlock / 32];
  __shared__ uint32_t folded[NFOLD];
  for (int r = blockIdx.x; r < a.R; r += gridDim.x) {     // a.R x a.C: the shape the folds reduce
    uint32_t acc[N];
    float comp[N] = {};                                  // see fold_step
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_inner_row_fold(nd)) acc[i] = identity_of<nd.fn, nd.dtype>();
    });
    for (int c = threadIdx.x * W; c < a.C; c += kBlock * W) {
      const IX ix{r, c};
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr CNode nd = CL::c.nodes[i];
        if constexpr (is_inner_row_fold(nd)) {
          const auto v = eval<CL, nd.in[0]>(a, ix);
          if constexpr (VEC) {
#pragma unroll
            for (int j = 0; j < 4; ++j) fold_step<nd.fn, nd.dtype>(acc[i], comp[i], v.v[j]);
          } else {
            fold_step<nd.fn, nd.dtype>(acc[i], comp[i], v);
          }
        }
      });
    }
    static_for<0, N>([&](auto ic) {
      constexpr int i = decltype(ic)::value;
      constexpr CNode nd = CL::c.nodes[i];
      if constexpr (is_inner_row_fold(nd)) {
        const uint32_t v = block_reduce<nd.fn, nd.dtype>(acc[i], red);
        if (threadIdx.x == 0) {
          folded[fold_slot<CL>(i)] = v;
          if constexpr (nd.manifest) reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[r] = v;
        }
      }
    });
    if (threadIdx.x == 0) {
      const IxAfter ix{0, r, folded};
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        if constexpr (is_store_root(CL::c.nodes[i]))
          reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr))[r] = eval<CL, i>(a, ix);
      });
    }
    __syncthreads();                                       // `folded` is rewritten for the next row
  }
}

// =========================================================================================
// Scratch layout of k_scan: word [0] ticket; from byte 16 one 64-bit tile state per tile:
// (value << 32) | low, the two lowest bits of `low` being the flag: 0 = nothing yet, 1 = the tile's
// own total, 2 = inclusive prefix.  The prefix of an fp32 sum is carried as two floats, hi in `value`
// and lo (its two lowest mantissa bits dropped) in the rest of `low`: the chain of tile prefixes is a
// running sum over up to 2^31 / 4096 tiles, and in plain fp32 its rounding errors pile up on inputs
// where they do not cancel.
// Tile shape: 256 threads x 16 elements where the scanned operand gathers (the random reads bound the
// kernel and small tiles keep more of them in flight), 512 threads x 32 elements where it streams (per
// tile the ticket, three barriers and the look-back are then paid once per 64 KB: 0.156 against 0.209 ms
// for 2^26 floats, with no change for the gathering cluster).
template <class CL> constexpr bool scan_gathers() {
  for (int i = 0; i < CL::c.n; ++i)
    if (CL::c.nodes[i].member && CL::c.nodes[i].kind == ACC_GATHER) return true;
  return false;
}
template <class CL> constexpr int scan_block() { return scan_gathers<CL>() ? 256 : 512; }
template <class CL> constexpr int scan_rows() { return scan_gathers<CL>() ? 4 : 8; }     // 128-bit chunks per thread
constexpr uint32_t kFlagAggregate = 1, kFlagPrefix = 2;

__device__ __forceinline__ uint64_t ld_state(const uint64_t* p) {
  return *reinterpret_cast<const volatile uint64_t*>(p);
}
__device__ __forceinline__ void st_state(uint64_t* p, uint32_t flag, uint32_t v, uint32_t low = 0u) {
  *reinterpret_cast<volatile uint64_t*>(p) = ((uint64_t)v << 32) | (low & ~3u) | flag;
}
__device__ __forceinline__ uint32_t flag_of(uint64_t s) { return (uint32_t)s & 3u; }
__device__ __forceinline__ uint32_t value_of(uint64_t s) { return (uint32_t)(s >> 32); }
// hi + lo of a state of an fp32 sum (lo is zero for a tile's own total)
__device__ __forceinline__ double wide_of(uint64_t s) {
  return (double)__uint_as_float(value_of(s)) + (double)__uint_as_float((uint32_t)s & ~3u);
}
__device__ __forceinline__ void st_wide(uint64_t* p, double prefix) {
  const float hi = (float)prefix;
  const float lo = isfinite(hi) ? (float)(prefix - (double)hi) : 0.0f;     // an overflowed sum stays infinite
  st_state(p, kFlagPrefix, __float_as_uint(hi), __float_as_uint(lo));
}

// stores at a descending chunk: the lanes go back into ascending memory order
__device__ __forceinline__ void st(uint32_t* p, int C, const IxR4& i, const V4& v) {
  *reinterpret_cast<uint4*>(p + (i.r * C + i.c - 3)) = make_uint4(v.v[3], v.v[2], v.v[1], v.v[0]);
}

// Element-wise members that consume the scan inside its cluster are evaluated where the scanned values
// are final, at an index that carries them: IxSc<B> is the plain index B plus the scan's values there,
// and the scan member reads as those values.  Only index-preserving paths (array operands of map and
// zipWith, the index operand of a gather) may lead from such a member to the scan; behind an index map
// the values would be lost, and no such cluster is instantiated.
template <class B> struct IxSc : B { val_of<B> sv; };
template <class B> struct width_of<IxSc<B>> { static constexpr int value = width_of<B>::value; };
template <class CL, int I, class B> struct reads_staged<CL, I, IxSc<B>> { static constexpr bool value = I == first_scan<CL>(); };
template <class CL, int I, class A, class B>
__device__ __forceinline__ val_of<B> ld_staged(const A&, const IxSc<B>& ix) { return ix.sv; }

// A gather whose values were brought in by an earlier launch (slabgather.cuh): the index carries them, and the
// gather member reads as those values.  As with IxSc, only index-preserving paths may lead to that member.
template <class B> struct IxGv : B { val_of<B> gv; };
template <class B> struct width_of<IxGv<B>> { static constexpr int value = width_of<B>::value; };
template <class CL> constexpr int the_gather() {
  int g = -1;
  for (int i = 0; i < CL::c.n; ++i)
    if (CL::c.nodes[i].member && CL::c.nodes[i].kind == ACC_GATHER) g = g < 0 ? i : -2;
  return g < 0 ? -1 : g;
}
template <class CL, int I, class B> struct reads_staged<CL, I, IxGv<B>> { static constexpr bool value = I == the_gather<CL>(); };
template <class CL, int I, class A, class B>
__device__ __forceinline__ val_of<B> ld_staged(const A&, const IxGv<B>& ix) { return ix.gv; }

// What the merging scan needs beside its cluster arguments (see slabgather.cuh); unused by the plain scan.
struct SlabIn {
  const uint32_t* codes = nullptr;     // per element of a full warp tile: which slab its gathered index fell in (2 bits; a word per lane)
  const uint32_t* counts = nullptr;    // per full warp tile: how many of its elements fell in slabs 0, 1, 2 (10 bits each)
  int full_tiles = 0;                  // warp tiles of kSlabWarpTile elements that the earlier launches covered
  const uint32_t* local = nullptr;     // how many of the `sampled` warp tiles that k_slab_probe looked at hold indices close together
  uint32_t sampled = 0;
};
// Whether the probe found the gather's indices local (most sampled warp tiles span few elements of the source): then
// the gather reads whole sectors and lines as it is, the slab passes stand back and their kernels return at once.
__device__ __forceinline__ bool slab_passes_stand_back(const SlabIn& slab) { return 2u * __ldg(slab.local) > slab.sampled; }
constexpr int kSlabWarpTile = 512;

// Whether `leaf` (an array from outside the cluster) is read by member i at i's own index: through array operands
// of maps and zipWiths only.
constexpr bool reads_in_place(const CCluster& c, int i, int leaf) {
  if (i == leaf) return true;
  const CNode& n = c.nodes[i];
  if (!n.member || (n.kind != ACC_MAP && n.kind != ACC_ZIPWITH)) return false;
  for (int k = 0; k < n.narr; ++k)
    if (reads_in_place(c, n.in[k], leaf)) return true;
  return false;
}

// The gathered values of warp tile `wt` (kSlabWarpTile elements, grouped by slab where `staged` holds them) in element
// order: lane's elements (j * 32 + lane) * 4 .. + 3 in gathered[j].  The stable counting sort of k_slab_partition is undone
// from the slab codes and the group sizes, through `stage` (kSlabWarpTile words of shared memory that the warp owns).
template <int ROWS>
__device__ __forceinline__ void unpermute_warp_tile(const uint32_t* staged_array, const SlabIn& slab, int wt, uint32_t* stage, V4 (&gathered)[ROWS]) {
  static_assert(ROWS * 128 == kSlabWarpTile, "a lane holds 16 elements of the warp tile");
  const int lane = threadIdx.x & 31;
  const uint32_t code = __ldg(slab.codes + (size_t)wt * 32 + lane), cnt3 = __ldg(slab.counts + wt);
  const uint32_t* staged = staged_array + (size_t)wt * kSlabWarpTile;
  uint4 st[ROWS];
#pragma unroll
  for (int j = 0; j < ROWS; ++j) st[j] = *reinterpret_cast<const uint4*>(staged + (j * 32 + lane) * 4);
  const uint32_t lo1 = code & 0x55555555u, hi1 = (code >> 1) & 0x55555555u;
  const uint32_t n3 = __popc(lo1 & hi1), n2 = __popc(hi1 & ~lo1), n1 = __popc(lo1 & ~hi1);
  const uint32_t c01 = (16u - n1 - n2 - n3) | (n1 << 16), c23 = n2 | (n3 << 16);     // this lane's elements per slab
  uint32_t i01 = c01, i23 = c23;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t u0 = __shfl_up_sync(0xFFFFFFFFu, i01, o), u1 = __shfl_up_sync(0xFFFFFFFFu, i23, o);
    if (lane >= o) { i01 += u0; i23 += u1; }
  }
  const uint32_t t0 = cnt3 & 1023u, t1 = (cnt3 >> 10) & 1023u, t2 = (cnt3 >> 20) & 1023u;
  uint32_t a01 = (i01 - c01) + (t0 << 16);                             // next position in the lists of slabs 0 | 1
  uint32_t a23 = (i23 - c23) + (t0 + t1) + ((t0 + t1 + t2) << 16);     // ... of slabs 2 | 3
  __syncwarp();
#pragma unroll
  for (int j = 0; j < ROWS; ++j) *reinterpret_cast<uint4*>(stage + (j * 32 + lane) * 4) = st[j];
  __syncwarp();
#pragma unroll
  for (int j = 0; j < ROWS; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t sl = (code >> (2 * (4 * j + e))) & 3u;
      const uint32_t sh = 16 * (sl & 1);
      gathered[j].v[e] = stage[((sl < 2 ? a01 : a23) >> sh) & (kSlabWarpTile - 1)];
      if (sl < 2) a01 += 1u << sh; else a23 += 1u << sh;
    }
}

// Whether member i needs the value of scan s (through any chain of operands inside the cluster).
constexpr bool needs_scan(const CCluster& c, int i, int s) {
  const CNode& n = c.nodes[i];
  if (!n.member) return false;
  for (int k = 0; k < n.nin; ++k)
    if (n.in[k] == s || needs_scan(c, n.in[k], s)) return true;
  return false;
}

// What one tile of a scan takes, in the three parts that the kernels below put together: a warp's share of the tile
// evaluated and scanned in registers, the look-back of one warp for the tile's prefix, and the final values stored.
// Rows of a rank-2 array are scanned independently: a row is cut into tiles of its own, the
// look-back of a tile stops at the first tile of its row.  A right-to-left scan walks its row
// from the far end: position p of the walk is element C-1-p of the row.
template <class CL, bool VEC, bool SLAB>
struct ScanTile {
  static constexpr int N = CL::c.n;
  static constexpr int W = VEC ? 4 : 1;
  static constexpr int BLOCK = scan_block<CL>();
  static constexpr int ROWS = VEC ? scan_rows<CL>() : scan_rows<CL>() * 4;   // as many elements per thread either way
  static constexpr int TILE = BLOCK * scan_rows<CL>() * 4;
  static constexpr int PART = TILE / (BLOCK / 32);         // elements of a tile that one warp takes
  static constexpr int S = first_scan<CL>();
  static_assert(S >= 0, "k_scan needs a scan member");
  static constexpr CNode sn = CL::c.nodes[S];
  static constexpr int FN = sn.fn, DT = sn.dtype;
  static constexpr bool REV = sn.kind == ACC_SCANR;
  static constexpr bool EXCL = sn.p0 == 1;                 // seeded and exclusive: element k leaves itself out
  static constexpr bool WIDE = FN == ACC_FN_ADD && DT == ACC_F32;
  using IX = std::conditional_t<VEC, std::conditional_t<REV, IxR4, Ix4>, Ix>;
  static_assert(!SLAB || (VEC && PART == kSlabWarpTile && !REV), "the merging scan walks rank-1 tiles of 512-element warp tiles");

  static __device__ __forceinline__ IX index_at(int n, int row, int p) {   // walk position p (a multiple of W) of a row of n -> index
    IX ix;
    ix.r = row;
    ix.c = REV ? n - 1 - p : p;
    return ix;
  }

  // The warp's PART elements from walk position warp_base of `row` on: evaluated, stored where a root does not need
  // the scan, and scanned within the warp (val: each element's scan over the warp's part).  Returns the part's total.
  // SLAB: the gathered values of warp tile `wt` lie, grouped by slab, where the scan's results will go; they are put
  // back into element order through `stage` (kSlabWarpTile words of shared memory that this warp owns).
  static __device__ __forceinline__ uint32_t scan_part(const Args<N>& a, int row, int warp_base, int wt, const SlabIn& slab,
                                                       uint32_t* stage, uint32_t (&val)[ROWS][W]) {
    const int lane = threadIdx.x & 31;
    const int n = a.C;                                     // length of a row
    V4 gathered[SLAB ? ROWS : 1];
    bool merged = false;                                   // the same for a whole warp
    if constexpr (SLAB) {
      if (wt < slab.full_tiles) {
        merged = true;
        unpermute_warp_tile<ROWS>(reinterpret_cast<const uint32_t*>(a.n[S].ptr), slab, wt, stage, gathered);
      }
    }
    uint32_t carry = identity_of<FN, DT>();                // running total of this warp's earlier rows
#pragma unroll
    for (int j = 0; j < ROWS; ++j) {
      const int c = warp_base + (j * 32 + lane) * W;
      const bool live = c < n;
      if (live) {
        const IX ix = index_at(n, row, c);
        val_of<IX> v;
        if constexpr (SLAB) {
          if (merged) {
            IxGv<IX> with;
            static_cast<IX&>(with) = ix;
            with.gv = gathered[j];
            v = eval<CL, sn.in[0]>(a, with);
          } else {
            v = eval<CL, sn.in[0]>(a, ix);
          }
        } else {
          v = eval<CL, sn.in[0]>(a, ix);
        }
        if constexpr (VEC) {
#pragma unroll
          for (int e = 0; e < 4; ++e) val[j][e] = v.v[e];
        } else {
          val[j][0] = v;
        }
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          if constexpr (is_store_root(CL::c.nodes[i]) && !needs_scan(CL::c, i, S))
            st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), a.n[i].C, ix, eval<CL, i>(a, ix));
        });
      } else {
#pragma unroll
        for (int e = 0; e < W; ++e) val[j][e] = identity_of<FN, DT>();
      }
      // inclusive scan inside the thread, then across the warp
#pragma unroll
      for (int e = 1; e < W; ++e) val[j][e] = combine<FN, DT>(val[j][e - 1], val[j][e]);
      uint32_t incl = val[j][W - 1];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl = combine<FN, DT>(t, incl);
      }
      uint32_t excl = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
      if (lane == 0) excl = identity_of<FN, DT>();
      excl = combine<FN, DT>(carry, excl);
      if constexpr (EXCL) {
        // what came before each element: the thread's own earlier elements on top of `excl`
#pragma unroll
        for (int e = W - 1; e >= 1; --e) val[j][e] = combine<FN, DT>(excl, val[j][e - 1]);
        val[j][0] = excl;
      } else {
#pragma unroll
        for (int e = 0; e < W; ++e) val[j][e] = combine<FN, DT>(excl, val[j][e]);
      }
      carry = combine<FN, DT>(carry, __shfl_sync(0xFFFFFFFFu, incl, 31));
    }
    return carry;
  }

  // One warp publishes the tile's total, looks back over the tiles of its row before it and publishes the tile's
  // inclusive prefix.  Returns (in every lane) what came before the tile.  A wait that runs out sets the status flag.
  static __device__ __forceinline__ uint32_t look_back(const Args<N>& a, int tile, int in_row, uint32_t tile_total) {
    const int lane = threadIdx.x & 31;
    uint64_t* states = reinterpret_cast<uint64_t*>(a.scratch + 4);
    uint32_t exclusive = identity_of<FN, DT>();
    if (in_row == 0) {
      if (lane == 0) st_state(states + tile, kFlagPrefix, tile_total);
      return exclusive;
    }
    if (lane == 0) st_state(states + tile, kFlagAggregate, tile_total);
    int look = in_row - 1;                                 // tiles of this row before this one
    uint32_t spins = 0;
    bool gave_up = false;
    double wide = 0.0;                                     // WIDE: the sum of the tiles before this one
    for (;;) {
      const int idx = look - lane;
      const uint64_t* at = states + (tile - in_row) + idx;
      uint64_t s = idx >= 0 ? ld_state(at) : ((uint64_t)identity_of<FN, DT>() << 32) | kFlagPrefix;
      while (__any_sync(0xFFFFFFFFu, flag_of(s) == 0)) {
        if (++spins > a.spin_limit) { gave_up = true; break; }
        __nanosleep(20);
        if (idx >= 0) s = ld_state(at);
      }
      if (gave_up) break;
      const unsigned done = __ballot_sync(0xFFFFFFFFu, flag_of(s) == kFlagPrefix);
      const int stop = done ? __ffs(done) - 1 : 31;
      if constexpr (WIDE) {
        double part = lane <= stop ? wide_of(s) : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
        wide += part;
      } else {
        uint32_t part = lane <= stop ? value_of(s) : identity_of<FN, DT>();
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part = combine<FN, DT>(part, __shfl_xor_sync(0xFFFFFFFFu, part, o));
        exclusive = combine<FN, DT>(part, exclusive);
      }
      if (done) break;
      look -= 32;
    }
    if (gave_up && lane == 0) atomicOr(a.status, kStatusTimeout);
    if constexpr (WIDE) {
      exclusive = u_((float)wide);
      if (lane == 0) st_wide(states + tile, wide + (double)f_(tile_total));
    } else {
      if (lane == 0) st_state(states + tile, kFlagPrefix, combine<FN, DT>(exclusive, tile_total));
    }
    return exclusive;
  }

  // The warp's part once `before` (everything of the row ahead of the part) is known: the scan is stored, and so is
  // every root that reads it.
  static __device__ __forceinline__ void finish_part(const Args<N>& a, int row, int warp_base, uint32_t before, const uint32_t (&val)[ROWS][W]) {
    const int lane = threadIdx.x & 31;
    const int n = a.C;
    uint32_t base = before;
    if constexpr (EXCL) base = combine<FN, DT>(DT == ACC_F32 ? u_(a.n[S].fp0) : (uint32_t)a.n[S].ip0, base);   // the seed comes first
    uint32_t* out = reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[S].ptr));
#pragma unroll
    for (int j = 0; j < ROWS; ++j) {
      const int c = warp_base + (j * 32 + lane) * W;
      if (c < n) {
        const IX ix = index_at(n, row, c);
        IxSc<IX> scanned;
        static_cast<IX&>(scanned) = ix;
        if constexpr (VEC) {
          scanned.sv = V4{{combine<FN, DT>(base, val[j][0]), combine<FN, DT>(base, val[j][1]),
                           combine<FN, DT>(base, val[j][2]), combine<FN, DT>(base, val[j][3])}};
        } else {
          scanned.sv = combine<FN, DT>(base, val[j][0]);
        }
        if constexpr (sn.manifest) st(out, n, ix, scanned.sv);
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          if constexpr (is_store_root(CL::c.nodes[i]) && needs_scan(CL::c, i, S))
            st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), a.n[i].C, ix, eval<CL, i>(a, scanned));
        });
      }
    }
  }

  // The lines that the warp's part from walk position warp_base of `row` on will read in place, asked into L2
  // (left-to-right scans; arrays from outside the cluster that the scanned operand reads at its own index).
  static __device__ __forceinline__ void prefetch_operands(const Args<N>& a, int row, int warp_base) {
    if constexpr (!REV) {
      const int lane = threadIdx.x & 31;
      const int n = a.C;
      static_for<0, N>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        if constexpr (!CL::c.nodes[i].member && reads_in_place(CL::c, sn.in[0], i)) {
          const char* base = reinterpret_cast<const char*>(a.n[i].ptr) + (size_t)row * n * 4;
#pragma unroll
          for (int k = 0; k < PART; k += 1024) {
            const int at = warp_base + k + lane * 32;
            if (at < n) asm volatile("prefetch.global.L2 [%0];" ::"l"(base + (size_t)at * 4));
          }
        }
      });
    }
  }

  // SLAB: the staged values and codes of warp tile `wt` are asked into L2 ahead of their use
  static __device__ __forceinline__ void prefetch_part(const Args<N>& a, int wt, const SlabIn& slab) {
    const int lane = threadIdx.x & 31;
    if (wt < slab.full_tiles) {
      const char* q = lane < 16 ? reinterpret_cast<const char*>(reinterpret_cast<const uint32_t*>(a.n[S].ptr) + (size_t)wt * kSlabWarpTile) + lane * 128
                                : reinterpret_cast<const char*>(slab.codes + (size_t)wt * 32);
      if (lane <= 16) asm volatile("prefetch.global.L2 [%0];" ::"l"(q));
    }
  }
};

// Tile after tile with the whole block in step: every warp scans its part, one warp looks back, every warp stores.
// STATIC: block b walks tiles b, b + G, b + 2G, ... of a grid of G blocks that are all resident at once (a
// cooperative launch): no ticket, whose atomic every warp of the block would otherwise wait for at the top of every
// tile (measured on a streaming scan of 2^26 floats: 28 barrier-stall cycles per issued instruction, 19 % of the
// issue slots used).  A tile's predecessors belong to the blocks before this one in the same round, or to an
// earlier round, so they are running or done.  Without that guarantee the tiles are claimed from a ticket.
template <class CL, bool VEC, bool SLAB, bool STATIC = false>
__device__ __forceinline__ void scan_tiles(const Args<CL::c.n>& a, int tiles_per_row, int n_tiles, const SlabIn& slab) {
  using T = ScanTile<CL, VEC, SLAB>;
  constexpr int BLOCK = T::BLOCK, FN = T::FN, DT = T::DT;
  __shared__ uint32_t warp_total[BLOCK / 32];
  __shared__ uint32_t tile_prefix;
  __shared__ int tile_id;
  __shared__ __align__(16) uint32_t slab_stage[SLAB ? BLOCK / 32 : 1][SLAB ? kSlabWarpTile : 1];   // read and written 128 bits at a time
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  for (int round = 0;; ++round) {
    int tile;
    if constexpr (STATIC) {
      // (no barrier here: what a round shares through shared memory is read before its second barrier or right
      // after it, and written again only behind the next round's first barrier)
      tile = (int)blockIdx.x + round * (int)gridDim.x;
    } else {
      __syncthreads();
      if (threadIdx.x == 0) tile_id = (int)atomicAdd(a.scratch, 1u);
      __syncthreads();
      tile = tile_id;
    }
    if (tile >= n_tiles) return;
    const int row = tile / tiles_per_row, in_row = tile - row * tiles_per_row;
    const int warp_base = in_row * T::TILE + warp * T::PART;

    if constexpr (STATIC) {
      // this block's next tile is known: what it reads is on its way while this tile is scanned and looked back
      // for (config-3 shape, 2^26 elements: 0.726 -> 0.704 ms for the cluster)
      const int next = tile + (int)gridDim.x;
      if constexpr (SLAB) {
        T::prefetch_part(a, next * (BLOCK / 32) + warp, slab);
      } else if (next < n_tiles) {
        const int nrow = next / tiles_per_row;
        T::prefetch_operands(a, nrow, (next - nrow * tiles_per_row) * T::TILE + warp * T::PART);
      }
    }
    uint32_t val[T::ROWS][T::W];
    const uint32_t carry = T::scan_part(a, row, warp_base, tile * (BLOCK / 32) + warp, slab, slab_stage[SLAB ? warp : 0], val);
    if (lane == 0) warp_total[warp] = carry;
    __syncthreads();
    uint32_t offset = identity_of<FN, DT>();               // total of the warps before this one
    uint32_t tile_total = identity_of<FN, DT>();
#pragma unroll
    for (int w = 0; w < BLOCK / 32; ++w) {
      const uint32_t t = warp_total[w];
      if (w < warp) offset = combine<FN, DT>(offset, t);
      tile_total = combine<FN, DT>(tile_total, t);
    }
    if (warp == 0) {
      const uint32_t exclusive = T::look_back(a, tile, in_row, tile_total);
      if (lane == 0) tile_prefix = exclusive;
    }
    __syncthreads();
    T::finish_part(a, row, warp_base, combine<FN, DT>(tile_prefix, offset), val);
  }
}

// Named barriers (ids 1..4; id 0 is __syncthreads'): `count` threads take part, arriving or waiting.
template <int ID> __device__ __forceinline__ void bar_sync_id(int count) { asm volatile("bar.sync %0, %1;" ::"n"(ID), "r"(count) : "memory"); }
template <int ID> __device__ __forceinline__ void bar_arrive_id(int count) { asm volatile("bar.arrive %0, %1;" ::"n"(ID), "r"(count) : "memory"); }
// (barrier `first` for half 0, `first + 1` for half 1, as immediates)
template <int FIRST> __device__ __forceinline__ void bar_sync(int half, int count) { if (half) bar_sync_id<FIRST + 1>(count); else bar_sync_id<FIRST>(count); }
template <int FIRST> __device__ __forceinline__ void bar_arrive(int half, int count) { if (half) bar_arrive_id<FIRST + 1>(count); else bar_arrive_id<FIRST>(count); }

// The same tiles with the look-back taken out of the block's way: BLOCK / 32 warps scan parts and one more warp does
// nothing but look back.  A scanning warp leaves its part's values in shared memory, tells the look-back warp that
// the part's total is in, goes on to its part of the block's next tile, and only then comes back for the values,
// which it finishes with what the look-back warp has found meanwhile.  Where the whole block waits for the look-back
// (scan_tiles), the blocks of a cooperative grid fall into step and an SM's blocks all wait at once.
// Round r uses half r & 1 of everything shared.  Barrier 1 + half: a part's total is in shared memory (the scanning
// warps arrive, the look-back warp waits); barrier 3 + half: what comes before each part is in shared memory (the
// look-back warp arrives, the scanning warps wait).  Every warp of a block walks the same rounds, so that each
// barrier sees BLOCK + 32 threads once a round.  Only for grids whose blocks are all resident (STATIC tiles).
template <class CL, bool VEC, bool SLAB>
__device__ __forceinline__ void scan_tiles_pipelined(const Args<CL::c.n>& a, int tiles_per_row, int n_tiles, const SlabIn& slab) {
  using T = ScanTile<CL, VEC, SLAB>;
  constexpr int BLOCK = T::BLOCK, WARPS = BLOCK / 32, FN = T::FN, DT = T::DT, ROWS = T::ROWS, W = T::W;
  static_assert(WARPS <= 32, "one lane of the look-back warp per scanning warp");
  __shared__ __align__(16) uint32_t values[2][T::TILE];    // a part's scanned values between its two visits (SLAB: first the staging area of its merge)
  __shared__ uint32_t part_total[2][WARPS];
  __shared__ uint32_t part_before[2][WARPS];               // what of the row comes before each part
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int G = (int)gridDim.x;

  if (warp == WARPS) {
    for (int round = 0;; ++round) {
      const int tile = (int)blockIdx.x + round * G;
      if (tile >= n_tiles) return;
      const int half = round & 1;
      const int row = tile / tiles_per_row, in_row = tile - row * tiles_per_row;
      bar_sync<1>(half, BLOCK + 32);
      uint32_t incl = lane < WARPS ? part_total[half][lane] : identity_of<FN, DT>();
#pragma unroll
      for (int o = 1; o < WARPS; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl = combine<FN, DT>(t, incl);
      }
      uint32_t earlier = __shfl_up_sync(0xFFFFFFFFu, incl, 1);                 // total of the parts before lane's
      if (lane == 0) earlier = identity_of<FN, DT>();
      const uint32_t tile_total = __shfl_sync(0xFFFFFFFFu, incl, WARPS - 1);
      const uint32_t exclusive = T::look_back(a, tile, in_row, tile_total);
      if (lane < WARPS) part_before[half][lane] = combine<FN, DT>(exclusive, earlier);
      bar_arrive<3>(half, BLOCK + 32);
    }
  }

  auto finish = [&](int tile, int half) {
    const int row = tile / tiles_per_row, in_row = tile - row * tiles_per_row;
    bar_sync<3>(half, BLOCK + 32);
    const uint32_t before = part_before[half][warp];
    const uint32_t* mine = values[half] + warp * T::PART;
    uint32_t val[ROWS][W];
#pragma unroll
    for (int j = 0; j < ROWS; ++j) {
      if constexpr (VEC) {
        const uint4 q = *reinterpret_cast<const uint4*>(mine + (j * 32 + lane) * 4);
        val[j][0] = q.x; val[j][1] = q.y; val[j][2] = q.z; val[j][3] = q.w;
      } else {
        val[j][0] = mine[j * 32 + lane];
      }
    }
    T::finish_part(a, row, in_row * T::TILE + warp * T::PART, before, val);
  };

  int round = 0;
  for (;; ++round) {
    const int tile = (int)blockIdx.x + round * G;
    if (tile >= n_tiles) break;
    const int half = round & 1;
    const int row = tile / tiles_per_row, in_row = tile - row * tiles_per_row;
    uint32_t* mine = values[half] + warp * T::PART;
    if constexpr (SLAB) {
      T::prefetch_part(a, (tile + G) * WARPS + warp, slab);
    } else if (tile + G < n_tiles) {
      const int nrow = (tile + G) / tiles_per_row;
      T::prefetch_operands(a, nrow, (tile + G - nrow * tiles_per_row) * T::TILE + warp * T::PART);
    }
    {
      uint32_t val[ROWS][W];
      const uint32_t total = T::scan_part(a, row, in_row * T::TILE + warp * T::PART, tile * WARPS + warp, slab, mine, val);
      __syncwarp();                                        // (SLAB: every lane has taken its merged values out of `mine`)
#pragma unroll
      for (int j = 0; j < ROWS; ++j) {
        if constexpr (VEC) *reinterpret_cast<uint4*>(mine + (j * 32 + lane) * 4) = make_uint4(val[j][0], val[j][1], val[j][2], val[j][3]);
        else mine[j * 32 + lane] = val[j][0];
      }
      if (lane == 0) part_total[half][warp] = total;
    }
    bar_arrive<1>(half, BLOCK + 32);
    if (round > 0) finish(tile - G, half ^ 1);
  }
  if (round > 0) finish((int)blockIdx.x + (round - 1) * G, (round - 1) & 1);
}

template <class CL, bool VEC, bool STATIC = false>
__global__ void __launch_bounds__(scan_block<CL>()) k_scan(const __grid_constant__ Args<CL::c.n> a, int tiles_per_row, int n_tiles) {
  scan_tiles<CL, VEC, false, STATIC>(a, tiles_per_row, n_tiles, SlabIn{});
}

// (a tile's values stay in shared memory twice over: only for tiles of at most 16 KB)
template <class CL> constexpr bool scan_pipelines() { return scan_block<CL>() * scan_rows<CL>() * 4 <= 4096; }
template <class CL, bool VEC>
__global__ void __launch_bounds__(scan_block<CL>() + 32) k_scan_pipelined(const __grid_constant__ Args<CL::c.n> a, int tiles_per_row, int n_tiles) {
  if constexpr (scan_pipelines<CL>()) scan_tiles_pipelined<CL, VEC, false>(a, tiles_per_row, n_tiles, SlabIn{});
}

}  // namespace dev
}  // namespace acc
