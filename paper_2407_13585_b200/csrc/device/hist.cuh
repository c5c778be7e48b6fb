// k_hist: the skeleton for a cluster whose permute is an fp32 '+' scatter into few enough
// bins to keep them on chip.
//
// Measured on B200 (2^27 Zipf-skewed keys): shared-memory integer atomics sustain about
// 1000 G updates/s, fp32 shared-memory atomics about 56 G/s (they retry on every collision,
// and a hot bin collides all the time), atomics into a partner CTA's shared memory 140 G/s.
// So the bins are 32-bit *integers* in the CTA's own shared memory:
//
//  * a value x is added as the integer x * 2^S when that product is an integer of magnitude
//    below `cap` -- exact, one fire-and-forget native atomic.  `cap` is 2^31 divided by the
//    number of elements the CTA can meet, so a bin cannot overflow; S is picked per CTA from
//    the largest magnitude among the first elements it sees;
//  * any other value (not a multiple of 2^-S, too large, not finite) is added to the global
//    fp64 accumulator of its bin directly -- exact as well, slower;
//  * at the end every CTA adds its bins into the fp64 accumulators, and the block that
//    finishes last turns those into the fp32 result on top of the defaults.
//
// Every partial sum is exact, so the result is the fp32 rounding of the exact fp64-combined
// sum whatever the order of arrival.
//
// Bins beyond one CTA's shared memory: up to kHistOverflowBins more live in a private slice
// of global memory per CTA (integer atomics again; private, so a hot bin is not shared
// between SMs).  Beyond that a group of G = 2, 4 or 8 neighbouring CTAs splits the bins:
// all CTAs of a group walk the same elements (the later readers hit L2) and each updates
// only the bins it owns; store roots and whole-array folds of an element are handled by one
// CTA of the group.
#pragma once
#include "skeletons.cuh"

namespace acc {
namespace dev {

constexpr int kHistBlock = 1024;
constexpr int kHistMaxBinsPerCta = 56 * 1024;   // 224 KiB of 32-bit bins per CTA
constexpr int kHistOverflowBins = 16 * 1024;    // further bins kept per CTA in global memory
constexpr int kHistUnroll = 2;                  // independent chunks in flight per thread (4 measured no faster)
constexpr int kHistAhead = 2;                   // trips between asking L2 for a chunk and reading it

struct HistPlan {
  int group;        // CTAs that split the bins
  int per_cta;      // bins in each CTA's shared memory
  int shift;        // log2(per_cta) when it is a power of two and group > 1, else -1
  int overflow;     // bins per CTA kept in global memory (group == 1 only)
};

// How the bins are laid out, or false when they do not fit eight CTAs.
inline bool hist_plan(int64_t bins, int sms, HistPlan& p) {
  p = HistPlan{1, 0, -1, 0};
  if (bins <= 0) return false;
  if (bins <= kHistMaxBinsPerCta + kHistOverflowBins) {
    p.per_cta = (int)std::min<int64_t>(bins, kHistMaxBinsPerCta);
    p.overflow = (int)(bins - p.per_cta);
    return true;
  }
  while (p.group <= 8 && (bins + p.group - 1) / p.group > kHistMaxBinsPerCta) p.group *= 2;
  if (p.group > 8 || p.group > sms) return false;
  p.per_cta = (int)((bins + p.group - 1) / p.group);
  if ((p.per_cta & (p.per_cta - 1)) == 0)
    for (p.shift = 0; (1 << p.shift) < p.per_cta; ++p.shift) {}
  return true;
}

// Fire-and-forget integer add on global memory (no value comes back, so nothing waits for it).
__device__ __forceinline__ void red_add_global(int* p, int v) {
  asm volatile("red.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Adds v to bin k: bins below `per_cta` are words of shared memory from `bins_addr`, the others
// words of global memory from `rest` (which already points per_cta words before the first of
// them).  One comparison and two predicated fire-and-forget adds, no branch.
__device__ __forceinline__ void red_add_bin(uint32_t k, uint32_t per_cta, uint32_t bins_addr, const int* rest, int v) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .u32 sa;\n\t.reg .u64 ga;\n\t"
      "setp.lt.u32 p, %0, %1;\n\t"
      "mad.lo.u32 sa, %0, 4, %2;\n\t"
      "mad.wide.u32 ga, %0, 4, %3;\n\t"
      "@p red.shared.add.s32 [sa], %4;\n\t"
      "@!p red.global.add.s32 [ga], %4;\n\t}"
      ::"r"(k), "r"(per_cta), "r"(bins_addr), "l"(rest), "r"(v) : "memory");
}
__device__ __forceinline__ void red_add_global(double* p, double v) {
  asm volatile("red.global.add.f64 [%0], %1;" ::"l"(p), "d"(v) : "memory");
}

// Whether member I can only take integer values in [0, iparam[0]), known from its function alone
// (then a scatter of it needs no per-value test of what the integer bins can hold).
template <class CL> constexpr bool yields_small_integers(int i) {
  const CNode& n = CL::c.nodes[i];
  return n.member && n.kind == ACC_GENERATE && n.dtype == ACC_F32 && n.fn == ACC_FN_IMOD_TO_F32;
}

template <class CL> constexpr int the_f32_add_permute() {
  for (int i = 0; i < CL::c.n; ++i)
    if (is_f32_add_permute(CL::c.nodes[i])) return i;
  return -1;
}

template <class CL, bool VEC>
__global__ void __launch_bounds__(kHistBlock, 1)
k_hist(const __grid_constant__ Args<CL::c.n> a, const HistPlan plan, int* overflow_base) {
  constexpr int N = CL::c.n;
  constexpr int W = VEC ? 4 : 1;
  constexpr int U = kHistUnroll;
  constexpr int DR = domain_rank<CL>();
  constexpr int NF = count_if<CL>(is_scalar_fold);
  constexpr int P = the_f32_add_permute<CL>();
  static_assert(P >= 0, "k_hist needs an fp32 '+' permute");
  constexpr CNode pn = CL::c.nodes[P];
  using IX = std::conditional_t<VEC, Ix4, Ix>;
  using VAL = val_of<IX>;
  extern __shared__ int bins_smem[];
  __shared__ uint32_t red[kHistBlock / 32];
  __shared__ bool last_block;
  __shared__ float sample_max;

  const int per_cta = plan.per_cta;
  const uint32_t group = (uint32_t)plan.group;
  const uint32_t rank = blockIdx.x % group;                    // which slice of the bins this CTA owns
  const uint32_t team = blockIdx.x / group;                    // which share of the elements its group walks
  const uint32_t n_teams = gridDim.x / group;
  int* const spill = overflow_base + (size_t)blockIdx.x * plan.overflow;   // zeroed by the host with the scratch
  for (int i = threadIdx.x; i < per_cta; i += kHistBlock) bins_smem[i] = 0;

  uint32_t acc[N];
  float comp[N] = {};                                          // see fold_step
  static_for<0, N>([&](auto ic) {
    constexpr int i = decltype(ic)::value;
    constexpr CNode nd = CL::c.nodes[i];
    if constexpr (is_scalar_fold(nd)) acc[i] = identity_of<nd.fn, nd.dtype>();
  });
  const uint32_t n_bins = (uint32_t)(a.n[P].R * a.n[P].C);
  const uint32_t per_row = (uint32_t)a.C / W;
  const uint32_t total = (uint32_t)a.R * per_row;
  const uint32_t stride = n_teams * kHistBlock;
  double* acc64 = reinterpret_cast<double*>(a.scratch + stream_acc64_off(NF, a.grid));

  auto index_of = [&](uint32_t q) {
    IX ix;
    if constexpr (DR <= 1) { ix.r = 0; ix.c = (int)(q * W); }
    else { const uint32_t r = q / per_row; ix.r = (int)r; ix.c = (int)((q - r * per_row) * W); }
    return ix;
  };

  // scale: the first chunk of every thread gives the magnitude to expect
  {
    float m = 0.0f;
    const uint32_t q = team * kHistBlock + threadIdx.x;
    if (q < total) {
      const VAL v = eval<CL, pn.in[2]>(a, index_of(q));
      if constexpr (VEC) {
#pragma unroll
        for (int j = 0; j < 4; ++j) m = fmaxf(m, fabsf(f_(v.v[j])));
      } else {
        m = fabsf(f_(v));
      }
    }
    if (!(m < 3.0e38f)) m = 0.0f;                              // ignore infinities and NaNs here
    const uint32_t top = block_reduce_n<ACC_FN_MAX, ACC_F32, kHistBlock>(u_(m), red);
    if (threadIdx.x == 0) sample_max = f_(top);
  }
  __syncthreads();
  // a bin receives at most `mine` addends of magnitude < cap each: |sum| < 2^31
  const uint32_t mine = ((total + n_teams - 1) / n_teams + 1) * W;
  const int cap_log2 = min(30 - (32 - __clz(mine)), 22);      // 2^cap_log2 * mine < 2^30
  constexpr bool INTS = yields_small_integers<CL>(pn.in[2]);
  // values known to be integers below m: m - 1 is the magnitude to scale for, whatever the sample says
  const float largest = INTS ? (float)max(a.n[pn.in[2]].ip0 - 1, 0) : sample_max;
  int S = 0;
  if (largest > 0.0f) {
    int e;
    frexpf(largest, &e);                                       // largest = f * 2^e, f in [0.5, 1)
    S = min(max(cap_log2 - 1 - e, -100), 100);                 // largest * 2^S < cap / 2
  }
  const float cap = exp2f((float)cap_log2);
  const float up = exp2f((float)S);
  const double down = exp2((double)-S);

  auto scatter_one = [&](uint32_t k, uint32_t xbits) {
    if (k >= n_bins) { atomicOr(a.status, kStatusIndex); return; }
    uint32_t at = k;                                           // position among this CTA's bins
    if (group != 1) {
      const uint32_t owner = plan.shift >= 0 ? (k >> plan.shift) : (k / (uint32_t)per_cta);
      if (owner != rank) return;
      at = k - owner * (uint32_t)per_cta;
    }
    const float x = f_(xbits);
    if (x == 0.0f) return;
    const float t = __fmul_rn(x, up);                          // exact whenever |t| >= 1 (no underflow)
    // nearest integer without the conversion unit: adding 1.5 * 2^23 leaves |t| < 2^22 rounded
    // to an integer in the low mantissa bits (cap <= 2^22 keeps |t| in that range)
    const float shifted = __fadd_rn(t, 12582912.0f);
    const float rounded = __fadd_rn(shifted, -12582912.0f);
    if (fabsf(t) >= 1.0f && fabsf(t) < cap && t == rounded) {
      const int v = __float_as_int(shifted) - 0x4B400000;      // bits of 12582912.0f
      // two calls, so that each is an atomic on a known address space (shared / global)
      if (at < (uint32_t)per_cta) atomicAdd(bins_smem + at, v);
      else red_add_global(spill + (at - (uint32_t)per_cta), v);
    } else {
      red_add_global(acc64 + k, (double)x);
    }
  };

  const bool fast_ok = group == 1 && S >= 0;
  const uint32_t bins_addr = (uint32_t)__cvta_generic_to_shared(bins_smem);
  uint32_t it = 0;
  // FULL: every chunk of the trip and of the trips prefetched from it lies inside the array (no test per chunk)
  auto trip = [&](auto full_c, uint32_t q0) {
    constexpr bool FULL = decltype(full_c)::value;
    if constexpr (VEC) {
      // ask L2 for what the trip after next will read: there are too few registers to keep
      // enough loads in flight to cover DRAM latency, so the loads should find their lines in L2
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint32_t q = q0 + (kHistAhead * U + u) * stride;
        if (FULL || q < total) {
          const IX ix = index_of(q);
          eval<CL, pn.in[1]>(a, IxPF4{ix.r, ix.c});
          eval<CL, pn.in[2]>(a, IxPF4{ix.r, ix.c});
        }
      }
    }
    // evaluate U independent chunks first so that their loads are in flight together
    VAL key[U], val[U];
    bool live[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t q = q0 + u * stride;
      live[u] = FULL || q < total;
      if (live[u]) {
        const IX ix = index_of(q);
        key[u] = eval<CL, pn.in[1]>(a, ix);
        val[u] = eval<CL, pn.in[2]>(a, ix);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (!FULL && !live[u]) continue;
      if (group == 1 || (it + u) % group == rank) {            // this CTA's turn for the element-wise side
        const IX ix = index_of(q0 + u * stride);
        static_for<0, N>([&](auto ic) {
          constexpr int i = decltype(ic)::value;
          constexpr CNode nd = CL::c.nodes[i];
          if constexpr (is_store_root(nd)) {
            st(reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)), a.n[i].C, ix, eval<CL, i>(a, ix));
          } else if constexpr (is_scalar_fold(nd)) {
            // a fold over the scatter's own value or index operand shares its registers
            VAL v;
            if constexpr (nd.in[0] == CL::c.nodes[P].in[2]) v = val[u];
            else if constexpr (nd.in[0] == CL::c.nodes[P].in[1]) v = key[u];
            else v = eval<CL, nd.in[0]>(a, ix);
            // a thread adds thousands of chunks to its running value: that step is compensated; the four
            // elements of a chunk are of one magnitude and are combined as a small tree first
            if constexpr (VEC) {
              const uint32_t four = combine<nd.fn, nd.dtype>(combine<nd.fn, nd.dtype>(v.v[0], v.v[1]),
                                                             combine<nd.fn, nd.dtype>(v.v[2], v.v[3]));
              fold_step<nd.fn, nd.dtype>(acc[i], comp[i], four);
            } else {
              fold_step<nd.fn, nd.dtype>(acc[i], comp[i], v);
            }
          }
        });
      }
      if constexpr (VEC) {
        // The usual case in one piece, without a branch per element: all four indices in range and
        // all four values exact integers below `cap` after scaling.  (With up >= 1 a non-zero x
        // cannot underflow to a zero product; otherwise the careful path below is taken.)
        const uint32_t kmax = max(max(key[u].v[0], key[u].v[1]), max(key[u].v[2], key[u].v[3]));
        if constexpr (INTS) {
          // integers below m, and (m - 1) * 2^S below cap / 2 by the choice of S: every product is an
          // exact integer the bins can take, so only the indices are looked at
          if (fast_ok & (kmax < n_bins)) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              red_add_bin(key[u].v[j], (uint32_t)per_cta, bins_addr, spill - per_cta,
                          __float_as_int(__fadd_rn(__fmul_rn(f_(val[u].v[j]), up), 12582912.0f)) - 0x4B400000);
            continue;
          }
        }
        float t[4], shifted[4], off = 0.0f, big = 0.0f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          t[j] = __fmul_rn(f_(val[u].v[j]), up);
          shifted[j] = __fadd_rn(t[j], 12582912.0f);
          off = __fadd_rn(off, fabsf(__fadd_rn(__fadd_rn(shifted[j], -12582912.0f), -t[j])));   // 0 iff t is an integer (NaN otherwise)
          big = fmaxf(big, fabsf(t[j]));
        }
        if (fast_ok & (kmax < n_bins) & (off == 0.0f) & (big < cap)) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t k = key[u].v[j];
            // (a zero is added like any other value: skipping it would cost more than it saves)
            red_add_bin(k, (uint32_t)per_cta, bins_addr, spill - per_cta, __float_as_int(shifted[j]) - 0x4B400000);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) scatter_one(key[u].v[j], val[u].v[j]);
        }
      } else {
        scatter_one(key[u], val[u]);
      }
    }
  };
  {
    const uint64_t step = (uint64_t)stride * U;
    const uint64_t reach = (uint64_t)(kHistAhead * U + U - 1) * stride;     // the furthest chunk a trip touches, from its first
    uint64_t q0 = (uint64_t)team * kHistBlock + threadIdx.x;
    for (; q0 + reach < total; q0 += step, it += U) trip(std::true_type{}, (uint32_t)q0);
    for (; q0 < total; q0 += step, it += U) trip(std::false_type{}, (uint32_t)q0);
  }

  __syncthreads();
  // every CTA starts its sweep somewhere else, so that the CTAs that finish together do not all
  // queue up on the same accumulators
  const int turn = (int)((blockIdx.x * 2654435761u) >> 8);
  for (int i0 = threadIdx.x; i0 < per_cta; i0 += kHistBlock) {
    const int i = (int)((uint32_t)(i0 + turn) % (uint32_t)per_cta);
    const int v = bins_smem[i];
    const uint32_t bin = rank * (uint32_t)per_cta + i;
    if (v != 0 && bin < n_bins) red_add_global(acc64 + bin, (double)v * down);
  }
  for (int i0 = threadIdx.x; i0 < plan.overflow; i0 += kHistBlock) {
    const int i = (int)((uint32_t)(i0 + turn) % (uint32_t)plan.overflow);
    const int v = *reinterpret_cast<volatile int*>(spill + i);
    if (v != 0) red_add_global(acc64 + per_cta + i, (double)v * down);
  }

  static_for<0, N>([&](auto ic) {
    constexpr int i = decltype(ic)::value;
    constexpr CNode nd = CL::c.nodes[i];
    if constexpr (is_scalar_fold(nd)) {
      constexpr int ord = count_if<CL>(is_scalar_fold, i);
      const uint32_t v = block_reduce_n<nd.fn, nd.dtype, kHistBlock>(acc[i], red);
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
      for (int b = threadIdx.x; b < (int)gridDim.x; b += kHistBlock) v = combine<nd.fn, nd.dtype>(v, part[b]);
      v = block_reduce_n<nd.fn, nd.dtype, kHistBlock>(v, red);
      if (threadIdx.x == 0) *reinterpret_cast<uint32_t*>(const_cast<void*>(a.n[i].ptr)) = v;
    }
  });
  const volatile double* sums = acc64;
  const float* defaults = reinterpret_cast<const float*>(a.n[pn.in[0]].ptr);
  float* out = reinterpret_cast<float*>(const_cast<void*>(a.n[P].ptr));
  for (uint32_t b = threadIdx.x; b < n_bins; b += kHistBlock) out[b] = (float)((double)defaults[b] + sums[b]);
}

}  // namespace dev
}  // namespace acc
