// Kernels of  k = hash keys; vals = generate; hist = permute(+) zeros k vals;
// total = fold(+) vals; frac = hist / total  (all ten legal clusterings).
#include "../device/launch.cuh"
#include "programs.h"

namespace acc {
using programs::kHistogram;
ACC_CLUSTER(kHistogram, 0x04, hist_k)
ACC_CLUSTER(kHistogram, 0x08, hist_vals)
ACC_CLUSTER(kHistogram, 0x10, hist_hist)
ACC_CLUSTER(kHistogram, 0x20, hist_total)
ACC_CLUSTER(kHistogram, 0x40, hist_frac)
ACC_CLUSTER(kHistogram, 0x14, hist_k_hist)
ACC_CLUSTER(kHistogram, 0x18, hist_vals_hist)
ACC_CLUSTER(kHistogram, 0x28, hist_vals_total)
ACC_CLUSTER(kHistogram, 0x30, hist_hist_total)
ACC_CLUSTER(kHistogram, 0x1C, hist_k_vals_hist)
ACC_CLUSTER(kHistogram, 0x34, hist_k_hist_total)
ACC_CLUSTER(kHistogram, 0x38, hist_vals_hist_total)
ACC_CLUSTER(kHistogram, 0x3C, hist_all)
// the clusters that hold the hash, built for a modulus that is a power of two (one AND per key)
using programs::kHistogramPow2;
ACC_CLUSTER(kHistogramPow2, 0x04, hist_k_pow2)
ACC_CLUSTER(kHistogramPow2, 0x14, hist_k_hist_pow2)
ACC_CLUSTER(kHistogramPow2, 0x1C, hist_k_vals_hist_pow2)
ACC_CLUSTER(kHistogramPow2, 0x34, hist_k_hist_total_pow2)
ACC_CLUSTER(kHistogramPow2, 0x3C, hist_all_pow2)
ACC_CLUSTER(programs::kHistogramScatterOnlyPow2, 0x1C, hist_k_vals_hist_private_pow2)
// with a copy of `vals` in the cluster of `total`
ACC_CLUSTER(programs::kHistogramScatterOnly, 0x1C, hist_k_vals_hist_private)
ACC_CLUSTER(programs::kGeneratedTotal, 0x3, hist_vals_copy_total)
}  // namespace acc
