// Kernels of one Jacobi iteration (five clamped shifts, four zipWiths): the nodes alone,
// the whole iteration as one cluster, the intermediate cuts the greedy planners reach, and
// two to four whole iterations as one cluster.
#include "../device/launch.cuh"
#include "programs.h"

namespace acc {
using programs::kJacobi;
ACC_CLUSTER(kJacobi, 0x002, jac_shift)          // any single shift (the five are one pattern)
ACC_CLUSTER(kJacobi, 0x040, jac_add)            // t1, t2, t3 alone
ACC_CLUSTER(kJacobi, 0x200, jac_add_scale)      // Y alone
ACC_CLUSTER(kJacobi, 0x3FE, jac_iteration)      // all nine
ACC_CLUSTER(kJacobi, 0x046, jac_cn_t1)          // {c, n, t1}
ACC_CLUSTER(kJacobi, 0x0CE, jac_cns_t2)         // {c, n, s, t1, t2}
ACC_CLUSTER(kJacobi, 0x1DE, jac_cnse_t3)        // {c, n, s, e, t1, t2, t3}
ACC_CLUSTER(kJacobi, 0x220, jac_w_Y)            // {w, Y}
ACC_CLUSTER(kJacobi, 0x330, jac_ew_t3Y)         // {e, w, t3, Y}
ACC_CLUSTER(kJacobi, 0x3C0, jac_sums)           // {t1, t2, t3, Y} over five manifest shifts
ACC_CLUSTER(kJacobi, 0x380, jac_t2t3Y)          // {t2, t3, Y} over a manifest t1 and three manifest shifts
// Several iterations in one cluster (a clustering that recomputes: the iterate in between is
// read in five orders); the iterates in between stay in shared memory.
using programs::kJacobiChain;
// (built for the five-point offsets, which halves the instructions of a stacked kernel.  A single
// iteration is left to the kernel above that takes the offsets at run time: built for fixed
// offsets it ran 8192 x 8192 in 104 us per launch back to back against 93 us, although alone,
// from a cold cache, it is the faster one, 89 against 95 us)
ACC_CLUSTER(kJacobiChain, 0x7FFFEull, jac_two_iterations)
ACC_CLUSTER(kJacobiChain, 0xFFFFFFEull, jac_three_iterations)
ACC_CLUSTER(kJacobiChain, 0x1FFFFFFFFEull, jac_four_iterations)
}  // namespace acc
