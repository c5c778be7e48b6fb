// Kernels of  g = hash x; h = gather idx g; o = h & mask; out = scanl(+) o
// (all eight legal clusterings).
#include "../device/launch.cuh"
#include "programs.h"

namespace acc {
using programs::kGatherScan;
ACC_CLUSTER(kGatherScan, 0x04, gs_g)
ACC_CLUSTER(kGatherScan, 0x08, gs_h)
ACC_CLUSTER(kGatherScan, 0x10, gs_o)
ACC_CLUSTER(kGatherScan, 0x20, gs_out)
ACC_CLUSTER(kGatherScan, 0x0C, gs_gh)
ACC_CLUSTER(kGatherScan, 0x18, gs_ho)
ACC_CLUSTER(kGatherScan, 0x30, gs_oout)
ACC_CLUSTER(kGatherScan, 0x1C, gs_gho)
ACC_CLUSTER(kGatherScan, 0x38, gs_hoout)
ACC_CLUSTER(kGatherScan, 0x3C, gs_ghoout)
}  // namespace acc
