// Kernels of  B = transpose A; C = A*B + k; rowsum = fold(+) C  (all four legal clusterings).
#include "../device/launch.cuh"
#include "programs.h"

namespace acc {
using programs::kTransposeReduce;
ACC_CLUSTER(kTransposeReduce, 0x2, tr_B)
ACC_CLUSTER(kTransposeReduce, 0x4, tr_C)
ACC_CLUSTER(kTransposeReduce, 0x8, tr_rowsum)
ACC_CLUSTER(kTransposeReduce, 0x6, tr_BC)
ACC_CLUSTER(kTransposeReduce, 0xC, tr_Crowsum)
ACC_CLUSTER(kTransposeReduce, 0xE, tr_BCrowsum)
}  // namespace acc
