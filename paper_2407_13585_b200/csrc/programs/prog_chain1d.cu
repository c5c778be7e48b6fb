// Kernels of the 1-D chain  y = map x; z = reverse y; w = z * x; s = fold(+) w:
// every node alone and every connected sub-chain (all eight legal clusterings).
#include "../device/launch.cuh"
#include "programs.h"

namespace acc {
using programs::kChain1d;
ACC_CLUSTER(kChain1d, 0x02, chain_y)
ACC_CLUSTER(kChain1d, 0x04, chain_z)
ACC_CLUSTER(kChain1d, 0x08, chain_w)
ACC_CLUSTER(kChain1d, 0x10, chain_s)
ACC_CLUSTER(kChain1d, 0x06, chain_yz)
ACC_CLUSTER(kChain1d, 0x0C, chain_zw)
ACC_CLUSTER(kChain1d, 0x18, chain_ws)
ACC_CLUSTER(kChain1d, 0x0E, chain_yzw)
ACC_CLUSTER(kChain1d, 0x1C, chain_zws)
ACC_CLUSTER(kChain1d, 0x1E, chain_yzws)
}  // namespace acc
