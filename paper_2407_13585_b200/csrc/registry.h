// Registry of build-time kernel instantiations, keyed by cluster signature.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>
#include <string>

#include "cluster.h"
#include "device/eval.cuh"

namespace acc {

// Everything a launcher needs for one cluster of one run.  nodes[] is indexed by the
// cluster's local ids and carries pointers, constants and shapes.
struct ClusterLaunch {
  dev::NodeArg nodes[kMaxCluster];
  int n = 0;
  uint32_t* scratch = nullptr;   // scratch_bytes() bytes, 16-byte aligned, the first zeroed_bytes() of them zero
  uint32_t* status = nullptr;
  uint32_t spin_limit = 1u << 22;
  cudaStream_t stream = nullptr;
  mutable int extra_launches = 0;   // set by a launcher that took more launches than its entry's `passes` (data-dependent paths)
};

struct KernelEntry {
  std::string sig;
  const char* name;
  int64_t (*scratch_bytes)(const ClusterLaunch&);   // >= 0, or a negative acc_status
  int64_t (*zeroed_bytes)(const ClusterLaunch&);    // how much of the scratch, from its start, must be zero at launch
  int (*launch)(const ClusterLaunch&);               // acc_status; asynchronous
  int passes = 1;                                    // launches per run (see Passes in device/launch.cuh)
};

void register_kernel(const KernelEntry& e);
const KernelEntry* find_kernel(const std::string& sig);
int registry_size();
int sm_count();
bool cooperative_launch_ok();   // the current device can run a grid with all blocks resident
// Fills the CUtensorMap at `out` for box copies from a row-major rows x cols array of 4-byte
// elements; false if the driver call is unavailable or the array is not 16-byte friendly.
bool make_tensor_map_2d(void* out, const void* base, int rows, int cols, int box_rows, int box_cols);

}  // namespace acc
