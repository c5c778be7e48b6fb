// Schedule of one executor over one graph: clusters in execution order with their
// kernels, and the layout of the caller's workspace (control region, then arrays).
#pragma once
#include <cuda_runtime.h>

#include <utility>
#include <vector>

#include "cluster.h"
#include "graph.h"
#include "registry.h"

namespace acc {

struct ClusterStep {
  int first_node = 0, n_members = 0;
  CCluster cc{};
  const KernelEntry* kernel = nullptr;
  ClusterLaunch launch;
  size_t scratch_off = 0, scratch_bytes = 0, zero_bytes = 0;
};

struct Schedule {
  std::vector<ClusterStep> steps;
  std::vector<size_t> array_off;     // offset of each workspace-resident array, SIZE_MAX otherwise
  std::vector<uint8_t> manifest;
  std::vector<int32_t> pi;
  size_t ctrl_bytes = 0, array_bytes = 0, total_bytes = 0;
  std::vector<std::pair<size_t, size_t>> to_clear;   // (offset, bytes) of what a run zeroes first: the status slot and the zeroed part of every scratch
};

int build_schedule(Graph& g, int executor, Schedule& sch);
// Splits clusters of `pi` that have no instantiated kernel until every cluster has one (see acc_refine_to_kernels).
int refine_to_kernels(const Graph& g, std::vector<int32_t>& pi, int recompute_depth, int& splits);
// `marks`, if given, receives one recorded event before the first launch and one after each launch
int run_schedule(Graph& g, Schedule& sch, void* workspace, size_t ws_bytes, cudaStream_t stream,
                 std::vector<cudaEvent_t>* marks = nullptr);
int check_gather_indices(Graph& g, void* workspace, size_t ws_bytes, cudaStream_t stream);
int finish(Graph& g, void* workspace, cudaStream_t stream);

}  // namespace acc
