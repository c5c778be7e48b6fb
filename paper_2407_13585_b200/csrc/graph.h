// Runtime data-dependence graph of a combinator program (Section 4.1 of the paper:
// nodes, fusible edges F, infusible edges I) and the state attached to it.
#pragma once
#include <cstdarg>
#include <cstdint>
#include <memory>
#include <string>
#include <vector>

#include "acc.h"

namespace acc {

struct Node {
  acc_node_desc d{};
  bool     output = false;
  int64_t  count = 0;          // number of elements
  void*    dev = nullptr;      // caller-bound device buffer
  size_t   dev_bytes = 0;
  void*    host = nullptr;     // caller-bound host buffer (end-to-end runs)
  size_t   host_bytes = 0;
};

// One edge per input slot of the consumer.
struct Edge {
  int  a, b, slot;
  bool fusible;   // may be fused when a and b share a cluster
  bool ordered;   // the slot traverses the array in a definite order (Table 1)
};

struct Graph {
  std::vector<Node> nodes;
  std::vector<Edge> edges;
  std::vector<int32_t> pi;         // stored clustering, -1 for inputs
  bool has_pi = false;
  int recompute_depth = 0;         // the rules the stored clustering was checked under
  // A clustering with nodes copied into further clusters is run on a graph of its own in which
  // every copy is a node: `unfolded` (its own clustering stored in it), and where each node of
  // this graph went (`home_in_unfolded`).  Null for every other clustering.
  std::shared_ptr<Graph> unfolded;
  std::vector<int> home_in_unfolded;
  std::vector<uint8_t> manifest;   // under the stored clustering
  // bookkeeping of the last run
  int64_t plan_visited = 0;        // partial clusterings the last planner call looked at
  bool plan_proven = false;        // ... and whether its result is proven optimal
  int32_t launches = 0;
  std::string schedule;
  uint32_t host_status = 0;
  uint32_t run_serial = 0;         // bumped by every change that invalidates a schedule
  uint32_t spin_limit = 1u << 22;  // polls a scan tile spends on a predecessor before it gives up (acc_set_spin_limit)
};

inline bool is_input(const Node& n) { return n.d.kind == ACC_INPUT; }
inline bool gather_like(const Node& n) { return n.d.kind == ACC_GATHER || n.d.kind == ACC_BACKPERMUTE; }

int  set_error(int code, const char* fmt, ...);
const char* last_error();
void clear_error();

// graph.cpp
int  add_node(Graph& g, const acc_node_desc& d);

// legality.cpp
struct Solution {
  std::vector<uint8_t> manifest;   // per node
  std::vector<int32_t> order;      // d^o per node (for PERMUTE: order of its idx/vals slots), -1 for inputs
  std::vector<std::vector<int32_t>> copies;   // clusters that recompute: every order a node is evaluated in (else empty)
};
// recompute_depth 0: the paper's rules; k > 0: producers may be evaluated once per order they are
// read in, with at most k gather-like members stacked on a fused path
int  check_partition(const Graph& g, const int32_t* pi, Solution* sol, bool quiet = false, int recompute_depth = 0);
void manifest_of(const Graph& g, const int32_t* pi, std::vector<uint8_t>& man);
bool partial_clustering_possible(const Graph& g, const std::vector<int>& block_of, int n_blocks, const std::vector<uint8_t>& man,
                                 bool check_orders);
void forced_manifest(const Graph& g, std::vector<uint8_t>& forced, std::vector<uint8_t>& must_read);

// planner.cpp
int     plan(Graph& g, int mode, int cost, std::vector<int32_t>& out, int recompute_depth = 0);
int64_t enumerate_all(const Graph& g, std::vector<std::vector<int32_t>>& out, int recompute_depth = 0);
int     partition_cost(const Graph& g, const int32_t* pi, int cost, double* out, int recompute_depth = 0);
bool    canonical_numbering(const Graph& g, const std::vector<int>& block_of, int n_blocks, std::vector<int32_t>& pi);

}  // namespace acc

struct acc_graph : acc::Graph {};
