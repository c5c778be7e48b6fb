// extern "C" entry points declared in acc.h.
#include <cstring>
#include <map>
#include <memory>

#include "acc.h"
#include "exec.h"
#include "graph.h"

using namespace acc;

namespace {

// Schedules are rebuilt only when the graph, its clustering or its bindings change.
struct Cache {
  uint32_t serial = ~0u;
  Schedule sch;
};
std::map<const acc_graph*, std::unique_ptr<Cache[]>>& caches() {
  static std::map<const acc_graph*, std::unique_ptr<Cache[]>> c;
  return c;
}

// The graph a run works on: the caller's, or, for the fused executor under a clustering with
// copies, the graph in which the copies are nodes (buffers and output marks carried over).
Graph& run_target(acc_graph* g, int executor) {
  if (executor != ACC_EXEC_FUSED || !g->unfolded) return *g;
  Graph& u = *g->unfolded;
  u.spin_limit = g->spin_limit;
  for (size_t i = 0; i < g->nodes.size(); ++i) {
    Node& to = u.nodes[g->home_in_unfolded[i]];
    const Node& from = g->nodes[i];
    to.dev = from.dev;
    to.dev_bytes = from.dev_bytes;
    to.host = from.host;
    to.host_bytes = from.host_bytes;
  }
  return u;
}

int schedule_for(acc_graph* g, int executor, Schedule** out) {
  if (executor != ACC_EXEC_FUSED && executor != ACC_EXEC_UNFUSED) return set_error(ACC_ERR_ARG, "unknown executor %d", executor);
  auto& slot = caches()[g];
  if (!slot) slot.reset(new Cache[2]);
  Cache& c = slot[executor];
  if (c.serial != g->run_serial) {
    const int rc = build_schedule(run_target(g, executor), executor, c.sch);
    if (rc != ACC_OK) return rc;
    c.serial = g->run_serial;
  }
  *out = &c.sch;
  return ACC_OK;
}

bool bad_node(const acc_graph* g, acc_node n) { return n < 0 || n >= (acc_node)g->nodes.size(); }

}  // namespace

extern "C" {

int acc_graph_create(acc_graph** out) {
  clear_error();
  if (!out) return set_error(ACC_ERR_ARG, "out is null");
  *out = new acc_graph();
  return ACC_OK;
}

int acc_graph_destroy(acc_graph* g) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  caches().erase(g);
  delete g;
  return ACC_OK;
}

acc_node acc_add_node(acc_graph* g, const acc_node_desc* d) {
  clear_error();
  if (!g || !d) return set_error(ACC_ERR_ARG, "null argument");
  g->run_serial++;
  g->unfolded.reset();
  return add_node(*g, *d);
}

int acc_mark_output(acc_graph* g, acc_node n) {
  clear_error();
  if (!g || bad_node(g, n)) return set_error(ACC_ERR_ARG, "bad node id");
  if (is_input(g->nodes[n])) return set_error(ACC_ERR_ARG, "an input cannot be an output");
  g->nodes[n].output = true;
  g->has_pi = false;
  g->unfolded.reset();
  g->run_serial++;
  return ACC_OK;
}

int32_t acc_node_count(const acc_graph* g) { return g ? (int32_t)g->nodes.size() : ACC_ERR_ARG; }

int acc_edges(const acc_graph* g, int32_t* F, int32_t* nF, int32_t* I, int32_t* nI, int32_t cap) {
  clear_error();
  if (!g || !nF || !nI) return set_error(ACC_ERR_ARG, "null argument");
  int f = 0, i = 0;
  for (const Edge& e : g->edges) {
    int32_t* dst = e.fusible ? F : I;
    int& k = e.fusible ? f : i;
    if (dst && k < cap) { dst[2 * k] = e.a; dst[2 * k + 1] = e.b; }
    ++k;
  }
  *nF = f;
  *nI = i;
  return ACC_OK;
}

int acc_check_partition_recompute(acc_graph* g, const int32_t* pi, int32_t n_nodes, int32_t max_depth) {
  clear_error();
  if (!g || !pi) return set_error(ACC_ERR_ARG, "null argument");
  if (max_depth < 0) return set_error(ACC_ERR_ARG, "max_depth %d is negative", max_depth);
  if (n_nodes != (int32_t)g->nodes.size()) return set_error(ACC_ERR_ARG, "clustering has %d entries, graph has %zu nodes", n_nodes, g->nodes.size());
  for (int i = 0; i < n_nodes; ++i)
    if (!is_input(g->nodes[i]) && (pi[i] < 0 || pi[i] > n_nodes)) return set_error(ACC_ERR_ARG, "cluster number %d of node %d outside 0..n", pi[i], i);
  return check_partition(*g, pi, nullptr, false, max_depth);
}

int acc_check_partition(acc_graph* g, const int32_t* pi, int32_t n_nodes) { return acc_check_partition_recompute(g, pi, n_nodes, 0); }

int acc_set_partition_recompute(acc_graph* g, const int32_t* pi, int32_t n_nodes, int32_t max_depth) {
  const int rc = acc_check_partition_recompute(g, pi, n_nodes, max_depth);
  if (rc != ACC_OK) return rc;
  g->pi.assign(pi, pi + n_nodes);
  for (int i = 0; i < n_nodes; ++i)
    if (is_input(g->nodes[i])) g->pi[i] = -1;
  manifest_of(*g, g->pi.data(), g->manifest);
  g->has_pi = true;
  g->recompute_depth = max_depth;
  g->unfolded.reset();
  g->run_serial++;
  return ACC_OK;
}

int acc_set_partition(acc_graph* g, const int32_t* pi, int32_t n_nodes) { return acc_set_partition_recompute(g, pi, n_nodes, 0); }

int acc_set_partition_copies(acc_graph* g, const int32_t* pi, int32_t n_nodes, const int32_t* copy_node, const int32_t* copy_cluster,
                             int32_t n_copies, int32_t max_depth) {
  clear_error();
  if (!g || !pi || n_copies < 0 || (n_copies > 0 && (!copy_node || !copy_cluster))) return set_error(ACC_ERR_ARG, "null argument");
  if (max_depth < 0) return set_error(ACC_ERR_ARG, "max_depth %d is negative", max_depth);
  const int n = (int)g->nodes.size();
  if (n_nodes != n) return set_error(ACC_ERR_ARG, "clustering has %d entries, graph has %d nodes", n_nodes, n);
  for (int i = 0; i < n; ++i)
    if (!is_input(g->nodes[i]) && (pi[i] < 0 || pi[i] > n)) return set_error(ACC_ERR_ARG, "cluster number %d of node %d outside 0..n", pi[i], i);
  for (int k = 0; k < n_copies; ++k) {
    const int a = copy_node[k], c = copy_cluster[k];
    if (a < 0 || a >= n || is_input(g->nodes[a])) return set_error(ACC_ERR_ARG, "copy %d: node %d cannot be copied", k, a);
    if (c < 0 || c > n || c == pi[a]) return set_error(ACC_ERR_ARG, "copy %d: cluster %d is node %d's own or outside 0..n", k, c, a);
    for (int j = 0; j < k; ++j)
      if (copy_node[j] == a && copy_cluster[j] == c) return set_error(ACC_ERR_ARG, "copy %d repeats copy %d", k, j);
  }
  // the graph with every copy as a node, right after the node it copies (so inputs still come first)
  auto u = std::make_shared<Graph>();
  std::vector<int> home(n, -1);
  std::vector<int32_t> upi;
  std::vector<int> copy_id(n_copies, -1);
  auto instance = [&](int x, int cluster) {            // what a reader in `cluster` reads of node x
    if (!is_input(g->nodes[x]) && pi[x] != cluster)
      for (int k = 0; k < n_copies; ++k)
        if (copy_node[k] == x && copy_cluster[k] == cluster) return copy_id[k];
    return home[x];
  };
  for (int i = 0; i < n; ++i) {
    for (int k = -1; k < n_copies; ++k) {
      if (k >= 0 && copy_node[k] != i) continue;
      const int cluster = k < 0 ? (is_input(g->nodes[i]) ? -1 : pi[i]) : copy_cluster[k];
      acc_node_desc d = g->nodes[i].d;
      for (int s = 0; s < d.n_inputs; ++s) d.inputs[s] = instance(d.inputs[s], cluster);
      const int id = add_node(*u, d);
      if (id < 0) return id;
      upi.push_back(cluster);
      if (k < 0) { home[i] = id; u->nodes[id].output = g->nodes[i].output; }
      else copy_id[k] = id;
    }
  }
  const int rc = check_partition(*u, upi.data(), nullptr, false, max_depth);
  if (rc != ACC_OK) return rc;
  std::vector<uint8_t> uman;
  manifest_of(*u, upi.data(), uman);
  for (int k = 0; k < n_copies; ++k)
    if (uman[copy_id[k]])
      return set_error(ACC_ERR_ARG, "the copy of node %d in cluster %d has no reader there or would have to be stored", copy_node[k], copy_cluster[k]);
  u->pi = upi;
  u->manifest = uman;
  u->has_pi = true;
  u->recompute_depth = max_depth;
  g->pi.assign(pi, pi + n);
  g->manifest.assign(n, 0);
  for (int i = 0; i < n; ++i) {
    if (is_input(g->nodes[i])) g->pi[i] = -1;
    g->manifest[i] = uman[home[i]];
  }
  g->has_pi = true;
  g->recompute_depth = max_depth;
  g->unfolded = u;
  g->home_in_unfolded = home;
  g->run_serial++;
  return ACC_OK;
}

int acc_get_partition(const acc_graph* g, int32_t* out, int32_t n_nodes) {
  clear_error();
  if (!g || !out || n_nodes != (int32_t)g->nodes.size()) return set_error(ACC_ERR_ARG, "bad argument");
  if (!g->has_pi) return set_error(ACC_ERR_NO_PARTITION, "no clustering set");
  memcpy(out, g->pi.data(), sizeof(int32_t) * n_nodes);
  return ACC_OK;
}

int acc_manifest(const acc_graph* g, int32_t* out, int32_t n_nodes) {
  clear_error();
  if (!g || !out || n_nodes != (int32_t)g->nodes.size()) return set_error(ACC_ERR_ARG, "bad argument");
  if (!g->has_pi) return set_error(ACC_ERR_NO_PARTITION, "no clustering set");
  for (int i = 0; i < n_nodes; ++i) out[i] = g->manifest[i];
  return ACC_OK;
}

int acc_plan_recompute(acc_graph* g, int mode, int cost, int32_t max_depth, int32_t* out) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  if (max_depth < 0) return set_error(ACC_ERR_ARG, "max_depth %d is negative", max_depth);
  std::vector<int32_t> pi;
  const int rc = plan(*g, mode, cost, pi, max_depth);
  if (rc != ACC_OK) return rc;
  if (out) memcpy(out, pi.data(), sizeof(int32_t) * pi.size());
  return acc_set_partition_recompute(g, pi.data(), (int32_t)pi.size(), max_depth);
}

int acc_plan(acc_graph* g, int mode, int cost, int32_t* out) { return acc_plan_recompute(g, mode, cost, 0, out); }

int acc_refine_to_kernels(acc_graph* g, int32_t* out) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  if (!g->has_pi) return set_error(ACC_ERR_NO_PARTITION, "no clustering set: call acc_set_partition or acc_plan first");
  if (g->unfolded) return set_error(ACC_ERR_ARG, "a clustering with copies is not refined");
  std::vector<int32_t> pi(g->pi);
  int splits = 0;
  const int depth = g->recompute_depth;
  int rc = refine_to_kernels(*g, pi, depth, splits);
  if (rc != ACC_OK) return rc;
  if (splits > 0) {
    rc = acc_set_partition_recompute(g, pi.data(), (int32_t)pi.size(), depth);
    if (rc != ACC_OK) return rc;
  }
  if (out) memcpy(out, g->pi.data(), sizeof(int32_t) * g->pi.size());
  return splits;
}

int acc_plan_info(const acc_graph* g, int64_t* visited, int32_t* proven) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  if (visited) *visited = g->plan_visited;
  if (proven) *proven = g->plan_proven ? 1 : 0;
  return ACC_OK;
}

int64_t acc_enumerate(acc_graph* g, int32_t* out_pi, int64_t max_partitions) { return acc_enumerate_recompute(g, 0, out_pi, max_partitions); }

int64_t acc_enumerate_recompute(acc_graph* g, int32_t max_depth, int32_t* out_pi, int64_t max_partitions) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  if (max_depth < 0) return set_error(ACC_ERR_ARG, "max_depth %d is negative", max_depth);
  std::vector<std::vector<int32_t>> all;
  const int64_t cnt = enumerate_all(*g, all, max_depth);
  if (cnt < 0) return cnt;
  const size_t n = g->nodes.size();
  if (out_pi)
    for (int64_t i = 0; i < cnt && i < max_partitions; ++i) memcpy(out_pi + i * n, all[i].data(), sizeof(int32_t) * n);
  return cnt;
}

int acc_partition_cost_recompute(acc_graph* g, const int32_t* pi, int32_t n_nodes, int32_t max_depth, int cost, double* out) {
  clear_error();
  if (!g || !pi || !out || max_depth < 0 || n_nodes != (int32_t)g->nodes.size()) return set_error(ACC_ERR_ARG, "bad argument");
  return partition_cost(*g, pi, cost, out, max_depth);
}

int acc_partition_cost(acc_graph* g, const int32_t* pi, int32_t n_nodes, int cost, double* out) {
  return acc_partition_cost_recompute(g, pi, n_nodes, 0, cost, out);
}

int acc_bind(acc_graph* g, acc_node n, void* device_ptr, size_t bytes) {
  clear_error();
  if (!g || bad_node(g, n)) return set_error(ACC_ERR_ARG, "bad node id");
  Node& nd = g->nodes[n];
  if (bytes < (size_t)nd.count * 4) return set_error(ACC_ERR_UNBOUND, "node %d needs %zu bytes, buffer has %zu", n, (size_t)nd.count * 4, bytes);
  if (!device_ptr && nd.count > 0) return set_error(ACC_ERR_ARG, "device pointer is null");
  if (reinterpret_cast<uintptr_t>(device_ptr) & 15) return set_error(ACC_ERR_ARG, "device pointer is not 16-byte aligned");
  nd.dev = device_ptr;
  nd.dev_bytes = bytes;
  g->run_serial++;
  return ACC_OK;
}

int acc_bind_host(acc_graph* g, acc_node n, void* host_ptr, size_t bytes) {
  clear_error();
  if (!g || bad_node(g, n)) return set_error(ACC_ERR_ARG, "bad node id");
  Node& nd = g->nodes[n];
  if (!is_input(nd) && !nd.output) return set_error(ACC_ERR_ARG, "node %d is neither an input nor a marked output", n);
  if (bytes < (size_t)nd.count * 4 || (!host_ptr && nd.count > 0)) return set_error(ACC_ERR_UNBOUND, "host buffer of node %d is null or too small", n);
  nd.host = host_ptr;
  nd.host_bytes = bytes;
  return ACC_OK;
}

int acc_workspace_bytes(acc_graph* g, int executor, size_t* bytes) {
  clear_error();
  if (!g || !bytes) return set_error(ACC_ERR_ARG, "null argument");
  Schedule* sch = nullptr;
  const int rc = schedule_for(g, executor, &sch);
  if (rc != ACC_OK) return rc;
  *bytes = sch->total_bytes;
  return ACC_OK;
}

int acc_run(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream, int executor) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  Schedule* sch = nullptr;
  int rc = schedule_for(g, executor, &sch);
  if (rc != ACC_OK) return rc;
  Graph& target = run_target(g, executor);
  rc = run_schedule(target, *sch, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
  g->launches = target.launches;
  g->schedule = target.schedule;
  return rc;
}

int acc_run_timed(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream, int executor,
                  float* ms_out, int32_t cap, int32_t* n_out) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  Schedule* sch = nullptr;
  int rc = schedule_for(g, executor, &sch);
  if (rc != ACC_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  std::vector<cudaEvent_t> marks;
  Graph& target = run_target(g, executor);
  rc = run_schedule(target, *sch, workspace, workspace_bytes, stream, &marks);
  g->launches = target.launches;
  g->schedule = target.schedule;
  if (rc == ACC_OK) rc = finish(*g, workspace, stream);
  if (rc == ACC_OK) {
    const int n = (int)marks.size() - 1;
    for (int k = 0; k < n && k < cap && ms_out; ++k) {
      float ms = 0;
      if (cudaEventElapsedTime(&ms, marks[k], marks[k + 1]) != cudaSuccess) ms = -1.0f;
      ms_out[k] = ms;
    }
    if (n_out) *n_out = n < 0 ? 0 : n;
  }
  for (cudaEvent_t e : marks) cudaEventDestroy(e);
  cudaGetLastError();
  return rc;
}

int acc_check_gather_indices(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  return check_gather_indices(*g, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int acc_finish(acc_graph* g, void* workspace, void* cuda_stream) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  return finish(*g, workspace, static_cast<cudaStream_t>(cuda_stream));
}

int acc_run_e2e(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream, int executor,
                size_t* h2d_bytes, size_t* d2h_bytes) {
  const int rc = acc_run_e2e_async(g, workspace, workspace_bytes, cuda_stream, executor, h2d_bytes, d2h_bytes);
  if (rc != ACC_OK) return rc;
  return finish(*g, workspace, static_cast<cudaStream_t>(cuda_stream));
}

int acc_run_e2e_async(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream, int executor,
                      size_t* h2d_bytes, size_t* d2h_bytes) {
  clear_error();
  if (!g) return set_error(ACC_ERR_ARG, "graph is null");
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  size_t up = 0, down = 0;
  for (Node& nd : g->nodes)
    if (is_input(nd) && nd.host) {
      if (!nd.dev) return set_error(ACC_ERR_UNBOUND, "a host-bound input has no device buffer");
      const size_t b = (size_t)nd.count * 4;
      if (b && cudaMemcpyAsync(nd.dev, nd.host, b, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return set_error(ACC_ERR_CUDA, "host-to-device copy failed: %s", cudaGetErrorString(cudaGetLastError()));
      up += b;
    }
  const int rc = acc_run(g, workspace, workspace_bytes, cuda_stream, executor);
  if (rc != ACC_OK) return rc;
  for (Node& nd : g->nodes)
    if (nd.output && nd.host) {
      const size_t b = (size_t)nd.count * 4;
      if (b && cudaMemcpyAsync(nd.host, nd.dev, b, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return set_error(ACC_ERR_CUDA, "device-to-host copy failed: %s", cudaGetErrorString(cudaGetLastError()));
      down += b;
    }
  if (h2d_bytes) *h2d_bytes = up;
  if (d2h_bytes) *d2h_bytes = down;
  return ACC_OK;
}

int32_t acc_launch_count(const acc_graph* g) { return g ? g->launches : ACC_ERR_ARG; }

int acc_set_spin_limit(acc_graph* g, uint32_t max_polls) {
  if (!g) return set_error(ACC_ERR_ARG, "null graph");
  g->spin_limit = max_polls;
  return ACC_OK;
}

int acc_last_schedule(const acc_graph* g, char* buf, size_t cap) {
  if (!g || !buf || !cap) return ACC_ERR_ARG;
  strncpy(buf, g->schedule.c_str(), cap - 1);
  buf[cap - 1] = 0;
  return ACC_OK;
}

const char* acc_last_error(void) { return last_error(); }

int32_t acc_registry_size(void) { return registry_size(); }

}  // extern "C"
