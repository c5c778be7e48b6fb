// Execution of a program: clusters run by ascending cluster number (Section 4.1), one kernel
// launch each (or one per pass) on the caller's stream.  The unfused executor is the same
// machinery with every combinator its own cluster.
#include <algorithm>
#include <cstring>
#include <map>

#include "cluster.h"
#include "exec.h"
#include "graph.h"
#include "registry.h"

namespace acc {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Cuts the cluster formed by `members` (ascending) out of the graph, mirroring the
// build-time extract(): externals appear just before their first use.
static bool extract_runtime(const Graph& g, const std::vector<int>& members, const std::vector<uint8_t>& man, CCluster& c) {
  c = CCluster{};
  std::map<int, int> local;
  std::vector<uint8_t> in_cluster(g.nodes.size(), 0);
  for (int m : members) in_cluster[m] = 1;
  for (int m : members) {
    const acc_node_desc& d = g.nodes[m].d;
    for (int s = 0; s < d.n_inputs; ++s) {
      const int a = d.inputs[s];
      if (!in_cluster[a] && !local.count(a)) {
        if (c.n >= kMaxCluster) return false;
        CNode e{ACC_INPUT, g.nodes[a].d.dtype, g.nodes[a].d.rank, 0, 0, 0, 0, {-1, -1, -1, -1, -1, -1}, false, true};
        local[a] = c.n;
        c.source[c.n] = a;
        c.nodes[c.n++] = e;
      }
    }
    if (c.n >= kMaxCluster) return false;
    CNode n{d.kind, d.dtype, d.rank, d.fn_id, d.idx_fn_id, d.n_inputs, d.n_array_inputs, {-1, -1, -1, -1, -1, -1}, true, man[m] != 0};
    if (d.kind != ACC_BACKPERMUTE) n.idxfn = 0;
    if (d.kind == ACC_BACKPERMUTE || d.kind == ACC_GATHER) n.fn = 0;
    if (d.kind == ACC_BACKPERMUTE && d.idx_fn_id == ACC_IDX_SHIFT_CLAMP && d.iparam[0] >= -1 && d.iparam[0] <= 1 &&
        d.iparam[1] >= -1 && d.iparam[1] <= 1) {
      n.p0 = (int)d.iparam[0];                         // kernels built for these very offsets are looked up first
      n.p1 = (int)d.iparam[1];
    }
    if ((d.kind == ACC_SCANL || d.kind == ACC_SCANR) && (d.flags & ACC_FLAG_SCAN_EXCLUSIVE)) n.p0 = 1;   // other code, not another argument
    if (d.kind == ACC_MAP && d.fn_id == ACC_FN_MUL_MOD && d.iparam[1] > 0 && (d.iparam[1] & (d.iparam[1] - 1)) == 0)
      n.p0 = kPow2;                                    // a kernel built for power-of-two moduli is looked up first
    for (int s = 0; s < d.n_inputs; ++s) n.in[s] = local[d.inputs[s]];
    local[m] = c.n;
    c.source[c.n] = m;
    c.nodes[c.n++] = n;
  }
  return true;
}

static dev::NodeArg node_arg(const Node& n, const void* ptr) {
  dev::NodeArg a{};
  a.ptr = ptr;
  a.ip0 = (int32_t)(uint32_t)(n.d.iparam[0] & 0xFFFFFFFFll);
  a.ip1 = (int32_t)(uint32_t)(n.d.iparam[1] & 0xFFFFFFFFll);
  a.fp0 = (float)n.d.fparam[0];
  a.fp1 = (float)n.d.fparam[1];
  // branch-free division by d (Granlund and Montgomery's round-up multiplier, 33 bits with the
  // add-and-shift fix-up): l = ceil(log2 d), m = floor(2^32 (2^l - d) / d) + 1,
  // v / d = (t + ((v - t) >> min(l, 1))) >> max(l - 1, 0) with t = umulhi(v, m); d = 1 gives v
  const uint32_t d = (uint32_t)(n.d.fn_id == ACC_FN_MUL_MOD ? a.ip1 : a.ip0);
  if (d >= 1) {
    uint32_t l = 0;
    while (l < 32 && (1ull << l) < d) ++l;
    a.div_mul = (uint32_t)((((1ull << l) - d) << 32) / d + 1);
    a.div_sh1 = l < 1 ? l : 1;
    a.div_sh2 = l - a.div_sh1;
    a.div_mask = (d & (d - 1)) == 0 ? d - 1 : 0;
  }
  a.R = n.d.rank == 2 ? (int32_t)n.d.shape[0] : 1;
  a.C = n.d.rank == 2 ? (int32_t)n.d.shape[1] : (n.d.rank == 1 ? (int32_t)n.d.shape[0] : 1);
  return a;
}

// The kernel instantiated for a cluster: for its very constants, else the one that takes them at run time.
static const KernelEntry* lookup(CCluster& cc, std::string& sig) {
  sig = signature(cc);
  const KernelEntry* k = find_kernel(sig);
  if (!k) {
    for (int li = 0; li < cc.n; ++li)
      if (cc.nodes[li].kind == ACC_BACKPERMUTE || (cc.nodes[li].kind == ACC_MAP && cc.nodes[li].fn == ACC_FN_MUL_MOD))
        cc.nodes[li].p0 = cc.nodes[li].p1 = kRunTime;
    sig = signature(cc);
    k = find_kernel(sig);
  }
  return k;
}

int refine_to_kernels(const Graph& g, std::vector<int32_t>& pi, int recompute_depth, int& splits) {
  const int n = (int)g.nodes.size();
  splits = 0;
  for (;;) {
    std::vector<uint8_t> man;
    manifest_of(g, pi.data(), man);
    std::map<int, std::vector<int>> clusters;
    for (int i = 0; i < n; ++i)
      if (!is_input(g.nodes[i])) clusters[pi[i]].push_back(i);
    const std::vector<int>* bad = nullptr;
    std::string sig;
    for (auto& kv : clusters) {
      CCluster cc;
      if (!extract_runtime(g, kv.second, man, cc) || !lookup(cc, sig)) { bad = &kv.second; break; }
    }
    if (!bad) return ACC_OK;
    if (bad->size() == 1)
      return set_error(ACC_ERR_NO_KERNEL, "no kernel instantiated for node %d alone [%s]", bad->front(), sig.c_str());
    // the latest member that may leave and still leave a legal clustering becomes a cluster of its own;
    // failing that the whole cluster falls apart into its nodes
    const int n_blocks = (int)clusters.size();
    std::vector<int> block_of(pi.begin(), pi.end());
    std::vector<int32_t> trial;
    bool done = false;
    for (auto it = bad->rbegin(); it != bad->rend() && !done; ++it) {
      std::vector<int> b(block_of);
      b[*it] = n_blocks;
      done = canonical_numbering(g, b, n_blocks + 1, trial) && check_partition(g, trial.data(), nullptr, true, recompute_depth) == ACC_OK;
    }
    if (!done) {
      std::vector<int> b(block_of);
      int next = n_blocks;
      for (size_t k = 1; k < bad->size(); ++k) b[(*bad)[k]] = next++;
      if (!canonical_numbering(g, b, next, trial) || check_partition(g, trial.data(), nullptr, true, recompute_depth) != ACC_OK)
        return set_error(ACC_ERR_NO_KERNEL, "the cluster at node %d has no kernel and cannot be split legally [%s]", bad->front(), sig.c_str());
    }
    clear_error();
    pi = trial;
    ++splits;
  }
}

int build_schedule(Graph& g, int executor, Schedule& sch) {
  const int n = (int)g.nodes.size();
  sch = Schedule{};
  std::vector<int32_t> pi;
  if (executor == ACC_EXEC_FUSED) {
    if (!g.has_pi) return set_error(ACC_ERR_NO_PARTITION, "no clustering set: call acc_set_partition or acc_plan first");
    pi = g.pi;
  } else if (executor == ACC_EXEC_UNFUSED) {
    pi.assign(n, -1);
    int c = 0;
    for (int i = 0; i < n; ++i)
      if (!is_input(g.nodes[i])) pi[i] = c++;
  } else {
    return set_error(ACC_ERR_ARG, "unknown executor %d", executor);
  }
  std::vector<uint8_t> man;
  manifest_of(g, pi.data(), man);

  // buffers: bound ones stay where they are, other manifest arrays go into the workspace
  sch.array_off.assign(n, SIZE_MAX);
  size_t off = 0;
  for (int i = 0; i < n; ++i) {
    const Node& nd = g.nodes[i];
    if (is_input(nd) || nd.output) {
      if (!nd.dev && nd.count > 0)
        return set_error(ACC_ERR_UNBOUND, "node %d (%s) has no device buffer", i, is_input(nd) ? "input" : "output");
      continue;
    }
    if (!man[i] || nd.dev) continue;
    sch.array_off[i] = off;
    off += align_up((size_t)std::max<int64_t>(nd.count, 1) * 4, 256);
  }
  sch.array_bytes = off;

  std::map<int, std::vector<int>> clusters;
  for (int i = 0; i < n; ++i)
    if (!is_input(g.nodes[i])) clusters[pi[i]].push_back(i);
  size_t ctrl = 256;                                    // status word first
  for (auto& kv : clusters) {
    ClusterStep st;
    st.first_node = kv.second.front();
    st.n_members = (int)kv.second.size();
    if (!extract_runtime(g, kv.second, man, st.cc))
      return set_error(ACC_ERR_NO_KERNEL, "cluster at node %d has more than %d local nodes", st.first_node, kMaxCluster);
    std::string sig;
    st.kernel = lookup(st.cc, sig);
    if (!st.kernel)
      return set_error(ACC_ERR_NO_KERNEL, "no kernel instantiated for the cluster of %d nodes starting at node %d [%s]",
                       st.n_members, st.first_node, sig.c_str());
    st.launch.n = st.cc.n;
    for (int li = 0; li < st.cc.n; ++li) st.launch.nodes[li] = node_arg(g.nodes[st.cc.source[li]], nullptr);
    const int64_t sb = st.kernel->scratch_bytes(st.launch);
    if (sb < 0) return set_error((int)sb, "cluster at node %d: no scratch layout", st.first_node);
    const int64_t zb = st.kernel->zeroed_bytes(st.launch);
    st.scratch_off = ctrl;
    st.scratch_bytes = (size_t)sb;
    st.zero_bytes = (size_t)std::min<int64_t>(std::max<int64_t>(zb, 0), sb);
    ctrl += align_up((size_t)sb, 256);
    sch.steps.push_back(st);
  }
  sch.ctrl_bytes = ctrl;
  sch.to_clear.clear();
  sch.to_clear.emplace_back(0, 256);                       // the status slot
  for (const ClusterStep& st : sch.steps) {
    if (st.zero_bytes == 0) continue;
    auto& last = sch.to_clear.back();
    if (last.first + align_up(last.second, 256) == st.scratch_off) last.second = st.scratch_off - last.first + st.zero_bytes;   // one piece
    else sch.to_clear.emplace_back(st.scratch_off, st.zero_bytes);
  }
  sch.total_bytes = ctrl + sch.array_bytes;
  sch.manifest = man;
  sch.pi = pi;
  return ACC_OK;
}

static void* buffer_of(const Graph& g, const Schedule& sch, char* ws, int node) {
  const Node& nd = g.nodes[node];
  if (nd.dev) return nd.dev;
  if (sch.array_off[node] == SIZE_MAX) return nullptr;
  return ws + sch.ctrl_bytes + sch.array_off[node];
}

static bool mark(std::vector<cudaEvent_t>* marks, cudaStream_t stream) {
  if (!marks) return true;
  cudaEvent_t e;
  if (cudaEventCreate(&e) != cudaSuccess) return false;
  marks->push_back(e);
  return cudaEventRecord(e, stream) == cudaSuccess;
}

int run_schedule(Graph& g, Schedule& sch, void* workspace, size_t ws_bytes, cudaStream_t stream, std::vector<cudaEvent_t>* marks) {
  if (!workspace) return set_error(ACC_ERR_WORKSPACE, "workspace is null, %zu bytes needed", sch.total_bytes);
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return set_error(ACC_ERR_WORKSPACE, "workspace is not 256-byte aligned");
  if (ws_bytes < sch.total_bytes) return set_error(ACC_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", ws_bytes, sch.total_bytes);
  char* ws = static_cast<char*>(workspace);
  for (const auto& piece : sch.to_clear)
    if (cudaMemsetAsync(ws + piece.first, 0, piece.second, stream) != cudaSuccess)
      return set_error(ACC_ERR_CUDA, "clearing the control region failed: %s", cudaGetErrorString(cudaGetLastError()));
  g.launches = 0;
  g.schedule.clear();
  if (!mark(marks, stream)) return set_error(ACC_ERR_CUDA, "recording an event failed: %s", cudaGetErrorString(cudaGetLastError()));
  for (ClusterStep& st : sch.steps) {
    for (int li = 0; li < st.cc.n; ++li) {
      const int node = st.cc.source[li];
      const CNode& cn = st.cc.nodes[li];
      void* p = (!cn.member || cn.manifest) ? buffer_of(g, sch, ws, node) : nullptr;
      if ((!cn.member || cn.manifest) && !p && g.nodes[node].count > 0)
        return set_error(ACC_ERR_UNBOUND, "node %d is read or written by the cluster at node %d but has no buffer", node, st.first_node);
      st.launch.nodes[li].ptr = p;
    }
    st.launch.scratch = reinterpret_cast<uint32_t*>(ws + st.scratch_off);
    st.launch.status = reinterpret_cast<uint32_t*>(ws);
    st.launch.stream = stream;
    st.launch.spin_limit = g.spin_limit;
    st.launch.extra_launches = 0;
    const int rc = st.kernel->launch(st.launch);
    if (rc != ACC_OK) return rc;
    if (!mark(marks, stream)) return set_error(ACC_ERR_CUDA, "recording an event failed: %s", cudaGetErrorString(cudaGetLastError()));
    g.launches += st.kernel->passes + st.launch.extra_launches;
    char item[48];
    snprintf(item, sizeof item, "%s%d:%d", g.schedule.empty() ? "" : " ", st.first_node, st.n_members);
    g.schedule += item;
  }
  return ACC_OK;
}

// One word per index: out of range (as unsigned, so negative ones too) sets the index bit of the status word.
__global__ void k_index_range(const uint32_t* idx, int64_t n, uint32_t bound, uint32_t* status) {
  bool bad = false;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) bad = bad || idx[i] >= bound;
  if (__syncthreads_or(bad) && threadIdx.x == 0) atomicOr(status, 2u);
}

int check_gather_indices(Graph& g, void* workspace, size_t ws_bytes, cudaStream_t stream) {
  if (!workspace || ws_bytes < 256 || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return set_error(ACC_ERR_WORKSPACE, "the check needs a 256-byte aligned workspace of 256 bytes");
  if (cudaMemsetAsync(workspace, 0, 256, stream) != cudaSuccess)
    return set_error(ACC_ERR_CUDA, "clearing the status word failed: %s", cudaGetErrorString(cudaGetLastError()));
  for (const Node& nd : g.nodes) {
    if (nd.d.kind != ACC_GATHER) continue;
    const Node& idx = g.nodes[nd.d.inputs[0]];
    const Node& src = g.nodes[nd.d.inputs[1]];
    if (!is_input(idx) || !idx.dev || idx.count == 0) continue;
    const uint32_t bound = (uint32_t)std::min<int64_t>(src.count, 0x7FFFFFFF);
    const int grid = (int)std::min<int64_t>((idx.count + 255) / 256, (int64_t)sm_count() * 8);
    k_index_range<<<grid, 256, 0, stream>>>(static_cast<const uint32_t*>(idx.dev), idx.count, bound, static_cast<uint32_t*>(workspace));
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
  }
  return finish(g, workspace, stream);
}

int finish(Graph& g, void* workspace, cudaStream_t stream) {
  uint32_t status = 0;
  if (workspace && cudaMemcpyAsync(&status, workspace, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return set_error(ACC_ERR_CUDA, "reading the status word failed: %s", cudaGetErrorString(cudaGetLastError()));
  const cudaError_t e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "stream failed: %s", cudaGetErrorString(e));
  g.host_status = status;
  if (status & 1u) return set_error(ACC_ERR_DEVICE_TIMEOUT, "a device-side wait ran out of iterations");
  if (status & 2u) return set_error(ACC_ERR_INDEX_RANGE, "a scatter index, a segment offset or a checked gather index fell outside its array");
  if (status & 4u) return set_error(ACC_ERR_SHAPE, "an empty segment has no value: segment offsets must increase");
  return ACC_OK;
}

}  // namespace acc
