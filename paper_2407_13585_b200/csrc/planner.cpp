// Host planner: cost functions of Section 4.1 (a)-(e), exhaustive search over all legal
// clusterings of small graphs (in place of the ILP solver), and the two greedy
// algorithms of Section 5 ("Greedy"): walk the fusible edges from the top or from the
// bottom of the graph, fuse an edge, keep it if a legal clustering still exists.
#include <algorithm>
#include <functional>
#include <set>
#include <tuple>

#include "graph.h"

namespace acc {

// Numbers the blocks in an execution order that respects every edge and the scatter rule;
// ties go to the block holding the smallest node id.  False if no such order exists.
bool canonical_numbering(const Graph& g, const std::vector<int>& block_of, int n_blocks, std::vector<int32_t>& pi) {
  const int n = (int)g.nodes.size();
  std::vector<std::set<int>> before(n_blocks);
  std::vector<int> smallest(n_blocks, n);
  for (int i = 0; i < n; ++i)
    if (block_of[i] >= 0) smallest[block_of[i]] = std::min(smallest[block_of[i]], i);
  for (const Edge& e : g.edges) {
    if (block_of[e.a] < 0) continue;
    if (block_of[e.a] != block_of[e.b]) before[block_of[e.b]].insert(block_of[e.a]);
  }
  for (int j = 0; j < n; ++j) {
    if (g.nodes[j].d.kind != ACC_PERMUTE) continue;
    const int dest = g.nodes[j].d.inputs[0];
    for (const Edge& e : g.edges)
      if (e.a == dest && e.b != j) {
        if (block_of[e.b] == block_of[j]) return false;
        before[block_of[j]].insert(block_of[e.b]);
      }
  }
  std::vector<int> number(n_blocks, -1);
  for (int next = 0; next < n_blocks; ++next) {
    int pick = -1;
    for (int b = 0; b < n_blocks; ++b) {
      if (number[b] >= 0) continue;
      bool ready = true;
      for (int p : before[b]) ready = ready && number[p] >= 0;
      if (ready && (pick < 0 || smallest[b] < smallest[pick])) pick = b;
    }
    if (pick < 0) return false;
    number[pick] = next;
  }
  pi.assign(n, -1);
  for (int i = 0; i < n; ++i)
    if (block_of[i] >= 0) pi[i] = number[block_of[i]];
  return true;
}

int partition_cost(const Graph& g, const int32_t* pi, int cost, double* out, int recompute_depth) {
  Solution sol;
  const int rc = check_partition(g, pi, &sol, false, recompute_depth);
  if (rc != ACC_OK) return rc;
  const int n = (int)g.nodes.size();
  auto bytes = [&](int a) { return double(std::max<int64_t>(g.nodes[a].count, 1)) * 4.0; };
  std::set<int> clusters;
  for (int i = 0; i < n; ++i)
    if (!is_input(g.nodes[i])) clusters.insert(pi[i]);
  double unfused = 0;
  for (const Edge& e : g.edges)
    if (e.fusible && pi[e.a] != pi[e.b]) unfused += 1;
  double arrays = 0, write_bytes = 0;
  for (int i = 0; i < n; ++i)
    if (!is_input(g.nodes[i]) && sol.manifest[i]) { arrays += 1; write_bytes += bytes(i); }
  // one read per (array, consuming cluster, order of the consuming slot)
  std::set<std::tuple<int, int, int, int>> reads;
  int label = 2;
  std::vector<int> lab(n, 0);
  for (int i = 0; i < n; ++i)
    if (gather_like(g.nodes[i])) lab[i] = label++;
  for (const Edge& e : g.edges) {
    const bool inside = !is_input(g.nodes[e.a]) && pi[e.a] == pi[e.b];
    if (inside || e.slot >= g.nodes[e.b].d.n_array_inputs) continue;
    const int k = g.nodes[e.b].d.kind;
    int order, uniq = -1;
    if (!e.ordered) { order = -2; uniq = e.b * 8 + e.slot; }
    else if (k == ACC_BACKPERMUTE || (k == ACC_GATHER && e.slot == 1)) order = lab[e.b];
    else order = sol.order[e.b];
    reads.insert(std::make_tuple(e.a, pi[e.b], order, uniq));
    // a reader that is evaluated in several orders (a cluster that recomputes) reads once per order
    if (e.ordered && order == sol.order[e.b] && e.b < (int)sol.copies.size())
      for (int32_t o : sol.copies[e.b]) reads.insert(std::make_tuple(e.a, pi[e.b], (int)o, uniq));
  }
  double n_reads = 0, read_bytes = 0;
  for (auto& r : reads) { n_reads += 1; read_bytes += bytes(std::get<0>(r)); }
  switch (cost) {
    case ACC_COST_CLUSTERS: *out = (double)clusters.size(); break;
    case ACC_COST_FUSED_EDGES: *out = unfused; break;
    case ACC_COST_ARRAYS: *out = arrays; break;
    case ACC_COST_READS: *out = n_reads; break;
    case ACC_COST_READS_WRITES: *out = n_reads + arrays; break;
    case ACC_COST_EVERYTHING: *out = (double)clusters.size() + unfused + arrays + n_reads + (n_reads + arrays); break;
    case ACC_COST_BYTES: *out = read_bytes + write_bytes; break;
    default: return set_error(ACC_ERR_ARG, "unknown cost function %d", cost);
  }
  return ACC_OK;
}

int64_t enumerate_all(const Graph& g, std::vector<std::vector<int32_t>>& out, int recompute_depth) {
  const int n = (int)g.nodes.size();
  std::vector<int> items;
  for (int i = 0; i < n; ++i)
    if (!is_input(g.nodes[i])) items.push_back(i);
  if (items.size() > 12) return set_error(ACC_ERR_TOO_LARGE, "%zu nodes: exhaustive enumeration is limited to 12", items.size());
  // infusible pairs can never share a block: prune while growing
  std::vector<std::vector<uint8_t>> apart(n, std::vector<uint8_t>(n, 0));
  for (const Edge& e : g.edges)
    if (!e.fusible) apart[e.a][e.b] = apart[e.b][e.a] = 1;
  std::vector<int> block_of(n, -1);
  std::vector<int32_t> pi;
  std::function<void(size_t, int)> grow = [&](size_t at, int n_blocks) {
    if (at == items.size()) {
      if (canonical_numbering(g, block_of, n_blocks, pi) && check_partition(g, pi.data(), nullptr, true, recompute_depth) == ACC_OK) out.push_back(pi);
      return;
    }
    const int node = items[at];
    for (int b = 0; b <= n_blocks; ++b) {
      bool ok = true;
      for (size_t j = 0; j < at && ok; ++j)
        if (block_of[items[j]] == b && apart[items[j]][node]) ok = false;
      if (!ok) continue;
      block_of[node] = b;
      grow(at + 1, b == n_blocks ? n_blocks + 1 : n_blocks);
    }
    block_of[node] = -1;
  };
  grow(0, 0);
  std::sort(out.begin(), out.end());
  return (int64_t)out.size();
}

namespace {

// Greedy over fusible edges.  Fusing (a, b) merges their blocks and pulls in every node
// lying on a path between the two blocks (otherwise no execution order exists).
int greedy(const Graph& g, bool top_down, std::vector<int32_t>& out, int recompute_depth) {
  const int n = (int)g.nodes.size();
  std::vector<std::vector<uint8_t>> reach(n, std::vector<uint8_t>(n, 0));   // reach[a][b]: path a -> b
  for (int b = 0; b < n; ++b)
    for (const Edge& e : g.edges)
      if (e.b == b) {
        reach[e.a][b] = 1;
        for (int a = 0; a < n; ++a)
          if (reach[a][e.a]) reach[a][b] = 1;
      }
  std::vector<int> block(n, -1);
  int n_blocks = 0;
  for (int i = 0; i < n; ++i)
    if (!is_input(g.nodes[i])) block[i] = n_blocks++;
  std::vector<const Edge*> order;
  for (const Edge& e : g.edges)
    if (e.fusible) order.push_back(&e);
  std::stable_sort(order.begin(), order.end(), [&](const Edge* x, const Edge* y) {
    return top_down ? std::make_pair(x->a, x->b) < std::make_pair(y->a, y->b)
                    : std::make_pair(x->b, x->a) > std::make_pair(y->b, y->a);
  });
  auto densify = [&](const std::vector<int>& blk, std::vector<int>& dense) {
    std::vector<int> remap(n_blocks, -1);
    dense.assign(n, -1);
    int nb = 0;
    for (int i = 0; i < n; ++i)
      if (blk[i] >= 0) {
        if (remap[blk[i]] < 0) remap[blk[i]] = nb++;
        dense[i] = remap[blk[i]];
      }
    return nb;
  };
  std::vector<int32_t> pi;
  std::vector<int> dense;
  for (const Edge* e : order) {
    if (block[e->a] == block[e->b]) continue;
    std::vector<int> trial(block);
    const int keep = trial[e->a], gone = trial[e->b];
    for (int i = 0; i < n; ++i)
      if (trial[i] == gone) trial[i] = keep;
    bool grew = true;
    while (grew) {                                    // convex closure of the merged block
      grew = false;
      for (int i = 0; i < n; ++i) {
        if (trial[i] < 0 || trial[i] == keep) continue;
        bool below = false, above = false;
        for (int j = 0; j < n; ++j)
          if (trial[j] == keep) { below = below || reach[j][i]; above = above || reach[i][j]; }
        if (below && above) {
          const int was = trial[i];
          for (int j = 0; j < n; ++j)
            if (trial[j] == was) trial[j] = keep;
          grew = true;
        }
      }
    }
    const int nb = densify(trial, dense);
    if (canonical_numbering(g, dense, nb, pi) && check_partition(g, pi.data(), nullptr, true, recompute_depth) == ACC_OK) block = trial;
  }
  const int nb = densify(block, dense);
  if (!canonical_numbering(g, dense, nb, out)) return set_error(ACC_ERR_ARG, "greedy planner lost its execution order");
  return ACC_OK;
}

// Exact search for the cheapest clustering under the reads-and-writes objective of Section 4.1
// (e), in arrays or in bytes.  Nodes are placed in program order, each into one of the blocks
// that exist or into a new one (its producers' blocks first, so that the first leaves look like
// the greedy results).  A partial clustering is dropped when it can no longer become legal
// (partial_clustering_possible) or when the traffic it is already sure of is no less than the
// best complete clustering known: every array that is manifest for certain is written once, and
// read once by every placed block that reads it from outside and once more by each gather-like
// reader, whose order no other read shares (at least once by somebody if that is certain too).
struct BranchBound {
  static constexpr int64_t kLimit = int64_t(1) << 22;
  Graph& g;
  const int cost, depth;
  std::vector<int> items, block_of;
  std::vector<uint8_t> forced, must_read, apart;
  int n = 0, n_blocks = 0;
  double best = 0;
  std::vector<int32_t> best_pi;
  int64_t visited = 0;
  bool complete = true;

  BranchBound(Graph& g_, int cost_, int depth_) : g(g_), cost(cost_), depth(depth_) {
    n = (int)g.nodes.size();
    block_of.assign(n, -1);
    for (int i = 0; i < n; ++i)
      if (!is_input(g.nodes[i])) items.push_back(i);
    forced_manifest(g, forced, must_read);
    if (depth > 0) {                       // with copies an array read in two orders can be fused away after all
      for (int i = 0; i < n; ++i) {
        bool infusible_out = false;
        int readers = 0;
        for (const Edge& e : g.edges)
          if (e.a == i) { ++readers; infusible_out = infusible_out || !e.fusible; }
        forced[i] = is_input(g.nodes[i]) || g.nodes[i].output || readers == 0 || infusible_out;
        if (!is_input(g.nodes[i]) && !infusible_out) must_read[i] = 0;
      }
    }
    apart.assign((size_t)n * n, 0);
    for (const Edge& e : g.edges)
      if (!e.fusible) apart[(size_t)e.a * n + e.b] = apart[(size_t)e.b * n + e.a] = 1;
  }

  double weight(int a) const { return cost == ACC_COST_BYTES ? double(std::max<int64_t>(g.nodes[a].count, 1)) * 4.0 : 1.0; }

  // arrays that are manifest whatever happens to the nodes not placed yet
  void certain_manifest(std::vector<uint8_t>& man) const {
    man = forced;
    for (const Edge& e : g.edges)
      if (block_of[e.b] >= 0 && block_of[e.a] >= 0 && block_of[e.a] != block_of[e.b]) man[e.a] = 1;
  }

  double bound(const std::vector<uint8_t>& man) const {
    double sum = 0;
    std::vector<int> seen;
    for (int a = 0; a < n; ++a) {
      if (!man[a]) continue;
      if (!is_input(g.nodes[a])) sum += weight(a);
      seen.clear();
      size_t by_label = 0;                                // a gather-like reader has an order of its own: a read of its own
      for (const Edge& e : g.edges) {
        if (e.a != a || e.slot >= g.nodes[e.b].d.n_array_inputs) continue;
        const int k = g.nodes[e.b].d.kind;
        const bool label_slot = k == ACC_BACKPERMUTE || (k == ACC_GATHER && e.slot == 1);
        // in the paper's model a stored array cannot be fused into such a reader, placed or not
        if (label_slot && depth == 0) { ++by_label; continue; }
        if (block_of[e.b] < 0) continue;
        if (!is_input(g.nodes[a]) && block_of[e.b] == block_of[a]) continue;
        if (label_slot) { ++by_label; continue; }
        if (std::find(seen.begin(), seen.end(), block_of[e.b]) == seen.end()) seen.push_back(block_of[e.b]);
      }
      sum += weight(a) * (double)std::max<size_t>(seen.size() + by_label, must_read[a] ? 1 : 0);
    }
    return sum;
  }

  void leaf() {
    std::vector<int32_t> pi;
    if (!canonical_numbering(g, block_of, n_blocks, pi)) return;
    double c = 0;
    if (check_partition(g, pi.data(), nullptr, true, depth) != ACC_OK) return;
    if (partition_cost(g, pi.data(), cost, &c, depth) != ACC_OK) return;
    if (c < best) { best = c; best_pi = pi; }
  }

  void search(size_t at) {
    if (at == items.size()) { leaf(); return; }
    const int node = items[at];
    std::vector<int> order;                               // blocks to try: producers' first, then the rest, then a new one
    for (int s = g.nodes[node].d.n_inputs - 1; s >= 0; --s) {
      const int b = block_of[g.nodes[node].d.inputs[s]];
      if (b >= 0 && std::find(order.begin(), order.end(), b) == order.end()) order.push_back(b);
    }
    for (int b = n_blocks - 1; b >= 0; --b)
      if (std::find(order.begin(), order.end(), b) == order.end()) order.push_back(b);
    order.push_back(n_blocks);
    std::vector<uint8_t> man;
    for (int b : order) {
      bool ok = true;
      for (size_t j = 0; j < at && ok; ++j)
        if (block_of[items[j]] == b && apart[(size_t)items[j] * n + node]) ok = false;
      if (!ok) continue;
      if (++visited > kLimit) { complete = false; return; }
      block_of[node] = b;
      const int grown = b == n_blocks ? 1 : 0;
      n_blocks += grown;
      certain_manifest(man);
      if (partial_clustering_possible(g, block_of, n_blocks, man, depth == 0) && bound(man) < best) search(at + 1);
      n_blocks -= grown;
      block_of[node] = -1;
      if (!complete) return;
    }
  }
};

}  // namespace

int plan(Graph& g, int mode, int cost, std::vector<int32_t>& out, int recompute_depth) {
  g.plan_visited = 0;
  g.plan_proven = false;
  const int n = (int)g.nodes.size();
  switch (mode) {
    case ACC_PLAN_UNFUSED: {
      out.assign(n, -1);
      int c = 0;
      for (int i = 0; i < n; ++i)
        if (!is_input(g.nodes[i])) out[i] = c++;
      return check_partition(g, out.data(), nullptr);
    }
    case ACC_PLAN_ENUMERATE: {
      std::vector<std::vector<int32_t>> all;
      const int64_t cnt = enumerate_all(g, all, recompute_depth);
      if (cnt < 0) return (int)cnt;
      if (cnt == 0) return set_error(ACC_ERR_ARG, "no legal clustering");
      double best = 0;
      int best_i = -1;
      for (int i = 0; i < (int)all.size(); ++i) {
        double c = 0;
        const int rc = partition_cost(g, all[i].data(), cost, &c, recompute_depth);
        if (rc != ACC_OK) return rc;
        if (best_i < 0 || c < best) { best = c; best_i = i; }
      }
      out = all[best_i];
      g.plan_visited = cnt;
      g.plan_proven = true;
      return ACC_OK;
    }
    case ACC_PLAN_BRANCH_BOUND: {
      if (cost != ACC_COST_BYTES && cost != ACC_COST_READS_WRITES)
        return set_error(ACC_ERR_ARG, "branch and bound minimises reads and writes (cost READS_WRITES or BYTES)");
      BranchBound bb(g, cost, recompute_depth);
      for (int top_down = 0; top_down < 2; ++top_down) {           // the better greedy result is the first incumbent
        std::vector<int32_t> pi;
        double c = 0;
        if (greedy(g, top_down != 0, pi, recompute_depth) != ACC_OK) continue;
        if (partition_cost(g, pi.data(), cost, &c, recompute_depth) != ACC_OK) continue;
        if (bb.best_pi.empty() || c < bb.best) { bb.best = c; bb.best_pi = pi; }
      }
      if (bb.best_pi.empty()) bb.best = 1e300;                     // no greedy result: any legal clustering is better
      clear_error();
      bb.search(0);
      if (bb.best_pi.empty()) return set_error(ACC_ERR_ARG, "no legal clustering");
      out = bb.best_pi;
      g.plan_visited = bb.visited;
      g.plan_proven = bb.complete;
      return ACC_OK;
    }
    case ACC_PLAN_GREEDY_TOPDOWN: return greedy(g, true, out, recompute_depth);
    case ACC_PLAN_GREEDY_BOTTOMUP: return greedy(g, false, out, recompute_depth);
    default: return set_error(ACC_ERR_ARG, "unknown planner mode %d", mode);
  }
}

}  // namespace acc
