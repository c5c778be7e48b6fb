// Legality of a clustering pi: the paper's Figure 3 evaluated for given pi, plus the
// top-level rules of Section 3.4 and the splitting step of Section 4.1.
//
// Within a cluster, x_ab = 0 is forced for every edge (Figure 3: x_ab <= pi_b - pi_a), so
// the order equalities d^o_a = d^i_b of all inner edges must hold together.  They are
// solved by union-find over one order variable per node; constants come from scans (0/1)
// and from the source slot of gather-like nodes (their label).  Manifest arrays need an
// order in {0,1}.  Order classes that stay free are 0 or 1; which one matters only for
// whether two reads of a common outside parent are shared, i.e. for connectivity, and is
// settled by a small exhaustive search.
//
// Recomputing clusterings (an extension; the paper leaves work duplication to future work in
// its Section 6).  With `recompute_depth` > 0 an array that is fused away may be evaluated
// once per order it is asked for, as if every consumer had a private copy of its producer (and
// of that producer's producers inside the cluster).  The order equalities then only run from a
// consumer to its own copies, so they can only fail at a scan (whose order is fixed) or at the
// one stored copy of a manifest array (order 0 or 1).  At most `recompute_depth` gather-like
// members may be stacked on a fused path of a cluster that needs such copies; a cluster that is
// legal in the paper's model stays legal whatever its depth.
#include <algorithm>
#include <map>

#include "graph.h"

namespace acc {

void manifest_of(const Graph& g, const int32_t* pi, std::vector<uint8_t>& man) {
  const int n = (int)g.nodes.size();
  man.assign(n, 0);
  std::vector<uint8_t> has_out(n, 0);
  for (const Edge& e : g.edges) {
    has_out[e.a] = 1;
    if (is_input(g.nodes[e.a]) || pi[e.a] != pi[e.b] || !e.fusible) man[e.a] = 1;
  }
  for (int i = 0; i < n; ++i)
    if (is_input(g.nodes[i]) || g.nodes[i].output || !has_out[i]) man[i] = 1;
}

namespace {

struct Dsu {
  std::vector<int> p;
  explicit Dsu(int n) : p(n) { for (int i = 0; i < n; ++i) p[i] = i; }
  int find(int x) { while (p[x] != x) { p[x] = p[p[x]]; x = p[x]; } return x; }
  void unite(int a, int b) { p[find(a)] = find(b); }
};

constexpr int kFree = -1;

struct ClusterCheck {
  const Graph& g;
  const std::vector<int>& members;         // ascending node ids
  const std::vector<uint8_t>& man;
  const std::vector<int>& label;           // label per gather-like node, else 0
  std::vector<int> local;                  // node id -> index in members, -1 outside

  ClusterCheck(const Graph& g_, const std::vector<int>& m, const std::vector<uint8_t>& man_, const std::vector<int>& lab)
      : g(g_), members(m), man(man_), label(lab), local(g_.nodes.size(), -1) {
    for (int i = 0; i < (int)m.size(); ++i) local[m[i]] = i;
  }

  // Order of slot `slot` of member b: a constant label, or b's own order variable (kFree).
  int slot_const(int b, int slot) const {
    const int k = g.nodes[b].d.kind;
    if (k == ACC_BACKPERMUTE || (k == ACC_GATHER && slot == 1)) return label[b];
    return kFree;
  }

  // With need_connected = false only the order equalities are checked: what a cluster that is
  // still growing can already get wrong for good.
  int run(std::vector<int32_t>* order_out, bool need_connected = true) {
    const int m = (int)members.size();
    Dsu cls(m);
    for (const Edge& e : g.edges) {
      if (local[e.a] < 0 || local[e.b] < 0) continue;
      if (slot_const(e.b, e.slot) == kFree) cls.unite(local[e.a], local[e.b]);
    }
    std::vector<int> value(m, kFree);        // per class root
    std::vector<uint8_t> zero_one(m, 0);
    auto pin = [&](int node_local, int v) -> bool {
      const int r = cls.find(node_local);
      if (value[r] != kFree && value[r] != v) return false;
      value[r] = v;
      return true;
    };
    for (int i = 0; i < m; ++i) {
      const int a = members[i];
      const int k = g.nodes[a].d.kind;
      if (k == ACC_SCANL && !pin(i, 0)) return ACC_ERR_ILLEGAL_TRAVERSAL;
      if (k == ACC_SCANR && !pin(i, 1)) return ACC_ERR_ILLEGAL_TRAVERSAL;
      if (man[a] || k == ACC_PERMUTE) zero_one[cls.find(i)] = 1;
    }
    for (const Edge& e : g.edges) {
      if (local[e.a] < 0 || local[e.b] < 0) continue;
      const int c = slot_const(e.b, e.slot);
      if (c != kFree && !pin(local[e.a], c)) return ACC_ERR_ILLEGAL_TRAVERSAL;
    }
    for (int i = 0; i < m; ++i) {
      const int r = cls.find(i);
      if (zero_one[r] && value[r] > 1) return ACC_ERR_ILLEGAL_TRAVERSAL;
    }
    if (!need_connected) return ACC_OK;
    // connectivity: fused edges, or reads of one outside parent in one order
    Dsu base(m);
    for (const Edge& e : g.edges)
      if (local[e.a] >= 0 && local[e.b] >= 0) base.unite(local[e.a], local[e.b]);
    struct Read { int parent, cls, node; };
    std::vector<Read> reads;                 // reads through a node's own order variable
    for (const Edge& e : g.edges) {
      if (local[e.b] < 0 || local[e.a] >= 0 || !e.ordered) continue;
      if (slot_const(e.b, e.slot) != kFree) continue;   // a label is unique: never shared with another node
      reads.push_back({e.a, cls.find(local[e.b]), local[e.b]});
    }
    std::vector<int> free_cls;
    for (const Read& r : reads)
      if (value[r.cls] == kFree && std::find(free_cls.begin(), free_cls.end(), r.cls) == free_cls.end()) free_cls.push_back(r.cls);
    const int k = (int)free_cls.size();
    const uint32_t combos = k > 16 ? 1u : (1u << k);
    std::vector<int> trial(value);
    for (uint32_t bits = 0; bits < combos; ++bits) {
      for (int j = 0; j < k; ++j) trial[free_cls[j]] = k > 16 ? 0 : int((bits >> j) & 1u);
      Dsu conn = base;
      std::map<std::pair<int, int>, int> first;
      for (const Read& r : reads) {
        auto key = std::make_pair(r.parent, trial[r.cls]);
        auto it = first.find(key);
        if (it == first.end()) first[key] = r.node; else conn.unite(it->second, r.node);
      }
      bool one = true;
      for (int i = 1; i < m && one; ++i) one = conn.find(i) == conn.find(0);
      if (one) {
        if (order_out)
          for (int i = 0; i < m; ++i) {
            const int r = cls.find(i);
            (*order_out)[members[i]] = trial[r] == kFree ? 0 : trial[r];
          }
        return ACC_OK;
      }
    }
    return ACC_ERR_DISCONNECTED;
  }

  // The recomputing variant.  Orders are symbols: a constant (0, 1, a label) or the variable of
  // a stored copy / a scatter / a member nobody in the cluster reads (encoded -1 - local id),
  // which is 0 or 1.  Members are visited consumers first; each passes the orders it is asked
  // for on to its producers, slot by slot.
  int run_recompute(std::vector<int32_t>* order_out, int max_depth, std::vector<std::vector<int32_t>>* copies_out = nullptr) {
    const int m = (int)members.size();
    std::vector<std::vector<int>> asked(m);
    std::vector<int> bound(m, kFree);                    // value of variable i once a scan fixed it
    std::vector<uint8_t> read_inside(m, 0);
    std::vector<int> depth(m, 0);
    for (const Edge& e : g.edges)
      if (local[e.a] >= 0 && local[e.b] >= 0) read_inside[local[e.a]] = 1;
    auto resolve = [&](int o) { return o < 0 && bound[-1 - o] != kFree ? bound[-1 - o] : o; };
    auto ask = [&](int i, int o) {
      if (std::find(asked[i].begin(), asked[i].end(), o) == asked[i].end()) asked[i].push_back(o);
    };
    for (int i = m - 1; i >= 0; --i) {
      const int a = members[i];
      const int k = g.nodes[a].d.kind;
      if (man[a] || k == ACC_PERMUTE || !read_inside[i]) ask(i, -1 - i);
      if (k == ACC_SCANL || k == ACC_SCANR) {
        const int fixed = k == ACC_SCANL ? 0 : 1;
        for (int o : asked[i]) {
          const int r = resolve(o);
          if (r >= 0 && r != fixed) return ACC_ERR_ILLEGAL_TRAVERSAL;
          if (r < 0) bound[-1 - r] = fixed;
        }
        asked[i].assign(1, fixed);
      }
      for (const Edge& e : g.edges) {
        if (e.b != a || local[e.a] < 0) continue;
        const int c = slot_const(a, e.slot);
        for (int o : asked[i]) ask(local[e.a], c != kFree ? c : o);
      }
    }
    // depth of stacking, producers first
    int deepest = 0;
    for (int i = 0; i < m; ++i) {
      const int a = members[i];
      int d = 0;
      for (const Edge& e : g.edges)
        if (e.b == a && local[e.a] >= 0) d = std::max(d, depth[local[e.a]]);
      depth[i] = d + (gather_like(g.nodes[a]) ? 1 : 0);
      deepest = std::max(deepest, depth[i]);
    }
    if (deepest > max_depth) return ACC_ERR_ILLEGAL_TRAVERSAL;
    // connectivity: fused edges, or reads of one outside parent in one order
    Dsu base(m);
    for (const Edge& e : g.edges)
      if (local[e.a] >= 0 && local[e.b] >= 0) base.unite(local[e.a], local[e.b]);
    struct Read { int parent, order, node; };
    std::vector<Read> reads;
    for (const Edge& e : g.edges) {
      if (local[e.b] < 0 || local[e.a] >= 0 || !e.ordered) continue;
      if (slot_const(e.b, e.slot) != kFree) continue;
      for (int o : asked[local[e.b]]) reads.push_back({e.a, resolve(o), local[e.b]});
    }
    std::vector<int> free_var;
    for (const Read& r : reads)
      if (r.order < 0 && std::find(free_var.begin(), free_var.end(), r.order) == free_var.end()) free_var.push_back(r.order);
    const int k = (int)free_var.size();
    const uint32_t combos = k > 16 ? 1u : (1u << k);
    for (uint32_t bits = 0; bits < combos; ++bits) {
      auto value_of = [&](int o) {
        if (o >= 0) return o;
        for (int j = 0; j < k; ++j)
          if (free_var[j] == o) return k > 16 ? 0 : int((bits >> j) & 1u);
        return 0;
      };
      Dsu conn = base;
      std::map<std::pair<int, int>, int> first;
      for (const Read& r : reads) {
        auto key = std::make_pair(r.parent, value_of(r.order));
        auto it = first.find(key);
        if (it == first.end()) first[key] = r.node; else conn.unite(it->second, r.node);
      }
      bool one = true;
      for (int i = 1; i < m && one; ++i) one = conn.find(i) == conn.find(0);
      if (one) {
        if (order_out)
          for (int i = 0; i < m; ++i) {
            const int o = asked[i].empty() ? 0 : value_of(resolve(asked[i].front()));
            (*order_out)[members[i]] = o;
            if (copies_out) {
              std::vector<int32_t>& all = (*copies_out)[members[i]];
              all.clear();
              for (int q : asked[i]) {
                const int v = value_of(resolve(q));
                if (std::find(all.begin(), all.end(), v) == all.end()) all.push_back(v);
              }
            }
          }
        return ACC_OK;
      }
    }
    return ACC_ERR_DISCONNECTED;
  }
};

}  // namespace

// For a clustering of only some nodes (block_of[i] < 0: not placed yet): false if the placed
// nodes already break a rule of the paper's model that placing more nodes cannot mend: an
// infusible edge or a scatter and another reader of its destination inside one block, blocks
// that need each other's results, or order equalities without a solution.  `man` marks arrays
// that are manifest whatever happens to the nodes not placed yet.
bool partial_clustering_possible(const Graph& g, const std::vector<int>& block_of, int n_blocks, const std::vector<uint8_t>& man,
                                 bool check_orders) {
  const int n = (int)g.nodes.size();
  std::vector<std::vector<int>> after(n_blocks);
  std::vector<int> waiting(n_blocks, 0);
  auto link = [&](int from, int to) {
    if (std::find(after[from].begin(), after[from].end(), to) == after[from].end()) { after[from].push_back(to); ++waiting[to]; }
  };
  for (const Edge& e : g.edges) {
    if (block_of[e.a] < 0 || block_of[e.b] < 0) continue;
    if (block_of[e.a] == block_of[e.b]) { if (!e.fusible) return false; }
    else link(block_of[e.a], block_of[e.b]);
  }
  for (int j = 0; j < n; ++j) {
    if (g.nodes[j].d.kind != ACC_PERMUTE || block_of[j] < 0) continue;
    const int dest = g.nodes[j].d.inputs[0];
    for (const Edge& e : g.edges)
      if (e.a == dest && e.b != j && block_of[e.b] >= 0) {
        if (block_of[e.b] == block_of[j]) return false;
        link(block_of[e.b], block_of[j]);
      }
  }
  std::vector<int> ready;
  for (int b = 0; b < n_blocks; ++b)
    if (waiting[b] == 0) ready.push_back(b);
  int done = 0;
  while (!ready.empty()) {
    const int b = ready.back();
    ready.pop_back();
    ++done;
    for (int t : after[b])
      if (--waiting[t] == 0) ready.push_back(t);
  }
  if (done != n_blocks) return false;
  if (!check_orders) return true;
  std::vector<int> label(n, 0);
  int next = 2;
  for (int i = 0; i < n; ++i)
    if (gather_like(g.nodes[i])) label[i] = next++;
  std::vector<std::vector<int>> members(n_blocks);
  for (int i = 0; i < n; ++i)
    if (block_of[i] >= 0) members[block_of[i]].push_back(i);
  for (int b = 0; b < n_blocks; ++b) {
    if (members[b].size() < 2) continue;
    ClusterCheck cc(g, members[b], man, label);
    if (cc.run(nullptr, false) != ACC_OK) return false;
  }
  return true;
}

// Arrays that are manifest in every clustering of the paper's model: program outputs, arrays
// nobody reads, arrays with an infusible out-edge, arrays read through a gather-like source slot
// and by anyone else (fused with the gather-like reader its order is that reader's label, which
// no second reader and no stored copy can have), arrays read by a scanl and a scanr.  must_read
// marks those of them (and the inputs) that some cluster is sure to read from memory.
void forced_manifest(const Graph& g, std::vector<uint8_t>& forced, std::vector<uint8_t>& must_read) {
  const int n = (int)g.nodes.size();
  forced.assign(n, 0);
  must_read.assign(n, 0);
  std::vector<int> readers(n, 0), label_readers(n, 0), array_readers(n, 0);
  std::vector<uint8_t> infusible(n, 0), scanl(n, 0), scanr(n, 0);
  for (const Edge& e : g.edges) {
    ++readers[e.a];
    const Node& b = g.nodes[e.b];
    const bool array_slot = e.slot < b.d.n_array_inputs;
    if (array_slot) ++array_readers[e.a];
    if (!e.fusible && array_slot) infusible[e.a] = 1;
    if (!e.fusible) forced[e.a] = 1;
    if (b.d.kind == ACC_BACKPERMUTE || (b.d.kind == ACC_GATHER && e.slot == 1)) ++label_readers[e.a];
    if (b.d.kind == ACC_SCANL) scanl[e.a] = 1;
    if (b.d.kind == ACC_SCANR) scanr[e.a] = 1;
  }
  for (int i = 0; i < n; ++i) {
    const bool clash = (label_readers[i] > 0 && readers[i] > 1) || (scanl[i] && scanr[i]);
    if (is_input(g.nodes[i]) || g.nodes[i].output || readers[i] == 0 || clash) forced[i] = 1;
    must_read[i] = (is_input(g.nodes[i]) && array_readers[i] > 0) || infusible[i] || clash;
  }
}

int check_partition(const Graph& g, const int32_t* pi, Solution* sol, bool quiet, int recompute_depth) {
  const int n = (int)g.nodes.size();
  auto fail = [&](int code, const char* what, int a, int b) {
    return quiet ? code : set_error(code, "illegal clustering: %s (nodes %d, %d)", what, a, b);
  };
  for (const Edge& e : g.edges) {
    if (is_input(g.nodes[e.a])) continue;
    if (pi[e.a] > pi[e.b]) return fail(ACC_ERR_ILLEGAL_ORDER, "a consumer runs before its producer", e.a, e.b);
    if (!e.fusible && pi[e.a] == pi[e.b]) return fail(ACC_ERR_ILLEGAL_INFUSIBLE, "infusible edge inside one cluster", e.a, e.b);
  }
  for (int j = 0; j < n; ++j) {
    if (g.nodes[j].d.kind != ACC_PERMUTE) continue;
    const int dest = g.nodes[j].d.inputs[0];
    for (const Edge& e : g.edges)
      if (e.a == dest && e.b != j && !(pi[e.b] < pi[j]))
        return fail(ACC_ERR_ILLEGAL_SCATTER, "another use of a scatter destination is not earlier", e.b, j);
  }
  std::vector<uint8_t> man;
  manifest_of(g, pi, man);
  std::vector<int> label(n, 0);
  int next = 2;
  for (int i = 0; i < n; ++i)
    if (gather_like(g.nodes[i])) label[i] = next++;
  std::map<int, std::vector<int>> clusters;
  for (int i = 0; i < n; ++i)
    if (!is_input(g.nodes[i])) clusters[pi[i]].push_back(i);
  std::vector<int32_t> order(n, -1);
  std::vector<std::vector<int32_t>> copies(n);
  for (auto& kv : clusters) {
    ClusterCheck cc(g, kv.second, man, label);
    int rc = cc.run(&order);                             // a cluster of the paper's model needs no copies
    if (rc != ACC_OK && recompute_depth > 0) rc = cc.run_recompute(&order, recompute_depth, &copies);
    if (rc != ACC_OK)
      return fail(rc, rc == ACC_ERR_DISCONNECTED ? "a cluster does not hang together through a fused array"
                                                 : "traversal orders cannot be matched",
                  kv.second.front(), kv.second.back());
  }
  if (sol) {
    sol->manifest = man;
    sol->order = order;
    sol->copies = copies;
  }
  return ACC_OK;
}

}  // namespace acc
