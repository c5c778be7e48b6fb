// Cluster descriptions shared by the build-time kernel instantiations and the run-time
// matcher.  A cluster is a small program of its own: local nodes in topological order,
// each either EXTERNAL (an array produced outside the cluster and read from memory) or a
// MEMBER (a combinator evaluated inside the kernel), with a manifest flag per member
// (m_a = 0 in the paper's Figure 3: the array is written to memory).
//
// Build time: `extract(program, mask)` cuts a cluster out of a constexpr program.
// Run time: the executor cuts it out of the caller's graph in the same way.  Both give
// the same structure for the same sub-DAG, and `signature()` of that structure is the
// registry key, so a kernel instantiated for one program serves every program that
// contains the same sub-DAG (e.g. each iteration of a Jacobi chain).
#pragma once
#include <cstdint>
#include <cstdio>
#include <string>

#include "acc.h"

namespace acc {

constexpr int kMaxSlots = ACC_MAX_INPUTS;
constexpr int kMaxCluster = 40;   // local nodes per cluster
constexpr int kMaxProgram = 40;   // nodes per build-time program

// Constants of a node that select code instead of being run-time arguments: the row and
// column offsets of a clamped shift when both lie in -1..1 (kRunTime: not fixed), p0 = 1 for a
// seeded exclusive scan, and p0 = kPow2 for a modulus that is a power of two.  Except for the
// scan's, a kernel built with kRunTime in their place serves every value.
constexpr int kRunTime = 9;
// p0 of a map with ACC_FN_MUL_MOD: the modulus is a power of two (v mod d is one AND in such a kernel).
constexpr int kPow2 = 1;

struct PNode {                    // node of a build-time program
  int kind = 0, dtype = 0, rank = 0, fn = 0, idxfn = 0, nin = 0, narr = 0;
  int in[kMaxSlots] = {};
  int p0 = kRunTime, p1 = kRunTime;
};

struct CProgram {
  int n;
  uint64_t outputs;               // bit i: node i is a program output
  PNode nodes[kMaxProgram];
};

struct CNode {
  int kind = 0, dtype = 0, rank = 0, fn = 0, idxfn = 0, nin = 0, narr = 0;
  int in[kMaxSlots] = {};         // local ids
  bool member = false, manifest = false;
  int p0 = kRunTime, p1 = kRunTime;
};

struct CCluster {
  int n;
  int source[kMaxCluster];        // id in the program / graph the cluster was cut from
  CNode nodes[kMaxCluster];
};

constexpr PNode pnode(int kind, int dtype, int rank, int fn, int idxfn, int narr,
                      int i0 = -1, int i1 = -1, int i2 = -1, int i3 = -1, int i4 = -1, int i5 = -1) {
  PNode p{kind, dtype, rank, fn, idxfn, 0, narr, {i0, i1, i2, i3, i4, i5}};
  for (int s = 0; s < kMaxSlots; ++s)
    if (p.in[s] >= 0) p.nin = s + 1;
  return p;
}

// The same node with its two constants fixed at build time.
constexpr PNode fixed(PNode p, int p0, int p1) {
  p.p0 = p0;
  p.p1 = p1;
  return p;
}

// Cuts the members selected by `mask` out of `p`.  A member is manifest if it is a
// program output, has no consumer, or has a consumer outside the mask.
constexpr CCluster extract(const CProgram& p, uint64_t mask) {
  CCluster c{};
  int local[kMaxProgram] = {};
  for (int i = 0; i < kMaxProgram; ++i) local[i] = -1;
  for (int i = 0; i < p.n; ++i) {
    if (!((mask >> i) & 1)) continue;
    const PNode& nd = p.nodes[i];
    for (int s = 0; s < nd.nin; ++s) {
      const int a = nd.in[s];
      if (local[a] < 0) {               // an external, first used here
        CNode e{ACC_INPUT, p.nodes[a].dtype, p.nodes[a].rank, 0, 0, 0, 0, {-1, -1, -1, -1, -1, -1}, false, true};
        local[a] = c.n;
        c.source[c.n] = a;
        c.nodes[c.n++] = e;
      }
    }
    CNode m{nd.kind, nd.dtype, nd.rank, nd.fn, nd.idxfn, nd.nin, nd.narr, {-1, -1, -1, -1, -1, -1}, true, false};
    for (int s = 0; s < nd.nin; ++s) m.in[s] = local[nd.in[s]];
    m.p0 = nd.p0;
    m.p1 = nd.p1;
    bool consumed = false, outside = false;
    for (int j = i + 1; j < p.n; ++j)
      for (int s = 0; s < p.nodes[j].nin; ++s)
        if (p.nodes[j].in[s] == i) {
          consumed = true;
          if (!((mask >> j) & 1)) outside = true;
        }
    m.manifest = ((p.outputs >> i) & 1) || !consumed || outside;
    local[i] = c.n;
    c.source[c.n] = i;
    c.nodes[c.n++] = m;
  }
  return c;
}

// Registry key of a cluster: everything that selects code, nothing that is a run-time
// value (shapes, constants, pointers).
inline std::string signature(const CCluster& c) {
  std::string s;
  char buf[64];
  for (int i = 0; i < c.n; ++i) {
    const CNode& nd = c.nodes[i];
    if (!nd.member) {
      snprintf(buf, sizeof buf, "E%d.%d;", nd.dtype, nd.rank);
      s += buf;
      continue;
    }
    snprintf(buf, sizeof buf, "M%d.%d.%d.%d.%d.%d.%d.%d.%d(", nd.kind, nd.dtype, nd.rank, nd.fn, nd.idxfn, nd.narr, (int)nd.manifest,
             nd.p0, nd.p1);
    s += buf;
    for (int k = 0; k < nd.nin; ++k) {
      snprintf(buf, sizeof buf, "%d,", nd.in[k]);
      s += buf;
    }
    s += ");";
  }
  return s;
}

}  // namespace acc
