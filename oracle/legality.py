"""Which clusterings of a combinator program are legal (test infrastructure, CPU only).

Follows the paper's integer-programming model (Figure 3) and the top-level
rules of Section 3.4, evaluated for a *given* assignment pi of nodes to cluster
numbers instead of being solved:

  * every edge (a, b) needs pi_a <= pi_b, an infusible one pi_a < pi_b; two
    nodes of one cluster joined by a fusible edge are fused (x_ab = 0 is then
    forced by  x_ab <= pi_b - pi_a <= n * x_ab);
  * infusible edges: out of a program input; into a free-variable (indexed)
    slot; into the destination slot of a scatter and out of a scatter's
    result; through force();
  * a scatter comes strictly after every other consumer of its destination;
  * an array is fused away (m_a = 1) only if all of its out-edges are fused
    and it is not a program output; otherwise it is manifest and its order
    d^o_a is 0 or 1;
  * a fused edge needs d^o_a = d^i of the consuming slot, where map, zipWith
    and fold read every array slot in their own output order, a gather reads
    its index slot in its output order and its source slot in its own label,
    a backpermute (generate + gather already fused) reads its source in its
    label, scanl is all-0, scanr all-1, and a scatter reads index and value
    slots in one common order that is 0 or 1;
  * the nodes of a cluster hang together through fused edges or through a
    common parent outside the cluster read in the same order (Section 4.1's
    splitting step, with parents added once per order; Section 3.4 asks for
    at least one horizontally/vertically/diagonally fused array per merge).

The search over the free 0/1 orders of the manifest nodes of a cluster is
done by plain enumeration.

Clusterings that recompute (`recompute=k > 0`; not in the paper, whose
Section 6 leaves fusion that duplicates work to future work).  The model is
the paper's own, applied to an unfolded cluster: every member that is stored
(manifest), is a scatter, or has no reader inside the cluster is a root, and
below each root the cluster is unfolded into a tree in which every reader has
a private copy of each producer it reads inside the cluster.  A copy has one
reader, so its order is simply the order of the slot that reads it; roots are
0 or 1; a copy of a scan must come out in the scan's own order; copies of
gather-like nodes carry labels of their own.  No path of the tree may hold
more than k gather-like nodes (a cluster that is legal without copies is
legal whatever its depth).  Whether the cluster hangs together is judged
on the original members: through fused edges, or through a common outside
parent that copies of two members read in the same order.
"""
from itertools import product


class Edge:
    __slots__ = ("a", "b", "slot", "fusible", "ordered")

    def __init__(self, a, b, slot, fusible, ordered):
        self.a, self.b, self.slot, self.fusible, self.ordered = a, b, slot, fusible, ordered


def edges_of(nodes):
    """One edge per input slot, classified fusible/infusible and ordered/unordered."""
    out = []
    for b, nd in enumerate(nodes):
        for s, a in enumerate(nd.inputs):
            pa = nodes[a]
            free = s >= nd.n_array
            dest = nd.kind == "permute" and s == 0
            forced = s in tuple(getattr(nd, "force", ()))
            from_scatter = pa.kind == "permute"
            ordered = not (free or dest or forced or from_scatter)
            fusible = ordered and pa.kind != "input"
            out.append(Edge(a, b, s, fusible, ordered))
    return out


def graph_sets(nodes):
    """(F, I) as sets of node pairs, the form the paper prints a graph in."""
    F, I = set(), set()
    for e in edges_of(nodes):
        (F if e.fusible else I).add((e.a, e.b))
    return F - I, I


def labels_of(nodes):
    """A unique label 2..g+1 for every gather-like node."""
    lab, nxt = {}, 2
    for i, nd in enumerate(nodes):
        if nd.kind in ("gather", "backpermute"):
            lab[i] = nxt
            nxt += 1
    return lab


def _slot_order(nodes, lab, d, b, slot):
    """d^i of slot `slot` of node b, given b's own order d[b]."""
    k = nodes[b].kind
    if k == "gather":
        return d[b] if slot == 0 else lab[b]
    if k == "backpermute":
        return lab[b]
    return d[b]


def manifest_set(nodes, outputs, pi, edges):
    """Nodes whose array is written to memory under pi (m_a = 0)."""
    man = set()
    has_out = set()
    for e in edges:
        has_out.add(e.a)
        if pi[e.a] != pi[e.b] or not e.fusible:
            man.add(e.a)
    for i, nd in enumerate(nodes):
        if nd.kind == "input" or i in outputs or i not in has_out:
            man.add(i)
    return man


def check(nodes, outputs, pi, recompute=0):
    """(True, "") if pi is legal, else (False, reason).  pi[i] is ignored for inputs."""
    ok, why, _ = solve(nodes, outputs, pi, recompute)
    return ok, why


def solve(nodes, outputs, pi, recompute=0):
    """check() plus, when legal, one satisfying order d^o per node (for a scatter: the
    order of its index/value slots; under recompute: the order of a node's first copy)."""
    edges = edges_of(nodes)
    is_in = [nd.kind == "input" for nd in nodes]
    for e in edges:
        if is_in[e.a]:
            continue
        if pi[e.a] > pi[e.b]:
            return False, f"order: edge {e.a}->{e.b} runs backwards", None
        if not e.fusible and pi[e.a] == pi[e.b]:
            return False, f"infusible: edge {e.a}->{e.b} inside one cluster", None
    for j, nd in enumerate(nodes):
        if nd.kind != "permute":
            continue
        dest = nd.inputs[0]
        for e in edges:
            if e.a == dest and e.b != j and not pi[e.b] < pi[j]:
                return False, f"scatter: node {e.b} also uses the destination of {j} and is not earlier", None
    man = manifest_set(nodes, outputs, pi, edges)
    lab = labels_of(nodes)
    clusters = {}
    for i in range(len(nodes)):
        if not is_in[i]:
            clusters.setdefault(pi[i], []).append(i)
    orders = {}
    for c in sorted(clusters):
        ok, why, d = _cluster_ok(nodes, edges, clusters[c], man, lab, pi)
        if not ok and recompute:                    # a cluster of the paper's model needs no copies
            ok, why, d = _cluster_ok_recompute(nodes, edges, clusters[c], man, recompute)
        if not ok:
            return False, f"cluster {c}: {why}", None
        orders.update(d)
    return True, "", orders


def _cluster_ok(nodes, edges, members, man, lab, pi):
    mset = set(members)
    inner = [e for e in edges if e.a in mset and e.b in mset]          # all fused (fusible, same cluster)
    outer = [e for e in edges if e.b in mset and e.a not in mset and e.ordered]
    consumers = {a: [e for e in inner if e.a == a] for a in members}
    fixed = {}
    free_nodes = []
    for a in members:
        k = nodes[a].kind
        if k == "scanl":
            fixed[a] = 0
        elif k == "scanr":
            fixed[a] = 1
        elif a in man or k == "permute":
            free_nodes.append(a)
    why = "traversal orders cannot be matched"
    for choice in product((0, 1), repeat=len(free_nodes)):
        d = dict(fixed)
        d.update(zip(free_nodes, choice))
        ok = True
        for a in reversed(members):                 # consumers come later in program order
            want = {_slot_order(nodes, lab, d, e.b, e.slot) for e in consumers[a]}
            if a in d:
                if any(w != d[a] for w in want):
                    ok = False
            elif len(want) == 1:
                d[a] = want.pop()
            else:
                ok = False
            if not ok:
                break
            if a in man and nodes[a].kind != "permute" and d[a] > 1:
                ok = False
                break
        if not ok:
            continue
        if _connected(nodes, members, inner, outer, lab, d):
            return True, "", d
        why = "disconnected: no fused array links all of its nodes"
    return False, why, None


def _cluster_ok_recompute(nodes, edges, members, man, max_depth):
    """The unfolded-tree model described in the module text."""
    mset = set(members)
    inner = [e for e in edges if e.a in mset and e.b in mset]
    outer = [e for e in edges if e.b in mset and e.a not in mset and e.ordered]
    producers = {b: [e for e in inner if e.b == b] for b in members}
    read_inside = {e.a for e in inner}
    roots = [a for a in members if a in man or nodes[a].kind == "permute" or a not in read_inside]

    # depth of stacking first: it also bounds the size of the tree
    depth = {}
    for a in members:                                  # producers come earlier in program order
        below = max((depth[e.a] for e in producers[a]), default=0)
        depth[a] = below + (1 if nodes[a].kind in ("gather", "backpermute") else 0)
    if max(depth.values()) > max_depth:
        return False, f"more than {max_depth} gather-like nodes stacked on a fused path", None

    # the tree: copies[i] = (node, reader copy or None, slot of the reader)
    copies = []

    def unfold(a, reader, slot):
        me = len(copies)
        copies.append((a, reader, slot))
        for e in producers[a]:
            unfold(e.a, me, e.slot)

    for r in roots:
        unfold(r, None, None)

    def label_slot(b, slot):
        k = nodes[b].kind
        return k == "backpermute" or (k == "gather" and slot == 1)

    why = "traversal orders cannot be matched"
    for choice in product((0, 1), repeat=len(roots)):
        root_order = dict(zip(roots, choice))
        d = []
        ok = True
        for i, (a, reader, slot) in enumerate(copies):
            if reader is None:
                o = root_order[a]
            elif label_slot(copies[reader][0], slot):
                o = ("label", reader)                  # the reader copy's own label: shared with nobody
            else:
                o = d[reader]
            k = nodes[a].kind
            if k == "scanl" and o != 0 or k == "scanr" and o != 1:
                ok = False
                break
            d.append(o)
        if not ok:
            continue
        # hanging together, on the original members
        parent = {a: a for a in members}

        def find(x):
            while parent[x] != x:
                parent[x] = parent[parent[x]]
                x = parent[x]
            return x

        for e in inner:
            parent[find(e.a)] = find(e.b)
        groups = {}
        for i, (a, _, _) in enumerate(copies):
            for e in outer:
                if e.b == a and not label_slot(a, e.slot):
                    groups.setdefault((e.a, d[i]), []).append(a)
        for g in groups.values():
            for b in g[1:]:
                parent[find(g[0])] = find(b)
        if len({find(a) for a in members}) == 1:
            first = {}
            for i, (a, _, _) in enumerate(copies):
                first.setdefault(a, d[i] if not isinstance(d[i], tuple) else 2 + d[i][1])
            return True, "", first
        why = "disconnected: no fused array links all of its nodes"
    return False, why, None


def _connected(nodes, members, inner, outer, lab, d):
    parent = {a: a for a in members}

    def find(x):
        while parent[x] != x:
            parent[x] = parent[parent[x]]
            x = parent[x]
        return x

    for e in inner:
        parent[find(e.a)] = find(e.b)
    groups = {}
    for e in outer:
        key = (e.a, _slot_order(nodes, lab, d, e.b, e.slot))
        groups.setdefault(key, []).append(e.b)
    for g in groups.values():
        for b in g[1:]:
            parent[find(g[0])] = find(b)
    return len({find(a) for a in members}) == 1


def _set_partitions(items):
    """All set partitions of a list, as lists of blocks."""
    if not items:
        yield []
        return
    first, rest = items[0], items[1:]
    for part in _set_partitions(rest):
        for i in range(len(part)):
            yield part[:i] + [[first] + part[i]] + part[i + 1:]
        yield [[first]] + part


def canonical_pi(nodes, blocks):
    """Number the blocks in an execution order that respects every edge and the
    scatter rule (ties: the block holding the smallest node id first).
    Returns None when the blocks cannot be ordered."""
    edges = edges_of(nodes)
    blk = {}
    for bi, b in enumerate(blocks):
        for a in b:
            blk[a] = bi
    before = {bi: set() for bi in range(len(blocks))}
    for e in edges:
        if e.a in blk and blk[e.a] != blk[e.b]:
            before[blk[e.b]].add(blk[e.a])
    for j, nd in enumerate(nodes):
        if nd.kind == "permute":
            for e in edges:
                if e.a == nd.inputs[0] and e.b != j:
                    if blk[e.b] == blk[j]:
                        return None
                    before[blk[j]].add(blk[e.b])
    order, done = [], set()
    while len(order) < len(blocks):
        ready = [bi for bi in range(len(blocks)) if bi not in done and before[bi] <= done]
        if not ready:
            return None
        nxt = min(ready, key=lambda bi: min(blocks[bi]))
        order.append(nxt)
        done.add(nxt)
    pi = [-1] * len(nodes)
    for num, bi in enumerate(order):
        for a in blocks[bi]:
            pi[a] = num
    return pi


def enumerate_partitions(nodes, outputs, recompute=0):
    """Every legal clustering, each as a canonical pi list (inputs get -1), sorted."""
    items = [i for i, nd in enumerate(nodes) if nd.kind != "input"]
    found = []
    for blocks in _set_partitions(items):
        pi = canonical_pi(nodes, blocks)
        if pi is None:
            continue
        if check(nodes, outputs, pi, recompute)[0]:
            found.append(pi)
    return sorted(found)


def traffic(nodes, outputs, pi, weight=lambda nd: 1):
    """(reads, writes) of arrays under pi, each array weighted by weight(node).

    An array is read once per (consuming cluster, order) from outside that
    cluster -- consumers of one cluster that read it in one order share the
    read -- and written once if it is manifest.  Free-variable reads touch a
    single element and are not counted.
    """
    edges = edges_of(nodes)
    man = manifest_set(nodes, outputs, pi, edges)
    lab = labels_of(nodes)
    ok, why, d = solve(nodes, outputs, pi)
    if not ok:
        raise ValueError(why)
    reads = set()
    for e in edges:
        inside = nodes[e.a].kind != "input" and pi[e.a] == pi[e.b]
        if inside or e.slot >= nodes[e.b].n_array:
            continue
        order = _slot_order(nodes, lab, d, e.b, e.slot) if e.ordered else ("unordered", e.b, e.slot)
        reads.add((e.a, pi[e.b], order))
    r = sum(weight(nodes[a]) for a, _, _ in reads)
    w = sum(weight(nodes[a]) for a in man if nodes[a].kind != "input")
    return r, w


def unfold_copies(nodes, outputs, pi, copies):
    """A clustering with copies, written out: (nodes2, outputs2, pi2, home, copy_ids).

    `copies` are (node, cluster) pairs: readers of the node inside that cluster read a copy that
    is evaluated there.  Every copy becomes a node of its own right after the node it copies; a
    node instance in cluster c reads, input by input, the instance of the input that lives in c
    (the input itself or its copy there), else the input itself.  home[i] is where node i went.
    """
    import copy as _copy
    nodes2, pi2, home, copy_ids = [], [], {}, {}

    def instance(x, cluster):
        if nodes[x].kind != "input" and pi[x] != cluster and (x, cluster) in copy_ids:
            return copy_ids[(x, cluster)]
        return home[x]

    for i, nd in enumerate(nodes):
        places = [None] + [c for a, c in copies if a == i]
        for c in places:
            cluster = (-1 if nd.kind == "input" else pi[i]) if c is None else c
            m = _copy.copy(nd)
            m.inputs = tuple(instance(x, cluster) for x in nd.inputs)
            nodes2.append(m)
            pi2.append(cluster)
            if c is None:
                home[i] = len(nodes2) - 1
            else:
                copy_ids[(i, c)] = len(nodes2) - 1
    return nodes2, [home[o] for o in outputs], pi2, home, copy_ids


def check_with_copies(nodes, outputs, pi, copies, recompute=0):
    """Legality of a clustering with copies: the written-out clustering is legal and no copy is stored."""
    for a, c in copies:
        if nodes[a].kind == "input" or c == pi[a] or copies.count((a, c)) > 1:
            return False, "bad copy"
    nodes2, outputs2, pi2, home, copy_ids = unfold_copies(nodes, outputs, pi, copies)
    ok, why = check(nodes2, outputs2, pi2, recompute)
    if not ok:
        return False, why
    man = manifest_set(nodes2, outputs2, pi2, edges_of(nodes2))
    for key, j in copy_ids.items():
        if j in man:
            return False, f"the copy of node {key[0]} in cluster {key[1]} would be stored"
    return True, ""
