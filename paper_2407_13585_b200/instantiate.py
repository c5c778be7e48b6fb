"""Emits the build-time kernel instantiations of a program.

Fused kernels are compiled ahead of time, one per distinct cluster.  Given a program
(a list of node records as in `workloads/programs.py`), this prints a C++ translation
unit for `csrc/programs/` that describes the program as a constexpr table and
instantiates every cluster that occurs in any legal clustering of it (enumerated by
the library's own legality checker), plus every node alone.

    python -m paper_2407_13585_b200.instantiate [--fixed-shifts] workloads:simple1 workloads:random_program:3,64,5 > csrc/programs/prog_x.cu

(`module:function[:int,...]` names a program; the integers are the function's arguments.)

Clusters the kernel skeletons cannot express are skipped and listed in a comment: a
scan whose values are consumed inside its own cluster other than element for element, and a fold
that is both written to memory and consumed inside its own cluster.
"""
import importlib
import sys

from . import binding as B

_KIND = {"foldseg": "ACC_FOLDSEG", "input": "ACC_INPUT", "generate": "ACC_GENERATE", "map": "ACC_MAP", "zipwith": "ACC_ZIPWITH",
         "backpermute": "ACC_BACKPERMUTE", "gather": "ACC_GATHER", "permute": "ACC_PERMUTE", "fold": "ACC_FOLD",
         "scanl": "ACC_SCANL", "scanr": "ACC_SCANR"}
_DT = {"f32": "ACC_F32", "i32": "ACC_I32", "u32": "ACC_U32"}


def clusters_of(prog):
    """Distinct clusters (frozensets of node ids) over all legal clusterings, singletons included."""
    g = B.Graph(prog.nodes, prog.outputs)
    found = set()
    for pi in g.enumerate():
        blocks = {}
        for i, c in enumerate(pi):
            if c >= 0:
                blocks.setdefault(c, set()).add(i)
        found.update(frozenset(b) for b in blocks.values())
    return sorted(found, key=lambda s: (len(s), sorted(s)))


def scans_consumed_in_place(prog, members):
    """Whether every scan of the cluster that is consumed inside it is consumed element for element: only
    array operands of map and zipWith and the index operand of a gather lead from a consumer to the scan,
    and no consumer needs two scans or is itself a fold, a scan or a scatter."""
    nodes = prog.nodes
    needs = {}                                   # member -> scans of the cluster it consumes
    for i in sorted(members):
        nd = nodes[i]
        mine = set()
        for slot, j in enumerate(nd.inputs):
            if j not in members:
                continue
            got = {j} if nodes[j].kind in ("scanl", "scanr") else needs[j]
            if not got:
                continue
            in_place = (nd.kind in ("map", "zipwith") and slot < nd.n_array) or (nd.kind == "gather" and slot == 0)
            if not in_place:
                return False
            mine |= got
        if len(mine) > 1:
            return False
        needs[i] = mine
    return True


def expressible(prog, members):
    nodes = prog.nodes
    if not scans_consumed_in_place(prog, members):
        return False
    for i in members:
        k = nodes[i].kind
        inside = [j for j in members if i in nodes[j].inputs]
        outside = i in prog.outputs or any(i in nodes[j].inputs for j in range(len(nodes)) if j not in members)
        if k == "fold" and inside and outside:
            return False
        if k == "foldseg" and outside:
            # a segmented fold that is written shares its kernel with other such folds only
            others = [j for j in members if j != i and (j in prog.outputs or any(
                j in nodes[c].inputs for c in range(len(nodes)) if c not in members))]
            if any(nodes[j].kind != "foldseg" or nodes[j].inputs[1] != nodes[i].inputs[1] for j in others):
                return False
        if k == "foldseg" and inside and outside:
            return False
    return True


def emit(prog, out):
    name = prog.name
    n = len(prog.nodes)
    outputs = " | ".join("(1ull << %d)" % o for o in prog.outputs) or "0"
    out.write("constexpr CProgram make_%s() {\n  CProgram p{%d, %s, {}};\n" % (name, n, outputs))
    for i, nd in enumerate(prog.nodes):
        rank = len(nd.shape)
        if nd.kind == "input":
            out.write("  p.nodes[%d] = pnode(ACC_INPUT, %s, %d, 0, 0, 0);\n" % (i, _DT[nd.dtype], rank))
            continue
        fn = "ACC_FN_" + nd.fn.upper() if nd.fn else "0"
        idx = "ACC_IDX_" + nd.idx_fn.upper() if nd.idx_fn else "0"
        ins = "".join(", %d" % s for s in nd.inputs)
        node = "pnode(%s, %s, %d, %s, %s, %d%s)" % (_KIND[nd.kind], _DT[nd.dtype], rank, fn, idx, nd.n_array, ins)
        # constants that select code: a seeded exclusive scan; with --fixed-shifts the offsets of clamped
        # shifts within -1..1 (kernels for run-time offsets are what the library falls back to)
        if nd.kind in ("scanl", "scanr") and getattr(nd, "exclusive", False):
            node = "fixed(%s, 1, kRunTime)" % node
        elif FIXED_SHIFTS and nd.kind == "backpermute" and nd.idx_fn == "shift_clamp" and all(-1 <= v <= 1 for v in nd.iparam[:2]):
            node = "fixed(%s, %d, %d)" % (node, nd.iparam[0], nd.iparam[1])
        out.write("  p.nodes[%d] = %s;  // %s\n" % (i, node, nd.name))
    out.write("  return p;\n}\ninline constexpr CProgram k_%s = make_%s();\n" % (name, name))
    skipped = []
    for members in clusters_of(prog):
        mask = sum(1 << i for i in members)
        tag = "_".join(prog.nodes[i].name or str(i) for i in sorted(members))
        if expressible(prog, members):
            out.write("ACC_CLUSTER(k_%s, 0x%X, %s__%s)\n" % (name, mask, name, tag))
        else:
            skipped.append(tag)
    if skipped:
        out.write("// not instantiated (outside the skeletons): %s\n" % ", ".join(skipped))
    out.write("\n")


FIXED_SHIFTS = False


def main(argv):
    global FIXED_SHIFTS
    if "--fixed-shifts" in argv:
        FIXED_SHIFTS = True
        argv = [a for a in argv if a != "--fixed-shifts"]
    out = sys.stdout
    out.write("// Generated by `python -m paper_2407_13585_b200.instantiate %s`.\n" % " ".join(argv))
    out.write("// Every cluster of every legal clustering of the programs named above, and every node alone.\n")
    out.write('#include "device/launch.cuh"\n\nnamespace acc {\n\n')
    for spec in argv:
        mod, fn, *rest = spec.split(":")                  # module:function[:int,int,...]
        prog = getattr(importlib.import_module(mod), fn)(*[int(v) for v in rest[0].split(",")] if rest else [])
        emit(prog, out)
    out.write("}  // namespace acc\n")


if __name__ == "__main__":
    main(sys.argv[1:])
