"""ctypes binding of libacc.so: argument marshalling only, same names as include/acc.h.

Every step of a program runs in the library's CUDA kernels; this module converts
node records to `acc_node_desc`, passes tensor addresses and the current CUDA
stream, and turns negative status codes into exceptions.  There is no CPU
fallback: loading fails if the library has not been built.
"""
import ctypes as C
import os
import re

HERE = os.path.dirname(os.path.abspath(__file__))
HEADER = os.path.join(os.path.dirname(HERE), "include", "acc.h")
LIB_PATH = os.path.join(HERE, "libacc.so")

MAX_INPUTS = 6


def _parse_enums(path):
    """{enumerator: value} for every enum of the header (values counted as a C compiler does)."""
    text = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
    out = {}
    for body in re.findall(r"enum\s+\w+\s*\{(.*?)\}", text, flags=re.S):
        nxt = 0
        for item in body.split(","):
            item = item.strip()
            if not item:
                continue
            if "=" in item:
                name, val = (t.strip() for t in item.split("=", 1))
                nxt = int(val, 0)
            else:
                name = item
            out[name] = nxt
            nxt += 1
    return out


ENUM = _parse_enums(HEADER)
KIND = {k[4:].lower(): v for k, v in ENUM.items()
        if k in ("ACC_INPUT", "ACC_GENERATE", "ACC_MAP", "ACC_ZIPWITH", "ACC_BACKPERMUTE", "ACC_GATHER",
                 "ACC_PERMUTE", "ACC_FOLD", "ACC_FOLDSEG", "ACC_SCANL", "ACC_SCANR")}
DTYPE = {"f32": ENUM["ACC_F32"], "i32": ENUM["ACC_I32"], "u32": ENUM["ACC_U32"]}
FN = {k[7:].lower(): v for k, v in ENUM.items() if k.startswith("ACC_FN_")}
IDX_FN = {k[8:].lower(): v for k, v in ENUM.items() if k.startswith("ACC_IDX_")}
STATUS_NAME = {v: k for k, v in ENUM.items() if k.startswith("ACC_ERR_") or k == "ACC_OK"}
FUSED, UNFUSED = ENUM["ACC_EXEC_FUSED"], ENUM["ACC_EXEC_UNFUSED"]
PLAN = {"unfused": ENUM["ACC_PLAN_UNFUSED"], "enumerate": ENUM["ACC_PLAN_ENUMERATE"],
        "greedy_topdown": ENUM["ACC_PLAN_GREEDY_TOPDOWN"], "greedy_bottomup": ENUM["ACC_PLAN_GREEDY_BOTTOMUP"],
        "branch_bound": ENUM["ACC_PLAN_BRANCH_BOUND"]}
COST = {k[9:].lower(): v for k, v in ENUM.items() if k.startswith("ACC_COST_")}


class NodeDesc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("dtype", C.c_int32), ("rank", C.c_int32), ("shape", C.c_int64 * 2),
                ("n_inputs", C.c_int32), ("inputs", C.c_int32 * MAX_INPUTS), ("n_array_inputs", C.c_int32),
                ("fn_id", C.c_int32), ("idx_fn_id", C.c_int32), ("iparam", C.c_int64 * 4),
                ("fparam", C.c_double * 4), ("flags", C.c_uint32)]


class AccError(RuntimeError):
    def __init__(self, code, message):
        super().__init__("%s (%d): %s" % (STATUS_NAME.get(code, "?"), code, message))
        self.code = code
        self.status = STATUS_NAME.get(code, "?")


def load_library(path=LIB_PATH):
    if not os.path.exists(path):
        raise ImportError("%s is missing: build it with `python -m paper_2407_13585_b200.build`" % path)
    lib = C.CDLL(path)
    p, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    pi32 = C.POINTER(C.c_int32)
    sig = {
        "acc_graph_create": (C.c_int, [C.POINTER(p)]),
        "acc_graph_destroy": (C.c_int, [p]),
        "acc_add_node": (i32, [p, C.POINTER(NodeDesc)]),
        "acc_mark_output": (C.c_int, [p, i32]),
        "acc_node_count": (i32, [p]),
        "acc_edges": (C.c_int, [p, pi32, pi32, pi32, pi32, i32]),
        "acc_set_partition": (C.c_int, [p, pi32, i32]),
        "acc_check_partition": (C.c_int, [p, pi32, i32]),
        "acc_get_partition": (C.c_int, [p, pi32, i32]),
        "acc_manifest": (C.c_int, [p, pi32, i32]),
        "acc_plan": (C.c_int, [p, C.c_int, C.c_int, pi32]),
        "acc_enumerate": (i64, [p, pi32, i64]),
        "acc_partition_cost": (C.c_int, [p, pi32, i32, C.c_int, C.POINTER(C.c_double)]),
        "acc_check_partition_recompute": (C.c_int, [p, pi32, i32, i32]),
        "acc_set_partition_recompute": (C.c_int, [p, pi32, i32, i32]),
        "acc_plan_recompute": (C.c_int, [p, C.c_int, C.c_int, i32, pi32]),
        "acc_enumerate_recompute": (i64, [p, i32, pi32, i64]),
        "acc_partition_cost_recompute": (C.c_int, [p, pi32, i32, i32, C.c_int, C.POINTER(C.c_double)]),
        "acc_plan_info": (C.c_int, [p, C.POINTER(i64), C.POINTER(i32)]),
        "acc_refine_to_kernels": (C.c_int, [p, pi32]),
        "acc_set_partition_copies": (C.c_int, [p, pi32, i32, pi32, pi32, i32, i32]),
        "acc_bind": (C.c_int, [p, i32, p, sz]),
        "acc_bind_host": (C.c_int, [p, i32, p, sz]),
        "acc_workspace_bytes": (C.c_int, [p, C.c_int, C.POINTER(sz)]),
        "acc_run": (C.c_int, [p, p, sz, p, C.c_int]),
        "acc_finish": (C.c_int, [p, p, p]),
        "acc_run_e2e": (C.c_int, [p, p, sz, p, C.c_int, C.POINTER(sz), C.POINTER(sz)]),
        "acc_run_e2e_async": (C.c_int, [p, p, sz, p, C.c_int, C.POINTER(sz), C.POINTER(sz)]),
        "acc_run_timed": (C.c_int, [p, p, sz, p, C.c_int, C.POINTER(C.c_float), i32, pi32]),
        "acc_check_gather_indices": (C.c_int, [p, p, sz, p]),
        "acc_launch_count": (i32, [p]),
        "acc_set_spin_limit": (C.c_int, [p, C.c_uint32]),
        "acc_last_schedule": (C.c_int, [p, C.c_char_p, sz]),
        "acc_scanl_add_i32_static": (C.c_int, [p, p, i64, p]),
        "acc_last_error": (C.c_char_p, []),
        "acc_registry_size": (i32, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = load_library()
    return _lib


_kernel_libraries = {}


def load_kernel_library(path):
    """Loads a shared object of further kernel instantiations (built by `build.build_kernel_library`); its
    kernels register themselves with libacc.so while it loads.  Returns how many signatures were new."""
    path = os.path.abspath(path)
    before = registry_size()
    if path not in _kernel_libraries:
        if not os.path.exists(path):
            raise ImportError("%s is missing: build it with `python -m paper_2407_13585_b200.build --tests`" % path)
        _kernel_libraries[path] = C.CDLL(path, mode=C.RTLD_GLOBAL)
    return registry_size() - before


def _check(code):
    if code < 0:
        raise AccError(int(code), lib().acc_last_error().decode())
    return code


def make_desc(nd):
    """acc_node_desc from a node record (attributes kind, dtype, shape, inputs, n_array, fn, idx_fn, iparam, fparam, force)."""
    d = NodeDesc()
    d.kind = KIND[nd.kind]
    d.dtype = DTYPE[nd.dtype]
    d.rank = len(nd.shape)
    for k, e in enumerate(nd.shape):
        d.shape[k] = int(e)
    d.n_inputs = len(nd.inputs)
    for k, s in enumerate(nd.inputs):
        d.inputs[k] = int(s)
    d.n_array_inputs = int(nd.n_array)
    d.fn_id = FN[nd.fn] if nd.fn else 0
    d.idx_fn_id = IDX_FN[nd.idx_fn] if nd.idx_fn else 0
    for k, v in enumerate(nd.iparam):
        d.iparam[k] = int(v)
    for k, v in enumerate(nd.fparam):
        d.fparam[k] = float(v)
    flags = 0
    for s in getattr(nd, "force", ()):
        flags |= 1 << s
    if getattr(nd, "exclusive", False):
        flags |= 1 << 16                      # ACC_FLAG_SCAN_EXCLUSIVE
    d.flags = flags
    return d


def _i32_array(values):
    return (C.c_int32 * len(values))(*[int(v) for v in values])


class Graph:
    """A program handle.  Methods mirror the acc_* entry points one to one."""

    def __init__(self, nodes=None, outputs=()):
        self._h = C.c_void_p()
        _check(lib().acc_graph_create(C.byref(self._h)))
        self._keep = {}          # tensors bound to nodes stay alive with the graph
        self.workspace = None
        if nodes is not None:
            for nd in nodes:
                self.add_node(nd)
            for o in outputs:
                self.mark_output(o)

    def close(self):
        if self._h:
            lib().acc_graph_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- graph ------------------------------------------------------------------
    def add_node(self, nd):
        d = nd if isinstance(nd, NodeDesc) else make_desc(nd)
        return _check(lib().acc_add_node(self._h, C.byref(d)))

    def mark_output(self, n):
        _check(lib().acc_mark_output(self._h, n))

    @property
    def n(self):
        return lib().acc_node_count(self._h)

    def edges(self):
        cap = 8 * max(self.n, 1)
        F, I = (C.c_int32 * (2 * cap))(), (C.c_int32 * (2 * cap))()
        nF, nI = C.c_int32(), C.c_int32()
        _check(lib().acc_edges(self._h, F, C.byref(nF), I, C.byref(nI), cap))
        pairs = lambda a, k: [(a[2 * j], a[2 * j + 1]) for j in range(k)]
        return pairs(F, nF.value), pairs(I, nI.value)

    # ---- clustering -------------------------------------------------------------
    def set_partition(self, pi):
        _check(lib().acc_set_partition(self._h, _i32_array(pi), len(pi)))

    def check_partition(self, pi):
        """Status name: 'ACC_OK' or the ACC_ERR_* that says which rule failed."""
        return STATUS_NAME[lib().acc_check_partition(self._h, _i32_array(pi), len(pi))]

    # clusterings that recompute: max_depth > 0 lets a fused-away array be evaluated once per order
    # it is read in, with at most max_depth gather-like nodes stacked on a fused path
    def set_partition_recompute(self, pi, max_depth):
        _check(lib().acc_set_partition_recompute(self._h, _i32_array(pi), len(pi), max_depth))

    def check_partition_recompute(self, pi, max_depth):
        return STATUS_NAME[lib().acc_check_partition_recompute(self._h, _i32_array(pi), len(pi), max_depth)]

    def plan_recompute(self, mode, cost, max_depth):
        out = (C.c_int32 * self.n)()
        _check(lib().acc_plan_recompute(self._h, PLAN[mode], COST[cost], max_depth, out))
        return list(out)

    def enumerate_recompute(self, max_depth):
        cnt = _check(lib().acc_enumerate_recompute(self._h, max_depth, None, 0))
        buf = (C.c_int32 * (max(cnt, 1) * self.n))()
        _check(lib().acc_enumerate_recompute(self._h, max_depth, buf, cnt))
        return [list(buf[i * self.n:(i + 1) * self.n]) for i in range(cnt)]

    def partition_cost_recompute(self, pi, max_depth, cost="bytes"):
        out = C.c_double()
        _check(lib().acc_partition_cost_recompute(self._h, _i32_array(pi), len(pi), max_depth, COST[cost], C.byref(out)))
        return out.value

    def set_partition_copies(self, pi, copies, max_depth=0):
        """copies: (node, cluster) pairs; readers of the node in that cluster read a copy recomputed there."""
        nodes = _i32_array([a for a, _ in copies])
        clusters = _i32_array([c for _, c in copies])
        _check(lib().acc_set_partition_copies(self._h, _i32_array(pi), len(pi), nodes, clusters, len(copies), max_depth))

    def get_partition(self):
        out = (C.c_int32 * self.n)()
        _check(lib().acc_get_partition(self._h, out, self.n))
        return list(out)

    def manifest(self):
        out = (C.c_int32 * self.n)()
        _check(lib().acc_manifest(self._h, out, self.n))
        return [bool(v) for v in out]

    def plan(self, mode="enumerate", cost="bytes"):
        out = (C.c_int32 * self.n)()
        _check(lib().acc_plan(self._h, PLAN[mode], COST[cost], out))
        return list(out)

    def plan_info(self):
        """(partial clusterings visited, result proven optimal) of the last plan call."""
        visited, proven = C.c_int64(), C.c_int32()
        _check(lib().acc_plan_info(self._h, C.byref(visited), C.byref(proven)))
        return visited.value, bool(proven.value)

    def refine_to_kernels(self):
        """Splits clusters that have no instantiated kernel; returns (splits made, the clustering now stored)."""
        buf = (C.c_int32 * self.n)()
        splits = _check(lib().acc_refine_to_kernels(self._h, buf))
        return splits, list(buf)

    def enumerate(self):
        cnt = _check(lib().acc_enumerate(self._h, None, 0))
        buf = (C.c_int32 * (max(cnt, 1) * self.n))()
        _check(lib().acc_enumerate(self._h, buf, cnt))
        return [list(buf[i * self.n:(i + 1) * self.n]) for i in range(cnt)]

    def partition_cost(self, pi, cost="bytes"):
        out = C.c_double()
        _check(lib().acc_partition_cost(self._h, _i32_array(pi), len(pi), COST[cost], C.byref(out)))
        return out.value

    # ---- running ----------------------------------------------------------------
    def bind(self, n, tensor):
        """Binds a CUDA tensor (4-byte elements, contiguous) to node n."""
        assert tensor.is_cuda and tensor.is_contiguous() and tensor.element_size() == 4
        _check(lib().acc_bind(self._h, n, C.c_void_p(tensor.data_ptr()), tensor.numel() * 4))
        self._keep[("dev", n)] = tensor

    def bind_host(self, n, tensor):
        assert not tensor.is_cuda and tensor.is_contiguous() and tensor.element_size() == 4
        _check(lib().acc_bind_host(self._h, n, C.c_void_p(tensor.data_ptr()), tensor.numel() * 4))
        self._keep[("host", n)] = tensor

    def workspace_bytes(self, executor=FUSED):
        out = C.c_size_t()
        _check(lib().acc_workspace_bytes(self._h, executor, C.byref(out)))
        return out.value

    def ensure_workspace(self, executor=FUSED, device="cuda"):
        import torch
        need = self.workspace_bytes(executor)
        if self.workspace is None or self.workspace.numel() < need:
            self.workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=device)
        return self.workspace

    @staticmethod
    def _stream():
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)

    def run(self, executor=FUSED, finish=True):
        ws = self.ensure_workspace(executor)
        _check(lib().acc_run(self._h, C.c_void_p(ws.data_ptr()), ws.numel(), self._stream(), executor))
        if finish:
            self.finish()

    def finish(self):
        ws = self.workspace
        _check(lib().acc_finish(self._h, C.c_void_p(ws.data_ptr()) if ws is not None else None, self._stream()))

    def run_e2e(self, executor=FUSED, finish=True):
        """Host inputs in, program, host outputs out on the current stream; finish=False returns
        after enqueueing (call finish() under the same stream later)."""
        ws = self.ensure_workspace(executor)
        up, down = C.c_size_t(), C.c_size_t()
        fn = lib().acc_run_e2e if finish else lib().acc_run_e2e_async
        _check(fn(self._h, C.c_void_p(ws.data_ptr()), ws.numel(), self._stream(), executor, C.byref(up), C.byref(down)))
        return up.value, down.value

    def run_timed(self, executor=FUSED):
        """Runs and waits; returns the device time of every cluster launch in ms, in execution order."""
        ws = self.ensure_workspace(executor)
        ms = (C.c_float * 64)()
        n = C.c_int32()
        _check(lib().acc_run_timed(self._h, C.c_void_p(ws.data_ptr()), ws.numel(), self._stream(), executor, ms, 64, C.byref(n)))
        return [ms[k] for k in range(min(n.value, 64))]

    def check_gather_indices(self):
        """Raises AccError(ACC_ERR_INDEX_RANGE) if an input index array of a gather points outside its source."""
        ws = self.ensure_workspace(FUSED)
        _check(lib().acc_check_gather_indices(self._h, C.c_void_p(ws.data_ptr()), ws.numel(), self._stream()))

    def set_spin_limit(self, max_polls):
        _check(lib().acc_set_spin_limit(self._h, max_polls))

    def launch_count(self):
        return lib().acc_launch_count(self._h)

    def last_schedule(self):
        buf = C.create_string_buffer(4096)
        lib().acc_last_schedule(self._h, buf, 4096)
        return buf.value.decode()


def scanl_add_i32_static(src, dst):
    """acc_scanl_add_i32_static on two int32 CUDA tensors: inclusive wrapping prefix sum of `src`
    into `dst` using the library's built-in scratch array.  Nothing is allocated here or in the
    library, so it can be called from code that must not touch the device allocator.  Waits for
    the current stream; calls that overlap on one GPU race on the shared scratch."""
    assert src.is_cuda and dst.is_cuda and src.is_contiguous() and dst.is_contiguous()
    assert src.element_size() == 4 and dst.numel() >= src.numel()
    _check(lib().acc_scanl_add_i32_static(C.c_void_p(src.data_ptr()), C.c_void_p(dst.data_ptr()), src.numel(),
                                          Graph._stream()))


def registry_size():
    return lib().acc_registry_size()
