/*
 * acc.h -- C ABI of the fused-cluster executor for combinator array programs.
 *
 * A program is a data-dependence graph of array combinators (the paper's
 * Section 4.1: nodes, fusible and infusible edges).  A clustering is the map
 * pi from node to cluster number; clusters run in ascending number (Section
 * 4.1) and each legal cluster runs as ONE CUDA kernel.  Legality is the
 * paper's Figure 3 together with the top-level rules of Section 3.4.
 *
 * Conventions
 *   - Every call returns ACC_OK (0) or a negative acc_status; acc_add_node
 *     returns the new node id (>= 0) or a negative acc_status.  A message for
 *     the last failure on the calling thread is kept by acc_last_error().
 *   - The library never allocates, frees or owns device memory and never
 *     creates a stream.  Device pointers come from the caller through
 *     acc_bind / the workspace argument and must stay valid until the work
 *     that uses them has finished on the stream.
 *   - Arrays are dense, row-major, 4-byte elements (fp32, int32, uint32),
 *     rank 0..2, at most ACC_MAX_ELEMENTS (2^31 - 2^16) elements, base pointers
 *     16-byte aligned.
 *   - A graph handle is not thread-safe.
 */
#ifndef ACC_H
#define ACC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct acc_graph acc_graph; /* opaque, owned by the library */
typedef int32_t acc_node;           /* >= 0: node id; < 0: acc_status */

/* Combinators of Section 2 (Table 1).  ZIPWITH is a map over several arrays
 * of one shape (structure-of-arrays view, Section 2); BACKPERMUTE is
 * generate + gather already fused (Section 2.1); PERMUTE is the paper's
 * scatter with index and value arrays in separate slots. */
enum acc_kind {
  ACC_INPUT = 0,   /* array supplied by the caller                               */
  ACC_GENERATE,    /* ys[i] = f(i)                                                */
  ACC_MAP,         /* ys[i] = f(xs[i])                       slots {xs, free...}  */
  ACC_ZIPWITH,     /* ys[i] = f(xs1[i]..xsk[i]), k = 2..3    slots {xs.., free..} */
  ACC_BACKPERMUTE, /* ys[j] = xs[p(j)], p named by idx_fn    slots {xs}           */
  ACC_GATHER,      /* ys[j] = src[idx[j]] (linear index)     slots {idx, src}     */
  ACC_PERMUTE,     /* out = defaults; out[idx[j]] op= vals[j] slots {defaults, idx, vals} */
  ACC_FOLD,        /* reduce the innermost extent, no seed   slots {xs}           */
  ACC_FOLDSEG,     /* ys[s] = fold of xs[off[s] .. off[s+1]), rank-1 xs   slots {xs, off}: n_array_inputs = 1,
                      off is S+1 increasing int offsets read by index (the paper names foldSeg in a keyword
                      list only; segments must be non-empty since a fold has no seed)          */
  ACC_SCANL,       /* inclusive left-to-right scan per innermost row  slots {xs}  */
  ACC_SCANR        /* inclusive right-to-left scan per innermost row  slots {xs}  */
};

enum acc_dtype { ACC_F32 = 0, ACC_I32 = 1, ACC_U32 = 2 };

/* Element functions (the paper leaves them abstract; these are the ones the
 * build instantiates).  fp32 functions round after every operation (no FMA
 * contraction); integer functions wrap modulo 2^32 on the uint32 view.
 * "free0" is element 0 of the first free-variable slot. */
enum acc_fn {
  ACC_FN_NONE = 0,
  /* map / zipWith */
  ACC_FN_IDENTITY,          /* x                                                   */
  ACC_FN_AFFINE,            /* fparam[0]*x + fparam[1]                             */
  ACC_FN_MUL,               /* a*b                 (also a combine operator)       */
  ACC_FN_ADD,               /* a+b                 (also a combine operator)       */
  ACC_FN_ADD3,              /* (a+b)+c                                             */
  ACC_FN_MUL_ADD_CONST,     /* a*b + fparam[0]                                     */
  ACC_FN_ADD_SCALE,         /* fparam[0]*(a+b)                                     */
  ACC_FN_DIV_FREE,          /* x / free0                                           */
  ACC_FN_ADD_FREE,          /* x + free0                                           */
  ACC_FN_HASH_MUL_XORSHIFT, /* (v*iparam[0]) xor (v >> iparam[1]), logical shift   */
  ACC_FN_AND_MASK,          /* v and iparam[0]                                     */
  ACC_FN_MUL_MOD,           /* (v*iparam[0] mod 2^32) mod iparam[1]                */
  ACC_FN_MUL_CONST,         /* v*iparam[0]                                         */
  ACC_FN_ADD_CONST,         /* v+iparam[0]                                         */
  /* generate (i = row-major linear index) */
  ACC_FN_IOTA,              /* i converted to the node dtype                       */
  ACC_FN_IMOD_TO_F32,       /* float(i mod iparam[0])                              */
  ACC_FN_ROW_INDEX,         /* i / innermost extent                                */
  ACC_FN_IOTA_PLUS_FREE,    /* float(i) + free0                                    */
  /* further combine operators of fold / scan / permute */
  ACC_FN_MIN,
  ACC_FN_MAX,
  ACC_FN_COUNT_
};

/* Index maps of BACKPERMUTE: position in the output -> position in the source. */
enum acc_idx_fn {
  ACC_IDX_NONE = 0,
  ACC_IDX_IDENTITY,
  ACC_IDX_REVERSE,     /* linear index j -> count-1-j                                   */
  ACC_IDX_TRANSPOSE,   /* (r, c) -> (c, r); output shape (R, C) over a source (C, R)     */
  ACC_IDX_SHIFT_CLAMP  /* (r, c) -> (clamp(r+iparam[0]), clamp(c+iparam[1])), same shape */
};

enum acc_exec { ACC_EXEC_FUSED = 0, ACC_EXEC_UNFUSED = 1 };

enum acc_plan_mode {
  ACC_PLAN_UNFUSED = 0,      /* every node its own cluster                             */
  ACC_PLAN_ENUMERATE,        /* best of all legal clusterings (small graphs only)      */
  ACC_PLAN_GREEDY_TOPDOWN,   /* Section 5 "Greedy": edges from the top of the graph    */
  ACC_PLAN_GREEDY_BOTTOMUP,  /* Section 5 "Greedy": edges from the bottom              */
  ACC_PLAN_BRANCH_BOUND      /* exact search with a traffic lower bound (costs BYTES,
                                READS_WRITES), started from the better greedy result    */
};

/* Cost functions of Section 4.1 (a)-(e), the sum of them ("everything" in
 * Figure 6), and (e) with every array weighted by its size in bytes. */
enum acc_cost {
  ACC_COST_CLUSTERS = 0,
  ACC_COST_FUSED_EDGES,
  ACC_COST_ARRAYS,
  ACC_COST_READS,
  ACC_COST_READS_WRITES,
  ACC_COST_EVERYTHING,
  ACC_COST_BYTES
};

enum acc_status {
  ACC_OK = 0,
  ACC_ERR_ARG = -1,                /* null pointer, bad enum, id out of range             */
  ACC_ERR_SHAPE = -2,              /* shapes of a node and its inputs do not fit           */
  ACC_ERR_DTYPE = -3,
  ACC_ERR_UNSUPPORTED = -4,        /* a combination the build has no code for              */
  ACC_ERR_ILLEGAL_INFUSIBLE = -5,  /* an infusible edge inside one cluster                 */
  ACC_ERR_ILLEGAL_ORDER = -6,      /* pi_a > pi_b on an edge                                */
  ACC_ERR_ILLEGAL_TRAVERSAL = -7,  /* no assignment of traversal orders satisfies Figure 3  */
  ACC_ERR_ILLEGAL_SCATTER = -8,    /* another use of a scatter destination is not earlier   */
  ACC_ERR_DISCONNECTED = -9,       /* a cluster whose nodes share no fused array            */
  ACC_ERR_NO_KERNEL = -10,         /* legal cluster without a build-time instantiation      */
  ACC_ERR_UNBOUND = -11,           /* an input or output has no device buffer               */
  ACC_ERR_WORKSPACE = -12,         /* workspace null, misaligned or too small               */
  ACC_ERR_CUDA = -13,              /* a CUDA runtime call failed                            */
  ACC_ERR_DEVICE_TIMEOUT = -14,    /* a bounded device-side wait ran out                    */
  ACC_ERR_INDEX_RANGE = -15,       /* scatter index outside its destination                 */
  ACC_ERR_TOO_LARGE = -16,         /* graph too large for the requested planner mode        */
  ACC_ERR_NO_PARTITION = -17       /* acc_run(FUSED) before a clustering was set            */
};

#define ACC_MAX_INPUTS 6
/* Largest array (and largest single extent) acc_add_node accepts: the kernels
 * index with signed 32-bit arithmetic and keep one tile of head room. */
#define ACC_MAX_ELEMENTS ((1ll << 31) - (1ll << 16))
#define ACC_FLAG_FORCE_SLOT(s) (1u << (s)) /* the read of slot s goes through force() */
/* SCANL / SCANR only.  The paper's scans (Section 2) have no seed and keep the length, which is
 * read as inclusive.  With this flag the scan is seeded and exclusive: element k is the seed
 * (fparam[0] for F32, iparam[0] otherwise) combined with the elements before k in scan order, so
 * the first element is the seed itself and the last element of the source is left out. */
#define ACC_FLAG_SCAN_EXCLUSIVE (1u << 16)

typedef struct acc_node_desc {
  int32_t  kind;                 /* acc_kind                                             */
  int32_t  dtype;                /* acc_dtype of the result                              */
  int32_t  rank;                 /* 0 (scalar result of a rank-1 fold), 1 or 2           */
  int64_t  shape[2];             /* result shape, row-major                              */
  int32_t  n_inputs;
  acc_node inputs[ACC_MAX_INPUTS];
  int32_t  n_array_inputs;       /* inputs[n_array_inputs..] are free-variable reads     */
  int32_t  fn_id;                /* acc_fn: element function or combine operator         */
  int32_t  idx_fn_id;            /* acc_idx_fn (BACKPERMUTE only)                        */
  int64_t  iparam[4];
  double   fparam[4];
  uint32_t flags;                /* ACC_FLAG_FORCE_SLOT(s), ACC_FLAG_SCAN_EXCLUSIVE      */
} acc_node_desc;

/* ---- building the graph (Section 4.1, "Data dependence graph") ------------- */

/* Creates an empty graph in *out.  Host pointers only. */
int acc_graph_create(acc_graph** out);
/* Destroys the graph; buffers bound to it are not touched. */
int acc_graph_destroy(acc_graph* g);
/* Appends a node.  Every input must be an existing node, so the graph is a DAG
 * in node-id order.  Edges are classified here: infusible out of an INPUT,
 * into a free-variable slot, into PERMUTE's defaults slot, out of a PERMUTE
 * and through a forced slot (Sections 3.4 and 4.1); fusible otherwise.
 * The descriptor is copied. */
acc_node acc_add_node(acc_graph* g, const acc_node_desc* d);
/* Marks a node as a program output: its array is manifest under every clustering. */
int acc_mark_output(acc_graph* g, acc_node n);
/* Number of nodes added so far. */
int32_t acc_node_count(const acc_graph* g);
/* Writes the fusible edges as pairs (a,b) into F and the infusible ones into I
 * (each up to `cap` pairs, 2*cap int32); *nF and *nI receive the true counts. */
int acc_edges(const acc_graph* g, int32_t* F, int32_t* nF, int32_t* I, int32_t* nI, int32_t cap);

/* ---- clustering (Sections 3.4, 4.1, 4.2; Figure 3) -------------------------- */

/* Checks pi (cluster_of_node[i] for every node; entries of INPUT nodes are
 * ignored) against Figure 3 and the top-level rules, and stores it on success.
 * On failure the stored clustering is unchanged and the ACC_ERR_ILLEGAL_* /
 * ACC_ERR_DISCONNECTED code says which rule failed. */
int acc_set_partition(acc_graph* g, const int32_t* cluster_of_node, int32_t n_nodes);
/* Same checks, nothing stored. */
int acc_check_partition(acc_graph* g, const int32_t* cluster_of_node, int32_t n_nodes);
/* Reads back the stored clustering (INPUT nodes get -1). */
int acc_get_partition(const acc_graph* g, int32_t* cluster_of_node_out, int32_t n_nodes);
/* For the stored clustering: manifest_out[i] = 1 if node i is written to
 * memory (m_i = 0 in Figure 3), 0 if it is fused away. */
int acc_manifest(const acc_graph* g, int32_t* manifest_out, int32_t n_nodes);
/* Plans a clustering (Section 5, "Greedy"; exhaustive search or branch and
 * bound in place of the ILP solver of Section 4) under `cost`, writes it to
 * cluster_of_node_out (may be null) and stores it.  ENUMERATE fails with
 * ACC_ERR_TOO_LARGE beyond 12 non-input nodes.  BRANCH_BOUND minimises
 * Section 4.1's reads-and-writes objective (e), in arrays or in bytes: it assigns
 * nodes to clusters in program order, drops a partial clustering as soon as it
 * breaks a rule that more nodes cannot mend or as soon as the traffic it is
 * already sure of (arrays that must be manifest in every clustering included)
 * reaches the best clustering known, and gives up the proof, not the result,
 * after 2^22 partial clusterings. */
int acc_plan(acc_graph* g, int mode, int cost, int32_t* cluster_of_node_out);
/* Makes the stored clustering runnable.  Kernels are instantiated at build
 * time per cluster shape, and the rules of Figure 3 know nothing of that: a
 * planner may return a legal cluster nobody built a kernel for (ACC_ERR_NO_KERNEL
 * from acc_run).  While such a cluster exists, its latest node (in program
 * order) that can leave it with the clustering still legal becomes a cluster of
 * its own; if no single node can, the cluster falls apart into its nodes.
 * Stores the result, writes it to cluster_of_node_out (may be null) and returns
 * the number of splits (0: every cluster had a kernel), or a negative
 * acc_status (ACC_ERR_NO_KERNEL if a node alone has none).  Host only. */
int acc_refine_to_kernels(acc_graph* g, int32_t* cluster_of_node_out);
/* Every legal clustering, each as n_nodes int32 with canonical numbering
 * (clusters numbered in an execution order, ties by smallest node id), in
 * lexicographic order.  Returns the count (also when out_pi is null or
 * max_partitions is smaller) or a negative acc_status. */
int64_t acc_enumerate(acc_graph* g, int32_t* out_pi, int64_t max_partitions);
/* Cost of a legal clustering under `cost` (lower is better). */
int acc_partition_cost(acc_graph* g, const int32_t* cluster_of_node, int32_t n_nodes, int cost, double* out);

/* About the last acc_plan / acc_plan_recompute call on g: how many partial
 * clusterings the search visited, and whether the result is proven to have the
 * least cost (always for ENUMERATE; for BRANCH_BOUND unless the search stopped
 * at its limit of visited clusterings; never for the greedy planners). */
int acc_plan_info(const acc_graph* g, int64_t* visited_out, int32_t* proven_optimal_out);

/* ---- clusterings that recompute (the paper's future work, Section 6) ----------- */

/* The paper's model gives every array one traversal order, so an array read in
 * two orders by one cluster (once as it lies and once through a backpermute, or
 * through several backpermutes) cannot be fused away there: Section 3.3's
 * `simple5` reads it twice from memory instead, and Section 6 leaves fusion
 * that duplicates work to future work.  The calls below accept such clusters:
 * with max_depth > 0 a fused-away array may be evaluated once per order it is
 * read in, as if each consumer had its own copy of the producer (and of the
 * producer's producers inside the cluster).  What still fails: a scan asked for
 * an order other than its own, the one stored copy of a manifest array asked
 * for an order above 1, every rule that is not about orders, and more than
 * max_depth gather-like nodes stacked on one fused path of a cluster that needs
 * such copies (a cluster that is legal in the paper's model stays legal).
 * max_depth = 0 is the paper's model (the calls above).  The arrays computed are the same as under
 * any legal clustering; only the work and the traffic differ.
 * Arguments and results as for the calls of the same name above. */
int acc_check_partition_recompute(acc_graph* g, const int32_t* cluster_of_node, int32_t n_nodes, int32_t max_depth);
int acc_set_partition_recompute(acc_graph* g, const int32_t* cluster_of_node, int32_t n_nodes, int32_t max_depth);
int acc_plan_recompute(acc_graph* g, int mode, int cost, int32_t max_depth, int32_t* cluster_of_node_out);
int64_t acc_enumerate_recompute(acc_graph* g, int32_t max_depth, int32_t* out_pi, int64_t max_partitions);
int acc_partition_cost_recompute(acc_graph* g, const int32_t* cluster_of_node, int32_t n_nodes, int32_t max_depth, int cost,
                                 double* out);

/* A clustering in which some nodes are evaluated in several clusters: besides
 * cluster_of_node (each node's own cluster), n_copies pairs (copy_node[k],
 * copy_cluster[k]) put a copy of a node into a further cluster.  Every reader of
 * the node that lies in such a cluster reads the copy (fused, recomputed there)
 * instead of the stored array; the copy itself reads, input by input, what its
 * cluster holds of the input (the input's own node or its copy there) and
 * otherwise the stored array.  A copy must be fused away: it is an error if it
 * has no reader in its cluster or would have to be stored.  The clustering with
 * the copies written out as nodes is checked like any other (max_depth as
 * above; 0: the paper's rules).  acc_get_partition and acc_manifest keep
 * speaking of the original nodes.  Example: the total of the histogram program
 * can regenerate `vals` in its own kernel instead of reading them from memory. */
int acc_set_partition_copies(acc_graph* g, const int32_t* cluster_of_node, int32_t n_nodes, const int32_t* copy_node,
                             const int32_t* copy_cluster, int32_t n_copies, int32_t max_depth);

/* ---- running ------------------------------------------------------------------ */

/* Binds a caller-owned DEVICE buffer to a node.  Required for INPUT nodes and
 * marked outputs; allowed for any node (its array is then written there when
 * manifest instead of into the workspace).  bytes must cover the array. */
int acc_bind(acc_graph* g, acc_node n, void* device_ptr, size_t bytes);
/* Binds a caller-owned HOST buffer (pinned for asynchronous copies) to an
 * INPUT node or a marked output, used by acc_run_e2e only. */
int acc_bind_host(acc_graph* g, acc_node n, void* host_ptr, size_t bytes);
/* Device bytes acc_run needs beyond bound buffers for `executor` under the
 * stored clustering: unbound manifest arrays plus tickets, partials and scan
 * tile states.  The workspace must be 256-byte aligned. */
int acc_workspace_bytes(acc_graph* g, int executor, size_t* bytes);
/* Enqueues the whole program on `cuda_stream` (a cudaStream_t; null = default
 * stream): FUSED = one kernel per cluster of the stored clustering in
 * ascending cluster number; UNFUSED = one kernel per combinator in node order.
 * Asynchronous: returns after the launches; launch failures are reported here,
 * device-side status by acc_finish.  `workspace` is a DEVICE pointer. */
int acc_run(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream, int executor);
/* Waits for the stream and returns the device status of the last acc_run
 * (ACC_OK, ACC_ERR_DEVICE_TIMEOUT, ACC_ERR_INDEX_RANGE, ACC_ERR_CUDA). */
int acc_finish(acc_graph* g, void* workspace, void* cuda_stream);
/* acc_run followed by acc_finish, with a CUDA event before the first launch and
 * after every cluster: ms_per_cluster_out[k] receives the device time of the
 * k-th launch in execution order (up to `cap` entries), *n_out their number.
 * For looking at where a program's time goes; the events cost a little, so time
 * whole programs with acc_run. */
int acc_run_timed(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream, int executor,
                  float* ms_per_cluster_out, int32_t cap, int32_t* n_out);
/* Gather is defined for valid indices only (Section 2), and the kernels do not
 * check them: an index outside the source reads memory that is not the
 * caller's.  This call checks, on the device and without running the program,
 * every GATHER whose index array is a program INPUT with a bound device buffer
 * against the size of its source; it waits for the stream and returns ACC_OK or
 * ACC_ERR_INDEX_RANGE.  `workspace` needs 256 bytes (the status word). */
int acc_check_gather_indices(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream);
/* End to end with HOST buffers: copies every host-bound INPUT to its device
 * buffer, runs as acc_run, copies every host-bound output back, waits, and
 * returns as acc_finish.  h2d/d2h receive the bytes copied (may be null). */
int acc_run_e2e(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream, int executor,
                size_t* h2d_bytes, size_t* d2h_bytes);
/* The same without the wait: the copies and the launches are enqueued and the
 * call returns; acc_finish on the same stream waits and reports.  Programs
 * enqueued this way on different streams overlap their copies in both
 * directions with each other and with the kernels. */
int acc_run_e2e_async(acc_graph* g, void* workspace, size_t workspace_bytes, void* cuda_stream, int executor,
                      size_t* h2d_bytes, size_t* d2h_bytes);
/* Bound of the one device-side wait that polls plain memory: a tile of a
 * single-pass scan (Section 2: "prefix sum", computed with decoupled look-back)
 * polls the state of the tiles before it until they have published a total.
 * A tile that has polled max_polls times without success gives up, the run
 * goes on and ends with ACC_ERR_DEVICE_TIMEOUT (the scan's output is then not
 * valid); 0 gives up at the first unsuccessful poll.  Default 2^22 (seconds).
 * Applies to later runs of this graph; the waits on copy barriers in the
 * tile-staging kernels have a fixed bound and are not affected. */
int acc_set_spin_limit(acc_graph* g, uint32_t max_polls);
/* Kernels launched by the last acc_run / acc_run_e2e on this graph. */
int32_t acc_launch_count(const acc_graph* g);
/* Clusters of the last run, as "first_node:count" items separated by blanks,
 * copied into buf (truncated to cap-1 characters). */
int acc_last_schedule(const acc_graph* g, char* buf, size_t cap);

/* Inclusive left-to-right prefix sum of n int32 values with wrap-around,
 * out[i] = in[0] + ... + in[i], for callers that cannot give the library a
 * workspace.  (The paper has no counterpart: this is a packaging variant of
 * the scan kernel, not a combinator or a rule of its own.)
 *
 * Who needs it: code that may not allocate device memory where it calls us --
 * a plug-in or callback that receives raw device pointers but no allocator, a
 * process whose device-memory budget is fixed up front and fully handed out,
 * a component that must not call cudaMalloc or cudaFree because other work
 * shares the device with it.  acc_run needs a caller-allocated workspace for
 * the scan's tile states; this entry point keeps them in a fixed array inside
 * the library's device image instead (about 128 KiB, resident on every GPU
 * that loads the library until the process exits) and calls no cudaMalloc,
 * cudaFree or any other allocating routine.  It is not a low-latency call:
 * it blocks the host until the scan has finished (see below).
 *
 *   in, out      DEVICE pointers to n int32 each, owned by the caller, not
 *                overlapping; 16-byte alignment and n % 4 == 0 select the
 *                128-bit path, anything else the scalar one.
 *   n            0 .. ACC_STATIC_SCAN_MAX_ELEMENTS; more is refused with
 *                ACC_ERR_TOO_LARGE and nothing is launched.
 *   cuda_stream  a cudaStream_t of the current device (null = default stream).
 *
 * The call enqueues a clear of the part of the array it uses and the scan, then
 * BLOCKS THE HOST until the stream has finished (it copies the status word
 * back and synchronises the stream) and returns ACC_OK, ACC_ERR_DEVICE_TIMEOUT
 * (a bounded wait between tiles ran out; out is then not valid) or
 * ACC_ERR_CUDA.  Because of that copy and wait, never call it on a stream that
 * is being captured.  The first call on each device also looks up the array's
 * device address (with that device current).
 * All calls on one GPU share the one array, which keeps the previous call's
 * contents between calls: two calls whose work overlaps on the same GPU
 * (different streams or threads) race on it and give undefined results --
 * serialise them.  Calls on different GPUs are independent. */
#define ACC_STATIC_SCAN_MAX_ELEMENTS (1ll << 26)
int acc_scanl_add_i32_static(const int32_t* in, int32_t* out, int64_t n, void* cuda_stream);

/* Message for the last failing call on this thread ("" if none). */
const char* acc_last_error(void);
/* Number of build-time kernel instantiations in the registry. */
int32_t acc_registry_size(void);

#ifdef __cplusplus
}
#endif
#endif /* ACC_H */
