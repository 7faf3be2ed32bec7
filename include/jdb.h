/*
 * jdb.h - C ABI of the dynamically batched Child-Sum Tree-LSTM forward for B200 (sm_100a).
 *
 * The paper ("Just-in-Time Dynamic-Batching") collects the computation graphs of a
 * batch of samples, files every node in a table by depth, and runs the table in depth
 * order, one batched launch per slot (Sections 4.2 and 4.3).  For a forest of Tree-LSTM
 * cells that is two calls:
 *
 *   jdb_schedule          the batching analysis: depth per node, level offsets and the
 *                         level-ordered node permutation, from the forest's child CSR;
 *   jdb_treelstm_forward  the batched execution: every level evaluated as one batch.
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its comment says "host".
 *   - The library allocates no device memory: outputs and workspaces are the caller's.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     All work is enqueued on it; see each call for where it synchronises.
 *   - Errors are returned as jdb_status; nothing aborts, throws or traps the device.
 *   - Node and edge ids are int32; row offsets are computed in 64 bits.
 */
#ifndef JDB_H_
#define JDB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    JDB_OK = 0,
    JDB_ERR_INVALID_ARG = 1,   /* null pointer, negative size, bad enum, misaligned buffer      */
    JDB_ERR_NOT_A_FOREST = 2,  /* child id out of range, node with two parents, cycle, bad ptr  */
    JDB_ERR_WORKSPACE = 3,     /* workspace or packed-weight buffer too small                    */
    JDB_ERR_UNSUPPORTED = 4,   /* sizes outside what the kernels were built for                  */
    JDB_ERR_CUDA = 5,          /* a CUDA runtime call failed (see jdb_last_cuda_error)           */
    JDB_ERR_TIMEOUT = 6,       /* a bounded device-side wait ran out; outputs are undefined      */
    JDB_ERR_CHECK = 7          /* JDB_FLAG_DEBUG_CHECKS: a kernel met an index outside its arrays (the access was
                                  skipped; see jdb_debug_report)                                  */
} jdb_status;

/* precision of the GEMM operands; accumulation and the c/h state are always fp32 */
enum { JDB_FP32 = 0, JDB_BF16 = 1 };
/* how the level loop runs */
enum { JDB_MODE_AUTO = 0, JDB_MODE_PER_LEVEL = 1, JDB_MODE_PERSISTENT = 2 };

/* jdb_opts.flags */
enum {
    JDB_FLAG_NO_SYNC = 1,      /* jdb_treelstm_forward never synchronises; ask jdb_sched_status afterwards */
    JDB_FLAG_ROOTS_ONLY = 4,   /* host entries (jdb_treelstm_forward_host, jdb_online_submit) only: h and c receive the
                                  states of the ROOTS alone, dense [n_nodes - n_edges, H], roots in ascending node id
                                  (what a sentence-level task reads; the other rows stay on the device)            */
    JDB_FLAG_DEBUG_CHECKS = 2  /* every kernel of the forward pass checks the indices it is about to follow (child ids,
                                  positions in level order, level offsets, rows of the workspace arrays) against the
                                  sizes of the arrays they index, skips an access that would leave them and records the
                                  first offender in sched->meta; the call then synchronises and returns JDB_ERR_CHECK.
                                  Slower; meant for tests and for bringing up a new caller.                          */
};

/* jdb_opts.tuning: 0 takes the library's defaults (the measured best, which the environment variables JDB_GEMM_PAIR,
 * JDB_GEMM_ISSUERS, JDB_PDL, JDB_P_TMA, JDB_GATHER_X and JDB_TREE_GROUPS may change, read at every call).  With JDB_TUNE_SET the other bits
 * replace those defaults for this call; every combination computes the same values. */
enum {
    JDB_TUNE_SET = 1,
    JDB_TUNE_PAIR_XPROJ = 2,    /* input-projection GEMM as CTA pairs (forests of at least 256 rows per SM); default   */
    JDB_TUNE_PAIR_LEVEL = 4,    /* per-level gate GEMM as CTA pairs (launches with at least 32 tiles per pair); default */
    JDB_TUNE_PAIR_FORGET = 8,   /* per-level forget-gate GEMM as CTA pairs (launches with at least 32 tiles per pair); default */
    JDB_TUNE_TWO_ISSUERS = 16,  /* two MMA-issuing warps per lone CTA, half of the tile's columns each               */
    JDB_TUNE_NO_PDL = 32,       /* ordinary launches instead of programmatic dependent launches                      */
    JDB_TUNE_PLAIN_STORES = 64, /* level-ordered outputs through the load/store units instead of TMA stores           */
    JDB_TUNE_GATHER_X = 128,    /* bf16 x with 16-byte aligned rows is read in place by the input projection (TMA row
                                   gathers keyed by perm) instead of being laid out in level order first; slower      */
    JDB_TUNE_TREE_GROUPS = 256  /* cooperative level loop (JDB_BF16, H <= 192): partition the forest by tree over the groups
                                   of CTAs, which then synchronise inside a group only instead of ending every level in
                                   a barrier over the whole grid (needs a schedule from jdb_schedule; not faster on the
                                   workloads measured, so off by default)                                                */
};

#define JDB_META_INTS 16 /* size of jdb_sched.meta in int32 */

/* A forest as a child CSR: the children of node v are child_idx[child_ptr[v] .. child_ptr[v+1]-1],
 * in that order.  Roots are the nodes no list mentions; any number of trees; ids need not be
 * topologically ordered.  (The per-sample graphs of Section 1, stacked.) */
typedef struct {
    const int32_t *child_ptr; /* [n_nodes + 1], child_ptr[0] = 0, non-decreasing, last = n_edges */
    const int32_t *child_idx; /* [n_edges] */
    int32_t n_nodes;
    int32_t n_edges;
} jdb_forest;

/* The depth table of Section 4.2.  depth(v) = 0 for a leaf, else 1 + max over its children: no node depends on
 * another node of its own depth, and levels run in ascending order.
 * All arrays are caller-allocated device memory. */
typedef struct {
    int32_t *depth;     /* [n_nodes]                                                            */
    int32_t *level_ptr; /* [n_nodes + 2] capacity; entries 0..n_levels valid:
                           level_ptr[d] = number of nodes with depth < d                        */
    int32_t *perm;      /* [n_nodes] node ids ordered by (depth, id)                            */
    int32_t *meta;      /* [JDB_META_INTS] device-side copy of n_levels, n_leaves, error flags   */
    int32_t n_levels;   /* host; written by jdb_schedule, -1 after jdb_schedule_async            */
    int32_t n_leaves;   /* host; = level_ptr[1]; -1 after jdb_schedule_async                     */
    int32_t n_wide_levels; /* host; how many of the levels 1, 2, ... in a row hold at least 65536 nodes
                           (a statistic of the depth table; the forward pass does not depend on it);
                           -1 after jdb_schedule_async                                             */
    int32_t reserved0;  /* 0 */
} jdb_sched;

typedef struct {
    int32_t precision;  /* JDB_FP32 | JDB_BF16: must match the packed weights                    */
    int32_t mode;       /* JDB_MODE_*                                                            */
    int32_t flags;      /* JDB_FLAG_* ORed together                                              */
    int32_t tuning;     /* JDB_TUNE_* ORed together; 0 = defaults                                */
    uint64_t barrier_timeout_ns; /* limit of one grid-barrier wait in persistent mode; 0 = 2 s   */
    /* Optional timing hooks: cudaEvent_t handles (as void*, NULL = none) recorded on `stream` before
     * the input projection, after it, and after the level loop, so that a caller can time the two
     * phases of one call with cudaEventElapsedTime. */
    void *ev_begin;
    void *ev_xproj_done;
    void *ev_levels_done;
    /* Optional trace of the cooperative level loop: device array of trace_cap uint64 (NULL = none).  CTA 0
     * writes %globaltimer stamps (ns) per level at [8*level + s]: s=0 level start, 1 description of the first
     * pass received, 2 child rows gathered into the tensor-core operand, 4 tensor-core product done,
     * 5 accumulators read out, 6 rows stored, 7 level barrier passed (s=3 is not written).  Only its first
     * tile of a level is stamped. */
    uint64_t *trace;
    int64_t trace_cap;
} jdb_opts;

const char *jdb_status_string(jdb_status s);
/* cudaError_t (as int) of the most recent failing runtime call made by this thread's last API call */
int jdb_last_cuda_error(void);

/* ---- batching analysis (Section 4.2: depth-organised look-up table) ------------------------ */

/* Bytes of device scratch jdb_schedule needs for a forest of this size. */
size_t jdb_schedule_workspace_bytes(int32_t n_nodes, int32_t n_edges);

/* Computes depth, level_ptr, perm and meta on `stream`, then synchronises the stream ONCE to read
 * back n_levels, n_leaves and the validation result (the level count decides what the caller may
 * read and how many level launches follow).  n_nodes = 0 gives JDB_OK, n_levels = 0, level_ptr[0] = 0.
 * A malformed forest gives JDB_ERR_NOT_A_FOREST; the outputs are then undefined but no access
 * leaves the buffers.  ws must be 256-byte aligned. */
jdb_status jdb_schedule(const jdb_forest *forest, jdb_sched *out, void *ws, size_t ws_bytes, void *stream);

/* The same work without the synchronisation: n_levels/n_leaves are left at -1 on the host and live
 * only in out->meta.  A following jdb_treelstm_forward then runs its level loop from the device-side
 * values (persistent mode) and reports a malformed forest itself. */
jdb_status jdb_schedule_async(const jdb_forest *forest, jdb_sched *out, void *ws, size_t ws_bytes, void *stream);

/* The paper has no counterpart to this call: it is jdb_schedule for callers that cannot allocate device
 * memory at all and so cannot bring a workspace (a serving loop that may not stall in an allocator, a plug-in
 * inside a memory pool it does not own).  The scratch of the analysis kernels is a fixed array inside the
 * library image (about 1.2 MB, held by every GPU that loads the library until the process ends), so:
 *   - forests of more than JDB_STATIC_MAX_NODES nodes are refused with JDB_ERR_UNSUPPORTED;
 *   - the first call on a device looks the array's device address up; make that first call outside any
 *     stream capture;
 *   - all calls on one device share the array: two calls whose kernels can overlap on the GPU (different
 *     streams, different host threads) race and give wrong schedules.  Calls on one stream are safe, and a
 *     call never depends on what an earlier one left in the array.
 * No allocation routine of CUDA or of any library is called.  Outputs, errors and the one synchronisation
 * are those of jdb_schedule. */
#define JDB_STATIC_MAX_NODES 65536
jdb_status jdb_schedule_static(const jdb_forest *forest, jdb_sched *out, void *stream);

/* ---- launch counts at two granularities (Section 3: kernel versus subgraph statistics) ------- */

/* How many launches the forest costs without and with batching, counted at cell (subgraph) granularity, where two
 * cells share a launch only if they agree in depth and in their number of children, and at operator (kernel)
 * granularity, where 29 of a cell's 33 operators are shared by all cells of a depth and the 4 that depend on the
 * number of children are shared per (depth, number of children):
 *     cells:      n_nodes                 ->  number of distinct (depth, children) pairs
 *     operators:  33 * n_nodes            ->  sum over depths of (29 + 4 * kinds of cell at that depth)
 * The ratio unbatched / batched of a column is that granularity's batching ratio.  `sched` must come from
 * jdb_schedule on `forest`; `out` is a HOST struct; `ws` is device scratch of jdb_launch_counts_workspace_bytes
 * bytes, 8-byte aligned.  Synchronises `stream` once. */
typedef struct {
    int64_t cells_unbatched, cells_batched, ops_unbatched, ops_batched;
    int32_t n_levels, reserved;
} jdb_launch_stats;
size_t jdb_launch_counts_workspace_bytes(int32_t n_nodes);
jdb_status jdb_launch_counts(const jdb_forest *forest, const jdb_sched *sched, jdb_launch_stats *out, void *ws,
                             size_t ws_bytes, void *stream);

/* ---- batched execution (Section 4.3: stack, run the common subgraph once, slice) ------------ */

/* Weights arrive as the cell's natural matrices: W [4H, D], U [4H, H], b [4H], fp32 row-major, gate
 * row blocks in the order (i, o, u, f).  They are re-laid-out once for the kernels (and rounded to
 * bf16 for JDB_BF16); the packed buffer is reusable across forward calls. */
size_t jdb_packed_weights_bytes(int32_t D, int32_t H, int32_t precision);
jdb_status jdb_pack_weights(const float *W, const float *U, const float *b, int32_t D, int32_t H,
                            int32_t precision, void *packed, size_t packed_bytes, void *stream);

/* Bytes of device scratch for one forward call.  n_internal_bound is an upper bound on the number of
 * nodes that have children (n_nodes - sched.n_leaves when known, else n_nodes). */
size_t jdb_forward_workspace_bytes(int32_t n_nodes, int32_t n_internal_bound, int32_t D, int32_t H,
                                   int32_t precision);

/* Child-Sum Tree-LSTM over the whole forest, level by level (the cell cited in Section 3):
 *     h~_j = sum_k h_k;  (i, o, u) = (sig, sig, tanh)(W x_j + U h~_j + b);
 *     f_jk = sig(W_f x_j + U_f h_k + b_f);  c_j = i*u + sum_k f_jk*c_k;  h_j = o*tanh(c_j).
 * x        [n_nodes, D] row-major with leading dimension ldx (elements); x_dtype JDB_FP32 (float) or
 *          JDB_BF16 (bfloat16 bits).  JDB_FP32 precision requires fp32 x.
 * packed   from jdb_pack_weights with the same D, H, precision.
 * h, c     [n_nodes, H] fp32 outputs with leading dimension ldh, row v = node v; every node's state
 *          is returned.  Columns H..ldh-1 are not written.
 * Asynchronous on `stream` unless the level loop runs as one cooperative launch (persistent mode, or a
 * schedule from jdb_schedule_async), in which case the call synchronises at the end to report
 * JDB_ERR_NOT_A_FOREST / JDB_ERR_TIMEOUT.  With JDB_FLAG_NO_SYNC it does not synchronise either (as long as
 * the level count is known or H <= 192) and those two conditions are reported by jdb_sched_status.
 * JDB_FP32 with H > 192 and a schedule from jdb_schedule runs level by level through a tiled GEMM and synchronises once, at
 * its start, to read the level table (with JDB_FLAG_NO_SYNC, an explicit mode or the debug checks: the plain-ALU kernels).
 * A bounded wait that runs out inside one of the per-level launches (which are asynchronous) is likewise
 * visible through jdb_sched_status only.  JDB_BF16 with H > 192 runs one set of launches per level and needs the
 * level count on the host: after jdb_schedule_async the call first synchronises once to read it. */
jdb_status jdb_treelstm_forward(const jdb_forest *forest, const jdb_sched *sched, const void *x,
                                int32_t x_dtype, int64_t ldx, const void *packed, int32_t D, int32_t H,
                                float *h, float *c, int64_t ldh, const jdb_opts *opts, void *ws,
                                size_t ws_bytes, void *stream);

/* Synchronises `stream` and reports what the device recorded in sched->meta for the calls enqueued so far:
 * JDB_ERR_NOT_A_FOREST (analysis), JDB_ERR_TIMEOUT (a bounded wait ran out), else JDB_OK.  n_levels_out and
 * n_leaves_out (host, may be NULL) receive the counts.  The companion of jdb_schedule_async and
 * JDB_FLAG_NO_SYNC (deferred error reporting of the depth-ordered execution of Section 4.2). */
jdb_status jdb_sched_status(const jdb_sched *sched, int32_t *n_levels_out, int32_t *n_leaves_out, void *stream);

/* What JDB_FLAG_DEBUG_CHECKS recorded for the calls enqueued so far on this schedule (synchronises `stream`):
 * out[0] which check failed first (0 none; 1 node id from perm, 2 child id, 3 position in level order, 4 edge slot,
 * 5 parent row, 6 level offset, 7 edge offset), out[1] the offending value, out[2] the bound it was held against
 * (valid values are 0 .. bound-1), out[3] the position, slot, node or level at which it was met.  `out` is a host array.
 * The companion of the depth-ordered execution of Section 4.2 for callers that assemble schedules themselves. */
jdb_status jdb_debug_report(const jdb_sched *sched, int32_t out[4], void *stream);

/* ---- relatedness head (the scoring function of the workload of Section 5) --------------------- */

/* Scores pairs of trees from the states of their roots, with the head of the Tree-LSTM model the paper cites:
 *     h_s = sig(W_x (h_L * h_R) + W_+ |h_L - h_R| + b_h);  p = softmax(W_p h_s + b_p);  y = sum_k k p_k, k = 1..K.
 * h        [n_nodes, H] fp32 with leading dimension ldh: the h output of jdb_treelstm_forward.
 * left, right  [n_pairs] node ids of the two roots of every pair.
 * Wx, Wp   [Hs, H] row-major (the weights of the product and of the difference features), bh [Hs];
 * Wq [K, Hs], bq [K]; K <= 32; 4 (2 H + Hs) floats must fit 48 KB of shared memory (H up to about 1500), else
 * JDB_ERR_UNSUPPORTED.
 * y        [n_pairs] fp32 out;  p [n_pairs, K] fp32 out, may be NULL.
 * bad_flag one int32 on the device, set to 1 if a root id lies outside 0 .. n_nodes-1 (that pair is skipped), else 0.
 * All pointers are device pointers.  Asynchronous on `stream`; allocates nothing. */
jdb_status jdb_relatedness_head(const float *h, int64_t ldh, int32_t n_nodes, const int32_t *left, const int32_t *right,
                                int32_t n_pairs, const float *Wx, const float *Wp, const float *bh, const float *Wq,
                                const float *bq, int32_t H, int32_t Hs, int32_t K, float *y, float *p, int32_t *bad_flag,
                                void *stream);

/* ---- backward pass (training: the listing of Section 4.3 calls backward() inside the batching scope) ---------- */

/* Bytes of device scratch for one backward call.  n_internal_bound as for the forward workspace. */
size_t jdb_treelstm_backward_workspace_bytes(int32_t n_nodes, int32_t n_edges, int32_t n_internal_bound, int32_t H);

/* Gradients of L = sum_v <grad_h[v], h_v> + <grad_c[v], c_v> for the cell of jdb_treelstm_forward, over the same depth
 * table with the levels in DESCENDING order (a node's gradient is complete once its parent's level is done; Section 5
 * reports the training speed-up this pass takes part in).  fp32 throughout.
 * sched    from jdb_schedule on `forest` (the level count and level offsets are needed on the host: the call copies the
 *          level table back and synchronises `stream` ONCE before its launches; a schedule from jdb_schedule_async,
 *          whose counts were never read back, gives JDB_ERR_INVALID_ARG, and so does one whose node, leaf or edge
 *          totals do not fit this forest).
 * x        [n_nodes, D] fp32, leading dimension ldx.  W [4H, D], U [4H, H], b [4H]: the natural matrices, fp32
 *          row-major, gate row blocks (i, o, u, f), as given to jdb_pack_weights.
 * h, c     [n_nodes, H] fp32, leading dimension ldh: the outputs of the forward pass on the same inputs.
 * grad_h   [n_nodes, H] fp32, leading dimension ldg: dL/dh of every node (rows of nodes the loss does not see are
 *          zero); grad_c the same for c, or NULL for zeros.
 * dW [4H, D], dU [4H, H], db [4H]: outputs, dense, OVERWRITTEN (not accumulated).  dx [n_nodes, D] with leading
 * dimension lddx, or NULL to skip it.  The sums over nodes and edges behind dW, dU and db are split over CTAs whose
 * partial sums are added atomically, and so are the products of levels too small to fill the GPU otherwise: the last
 * bits of every output can differ from run to run.
 * ws       device scratch of jdb_treelstm_backward_workspace_bytes bytes, 256-byte aligned.
 * Everything after the one synchronisation is asynchronous on `stream`; allocates nothing on the device. */
jdb_status jdb_treelstm_backward(const jdb_forest *forest, const jdb_sched *sched, const float *x, int64_t ldx,
                                 const float *W, const float *U, const float *b, int32_t D, int32_t H, const float *h,
                                 const float *c, int64_t ldh, const float *grad_h, const float *grad_c, int64_t ldg,
                                 float *dW, float *dU, float *db, float *dx, int64_t lddx, void *ws, size_t ws_bytes,
                                 void *stream);

/* ---- nodes of several kinds: the table keyed by (depth, key) and its execution (Sections 4.2 and 4.3) ---------- */

/* Section 4.2 files every node under its depth and a key made of its type, its settings and the layout of its
 * arguments; nodes that share both share a slot, and the slots run in depth order, one batched launch each
 * (Section 4.3).  Here `key[v]` (0 .. n_keys-1) stands for that triple: equal keys are batchable with each other.
 * All arrays are caller-allocated device memory. */
typedef struct {
    int32_t *perm;       /* [n_nodes] node ids ordered by (depth, key, id)                                  */
    int32_t *slot_ptr;   /* [n_nodes + 1] capacity; entries 0..n_slots valid: first position of every slot  */
    int32_t *slot_depth; /* [n_nodes] capacity; depth of the nodes of slot s                                */
    int32_t *slot_key;   /* [n_nodes] capacity; their key                                                   */
    int32_t n_slots;     /* host; written by jdb_batch_plan                                                 */
    int32_t bad_key;     /* host; 1 if some key lay outside 0 .. n_keys-1 (it was filed as key 0)           */
} jdb_plan;

size_t jdb_batch_plan_workspace_bytes(int32_t n_nodes);

/* Builds the table from the depths of a schedule made by jdb_schedule on `forest` (its level count bounds the sort
 * key; n_levels * n_keys must stay below 2^31, else JDB_ERR_UNSUPPORTED).  Synchronises `stream` once to read back the
 * slot count.  A key out of range gives JDB_ERR_INVALID_ARG (the table is still complete, with that key taken as 0).
 * n_nodes = 0 gives n_slots = 0 and slot_ptr[0] = 0.  ws: device scratch, 256-byte aligned. */
jdb_status jdb_batch_plan(const jdb_forest *forest, const jdb_sched *sched, const int32_t *key, int32_t n_keys,
                          jdb_plan *out, void *ws, size_t ws_bytes, void *stream);

/* One kind of cell with its own parameters (Section 1 lets nodes share a batch only if they also share their parameters: nodes batch only with
 * nodes of the same cell).  W [4H, D], b [4H] in row blocks (i, o, u, f), fp32 row-major device arrays.
 * JDB_CELL_CHILDSUM: the cell of jdb_treelstm_forward, U [4H, H], any number of children.
 * JDB_CELL_NARY: the N-ary Tree-LSTM cell of the same cited model, one recurrent matrix per child position:
 *     (i, o, u) = (sig, sig, tanh)(W x + sum_l U^l h_l + b);  f_k = sig(W_f x + sum_l U_f^kl h_l + b_f);
 *     c = i*u + sum_k f_k*c_k;  h = o*tanh(c);
 *   U [(3 + arity) H, arity H]: row blocks (i, o, u, f_1 .. f_arity), column block l multiplies child l's h; a node
 *   with fewer children than `arity` (1 .. 8) treats the missing ones as zero states, one with more is an error. */
enum { JDB_CELL_CHILDSUM = 0, JDB_CELL_NARY = 1 };
typedef struct {
    int32_t kind;   /* JDB_CELL_* */
    int32_t arity;  /* JDB_CELL_NARY: child positions; ignored for JDB_CELL_CHILDSUM */
    const float *W;
    const float *U;
    const float *b;
} jdb_cell;

size_t jdb_cells_forward_workspace_bytes(int32_t n_nodes, int32_t n_edges, int32_t H, int32_t max_arity, int32_t n_keys);

/* Runs the table: for every slot in order, the cell `cells[slot_key]` over the slot's nodes as one batch (fp32 on the
 * CUDA cores: W x + b of the slot's rows, the recurrent products of the cell's kind, then its pointwise part).
 * cells    HOST array of n_keys descriptors (their W, U, b are device pointers).
 * key      the array given to jdb_batch_plan.  x [n_nodes, D] fp32 (ldx); h, c [n_nodes, H] fp32 outputs (ldh).
 * Copies the slot table to the host and synchronises `stream` once before its launches; a node with more children
 * than its cell's arity, or a plan that does not fit the forest's totals, gives JDB_ERR_INVALID_ARG.  Allocates nothing
 * on the device.  ws: device scratch of jdb_cells_forward_workspace_bytes bytes, 256-byte aligned. */
jdb_status jdb_cells_forward(const jdb_forest *forest, const jdb_plan *plan, const int32_t *key, const jdb_cell *cells,
                             int32_t n_keys, const float *x, int64_t ldx, int32_t D, int32_t H, float *h, float *c,
                             int64_t ldh, void *ws, size_t ws_bytes, void *stream);

/* ---- one call from host buffers (what a user without device arrays calls) -------------------- */

/* Device scratch needed by jdb_treelstm_forward_host (CSR, x, schedule, h, c and both workspaces). */
size_t jdb_forward_host_workspace_bytes(int32_t n_nodes, int32_t n_edges, int32_t D, int32_t H,
                                        int32_t precision, int32_t x_dtype);

/* child_ptr, child_idx, x, h, c are HOST pointers (pinned memory makes the copies asynchronous);
 * x is dense [n_nodes, D], h and c dense [n_nodes, H].  Copies the inputs to `dev_ws`, runs the
 * analysis and the forward there, copies h and c back and synchronises the stream at the end, where
 * JDB_ERR_NOT_A_FOREST and JDB_ERR_TIMEOUT are reported.  That is the only synchronisation for JDB_FP32 and for
 * JDB_BF16 with H <= 192; JDB_BF16 with H > 192 launches per level and synchronises once more, after the analysis,
 * to read the level count.  n_levels_out (host, may be NULL) receives the level count. */
jdb_status jdb_treelstm_forward_host(const int32_t *child_ptr, const int32_t *child_idx, int32_t n_nodes,
                                     int32_t n_edges, const void *x, int32_t x_dtype, const void *packed,
                                     int32_t D, int32_t H, float *h, float *c, const jdb_opts *opts,
                                     void *dev_ws, size_t dev_ws_bytes, int32_t *n_levels_out, void *stream);

/* ---- requests arriving one after the other (Section 2: serving, where requests arrive irregularly) ---------- */

/* Every request is a forest of its own, given as HOST buffers (pinned memory makes the copies asynchronous).  A request
 * takes the next of `slots` slots; a slot owns a stream and 1/slots of the caller's device scratch, so the copies and the
 * batching analysis of a new request run while earlier requests execute, and nothing waits for a batch to fill.
 * The object is host state only (streams, tickets); it allocates no device memory.  Not thread-safe: one thread submits
 * and waits. */
typedef struct jdb_online jdb_online;

size_t jdb_online_workspace_bytes(int32_t slots, int32_t max_nodes, int32_t max_edges, int32_t D, int32_t H,
                                  int32_t precision, int32_t x_dtype);

/* slots 1 .. 16; max_nodes / max_edges bound a single request; packed from jdb_pack_weights (opts->precision, D, H);
 * x_dtype of every request's x; dev_ws: jdb_online_workspace_bytes bytes of device memory, 256-byte aligned, owned by
 * the caller and in use until jdb_online_destroy.  opts' timing events and trace are ignored. */
jdb_status jdb_online_create(jdb_online **out, int32_t slots, int32_t max_nodes, int32_t max_edges, const void *packed,
                             int32_t D, int32_t H, const jdb_opts *opts, int32_t x_dtype, void *dev_ws,
                             size_t dev_ws_bytes);

/* Enqueues one request (arguments as jdb_treelstm_forward_host: child_ptr, child_idx, x dense [n_nodes, D] in; h, c
 * dense [n_nodes, H] out; all HOST pointers that must stay valid until the request has been waited for) and returns
 * its ticket (0, 1, 2, ... in submission order).  If the slot it takes still holds an earlier request, that one is
 * completed first (its status is kept for a later jdb_online_wait).  Does not wait for the new request, except that
 * JDB_BF16 with H > 192 synchronises once for its level count.  A request larger than max_nodes / max_edges gives
 * JDB_ERR_WORKSPACE and takes no ticket. */
jdb_status jdb_online_submit(jdb_online *o, const int32_t *child_ptr, const int32_t *child_idx, int32_t n_nodes,
                             int32_t n_edges, const void *x, float *h, float *c, int64_t *ticket);

/* Waits for one request (in any order) and returns ITS status: JDB_OK, JDB_ERR_NOT_A_FOREST, JDB_ERR_TIMEOUT...; other
 * requests are not affected by it.  n_levels_out (host, may be NULL) receives its level count. */
jdb_status jdb_online_wait(jdb_online *o, int64_t ticket, int32_t *n_levels_out);

/* Waits for everything in flight, destroys the streams and frees the host object. */
jdb_status jdb_online_destroy(jdb_online *o);

#ifdef __cplusplus
}
#endif
#endif /* JDB_H_ */
