/*
 * codedreduce.h -- C ABI of the B200 coded tree aggregation library (libcodedreduce.so).
 *
 * The library simulates, on ONE GPU, the per-iteration gradient aggregation of
 * CodedReduce (CR): N = n + n^2 + .. + n^L workers arranged in an (n, L)-regular
 * tree below a master (Section III-A), every worker holding r_CR * P data
 * partitions with combining coefficients (CR.Allocate, Algorithm 2; CompAlloc,
 * Algorithm 1), every parent recovering a combination of its children's
 * messages from any n-s of them with a gradient-coding decode row and adding
 * its own coded gradient (CR.Execute, Algorithm 2), the master ending with the
 * exact gradient sum of Eq. (g).  Straggler sets are inputs (bit masks).
 *
 * Conventions common to all calls
 *   - Indices are 0-based.  Layer l = 1..L holds n^l nodes; node (l, i) has flat
 *     index offset(l) + i with offset(l) = n + .. + n^(l-1); its children are
 *     (l+1, n*i .. n*i + n-1).  The master is layer 0.
 *   - A sibling group is the n children of one parent.  Group 0 is the master's;
 *     the group below flat node v is v + 1.  There are 1 + n + .. + n^(L-1) groups.
 *   - A straggler mask is a uint32 whose bit j marks child j of the group as a
 *     straggler.  More than s bits set in a group that is consulted makes the
 *     pattern undecodable (the failure case of the second remark after
 *     Theorem 1); masks of groups below an unused child are ignored.
 *   - "device pointer" = memory of the plan's CUDA device, owned by the caller
 *     (e.g. allocated through PyTorch); "host pointer" = ordinary host memory.
 *     The library never frees or keeps caller buffers beyond the work it
 *     enqueues.  Device buffers of element type float (CR_F32) or int32_t
 *     (CR_I32) must be 4-byte aligned; 16-byte alignment and d % 4 == 0 enable
 *     the TMA path, anything else silently takes the plain-load kernels.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Device
 *     calls only enqueue work and small async copies; they do not synchronise.
 *     A plan is not thread-safe, and its device calls share plan-owned staging and
 *     scratch buffers: work of one plan that may overlap on the device (two streams)
 *     must be ordered by the caller (one stream, or events between the streams).
 *   - Every function returns a cr_status_t (CR_OK = 0) unless stated; nothing
 *     aborts or traps.  All argument and mask validation happens on the host
 *     before anything is launched.  There is no CPU fallback: device calls on a
 *     host-only plan return CR_ERR_CUDA.
 */
#ifndef CODEDREDUCE_H
#define CODEDREDUCE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cr_plan cr_plan_t;
typedef struct cr_schedule cr_schedule_t;

typedef enum {
    CR_OK = 0,
    CR_ERR_INVALID_ARG = 1,         /* NULL pointer, n/L/s/d out of range, bad flags, mask bit >= n */
    CR_ERR_BAD_PARTITION_COUNT = 2, /* P is not a multiple of sum_l n^l (s+1)^(L-l) */
    CR_ERR_CODE_UNAVAILABLE = 3,    /* code does not exist for this (n, s) */
    CR_ERR_ILL_CONDITIONED = 4,     /* no encoding matrix with kappa <= max_kappa / span property fails */
    CR_ERR_UNDECODABLE_MASK = 5,    /* > s stragglers in a consulted group */
    CR_ERR_DTYPE = 6,               /* integer mode asked of a non-integer code, or dtype mismatch */
    CR_ERR_CUDA = 7,                /* a CUDA call failed, or device work asked of a host-only plan */
    CR_ERR_OOM = 8,                 /* workspace too small / allocation failed */
    CR_ERR_TIMEOUT = 9              /* a bounded device-side wait gave up (reported by cr_plan_device_status) */
} cr_status_t;

/* Which gradient-coding encoding matrix B the plan builds (Section II-C). */
typedef enum {
    CR_CODE_CYCLIC_RANDOM = 0,         /* cyclic support {i..i+s}, random null-space construction */
    CR_CODE_FRACTIONAL_REPETITION = 1, /* 0/1 rows, n/(s+1) blocks of s+1 identical workers */
    CR_CODE_PAPER_3_1 = 2,             /* the (A, B) printed in Eq. (gc3nodes); n = 3, s = 1 only */
    CR_CODE_EXPLICIT = 3               /* caller supplies B per level */
} cr_code_t;

typedef enum { CR_F32 = 0, CR_I32 = 1 } cr_dtype_t;

/* Problem statement, mirroring the inputs of Algorithm 2: the (n, L) tree, the
 * straggler tolerance s per parent, the data set as P atomic partitions, the
 * gradient length d (the paper's p). */
typedef struct {
    int32_t n;          /* children per parent, 2..16 */
    int32_t L;          /* worker layers, 1..8 */
    int32_t s;          /* stragglers tolerated per sibling group, 0..n-1 */
    int32_t P;          /* atomic data partitions; multiple of sum_l n^l (s+1)^(L-l) */
    int64_t d;          /* gradient length, >= 1 */
    int32_t code;       /* cr_code_t */
    int32_t dtype;      /* cr_dtype_t of G_slots / outputs */
    uint64_t seed;      /* CR_CODE_CYCLIC_RANDOM: first sub-seed tried */
    const double *B_explicit; /* host, [L][n][n] row-major (level l = matrix used by parents at layer l),
                                 read during cr_plan_create only; NULL unless CR_CODE_EXPLICIT */
    double max_kappa;   /* conditioning screen for random codes; <= 0 selects 100 */
    int32_t device;     /* CUDA device ordinal, or -1 for a host-only plan (queries only) */
    int32_t reserved;   /* must be 0 */
} cr_plan_desc_t;

/* Variants of cr_aggregate (low byte of `flags`) and option bits. */
enum {
    CR_AGG_FUSED = 0,        /* one kernel, TMA-staged tiles, all levels in registers/shared memory.  Single
                                patterns for which the plain-load form measures faster take it unless
                                cr_plan_tune fixed a TMA shape: m <= 4 or m = 8 slot rows per node at
                                d >= 2^19, m = 12, 16, .. for 2^19 <= d <= 2^23, and CR_AGG_FROM_CODED;
                                cr_plan_last_kernel tells which kernel served a call */
    CR_AGG_FUSED_LDG = 1,    /* same dataflow with plain 128-bit loads (any d, any alignment) */
    CR_AGG_UNFUSED = 2,      /* cr_encode + cr_decode per level through the workspace */
    CR_AGG_UNCODED_SUM = 3,  /* comparator: plain sum of the same used slots, all weights 1 */
    CR_AGG_VARIANT_MASK = 0xff,
    CR_AGG_ALL_NODES = 0x100, /* CR_AGG_UNFUSED only: encode and decode every node, not just used ones */
    CR_AGG_FROM_CODED = 0x200 /* the first buffer is E [N][d] (coded gradients of cr_coded_gradients or cr_encode),
                                 not G_slots: the encode step is skipped.  Not with CR_AGG_UNFUSED. */
};

/* Per-sample loss whose gradient the workers compute (Eq. (g) leaves the loss generic; the paper's
 * experiments use linear regression on synthetic data and logistic regression on real data, Section V). */
typedef enum {
    CR_LOSS_SQUARED = 0,  /* 1/2 (x.w - y)^2        : gradient X^T (X w - y) */
    CR_LOSS_LOGISTIC = 1  /* log(1+e^{x.w}) - y x.w : gradient X^T (sigmoid(X w) - y), labels y in {0,1} */
} cr_loss_t;

/* ---- plan: CR.Allocate + the gradient-coding tables (host work, once) ------------------------
 * cr_plan_create builds the tree indexing, the per-level encoding matrices B (Section II-C), the
 * allocation of (partition, coefficient) pairs to every node by the recursion of Algorithm 2
 * (CR.Allocate) over CompAlloc (Algorithm 1): a parent's pass-down list is cut into n equal
 * consecutive chunks, child i receives chunk kappa scaled by b_{i,kappa} for every non-zero entry in
 * increasing kappa, keeps the first m = r_CR * P pairs (Theorem 1) and passes the rest down.  It also
 * solves, in fp64, the decode row a (a B = 1, supported on the lowest-indexed n-s non-stragglers)
 * for every straggler mask with at most s bits, per level.  With device >= 0 it makes that device
 * current for the call and allocates small device mirrors of the tables and a ring of eight staging
 * buffers (pinned host + device; 64 KB to 1 MB each, sized for batches of 64 patterns), through which
 * cr_aggregate and cr_decode send the expanded straggler patterns.  The first call whose tables exceed a
 * buffer (a larger batch) re-allocates the ring once, which synchronises the device; cr_schedule_create
 * keeps even that out of a loop.  cr_plan_destroy frees everything.  *out is written only on CR_OK. */
cr_status_t cr_plan_create(const cr_plan_desc_t *desc, cr_plan_t **out);
cr_status_t cr_plan_destroy(cr_plan_t *plan);

/* Human-readable name of a status code (static storage). */
const char *cr_status_string(int status);
/* Text of the last CUDA error seen by the calling thread ("" if none); valid until the next error. */
const char *cr_last_cuda_error(void);

/* Read-only queries; outputs are caller-allocated host memory. */
int32_t cr_plan_num_nodes(const cr_plan_t *plan);   /* N */
int32_t cr_plan_num_groups(const cr_plan_t *plan);  /* N / n */
int32_t cr_plan_load(const cr_plan_t *plan);        /* m = r_CR * P slots per node */
int64_t cr_plan_int_scale(const cr_plan_t *plan);   /* CR_I32: S = sigma^L with sigma*B integer; else 1 */
/* B used by the parents at `level` (0 = master .. L-1), n*n row-major; kappa and the sub-seed that
 * produced it (either pointer may be NULL). */
cr_status_t cr_plan_get_B(const cr_plan_t *plan, int32_t level, double *B, double *kappa, uint64_t *sub_seed);
/* D(l,i) of flat node `node`: m partition ids and their combining coefficients (Section III-A,
 * "scaled data sets").  In CR_I32 plans the coefficients returned are still the real ones; the
 * device uses S * coeff. */
cr_status_t cr_plan_get_slots(const cr_plan_t *plan, int32_t node, int32_t *part, double *coeff);
/* Decode row (n doubles) a parent at `level` uses for `straggler_mask`; CR_ERR_UNDECODABLE_MASK if
 * the mask has more than s bits. */
cr_status_t cr_plan_get_decode(const cr_plan_t *plan, int32_t level, uint32_t straggler_mask, double *a);
/* Host expansion of one straggler pattern (masks[num_groups]) into the post-order list of nodes
 * whose data is consumed: nodes[k], layers[k] (1..L) and the decode weight with which node k's
 * message enters its parent.  capacity >= N always suffices; *count receives the length. */
cr_status_t cr_plan_expand(const cr_plan_t *plan, const uint32_t *masks, int32_t capacity,
                           int32_t *nodes, int32_t *layers, double *weights, int32_t *count);
/* Which children each parent ends up not waiting for, from the workers' computation times: the
 * run-time model of Section III-C.  compute_time[v] (host, N doubles, >= 0) is the time node v needs
 * for its local coded gradient (the paper draws it from the shifted exponential of Eq. (comp_model));
 * a parent receives one message at a time (single-port model), each taking t_c, in the order in which
 * its children's messages become ready (ties: lower index first); a node's message is ready once it
 * holds n-s children messages and its own gradient (leaves: their own gradient).  The s children of
 * every group whose messages would come last are marked in masks_out[num_groups] (host), ready to be
 * passed to cr_aggregate; *t_total (may be NULL) receives the time at which the master holds its n-s
 * messages, i.e. one sample of T_CR of Theorem 2.  Host work only. */
cr_status_t cr_latency_masks(const cr_plan_t *plan, const double *compute_time, double t_c, uint32_t *masks_out,
                             double *t_total);

/* Status word written by bounded device-side waits: CR_OK, or CR_ERR_TIMEOUT if a kernel of this plan
 * gave up waiting for a copy.  The word is sticky on purpose -- results produced after a timeout are
 * not to be trusted until someone has looked -- and stays set until cr_plan_clear_status.  Both calls
 * synchronise the device. */
cr_status_t cr_plan_device_status(cr_plan_t *plan);
cr_status_t cr_plan_clear_status(cr_plan_t *plan);
/* Bound of every device-side wait of this plan's kernels, in nanoseconds (default 2e9; accepted range
 * 1e3 .. 6e10).  It travels to the kernels as an argument of each launch. */
cr_status_t cr_plan_set_wait_limit(cr_plan_t *plan, uint64_t limit_ns);
/* Shows the give-up path without harming anything: enqueues one small kernel whose single thread waits
 * limit_ns (1e3 .. 1e8) on a barrier that nobody completes, through the same bounded wait as the
 * aggregation and gradient kernels, and then sets the status word as they would.  No copy is in flight
 * and nothing traps; afterwards cr_plan_device_status returns CR_ERR_TIMEOUT until the word is cleared. */
cr_status_t cr_selftest_wait(cr_plan_t *plan, uint64_t limit_ns, void *stream);

/* ---- CR.Execute step 1, the workers' local partial gradients (Section III-A, Algorithm 2) ------
 * Linear-regression instance of Eq. (g): for every node v and slot j holding partition p,
 *   G_slots[v][j][:] = X_p^T (X_p w - y_p).
 * X [P][rows][d], y [P][rows], w [d], G_slots [N][m][d]: device pointers, fp32, row-major.
 * Two kernels serve it: when d % 4 == 0, d <= 8192 and X, w, G_slots are 16-byte aligned, a one-pass
 * kernel (row blocks staged by TMA bulk copies, a cluster of CTAs per slot, reduction through
 * distributed shared memory) that needs no scratch; otherwise a two-pass kernel pair that keeps the
 * residuals (one per node, slot and row) in `workspace`, device scratch of at least
 * cr_partial_gradients_workspace_bytes(plan, rows) bytes (CR_ERR_OOM if it is needed and missing).
 * CR_F32 plans only. */
size_t cr_partial_gradients_workspace_bytes(const cr_plan_t *plan, int32_t rows);
cr_status_t cr_partial_gradients(cr_plan_t *plan, const float *X, const float *y, int32_t rows,
                                 const float *w, float *G_slots, void *workspace,
                                 size_t workspace_bytes, void *stream);

/* The same pass for either loss (cr_partial_gradients is the CR_LOSS_SQUARED case). */
cr_status_t cr_partial_gradients_loss(cr_plan_t *plan, int32_t loss, const float *X, const float *y, int32_t rows,
                                      const float *w, float *G_slots, void *workspace, size_t workspace_bytes,
                                      void *stream);

/* ---- CR.Execute step 1 in coded form: every node's local coded gradient in one pass (Section III-A) ----
 * E[v][:] = g_{D(l,i)} = sum_j c_{v,j} * X_p^T r_p with p the partition of slot j of node v
 * (Section III-A: D(l,i) carries the combining coefficients along with its data points), r_p the
 * residuals of `loss` at w.  The slot gradients are never written: each node's cluster of CTAs walks
 * the rows of all its m slots and scales the residuals by the slot's coefficient.  X [P][rows][d],
 * y [P][rows], w [d], E [N][d]: device pointers, fp32.  Needs d % 4 == 0, d <= 8192 and 16-byte
 * aligned X, w, E (CR_ERR_INVALID_ARG otherwise: use cr_partial_gradients_loss + cr_encode).  Feed E
 * to cr_aggregate with CR_AGG_FROM_CODED, or to cr_decode level by level.  CR_F32 plans only. */
cr_status_t cr_coded_gradients(cr_plan_t *plan, int32_t loss, const float *X, const float *y, int32_t rows,
                               const float *w, float *E, void *stream);

/* ---- partial gradients of K models in one pass (tensor cores) ----------------------------------
 * Eq. (g) evaluated at K <= 32 models w_1..w_K at once (the candidates of a line search, several step
 * sizes, an ensemble): for every node v, slot j with partition p and every k,
 *   G_multi[k][v][j][:] = X_p^T (link(X_p w_k) - y_p),   link = identity or sigmoid by `loss`.
 * With K columns the two products are dense contractions and run on the tensor cores (tcgen05,
 * kind::tf32, fp32 accumulation in tensor memory).  Precision: the tensor core reads the upper 19 bits
 * of each fp32 of X, so results carry fp32 accuracy only for X whose values are TF32-representable
 * (low 13 mantissa bits zero); otherwise X is in effect truncated to TF32.  W and the residuals are
 * split into two TF32 terms and are not truncated.  The tensor core's fp32 accumulator truncates on
 * every addition; the kernels spread each sum over 8 accumulators, which keeps the relative L2 error
 * against exact arithmetic under 1e-5 for d <= 32768 and rows <= 16384 (it grows linearly beyond).
 * X [P][rows][d], y [P][rows], W [K][d], G_multi [K][N][m][d], R_out [N][m][rows][K] or NULL
 * (the residuals, for inspection): device pointers, fp32.  `workspace`: device scratch of at least
 * cr_partial_gradients_multi_workspace_bytes(plan, rows) bytes (CR_ERR_OOM if smaller).  Needs
 * d % 4 == 0, d >= 32, 1 <= K <= 32, N*m <= 65535 and 16-byte aligned X, G_multi, workspace
 * (CR_ERR_INVALID_ARG otherwise).  Each G_multi[k] is a G_slots buffer for cr_aggregate.  CR_F32
 * plans only. */
size_t cr_partial_gradients_multi_workspace_bytes(const cr_plan_t *plan, int32_t rows);
cr_status_t cr_partial_gradients_multi(cr_plan_t *plan, int32_t loss, const float *X, const float *y, int32_t rows,
                                       const float *W, int32_t K, float *G_multi, float *R_out, void *workspace,
                                       size_t workspace_bytes, void *stream);

/* ---- the same partial-gradient pass for callers that cannot allocate device memory ----------------
 * (No counterpart in the paper: this is a packaging variant of cr_partial_gradients.)
 * Some callers have no way to provide the residual workspace: a host thread that runs inside a
 * latency-critical loop where cudaMalloc would stall the whole device, a process whose device memory
 * has been handed in full to another component's pool, a plug-in that is given raw pointers and a
 * stream but no allocator.  For them the residuals (one float per node, slot and row) live in a fixed
 * array inside the library: 4 MiB of device memory on every GPU that loads the library, kept until the
 * process exits.  Arguments, layouts and results are those of cr_partial_gradients (squared loss);
 * the work is always done by the two-pass kernel pair, whatever d is, since that is the form that
 * needs the scratch.
 *   - N * m * rows must not exceed cr_partial_gradients_static_capacity() (1,048,576 residuals);
 *     larger problems return CR_ERR_OOM with an explanatory cr_last_cuda_error() text and launch nothing.
 *   - The call never allocates or frees (no cudaMalloc/cudaFree, no staging buffers, no library
 *     allocator).  The first call on each device looks up the array's device address; make that first
 *     call outside of any stream capture.
 *   - Every call on a device shares the one array and finds the previous call's residuals in it; each
 *     call overwrites every entry it later reads, so nothing needs clearing.  Two calls whose kernels
 *     can overlap on the same GPU (different streams, different plans, different threads) race on it:
 *     order them on one stream or with events. */
size_t cr_partial_gradients_static_capacity(void);
cr_status_t cr_partial_gradients_static(cr_plan_t *plan, const float *X, const float *y, int32_t rows,
                                        const float *w, float *G_slots, void *stream);

/* ---- CR.Execute, local coded gradient g_{D(l,i)} (Section III-A) ------------------------------
 * E[v][:] = sum_j c_{v,j} * G_slots[v][j][:] for every node v.  G_slots [N][m][d], E [N][d]:
 * device pointers of the plan's dtype.  (Verification path; the fused kernel never writes E.) */
cr_status_t cr_encode(cr_plan_t *plan, const void *G_slots, void *E, void *stream);

/* ---- CR.Execute, one level of "decode from any n-s children, add own, upload" -----------------
 * For every parent i at `parent_layer` (L-1 .. 0; 0 = master):
 *   M_parent[i][:] = sum_j a[j] * M_child[n*i + j][:]  (+ E_parent[i][:] unless parent_layer == 0)
 * with a the decode row for masks_host[i].  M_child [n^(parent_layer+1)][d], E_parent
 * [n^parent_layer][d] (the slice of E for that layer; NULL at layer 0), M_parent
 * [n^parent_layer][d]: device pointers.  masks_host: host, one per parent of the layer.
 * Children with zero weight are not read. */
cr_status_t cr_decode(cr_plan_t *plan, int32_t parent_layer, const void *M_child, const void *E_parent,
                      const uint32_t *masks_host, void *M_parent, void *stream);

/* ---- CR.Execute end to end for `batch` straggler patterns --------------------------------------
 * g_out[b][:] = root result for pattern b.  G_slots [N][m][d] and g_out [batch][d] are device
 * pointers; masks_host is host memory [batch][num_groups].  Only nodes with non-zero decode weight
 * along the tree are read.  In CR_I32 plans all arithmetic is int32 on S-scaled integer
 * coefficients and the root divides by S exactly (wrap-around on overflow is the caller's concern).
 * workspace: device scratch, needed by CR_AGG_UNFUSED only
 * (cr_aggregate_workspace_bytes); may be NULL otherwise. */
size_t cr_aggregate_workspace_bytes(const cr_plan_t *plan, int32_t batch, uint32_t flags);
cr_status_t cr_aggregate(cr_plan_t *plan, const void *G_slots, const uint32_t *masks_host, int32_t batch,
                         void *g_out, uint32_t flags, void *workspace, size_t workspace_bytes, void *stream);

/* ---- CR.Execute with the straggler sets fixed in advance ------------------------------------------
 * The straggler sets are an input of CR.Execute (Algorithm 2); everything cr_aggregate derives from them
 * -- the post-order list of consumed nodes with their decode weights, the union of a batch, the tables
 * of the batch kernel -- depends on the masks alone, not on the gradients.  cr_schedule_create does that
 * work once for `batch` patterns (masks_host [batch][num_groups], host) and `flags` (as cr_aggregate) and
 * keeps the tables in device memory it allocates; cr_aggregate_scheduled then only launches: no mask is
 * validated or expanded, nothing is allocated and nothing is copied.  A schedule belongs to its plan,
 * may be used any number of times, by one stream at a time like the plan itself, and must be destroyed
 * before the plan.  Results are those of cr_aggregate with the same masks and flags, bit for bit.
 * Since it only enqueues kernels, a cr_aggregate_scheduled call (and a cr_partial_gradients_loss call in
 * front of it) may be captured in a CUDA graph on a capturing stream and replayed; the graph then holds
 * the schedule, the buffers and the plan by address, so they must outlive it.
 * cr_schedule_bytes: the algorithmic bytes of one call (as cr_aggregate_bytes). */
cr_status_t cr_schedule_create(cr_plan_t *plan, const uint32_t *masks_host, int32_t batch, uint32_t flags,
                               cr_schedule_t **out);
cr_status_t cr_schedule_destroy(cr_schedule_t *sched);
cr_status_t cr_schedule_bytes(const cr_schedule_t *sched, int64_t *bytes, int32_t *used_nodes);
cr_status_t cr_aggregate_scheduled(cr_plan_t *plan, const void *G_slots, const cr_schedule_t *sched, void *g_out,
                                   void *workspace, size_t workspace_bytes, void *stream);

/* Same computation with HOST buffers: copies from G_slots_host (pinned or pageable host memory,
 * [N][m][d]) into dev_slots the slots of the nodes that the batch consumes (the rest of dev_slots is
 * left as it is: a straggler's data is never waited for; all nodes with CR_AGG_ALL_NODES), runs
 * cr_aggregate, copies the result into g_out_host and waits for the stream.  dev_slots [N][m][d] and
 * dev_out [batch][d] are caller-owned device staging buffers.  The bytes that cross the bus are those
 * of cr_aggregate_bytes. */
cr_status_t cr_aggregate_host(cr_plan_t *plan, const void *G_slots_host, const uint32_t *masks_host,
                              int32_t batch, void *g_out_host, uint32_t flags, void *dev_slots,
                              void *dev_out, void *workspace, size_t workspace_bytes, void *stream);

/* Algorithmic bytes of one cr_aggregate call: element size * d * (m * |union of used nodes| + batch),
 * i.e. every used slot read once and every output written once.  *used_nodes (may be NULL)
 * receives the size of the union. */
cr_status_t cr_aggregate_bytes(const cr_plan_t *plan, const uint32_t *masks_host, int32_t batch,
                               int64_t *bytes, int32_t *used_nodes);

/* Launch shape of the TMA kernels of cr_aggregate; 0 keeps the built-in choice for that field.
 * Single-pattern kernel: consumer_warps in {2,4,8} (column tile = 128 * consumer_warps), stages = depth
 * of the shared-memory ring (2..16), ctas_per_sm = persistent CTAs per SM (1..8), rows_per_box = slot
 * rows per TMA box (must divide m, at most 16).  Batch kernel (one CTA per SM): consumer_warps = replay
 * warps (4 or 8), stages = boxes per loader warp, ctas_per_sm = loader warps (4 or 6), rows_per_box as
 * above.  With both left at 0, a batch whose union is small enough for two CTAs of eight warps (four loaders,
 * four replay warps) to share an SM runs in that form.  Shapes that do not fit shared memory fall back to
 * smaller ones or to plain loads. */
cr_status_t cr_plan_tune(cr_plan_t *plan, int32_t consumer_warps, int32_t stages, int32_t ctas_per_sm,
                         int32_t rows_per_box);

/* Batches of patterns (CR_AGG_FUSED, batch > 1, L >= 2): a parent's message depends only on the straggler
 * sets of its own sub-tree (CR.Execute), so the patterns of a batch can share the messages of the nodes
 * whose children are leaves.  share_messages: 0 = share when it halves the replay work (built-in
 * choice), 1 = never, 2 = whenever the tables fit.  Read when a batch is expanded
 * (cr_aggregate, cr_schedule_create).  e_buffers: buffers of coded gradients the batch kernel keeps in
 * shared memory, 0 = built-in choice (two when they fit beside tall boxes), 1 or 2; one buffer leaves
 * room for more and deeper loader rings (cr_plan_tune). */
cr_status_t cr_plan_tune_batch(cr_plan_t *plan, int32_t share_messages, int32_t e_buffers);
/* Host work only (also on host-only plans): what the expansion of `batch` patterns (masks_host
 * [batch][num_groups]) amounts to under the sharing rule `share_messages` (as above).  stats[0] = entries of the
 * patterns' schedules (consumed nodes, summed over the batch), [1] = nodes in the union, [2] = nodes of layer L-1
 * whose messages are shared (0: the batch does not share), [3] = distinct message variants over those nodes
 * (a variant = a distinct decode row over the node's children in the union), [4] = entries of the reduced
 * schedules (a consumed node of layer L-1 counts once, its leaves not at all), [5] = rows of a buffer of coded
 * gradients in the batch kernel (the union, plus variants that found no dead row to reuse). */
cr_status_t cr_plan_batch_stats(const cr_plan_t *plan, const uint32_t *masks_host, int32_t batch, int32_t share_messages,
                                int64_t *stats);

/* Launch shape of the one-pass partial-gradient kernel; 0 keeps the built-in choice for that field.
 * block_kb = KB of X per staged row block (1..128), stages = row-block buffers per CTA (2..8),
 * cluster = CTAs that share one (node, slot) item (1, 2, 4 or 8).  A shape that does not fit shared
 * memory makes cr_partial_gradients return CR_ERR_CUDA. */
cr_status_t cr_plan_tune_gradients(cr_plan_t *plan, int32_t block_kb, int32_t stages, int32_t cluster);

/* Order in which the partial-gradient kernels launch the (node, slot) items, and ring depth of the
 * second kernel of cr_partial_gradients_multi; 0 keeps the built-in choice for that field.
 * item_order: 1 = by node, then slot; 2 = grouped by partition (items that hold the same partition
 * run side by side and share its rows through L2; the built-in choice of every partial-gradient kernel).
 * multi_stages: 2..4 (2 lets two CTAs share an SM). */
cr_status_t cr_plan_tune_items(cr_plan_t *plan, int32_t item_order, int32_t multi_stages);

/* Kernel launches enqueued by this plan's device calls so far. */
int64_t cr_plan_launch_count(const cr_plan_t *plan);

/* Name of the kernel (family) that served this plan's latest cr_aggregate call; "" before the first.
 * The string is static storage owned by the library. */
const char *cr_plan_last_kernel(const cr_plan_t *plan);

#ifdef __cplusplus
}
#endif
#endif /* CODEDREDUCE_H */
