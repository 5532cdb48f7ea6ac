// Launch wrappers of the sm_100a kernels (implemented in cr_kernels.cu).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace cr {

// One consumed node of an expanded straggler pattern, as the kernels read it (16 bytes).
struct Step {
    int32_t node;    // flat node index: its slots are rows node*m .. node*m+m-1 of G_slots
    int32_t layer;   // bits 0..7: layer 1..L; bit 8: first consumed child of its parent
    uint32_t wbits;  // decode weight of the node's message at its parent: float bits (CR_F32) or int32 (CR_I32)
    int32_t index;   // batch kernel: position of the node in the union list (bits 0..11) and, when the batch
                     // has a weight table, the index of wbits in it (bits 12..); otherwise unused
};

// Tuning of the TMA kernels; 0 selects the built-in choice.
struct Tuning {
    int ncw = 0;          // consumer warps per CTA (single-pattern kernel: tile = 128 * ncw columns)
    int stages = 0;       // depth of the shared-memory ring
    int ctas_per_sm = 0;  // persistent CTAs per SM (batch kernel, always one CTA per SM: loader warps, 4 or 6)
    int rows = 0;         // slot rows per TMA box (must divide m)
    int pg_block_kb = 0;  // partial gradients: KB of X per staged row block
    int pg_stages = 0;    // partial gradients: row-block buffers per CTA
    int pg_cluster = 0;   // partial gradients: CTAs per (node, slot) item (1, 2, 4 or 8)
    int pg_order = 0;     // partial gradients: launch order of the items: 1 (node, slot), 2 grouped by partition
    int tc_stages = 0;    // multi-model gradients: ring depth of the X^T R kernel (2..4)
    int share = 0;        // batch kernel, messages shared by the patterns of a batch: 0 when it pays, 1 never, 2 always
    int e_buffers = 0;    // batch kernel: buffers of coded gradients in shared memory (1 or 2)
    unsigned long long wait_limit_ns = 2000000000ull;  // bound of every device-side wait
};

struct DeviceInfo {
    int sm_count = 0;
    int smem_optin = 0;  // bytes of dynamic shared memory a CTA may opt in to
    int smem_per_sm = 0;
};

struct AggArgs {
    const void *G;        // [N*m][d]
    const void *coeff;    // [N*m] element type T
    const Step *steps;    // device: all patterns' steps, concatenated (may be null for launch_fused_tma
                          // when host_steps is given and short enough to travel in the kernel parameters)
    const Step *host_steps;  // host copy of the same entries, or null
    const int32_t *pat_off;  // device [batch+1]: pattern b owns steps pat_off[b] .. pat_off[b+1]-1
    const int32_t *unodes;   // device [n_union]: union of used nodes (batch kernel)
    const uint32_t *wtab;    // device [n_wtab]: distinct weight bit patterns of the batch (n_wtab = 0: none)
    int n_wtab;
    // batch kernel, few slot rows per node: n_boxes TMA boxes that each cover up to `npb` union nodes with
    // consecutive ids (their slot rows are contiguous); npb <= 1: one node per box.
    int n_boxes = 0;
    int npb = 0;
    // batch kernel: device table of unit records, one per box of a tile, laid out for the BatchShape the
    // launch uses (16-byte aligned)
    const uint32_t *units = nullptr;
    int n_union;
    int batch;
    int total_steps;
    int m;
    int L;                // layers of the schedules (with shared messages: of the reduced ones, one less than the tree's)
    int64_t d;
    int64_t rows_total;   // N*m
    void *out;            // [batch][d]
    int shift;            // CR_I32: arithmetic right shift applied at the root
    int *status;          // device status word (bounded waits)
    int is_int;
    int same_shape;       // batch > 1: all patterns' schedules share length and layer sequence
    // batch kernel, messages shared by the patterns (n_ops > 0): an E buffer has n_rows rows (the union nodes,
    // then extra message rows); ops / vtab as in BatchArgs (device pointers)
    int n_rows = 0;
    int n_ops = 0;
    const int4 *ops = nullptr;
    const uint32_t *vtab = nullptr;
    int vtab_words = 0;
    void *split_scratch = nullptr;  // launch_fused_ldg, single inline schedule: [n][d] scratch; when set, the
                                    // sub-trees below the master run as separate blocks (see launch_fused_ldg)
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Each returns cudaSuccess or the first CUDA error; *launches is incremented per kernel launched.
// `can_tma` tells whether d and the pointers meet the TMA alignment rules.
bool tma_eligible(const AggArgs &a);
// Longest single-pattern schedule that launch_fused_tma can pass inside the kernel parameters.
int inline_schedule_limit();

cudaError_t launch_fused_tma(const AggArgs &a, const DeviceInfo &dev, const Tuning &tune, EncodeTiledFn encode,
                             cudaStream_t stream, int64_t *launches, bool *done);
// Launch shape of the batch kernel for one expanded batch: depends on the tree, the union, the tables and the
// device, not on any pointer, so it is fixed when the batch is expanded (the unit records are laid out for it).
struct BatchShape {
    bool ok = false;       // false: the union does not fit shared memory, the batch kernel cannot serve this batch
    int nbuf = 0;          // buffers of coded gradients
    int stages = 0;        // boxes per loader ring
    int R = 0;             // slot rows per box
    int nlw = 0, nrw = 0;  // loader and replay warps
    int multi = 0;         // a box covers several small nodes
    int cpn = 1;           // boxes per group (a tall node cut into cpn boxes)
    int n_groups = 0;      // groups of boxes per tile
    int nst = 0;           // same-shape batches: entries per schedule
    int n_rows = 0;        // rows of a buffer of coded gradients
    int vtab_smem = 0;
    int grid = 0;
    size_t sched_bytes = 0, smem = 0;
};
BatchShape batch_shape(const AggArgs &a, const DeviceInfo &dev, const Tuning &tune);
// Words of a unit record: 16 coefficients (zero beyond the rows in use), then {first slot row of the box, E row
// of the first node the box completes, rows after which a node is complete (0: it continues in the next box of
// the group), rows of the box in use}.
int unit_words();
cudaError_t launch_fused_batch_tma(const AggArgs &a, const BatchShape &shape, const Tuning &tune, EncodeTiledFn encode,
                                   cudaStream_t stream, int64_t *launches, bool *done);
// With a.split_scratch the schedule of a single pattern is cut at the master's children: every layer-1
// sub-tree is folded by its own blocks into a row of the scratch, and a second small kernel adds the
// rows (the master's decode).  For short vectors, where one block per column range would walk all the
// nodes of a large tree one after the other.
cudaError_t launch_fused_ldg(const AggArgs &a, cudaStream_t stream, int64_t *launches);
// Largest number of sub-trees below the master that the split form handles (= largest n).
int split_limit();
cudaError_t launch_uncoded_sum(const AggArgs &a, cudaStream_t stream, int64_t *launches);

// E[v][:] = sum_j coeff[v*m+j] * G[v*m+j][:] for the nodes listed in `nodes` (device, count entries) or
// for all N nodes when nodes == nullptr.
cudaError_t launch_encode(const void *G, const void *coeff, const int32_t *nodes, int count, int m, int64_t d,
                          void *E, int is_int, cudaStream_t stream, int64_t *launches);

// One level of decode: for parent i < parents: M_parent[i] = sum_j W[i*n+j] * M_child[n*i+j] (+ E_parent[i]);
// parents with active[i] == 0 are skipped.  W and active are device arrays.
cudaError_t launch_decode(const void *M_child, const void *E_parent, const void *W, const int32_t *active,
                          int parents, int n, int64_t d, void *M_parent, int shift, int is_int,
                          cudaStream_t stream, int64_t *launches);

// Partial gradients of linear regression, two passes over X: residuals r = X_p w - y_p into `resid`
// ([items][rows]), then G[item][:] = X_p^T r.  part[item] is the partition of slot `item`.  Any d.
// loss: 0 squared, 1 logistic (r = sigmoid(X_p w) - y_p).
// `order` (device [items], may be null): launch order of the items, e.g. grouped by partition.
cudaError_t launch_partial_gradients_two_pass(const float *X, const float *y, const float *w, const int32_t *part,
                                              const int32_t *order, int items, int rows, int64_t d, float *resid,
                                              float *G, int loss, int sm_count, cudaStream_t stream, int64_t *launches);

// One CTA that waits `limit_ns` on an mbarrier nobody arrives on -- through the same bounded wait as the
// production kernels -- and then sets *status, as they do when a wait runs out.  No copy is in flight.
cudaError_t launch_wait_selftest(int *status, unsigned long long limit_ns, cudaStream_t stream, int64_t *launches);

// The same in one pass over X (row blocks staged in shared memory, cluster reduction), no scratch;
// needs d % 4 == 0, d <= 8192 and 16-byte aligned X, w, G (partial_fused_eligible).
bool partial_fused_eligible(const float *X, const float *w, const float *G, int64_t d, int items);
// slots_per_item = 1: G[item] for every (node, slot) item; slots_per_item = m with `coeff`: item = node,
// G[node] = sum_j coeff[node*m+j] * (gradient of slot j), the node's coded gradient.
// loss: 0 squared (r = X w - y), 1 logistic (r = sigmoid(X w) - y).  `order` ([items], may be null;
// used when slots_per_item = 1): the order in which the items are launched.
cudaError_t launch_partial_gradients_fused(const float *X, const float *y, const float *w, const int32_t *part,
                                           const int32_t *order, const float *coeff, int items, int slots_per_item,
                                           int rows, int64_t d,
                                           float *G, int loss, int *status, const DeviceInfo &dev,
                                           const Tuning &tune, cudaStream_t stream, int64_t *launches);

// Partial gradients of K <= 32 models at once on the tensor cores (cr_tc.cu): G [K][items][d]; R_out
// optional [items][rows][K]; workspace of multi_model_workspace_bytes bytes.
size_t multi_model_workspace_bytes(int items, int rows, int64_t d);
bool multi_model_eligible(const float *X, const float *G, const void *workspace, int64_t d, int rows, int K, int items);
cudaError_t launch_partial_gradients_multi(const float *X, const float *y, const float *W, int K, const int32_t *part,
                                           const int32_t *order, int items, int P, int rows, int64_t d, float *G,
                                           float *R_out, int loss,
                                           void *workspace, int *status, const Tuning &tune, EncodeTiledFn encode,
                                           cudaStream_t stream, int64_t *launches);

}  // namespace cr
