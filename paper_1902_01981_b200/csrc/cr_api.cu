// C ABI of libcodedreduce.so: argument checking, host expansion of straggler patterns into
// schedules, staging of those small tables to the device, kernel dispatch.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "codedreduce.h"
#include "cr_kernels.hpp"
#include "cr_plan.hpp"

namespace {

thread_local char g_last_error[256] = "";

void note_cuda(cudaError_t e, const char *where) {
    std::snprintf(g_last_error, sizeof(g_last_error), "%s: %s", where, cudaGetErrorString(e));
}

#define CR_CUDA(call)                              \
    do {                                           \
        cudaError_t e__ = (call);                  \
        if (e__ != cudaSuccess) {                  \
            note_cuda(e__, #call);                 \
            return CR_ERR_CUDA;                    \
        }                                          \
    } while (0)

constexpr int kRing = 8;

struct StageSlot {
    unsigned char *host = nullptr;
    unsigned char *dev = nullptr;
    size_t bytes = 0;
    cudaEvent_t ev = nullptr;
    bool pending = false;
};

size_t align16(size_t x) { return (x + 15) & ~(size_t)15; }

}  // namespace

// The split form of short aggregations (cr_aggregate): vectors of at most this length, under trees whose
// master has at least this many children.
constexpr long long kSplitMaxD = 1ll << 17;
constexpr int kSplitMinSubtrees = 6;

struct cr_plan {
    cr::HostPlan hp;
    int device = -1;
    void *d_coeff = nullptr;     // [N*m] float or int32
    void *d_ones = nullptr;      // [N] the value 1 in the plan's element type (aggregation of coded gradients)
    int32_t *d_part = nullptr;   // [N*m]
    int32_t *d_order = nullptr;  // [N*m] slot items sorted by partition: launch order of the gradient kernels
    void *d_split = nullptr;     // [n][d] scratch of the split form of short aggregations (plans that can take it)
    const char *last_kernel = "";  // kernel that served the latest cr_aggregate call
    int *d_status = nullptr;
    cr::DeviceInfo dev;
    cr::Tuning tune;
    cr::EncodeTiledFn encode = nullptr;
    StageSlot ring[kRing];
    int next = 0;
    int64_t launches = 0;
};

namespace {

// Takes the next staging slot, waiting for the work that last used it, and makes it large enough.
cr_status_t stage_acquire(cr_plan *p, size_t bytes, StageSlot **out) {
    StageSlot &s = p->ring[p->next];
    p->next = (p->next + 1) % kRing;
    if (s.pending) {
        CR_CUDA(cudaEventSynchronize(s.ev));
        s.pending = false;
    }
    if (s.bytes < bytes) {
        if (s.host) cudaFreeHost(s.host);
        if (s.dev) cudaFree(s.dev);
        s.host = nullptr; s.dev = nullptr; s.bytes = 0;
        const size_t cap = std::max<size_t>(align16(bytes) * 2, 4096);
        CR_CUDA(cudaMallocHost(reinterpret_cast<void **>(&s.host), cap));
        CR_CUDA(cudaMalloc(reinterpret_cast<void **>(&s.dev), cap));
        s.bytes = cap;
    }
    if (!s.ev) CR_CUDA(cudaEventCreateWithFlags(&s.ev, cudaEventDisableTiming));
    *out = &s;
    return CR_OK;
}

cr_status_t stage_commit(StageSlot *s, size_t bytes, cudaStream_t stream) {
    CR_CUDA(cudaMemcpyAsync(s->dev, s->host, bytes, cudaMemcpyHostToDevice, stream));
    return CR_OK;
}

cr_status_t stage_release(StageSlot *s, cudaStream_t stream) {
    CR_CUDA(cudaEventRecord(s->ev, stream));
    s->pending = true;
    return CR_OK;
}

uint32_t weight_bits(const cr::HostPlan &hp, double w) {
    if (hp.dtype == CR_I32) return (uint32_t)(int32_t)std::llround(w);
    const float f = (float)w;
    uint32_t bits;
    std::memcpy(&bits, &f, 4);
    return bits;
}

struct Expanded {
    std::vector<cr::Step> steps;       // all patterns, concatenated
    std::vector<int32_t> pat_off;      // [batch+1]
    std::vector<int32_t> unodes;       // union of used nodes, ascending
    std::vector<uint32_t> wtab;        // distinct decode-weight bit patterns of the batch (empty: none / too many)
    std::vector<std::vector<cr::UsedNode>> per_pattern;
};

cr_status_t expand_all(const cr::HostPlan &hp, const uint32_t *masks, int batch, Expanded &ex) {
    std::vector<int32_t> pos(hp.N, -1);
    ex.pat_off.assign(1, 0);
    ex.per_pattern.resize(batch);
    std::vector<char> seen(hp.N, 0);
    for (int b = 0; b < batch; ++b) {
        cr_status_t st = hp.expand(masks + (size_t)b * hp.groups, ex.per_pattern[b]);
        if (st != CR_OK) return st;
        for (const cr::UsedNode &u : ex.per_pattern[b]) seen[u.node] = 1;
    }
    for (int v = 0; v < hp.N; ++v)
        if (seen[v]) { pos[v] = (int32_t)ex.unodes.size(); ex.unodes.push_back(v); }
    // Step.index = position of the node in the union list (bits 0..11 when it fits) and, above it, the
    // index of the step's weight in the table of distinct weights: the batch kernel can then keep a
    // 4-byte entry per step and pattern in shared memory.
    bool table_ok = batch > 1 && ex.unodes.size() <= 4096;
    for (int b = 0; b < batch; ++b) {
        for (const cr::UsedNode &u : ex.per_pattern[b]) {
            const uint32_t wb = weight_bits(hp, u.weight);
            int32_t index = pos[u.node];
            if (table_ok) {
                size_t wi = 0;
                while (wi < ex.wtab.size() && ex.wtab[wi] != wb) ++wi;
                if (wi == ex.wtab.size()) {
                    if (ex.wtab.size() >= 1024) table_ok = false;
                    else ex.wtab.push_back(wb);
                }
                if (table_ok) index |= (int32_t)(wi << 12);
            }
            ex.steps.push_back(cr::Step{u.node, u.layer | (u.first ? 0x100 : 0), wb, index});
        }
        ex.pat_off.push_back((int32_t)ex.steps.size());
    }
    if (!table_ok) {
        ex.wtab.clear();
        for (cr::Step &st : ex.steps) st.index = pos[st.node];   // plain positions
    }
    return CR_OK;
}

cr_status_t check_device_plan(cr_plan *p) {
    if (!p) return CR_ERR_INVALID_ARG;
    if (p->device < 0) {
        std::snprintf(g_last_error, sizeof(g_last_error), "device work asked of a host-only plan");
        return CR_ERR_CUDA;
    }
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current != p->device) CR_CUDA(cudaSetDevice(p->device));
    return CR_OK;
}

}  // namespace

extern "C" {

const char *cr_status_string(int status) {
    switch (status) {
        case CR_OK: return "CR_OK";
        case CR_ERR_INVALID_ARG: return "CR_ERR_INVALID_ARG";
        case CR_ERR_BAD_PARTITION_COUNT: return "CR_ERR_BAD_PARTITION_COUNT";
        case CR_ERR_CODE_UNAVAILABLE: return "CR_ERR_CODE_UNAVAILABLE";
        case CR_ERR_ILL_CONDITIONED: return "CR_ERR_ILL_CONDITIONED";
        case CR_ERR_UNDECODABLE_MASK: return "CR_ERR_UNDECODABLE_MASK";
        case CR_ERR_DTYPE: return "CR_ERR_DTYPE";
        case CR_ERR_CUDA: return "CR_ERR_CUDA";
        case CR_ERR_OOM: return "CR_ERR_OOM";
        case CR_ERR_TIMEOUT: return "CR_ERR_TIMEOUT";
        default: return "CR_ERR_UNKNOWN";
    }
}

const char *cr_last_cuda_error(void) { return g_last_error; }

cr_status_t cr_plan_destroy(cr_plan_t *plan) {
    if (!plan) return CR_OK;
    if (plan->device >= 0) {
        cudaSetDevice(plan->device);
        for (StageSlot &s : plan->ring) {
            if (s.pending) cudaEventSynchronize(s.ev);
            if (s.ev) cudaEventDestroy(s.ev);
            if (s.host) cudaFreeHost(s.host);
            if (s.dev) cudaFree(s.dev);
        }
        if (plan->d_coeff) cudaFree(plan->d_coeff);
        if (plan->d_ones) cudaFree(plan->d_ones);
        if (plan->d_part) cudaFree(plan->d_part);
        if (plan->d_order) cudaFree(plan->d_order);
        if (plan->d_split) cudaFree(plan->d_split);
        if (plan->d_status) cudaFree(plan->d_status);
    }
    delete plan;
    return CR_OK;
}

cr_status_t cr_plan_create(const cr_plan_desc_t *desc, cr_plan_t **out) {
    if (!desc || !out) return CR_ERR_INVALID_ARG;
    if (desc->device < -1) return CR_ERR_INVALID_ARG;
    cr_plan *p = new (std::nothrow) cr_plan();
    if (!p) return CR_ERR_OOM;
    cr_status_t st = cr::build_host_plan(*desc, p->hp);
    if (st != CR_OK) { delete p; return st; }
    p->device = desc->device;
    if (p->device >= 0) {
        auto fail = [&](cr_status_t code) { cr_plan_destroy(p); return code; };
#define CR_CUDA_P(call)                                                                          \
    do {                                                                                         \
        cudaError_t e__ = (call);                                                                \
        if (e__ != cudaSuccess) { note_cuda(e__, #call); return fail(CR_ERR_CUDA); }             \
    } while (0)
        CR_CUDA_P(cudaSetDevice(p->device));
        CR_CUDA_P(cudaDeviceGetAttribute(&p->dev.sm_count, cudaDevAttrMultiProcessorCount, p->device));
        CR_CUDA_P(cudaDeviceGetAttribute(&p->dev.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, p->device));
        CR_CUDA_P(cudaDeviceGetAttribute(&p->dev.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, p->device));
        int major = 0;
        CR_CUDA_P(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, p->device));
        if (major != 10) {
            std::snprintf(g_last_error, sizeof(g_last_error), "device is not sm_100 (compute capability %d.x)", major);
            return fail(CR_ERR_CUDA);
        }
        const size_t slots = (size_t)p->hp.N * p->hp.m;
        std::vector<int32_t> part(slots);
        std::vector<uint32_t> coeff(slots);
        for (size_t i = 0; i < slots; ++i) {
            part[i] = p->hp.slots[i].part;
            coeff[i] = weight_bits(p->hp, p->hp.slots[i].coeff * (double)p->hp.int_scale);
        }
        CR_CUDA_P(cudaMalloc(&p->d_coeff, slots * 4));
        CR_CUDA_P(cudaMalloc(reinterpret_cast<void **>(&p->d_part), slots * 4));
        CR_CUDA_P(cudaMalloc(reinterpret_cast<void **>(&p->d_status), sizeof(int)));
        CR_CUDA_P(cudaMemcpy(p->d_coeff, coeff.data(), slots * 4, cudaMemcpyHostToDevice));
        {
            std::vector<uint32_t> ones((size_t)p->hp.N, weight_bits(p->hp, 1.0));
            CR_CUDA_P(cudaMalloc(&p->d_ones, ones.size() * 4));
            CR_CUDA_P(cudaMemcpy(p->d_ones, ones.data(), ones.size() * 4, cudaMemcpyHostToDevice));
        }
        CR_CUDA_P(cudaMemcpy(p->d_part, part.data(), slots * 4, cudaMemcpyHostToDevice));
        {
            // items that hold the same partition compute the same gradient from the same rows of X:
            // launched side by side, they fetch those rows from HBM once and share them through L2
            std::vector<int32_t> order(slots);
            for (size_t i = 0; i < slots; ++i) order[i] = (int32_t)i;
            std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return part[a] < part[b]; });
            CR_CUDA_P(cudaMalloc(reinterpret_cast<void **>(&p->d_order), slots * 4));
            CR_CUDA_P(cudaMemcpy(p->d_order, order.data(), slots * 4, cudaMemcpyHostToDevice));
        }
        CR_CUDA_P(cudaMemset(p->d_status, 0, sizeof(int)));
        // scratch of the split form of short aggregations under wide trees (see cr_aggregate): reserved
        // here, so that no device call ever allocates
        if (p->hp.L >= 2 && p->hp.d <= kSplitMaxD && p->hp.n >= kSplitMinSubtrees && p->hp.n <= cr::split_limit())
            CR_CUDA_P(cudaMalloc(&p->d_split, (size_t)p->hp.n * (size_t)p->hp.d * 4));
        // cuTensorMapEncodeTiled through the runtime, so that the library needs no link to libcuda
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            p->encode = reinterpret_cast<cr::EncodeTiledFn>(fn);
        else
            (void)cudaGetLastError();
#undef CR_CUDA_P
    }
    *out = p;
    return CR_OK;
}

int32_t cr_plan_num_nodes(const cr_plan_t *plan) { return plan ? plan->hp.N : -1; }
int32_t cr_plan_num_groups(const cr_plan_t *plan) { return plan ? plan->hp.groups : -1; }
int32_t cr_plan_load(const cr_plan_t *plan) { return plan ? plan->hp.m : -1; }
int64_t cr_plan_int_scale(const cr_plan_t *plan) { return plan ? plan->hp.int_scale : -1; }
int64_t cr_plan_launch_count(const cr_plan_t *plan) { return plan ? plan->launches : -1; }
const char *cr_plan_last_kernel(const cr_plan_t *plan) { return plan ? plan->last_kernel : ""; }

cr_status_t cr_plan_tune(cr_plan_t *plan, int32_t consumer_warps, int32_t stages, int32_t ctas_per_sm, int32_t rows_per_box) {
    if (!plan || consumer_warps < 0 || stages < 0 || ctas_per_sm < 0 || rows_per_box < 0) return CR_ERR_INVALID_ARG;
    if (consumer_warps != 0 && consumer_warps != 2 && consumer_warps != 4 && consumer_warps != 8) return CR_ERR_INVALID_ARG;
    if (stages == 1 || stages > 16 || ctas_per_sm > 8) return CR_ERR_INVALID_ARG;
    if (rows_per_box != 0 && (plan->hp.m % rows_per_box != 0 || rows_per_box > 16)) return CR_ERR_INVALID_ARG;
    plan->tune.ncw = consumer_warps; plan->tune.stages = stages; plan->tune.ctas_per_sm = ctas_per_sm;
    plan->tune.rows = rows_per_box;
    return CR_OK;
}

cr_status_t cr_plan_tune_gradients(cr_plan_t *plan, int32_t block_kb, int32_t stages, int32_t cluster) {
    if (!plan || block_kb < 0 || block_kb > 128 || stages < 0 || stages == 1 || stages > 8) return CR_ERR_INVALID_ARG;
    if (cluster != 0 && cluster != 1 && cluster != 2 && cluster != 4 && cluster != 8 && cluster != 16) return CR_ERR_INVALID_ARG;
    plan->tune.pg_block_kb = block_kb; plan->tune.pg_stages = stages; plan->tune.pg_cluster = cluster;
    return CR_OK;
}

cr_status_t cr_plan_tune_items(cr_plan_t *plan, int32_t item_order, int32_t multi_stages) {
    if (!plan || item_order < 0 || item_order > 2 || multi_stages < 0 || multi_stages == 1 || multi_stages > 4) return CR_ERR_INVALID_ARG;
    plan->tune.pg_order = item_order; plan->tune.tc_stages = multi_stages;
    return CR_OK;
}

cr_status_t cr_plan_get_B(const cr_plan_t *plan, int32_t level, double *B, double *kappa, uint64_t *sub_seed) {
    if (!plan || !B || level < 0 || level >= plan->hp.L) return CR_ERR_INVALID_ARG;
    std::copy(plan->hp.B[level].begin(), plan->hp.B[level].end(), B);
    if (kappa) *kappa = plan->hp.kappa[level];
    if (sub_seed) *sub_seed = plan->hp.sub_seed[level];
    return CR_OK;
}

cr_status_t cr_plan_get_slots(const cr_plan_t *plan, int32_t node, int32_t *part, double *coeff) {
    if (!plan || !part || !coeff || node < 0 || node >= plan->hp.N) return CR_ERR_INVALID_ARG;
    for (int j = 0; j < plan->hp.m; ++j) {
        part[j] = plan->hp.slots[(size_t)node * plan->hp.m + j].part;
        coeff[j] = plan->hp.slots[(size_t)node * plan->hp.m + j].coeff;
    }
    return CR_OK;
}

cr_status_t cr_plan_get_decode(const cr_plan_t *plan, int32_t level, uint32_t straggler_mask, double *a) {
    if (!plan || !a || level < 0 || level >= plan->hp.L || (straggler_mask >> plan->hp.n) != 0) return CR_ERR_INVALID_ARG;
    if (!plan->hp.mask_ok(straggler_mask)) return CR_ERR_UNDECODABLE_MASK;
    const double *row = plan->hp.decode_row(level, straggler_mask);
    std::copy(row, row + plan->hp.n, a);
    return CR_OK;
}

cr_status_t cr_plan_expand(const cr_plan_t *plan, const uint32_t *masks, int32_t capacity, int32_t *nodes,
                           int32_t *layers, double *weights, int32_t *count) {
    if (!plan || !masks || !nodes || !layers || !weights || !count || capacity < 0) return CR_ERR_INVALID_ARG;
    std::vector<cr::UsedNode> used;
    cr_status_t st = plan->hp.expand(masks, used);
    if (st != CR_OK) return st;
    if ((int)used.size() > capacity) return CR_ERR_OOM;
    for (size_t k = 0; k < used.size(); ++k) { nodes[k] = used[k].node; layers[k] = used[k].layer; weights[k] = used[k].weight; }
    *count = (int32_t)used.size();
    return CR_OK;
}

cr_status_t cr_latency_masks(const cr_plan_t *plan, const double *compute_time, double t_c, uint32_t *masks_out,
                             double *t_total) {
    if (!plan || !compute_time || !masks_out || !(t_c >= 0.0)) return CR_ERR_INVALID_ARG;
    for (int v = 0; v < plan->hp.N; ++v)
        if (!(compute_time[v] >= 0.0)) return CR_ERR_INVALID_ARG;
    const double t = plan->hp.latency_masks(compute_time, t_c, masks_out);
    if (t_total) *t_total = t;
    return CR_OK;
}

cr_status_t cr_plan_device_status(cr_plan_t *plan) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    int word = 0;
    CR_CUDA(cudaDeviceSynchronize());
    CR_CUDA(cudaMemcpy(&word, plan->d_status, sizeof(int), cudaMemcpyDeviceToHost));
    return word == 0 ? CR_OK : CR_ERR_TIMEOUT;
}

cr_status_t cr_aggregate_bytes(const cr_plan_t *plan, const uint32_t *masks_host, int32_t batch, int64_t *bytes,
                               int32_t *used_nodes) {
    if (!plan || !masks_host || batch < 1 || !bytes) return CR_ERR_INVALID_ARG;
    Expanded ex;
    cr_status_t st = expand_all(plan->hp, masks_host, batch, ex);
    if (st != CR_OK) return st;
    *bytes = 4ll * plan->hp.d * ((int64_t)plan->hp.m * (int64_t)ex.unodes.size() + batch);
    if (used_nodes) *used_nodes = (int32_t)ex.unodes.size();
    return CR_OK;
}

size_t cr_partial_gradients_workspace_bytes(const cr_plan_t *plan, int32_t rows) {
    if (!plan || rows < 1) return 0;
    return (size_t)plan->hp.N * plan->hp.m * (size_t)rows * sizeof(float);
}

cr_status_t cr_partial_gradients_loss(cr_plan_t *plan, int32_t loss, const float *X, const float *y, int32_t rows,
                                      const float *w, float *G_slots, void *workspace, size_t workspace_bytes,
                                      void *stream) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    if (!X || !y || !w || !G_slots || rows < 1 || (loss != CR_LOSS_SQUARED && loss != CR_LOSS_LOGISTIC)) return CR_ERR_INVALID_ARG;
    if (plan->hp.dtype != CR_F32) return CR_ERR_DTYPE;
    const int items = plan->hp.N * plan->hp.m;
    cudaError_t e;
    if (cr::partial_fused_eligible(X, w, G_slots, plan->hp.d, items)) {
        // one pass over X, no scratch
        e = cr::launch_partial_gradients_fused(X, y, w, plan->d_part, plan->tune.pg_order == 2 ? plan->d_order : nullptr, nullptr, items, 1, rows, plan->hp.d, G_slots, loss,
                                               plan->d_status, plan->dev, plan->tune,
                                               reinterpret_cast<cudaStream_t>(stream), &plan->launches);
    } else {
        if (!workspace || workspace_bytes < cr_partial_gradients_workspace_bytes(plan, rows)) return CR_ERR_OOM;
        // items grouped by partition unless the caller asked for (node, slot) order: the items that hold the
        // same partition then read its rows from HBM once and share them through L2
        e = cr::launch_partial_gradients_two_pass(X, y, w, plan->d_part, plan->tune.pg_order == 1 ? nullptr : plan->d_order, items, rows, plan->hp.d,
                                                  reinterpret_cast<float *>(workspace), G_slots, loss,
                                                  reinterpret_cast<cudaStream_t>(stream), &plan->launches);
    }
    if (e != cudaSuccess) { note_cuda(e, "cr_partial_gradients"); return CR_ERR_CUDA; }
    return CR_OK;
}

cr_status_t cr_partial_gradients(cr_plan_t *plan, const float *X, const float *y, int32_t rows, const float *w,
                                 float *G_slots, void *workspace, size_t workspace_bytes, void *stream) {
    return cr_partial_gradients_loss(plan, CR_LOSS_SQUARED, X, y, rows, w, G_slots, workspace, workspace_bytes, stream);
}

cr_status_t cr_coded_gradients(cr_plan_t *plan, int32_t loss, const float *X, const float *y, int32_t rows,
                               const float *w, float *E, void *stream) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    if (!X || !y || !w || !E || rows < 1 || (loss != CR_LOSS_SQUARED && loss != CR_LOSS_LOGISTIC)) return CR_ERR_INVALID_ARG;
    if (plan->hp.dtype != CR_F32) return CR_ERR_DTYPE;
    if (!cr::partial_fused_eligible(X, w, E, plan->hp.d, plan->hp.N)) {
        std::snprintf(g_last_error, sizeof(g_last_error),
                      "cr_coded_gradients needs d %% 4 == 0, d <= 8192 and 16-byte aligned X, w, E");
        return CR_ERR_INVALID_ARG;
    }
    cudaError_t e = cr::launch_partial_gradients_fused(X, y, w, plan->d_part, nullptr, reinterpret_cast<const float *>(plan->d_coeff),
                                                       plan->hp.N, plan->hp.m, rows, plan->hp.d, E, loss, plan->d_status,
                                                       plan->dev, plan->tune, reinterpret_cast<cudaStream_t>(stream),
                                                       &plan->launches);
    if (e != cudaSuccess) { note_cuda(e, "cr_coded_gradients"); return CR_ERR_CUDA; }
    return CR_OK;
}

size_t cr_partial_gradients_multi_workspace_bytes(const cr_plan_t *plan, int32_t rows) {
    if (!plan || rows < 1) return 0;
    return cr::multi_model_workspace_bytes(plan->hp.N * plan->hp.m, rows, plan->hp.d);
}

cr_status_t cr_partial_gradients_multi(cr_plan_t *plan, int32_t loss, const float *X, const float *y, int32_t rows,
                                       const float *W, int32_t K, float *G_multi, float *R_out, void *workspace,
                                       size_t workspace_bytes, void *stream) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    if (!X || !y || !W || !G_multi || rows < 1 || (loss != CR_LOSS_SQUARED && loss != CR_LOSS_LOGISTIC)) return CR_ERR_INVALID_ARG;
    if (plan->hp.dtype != CR_F32) return CR_ERR_DTYPE;
    if (!plan->encode) return CR_ERR_CUDA;
    const int items = plan->hp.N * plan->hp.m;
    if (!workspace || workspace_bytes < cr::multi_model_workspace_bytes(items, rows, plan->hp.d)) return CR_ERR_OOM;
    if (!cr::multi_model_eligible(X, G_multi, workspace, plan->hp.d, rows, K, items)) {
        std::snprintf(g_last_error, sizeof(g_last_error),
                      "cr_partial_gradients_multi needs d %% 4 == 0, d >= 32, 1 <= K <= 32, N*m <= 65535 and 16-byte "
                      "aligned X, G_multi, workspace");
        return CR_ERR_INVALID_ARG;
    }
    cudaError_t e = cr::launch_partial_gradients_multi(X, y, W, K, plan->d_part, plan->tune.pg_order == 1 ? nullptr : plan->d_order, items, plan->hp.P, rows, plan->hp.d,
                                                       G_multi, R_out, loss, workspace, plan->d_status, plan->tune, plan->encode,
                                                       reinterpret_cast<cudaStream_t>(stream), &plan->launches);
    if (e != cudaSuccess) { note_cuda(e, "cr_partial_gradients_multi"); return CR_ERR_CUDA; }
    return CR_OK;
}

cr_status_t cr_encode(cr_plan_t *plan, const void *G_slots, void *E, void *stream) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    if (!G_slots || !E) return CR_ERR_INVALID_ARG;
    cudaError_t e = cr::launch_encode(G_slots, plan->d_coeff, nullptr, plan->hp.N, plan->hp.m, plan->hp.d, E,
                                      plan->hp.dtype == CR_I32, reinterpret_cast<cudaStream_t>(stream), &plan->launches);
    if (e != cudaSuccess) { note_cuda(e, "cr_encode"); return CR_ERR_CUDA; }
    return CR_OK;
}

cr_status_t cr_decode(cr_plan_t *plan, int32_t parent_layer, const void *M_child, const void *E_parent,
                      const uint32_t *masks_host, void *M_parent, void *stream) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    const cr::HostPlan &hp = plan->hp;
    if (!M_child || !masks_host || !M_parent || parent_layer < 0 || parent_layer >= hp.L) return CR_ERR_INVALID_ARG;
    if ((parent_layer == 0) != (E_parent == nullptr)) return CR_ERR_INVALID_ARG;
    const int parents = hp.nodes_in_layer(parent_layer);
    for (int i = 0; i < parents; ++i) {
        if ((masks_host[i] >> hp.n) != 0) return CR_ERR_INVALID_ARG;
        if (!hp.mask_ok(masks_host[i])) return CR_ERR_UNDECODABLE_MASK;
    }
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)parents * hp.n * 4;
    StageSlot *slot = nullptr;
    st = stage_acquire(plan, bytes, &slot);
    if (st != CR_OK) return st;
    uint32_t *W = reinterpret_cast<uint32_t *>(slot->host);
    for (int i = 0; i < parents; ++i) {
        const double *a = hp.decode_row(parent_layer, masks_host[i]);
        for (int j = 0; j < hp.n; ++j) W[(size_t)i * hp.n + j] = weight_bits(hp, a[j]);
    }
    st = stage_commit(slot, bytes, s);
    if (st != CR_OK) return st;
    const int shift = (hp.dtype == CR_I32 && parent_layer == 0) ? hp.int_shift : 0;
    cudaError_t e = cr::launch_decode(M_child, E_parent, slot->dev, nullptr, parents, hp.n, hp.d, M_parent, shift,
                                      hp.dtype == CR_I32, s, &plan->launches);
    if (e != cudaSuccess) { note_cuda(e, "cr_decode"); return CR_ERR_CUDA; }
    return stage_release(slot, s);
}

size_t cr_aggregate_workspace_bytes(const cr_plan_t *plan, int32_t batch, uint32_t flags) {
    (void)batch;
    if (!plan) return 0;
    if ((flags & CR_AGG_VARIANT_MASK) != CR_AGG_UNFUSED) return 0;
    // E for all nodes plus one message buffer per non-leaf worker layer (leaf messages are E itself)
    const cr::HostPlan &hp = plan->hp;
    const int64_t nonleaf = hp.layer_offset[hp.L];
    return (size_t)(hp.N + nonleaf) * (size_t)hp.d * 4;
}

static cr_status_t aggregate_unfused(cr_plan *plan, const void *G_slots, const uint32_t *masks_host, int batch,
                                     void *g_out, bool all_nodes, void *workspace, const Expanded &ex,
                                     cudaStream_t s) {
    const cr::HostPlan &hp = plan->hp;
    const int n = hp.n, L = hp.L;
    const bool is_int = hp.dtype == CR_I32;
    // staging: union node list, then per pattern and level the weight rows and the active flags
    size_t per_pattern = 0;
    std::vector<size_t> w_off(L), a_off(L);
    for (int l = 0; l < L; ++l) {
        const size_t parents = (size_t)hp.nodes_in_layer(l);
        w_off[l] = per_pattern; per_pattern += align16(parents * n * 4);
        a_off[l] = per_pattern; per_pattern += align16(parents * 4);
    }
    const size_t nodes_bytes = align16(ex.unodes.size() * 4);
    const size_t total = nodes_bytes + per_pattern * (size_t)batch;
    StageSlot *slot = nullptr;
    cr_status_t st = stage_acquire(plan, total, &slot);
    if (st != CR_OK) return st;
    std::memset(slot->host, 0, total);
    std::memcpy(slot->host, ex.unodes.data(), ex.unodes.size() * 4);
    for (int b = 0; b < batch; ++b) {
        const uint32_t *masks = masks_host + (size_t)b * hp.groups;
        std::vector<char> used(hp.N, 0);
        for (const cr::UsedNode &u : ex.per_pattern[b]) used[u.node] = 1;
        unsigned char *base = slot->host + nodes_bytes + per_pattern * (size_t)b;
        for (int l = 0; l < L; ++l) {
            uint32_t *W = reinterpret_cast<uint32_t *>(base + w_off[l]);
            int32_t *act = reinterpret_cast<int32_t *>(base + a_off[l]);
            const int parents = hp.nodes_in_layer(l);
            for (int i = 0; i < parents; ++i) {
                const int group = l == 0 ? 0 : hp.layer_offset[l] + i + 1;
                const bool active = all_nodes || l == 0 || used[hp.layer_offset[l] + i];
                act[i] = active ? 1 : 0;
                if (!active) continue;
                if ((masks[group] >> n) != 0) return CR_ERR_INVALID_ARG;
                if (!hp.mask_ok(masks[group])) return CR_ERR_UNDECODABLE_MASK;
                const double *a = hp.decode_row(l, masks[group]);
                for (int j = 0; j < n; ++j) W[(size_t)i * n + j] = weight_bits(hp, a[j]);
            }
        }
    }
    st = stage_commit(slot, total, s);
    if (st != CR_OK) return st;

    char *ws = reinterpret_cast<char *>(workspace);
    char *E = ws;
    std::vector<char *> M(L + 1, nullptr);  // M[l] for l = 1..L-1
    size_t off = (size_t)hp.N * hp.d * 4;
    for (int l = 1; l < L; ++l) { M[l] = ws + off; off += (size_t)hp.nodes_in_layer(l) * hp.d * 4; }
    M[L] = E + (size_t)hp.layer_offset[L] * hp.d * 4;  // a leaf's message is its coded gradient

    cudaError_t e;
    if (all_nodes) e = cr::launch_encode(G_slots, plan->d_coeff, nullptr, hp.N, hp.m, hp.d, E, is_int, s, &plan->launches);
    else e = cr::launch_encode(G_slots, plan->d_coeff, reinterpret_cast<const int32_t *>(slot->dev),
                               (int)ex.unodes.size(), hp.m, hp.d, E, is_int, s, &plan->launches);
    if (e != cudaSuccess) { note_cuda(e, "encode"); return CR_ERR_CUDA; }
    for (int b = 0; b < batch; ++b) {
        const unsigned char *base = slot->dev + nodes_bytes + per_pattern * (size_t)b;
        for (int l = L - 1; l >= 0; --l) {
            const void *child = M[l + 1];
            const void *own = l == 0 ? nullptr : E + (size_t)hp.layer_offset[l] * hp.d * 4;
            void *dst = l == 0 ? reinterpret_cast<char *>(g_out) + (size_t)b * hp.d * 4 : M[l];
            e = cr::launch_decode(child, own, base + w_off[l], reinterpret_cast<const int32_t *>(base + a_off[l]),
                                  hp.nodes_in_layer(l), n, hp.d, dst, (is_int && l == 0) ? hp.int_shift : 0, is_int, s,
                                  &plan->launches);
            if (e != cudaSuccess) { note_cuda(e, "decode"); return CR_ERR_CUDA; }
        }
    }
    return stage_release(slot, s);
}

cr_status_t cr_aggregate(cr_plan_t *plan, const void *G_slots, const uint32_t *masks_host, int32_t batch, void *g_out,
                         uint32_t flags, void *workspace, size_t workspace_bytes, void *stream) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    const cr::HostPlan &hp = plan->hp;
    if (!G_slots || !masks_host || !g_out || batch < 1 || batch > (1 << 16)) return CR_ERR_INVALID_ARG;
    const uint32_t variant = flags & CR_AGG_VARIANT_MASK;
    if (variant > CR_AGG_UNCODED_SUM || (flags & ~(uint32_t)(CR_AGG_VARIANT_MASK | CR_AGG_ALL_NODES | CR_AGG_FROM_CODED)) != 0)
        return CR_ERR_INVALID_ARG;
    if ((flags & CR_AGG_ALL_NODES) && variant != CR_AGG_UNFUSED) return CR_ERR_INVALID_ARG;
    if ((flags & CR_AGG_FROM_CODED) && variant == CR_AGG_UNFUSED) return CR_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

    Expanded ex;
    st = expand_all(hp, masks_host, batch, ex);
    if (st != CR_OK) return st;

    if (variant == CR_AGG_UNFUSED) {
        if (!workspace || workspace_bytes < cr_aggregate_workspace_bytes(plan, batch, flags)) return CR_ERR_OOM;
        plan->last_kernel = "cr_encode_kernel + cr_decode_kernel per level";
        return aggregate_unfused(plan, G_slots, masks_host, batch, g_out, (flags & CR_AGG_ALL_NODES) != 0, workspace, ex, s);
    }

    cr::AggArgs a;
    a.G = G_slots; a.coeff = plan->d_coeff;
    a.steps = nullptr; a.pat_off = nullptr; a.unodes = nullptr; a.wtab = nullptr;
    a.host_steps = ex.steps.data();
    a.n_wtab = (int)ex.wtab.size();
    a.n_union = (int)ex.unodes.size(); a.batch = batch; a.total_steps = (int)ex.steps.size();
    a.m = hp.m; a.L = hp.L; a.d = hp.d; a.rows_total = (int64_t)hp.N * hp.m; a.out = g_out;
    if (flags & CR_AGG_FROM_CODED) {
        // the input is E [N][d]: one row per node, already combined with the slot coefficients
        a.m = 1; a.coeff = plan->d_ones; a.rows_total = hp.N;
    }
    a.shift = hp.dtype == CR_I32 ? hp.int_shift : 0; a.status = plan->d_status; a.is_int = hp.dtype == CR_I32;
    a.same_shape = 1;
    for (int b = 1; b < batch && a.same_shape; ++b) {
        const auto &p0 = ex.per_pattern[0], &pb = ex.per_pattern[b];
        if (pb.size() != p0.size()) { a.same_shape = 0; break; }
        for (size_t k = 0; k < p0.size(); ++k)
            if (pb[k].layer != p0[k].layer) { a.same_shape = 0; break; }
    }

    // Few slot rows per node make small TMA boxes (m = 4: 4 KB; a coded gradient, one row per node:
    // 1 KB), too small for the copy engine to keep HBM busy (measured at d = 2^22 on the (12,2) tree:
    // 6.0-6.6 TB/s with m = 4, 1.7 TB/s from coded gradients).  The plain-load kernel, which requests
    // the next group of rows before it combines the current one, reaches 7.3 and 7.0 TB/s there, and
    // is still 2 % ahead at m = 8 ((4,3) tree: 7.32 against 7.16 TB/s).  Unless the caller fixed a TMA
    // launch shape, single patterns of these shapes take that kernel.  Taller nodes whose rows come in fours
    // (m = 12, 16, ..) do too up to d = 2^23, where the prefetching form is still ahead (m = 16, (4,2,3) tree:
    // 6.8 against 6.2 TB/s at d = 2^22, 7.0 against 6.6 at 2^23, 6.8 against 6.9 at 2^24).  So do two or three rows per node
    // (flat gradient coding, L = 1; n = 12, s = 1 at d = 2^22: 4.9 against 3.0 TB/s).
    // Short vectors stay with the TMA kernel unless they are coded gradients: its narrow tiles and
    // deep rings fill more SMs (m = 4, d = 5004: 70 against 109 us; from coded gradients 51 against 37 us).
    const bool prefer_plain = batch == 1 &&
                              (a.m == 1 || ((a.m <= 4 || a.m % 4 == 0) && hp.d >= (1ll << 19) && (a.m <= 8 || hp.d <= (1ll << 23)))) &&
                              hp.d % 4 == 0 && !plan->tune.ncw && !plan->tune.stages && !plan->tune.ctas_per_sm &&
                              !plan->tune.rows;

    // Short vectors under a large tree: one block per column range would walk all the consumed nodes
    // one after the other (d = 5004 under the (12,2) tree: 132 nodes, 53 us).  The sub-trees below the
    // master are independent until its decode, so each gets its own blocks and a second small kernel
    // adds their weighted messages.
    // Measured (us per call, split / TMA kernel): (12,2,1) d = 5004: 24 / 53, d = 120000: 48 / 113;
    // with few sub-trees it does not pay: (4,3,1) d = 6500: 18.5 / 20.6, (3,4,1) d = 4096: 31 / 18.5.
    const bool untuned = !plan->tune.ncw && !plan->tune.stages && !plan->tune.ctas_per_sm && !plan->tune.rows;
    int subtrees = 0;
    for (const cr::Step &st : ex.steps) subtrees += (st.layer & 0xff) == 1;
    if (variant == CR_AGG_FUSED && untuned && batch == 1 && plan->d_split && subtrees >= kSplitMinSubtrees &&
        a.total_steps >= 24 && a.total_steps <= cr::inline_schedule_limit() && subtrees <= cr::split_limit()) {
        a.split_scratch = plan->d_split;
        cudaError_t e0 = cr::launch_fused_ldg(a, s, &plan->launches);
        if (e0 != cudaSuccess) { note_cuda(e0, "cr_aggregate"); return CR_ERR_CUDA; }
        plan->last_kernel = "cr_fused_ldg_kernel (one row of blocks per sub-tree) + cr_sum_rows_kernel";
        return CR_OK;
    }

    // A single short pattern needs no staging: its schedule travels in the kernel parameters.
    if (variant == CR_AGG_FUSED && !prefer_plain && batch == 1 && a.total_steps <= cr::inline_schedule_limit()) {
        bool done = false;
        cudaError_t e0 = cr::launch_fused_tma(a, plan->dev, plan->tune, plan->encode, s, &plan->launches, &done);
        if (e0 != cudaSuccess) { note_cuda(e0, "cr_aggregate"); return CR_ERR_CUDA; }
        if (done) { plan->last_kernel = "cr_fused_tma_kernel"; return CR_OK; }
    }

    if ((variant == CR_AGG_FUSED_LDG || (variant == CR_AGG_FUSED && prefer_plain)) && batch == 1 &&
        a.total_steps <= cr::inline_schedule_limit()) {
        cudaError_t e0 = cr::launch_fused_ldg(a, s, &plan->launches);
        if (e0 != cudaSuccess) { note_cuda(e0, "cr_aggregate"); return CR_ERR_CUDA; }
        plan->last_kernel = "cr_fused_ldg_kernel";
        return CR_OK;
    }

    // staging layout: steps | pattern offsets | union nodes
    const size_t steps_bytes = align16(ex.steps.size() * sizeof(cr::Step));
    const size_t off_bytes = align16(ex.pat_off.size() * 4);
    const size_t nodes_bytes = align16(ex.unodes.size() * 4);
    const size_t wtab_bytes = align16(ex.wtab.size() * 4);
    // Batches over nodes with few slot rows (m <= 8, or coded gradients): one TMA box takes the rows of up
    // to 16 / m union nodes with consecutive ids, which lie next to each other in the slot buffer.
    std::vector<int2> boxes;
    const int npb = (batch > 1 && variant == CR_AGG_FUSED && a.m <= 8) ? 16 / a.m : 1;
    if (npb > 1 && ex.unodes.size() < (1u << 20)) {
        for (size_t u = 0; u < ex.unodes.size();) {
            size_t g = 1;
            while (g < (size_t)npb && u + g < ex.unodes.size() && ex.unodes[u + g] == ex.unodes[u] + (int32_t)g) ++g;
            boxes.push_back(make_int2(ex.unodes[u] * a.m, (int)u | (int)(g << 20)));
            u += g;
        }
    }
    const size_t boxes_bytes = align16(boxes.size() * sizeof(int2));
    const size_t total = steps_bytes + off_bytes + nodes_bytes + wtab_bytes + boxes_bytes;
    StageSlot *slot = nullptr;
    st = stage_acquire(plan, total, &slot);
    if (st != CR_OK) return st;
    std::memcpy(slot->host, ex.steps.data(), ex.steps.size() * sizeof(cr::Step));
    std::memcpy(slot->host + steps_bytes, ex.pat_off.data(), ex.pat_off.size() * 4);
    std::memcpy(slot->host + steps_bytes + off_bytes, ex.unodes.data(), ex.unodes.size() * 4);
    std::memcpy(slot->host + steps_bytes + off_bytes + nodes_bytes, ex.wtab.data(), ex.wtab.size() * 4);
    if (!boxes.empty())
        std::memcpy(slot->host + steps_bytes + off_bytes + nodes_bytes + wtab_bytes, boxes.data(), boxes.size() * sizeof(int2));
    st = stage_commit(slot, total, s);
    if (st != CR_OK) return st;

    a.steps = reinterpret_cast<const cr::Step *>(slot->dev);
    a.pat_off = reinterpret_cast<const int32_t *>(slot->dev + steps_bytes);
    a.unodes = reinterpret_cast<const int32_t *>(slot->dev + steps_bytes + off_bytes);
    a.wtab = reinterpret_cast<const uint32_t *>(slot->dev + steps_bytes + off_bytes + nodes_bytes);
    if (!boxes.empty()) {
        a.boxes = reinterpret_cast<const int2 *>(slot->dev + steps_bytes + off_bytes + nodes_bytes + wtab_bytes);
        a.n_boxes = (int)boxes.size();
        a.npb = npb;
    }
    a.host_steps = nullptr;

    cudaError_t e = cudaSuccess;
    if (variant == CR_AGG_UNCODED_SUM) {
        e = cr::launch_uncoded_sum(a, s, &plan->launches);
        plan->last_kernel = "cr_uncoded_sum_kernel";
    } else {
        bool done = false;
        if (variant == CR_AGG_FUSED && !prefer_plain) {
            if (batch == 1) e = cr::launch_fused_tma(a, plan->dev, plan->tune, plan->encode, s, &plan->launches, &done);
            else e = cr::launch_fused_batch_tma(a, plan->dev, plan->tune, plan->encode, s, &plan->launches, &done);
        }
        plan->last_kernel = done ? (batch == 1 ? "cr_fused_tma_kernel" : "cr_fused_batch_tma_kernel") : "cr_fused_ldg_kernel";
        if (e == cudaSuccess && !done) e = cr::launch_fused_ldg(a, s, &plan->launches);
    }
    if (e != cudaSuccess) { note_cuda(e, "cr_aggregate"); return CR_ERR_CUDA; }
    return stage_release(slot, s);
}

cr_status_t cr_aggregate_host(cr_plan_t *plan, const void *G_slots_host, const uint32_t *masks_host, int32_t batch,
                              void *g_out_host, uint32_t flags, void *dev_slots, void *dev_out, void *workspace,
                              size_t workspace_bytes, void *stream) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    if (!G_slots_host || !g_out_host || !dev_slots || !dev_out || batch < 1) return CR_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t out_bytes = (size_t)batch * (size_t)plan->hp.d * 4;
    // Only the slots of the nodes that some pattern of the batch consumes cross the bus: what a
    // straggler holds is never waited for.  (One copy per run of consecutive used nodes.)
    const bool from_coded = (flags & CR_AGG_FROM_CODED) != 0;
    const size_t node_bytes = (from_coded ? (size_t)1 : (size_t)plan->hp.m) * (size_t)plan->hp.d * 4;
    if (flags & CR_AGG_ALL_NODES) {
        CR_CUDA(cudaMemcpyAsync(dev_slots, G_slots_host, node_bytes * plan->hp.N, cudaMemcpyHostToDevice, s));
    } else {
        if (!masks_host) return CR_ERR_INVALID_ARG;
        std::vector<char> used((size_t)plan->hp.N, 0);
        std::vector<cr::UsedNode> one;
        for (int b = 0; b < batch; ++b) {
            one.clear();
            st = plan->hp.expand(masks_host + (size_t)b * plan->hp.groups, one);
            if (st != CR_OK) return st;
            for (const cr::UsedNode &u : one) used[u.node] = 1;
        }
        for (int v = 0; v < plan->hp.N;) {
            if (!used[v]) { ++v; continue; }
            int w = v;
            while (w < plan->hp.N && used[w]) ++w;
            CR_CUDA(cudaMemcpyAsync(static_cast<unsigned char *>(dev_slots) + node_bytes * v,
                                    static_cast<const unsigned char *>(G_slots_host) + node_bytes * v,
                                    node_bytes * (size_t)(w - v), cudaMemcpyHostToDevice, s));
            v = w;
        }
    }
    st = cr_aggregate(plan, dev_slots, masks_host, batch, dev_out, flags, workspace, workspace_bytes, stream);
    if (st != CR_OK) return st;
    CR_CUDA(cudaMemcpyAsync(g_out_host, dev_out, out_bytes, cudaMemcpyDeviceToHost, s));
    CR_CUDA(cudaStreamSynchronize(s));
    return CR_OK;
}

// ---- partial gradients without any allocation -------------------------------------------------
//
// Residual scratch of cr_partial_gradients_static: one fixed array per device that loads this
// library, held until the process exits.  4 MiB = 1,048,576 residuals (slots x rows).
#define CR_STATIC_RESIDUALS (1u << 20)
static __device__ __align__(256) float cr_static_residuals[CR_STATIC_RESIDUALS];

namespace {
std::mutex g_static_mutex;
float *g_static_ptr[64] = {nullptr};  // device address of the array, per device ordinal
}  // namespace

size_t cr_partial_gradients_static_capacity(void) { return (size_t)CR_STATIC_RESIDUALS; }

cr_status_t cr_partial_gradients_static(cr_plan_t *plan, const float *X, const float *y, int32_t rows,
                                        const float *w, float *G_slots, void *stream) {
    cr_status_t st = check_device_plan(plan);  // makes the plan's device current
    if (st != CR_OK) return st;
    if (!X || !y || !w || !G_slots || rows < 1) return CR_ERR_INVALID_ARG;
    if (plan->hp.dtype != CR_F32) return CR_ERR_DTYPE;
    if (plan->device >= 64) return CR_ERR_INVALID_ARG;
    const size_t need = (size_t)plan->hp.N * plan->hp.m * (size_t)rows;
    if (need > (size_t)CR_STATIC_RESIDUALS) {
        std::snprintf(g_last_error, sizeof(g_last_error),
                      "cr_partial_gradients_static: %zu residuals (slots x rows) exceed the fixed scratch of %u",
                      need, CR_STATIC_RESIDUALS);
        return CR_ERR_OOM;
    }
    float *scratch = nullptr;
    {
        // In host code the array's name is only a handle; the kernels need its address on this
        // device, looked up once per device while that device is current.
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[plan->device]) {
            void *addr = nullptr;
            CR_CUDA(cudaGetSymbolAddress(&addr, cr_static_residuals));
            g_static_ptr[plan->device] = reinterpret_cast<float *>(addr);
        }
        scratch = g_static_ptr[plan->device];
    }
    // items grouped by partition, as in cr_partial_gradients, unless the plan was tuned to (node, slot) order
    cudaError_t e = cr::launch_partial_gradients_two_pass(X, y, w, plan->d_part, plan->tune.pg_order == 1 ? nullptr : plan->d_order,
                                                 plan->hp.N * plan->hp.m, rows, plan->hp.d, scratch, G_slots, CR_LOSS_SQUARED,
                                                 reinterpret_cast<cudaStream_t>(stream), &plan->launches);
    if (e != cudaSuccess) { note_cuda(e, "cr_partial_gradients_static"); return CR_ERR_CUDA; }
    return CR_OK;
}

}  // extern "C"
