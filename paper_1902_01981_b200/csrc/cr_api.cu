// C ABI of libcodedreduce.so: argument checking, host expansion of straggler patterns into
// schedules, staging of those small tables to the device, kernel dispatch.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <map>
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

// Takes the next staging slot, waiting for the work that last used it.  A call whose tables do not fit
// the slots grows the whole ring at once (every slot to twice the size asked for), so that this happens
// once and not again for each of the eight slots as the loop reaches them: freeing and allocating pinned
// memory waits for the device and can take milliseconds.
cr_status_t stage_acquire(cr_plan *p, size_t bytes, StageSlot **out) {
    if (p->ring[p->next].bytes < bytes) {
        const size_t cap = std::max<size_t>(align16(bytes) * 2, 4096);
        for (StageSlot &s : p->ring) {
            if (s.pending) {
                CR_CUDA(cudaEventSynchronize(s.ev));
                s.pending = false;
            }
            if (s.host) cudaFreeHost(s.host);
            if (s.dev) cudaFree(s.dev);
            s.host = nullptr; s.dev = nullptr; s.bytes = 0;
            CR_CUDA(cudaMallocHost(reinterpret_cast<void **>(&s.host), cap));
            CR_CUDA(cudaMalloc(reinterpret_cast<void **>(&s.dev), cap));
            s.bytes = cap;
        }
    }
    StageSlot &s = p->ring[p->next];
    p->next = (p->next + 1) % kRing;
    if (s.pending) {
        CR_CUDA(cudaEventSynchronize(s.ev));
        s.pending = false;
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
    std::vector<cr::Step> steps;       // all patterns, concatenated: every consumed node in post-order
    std::vector<int32_t> pat_off;      // [batch+1]
    std::vector<int32_t> unodes;       // union of used nodes, ascending
    std::vector<uint32_t> wtab;        // distinct decode-weight bit patterns of the batch (empty: none / too many)
    std::vector<std::vector<cr::UsedNode>> per_pattern;
    // Messages shared by the patterns of a batch (batch kernel).  The message of a node of layer L-1, whose
    // children are leaves, depends only on the decode row of its own group, so the batch needs one copy per
    // distinct row.  `ops` lists those nodes, `vtab` their weight records and variant lists (layouts: BatchArgs), and the
    // reduced schedules name a message row where the full ones have the node and its leaves.
    std::vector<int4> ops;
    std::vector<uint32_t> vtab;
    std::vector<cr::Step> red_steps;
    std::vector<int32_t> red_off;
    int n_rows = 0;                    // rows of an E buffer: the union, then extra message rows
};

// share: 0 = build the shared-message tables when they save replay work, 1 = never, 2 = whenever possible
cr_status_t expand_all(const cr::HostPlan &hp, const uint32_t *masks, int batch, int share, Expanded &ex) {
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
    std::vector<int32_t> widx;   // per step: index of its weight in the table
    for (int b = 0; b < batch; ++b) {
        for (const cr::UsedNode &u : ex.per_pattern[b]) {
            const uint32_t wb = weight_bits(hp, u.weight);
            int32_t index = pos[u.node];
            size_t wi = 0;
            if (table_ok) {
                while (wi < ex.wtab.size() && ex.wtab[wi] != wb) ++wi;
                if (wi == ex.wtab.size()) {
                    if (ex.wtab.size() >= 1024) table_ok = false;
                    else ex.wtab.push_back(wb);
                }
                if (table_ok) index |= (int32_t)(wi << 12);
            }
            widx.push_back((int32_t)wi);
            ex.steps.push_back(cr::Step{u.node, u.layer | (u.first ? 0x100 : 0), wb, index});
        }
        ex.pat_off.push_back((int32_t)ex.steps.size());
    }
    if (!table_ok) {
        ex.wtab.clear();
        for (cr::Step &st : ex.steps) st.index = pos[st.node];   // plain positions
    }
    ex.n_rows = (int)ex.unodes.size();
    if (!table_ok || batch < 2 || hp.L < 2 || share == 1) return CR_OK;

    // ---- shared messages of the bottom layer (parents of the leaves) ----
    const int lb = hp.L - 1;
    struct Build {
        int own_row, child_row0, cnt;
        std::vector<std::vector<uint32_t>> weights;   // per variant: decode weights of the children in the union
        std::vector<int> dst;                          // per variant: row of its message
    };
    std::vector<Build> builds;
    std::vector<int32_t> op_of(hp.N, -1);
    int extra = 0;
    ex.red_off.assign(1, 0);
    std::vector<uint32_t> key;
    for (int b = 0; b < batch; ++b) {
        const std::vector<cr::UsedNode> &pp = ex.per_pattern[b];
        const size_t base = (size_t)ex.pat_off[b];
        size_t leaf_from = 0;   // the leaves since the last inner node are the children of the next bottom node
        for (size_t k = 0; k < pp.size(); ++k) {
            const cr::UsedNode &u = pp[k];
            if (u.layer == hp.L) continue;
            if (u.layer != lb) {
                ex.red_steps.push_back(ex.steps[base + k]);
                leaf_from = k + 1;
                continue;
            }
            int32_t &op = op_of[u.node];
            if (op < 0) {
                op = (int32_t)builds.size();
                Build nb;
                nb.own_row = pos[u.node];
                const int first_child = hp.layer_offset[hp.L] + (u.node - hp.layer_offset[lb]) * hp.n;
                nb.child_row0 = -1; nb.cnt = 0;
                for (int j = 0; j < hp.n; ++j)
                    if (pos[first_child + j] >= 0) { if (nb.child_row0 < 0) nb.child_row0 = pos[first_child + j]; ++nb.cnt; }
                builds.push_back(nb);
            }
            Build &bd = builds[op];
            key.assign((size_t)bd.cnt, 0u);
            for (size_t c = leaf_from; c < k; ++c) key[(size_t)(pos[pp[c].node] - bd.child_row0)] = ex.steps[base + c].wbits;
            size_t v = 0;
            while (v < bd.weights.size() && bd.weights[v] != key) ++v;
            if (v == bd.weights.size()) {
                // the node's own row and its children's rows are dead once its variants are formed: they hold
                // the first variants, the others go behind the union
                const int reuse = 1 + bd.cnt;
                bd.dst.push_back((int)v == 0 ? bd.own_row : ((int)v < reuse ? bd.child_row0 + (int)v - 1 : ex.n_rows + extra++));
                bd.weights.push_back(key);
            }
            cr::Step st = ex.steps[base + k];
            st.layer |= 0x200;   // a complete message: no children of its own in the reduced schedule
            st.index = bd.dst[v] | (widx[base + k] << 12);
            ex.red_steps.push_back(st);
            leaf_from = k + 1;
        }
        ex.red_off.push_back((int32_t)ex.red_steps.size());
    }
    // Replay work in rows of shared memory read or written per tile: every schedule entry one row; with shared
    // messages the reduced entries plus, per bottom node, its own row, its children and its variants.  Sharing
    // is taken when it halves that work.  Measured (64 patterns, ms per launch without / with): (12,2,1) at
    // d = 2^20 4.85 / 1.08, (4,3,1) 1.39 / 0.63 (ratios 0.32 and 0.37); (3,4,1) at d = 2^22, ratio 0.57, where the
    // loads already set the pace: 5.12 / 5.15.
    size_t work_new = ex.red_steps.size();
    for (const Build &bd : builds) work_new += 1 + (size_t)bd.cnt + bd.weights.size();
    const bool pays = share == 2 || work_new * 2 <= ex.steps.size();
    if (!pays || ex.n_rows + extra > 4096) {
        ex.red_steps.clear(); ex.red_off.clear();
        return CR_OK;
    }
    ex.n_rows += extra;
    // weight records first (padded to four words, equal ones stored once: with the whole tree in the union
    // the nodes of a level all use the same few decode rows), then the variant lists of the nodes
    std::map<std::vector<uint32_t>, uint32_t> record_at;
    std::vector<std::vector<uint32_t>> rec_of(builds.size());
    for (size_t o = 0; o < builds.size(); ++o) {
        for (std::vector<uint32_t> w : builds[o].weights) {
            w.resize((w.size() + 3) & ~(size_t)3, 0u);
            auto it = record_at.find(w);
            if (it == record_at.end()) {
                it = record_at.emplace(w, (uint32_t)ex.vtab.size()).first;
                ex.vtab.insert(ex.vtab.end(), w.begin(), w.end());
            }
            rec_of[o].push_back(it->second);
        }
    }
    for (size_t o = 0; o < builds.size(); ++o) {
        const Build &bd = builds[o];
        ex.ops.push_back(make_int4(bd.own_row, bd.child_row0, bd.cnt | ((int)bd.weights.size() << 8), (int)ex.vtab.size()));
        for (size_t v = 0; v < bd.weights.size(); ++v) {
            ex.vtab.push_back((uint32_t)bd.dst[v]);
            ex.vtab.push_back(rec_of[o][v]);
        }
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
        // staging ring for the expanded schedules: sized here for single patterns and small batches, so
        // that the device calls of an ordinary loop never allocate (a larger batch grows its slot once)
        {
            // room for a batch of 64 patterns over the whole tree (two schedules of 16-byte entries per pattern
            // and node), within 64 KB .. 1 MB per slot
            const size_t cap = std::min<size_t>(1u << 20, std::max<size_t>(64 * 1024, align16((size_t)p->hp.N * 64 * 40)));
            for (StageSlot &s : p->ring) {
                CR_CUDA_P(cudaMallocHost(reinterpret_cast<void **>(&s.host), cap));
                CR_CUDA_P(cudaMalloc(reinterpret_cast<void **>(&s.dev), cap));
                CR_CUDA_P(cudaEventCreateWithFlags(&s.ev, cudaEventDisableTiming));
                s.bytes = cap;
            }
        }
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

cr_status_t cr_plan_clear_status(cr_plan_t *plan) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    CR_CUDA(cudaDeviceSynchronize());
    CR_CUDA(cudaMemset(plan->d_status, 0, sizeof(int)));
    return CR_OK;
}

cr_status_t cr_plan_set_wait_limit(cr_plan_t *plan, uint64_t limit_ns) {
    if (!plan || limit_ns < 1000 || limit_ns > 60000000000ull) return CR_ERR_INVALID_ARG;
    plan->tune.wait_limit_ns = limit_ns;
    return CR_OK;
}

cr_status_t cr_selftest_wait(cr_plan_t *plan, uint64_t limit_ns, void *stream) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    // a bounded range: the self-test is there to show the give-up path, not to hold the GPU
    if (limit_ns < 1000 || limit_ns > 100000000ull) return CR_ERR_INVALID_ARG;
    cudaError_t e = cr::launch_wait_selftest(plan->d_status, limit_ns, reinterpret_cast<cudaStream_t>(stream), &plan->launches);
    if (e != cudaSuccess) { note_cuda(e, "cr_selftest_wait"); return CR_ERR_CUDA; }
    return CR_OK;
}

cr_status_t cr_plan_batch_stats(const cr_plan_t *plan, const uint32_t *masks_host, int32_t batch, int32_t share_messages,
                                int64_t *stats) {
    if (!plan || !masks_host || !stats || batch < 1 || batch > (1 << 16) || share_messages < 0 || share_messages > 2)
        return CR_ERR_INVALID_ARG;
    Expanded ex;
    cr_status_t st = expand_all(plan->hp, masks_host, batch, share_messages, ex);
    if (st != CR_OK) return st;
    int64_t variants = 0;
    for (const int4 &op : ex.ops) variants += op.z >> 8;
    stats[0] = (int64_t)ex.steps.size();
    stats[1] = (int64_t)ex.unodes.size();
    stats[2] = (int64_t)ex.ops.size();
    stats[3] = variants;
    stats[4] = (int64_t)ex.red_steps.size();
    stats[5] = ex.n_rows;
    return CR_OK;
}

cr_status_t cr_plan_tune_batch(cr_plan_t *plan, int32_t share_messages, int32_t e_buffers) {
    if (!plan || share_messages < 0 || share_messages > 2 || e_buffers < 0 || e_buffers > 2) return CR_ERR_INVALID_ARG;
    plan->tune.share = share_messages;
    plan->tune.e_buffers = e_buffers;
    return CR_OK;
}

cr_status_t cr_aggregate_bytes(const cr_plan_t *plan, const uint32_t *masks_host, int32_t batch, int64_t *bytes,
                               int32_t *used_nodes) {
    if (!plan || !masks_host || batch < 1 || !bytes) return CR_ERR_INVALID_ARG;
    Expanded ex;
    cr_status_t st = expand_all(plan->hp, masks_host, batch, 1, ex);
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
        // one pass over X, no scratch; items grouped by partition unless the caller asked for (node, slot) order:
        // the clusters that hold the same partition then run side by side and share its rows through L2 (since
        // the kernel reads shared memory once per block it is close to the DRAM bound and gains from that:
        // 2048 x 4096 partitions 0.557 -> 0.533 ms)
        e = cr::launch_partial_gradients_fused(X, y, w, plan->d_part, plan->tune.pg_order == 1 ? nullptr : plan->d_order, nullptr, items, 1, rows, plan->hp.d, G_slots, loss,
                                               plan->d_status, plan->dev, plan->tune,
                                               reinterpret_cast<cudaStream_t>(stream), &plan->launches);
    } else {
        if (!workspace || workspace_bytes < cr_partial_gradients_workspace_bytes(plan, rows)) return CR_ERR_OOM;
        // items grouped by partition unless the caller asked for (node, slot) order: the items that hold the
        // same partition then read its rows from HBM once and share them through L2
        e = cr::launch_partial_gradients_two_pass(X, y, w, plan->d_part, plan->tune.pg_order == 1 ? nullptr : plan->d_order, items, rows, plan->hp.d,
                                                  reinterpret_cast<float *>(workspace), G_slots, loss, plan->dev.sm_count,
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
    // the slot is guarded by an event on the error path too: its copy may still be queued
    st = stage_release(slot, s);
    if (e != cudaSuccess) { note_cuda(e, "cr_decode"); return CR_ERR_CUDA; }
    return st;
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

}  // extern "C"

namespace {

// A batch of straggler patterns, expanded: everything cr_aggregate derives from the masks before it can
// launch, with the tables the kernels read laid out as one block of bytes (`blob`) ready to be copied to
// the device.  Built per call by cr_aggregate, once by cr_schedule_create.
struct Prepared {
    int batch = 0;
    uint32_t flags = 0, variant = 0;
    Expanded ex;
    int same_shape = 1;       // fused forms: all full schedules share length and layer sequence
    int red_same_shape = 1;   // the same for the reduced schedules (shared messages)
    int subtrees = 0;         // single pattern: consumed children of the master
    int m_eff = 0;            // slot rows per node as the kernels see them (1 when the input is coded gradients)
    std::vector<unsigned char> blob;
    // fused forms: offsets of the tables inside the blob
    size_t off_steps = 0, off_pat = 0, off_unodes = 0, off_wtab = 0, off_units = 0, off_ops = 0, off_vtab = 0,
           off_red_steps = 0, off_red_pat = 0;
    int n_boxes = 0, npb = 1;
    cr::BatchShape shape;     // batches: launch shape of the batch kernel (ok = false: it cannot serve this batch)
    // unfused form: per pattern and level the weight rows and the active flags
    std::vector<size_t> w_off, a_off;
    size_t per_pattern = 0, nodes_bytes = 0;
};

bool same_layers(const std::vector<cr::Step> &steps, const std::vector<int32_t> &off, int batch) {
    const int32_t len = off[1] - off[0];
    for (int b = 1; b < batch; ++b) {
        if (off[b + 1] - off[b] != len) return false;
        for (int32_t k = 0; k < len; ++k)
            if ((steps[off[b] + k].layer & 0xff) != (steps[off[0] + k].layer & 0xff)) return false;
    }
    return true;
}

size_t append(std::vector<unsigned char> &blob, const void *src, size_t bytes) {
    const size_t off = blob.size();
    blob.resize(off + align16(bytes));
    if (bytes) std::memcpy(blob.data() + off, src, bytes);
    return off;
}

cr_status_t prepare(const cr_plan *plan, const uint32_t *masks_host, int batch, uint32_t flags, Prepared &pr) {
    const cr::HostPlan &hp = plan->hp;
    if (!masks_host || batch < 1 || batch > (1 << 16)) return CR_ERR_INVALID_ARG;
    const uint32_t variant = flags & CR_AGG_VARIANT_MASK;
    if (variant > CR_AGG_UNCODED_SUM || (flags & ~(uint32_t)(CR_AGG_VARIANT_MASK | CR_AGG_ALL_NODES | CR_AGG_FROM_CODED)) != 0)
        return CR_ERR_INVALID_ARG;
    if ((flags & CR_AGG_ALL_NODES) && variant != CR_AGG_UNFUSED) return CR_ERR_INVALID_ARG;
    if ((flags & CR_AGG_FROM_CODED) && variant == CR_AGG_UNFUSED) return CR_ERR_INVALID_ARG;
    pr.batch = batch; pr.flags = flags; pr.variant = variant;
    pr.m_eff = (flags & CR_AGG_FROM_CODED) ? 1 : hp.m;
    const int share = variant == CR_AGG_FUSED ? plan->tune.share : 1;
    cr_status_t st = expand_all(hp, masks_host, batch, share, pr.ex);
    if (st != CR_OK) return st;
    const Expanded &ex = pr.ex;

    if (variant == CR_AGG_UNFUSED) {
        // union node list, then per pattern and level the weight rows and the active flags
        const int n = hp.n, L = hp.L;
        const bool all_nodes = (flags & CR_AGG_ALL_NODES) != 0;
        pr.w_off.resize(L); pr.a_off.resize(L);
        for (int l = 0; l < L; ++l) {
            const size_t parents = (size_t)hp.nodes_in_layer(l);
            pr.w_off[l] = pr.per_pattern; pr.per_pattern += align16(parents * n * 4);
            pr.a_off[l] = pr.per_pattern; pr.per_pattern += align16(parents * 4);
        }
        pr.nodes_bytes = align16(ex.unodes.size() * 4);
        pr.blob.assign(pr.nodes_bytes + pr.per_pattern * (size_t)batch, 0);
        std::memcpy(pr.blob.data(), ex.unodes.data(), ex.unodes.size() * 4);
        std::vector<char> used(hp.N, 0);
        for (int b = 0; b < batch; ++b) {
            const uint32_t *masks = masks_host + (size_t)b * hp.groups;
            std::fill(used.begin(), used.end(), 0);
            for (const cr::UsedNode &u : ex.per_pattern[b]) used[u.node] = 1;
            unsigned char *base = pr.blob.data() + pr.nodes_bytes + pr.per_pattern * (size_t)b;
            for (int l = 0; l < L; ++l) {
                uint32_t *W = reinterpret_cast<uint32_t *>(base + pr.w_off[l]);
                int32_t *act = reinterpret_cast<int32_t *>(base + pr.a_off[l]);
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
        return CR_OK;
    }

    pr.same_shape = batch == 1 || same_layers(ex.steps, ex.pat_off, batch);
    pr.red_same_shape = !ex.ops.empty() && same_layers(ex.red_steps, ex.red_off, batch);
    for (const cr::Step &s : ex.steps) pr.subtrees += (s.layer & 0xff) == 1;
    // Batches over nodes with few slot rows (m <= 8, or coded gradients): one TMA box takes the rows of up
    // to 16 / m union nodes with consecutive ids, which lie next to each other in the slot buffer.
    std::vector<int2> boxes;
    pr.npb = (batch > 1 && variant == CR_AGG_FUSED && pr.m_eff <= 8) ? 16 / pr.m_eff : 1;
    if (pr.npb > 1 && ex.unodes.size() < (1u << 20)) {
        for (size_t u = 0; u < ex.unodes.size();) {
            size_t g = 1;
            while (g < (size_t)pr.npb && u + g < ex.unodes.size() && ex.unodes[u + g] == ex.unodes[u] + (int32_t)g) ++g;
            boxes.push_back(make_int2(ex.unodes[u] * pr.m_eff, (int)u | (int)(g << 20)));
            u += g;
        }
    }
    pr.n_boxes = (int)boxes.size();
    // Batches: the launch shape of the batch kernel is fixed here, first with the shared messages and, if
    // their tables do not fit, without them; then the unit records of the boxes are laid out for it.
    std::vector<uint32_t> units;
    if (batch > 1 && variant == CR_AGG_FUSED) {
        cr::AggArgs q;
        q.G = nullptr; q.coeff = nullptr; q.steps = nullptr; q.host_steps = nullptr; q.pat_off = nullptr; q.unodes = nullptr;
        q.wtab = nullptr; q.out = nullptr; q.status = nullptr; q.shift = 0; q.rows_total = 0;
        q.n_wtab = (int)ex.wtab.size(); q.n_union = (int)ex.unodes.size(); q.batch = batch;
        q.m = pr.m_eff; q.L = hp.L; q.d = hp.d; q.is_int = hp.dtype == CR_I32;
        q.npb = pr.npb; q.n_boxes = pr.n_boxes;
        if (!pr.ex.ops.empty()) {
            q.total_steps = (int)ex.red_steps.size(); q.same_shape = pr.red_same_shape;
            q.n_rows = ex.n_rows; q.n_ops = (int)ex.ops.size(); q.vtab_words = (int)ex.vtab.size();
            q.L = hp.L - 1;   // the reduced schedules end at the layer above the leaves
            pr.shape = cr::batch_shape(q, plan->dev, plan->tune);
            q.L = hp.L;
            if (!pr.shape.ok) {   // the shared form does not fit: the plain one
                pr.ex.ops.clear(); pr.ex.vtab.clear(); pr.ex.red_steps.clear(); pr.ex.red_off.clear();
                pr.ex.n_rows = (int)ex.unodes.size();
            }
        }
        if (pr.ex.ops.empty()) {
            q.total_steps = (int)ex.steps.size(); q.same_shape = pr.same_shape;
            q.n_rows = 0; q.n_ops = 0; q.vtab_words = 0;
            pr.shape = cr::batch_shape(q, plan->dev, plan->tune);
        }
        if (pr.shape.ok) {
            const int W = cr::unit_words();
            const bool coded = (flags & CR_AGG_FROM_CODED) != 0;
            auto coef_at = [&](int64_t row) {   // coefficient of slot row `row` as the kernels see it
                return coded ? weight_bits(hp, 1.0) : weight_bits(hp, hp.slots[(size_t)row].coeff * (double)hp.int_scale);
            };
            auto put = [&](int row0, int erow, int every, int valid) {
                const size_t at = units.size();
                units.resize(at + W, 0u);
                for (int j = 0; j < valid; ++j) units[at + j] = coef_at((int64_t)row0 + j);
                units[at + 16] = (uint32_t)row0; units[at + 17] = (uint32_t)erow;
                units[at + 18] = (uint32_t)every; units[at + 19] = (uint32_t)valid;
            };
            if (pr.shape.multi) {
                for (const int2 &bx : boxes) put(bx.x, bx.y & 0xfffff, pr.m_eff, (bx.y >> 20) * pr.m_eff);
            } else {
                for (size_t u = 0; u < ex.unodes.size(); ++u)
                    for (int c = 0; c < pr.shape.cpn; ++c)
                        put(ex.unodes[u] * pr.m_eff + c * pr.shape.R, (int)u, c + 1 == pr.shape.cpn ? pr.shape.R : 0, pr.shape.R);
            }
        }
    }
    pr.off_steps = append(pr.blob, ex.steps.data(), ex.steps.size() * sizeof(cr::Step));
    pr.off_pat = append(pr.blob, ex.pat_off.data(), ex.pat_off.size() * 4);
    pr.off_unodes = append(pr.blob, ex.unodes.data(), ex.unodes.size() * 4);
    pr.off_wtab = append(pr.blob, ex.wtab.data(), ex.wtab.size() * 4);
    pr.off_units = append(pr.blob, units.data(), units.size() * 4);
    pr.off_ops = append(pr.blob, ex.ops.data(), ex.ops.size() * sizeof(int4));
    pr.off_vtab = append(pr.blob, ex.vtab.data(), ex.vtab.size() * 4);
    pr.off_red_steps = append(pr.blob, ex.red_steps.data(), ex.red_steps.size() * sizeof(cr::Step));
    pr.off_red_pat = append(pr.blob, ex.red_off.data(), ex.red_off.size() * 4);
    return CR_OK;
}

cr_status_t run_unfused(cr_plan *plan, const Prepared &pr, const unsigned char *tables, const void *G_slots, void *g_out,
                        void *workspace, cudaStream_t s) {
    const cr::HostPlan &hp = plan->hp;
    const int n = hp.n, L = hp.L;
    const bool is_int = hp.dtype == CR_I32;
    const bool all_nodes = (pr.flags & CR_AGG_ALL_NODES) != 0;
    char *ws = reinterpret_cast<char *>(workspace);
    char *E = ws;
    std::vector<char *> M(L + 1, nullptr);  // M[l] for l = 1..L-1
    size_t off = (size_t)hp.N * hp.d * 4;
    for (int l = 1; l < L; ++l) { M[l] = ws + off; off += (size_t)hp.nodes_in_layer(l) * hp.d * 4; }
    M[L] = E + (size_t)hp.layer_offset[L] * hp.d * 4;  // a leaf's message is its coded gradient

    cudaError_t e;
    if (all_nodes) e = cr::launch_encode(G_slots, plan->d_coeff, nullptr, hp.N, hp.m, hp.d, E, is_int, s, &plan->launches);
    else e = cr::launch_encode(G_slots, plan->d_coeff, reinterpret_cast<const int32_t *>(tables),
                               (int)pr.ex.unodes.size(), hp.m, hp.d, E, is_int, s, &plan->launches);
    if (e != cudaSuccess) { note_cuda(e, "encode"); return CR_ERR_CUDA; }
    for (int b = 0; b < pr.batch; ++b) {
        const unsigned char *base = tables + pr.nodes_bytes + pr.per_pattern * (size_t)b;
        for (int l = L - 1; l >= 0; --l) {
            const void *child = M[l + 1];
            const void *own = l == 0 ? nullptr : E + (size_t)hp.layer_offset[l] * hp.d * 4;
            void *dst = l == 0 ? reinterpret_cast<char *>(g_out) + (size_t)b * hp.d * 4 : M[l];
            e = cr::launch_decode(child, own, base + pr.w_off[l], reinterpret_cast<const int32_t *>(base + pr.a_off[l]),
                                  hp.nodes_in_layer(l), n, hp.d, dst, (is_int && l == 0) ? hp.int_shift : 0, is_int, s,
                                  &plan->launches);
            if (e != cudaSuccess) { note_cuda(e, "decode"); return CR_ERR_CUDA; }
        }
    }
    return CR_OK;
}

// Launches the work of a prepared batch.  `tables` is the device copy of pr.blob, or null when it has
// not been made yet: forms that can pass a single short schedule in the kernel parameters then run
// without it, and the others return kNeedTables so that the caller stages the blob and calls again.
constexpr int kNeedTables = -1;

int run_prepared(cr_plan *plan, const Prepared &pr, const unsigned char *tables, const void *G_slots, void *g_out,
                 void *workspace, size_t workspace_bytes, cudaStream_t s) {
    const cr::HostPlan &hp = plan->hp;
    const int batch = pr.batch;
    const uint32_t variant = pr.variant;
    const Expanded &ex = pr.ex;

    if (variant == CR_AGG_UNFUSED) {
        if (!workspace || workspace_bytes < cr_aggregate_workspace_bytes(plan, batch, pr.flags)) return CR_ERR_OOM;
        if (!tables) return kNeedTables;
        plan->last_kernel = "cr_encode_kernel + cr_decode_kernel per level";
        return run_unfused(plan, pr, tables, G_slots, g_out, workspace, s);
    }

    cr::AggArgs a;
    a.G = G_slots; a.coeff = plan->d_coeff;
    a.steps = nullptr; a.pat_off = nullptr; a.unodes = nullptr; a.wtab = nullptr;
    a.host_steps = ex.steps.data();
    a.n_wtab = (int)ex.wtab.size();
    a.n_union = (int)ex.unodes.size(); a.batch = batch; a.total_steps = (int)ex.steps.size();
    a.m = hp.m; a.L = hp.L; a.d = hp.d; a.rows_total = (int64_t)hp.N * hp.m; a.out = g_out;
    if (pr.flags & CR_AGG_FROM_CODED) {
        // the input is E [N][d]: one row per node, already combined with the slot coefficients
        a.m = 1; a.coeff = plan->d_ones; a.rows_total = hp.N;
    }
    a.shift = hp.dtype == CR_I32 ? hp.int_shift : 0; a.status = plan->d_status; a.is_int = hp.dtype == CR_I32;
    a.same_shape = pr.same_shape;

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
    const bool untuned = !plan->tune.ncw && !plan->tune.stages && !plan->tune.ctas_per_sm && !plan->tune.rows;
    const bool prefer_plain = batch == 1 &&
                              (a.m == 1 || ((a.m <= 4 || a.m % 4 == 0) && hp.d >= (1ll << 19) && (a.m <= 8 || hp.d <= (1ll << 23)))) &&
                              hp.d % 4 == 0 && untuned;

    // Short vectors under a large tree: one block per column range would walk all the consumed nodes
    // one after the other (d = 5004 under the (12,2) tree: 132 nodes, 53 us).  The sub-trees below the
    // master are independent until its decode, so each gets its own blocks and a second small kernel
    // adds their weighted messages.
    // Measured (us per call, split / TMA kernel): (12,2,1) d = 5004: 24 / 53, d = 120000: 48 / 113;
    // with few sub-trees it does not pay: (4,3,1) d = 6500: 18.5 / 20.6, (3,4,1) d = 4096: 31 / 18.5.
    if (variant == CR_AGG_FUSED && untuned && batch == 1 && plan->d_split && pr.subtrees >= kSplitMinSubtrees &&
        a.total_steps >= 24 && a.total_steps <= cr::inline_schedule_limit() && pr.subtrees <= cr::split_limit()) {
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

    if (!tables) return kNeedTables;
    a.steps = reinterpret_cast<const cr::Step *>(tables + pr.off_steps);
    a.pat_off = reinterpret_cast<const int32_t *>(tables + pr.off_pat);
    a.unodes = reinterpret_cast<const int32_t *>(tables + pr.off_unodes);
    a.wtab = reinterpret_cast<const uint32_t *>(tables + pr.off_wtab);
    a.n_boxes = pr.n_boxes;
    a.npb = pr.npb;
    a.units = reinterpret_cast<const uint32_t *>(tables + pr.off_units);
    a.host_steps = nullptr;

    cudaError_t e = cudaSuccess;
    if (variant == CR_AGG_UNCODED_SUM) {
        e = cr::launch_uncoded_sum(a, s, &plan->launches);
        plan->last_kernel = "cr_uncoded_sum_kernel";
    } else {
        bool done = false;
        if (variant == CR_AGG_FUSED && !prefer_plain) {
            if (batch == 1) {
                e = cr::launch_fused_tma(a, plan->dev, plan->tune, plan->encode, s, &plan->launches, &done);
                if (done) plan->last_kernel = "cr_fused_tma_kernel";
            } else {
                if (!ex.ops.empty()) {
                    // the patterns share the messages of the bottom layer: reduced schedules
                    cr::AggArgs r = a;
                    r.steps = reinterpret_cast<const cr::Step *>(tables + pr.off_red_steps);
                    r.pat_off = reinterpret_cast<const int32_t *>(tables + pr.off_red_pat);
                    r.total_steps = (int)ex.red_steps.size();
                    r.same_shape = pr.red_same_shape;
                    r.L = hp.L - 1;   // depth of the reduced schedules: the kernel instance for that depth serves them
                    r.n_rows = ex.n_rows; r.n_ops = (int)ex.ops.size();
                    r.ops = reinterpret_cast<const int4 *>(tables + pr.off_ops);
                    r.vtab = reinterpret_cast<const uint32_t *>(tables + pr.off_vtab);
                    r.vtab_words = (int)ex.vtab.size();
                    e = cr::launch_fused_batch_tma(r, pr.shape, plan->tune, plan->encode, s, &plan->launches, &done);
                    if (done) plan->last_kernel = "cr_fused_batch_tma_kernel (shared messages)";
                } else {
                    e = cr::launch_fused_batch_tma(a, pr.shape, plan->tune, plan->encode, s, &plan->launches, &done);
                    if (done) plan->last_kernel = "cr_fused_batch_tma_kernel";
                }
            }
        }
        if (e == cudaSuccess && !done) {
            plan->last_kernel = "cr_fused_ldg_kernel";
            e = cr::launch_fused_ldg(a, s, &plan->launches);
        }
    }
    if (e != cudaSuccess) { note_cuda(e, "cr_aggregate"); return CR_ERR_CUDA; }
    return CR_OK;
}

}  // namespace

// A straggler pattern batch expanded once and kept on the device (cr_schedule_create).
struct cr_schedule {
    cr_plan *plan = nullptr;
    Prepared prep;
    unsigned char *dev = nullptr;
};

extern "C" {

cr_status_t cr_aggregate(cr_plan_t *plan, const void *G_slots, const uint32_t *masks_host, int32_t batch, void *g_out,
                         uint32_t flags, void *workspace, size_t workspace_bytes, void *stream) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    if (!G_slots || !g_out) return CR_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    Prepared pr;
    st = prepare(plan, masks_host, batch, flags, pr);
    if (st != CR_OK) return st;
    int rc = run_prepared(plan, pr, nullptr, G_slots, g_out, workspace, workspace_bytes, s);
    if (rc != kNeedTables) return (cr_status_t)rc;
    StageSlot *slot = nullptr;
    st = stage_acquire(plan, pr.blob.size(), &slot);
    if (st != CR_OK) return st;
    std::memcpy(slot->host, pr.blob.data(), pr.blob.size());
    st = stage_commit(slot, pr.blob.size(), s);
    if (st != CR_OK) return st;
    rc = run_prepared(plan, pr, slot->dev, G_slots, g_out, workspace, workspace_bytes, s);
    // the slot is guarded by an event on every path, so that it is not reused under a copy still queued
    st = stage_release(slot, s);
    return rc != CR_OK ? (cr_status_t)rc : st;
}

cr_status_t cr_schedule_create(cr_plan_t *plan, const uint32_t *masks_host, int32_t batch, uint32_t flags,
                               cr_schedule_t **out) {
    cr_status_t st = check_device_plan(plan);
    if (st != CR_OK) return st;
    if (!out) return CR_ERR_INVALID_ARG;
    cr_schedule *sc = new (std::nothrow) cr_schedule();
    if (!sc) return CR_ERR_OOM;
    sc->plan = plan;
    st = prepare(plan, masks_host, batch, flags, sc->prep);
    if (st != CR_OK) { delete sc; return st; }
    const size_t bytes = std::max<size_t>(sc->prep.blob.size(), 16);
    cudaError_t e = cudaMalloc(reinterpret_cast<void **>(&sc->dev), bytes);
    if (e == cudaSuccess && !sc->prep.blob.empty())
        e = cudaMemcpy(sc->dev, sc->prep.blob.data(), sc->prep.blob.size(), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        note_cuda(e, "cr_schedule_create");
        if (sc->dev) cudaFree(sc->dev);
        delete sc;
        return CR_ERR_CUDA;
    }
    *out = sc;
    return CR_OK;
}

cr_status_t cr_schedule_destroy(cr_schedule_t *sched) {
    if (!sched) return CR_OK;
    if (sched->plan && sched->plan->device >= 0) cudaSetDevice(sched->plan->device);
    if (sched->dev) cudaFree(sched->dev);
    delete sched;
    return CR_OK;
}

cr_status_t cr_schedule_bytes(const cr_schedule_t *sched, int64_t *bytes, int32_t *used_nodes) {
    if (!sched || !bytes) return CR_ERR_INVALID_ARG;
    const cr::HostPlan &hp = sched->plan->hp;
    *bytes = 4ll * hp.d * ((int64_t)sched->prep.m_eff * (int64_t)sched->prep.ex.unodes.size() + sched->prep.batch);
    if (used_nodes) *used_nodes = (int32_t)sched->prep.ex.unodes.size();
    return CR_OK;
}

cr_status_t cr_aggregate_scheduled(cr_plan_t *plan, const void *G_slots, const cr_schedule_t *sched, void *g_out,
                                   void *workspace, size_t workspace_bytes, void *stream) {
    if (!plan || !sched || sched->plan != plan || !G_slots || !g_out) return CR_ERR_INVALID_ARG;
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current != plan->device) CR_CUDA(cudaSetDevice(plan->device));
    return (cr_status_t)run_prepared(plan, sched->prep, sched->dev, G_slots, g_out, workspace, workspace_bytes,
                                     reinterpret_cast<cudaStream_t>(stream));
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
                                                 plan->dev.sm_count, reinterpret_cast<cudaStream_t>(stream), &plan->launches);
    if (e != cudaSuccess) { note_cuda(e, "cr_partial_gradients_static"); return CR_ERR_CUDA; }
    return CR_OK;
}

}  // extern "C"
