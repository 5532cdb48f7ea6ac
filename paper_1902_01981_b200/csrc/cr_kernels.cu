// sm_100a kernels of the coded tree aggregation (CR.Execute, Algorithm 2).
//
// The aggregation is a chain of axpy-like passes over length-d vectors, one FMA per element read:
// bound by HBM bandwidth, no dense contraction, so no tensor cores.  The fused kernels give each CTA
// a tile of columns, stream the slot rows of the consumed nodes through a TMA -> shared-memory ring
// and keep every intermediate coded vector (a node's coded gradient, every message) in registers
// or shared memory; only the root tile is written.
#include "cr_kernels.hpp"

#include <cooperative_groups.h>

#include <algorithm>
#include <cmath>
#include <map>
#include <mutex>
#include <tuple>
#include <type_traits>
#include <cstdio>

namespace cr {

// ------------------------------------------------------------------------------------------------
// PTX helpers: mbarrier, TMA, timers
// ------------------------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One probe of a barrier phase.  (A suspend-time hint on the probe, 200 ns or 1 us, changed nothing measurable
// in any kernel here and is not used.)
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Every wait in these kernels is bounded: `limit_ns` of wall time (a kernel argument; two seconds
// unless the plan was told otherwise) or 2^30 polls, whichever comes first, or as soon as another
// thread of the CTA has given up.  A correct launch never gets near the bound; it exists so that a
// broken one returns with a status instead of hanging the GPU.

// Most slot rows one TMA box may hold (the consumers keep that many coefficients in registers).
constexpr int kMaxBoxRows = 16;
// Most children of a parent (the batch kernel keeps their coded gradients in registers when it forms
// the messages that the patterns of a batch share).
constexpr int kMaxKids = 16;
// Words of a unit record of the batch kernel: 16 coefficients, then {first slot row, first E row, rows per
// node (0: the node continues in the next box), rows in use}.
constexpr int kUnitWords = 20;

// `abort_flag` points at a shared-memory word that the other side of the pipeline sets when it has
// given up (flags[0]: a consumer did, flags[1]: the producer did, flags[2]: never set).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint64_t limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (int outer = 0; outer < (1 << 22); ++outer) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > limit_ns) return false;
    }
    return false;
}

// The same wait for a whole warp (all 32 lanes call it): the answer is made uniform, so that the lanes
// take the give-up path together or not at all.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t *bar, uint32_t parity, volatile int *abort_flag, uint64_t limit_ns) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, limit_ns) ? 1 : 0) != 0;
}

// 2-D tiled TMA load global -> shared, completion counted in bytes on an mbarrier.  x (innermost
// coordinate) times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void *smem_dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

// 1-D bulk copy global -> shared (no tensor map): both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_load_1d(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void consumer_barrier(int threads) {
    asm volatile("bar.sync 1, %0;" ::"r"(threads) : "memory");
}

// ------------------------------------------------------------------------------------------------
// element-type helpers
// ------------------------------------------------------------------------------------------------

template <typename T> struct Vec4;
template <> struct Vec4<float> { typedef float4 type; };
template <> struct Vec4<int> { typedef int4 type; };

template <typename T> __device__ __forceinline__ T weight_of(uint32_t bits);
template <> __device__ __forceinline__ float weight_of<float>(uint32_t bits) { return __uint_as_float(bits); }
template <> __device__ __forceinline__ int weight_of<int>(uint32_t bits) { return (int)bits; }

template <typename T> __device__ __forceinline__ T finish(T v, int shift) { return v; }
template <> __device__ __forceinline__ int finish<int>(int v, int shift) { return v >> shift; }

// Reads one schedule entry; `layer` is returned without the first-child flag.
__device__ __forceinline__ Step load_step(const Step *p) {
    const int4 raw = __ldg(reinterpret_cast<const int4 *>(p));
    Step s;
    s.node = raw.x; s.layer = raw.y & 0xff; s.wbits = (uint32_t)raw.z; s.index = raw.w;
    return s;
}

// The tree recursion in registers.  acc[l] (l = 0..LMAX-1) holds, for the node of layer l currently
// being assembled, the decoded combination of the children messages seen so far.  Visiting a node of
// layer `layer` in post-order with coded gradient e and decode weight w at its parent:
//     message = acc[layer] + e;   acc[layer-1] += w * message;   acc[layer] = 0
// (leaves have no acc of their own: message = e).  After the last step acc[0] is the root's result.
template <typename T, int LMAX, int V>
__device__ __forceinline__ void fold(T (&acc)[LMAX][V], const T (&e)[V], int layer, T w) {
#pragma unroll
    for (int l = 1; l <= LMAX; ++l) {
        if (layer == l) {
#pragma unroll
            for (int q = 0; q < V; ++q) {
                T msg = e[q];
                if (l < LMAX) { msg += acc[l < LMAX ? l : 0][q]; acc[l < LMAX ? l : 0][q] = T(0); }
                acc[l - 1][q] += w * msg;
            }
        }
    }
}

// The same recursion for NP patterns whose schedules visit the same layers in the same order (they
// differ in which children are used and with what weights): one uniform branch on the layer, NP
// independent dependency chains inside it.  This form never clears an accumulator: the first consumed
// child of a parent ASSIGNS acc[layer-1] = w * message, later children add to it (`lf` carries the
// layer in bits 0..7 and the first-child flag in bit 8).  acc must start at zero so that leaves, whose
// own acc is never written, add nothing.  Bit 9 of `lf` marks an entry whose row already is a complete
// message (formed once for all patterns of the batch, see the batch kernel): it is taken as it is,
// without the accumulator of its layer, which may still hold another node's children.
template <typename T, int LMAX, int NP, bool WHOLE>
__device__ __forceinline__ void fold_many(T (&acc)[NP][LMAX][4], const T (&e)[NP][4], int lf, const T (&w)[NP]) {
    const int layer = lf & 0xff;
    const bool first = (lf & 0x100) != 0;
    const bool whole = WHOLE && (lf & 0x200) != 0;   // only schedules with shared messages carry such entries
#pragma unroll
    for (int l = 1; l <= LMAX; ++l) {
        if (layer == l) {
            if (first) {
#pragma unroll
                for (int p = 0; p < NP; ++p)
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        T msg = e[p][q];
                        if (l < LMAX && !whole) msg += acc[p][l < LMAX ? l : 0][q];
                        acc[p][l - 1][q] = w[p] * msg;
                    }
            } else {
#pragma unroll
                for (int p = 0; p < NP; ++p)
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        T msg = e[p][q];
                        if (l < LMAX && !whole) msg += acc[p][l < LMAX ? l : 0][q];
                        acc[p][l - 1][q] += w[p] * msg;
                    }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// K4: fused aggregation, one straggler pattern, TMA-staged
// ------------------------------------------------------------------------------------------------
//
// CTA = NCW consumer warps + 1 producer warp, persistent over column tiles of TILE = 128*NCW
// elements.  Per tile the producer streams, for every consumed node in post-order, boxes of R slot
// rows x TILE columns into a ring of `stages` buffers; consumer thread t owns 4 consecutive columns,
// forms the node's coded gradient e = sum_j c_j * row_j from shared memory and folds it into the
// register recursion above.  Shared-memory layout of a stage: [box][R][BOXW] with BOXW = min(TILE,256)
// (a TMA box is at most 256 elements wide).

// Schedules of at most kInlineSteps entries travel inside the kernel parameters (constant bank), which
// saves the host-to-device copy in front of short launches.
constexpr int kInlineSteps = 160;

struct FusedArgs {
    const void *coeff;
    const Step *steps;      // device schedule, unless n_inline > 0
    int n_inline;           // entries of steps_inline in use (0: read `steps`)
    Step steps_inline[kInlineSteps];
    int n_steps;
    int steps_smem;         // a staged schedule (n_inline == 0) is copied into shared memory at the start
    int m, R, cpn, stages;
    long long d;
    long long ntiles;
    void *out;
    int shift;
    int *status;
    unsigned long long wait_ns;  // bound of every wait, in nanoseconds
};

// Longest staged schedule that the single-pattern kernel copies into shared memory (16 KB).  Read from global
// memory instead, the node id in front of every box is a dependent L2 latency on the producer's path: a
// 182-node pattern ran at 1.9 TB/s where the plain-load kernel reaches 4.4.
constexpr int kSmemSteps = 1024;

// (Four 160-thread CTAs per SM need at most 96 registers per thread; the L <= 4 instances sit at 97 without
// the bound and lose nothing to it.)
template <typename T, int LMAX, int NCW>
__global__ void __launch_bounds__((NCW + 1) * 32, (LMAX <= 4 && NCW == 4) ? 4 : 1)
cr_fused_tma_kernel(const __grid_constant__ CUtensorMap tmap, const FusedArgs a) {
    constexpr int TILE = NCW * 128;
    constexpr int BOXW = TILE < 256 ? TILE : 256;
    constexpr int NBOX = TILE / BOXW;
    typedef typename Vec4<T>::type V4;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int R = a.R, S = a.stages;
    const size_t stage_elems = (size_t)R * TILE;
    T *ring = reinterpret_cast<T *>(smem_raw);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem_raw + (size_t)S * stage_elems * sizeof(T));
    uint64_t *empty = full + S;
    volatile int *flags = reinterpret_cast<volatile int *>(empty + S);
    Step *steps_s = reinterpret_cast<Step *>(smem_raw + (((size_t)S * stage_elems * sizeof(T) + (size_t)S * 16 + 32 + 15) & ~(size_t)15));

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], NCW); }
        flags[0] = 0; flags[1] = 0; flags[2] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (a.steps_smem)
        for (int k = tid; k < a.n_steps; k += blockDim.x)
            reinterpret_cast<int4 *>(steps_s)[k] = __ldg(reinterpret_cast<const int4 *>(a.steps) + k);
    __syncthreads();

    const T *coeff = reinterpret_cast<const T *>(a.coeff);
    const uint32_t stage_bytes = (uint32_t)(stage_elems * sizeof(T));

    if (warp == NCW) {
        // ---------------- producer: one thread issues every TMA of this CTA ----------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (long long tile = blockIdx.x; tile < a.ntiles && ok; tile += gridDim.x) {
                const int x0 = (int)(tile * TILE);
                for (int k = 0; k < a.n_steps && ok; ++k) {
                    const int row0 = (a.n_inline ? a.steps_inline[k].node : (a.steps_smem ? steps_s[k].node : __ldg(&a.steps[k].node))) * a.m;
                    for (int c = 0; c < a.cpn; ++c) {
                        if (!mbar_wait(&empty[stage], phase ^ 1u, &flags[0], a.wait_ns)) { ok = false; break; }
                        mbar_expect_tx(&full[stage], stage_bytes);
                        T *dst = ring + (size_t)stage * stage_elems;
#pragma unroll
                        for (int b = 0; b < NBOX; ++b)
                            tma_load_2d(dst + (size_t)b * R * BOXW, &tmap, x0 + b * BOXW, row0 + c * R, &full[stage]);
                        ++issued;
                        if (++stage == S) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (!ok) {
                // give up: flag it, then wait (bounded) for the copies still in flight so that none
                // lands in shared memory after the CTA has gone
                flags[1] = 1;
                atomicExch(a.status, 1);
                for (long long i = issued > S ? issued - S : 0; i < issued; ++i)
                    mbar_wait(&full[i % S], (uint32_t)((i / S) & 1), &flags[2], a.wait_ns);
            }
        }
    } else {
        // ---------------- consumers ----------------
        // The schedule entry and the R coefficients of a box are fetched one box ahead, before the
        // wait on the current box, so that their latency hides behind the wait for the data.
        T acc[LMAX][4];
#pragma unroll
        for (int l = 0; l < LMAX; ++l)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[l][q] = T(0);
        const int col = tid * 4;
        const int box = col / BOXW, within = col % BOXW;
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        auto step_at = [&](int k) {
            if (a.n_inline) { Step t = a.steps_inline[k]; t.layer &= 0xff; return t; }
            if (a.steps_smem) { Step t = steps_s[k]; t.layer &= 0xff; return t; }
            return load_step(&a.steps[k]);
        };
        Step st_next = step_at(0);
        T cj_next[kMaxBoxRows];
        {
            const T *cf = coeff + (size_t)st_next.node * a.m;
#pragma unroll
            for (int j = 0; j < kMaxBoxRows; ++j) cj_next[j] = j < R ? __ldg(cf + j) : T(0);
        }
        for (long long tile = blockIdx.x; tile < a.ntiles && ok; tile += gridDim.x) {
            for (int k = 0; k < a.n_steps && ok; ++k) {
                T e[4] = {T(0), T(0), T(0), T(0)};
                Step st = st_next;
                for (int c = 0; c < a.cpn; ++c) {
                    T cj[kMaxBoxRows];
#pragma unroll
                    for (int j = 0; j < kMaxBoxRows; ++j) cj[j] = cj_next[j];
                    st = st_next;
                    {
                        int kn = k, cn = c + 1;
                        if (cn == a.cpn) { cn = 0; kn = k + 1 == a.n_steps ? 0 : k + 1; }
                        st_next = step_at(kn);
                        const T *cf = coeff + (size_t)st_next.node * a.m + cn * R;
#pragma unroll
                        for (int j = 0; j < kMaxBoxRows; ++j) cj_next[j] = j < R ? __ldg(cf + j) : T(0);
                    }
                    if (!mbar_wait_warp(&full[stage], phase, &flags[1], a.wait_ns)) { ok = false; break; }
                    const T *src = ring + (size_t)stage * stage_elems + (size_t)box * R * BOXW + within;
#pragma unroll
                    for (int j = 0; j < kMaxBoxRows; ++j) {
                        if (j < R) {
                            const V4 v = *reinterpret_cast<const V4 *>(src + (size_t)j * BOXW);
                            e[0] += cj[j] * v.x; e[1] += cj[j] * v.y; e[2] += cj[j] * v.z; e[3] += cj[j] * v.w;
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&empty[stage]);
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                fold<T, LMAX, 4>(acc, e, st.layer, weight_of<T>(st.wbits));
            }
            if (!ok) break;
            const long long gcol = tile * TILE + col;
            if (gcol < a.d) {
                V4 o;
                o.x = finish<T>(acc[0][0], a.shift); o.y = finish<T>(acc[0][1], a.shift);
                o.z = finish<T>(acc[0][2], a.shift); o.w = finish<T>(acc[0][3], a.shift);
                *reinterpret_cast<V4 *>(reinterpret_cast<T *>(a.out) + gcol) = o;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[0][q] = T(0);
        }
        if (!ok) { flags[0] = 1; atomicExch(a.status, 1); }
    }
}

// ------------------------------------------------------------------------------------------------
// K4b: fused aggregation, a batch of straggler patterns over the same slots
// ------------------------------------------------------------------------------------------------
//
// The coded gradient e_v of a node does not depend on the straggler pattern, so the slots are read
// from HBM once for the whole batch.  One persistent CTA per SM works on tiles of 128 columns with
// two kinds of warps:
//   * NLW loader warps each own a PRIVATE ring of `stages` TMA boxes (R slot rows x 128 columns) that
//     only they fill and drain, in order: after consuming box q a loader's lane 0 issues box
//     q + stages into the buffer it has just read (a single serial producer thread for all rings could
//     not keep up: each of its waits costs several hundred nanoseconds).  Loader w forms e_v (a full
//     tile row of float4s per warp) for union nodes w, w+NLW, .. and stores it in the tile's E buffer
//     in shared memory, E[buf][n_union][128];
//   * NRW replay warps replay every pattern's post-order schedule from E (warp r takes pattern groups
//     r, r+NRW, ..) and write one output tile per pattern.
// E is double buffered (when it fits), so the loaders stream tile t+1 while tile t is replayed and HBM
// never idles; loaders and replayers hand the buffers over with two mbarriers per buffer.
//
// Shared messages.  A parent's message depends only on the straggler sets of its own sub-tree
// (CR.Execute: m_(l,i) = a_f [children's messages] + g_D(l,i)), so for a node of layer L-1, whose
// children are leaves, the whole batch needs at most one message per distinct decode row of its group
// -- a dozen for a 12-ary tree with one straggler, against one evaluation per pattern.  When the host
// finds that this pays (n_ops > 0), the replay warps first form those message variants, once per tile:
// a warp takes a bottom-layer node, reads its own E row and the rows of its children in the union into
// registers once and writes every variant own + sum_j a[j] * child_j back into rows of the same buffer
// (the node's and its children's rows, which are dead from then on, then extra rows behind the union).
// The patterns' schedules then name a message row where they had the node and its leaves.
//
// Why private rings: with one ring shared by warps that each take every NLW-th box, a warp can reach a
// buffer whose previous box -- another warp's -- has not landed yet, since TMA completions are
// unordered; a parity wait cannot tell "one phase behind" from "done", the warp would read early and
// release the buffer twice.  Box number q of a loader (counted over the whole kernel) lives in its
// buffer q % stages with phase (q / stages) & 1.  Every warp passes every phase of every barrier it
// waits on, in order, so no wait can alias.

struct BatchArgs {
    const void *coeff;
    const Step *steps;
    const int32_t *pat_off;
    const int32_t *unodes;
    const uint32_t *wtab;  // distinct weight bit patterns of the batch
    int n_wtab;
    const uint32_t *units; // [n_groups * cpn][kUnitWords] unit records (see kUnitWords), 16-byte aligned
    int n_groups;          // groups of boxes per tile: loader w takes groups w, w + NLW, .., cpn boxes each
    int n_union, batch;
    int m, R, cpn, stages;
    int same_shape;  // every pattern's schedule has the same length and layer sequence
    int sched_smem;  // bytes of shared memory set aside for the staged schedules (0: replay reads them from global)
    int nst;         // same_shape: entries per schedule
    int nbuf;        // E buffers: 2, or 1 when two do not fit
    long long d;
    long long ntiles;
    void *out;
    int shift;
    int *status;
    unsigned long long wait_ns;  // bound of every wait, in nanoseconds
    // Messages shared by the patterns of the batch (see the kernel): rows of an E buffer (the union nodes,
    // then extra message rows), the bottom-layer nodes whose message variants are formed once per tile,
    // and their variant records.
    int n_rows;
    int n_ops;
    const int4 *ops;       // [n_ops] x = own row, y = row of the first child in the union, z = children in the
                           // union | variants << 8, w = word offset of the node's variant list in vtab
    const uint32_t *vtab;  // weight records (the decode weights of the children in the union, padded with zeros
                           // to a multiple of four words; equal records are stored once), then per node its
                           // variant list: pairs {destination row, word offset of the weight record}
    int vtab_words;
    int vtab_smem;         // the records are staged in shared memory behind the other tables
    int flat;              // two-layer tree, staged schedules: every entry of a pattern is a message row of layer 1
};

// The rows of one full box (kMaxBoxRows rows in use) combined into coded gradients, for a compile-time
// number EV of rows per node (0: the node continues in the next box): no predicate and no branch per row,
// eight loads in flight at a time, and the stores of completed nodes at fixed places.  `dst` is the E row of
// the first node the box completes.
template <typename T, int EV>
__device__ __forceinline__ void full_box_rows(const T *src, const uint32_t (&cb)[kMaxBoxRows], T (&e)[4], T *dst) {
    typedef typename Vec4<T>::type V4;
    constexpr int TILE = 128;
#pragma unroll
    for (int h = 0; h < kMaxBoxRows; h += 8) {
        V4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = *reinterpret_cast<const V4 *>(src + (size_t)(h + j) * TILE);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const T cj = weight_of<T>(cb[h + j]);
            e[0] += cj * v[j].x; e[1] += cj * v[j].y; e[2] += cj * v[j].z; e[3] += cj * v[j].w;
            if (EV > 0 && (h + j + 1) % (EV > 0 ? EV : 1) == 0) {
                V4 o; o.x = e[0]; o.y = e[1]; o.z = e[2]; o.w = e[3];
                *reinterpret_cast<V4 *>(dst) = o;
                dst += TILE;
                e[0] = e[1] = e[2] = e[3] = T(0);
            }
        }
    }
}

// SHARE: the instance that forms shared messages first; the other one is free of that code and of its
// registers (a node's children live in registers while its variants are formed).
// The eight-warp form (four loaders, four replay warps) is held to 128 registers so that two CTAs share an SM
// when the union is small: a tile of a small tree is a short chain of waits, and two chains overlap.
template <typename T, int LMAX, int NLW, int NRW, bool SHARE>
__global__ void __launch_bounds__((NLW + NRW) * 32, (NLW + NRW) <= 8 ? 2 : 1)
cr_fused_batch_tma_kernel(const __grid_constant__ CUtensorMap tmap, const BatchArgs a) {
    constexpr int TILE = 128;
    constexpr int NP = LMAX <= 4 ? 4 : 2;  // patterns replayed together by one warp
    typedef typename Vec4<T>::type V4;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int R = a.R, S = a.stages, NS = NLW * a.stages;
    const size_t stage_elems = (size_t)R * TILE;
    const size_t e_elems = (size_t)a.n_rows * TILE;
    T *ring = reinterpret_cast<T *>(smem_raw);
    T *E = ring + (size_t)NS * stage_elems;  // [nbuf][n_union][TILE]
    // staged schedules (same-shape batches with a weight table): lf[nst] = layer | first-child flag of
    // every step, ent[nst][batch_pad] = position of the node in E (bits 0..11) | index of the decode
    // weight in the table (bits 12..) per step and pattern, wtab_s[n_wtab] = the table
    int *lf = reinterpret_cast<int *>(E + (size_t)a.nbuf * e_elems);
    const int batch_pad = (a.batch + NP - 1) / NP * NP;
    uint32_t *ent = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned char *>(lf) + (((size_t)a.nst * 4 + 15) & ~(size_t)15));
    uint32_t *wtab_s = ent + (((size_t)a.nst * batch_pad + 3) & ~(size_t)3);
    // shared messages: the node table and, when it fits, the variant records behind the weight table
    int4 *ops_s = reinterpret_cast<int4 *>(wtab_s + (((size_t)a.n_wtab + 3) & ~(size_t)3));
    uint32_t *vtab_s = reinterpret_cast<uint32_t *>(ops_s + a.n_ops);
    const int pos_mask = a.n_wtab ? 0xfff : 0x7fffffff;
    uint64_t *full = reinterpret_cast<uint64_t *>(reinterpret_cast<unsigned char *>(lf) + a.sched_smem);
    uint64_t *e_full = full + NS;    // [2] E buffer written by all loaders
    uint64_t *e_free = e_full + 2;   // [2] E buffer released by all replayers
    volatile int *flags = reinterpret_cast<volatile int *>(e_free + 2);  // [0] someone gave up, [1] never set

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(&full[s], 1);
        for (int b = 0; b < 2; ++b) { mbar_init(&e_full[b], NLW); mbar_init(&e_free[b], NRW); }
        flags[0] = 0; flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (a.sched_smem) {
        for (int k = tid; k < a.nst; k += blockDim.x) lf[k] = __ldg(&a.steps[k].layer);
        for (int idx = tid; idx < a.nst * batch_pad; idx += blockDim.x) {
            const int k = idx / batch_pad, b = min(idx - k * batch_pad, a.batch - 1);  // padding repeats the last pattern
            ent[idx] = (uint32_t)__ldg(&a.steps[__ldg(&a.pat_off[b]) + k].index);
        }
        for (int i = tid; i < a.n_wtab; i += blockDim.x) wtab_s[i] = __ldg(&a.wtab[i]);
        for (int i = tid; i < a.n_ops; i += blockDim.x) ops_s[i] = __ldg(&a.ops[i]);
        if (a.vtab_smem)
            for (int i = tid; i < a.vtab_words; i += blockDim.x) vtab_s[i] = __ldg(&a.vtab[i]);
    }
    __syncthreads();

    const uint32_t stage_bytes = (uint32_t)(stage_elems * sizeof(T));

    if (warp < NLW) {
        // ---------------- loaders: stream their boxes, coded gradients of the union nodes -> E[buf] ----------------
        // A loader's work per tile is a fixed list of units (boxes): groups warp, warp + NLW, .. of `upg` units
        // each (a group is a box over several small nodes, or a tall node cut into upg boxes).  What a box is
        // -- its first slot row, the E row of its first node, after how many rows a node's coded gradient is
        // complete, its rows' coefficients -- is its unit record.  The list is the same for every tile, so with
        // at most 32 units per loader and tile (the usual case) lane k keeps the record of the loader's k-th
        // unit in registers for the whole kernel and hands it round by shuffles: the loop below then touches
        // global memory only through the copy engine.  (Read with plain loads in front of every box, the tables
        // cost three dependent L2 latencies per box and the loaders, not HBM, set the pace: 2800 cycles per 8 KB
        // box on the 156-node tree.  Sent along with each box as a second small bulk copy, they double the
        // number of requests to the copy engine, which then becomes the limit.)
        bool ok = true;
        const unsigned upg = (unsigned)a.cpn;
        const unsigned groups_w = warp < a.n_groups ? (unsigned)(a.n_groups - warp + NLW - 1) / NLW : 0u;   // groups of this loader per tile
        const unsigned units_w = groups_w * upg;
        const unsigned my_tiles = blockIdx.x < a.ntiles ? (unsigned)((a.ntiles - 1 - blockIdx.x) / gridDim.x + 1) : 0u;
        const unsigned total_boxes = my_tiles * units_w;
        T *my_ring = ring + (size_t)warp * S * stage_elems;
        uint64_t *my_full = full + warp * S;
        auto unit_at = [&](unsigned k) { return (unsigned)(warp + (int)(k / upg) * NLW) * upg + k % upg; };   // k-th unit of a tile
        const bool in_regs = units_w <= 32u;
        uint32_t myrec[kUnitWords];
#pragma unroll
        for (int w = 0; w < kUnitWords; ++w) myrec[w] = 0u;
        if (in_regs && (unsigned)lane < units_w) {
            const uint4 *g = reinterpret_cast<const uint4 *>(a.units + (size_t)unit_at((unsigned)lane) * kUnitWords);
#pragma unroll
            for (int w = 0; w < kUnitWords / 4; ++w) {
                const uint4 v = __ldg(g + w);
                myrec[4 * w] = v.x; myrec[4 * w + 1] = v.y; myrec[4 * w + 2] = v.z; myrec[4 * w + 3] = v.w;
            }
        }
        // cursor of the next box to issue: tile number of this CTA and unit within the tile (kept by all lanes,
        // so that all of them can take part in the shuffle that fetches the unit's first slot row)
        unsigned issued = 0, it_t = 0, it_k = 0;
        auto issue_next = [&]() {   // all lanes; lane 0 issues
            const int row0 = in_regs ? (int)__shfl_sync(0xffffffffu, myrec[16], (int)it_k)
                                     : (int)__ldg(a.units + (size_t)unit_at(it_k) * kUnitWords + 16);
            if (lane == 0) {
                const int slot = (int)(issued % (unsigned)S);
                const long long tile = (long long)blockIdx.x + (long long)it_t * gridDim.x;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(&my_full[slot], stage_bytes);
                tma_load_2d(my_ring + (size_t)slot * stage_elems, &tmap, (int)(tile * TILE), row0, &my_full[slot]);
            }
            ++issued;
            if (++it_k == units_w) { it_k = 0; ++it_t; }
        };
        while (issued < total_boxes && issued < (unsigned)S) issue_next();
        unsigned q = 0;  // next box to consume
        unsigned t = 0;  // tiles handled by this CTA so far
        T e[4] = {T(0), T(0), T(0), T(0)};
        for (long long tile = blockIdx.x; tile < a.ntiles && ok; tile += gridDim.x, ++t) {
            const int buf = (int)(t % (unsigned)a.nbuf);
            const unsigned use = t / (unsigned)a.nbuf;  // how many times this buffer has been filled before
            // the buffer must have been released by the replay of its previous tile
            if (!mbar_wait_warp(&e_free[buf], (use & 1u) ^ 1u, &flags[0], a.wait_ns)) { ok = false; break; }
            T *Eb = E + (size_t)buf * e_elems;
            for (unsigned k = 0; k < units_w && ok; ++k, ++q) {
                const int slot = (int)(q % (unsigned)S);
                const uint32_t phase = (q / (unsigned)S) & 1u;
                // the unit's record: coefficients of its rows and what the rows are (fetched before the wait)
                uint32_t cb[kMaxBoxRows], dsc[4];
                if (in_regs) {
#pragma unroll
                    for (int j = 0; j < kMaxBoxRows; ++j) cb[j] = __shfl_sync(0xffffffffu, myrec[j], (int)k);
#pragma unroll
                    for (int j = 1; j < 4; ++j) dsc[j] = __shfl_sync(0xffffffffu, myrec[16 + j], (int)k);
                } else {
                    const uint4 *g = reinterpret_cast<const uint4 *>(a.units + (size_t)unit_at(k) * kUnitWords);
                    const uint4 c0 = __ldg(g), c1 = __ldg(g + 1), c2 = __ldg(g + 2), c3 = __ldg(g + 3), d4 = __ldg(g + 4);
                    cb[0] = c0.x; cb[1] = c0.y; cb[2] = c0.z; cb[3] = c0.w; cb[4] = c1.x; cb[5] = c1.y; cb[6] = c1.z; cb[7] = c1.w;
                    cb[8] = c2.x; cb[9] = c2.y; cb[10] = c2.z; cb[11] = c2.w; cb[12] = c3.x; cb[13] = c3.y; cb[14] = c3.z; cb[15] = c3.w;
                    dsc[1] = d4.y; dsc[2] = d4.z; dsc[3] = d4.w;
                }
                // dsc: [1] = E row of the first node that this box completes, [2] = rows after which a node is
                // complete (0: the node continues in the loader's next box), [3] = rows of the box in use
                const int valid = (int)dsc[3], every = (int)dsc[2];
                int node_end = every ? every : kMaxBoxRows + 1, erow = (int)dsc[1];
                if (!mbar_wait_warp(&my_full[slot], phase, &flags[0], a.wait_ns)) { ok = false; break; }
                const T *src = my_ring + (size_t)slot * stage_elems + lane * 4;
                // Full boxes of the usual shapes take a branch-free body; the loop below serves ragged boxes
                // and odd node heights.  (The warps of this kernel run at about one instruction in seven
                // cycles -- dependent chains, three warps per scheduler -- so the instructions per row are
                // what a box costs: 1500 cycles with a predicate and a compare per row.)
                bool fast = valid == kMaxBoxRows;
                if (fast) {
                    T *dst = Eb + (size_t)erow * TILE + lane * 4;
                    switch (every) {
                        case 0: full_box_rows<T, 0>(src, cb, e, dst); break;
                        case 1: full_box_rows<T, 1>(src, cb, e, dst); break;
                        case 2: full_box_rows<T, 2>(src, cb, e, dst); break;
                        case 4: full_box_rows<T, 4>(src, cb, e, dst); break;
                        case 8: full_box_rows<T, 8>(src, cb, e, dst); break;
                        case 16: full_box_rows<T, 16>(src, cb, e, dst); break;
                        default: fast = false; break;
                    }
                }
                if (!fast)
#pragma unroll
                for (int h = 0; h < kMaxBoxRows; h += 8) {
                    V4 v[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (h + j < valid) v[j] = *reinterpret_cast<const V4 *>(src + (size_t)(h + j) * TILE);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (h + j < valid) {
                            const T cj = weight_of<T>(cb[h + j]);
                            e[0] += cj * v[j].x; e[1] += cj * v[j].y; e[2] += cj * v[j].z; e[3] += cj * v[j].w;
                            if (h + j + 1 == node_end) {   // last row of a node: its coded gradient is complete
                                V4 o; o.x = e[0]; o.y = e[1]; o.z = e[2]; o.w = e[3];
                                *reinterpret_cast<V4 *>(Eb + (size_t)erow * TILE + lane * 4) = o;
                                e[0] = e[1] = e[2] = e[3] = T(0);
                                ++erow; node_end += every;
                            }
                        }
                    }
                }
                // every lane has read the box: refill its buffer with box q + stages
                __syncwarp();
                if (issued < total_boxes) issue_next();
            }
            if (!ok) break;
            __syncwarp();
            if (lane == 0) mbar_arrive(&e_full[buf]);
        }
        if (!ok) {
            // give up: flag it, then wait (bounded) for this loader's copies still in flight, so that
            // none lands in shared memory after the CTA has gone
            flags[0] = 1;
            atomicExch(a.status, 1);
            for (unsigned b = q; b < issued; ++b)
                mbar_wait(&my_full[b % (unsigned)S], (b / (unsigned)S) & 1u, &flags[1], a.wait_ns);
        }
    } else {
        // ---------------- replayers: every pattern's schedule from E[buf] ----------------
        const int rw = warp - NLW;
        bool ok = true;
        unsigned t = 0;
        for (long long tile = blockIdx.x; tile < a.ntiles; tile += gridDim.x, ++t) {
            const int buf = (int)(t % (unsigned)a.nbuf);
            const unsigned use = t / (unsigned)a.nbuf;
            if (!mbar_wait_warp(&e_full[buf], use & 1u, &flags[0], a.wait_ns)) { ok = false; break; }
            T *Eb = E + (size_t)buf * e_elems;
            const long long gcol = tile * TILE + lane * 4;
            if constexpr (SHARE) {
                // messages of the bottom-layer nodes, every distinct variant once for the whole batch
                const int4 *ops_p = a.sched_smem ? ops_s : a.ops;
                const uint32_t *vt = a.vtab_smem ? vtab_s : a.vtab;
                for (int op = rw; op < a.n_ops; op += NRW) {
                    const int4 o = ops_p[op];
                    const int cnt = o.z & 0xff, nvar = o.z >> 8;
                    T own[4], ch[kMaxKids][4];
                    {
                        const V4 v = *reinterpret_cast<const V4 *>(Eb + (size_t)o.x * TILE + lane * 4);
                        own[0] = v.x; own[1] = v.y; own[2] = v.z; own[3] = v.w;
                    }
#pragma unroll
                    for (int j = 0; j < kMaxKids; ++j) {
                        if (j < cnt) {
                            const V4 v = *reinterpret_cast<const V4 *>(Eb + (size_t)(o.y + j) * TILE + lane * 4);
                            ch[j][0] = v.x; ch[j][1] = v.y; ch[j][2] = v.z; ch[j][3] = v.w;
                        } else {
                            ch[j][0] = ch[j][1] = ch[j][2] = ch[j][3] = T(0);
                        }
                    }
                    // per variant: the row its message goes to and where its weights are (nodes whose
                    // children in the union coincide share the weight records of their decode rows)
                    // (the next variant's entry and weights are read before the current message is stored:
                    // behind the store the compiler could not move them up, and every variant would cost
                    // two shared-memory latencies in a row)
                    const uint2 *list = reinterpret_cast<const uint2 *>(vt + o.w);
                    uint2 dv_next = list[0];
                    uint4 w_next[kMaxKids / 4];
#pragma unroll
                    for (int g = 0; g < kMaxKids / 4; ++g)
                        w_next[g] = g * 4 < cnt ? reinterpret_cast<const uint4 *>(vt + dv_next.y)[g] : make_uint4(0u, 0u, 0u, 0u);
                    for (int v = 0; v < nvar; ++v) {
                        const uint2 dv = dv_next;
                        uint4 w_cur[kMaxKids / 4];
#pragma unroll
                        for (int g = 0; g < kMaxKids / 4; ++g) w_cur[g] = w_next[g];
                        if (v + 1 < nvar) {
                            dv_next = list[v + 1];
#pragma unroll
                            for (int g = 0; g < kMaxKids / 4; ++g)
                                if (g * 4 < cnt) w_next[g] = reinterpret_cast<const uint4 *>(vt + dv_next.y)[g];
                        }
                        T msg[4] = {own[0], own[1], own[2], own[3]};
#pragma unroll
                        for (int g = 0; g < kMaxKids / 4; ++g) {
                            if (g * 4 < cnt) {
                                const uint4 wb = w_cur[g];
                                const T w0 = weight_of<T>(wb.x), w1 = weight_of<T>(wb.y), w2 = weight_of<T>(wb.z), w3 = weight_of<T>(wb.w);
#pragma unroll
                                for (int q = 0; q < 4; ++q)
                                    msg[q] += w0 * ch[g * 4][q] + w1 * ch[g * 4 + 1][q] + w2 * ch[g * 4 + 2][q] + w3 * ch[g * 4 + 3][q];
                            }
                        }
                        V4 o4; o4.x = msg[0]; o4.y = msg[1]; o4.z = msg[2]; o4.w = msg[3];
                        *reinterpret_cast<V4 *>(Eb + (size_t)dv.x * TILE + lane * 4) = o4;
                    }
                }
                // every replay warp reads message rows written by the others
                asm volatile("bar.sync 2, %0;" ::"r"(NRW * 32) : "memory");
            }
            if (SHARE && a.flat) {
                // Two-layer tree with shared messages: a pattern's schedule is the master's decode alone, a
                // weighted sum of n-s message rows.  NP patterns at a time, no layer bookkeeping.
                const int nst = a.nst;
                const int ngroups = (a.batch + NP - 1) / NP;
                const int g0 = ngroups < NRW ? (int)((rw + NRW - (t * (unsigned)ngroups) % NRW) % NRW) : rw;
                for (int g = g0; g < ngroups; g += NRW) {
                    T acc[NP][4];
#pragma unroll
                    for (int p = 0; p < NP; ++p)
#pragma unroll
                        for (int q = 0; q < 4; ++q) acc[p][q] = T(0);
                    const uint32_t *mine = ent + g * NP;
#pragma unroll 4
                    for (int k = 0; k < nst; ++k) {
                        uint32_t en[NP];
                        if (NP == 4) {
                            const uint4 t4 = *reinterpret_cast<const uint4 *>(mine + (size_t)k * batch_pad);
                            en[0] = t4.x; en[1] = t4.y; en[NP - 2] = t4.z; en[NP - 1] = t4.w;
                        } else {
                            const uint2 t2 = *reinterpret_cast<const uint2 *>(mine + (size_t)k * batch_pad);
                            en[0] = t2.x; en[1] = t2.y;
                        }
#pragma unroll
                        for (int p = 0; p < NP; ++p) {
                            const T w = weight_of<T>(wtab_s[en[p] >> 12]);
                            const V4 v = *reinterpret_cast<const V4 *>(Eb + (size_t)(en[p] & 0xfffu) * TILE + lane * 4);
                            acc[p][0] += w * v.x; acc[p][1] += w * v.y; acc[p][2] += w * v.z; acc[p][3] += w * v.w;
                        }
                    }
                    if (gcol < a.d) {
#pragma unroll
                        for (int p = 0; p < NP; ++p) {
                            const int b = g * NP + p;
                            if (b < a.batch) {
                                V4 o;
                                o.x = finish<T>(acc[p][0], a.shift); o.y = finish<T>(acc[p][1], a.shift);
                                o.z = finish<T>(acc[p][2], a.shift); o.w = finish<T>(acc[p][3], a.shift);
                                *reinterpret_cast<V4 *>(reinterpret_cast<T *>(a.out) + (size_t)b * a.d + gcol) = o;
                            }
                        }
                    }
                }
            } else if (a.sched_smem) {
                // NP patterns at a time per warp: their schedules visit the same layers, so one
                // branch per step serves NP independent chains.  Step entries come from the staged
                // table (broadcast shared-memory loads); the loop is unrolled by two so that the E rows
                // of the next step are in flight while the current one is folded.
                const int nst = a.nst;
                // fewer pattern groups than replay warps: the groups of consecutive tiles go to different
                // warps, so that all of them work (on different E buffers) instead of the first few
                const int ngroups = (a.batch + NP - 1) / NP;
                const int g0 = ngroups < NRW ? (int)((rw + NRW - (t * (unsigned)ngroups) % NRW) % NRW) : rw;
                for (int g = g0; g < ngroups; g += NRW) {
                    T acc[NP][LMAX][4];
#pragma unroll
                    for (int p = 0; p < NP; ++p)
#pragma unroll
                        for (int l = 0; l < LMAX; ++l)
#pragma unroll
                            for (int q = 0; q < 4; ++q) acc[p][l][q] = T(0);
                    const uint32_t *mine = ent + g * NP;
                    auto fetch = [&](int k, int &lfk, T (&e)[NP][4], T (&w)[NP]) {
                        lfk = lf[k];
                        uint32_t en[NP];
                        if (NP == 4) {
                            const uint4 t4 = *reinterpret_cast<const uint4 *>(mine + (size_t)k * batch_pad);
                            en[0] = t4.x; en[1] = t4.y; en[NP - 2] = t4.z; en[NP - 1] = t4.w;
                        } else {
                            const uint2 t2 = *reinterpret_cast<const uint2 *>(mine + (size_t)k * batch_pad);
                            en[0] = t2.x; en[1] = t2.y;
                        }
#pragma unroll
                        for (int p = 0; p < NP; ++p) {
                            w[p] = weight_of<T>(wtab_s[en[p] >> 12]);
                            const V4 v = *reinterpret_cast<const V4 *>(Eb + (size_t)(en[p] & 0xfffu) * TILE + lane * 4);
                            e[p][0] = v.x; e[p][1] = v.y; e[p][2] = v.z; e[p][3] = v.w;
                        }
                    };
                    int lfA, lfB;
                    T eA[NP][4], wA[NP], eB[NP][4], wB[NP];
                    fetch(0, lfA, eA, wA);
                    for (int k = 0; k < nst; k += 2) {
                        if (k + 1 < nst) fetch(k + 1, lfB, eB, wB);
                        fold_many<T, LMAX, NP, SHARE>(acc, eA, lfA, wA);
                        if (k + 1 < nst) {
                            if (k + 2 < nst) fetch(k + 2, lfA, eA, wA);
                            fold_many<T, LMAX, NP, SHARE>(acc, eB, lfB, wB);
                        }
                    }
                    if (gcol < a.d) {
#pragma unroll
                        for (int p = 0; p < NP; ++p) {
                            const int b = g * NP + p;
                            if (b < a.batch) {
                                V4 o;
                                o.x = finish<T>(acc[p][0][0], a.shift); o.y = finish<T>(acc[p][0][1], a.shift);
                                o.z = finish<T>(acc[p][0][2], a.shift); o.w = finish<T>(acc[p][0][3], a.shift);
                                *reinterpret_cast<V4 *>(reinterpret_cast<T *>(a.out) + (size_t)b * a.d + gcol) = o;
                            }
                        }
                    }
                }
            } else {
                // General case, one pattern at a time: lane i fetches entry i of the pattern's schedule
                // (one coalesced load per 32 entries); entries are broadcast with shuffles.
                const int b0 = a.batch < NRW ? (int)((rw + NRW - (t * (unsigned)a.batch) % NRW) % NRW) : rw;
                for (int b = b0; b < a.batch; b += NRW) {
                    T acc[LMAX][4];
#pragma unroll
                    for (int l = 0; l < LMAX; ++l)
#pragma unroll
                        for (int q = 0; q < 4; ++q) acc[l][q] = T(0);
                    const int k0 = __ldg(&a.pat_off[b]), k1 = __ldg(&a.pat_off[b + 1]);
                    for (int kb = k0; kb < k1; kb += 32) {
                        int4 mine = make_int4(0, 0, 0, 0);
                        if (kb + lane < k1) mine = __ldg(reinterpret_cast<const int4 *>(&a.steps[kb + lane]));
                        const int cnt = k1 - kb < 32 ? k1 - kb : 32;
                        for (int i = 0; i < cnt; ++i) {
                            const int layer = __shfl_sync(0xffffffffu, mine.y, i) & 0xff;
                            const uint32_t wb = (uint32_t)__shfl_sync(0xffffffffu, mine.z, i);
                            const int idx = __shfl_sync(0xffffffffu, mine.w, i) & pos_mask;
                            const V4 v = *reinterpret_cast<const V4 *>(Eb + (size_t)idx * TILE + lane * 4);
                            const T e[4] = {v.x, v.y, v.z, v.w};
                            fold<T, LMAX, 4>(acc, e, layer, weight_of<T>(wb));
                        }
                    }
                    if (gcol < a.d) {
                        V4 o;
                        o.x = finish<T>(acc[0][0], a.shift); o.y = finish<T>(acc[0][1], a.shift);
                        o.z = finish<T>(acc[0][2], a.shift); o.w = finish<T>(acc[0][3], a.shift);
                        *reinterpret_cast<V4 *>(reinterpret_cast<T *>(a.out) + (size_t)b * a.d + gcol) = o;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&e_free[buf]);  // this warp has finished reading E[buf]
        }
        if (!ok) { flags[0] = 1; atomicExch(a.status, 1); }
    }
}

// ------------------------------------------------------------------------------------------------
// Fused aggregation with plain loads (any d, any alignment); grid.y = pattern
// ------------------------------------------------------------------------------------------------

template <typename T, int V> struct Loader;
template <typename T> struct Loader<T, 1> {
    static __device__ __forceinline__ void load(const T *p, T (&v)[1]) { v[0] = __ldg(p); }
    static __device__ __forceinline__ void store(T *p, const T (&v)[1]) { p[0] = v[0]; }
};
template <> struct Loader<float, 4> {
    static __device__ __forceinline__ void load(const float *p, float (&v)[4]) {
        float4 t;
        asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(t.x), "=f"(t.y), "=f"(t.z), "=f"(t.w) : "l"(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&v)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};
template <> struct Loader<int, 4> {
    static __device__ __forceinline__ void load(const int *p, int (&v)[4]) {
        int4 t;
        asm volatile("ld.global.nc.L1::no_allocate.v4.s32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(t.x), "=r"(t.y), "=r"(t.z), "=r"(t.w) : "l"(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    static __device__ __forceinline__ void store(int *p, const int (&v)[4]) {
        *reinterpret_cast<int4 *>(p) = make_int4(v[0], v[1], v[2], v[3]);
    }
};

// PIPE = 4 (m % 4 == 0): the next four slot rows (of this node or the next) are requested before the
// current four are combined, so that eight row loads per thread are in flight instead of four.
// PIPE = 1 (m == 1, aggregation of coded gradients): the rows of four schedule entries are requested
// at once, and the next four before these are folded.
// A single short schedule travels in the kernel parameters (inl.n > 0; `steps` and `pat_off` unused).
constexpr int kMaxSplit = 16;
struct InlineSchedule {
    int n;
    int nseg;                      // > 0: block row b folds entries seg_off[b] .. seg_off[b+1]-1 only
    int seg_off[kMaxSplit + 1];
    Step steps[kInlineSteps];
};

// (Four 256-thread blocks per SM, 64 registers per thread, keep the most loads in flight; the instances
// bounded here fit that without spilling.  PIPE = 5 is the generic path (PIPE = 0) for two or three rows
// per node, the short launches of flat gradient coding with a few dozen rows per thread, which gain from
// more resident threads instead: six blocks at 40 registers (five for int32), n = 12, s = 1 at d = 2^22:
// 4.9 -> 5.8 TB/s.  With nine rows per node the same bound costs 14 % at d = 2^20, so it is not general.  Unbounded, the four-layer float instance took 75 registers,
// three blocks per SM, and lost a tenth of its throughput.)
template <typename T, int LMAX, int V, int PIPE>
__global__ void __launch_bounds__(256, (LMAX <= 2 && PIPE == 5) ? (std::is_floating_point<T>::value ? 6 : 5)
                                                                     : ((LMAX <= 2 || (LMAX <= 4 && PIPE != 1)) ? 4 : 1))
cr_fused_ldg_kernel(const T *__restrict__ G, const T *__restrict__ coeff, const Step *__restrict__ steps,
                    const int32_t *__restrict__ pat_off, int m, long long d, T *__restrict__ out, int shift,
                    const __grid_constant__ InlineSchedule inl) {
    // The split form launches the kernel that adds the sub-trees' rows as a programmatic dependent: it may be
    // set up while this grid still runs (it waits for this grid's completion before it reads anything).
    asm volatile("griddepcontrol.launch_dependents;");
    const int b = blockIdx.y;
    const long long col = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * V;
    if (col >= d) return;
    const int k0 = inl.n ? (inl.nseg ? inl.seg_off[b] : 0) : __ldg(&pat_off[b]);
    const int k1 = inl.n ? (inl.nseg ? inl.seg_off[b + 1] : inl.n) : __ldg(&pat_off[b + 1]);
    auto step_at = [&](int k) {
        if (inl.n) { Step t = inl.steps[k]; t.layer &= 0xff; return t; }
        return load_step(&steps[k]);
    };
    T acc[LMAX][V];
#pragma unroll
    for (int l = 0; l < LMAX; ++l)
#pragma unroll
        for (int q = 0; q < V; ++q) acc[l][q] = T(0);
    if constexpr (PIPE == 1) {
        T cur[4][V], nxt[4][V];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (k0 + j < k1) Loader<T, V>::load(G + (size_t)step_at(k0 + j).node * d + col, cur[j]);
#pragma unroll 2
        for (int k = k0; k < k1; k += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (k + 4 + j < k1) Loader<T, V>::load(G + (size_t)step_at(k + 4 + j).node * d + col, nxt[j]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (k + j < k1) {
                    const Step st = step_at(k + j);
                    const T c = __ldg(coeff + st.node);
                    T e[V];
#pragma unroll
                    for (int q = 0; q < V; ++q) e[q] = c * cur[j][q];
                    fold<T, LMAX, V>(acc, e, st.layer, weight_of<T>(st.wbits));
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int q = 0; q < V; ++q) cur[j][q] = nxt[j][q];
        }
    } else if constexpr (PIPE == 4) {
        // m % 4 == 0: the work is a list of groups of four slot rows, node by node
        T cur[4][V], nxt[4][V];
        const int gpn = m >> 2;
        int k = k0, g = 0;
        Step st = k0 < k1 ? step_at(k0) : Step{0, 0, 0u, 0};
        if (k0 < k1) {
            const T *row = G + (size_t)st.node * m * d + col;
#pragma unroll
            for (int j = 0; j < 4; ++j) Loader<T, V>::load(row + (size_t)j * d, cur[j]);
        }
        T e[V];
#pragma unroll
        for (int q = 0; q < V; ++q) e[q] = T(0);
#pragma unroll 2
        while (k < k1) {
            int kn = k, gn = g + 1;
            Step sn = st;
            if (gn == gpn) {
                gn = 0; ++kn;
                if (kn < k1) sn = step_at(kn);
            }
            if (kn < k1) {
                const T *row = G + ((size_t)sn.node * m + 4 * gn) * d + col;
#pragma unroll
                for (int j = 0; j < 4; ++j) Loader<T, V>::load(row + (size_t)j * d, nxt[j]);
            }
            const T *cf = coeff + (size_t)st.node * m + 4 * g;
            const T c0 = __ldg(cf), c1 = __ldg(cf + 1), c2 = __ldg(cf + 2), c3 = __ldg(cf + 3);
#pragma unroll
            for (int q = 0; q < V; ++q) e[q] += c0 * cur[0][q] + c1 * cur[1][q] + c2 * cur[2][q] + c3 * cur[3][q];
            if (gn == 0) {
                fold<T, LMAX, V>(acc, e, st.layer, weight_of<T>(st.wbits));
#pragma unroll
                for (int q = 0; q < V; ++q) e[q] = T(0);
            }
            k = kn; g = gn; st = sn;
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int q = 0; q < V; ++q) cur[j][q] = nxt[j][q];
        }
    } else
    for (int k = k0; k < k1; ++k) {
        const Step st = step_at(k);
        const T *row = G + (size_t)st.node * m * d + col;
        const T *cf = coeff + (size_t)st.node * m;
        T e[V];
#pragma unroll
        for (int q = 0; q < V; ++q) e[q] = T(0);
        int j = 0;
        for (; j + 4 <= m; j += 4) {
            T v0[V], v1[V], v2[V], v3[V];
            Loader<T, V>::load(row + (size_t)(j + 0) * d, v0);
            Loader<T, V>::load(row + (size_t)(j + 1) * d, v1);
            Loader<T, V>::load(row + (size_t)(j + 2) * d, v2);
            Loader<T, V>::load(row + (size_t)(j + 3) * d, v3);
            const T c0 = __ldg(cf + j), c1 = __ldg(cf + j + 1), c2 = __ldg(cf + j + 2), c3 = __ldg(cf + j + 3);
#pragma unroll
            for (int q = 0; q < V; ++q) e[q] += c0 * v0[q] + c1 * v1[q] + c2 * v2[q] + c3 * v3[q];
        }
        for (; j < m; ++j) {
            T v0[V];
            Loader<T, V>::load(row + (size_t)j * d, v0);
            const T c0 = __ldg(cf + j);
#pragma unroll
            for (int q = 0; q < V; ++q) e[q] += c0 * v0[q];
        }
        fold<T, LMAX, V>(acc, e, st.layer, weight_of<T>(st.wbits));
    }
    T o[V];
#pragma unroll
    for (int q = 0; q < V; ++q) o[q] = finish<T>(acc[0][q], shift);
    Loader<T, V>::store(out + (size_t)b * d + col, o);
}

// ------------------------------------------------------------------------------------------------
// K5: uncoded comparator -- plain sum of the same slot rows, all weights 1
// ------------------------------------------------------------------------------------------------

// out[col] = finish(sum_r rows[r][col]): the master's decode of the split form (the decode weights are
// already applied by the sub-tree blocks).
template <typename T>
__global__ void __launch_bounds__(256)
cr_sum_rows_kernel(const T *__restrict__ rows, int nrows, long long d, T *__restrict__ out, int shift) {
    const long long col = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    // launched as a programmatic dependent of the kernel that writes `rows`: wait until that grid has
    // completed and its writes are visible (returns at once when there is no such dependency)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (col >= d) return;
    T sum = T(0);
    for (int r = 0; r < nrows; ++r) sum += rows[(size_t)r * d + col];
    out[col] = finish<T>(sum, shift);
}

template <typename T, int V>
__global__ void __launch_bounds__(256)
cr_uncoded_sum_kernel(const T *__restrict__ G, const Step *__restrict__ steps, const int32_t *__restrict__ pat_off,
                      int m, long long d, T *__restrict__ out) {
    const int b = blockIdx.y;
    const long long col = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * V;
    if (col >= d) return;
    const int k0 = __ldg(&pat_off[b]), k1 = __ldg(&pat_off[b + 1]);
    T acc[V];
#pragma unroll
    for (int q = 0; q < V; ++q) acc[q] = T(0);
    for (int k = k0; k < k1; ++k) {
        const T *row = G + (size_t)__ldg(&steps[k].node) * m * d + col;
        int j = 0;
        for (; j + 4 <= m; j += 4) {
            T v0[V], v1[V], v2[V], v3[V];
            Loader<T, V>::load(row + (size_t)(j + 0) * d, v0);
            Loader<T, V>::load(row + (size_t)(j + 1) * d, v1);
            Loader<T, V>::load(row + (size_t)(j + 2) * d, v2);
            Loader<T, V>::load(row + (size_t)(j + 3) * d, v3);
#pragma unroll
            for (int q = 0; q < V; ++q) acc[q] += (v0[q] + v1[q]) + (v2[q] + v3[q]);
        }
        for (; j < m; ++j) {
            T v0[V];
            Loader<T, V>::load(row + (size_t)j * d, v0);
#pragma unroll
            for (int q = 0; q < V; ++q) acc[q] += v0[q];
        }
    }
    Loader<T, V>::store(out + (size_t)b * d + col, acc);
}

// ------------------------------------------------------------------------------------------------
// K2 / K3: unfused verification path
// ------------------------------------------------------------------------------------------------

template <typename T, int V>
__global__ void __launch_bounds__(256)
cr_encode_kernel(const T *__restrict__ G, const T *__restrict__ coeff, const int32_t *__restrict__ nodes, int y0, int m,
                 long long d, T *__restrict__ E) {
    // (y0: first entry served by this launch; a grid has at most 65535 rows of blocks)
    const int v = nodes ? __ldg(&nodes[y0 + blockIdx.y]) : y0 + (int)blockIdx.y;
    const long long col = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * V;
    if (col >= d) return;
    const T *row = G + (size_t)v * m * d + col;
    const T *cf = coeff + (size_t)v * m;
    T e[V];
#pragma unroll
    for (int q = 0; q < V; ++q) e[q] = T(0);
    for (int j = 0; j < m; ++j) {
        T x[V];
        Loader<T, V>::load(row + (size_t)j * d, x);
        const T c = __ldg(cf + j);
#pragma unroll
        for (int q = 0; q < V; ++q) e[q] += c * x[q];
    }
    Loader<T, V>::store(E + (size_t)v * d + col, e);
}

template <typename T, int V>
__global__ void __launch_bounds__(256)
cr_decode_kernel(const T *__restrict__ M_child, const T *__restrict__ E_parent, const T *__restrict__ W,
                 const int32_t *__restrict__ active, int y0, int n, long long d, T *__restrict__ M_parent, int shift) {
    const int i = y0 + (int)blockIdx.y;
    if (active && __ldg(&active[i]) == 0) return;
    const long long col = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * V;
    if (col >= d) return;
    T acc[V];
#pragma unroll
    for (int q = 0; q < V; ++q) acc[q] = T(0);
    for (int j = 0; j < n; ++j) {
        const T w = __ldg(&W[(size_t)i * n + j]);
        if (w == T(0)) continue;  // stragglers and unused survivors are never read
        T x[V];
        Loader<T, V>::load(M_child + ((size_t)i * n + j) * d + col, x);
#pragma unroll
        for (int q = 0; q < V; ++q) acc[q] += w * x[q];
    }
    if (E_parent) {
        T x[V];
        Loader<T, V>::load(E_parent + (size_t)i * d + col, x);
#pragma unroll
        for (int q = 0; q < V; ++q) acc[q] += x[q];
    }
#pragma unroll
    for (int q = 0; q < V; ++q) acc[q] = finish<T>(acc[q], shift);
    Loader<T, V>::store(M_parent + (size_t)i * d + col, acc);
}

// ------------------------------------------------------------------------------------------------
// K1: partial gradients of linear regression, X_p^T (X_p w - y_p), two passes
// ------------------------------------------------------------------------------------------------

// Pass 1: one warp per (slot item, row): r = <X_p[row,:], w> - y_p[row].
template <int V>
__global__ void __launch_bounds__(256)
cr_residual_kernel(const float *__restrict__ X, const float *__restrict__ y, const float *__restrict__ w,
                   const int32_t *__restrict__ part, const int32_t *__restrict__ order, long long total_rows, int rows,
                   long long d, float *__restrict__ resid, int loss) {
    const int lane = threadIdx.x & 31;
    const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (long long idx = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; idx < total_rows; idx += warps) {
        // `order` (may be null) lists the items grouped by partition: the warps that run side by side then
        // read the same rows of X and share them through L2
        const long long pos = idx / rows;
        const int row = (int)(idx - pos * rows);
        const long long item = order ? (long long)__ldg(&order[pos]) : pos;
        const int p = __ldg(&part[item]);
        const float *xr = X + ((size_t)p * rows + row) * d;
        float acc = 0.f;
        if (V == 4) {
            // four 16-byte loads of the row in flight per lane (one per step left the pass bound by the
            // latency of its loads), four partial sums
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            long long c = lane * 4;
            for (; c + 384 < d; c += 512) {
                const float4 x0 = __ldg(reinterpret_cast<const float4 *>(xr + c));
                const float4 x1 = __ldg(reinterpret_cast<const float4 *>(xr + c + 128));
                const float4 x2 = __ldg(reinterpret_cast<const float4 *>(xr + c + 256));
                const float4 x3 = __ldg(reinterpret_cast<const float4 *>(xr + c + 384));
                const float4 w0 = __ldg(reinterpret_cast<const float4 *>(w + c));
                const float4 w1 = __ldg(reinterpret_cast<const float4 *>(w + c + 128));
                const float4 w2 = __ldg(reinterpret_cast<const float4 *>(w + c + 256));
                const float4 w3 = __ldg(reinterpret_cast<const float4 *>(w + c + 384));
                a0 += x0.x * w0.x + x0.y * w0.y + x0.z * w0.z + x0.w * w0.w;
                a1 += x1.x * w1.x + x1.y * w1.y + x1.z * w1.z + x1.w * w1.w;
                a2 += x2.x * w2.x + x2.y * w2.y + x2.z * w2.z + x2.w * w2.w;
                a3 += x3.x * w3.x + x3.y * w3.y + x3.z * w3.z + x3.w * w3.w;
            }
            for (; c < d; c += 128) {
                const float4 xv = __ldg(reinterpret_cast<const float4 *>(xr + c));
                const float4 wv = __ldg(reinterpret_cast<const float4 *>(w + c));
                a0 += xv.x * wv.x + xv.y * wv.y + xv.z * wv.z + xv.w * wv.w;
            }
            acc = (a0 + a1) + (a2 + a3);
        } else {
            for (long long c = lane; c < d; c += 32) acc += __ldg(xr + c) * __ldg(w + c);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) {
            if (loss == 1) acc = 1.f / (1.f + expf(-acc));   // logistic: sigmoid of the score
            resid[item * rows + row] = acc - __ldg(&y[(size_t)p * rows + row]);
        }
    }
}

// Pass 2: grid (column tiles, items); a thread owns V columns and walks all rows of the item.
template <int V>
__global__ void __launch_bounds__(128)
cr_xt_r_kernel(const float *__restrict__ X, const int32_t *__restrict__ part, const int32_t *__restrict__ order,
               const float *__restrict__ resid, int y0, int rows, long long d, float *__restrict__ G) {
    const long long item = order ? (long long)__ldg(&order[y0 + blockIdx.y]) : (long long)y0 + blockIdx.y;
    const long long col = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * V;
    if (col >= d) return;
    const int p = __ldg(&part[item]);
    const float *xp = X + (size_t)p * rows * d + col;
    const float *r = resid + item * rows;
    float acc[V];
#pragma unroll
    for (int q = 0; q < V; ++q) acc[q] = 0.f;
    int row = 0;
    for (; row + 4 <= rows; row += 4) {
        float v0[V], v1[V], v2[V], v3[V];
        Loader<float, V>::load(xp + (size_t)(row + 0) * d, v0);
        Loader<float, V>::load(xp + (size_t)(row + 1) * d, v1);
        Loader<float, V>::load(xp + (size_t)(row + 2) * d, v2);
        Loader<float, V>::load(xp + (size_t)(row + 3) * d, v3);
        const float r0 = __ldg(r + row), r1 = __ldg(r + row + 1), r2 = __ldg(r + row + 2), r3 = __ldg(r + row + 3);
#pragma unroll
        for (int q = 0; q < V; ++q) acc[q] += r0 * v0[q] + r1 * v1[q] + r2 * v2[q] + r3 * v3[q];
    }
    for (; row < rows; ++row) {
        float v0[V];
        Loader<float, V>::load(xp + (size_t)row * d, v0);
        const float r0 = __ldg(r + row);
#pragma unroll
        for (int q = 0; q < V; ++q) acc[q] += r0 * v0[q];
    }
    Loader<float, V>::store(G + (size_t)item * d + col, acc);
}

// ------------------------------------------------------------------------------------------------
// K1 (one pass): X_p^T (X_p w - y_p) with every X element read from HBM once
// ------------------------------------------------------------------------------------------------
//
// A cluster of `csplit` CTAs owns one (node, slot) item; CTA c takes a contiguous range of the
// partition's rows.  A block of RB consecutive rows is one contiguous piece of X, so it is staged with a
// single bulk copy (TMA, no tensor map) into a ring of shared-memory buffers.  Per block: pass A forms
// the residuals r = X_b w - y_b (warp-shuffle reduction, then across the 8 warps through shared
// memory), pass B adds r^T X_b to the thread's column accumulators, both from shared memory.  Thread t
// owns columns 4t + 1024k .. +3 (k < KPT), so d <= 1024 * KPT.  At the end the CTAs of the cluster add
// their partial gradients through distributed shared memory, each CTA reducing and storing one slice
// of the columns: deterministic, no atomics, no scratch in global memory.

struct PgArgs {
    const float *X;
    const float *y;
    const float *w;
    const int32_t *part;
    const int32_t *order; // [items] or null: cluster y works on item order[y] (items that read the same
                          // partition launched next to each other share its rows through L2)
    const float *coeff;   // [N*m] slot coefficients, or null: every slot weighs 1
    float *G;             // [items][d]
    int rows;
    int slots_per_item;   // 1: an item is one (node, slot); m: an item is a node and its slots are
                          //    combined with their coefficients (the coded gradient of the node)
    int loss;             // 0: squared loss, r = X w - y; 1: logistic loss, r = sigmoid(X w) - y
    int RB;
    int stages;
    long long d;
    int *status;
    unsigned long long wait_ns;  // bound of every wait, in nanoseconds
};

// Rows of a block: as many as a thread can keep in registers (its KPT column groups of each row).
__host__ __device__ constexpr int pg_block_rows(int kpt) { return 12 / kpt > 0 ? 12 / kpt : 1; }
// Words of one buffer of per-warp partial residuals: chunks of four rows, [row in chunk][warp].
__host__ __device__ constexpr int pg_red_words(int kpt) { return (pg_block_rows(kpt) + 3) / 4 * 32; }

__device__ __forceinline__ float4 lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

// Sums over the warp of R per-lane values, four rows at a time: the first two exchange steps halve the
// number of values instead of repeating the butterfly per row (6 shuffles for 4 rows against 20), after which
// lane class (lane >> 3) holds row 2 * (bit 3) + (bit 4) of the chunk.  One lane per class stores the warp's
// sum at red[chunk][row][warp].
template <int R>
__device__ __forceinline__ void pg_warp_sums(const float (&part)[R], float *redb, int warp, int lane) {
    constexpr unsigned FULL = 0xffffffffu;
    const bool up16 = (lane & 16) != 0, up8 = (lane & 8) != 0;
#pragma unroll
    for (int c = 0; c < (R + 3) / 4; ++c) {
        const int n = R - 4 * c < 4 ? R - 4 * c : 4;   // rows of this chunk
        float b;
        if (n == 1) {
            b = part[4 * c];
            b += __shfl_xor_sync(FULL, b, 16);
            b += __shfl_xor_sync(FULL, b, 8);
        } else {
            // (indices clamped where the chunk has fewer rows: those values are not used)
            const float v0 = part[4 * c], v1 = part[4 * c + 1 < R ? 4 * c + 1 : 0];
            const float a0 = (up16 ? v1 : v0) + __shfl_xor_sync(FULL, up16 ? v0 : v1, 16);
            if (n == 2) {
                b = a0 + __shfl_xor_sync(FULL, a0, 8);
            } else {
                const float v2 = part[4 * c + 2 < R ? 4 * c + 2 : 0], v3 = n == 4 ? part[4 * c + 3 < R ? 4 * c + 3 : 0] : 0.f;
                const float a1 = (up16 ? v3 : v2) + __shfl_xor_sync(FULL, up16 ? v2 : v3, 16);
                b = (up8 ? a1 : a0) + __shfl_xor_sync(FULL, up8 ? a0 : a1, 8);
            }
        }
        b += __shfl_xor_sync(FULL, b, 4);
        b += __shfl_xor_sync(FULL, b, 2);
        b += __shfl_xor_sync(FULL, b, 1);
        // n == 1: every class holds row 0; n == 2: classes with bit 4 hold row 1 (both bit-3 classes alike)
        const int row = n == 1 ? 0 : (n == 2 ? (lane >> 4) & 1 : ((lane >> 3) & 1) * 2 + ((lane >> 4) & 1));
        if ((lane & 7) == 0) redb[c * 32 + row * 8 + warp] = b;
    }
}

// The residual sums of the block's rows from the eight warps' partial sums: every thread reads the eight
// values of each row (two broadcast loads) and adds them as a tree.  (Letting lane l read one entry and
// adding across lanes takes a third of the instructions but four dependent shuffles; the block's time
// is set by the length of this chain, not by the instruction count.)
template <int R>
__device__ __forceinline__ void pg_block_sums(const float *redb, int lane, float (&z)[R]) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const float4 p0 = *reinterpret_cast<const float4 *>(redb + (r / 4) * 32 + (r % 4) * 8);
        const float4 p1 = *reinterpret_cast<const float4 *>(redb + (r / 4) * 32 + (r % 4) * 8 + 4);
        z[r] = ((p0.x + p0.y) + (p0.z + p0.w)) + ((p1.x + p1.y) + (p1.z + p1.w));
    }
}

// GENERAL = false is the case of one slot per item without slot coefficient, kept free of the bookkeeping of
// the general one (measured: 5 % faster on 2048 x 4096 partitions).
// Per block a thread reads its share of every row from shared memory ONCE, into registers: the same
// values serve the residuals (pass A) and, once the residuals are known, the gradient update (pass B).
// One CTA-wide barrier per block is all the synchronisation there is -- it also tells that everybody has
// read the buffer, so the copy of block blk + S goes into it at once.  What a block costs besides its
// multiply-adds is a chain of dependent instructions that every warp runs once per block, whatever the
// number of rows (measured: blocks of one row take as long as blocks of three), so that chain is kept
// short: 32-bit shared-memory addresses, buffer and phase counted up instead of divided out, the warp
// sums of all rows in one butterfly, the cross-warp sums by shuffles.
// (The first version read X from shared memory in both passes and took three barriers per block:
// shared-memory wavefronts 48 %, DRAM 48 % of peak.)
template <int KPT, bool GENERAL, bool LOGISTIC>
__global__ void __launch_bounds__(256, 2)
cr_partial_fused_kernel(const PgArgs a) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    constexpr int RBC = pg_block_rows(KPT);
    constexpr int REDW = pg_red_words(KPT);
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int d = (int)a.d;              // d <= 1024 * KPT
    const int RB = a.RB, S = a.stages;   // RB <= RBC
    const size_t stage_elems = (size_t)RB * d;
    float *ring = reinterpret_cast<float *>(smem_raw);
    float *gpart = ring + (size_t)S * stage_elems;          // [d] this CTA's partial gradient
    float *red = gpart + d;                                 // [2][REDW] per-warp partial residuals, double buffered
    uint64_t *full = reinterpret_cast<uint64_t *>(red + 2 * REDW);
    volatile int *flags = reinterpret_cast<volatile int *>(full + S);

    if (tid == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&full[s], 1);
        flags[0] = 0; flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    // The item's work is a list of row blocks: slot by slot, `bps` blocks of RB rows per slot (a block
    // never straddles two slots, whose partitions lie apart).  CTA c of the cluster takes a contiguous
    // share of the list.
    const long long item = a.order ? (long long)__ldg(&a.order[blockIdx.y]) : (long long)blockIdx.y;
    const int spi = GENERAL ? a.slots_per_item : 1;
    const int bps = (a.rows + RB - 1) / RB;
    const int total_blocks = spi * bps;
    const int per_cta = (total_blocks + (int)gridDim.x - 1) / (int)gridDim.x;
    const int b0 = min(total_blocks, (int)blockIdx.x * per_cta);
    const int nblocks = min(total_blocks, b0 + per_cta) - b0;
    // Position in the list, kept incrementally (no division and no dependent load per block): slot
    // within the item, block within the slot, where the block's rows and labels start; one copy for the
    // thread that issues the copies (it runs S blocks ahead), one for the consumers.
    const int slot0 = b0 / bps;
    int i_slot = slot0, i_bi = b0 - slot0 * bps, c_slot = slot0, c_bi = i_bi;
    const float *i_src = a.X, *c_y = a.y;
    float c_scale = 1.f;
    if (nblocks > 0) {
        const int p0 = __ldg(&a.part[item * spi + slot0]);
        i_src = a.X + ((size_t)p0 * a.rows + (size_t)i_bi * RB) * d;
        c_y = a.y + (size_t)p0 * a.rows + (size_t)c_bi * RB;
        if (GENERAL && a.coeff) c_scale = __ldg(&a.coeff[item * spi + slot0]);
    }

    float4 wv[KPT], acc[KPT];
    uint32_t koff[KPT];   // byte offset of the thread's k-th column group in a row; a group beyond d reads
                          // the row's first four columns instead (always there: finite numbers, against a
                          // zero weight, never stored)
#pragma unroll
    for (int k = 0; k < KPT; ++k) {
        const int col = 4 * tid + 1024 * k;
        wv[k] = col < d ? __ldg(reinterpret_cast<const float4 *>(a.w + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
        koff[k] = col < d ? (uint32_t)col * 4u : 0u;
        acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const uint32_t ring_u32 = smem_u32(ring);
    const uint32_t row_bytes = (uint32_t)d * 4u, stage_bytes = (uint32_t)RB * row_bytes;

    int issued = 0, i_stage = 0;
    auto issue = [&]() {  // thread 0 only; blocks are issued in order
        const int nr_i = min(RB, a.rows - i_bi * RB);
        const uint32_t bytes = (uint32_t)nr_i * row_bytes;
        mbar_expect_tx(&full[i_stage], bytes);
        bulk_load_1d(ring + (size_t)i_stage * stage_elems, i_src, bytes, &full[i_stage]);
        i_src += (size_t)nr_i * d;
        if (++i_stage == S) i_stage = 0;
        ++i_bi;
        ++issued;
        if (GENERAL && i_bi == bps) {
            i_bi = 0; ++i_slot;
            if (issued < nblocks) i_src = a.X + (size_t)__ldg(&a.part[item * spi + i_slot]) * a.rows * d;
        }
    };
    if (tid == 0)
        while (issued < nblocks && issued < S) issue();

    int done = 0, stage = 0;
    uint32_t phase = 0;
    for (int blk = 0; blk < nblocks; ++blk) {
        const int nr = min(RB, a.rows - c_bi * RB);
        // labels of the block's rows, fetched before the wait so that their latency hides behind it
        float yv[RBC];
#pragma unroll
        for (int r = 0; r < RBC; ++r) yv[r] = r < nr ? __ldg(c_y + r) : 0.f;
        const float scale = c_scale;
        c_y += RB;
        ++c_bi;
        if (GENERAL && c_bi == bps) {     // the next block opens the next slot of the item
            c_bi = 0; ++c_slot;
            if (blk + 1 < nblocks) {
                c_y = a.y + (size_t)__ldg(&a.part[item * spi + c_slot]) * a.rows;
                if (a.coeff) c_scale = __ldg(&a.coeff[item * spi + c_slot]);
            }
        }
        const int ok = mbar_wait(&full[stage], phase, &flags[1], a.wait_ns) ? 1 : 0;
        const uint32_t xb = ring_u32 + (uint32_t)stage * stage_bytes;
        // this thread's share of the block, read once; pass A: partial residuals
        float4 xf[RBC][KPT];
        float part[RBC];
        if (nr == RBC) {
#pragma unroll
            for (int r = 0; r < RBC; ++r)
#pragma unroll
                for (int k = 0; k < KPT; ++k) xf[r][k] = lds128(xb + (uint32_t)r * row_bytes + koff[k]);
        } else {   // the last block of a slot: rows the copy did not bring count as zeros
#pragma unroll
            for (int r = 0; r < RBC; ++r)
#pragma unroll
                for (int k = 0; k < KPT; ++k)
                    xf[r][k] = r < nr ? lds128(xb + (uint32_t)r * row_bytes + koff[k]) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int r = 0; r < RBC; ++r) {
            // two chains of multiply-adds per row
            float p0 = xf[r][0].x * wv[0].x, p1 = xf[r][0].y * wv[0].y;
            p0 = fmaf(xf[r][0].z, wv[0].z, p0); p1 = fmaf(xf[r][0].w, wv[0].w, p1);
#pragma unroll
            for (int k = 1; k < KPT; ++k) {
                p0 = fmaf(xf[r][k].x, wv[k].x, p0); p1 = fmaf(xf[r][k].y, wv[k].y, p1);
                p0 = fmaf(xf[r][k].z, wv[k].z, p0); p1 = fmaf(xf[r][k].w, wv[k].w, p1);
            }
            part[r] = p0 + p1;
        }
        float *redb = red + (blk & 1) * REDW;
        pg_warp_sums<RBC>(part, redb, warp, lane);
        // the one barrier of the block: the partial sums are visible, and everybody has read the buffer
        if (!__syncthreads_and(ok)) break;
        if (tid == 0 && issued < nblocks) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue();
        }
        // pass B from the registers: acc += r[row] * X_b[row, cols]
        float z[RBC];
        pg_block_sums<RBC>(redb, lane, z);
#pragma unroll
        for (int r = 0; r < RBC; ++r) {
            float zr = z[r];
            if (LOGISTIC) zr = 1.f / (1.f + expf(-zr));
            float rr = GENERAL ? scale * (zr - yv[r]) : zr - yv[r];
            if (r >= nr) rr = 0.f;
#pragma unroll
            for (int k = 0; k < KPT; ++k) {
                acc[k].x = fmaf(rr, xf[r][k].x, acc[k].x); acc[k].y = fmaf(rr, xf[r][k].y, acc[k].y);
                acc[k].z = fmaf(rr, xf[r][k].z, acc[k].z); acc[k].w = fmaf(rr, xf[r][k].w, acc[k].w);
            }
        }
        if (++stage == S) { stage = 0; phase ^= 1u; }
        ++done;
    }
    if (done < nblocks) {
        // a wait gave up: report it and wait (bounded) for the copies still in flight; the cluster
        // reduction below still runs so that the other CTAs of the cluster are not left waiting
        if (tid == 0) {
            flags[1] = 1;
            atomicExch(a.status, 1);
            for (int b = done; b < issued; ++b) mbar_wait(&full[b % S], (uint32_t)((b / S) & 1), &flags[0], a.wait_ns);
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < KPT; ++k) {
        const long long col = 4ll * tid + 1024ll * k;
        if (col < d) *reinterpret_cast<float4 *>(gpart + col) = acc[k];
    }
    cluster.sync();
    {
        const unsigned C = cluster.num_blocks(), rank = cluster.block_rank();
        const long long vecs = d / 4;
        const long long per = (vecs + C - 1) / C;
        for (long long v = (long long)rank * per + tid; v < min(vecs, (long long)(rank + 1) * per); v += blockDim.x) {
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
            for (unsigned c = 0; c < C; ++c) {
                const float4 x = *reinterpret_cast<const float4 *>(cluster.map_shared_rank(gpart, c) + v * 4);
                sum.x += x.x; sum.y += x.y; sum.z += x.z; sum.w += x.w;
            }
            *reinterpret_cast<float4 *>(a.G + (size_t)item * d + v * 4) = sum;
        }
    }
    cluster.sync();  // nobody leaves while its shared memory may still be read
}

// ------------------------------------------------------------------------------------------------
// Self-test of the bounded wait: what a kernel does when a copy never arrives
// ------------------------------------------------------------------------------------------------

// One thread initialises an mbarrier that expects one arrival and waits for a phase nobody completes,
// with the wait the kernels above use; when the wait gives up it reports through the status word,
// exactly as they do.  Nothing is in flight, so there is nothing to drain.
__global__ void cr_wait_selftest_kernel(int *status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ volatile int never;
    if (threadIdx.x == 0) {
        never = 0;
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait(&bar, 0, &never, limit_ns)) atomicExch(status, 1);
    }
}

// ------------------------------------------------------------------------------------------------
// host side: launch wrappers
// ------------------------------------------------------------------------------------------------

cudaError_t launch_wait_selftest(int *status, unsigned long long limit_ns, cudaStream_t stream, int64_t *launches) {
    cr_wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    const cudaError_t err = cudaGetLastError();
    if (err == cudaSuccess) ++*launches;
    return err;
}

// Most rows of blocks in a grid: launches over more items (nodes, parents, slot items) go in chunks.
constexpr int kMaxGridY = 65535;

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool tma_eligible(const AggArgs &a) {
    return a.d % 4 == 0 && a.d >= 256 && a.d < (1ll << 31) && aligned16(a.G) && aligned16(a.out) &&
           a.rows_total < (1ll << 31);
}

int inline_schedule_limit() { return kInlineSteps; }

static bool vec4_ok(const void *G, const void *out, int64_t d) { return d % 4 == 0 && aligned16(G) && aligned16(out); }

static int pick_lmax(int L) { return L <= 2 ? 2 : (L <= 4 ? 4 : 8); }

static CUresult make_map(EncodeTiledFn encode, CUtensorMap *map, const AggArgs &a, int boxw, int boxrows) {
    const cuuint64_t dims[2] = {(cuuint64_t)a.d, (cuuint64_t)a.rows_total};
    const cuuint64_t strides[1] = {(cuuint64_t)a.d * 4u};
    const cuuint32_t box[2] = {(cuuint32_t)boxw, (cuuint32_t)boxrows};
    const cuuint32_t estr[2] = {1, 1};
    return encode(map, a.is_int ? CU_TENSOR_MAP_DATA_TYPE_INT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                  const_cast<void *>(a.G), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// Largest divisor of m not above `cap`.
static int rows_per_box(int m, int cap) {
    int best = 1;
    for (int r = 1; r <= m && r <= cap; ++r)
        if (m % r == 0) best = r;
    return best;
}

template <typename T, int LMAX, int NCW>
static cudaError_t run_fused(const CUtensorMap &map, const FusedArgs &fa, int grid, size_t smem, cudaStream_t stream) {
    auto kern = cr_fused_tma_kernel<T, LMAX, NCW>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, (NCW + 1) * 32, smem, stream>>>(map, fa);
    return cudaGetLastError();
}

template <typename T, int NCW>
static cudaError_t run_fused_l(int lmax, const CUtensorMap &map, const FusedArgs &fa, int grid, size_t smem,
                               cudaStream_t stream) {
    switch (lmax) {
        case 2: return run_fused<T, 2, NCW>(map, fa, grid, smem, stream);
        case 4: return run_fused<T, 4, NCW>(map, fa, grid, smem, stream);
        default: return run_fused<T, 8, NCW>(map, fa, grid, smem, stream);
    }
}

template <typename T>
static cudaError_t run_fused_ncw(int ncw, int lmax, const CUtensorMap &map, const FusedArgs &fa, int grid, size_t smem,
                                 cudaStream_t stream) {
    switch (ncw) {
        case 2: return run_fused_l<T, 2>(lmax, map, fa, grid, smem, stream);
        case 4: return run_fused_l<T, 4>(lmax, map, fa, grid, smem, stream);
        default: return run_fused_l<T, 8>(lmax, map, fa, grid, smem, stream);
    }
}

// CTAs of one instantiation that fit an SM together with `smem` bytes of dynamic shared memory each
// (0 if the query fails).
template <typename T, int LMAX, int NCW>
static int fused_resident(size_t smem) {
    auto kern = cr_fused_tma_kernel<T, LMAX, NCW>;
    int blocks = 0;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks, kern, (NCW + 1) * 32, smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return blocks;
}

template <typename T, int NCW>
static int fused_resident_l(int lmax, size_t smem) {
    switch (lmax) {
        case 2: return fused_resident<T, 2, NCW>(smem);
        case 4: return fused_resident<T, 4, NCW>(smem);
        default: return fused_resident<T, 8, NCW>(smem);
    }
}

static int fused_resident_any(bool is_int, int ncw, int lmax, size_t smem) {
    // the answer depends on the instantiation and the shared-memory size only: remembered per process
    static std::mutex mu;
    static std::map<std::tuple<bool, int, int, size_t>, int> seen;
    const auto key = std::make_tuple(is_int, ncw, lmax, smem);
    {
        std::lock_guard<std::mutex> lock(mu);
        auto it = seen.find(key);
        if (it != seen.end()) return it->second;
    }
    int blocks = 0;
    switch (ncw) {
        case 2: blocks = is_int ? fused_resident_l<int, 2>(lmax, smem) : fused_resident_l<float, 2>(lmax, smem); break;
        case 4: blocks = is_int ? fused_resident_l<int, 4>(lmax, smem) : fused_resident_l<float, 4>(lmax, smem); break;
        default: blocks = is_int ? fused_resident_l<int, 8>(lmax, smem) : fused_resident_l<float, 8>(lmax, smem); break;
    }
    std::lock_guard<std::mutex> lock(mu);
    seen[key] = blocks;
    return blocks;
}

cudaError_t launch_fused_tma(const AggArgs &a, const DeviceInfo &dev, const Tuning &tune, EncodeTiledFn encode,
                             cudaStream_t stream, int64_t *launches, bool *done) {
    *done = false;
    if (!encode || !tma_eligible(a) || a.batch != 1) return cudaSuccess;
    // Short vectors give few column tiles: halve the tile so that more CTAs take part.
    int ncw = tune.ncw ? tune.ncw : ((a.d + 511) / 512 < 3ll * dev.sm_count ? 2 : 4);
    if (ncw != 2 && ncw != 4 && ncw != 8) ncw = 4;
    const int tile = ncw * 128;
    const int boxw = tile < 256 ? tile : 256;
    // Launch shape.  Measured on B200 (d = 2^24, m = 9): throughput peaks with about 100 KB of loads
    // in flight per SM and falls off on both sides (too little: latency-bound; too much: the DRAM
    // pages of too many slot rows are open at once), and several small CTAs per SM beat one large
    // one.  So: boxes of at most ~18 KB (R = a divisor of m), three CTAs per SM, and as many stages
    // as bring the total to ~36 KB per CTA, at least two.
    const int cap = std::min(kMaxBoxRows, std::max(1, (18 * 1024) / (tile * 4)));
    int R = tune.rows && a.m % tune.rows == 0 && tune.rows <= kMaxBoxRows ? tune.rows : rows_per_box(a.m, cap);
    // A box holds a divisor of m rows.  When m has no divisor under the soft cap but one row (m = 11 or 13 with
    // 512-column tiles), a box of one row is 2 KB and the copy engine, not HBM, sets the pace (1.9 TB/s
    // measured): take the taller box if there is one, and leave nodes that only split into thin boxes to the
    // plain-load kernel.
    if (!tune.rows && R < 4 && a.m > R) {
        R = rows_per_box(a.m, kMaxBoxRows);
        if (R < 4) return cudaSuccess;
    }
    const size_t stage_bytes = (size_t)R * tile * 4;
    // a schedule too long for the kernel parameters rides in shared memory when it is short enough for that
    const bool inline_ok = a.host_steps && a.total_steps <= kInlineSteps;
    const size_t steps_bytes = (!inline_ok && a.total_steps <= kSmemSteps) ? (size_t)a.total_steps * sizeof(Step) + 16 : 0;
    int ctas = tune.ctas_per_sm ? tune.ctas_per_sm : 3;
    int stages = tune.stages ? tune.stages
                             : std::max(2, std::min(8, (int)((36 * 1024 + stage_bytes / 2) / stage_bytes)));
    // With fewer tiles than resident CTAs the launch is bound by the latency of each box, not by HBM:
    // deepen every CTA's ring so that about as many boxes are in flight as a full grid would have.
    const long long tiles_now = (a.d + tile - 1) / tile;
    if (!tune.stages && tiles_now < (long long)dev.sm_count * ctas)
        stages = (int)std::min<long long>(8, std::max<long long>(stages, ((long long)dev.sm_count * ctas * stages + tiles_now - 1) / tiles_now));
    // With only a few tiles per CTA the last pass over the tiles is partly empty (d = 120000, 256-column
    // tiles: 469 tiles on 444 CTAs, 26.7 us; on four CTAs per SM, one tile each, 22.4 us.  m = 9, d = 2^19:
    // 1024 tiles on 444 CTAs 41.9 us, on 592 CTAs 39.5 us).  Of the CTA counts per SM that fit the
    // registers and shared memory, take the one whose last pass is fullest, and thin every ring so that
    // the bytes in flight per SM stay about the same.
    if (!tune.ctas_per_sm && tiles_now > (long long)dev.sm_count * ctas && tiles_now < (long long)dev.sm_count * ctas * 6) {
        auto fill = [&](int c) {   // share of the CTA-passes that carry a tile
            const double x = (double)tiles_now / ((double)dev.sm_count * c);
            return x <= 1.0 ? 1.0 : x / std::ceil(x);
        };
        int best = ctas, best_stages = stages;
        double best_fill = fill(ctas);
        for (int c = ctas + 1; c <= 6; ++c) {
            const int thin = tune.stages ? stages : std::max(2, stages * ctas / c);
            if (fused_resident_any(a.is_int, ncw, pick_lmax(a.L), (size_t)thin * stage_bytes + (size_t)thin * 16 + 32 + steps_bytes) < c) break;
            if (fill(c) > best_fill + 0.03) { best = c; best_stages = thin; best_fill = fill(c); }
            if ((long long)dev.sm_count * c >= tiles_now) break;
        }
        ctas = best;
        stages = best_stages;
    }
    const size_t usable = (size_t)dev.smem_per_sm - 2048;  // leave room for the per-CTA reserve
    while (ctas > 1 && ((size_t)stages * stage_bytes + steps_bytes + 1024 + 256) * ctas > usable) --ctas;
    while (stages > 2 && (size_t)stages * stage_bytes + steps_bytes + 256 > (size_t)dev.smem_optin) --stages;
    const size_t smem = (size_t)stages * stage_bytes + (size_t)stages * 16 + 32 + steps_bytes;
    if (smem > (size_t)dev.smem_optin) return cudaSuccess;  // does not fit: caller falls back to plain loads

    CUtensorMap map;
    if (make_map(encode, &map, a, boxw, R) != CUDA_SUCCESS) return cudaSuccess;

    FusedArgs fa;
    fa.n_inline = 0;
    fa.steps_smem = steps_bytes ? 1 : 0;
    if (inline_ok) {
        fa.n_inline = a.total_steps;
        for (int k = 0; k < a.total_steps; ++k) fa.steps_inline[k] = a.host_steps[k];
    } else if (!a.steps) {
        return cudaSuccess;  // no staged schedule and too long to inline: caller stages it and retries
    }
    fa.coeff = a.coeff; fa.steps = a.steps; fa.n_steps = a.total_steps; fa.m = a.m; fa.R = R; fa.cpn = a.m / R;
    fa.stages = stages; fa.d = a.d; fa.ntiles = (a.d + tile - 1) / tile; fa.out = a.out; fa.shift = a.shift;
    fa.status = a.status; fa.wait_ns = tune.wait_limit_ns;
    const long long max_grid = (long long)dev.sm_count * ctas;
    const int grid = (int)std::min<long long>(fa.ntiles, max_grid);
    cudaError_t err = a.is_int ? run_fused_ncw<int>(ncw, pick_lmax(a.L), map, fa, grid, smem, stream)
                               : run_fused_ncw<float>(ncw, pick_lmax(a.L), map, fa, grid, smem, stream);
    if (err == cudaSuccess) { *done = true; ++*launches; }
    return err;
}

template <typename T, int LMAX, int NLW, int NRW, bool SHARE>
static cudaError_t run_batch(const CUtensorMap &map, const BatchArgs &ba, int grid, size_t smem, cudaStream_t stream) {
    auto kern = cr_fused_batch_tma_kernel<T, LMAX, NLW, NRW, SHARE>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, (NLW + NRW) * 32, smem, stream>>>(map, ba);
    return cudaGetLastError();
}

template <typename T, int NLW, int NRW, bool SHARE>
static cudaError_t run_batch_l(int lmax, const CUtensorMap &map, const BatchArgs &ba, int grid, size_t smem,
                               cudaStream_t stream) {
    switch (lmax) {
        case 2: return run_batch<T, 2, NLW, NRW, SHARE>(map, ba, grid, smem, stream);
        case 4: return run_batch<T, 4, NLW, NRW, SHARE>(map, ba, grid, smem, stream);
        default: return run_batch<T, 8, NLW, NRW, SHARE>(map, ba, grid, smem, stream);
    }
}

template <typename T>
static cudaError_t run_batch_w(int nlw, int nrw, int lmax, const CUtensorMap &map, const BatchArgs &ba, int grid,
                               size_t smem, cudaStream_t stream) {
    if (ba.n_ops)   // shared messages: eight replay warps, or four in the two-CTAs-per-SM form
        return nlw == 6 ? run_batch_l<T, 6, 8, true>(lmax, map, ba, grid, smem, stream)
                        : (nrw == 4 ? run_batch_l<T, 4, 4, true>(lmax, map, ba, grid, smem, stream)
                                    : run_batch_l<T, 4, 8, true>(lmax, map, ba, grid, smem, stream));
    if (nlw == 6) return nrw == 4 ? run_batch_l<T, 6, 4, false>(lmax, map, ba, grid, smem, stream)
                                  : run_batch_l<T, 6, 8, false>(lmax, map, ba, grid, smem, stream);
    return nrw == 4 ? run_batch_l<T, 4, 4, false>(lmax, map, ba, grid, smem, stream)
                    : run_batch_l<T, 4, 8, false>(lmax, map, ba, grid, smem, stream);
}

BatchShape batch_shape(const AggArgs &a, const DeviceInfo &dev, const Tuning &tune) {
    BatchShape sh;
    const int tile = 128;
    sh.nrw = (tune.ncw == 4 && !a.n_ops) ? 4 : 8;  // replay warps
    // same-shape batches stage their schedules in shared memory (layer word per step, one 4-byte entry
    // per step and pattern, patterns padded to the replay group size, the weight table) when small
    const int lmax = pick_lmax(a.L);
    const int np = lmax <= 4 ? 4 : 2;
    const int nst = a.same_shape && a.batch > 0 ? a.total_steps / a.batch : 0;
    size_t sched_bytes = 0;
    if (a.same_shape && nst > 0 && a.n_wtab > 0) {
        const size_t want = (((size_t)nst * 4 + 15) & ~(size_t)15) +
                            (((size_t)nst * ((a.batch + np - 1) / np * np) + 3) & ~(size_t)3) * 4 +
                            (((size_t)a.n_wtab * 4 + 15) & ~(size_t)15) + (size_t)a.n_ops * 16;
        if (want <= 24 * 1024) sched_bytes = (want + 15) & ~(size_t)15;
    }
    const int n_rows = a.n_ops ? a.n_rows : a.n_union;
    const size_t e_one = (size_t)n_rows * tile * 4;
    const size_t budget = (size_t)dev.smem_optin - 512;   // barriers and flags take the rest
    // Shared memory = nbuf x E + staged schedules + one private ring of `stages` boxes of R rows per loader warp.  Measured on B200 (d = 2^22, m = 16, 120 nodes, 64 patterns): six
    // loaders with two boxes of 8 KB each stream at the copy bandwidth; four loaders reach 90 % of it, boxes
    // of 4 KB two thirds, a third box per loader adds nothing.  So: boxes as tall as fit come first, then the
    // second E buffer, then six loaders rather than four.
    int nbuf = 0, stages = 0, R = 0, nlw = 0;
    const int want_loaders = tune.ctas_per_sm == 4 ? 4 : 6;
    // Few slot rows per node (m <= 8, coded gradients): a box of one node would be 0.5-4 KB, too small for
    // the copy engine.  Then a box takes the rows of npb consecutive union nodes; the selection below sees
    // such a box as one tall node, and falls back to one node per box if tall boxes do not fit beside E.
    bool multi = a.npb > 1 && a.n_boxes > 0 && a.npb * a.m <= kMaxBoxRows && !tune.rows;
    for (int attempt = 0; attempt < 2 && !nbuf; ++attempt) {
        if (attempt == 1) {
            if (!multi) break;
            multi = false;
        }
        const int node_rows = multi ? a.npb * a.m : a.m;
        for (int try_buf = tune.e_buffers == 1 ? 1 : 2; try_buf >= 1 && !nbuf; --try_buf) {
            if (budget <= try_buf * e_one + sched_bytes) continue;
            const size_t ring_budget = budget - try_buf * e_one - sched_bytes;
            const int want_stages = tune.stages ? tune.stages : 2;
            int best_r = 0, best_depth = 0, best_lw = 0;
            for (int lw = want_loaders; lw >= 4; lw -= 2) {
                for (int depth = want_stages; depth >= 2; --depth) {
                    const size_t per_row = (size_t)lw * depth * tile * 4, fixed = (size_t)lw * depth * 8;
                    if (ring_budget <= fixed) continue;
                    const int cap = (int)std::min<size_t>(kMaxBoxRows, (ring_budget - fixed) / per_row);
                    if (cap < 1) continue;
                    const int r = multi ? (node_rows <= cap ? node_rows : 0)
                                        : (tune.rows && a.m % tune.rows == 0 && tune.rows <= cap ? tune.rows : rows_per_box(a.m, cap));
                    if (r > best_r) { best_r = r; best_depth = depth; best_lw = lw; }
                }
            }
            // two buffers only if they do not cost more than half of the box height one buffer allows
            if (best_r && (try_buf == 1 || 2 * best_r >= std::min(node_rows, kMaxBoxRows))) {
                nbuf = try_buf; R = best_r; stages = best_depth; nlw = best_lw;
            }
        }
    }
    if (!nbuf) return sh;  // union too large for shared memory
    const size_t stage_bytes = (size_t)R * tile * 4;
    size_t smem = (size_t)nlw * stages * (stage_bytes + 8) + nbuf * e_one + sched_bytes + 64 + 16;
    if (smem > (size_t)dev.smem_optin) return sh;
    // the variant records of the shared messages ride in shared memory too when the rest leaves room
    const size_t vtab_bytes = ((size_t)a.vtab_words * 4 + 15) & ~(size_t)15;   // what follows stays 16-byte aligned
    if (a.n_ops && sched_bytes && smem + vtab_bytes <= (size_t)dev.smem_optin) {
        sh.vtab_smem = 1;
        sched_bytes += vtab_bytes;
        smem += vtab_bytes;
    }
    const long long ntiles = (a.d + tile - 1) / tile;
    int grid = (int)std::min<long long>(ntiles, (long long)std::max(1, dev.sm_count));
    // Small unions: with four loaders and four replay warps two CTAs fit an SM (shared memory and registers),
    // and a CTA's tile -- a handful of boxes, then the replay, each a chain of waits -- overlaps the other's.
    // Measured, 16 patterns on the (4,2,1) tree at d = 2^20: one CTA of 14 warps per SM 0.138 ms.
    if (!tune.ncw && !tune.ctas_per_sm && nbuf == 2) {
        const size_t smem4 = smem - (size_t)(nlw - 4) * stages * (stage_bytes + 8);
        if (smem4 + 1024 <= (size_t)dev.smem_per_sm / 2 && ntiles >= 4ll * dev.sm_count) {
            nlw = 4; sh.nrw = 4; smem = smem4;
            grid = (int)std::min<long long>(ntiles, 2ll * dev.sm_count);
        }
    }
    sh.cpn = multi ? 1 : a.m / R;
    sh.n_groups = multi ? a.n_boxes : a.n_union;
    // box counters are 32-bit
    if ((ntiles / grid + 1) * (long long)sh.n_groups * sh.cpn >= (1ll << 31)) return sh;
    sh.nbuf = nbuf; sh.stages = stages; sh.R = R; sh.nlw = nlw; sh.multi = multi ? 1 : 0; sh.nst = nst;
    sh.sched_bytes = sched_bytes; sh.smem = smem; sh.n_rows = n_rows; sh.grid = grid;
    sh.ok = true;
    return sh;
}

int unit_words() { return kUnitWords; }

cudaError_t launch_fused_batch_tma(const AggArgs &a, const BatchShape &sh, const Tuning &tune, EncodeTiledFn encode,
                                   cudaStream_t stream, int64_t *launches, bool *done) {
    *done = false;
    if (!encode || !sh.ok || !a.units || !tma_eligible(a)) return cudaSuccess;
    const int tile = 128;
    CUtensorMap map;
    if (make_map(encode, &map, a, tile, sh.R) != CUDA_SUCCESS) return cudaSuccess;

    BatchArgs ba;
    ba.coeff = a.coeff; ba.steps = a.steps; ba.pat_off = a.pat_off; ba.unodes = a.unodes; ba.n_union = a.n_union;
    ba.batch = a.batch; ba.same_shape = a.same_shape; ba.m = a.m; ba.R = sh.R; ba.cpn = sh.cpn; ba.stages = sh.stages;
    ba.d = a.d; ba.ntiles = (a.d + tile - 1) / tile; ba.out = a.out; ba.shift = a.shift; ba.status = a.status;
    ba.sched_smem = (int)sh.sched_bytes; ba.nst = sh.nst; ba.nbuf = sh.nbuf; ba.wtab = a.wtab; ba.n_wtab = a.n_wtab;
    ba.units = a.units; ba.n_groups = sh.n_groups;
    ba.wait_ns = tune.wait_limit_ns;
    ba.n_rows = sh.n_rows; ba.n_ops = a.n_ops; ba.ops = a.ops; ba.vtab = a.vtab; ba.vtab_words = a.vtab_words;
    ba.vtab_smem = sh.vtab_smem;
    ba.flat = (a.n_ops && a.L == 1 && sh.sched_bytes) ? 1 : 0;   // a.L: depth of the (reduced) schedules
    const int lmax = pick_lmax(a.L);
    const cudaError_t err = a.is_int ? run_batch_w<int>(sh.nlw, sh.nrw, lmax, map, ba, sh.grid, sh.smem, stream)
                                     : run_batch_w<float>(sh.nlw, sh.nrw, lmax, map, ba, sh.grid, sh.smem, stream);
    if (err == cudaSuccess) { *done = true; ++*launches; }
    return err;
}

template <typename T, int V>
static cudaError_t run_ldg_main(const AggArgs &a, dim3 grid, T *out, int shift, const InlineSchedule &inl, cudaStream_t stream) {
    const T *G = reinterpret_cast<const T *>(a.G);
    const T *cf = reinterpret_cast<const T *>(a.coeff);
    if (a.m % 4 == 0 && V == 4) {
        switch (pick_lmax(a.L)) {
            case 2: cr_fused_ldg_kernel<T, 2, V, 4><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl); break;
            case 4: cr_fused_ldg_kernel<T, 4, V, 4><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl); break;
            default: cr_fused_ldg_kernel<T, 8, V, 4><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl); break;
        }
        return cudaGetLastError();
    }
    if (a.m == 1 && V == 4) {
        switch (pick_lmax(a.L)) {
            case 2: cr_fused_ldg_kernel<T, 2, V, 1><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl); break;
            case 4: cr_fused_ldg_kernel<T, 4, V, 1><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl); break;
            default: cr_fused_ldg_kernel<T, 8, V, 1><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl); break;
        }
        return cudaGetLastError();
    }
    if (a.m < 4 && V == 4 && pick_lmax(a.L) == 2) {
        cr_fused_ldg_kernel<T, 2, V, 5><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl);
        return cudaGetLastError();
    }
    switch (pick_lmax(a.L)) {
        case 2: cr_fused_ldg_kernel<T, 2, V, 0><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl); break;
        case 4: cr_fused_ldg_kernel<T, 4, V, 0><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl); break;
        default: cr_fused_ldg_kernel<T, 8, V, 0><<<grid, 256, 0, stream>>>(G, cf, a.steps, a.pat_off, a.m, a.d, out, shift, inl); break;
    }
    return cudaGetLastError();
}


template <typename T, int V>
static cudaError_t run_ldg(const AggArgs &a, cudaStream_t stream, int64_t *launches) {
    const long long threads = (a.d + V - 1) / V;
    dim3 grid((unsigned)((threads + 255) / 256), (unsigned)a.batch);
    T *out = reinterpret_cast<T *>(a.out);
    InlineSchedule inl;
    inl.n = 0; inl.nseg = 0;
    int shift = a.shift;
    if (!a.steps) {   // single short pattern, not staged: the schedule rides in the parameters
        if (!a.host_steps || a.batch != 1 || a.total_steps > kInlineSteps) return cudaErrorInvalidValue;
        inl.n = a.total_steps;
        for (int k = 0; k < a.total_steps; ++k) inl.steps[k] = a.host_steps[k];
        if (a.split_scratch) {
            // post-order: the entries of a layer-1 sub-tree are contiguous and end with its root
            inl.seg_off[0] = 0;
            for (int k = 0; k < a.total_steps; ++k)
                if ((a.host_steps[k].layer & 0xff) == 1) {
                    if (inl.nseg == kMaxSplit) return cudaErrorInvalidValue;
                    inl.seg_off[++inl.nseg] = k + 1;
                }
            if (inl.nseg == 0 || inl.seg_off[inl.nseg] != a.total_steps) return cudaErrorInvalidValue;
            grid.y = (unsigned)inl.nseg;
            out = reinterpret_cast<T *>(a.split_scratch);
            shift = 0;   // applied once, by the kernel that adds the rows
        }
    }
    cudaError_t err = run_ldg_main<T, V>(a, grid, out, shift, inl, stream);
    if (err != cudaSuccess) return err;
    ++*launches;
    if (inl.nseg) {
        // a programmatic dependent launch: the set-up of this small grid overlaps the run of the first one
        // (two back-to-back launches cost a few microseconds between them, a fifth of these short calls)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)((a.d + 255) / 256), 1, 1);
        cfg.blockDim = dim3(256, 1, 1);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        err = cudaLaunchKernelEx(&cfg, cr_sum_rows_kernel<T>, reinterpret_cast<const T *>(a.split_scratch), inl.nseg,
                                 (long long)a.d, reinterpret_cast<T *>(a.out), a.shift);
        if (err == cudaSuccess) ++*launches;
    }
    return err;
}

cudaError_t launch_fused_ldg(const AggArgs &a, cudaStream_t stream, int64_t *launches) {
    const bool v4 = vec4_ok(a.G, a.out, a.d) && (!a.split_scratch || aligned16(a.split_scratch));
    if (a.is_int) return v4 ? run_ldg<int, 4>(a, stream, launches) : run_ldg<int, 1>(a, stream, launches);
    return v4 ? run_ldg<float, 4>(a, stream, launches) : run_ldg<float, 1>(a, stream, launches);
}

int split_limit() { return kMaxSplit; }

template <typename T, int V>
static cudaError_t run_uncoded(const AggArgs &a, cudaStream_t stream) {
    const long long threads = (a.d + V - 1) / V;
    dim3 grid((unsigned)((threads + 255) / 256), (unsigned)a.batch);
    cr_uncoded_sum_kernel<T, V><<<grid, 256, 0, stream>>>(reinterpret_cast<const T *>(a.G), a.steps, a.pat_off, a.m,
                                                          a.d, reinterpret_cast<T *>(a.out));
    return cudaGetLastError();
}

cudaError_t launch_uncoded_sum(const AggArgs &a, cudaStream_t stream, int64_t *launches) {
    const bool v4 = vec4_ok(a.G, a.out, a.d);
    cudaError_t err;
    if (a.is_int) err = v4 ? run_uncoded<int, 4>(a, stream) : run_uncoded<int, 1>(a, stream);
    else err = v4 ? run_uncoded<float, 4>(a, stream) : run_uncoded<float, 1>(a, stream);
    if (err == cudaSuccess) ++*launches;
    return err;
}

template <typename T, int V>
static cudaError_t run_encode(const void *G, const void *coeff, const int32_t *nodes, int count, int m, int64_t d,
                              void *E, cudaStream_t stream) {
    const long long threads = (d + V - 1) / V;
    for (int y0 = 0; y0 < count; y0 += kMaxGridY) {
        dim3 grid((unsigned)((threads + 255) / 256), (unsigned)std::min(kMaxGridY, count - y0));
        cr_encode_kernel<T, V><<<grid, 256, 0, stream>>>(reinterpret_cast<const T *>(G), reinterpret_cast<const T *>(coeff),
                                                         nodes, y0, m, d, reinterpret_cast<T *>(E));
        const cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    return cudaSuccess;
}

cudaError_t launch_encode(const void *G, const void *coeff, const int32_t *nodes, int count, int m, int64_t d,
                          void *E, int is_int, cudaStream_t stream, int64_t *launches) {
    if (count <= 0) return cudaSuccess;
    const bool v4 = vec4_ok(G, E, d);
    cudaError_t err;
    if (is_int) err = v4 ? run_encode<int, 4>(G, coeff, nodes, count, m, d, E, stream)
                         : run_encode<int, 1>(G, coeff, nodes, count, m, d, E, stream);
    else err = v4 ? run_encode<float, 4>(G, coeff, nodes, count, m, d, E, stream)
                  : run_encode<float, 1>(G, coeff, nodes, count, m, d, E, stream);
    if (err == cudaSuccess) ++*launches;
    return err;
}

template <typename T, int V>
static cudaError_t run_decode(const void *M_child, const void *E_parent, const void *W, const int32_t *active,
                              int parents, int n, int64_t d, void *M_parent, int shift, cudaStream_t stream) {
    const long long threads = (d + V - 1) / V;
    for (int y0 = 0; y0 < parents; y0 += kMaxGridY) {
        dim3 grid((unsigned)((threads + 255) / 256), (unsigned)std::min(kMaxGridY, parents - y0));
        cr_decode_kernel<T, V><<<grid, 256, 0, stream>>>(reinterpret_cast<const T *>(M_child),
                                                         reinterpret_cast<const T *>(E_parent),
                                                         reinterpret_cast<const T *>(W), active, y0, n, d,
                                                         reinterpret_cast<T *>(M_parent), shift);
        const cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    return cudaSuccess;
}

cudaError_t launch_decode(const void *M_child, const void *E_parent, const void *W, const int32_t *active,
                          int parents, int n, int64_t d, void *M_parent, int shift, int is_int,
                          cudaStream_t stream, int64_t *launches) {
    const bool v4 = d % 4 == 0 && aligned16(M_child) && aligned16(M_parent) && (!E_parent || aligned16(E_parent));
    cudaError_t err;
    if (is_int) err = v4 ? run_decode<int, 4>(M_child, E_parent, W, active, parents, n, d, M_parent, shift, stream)
                         : run_decode<int, 1>(M_child, E_parent, W, active, parents, n, d, M_parent, shift, stream);
    else err = v4 ? run_decode<float, 4>(M_child, E_parent, W, active, parents, n, d, M_parent, shift, stream)
                  : run_decode<float, 1>(M_child, E_parent, W, active, parents, n, d, M_parent, shift, stream);
    if (err == cudaSuccess) ++*launches;
    return err;
}

cudaError_t launch_partial_gradients_two_pass(const float *X, const float *y, const float *w, const int32_t *part,
                                              const int32_t *order, int items, int rows, int64_t d, float *resid,
                                              float *G, int loss, int sm_count, cudaStream_t stream, int64_t *launches) {
    const bool v4 = d % 4 == 0 && aligned16(X) && aligned16(w) && aligned16(G);
    const long long total_rows = (long long)items * rows;
    const long long want_blocks = (total_rows + 7) / 8;  // 8 warps per block
    const int blocks = (int)std::min<long long>(want_blocks, (long long)std::max(1, sm_count) * 32);
    if (v4) cr_residual_kernel<4><<<blocks, 256, 0, stream>>>(X, y, w, part, order, total_rows, rows, d, resid, loss);
    else cr_residual_kernel<1><<<blocks, 256, 0, stream>>>(X, y, w, part, order, total_rows, rows, d, resid, loss);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    ++*launches;
    for (int y0 = 0; y0 < items && err == cudaSuccess; y0 += kMaxGridY) {
        const unsigned gy = (unsigned)std::min(kMaxGridY, items - y0);
        if (v4) {
            dim3 grid((unsigned)((d / 4 + 127) / 128), gy);
            cr_xt_r_kernel<4><<<grid, 128, 0, stream>>>(X, part, order, resid, y0, rows, d, G);
        } else {
            dim3 grid((unsigned)((d + 127) / 128), gy);
            cr_xt_r_kernel<1><<<grid, 128, 0, stream>>>(X, part, order, resid, y0, rows, d, G);
        }
        err = cudaGetLastError();
        if (err == cudaSuccess) ++*launches;
    }
    return err;
}

template <int KPT>
static cudaError_t run_partial_fused(const PgArgs &pa, int csplit, bool fit_one_wave, int items, size_t smem,
                                     cudaStream_t stream) {
    const bool general = pa.slots_per_item != 1 || pa.coeff != nullptr;
    auto kern = general ? (pa.loss == 1 ? cr_partial_fused_kernel<KPT, true, true> : cr_partial_fused_kernel<KPT, true, false>)
                        : (pa.loss == 1 ? cr_partial_fused_kernel<KPT, false, true> : cr_partial_fused_kernel<KPT, false, false>);
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    if (csplit > 8) {
        err = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (err != cudaSuccess) return err;
    }
    if (fit_one_wave && csplit == 16) {
        // Few items, each a cluster of 16: if the GPU cannot hold all of them at once the stragglers
        // of a second wave double the run time.  Take the largest cluster size (16 .. 9) of which
        // `items` clusters are resident together; the answer is remembered per shape.
        static std::mutex mu;
        static std::map<std::tuple<const void *, size_t, int>, int> memo;
        const auto key = std::make_tuple(reinterpret_cast<const void *>(kern), smem, items);
        std::lock_guard<std::mutex> lock(mu);
        auto it = memo.find(key);
        if (it == memo.end()) {
            int best = 16;
            for (int c = 16; c >= 9; --c) {
                cudaLaunchConfig_t q = {};
                q.gridDim = dim3((unsigned)c, (unsigned)items, 1);
                q.blockDim = dim3(256, 1, 1);
                q.dynamicSmemBytes = smem;
                cudaLaunchAttribute qa[1];
                qa[0].id = cudaLaunchAttributeClusterDimension;
                qa[0].val.clusterDim.x = (unsigned)c; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
                q.attrs = qa; q.numAttrs = 1;
                int resident = 0;
                if (cudaOccupancyMaxActiveClusters(&resident, kern, &q) != cudaSuccess) { (void)cudaGetLastError(); break; }
                if (resident >= items) { best = c; break; }
            }
            it = memo.emplace(key, best).first;
        }
        csplit = it->second;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)csplit, (unsigned)items, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)csplit;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, pa);
}

bool partial_fused_eligible(const float *X, const float *w, const float *G, int64_t d, int items) {
    return d % 4 == 0 && d <= 8192 && aligned16(X) && aligned16(w) && aligned16(G) && items <= 65535;
}

cudaError_t launch_partial_gradients_fused(const float *X, const float *y, const float *w, const int32_t *part,
                                           const int32_t *order, const float *coeff, int items, int slots_per_item,
                                           int rows, int64_t d,
                                           float *G, int loss, int *status, const DeviceInfo &dev,
                                           const Tuning &tune, cudaStream_t stream, int64_t *launches) {
    // Measured on B200 (d = 4096, rows = 2048): two CTAs per SM hide each other's reduction latency
    // (one CTA per SM with four buffers: 3.1 TB/s), and with two buffers per CTA the largest row block
    // that still lets two CTAs share an SM is best (32 KB: 6.2 TB/s, 48 KB: 6.7 TB/s; 64 KB, which
    // leaves one CTA per SM: 4.5 TB/s).
    const size_t per_cta = (size_t)dev.smem_per_sm / 2 - 1024;
    const int stages = tune.pg_stages ? tune.pg_stages : 2;
    int64_t rb = tune.pg_block_kb ? ((int64_t)tune.pg_block_kb * 1024) / (d * 4)
                                  : ((int64_t)per_cta - d * 4 - 512) / ((int64_t)stages * d * 4);
    // ... and no more rows than a thread keeps in registers
    const int kpt = d <= 1024 ? 1 : (d <= 2048 ? 2 : (d <= 4096 ? 4 : (int)((d + 1023) / 1024)));   // as the instances below
    const int rbc = pg_block_rows(kpt);
    const int RB = (int)std::max<int64_t>(1, std::min<int64_t>(rbc, rb));
    // the row blocks of one item are split over a cluster of up to 8 CTAs, each with at least 4 blocks
    const int item_blocks = slots_per_item * ((rows + RB - 1) / RB);
    int csplit = 1;
    while (csplit < 8 && item_blocks / (csplit * 2) >= 4) csplit *= 2;
    // ... and no wider than it takes to give the GPU about four waves of CTAs: with many small items a wide
    // cluster only adds reduction traffic and start-up cost (624 items of 39 x 5004: cluster of 4 114 us,
    // of 2 98 us, of 1 105 us; 64 rows: 154 / 142 / 154; 160 items of 2048 x 4096 keep 8)
    if (!tune.pg_cluster) {
        int cap = 1;
        while (cap < 8 && (long long)items * cap < 8ll * dev.sm_count) cap *= 2;
        csplit = std::min(csplit, cap);
    }
    // few items (coded gradients of a small tree): a cluster of 16 fills more of the GPU
    if (csplit == 8 && items * 8 < 2 * dev.sm_count && item_blocks / 16 >= 4) csplit = 16;
    if (tune.pg_cluster) csplit = tune.pg_cluster;
    const size_t smem = (size_t)stages * RB * d * 4 + (size_t)d * 4 + (size_t)2 * pg_red_words(kpt) * 4 + (size_t)stages * 8 + 16;
    if (smem > (size_t)dev.smem_optin) return cudaErrorInvalidConfiguration;
    PgArgs pa;
    pa.X = X; pa.y = y; pa.w = w; pa.part = part; pa.order = slots_per_item == 1 ? order : nullptr; pa.coeff = coeff; pa.G = G; pa.rows = rows;
    pa.slots_per_item = slots_per_item; pa.loss = loss; pa.RB = RB; pa.stages = stages; pa.d = d; pa.status = status;
    pa.wait_ns = tune.wait_limit_ns;
    cudaError_t err;
    const bool fit = !tune.pg_cluster;
    if (d <= 1024) err = run_partial_fused<1>(pa, csplit, fit, items, smem, stream);
    else if (d <= 2048) err = run_partial_fused<2>(pa, csplit, fit, items, smem, stream);
    else if (d <= 4096) err = run_partial_fused<4>(pa, csplit, fit, items, smem, stream);
    // between 4096 and 8192 in steps of 1024 columns: a thread's column groups beyond d are predicated off
    // but still issue, and the model sizes of the paper's regressions (p = 5001, 6500) lie here
    else if (d <= 5120) err = run_partial_fused<5>(pa, csplit, fit, items, smem, stream);
    else if (d <= 6144) err = run_partial_fused<6>(pa, csplit, fit, items, smem, stream);
    else if (d <= 7168) err = run_partial_fused<7>(pa, csplit, fit, items, smem, stream);
    else err = run_partial_fused<8>(pa, csplit, fit, items, smem, stream);
    if (err == cudaSuccess) ++*launches;
    return err;
}

}  // namespace cr
