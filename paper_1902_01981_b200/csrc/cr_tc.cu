// Partial gradients for SEVERAL models at once on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// With K models (a line search, an ensemble, several step sizes) the partial gradient of a partition
// becomes two dense contractions, R = X_p W^T - y 1^T (rows x K) and G = X_p^T R (d x K): 2K flops per
// byte of X each, enough to leave the HBM roofline of the single-model kernels, so this is the one
// place on the path where tensor cores apply.  Two kernels, both streaming X through TMA into
// 128-byte-swizzled shared memory and issuing tcgen05.mma (kind::tf32, M = 128, N = 32) from one
// thread with the accumulator in tensor memory:
//   cr_tc_residual_kernel : CTA = (slot item, tile of 128 rows); contraction over d.
//   cr_tc_gradient_kernel : CTA = (slot item, tile of 128 columns); contraction over the rows; the same
//                           X tile now acts as an MN-major operand (its transpose is never formed).
// Precision: X enters the tensor core as TF32 (the low 13 mantissa bits of each fp32 are ignored), so
// exact results need X whose values are TF32-representable; the small operands (W, R) are split into a
// TF32 head and a TF32 tail and both parts are multiplied, which keeps them at fp32 accuracy.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstdio>

#include "cr_kernels.hpp"

namespace cr {

namespace tc {

constexpr int kModels = 32;       // N of every MMA: models are padded to 32
constexpr int kTileM = 128;       // rows (residual kernel) or columns (gradient kernel) per CTA
constexpr int kBoxCols = 32;      // 32 fp32 = 128 bytes: one swizzle row
// The tensor core adds into its fp32 accumulator with truncation, an error that grows with the number
// of additions into one accumulator (about 1.5e-8 of the sum per addition, measured).  The head
// products are therefore spread round-robin over kHeadAccs accumulators and the (2^-11 times smaller)
// tail products go to one more; the epilogue adds the kAccs partial sums in registers.
constexpr int kHeadAccs = 7;
constexpr int kAccs = kHeadAccs + 1;
constexpr uint32_t kTmemCols = kAccs * kModels;   // 256 columns: two CTAs fit one SM's tensor memory

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
// Bounded wait (`limit_ns`, a kernel argument: two seconds by default): false when it gave up or when
// *abort_flag is set.
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

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int x, int y, int z, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}

// ---- tensor memory and tcgen05 -------------------------------------------------------------------

// One warp allocates `cols` (a power of two >= 32) columns of tensor memory; the base address lands in
// shared memory.  The same warp frees them.
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], one thread issues.  `accumulate` = 0 overwrites D.
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)   // no output lane disabled
        : "memory");
}
// Arrives on the mbarrier once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void mma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 consecutive accumulator columns of this thread's lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_load_32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Sum over the accumulators that `ksteps` k-steps have written (the tail accumulator and the first
// min(ksteps, kHeadAccs) head accumulators), for this thread's lane: out[k] = column k.
__device__ __forceinline__ void tmem_sum_accs(uint32_t taddr_lane, int ksteps, float (&out)[kModels]) {
    uint32_t r[32];
    tmem_load_32(taddr_lane + (uint32_t)(kHeadAccs * kModels), r);
#pragma unroll
    for (int k = 0; k < kModels; ++k) out[k] = __uint_as_float(r[k]);
    const int heads = ksteps < kHeadAccs ? ksteps : kHeadAccs;
#pragma unroll 1
    for (int h = 0; h < heads; ++h) {       // warp-uniform trip count
        tmem_load_32(taddr_lane + (uint32_t)(h * kModels), r);
#pragma unroll
        for (int k = 0; k < kModels; ++k) out[k] += __uint_as_float(r[k]);
    }
}

// Shared-memory matrix descriptor for a tile of 128-byte rows written by TMA with a 128-byte swizzle.
// K-major operand (kLayoutSw128, 16-byte chunks swizzled): groups of 8 rows `sbo` = 1024 bytes apart,
// `lbo` unused.  MN-major operand of 32-bit elements (kLayoutSw128Base32, 32-byte chunks swizzled,
// the only layout tcgen05 takes for MN-major tf32): a row holds 32 consecutive elements along M/N,
// rows follow along K, groups of 4 rows `sbo` = 512 bytes apart, and `lbo` is the distance between
// successive 32-element groups along M/N.
constexpr uint64_t kLayoutSw128 = 2, kLayoutSw128Base32 = 1;
__device__ __forceinline__ uint64_t smem_desc(const void *p, uint32_t lbo_bytes, uint32_t sbo_bytes, uint64_t layout) {
    uint64_t desc = 0;
    desc |= (uint64_t)((smem_u32(p) >> 4) & 0x3fffu);
    desc |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    desc |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    desc |= 1ull << 46;   // descriptor version of this architecture
    desc |= layout << 61;
    return desc;
}

// Instruction descriptor of kind::tf32 with fp32 accumulation.
__host__ __device__ constexpr uint32_t instr_desc_tf32(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ float tf32_head(float x) { return __uint_as_float(__float_as_uint(x) & 0xffffe000u); }

}  // namespace tc

// W [K][d] fp32 -> head and tail, each [32][d] (rows K..31 zero): head = the TF32 truncation, tail = the rest.
__global__ void cr_tc_split_models_kernel(const float *__restrict__ W, int K, long long d, float *__restrict__ Wh,
                                          float *__restrict__ Wl) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)tc::kModels * d) return;
    const int k = (int)(i / d);
    const float w = k < K ? W[i] : 0.f;
    const float h = tc::tf32_head(w);
    Wh[i] = h;
    Wl[i] = w - h;
}


// ------------------------------------------------------------------------------------------------
// Residuals of K models: R[item][row][k] = link(<X_p[row,:], w_k>) - y_p[row]
// ------------------------------------------------------------------------------------------------
//
// grid (row tiles, items), 192 threads: warp 0 streams boxes of 128 rows x 32 columns of X_p and
// 32 models x 32 columns of the two halves of W into a ring (TMA, 128-byte swizzle); warp 1 owns the
// tensor-memory accumulator (128 lanes x 32 columns) and issues, per box, 4 k-steps x 2 MMAs
// (X * W_head^T and X * W_tail^T); warps 2..5 read the accumulator (each its quarter of the lanes),
// subtract the label, and store head and tail of the residual for the gradient kernel.

struct TcResidualArgs {
    const float *y;        // [P][rows]
    const int32_t *part;   // [items]
    const int32_t *order;  // [items] or null: launch order of the items (same partition side by side)
    float *Rh, *Rl;        // [items][rows_pad][32]
    float *R_out;          // optional [items][rows][K]
    int items;
    int ipt;               // items per 128-row tile: 1, or 128 / sub_rows for partitions of few rows
    int sub_rows;          // ipt > 1: rows of a tile that one item takes (its rows rounded up to a multiple of 8)
    int rows, rows_pad, K, loss, stages;
    int kchunks;           // ceil(d / 32)
    int *status;
    unsigned long long wait_ns;  // bound of every wait, in nanoseconds
};

__global__ void __launch_bounds__(192, 1)
cr_tc_residual_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapWh,
                      const __grid_constant__ CUtensorMap mapWl, const TcResidualArgs a) {
    using namespace tc;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr uint32_t kXBytes = kTileM * kBoxCols * 4;     // 16 KB
    constexpr uint32_t kWBytes = kModels * kBoxCols * 4;    // 4 KB
    constexpr uint32_t kStageBytes = kXBytes + 2 * kWBytes;
    const int S = a.stages;
    // the swizzled tiles need 1024-byte alignment; the launch reserves 1 KB of slack for this
    unsigned char *ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t *full = reinterpret_cast<uint64_t *>(ring + (size_t)S * kStageBytes);
    uint64_t *empty = full + S;
    uint64_t *acc_full = empty + S;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
    volatile int *flags = reinterpret_cast<volatile int *>(tmem_slot + 1);   // [0] someone gave up, [1] never set

    // Partitions of few rows (the paper's logistic run has 39 per partition) would leave most of a 128-row
    // tile empty and drag the two W tiles through shared memory once per item.  Then `ipt` items share a
    // tile: item j of the group takes tile rows j * sub_rows .. (its box is sub_rows rows high, rows beyond
    // the partition are zero-filled by the copy engine), and W is fetched once for all of them.
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int first = (int)blockIdx.y * a.ipt;                       // first item of this CTA's group (launch order)
    const int in_group = min(a.ipt, a.items - first);
    const int row0 = blockIdx.x * kTileM;                            // ipt == 1: tile of the partition's rows

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_full, 1);
        flags[0] = 0; flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            int parts[kTileM / 8];
            for (int j = 0; j < in_group; ++j) {
                const int it = a.order ? __ldg(&a.order[first + j]) : first + j;
                parts[j] = __ldg(&a.part[it]);
            }
            const uint32_t sub_bytes = (uint32_t)a.sub_rows * kBoxCols * 4;
            const uint32_t x_bytes = a.ipt > 1 ? (uint32_t)in_group * sub_bytes : kXBytes;
            for (int kc = 0; kc < a.kchunks; ++kc) {
                const int s = kc % S;
                if (!mbar_wait(&empty[s], (uint32_t)(((kc / S) & 1) ^ 1), &flags[0], a.wait_ns)) { ok = false; break; }
                unsigned char *st = ring + (size_t)s * kStageBytes;
                mbar_expect_tx(&full[s], x_bytes + 2 * kWBytes);
                if (a.ipt > 1) {
                    for (int j = 0; j < in_group; ++j)
                        tma_load_3d(st + (size_t)j * sub_bytes, &mapX, kc * kBoxCols, 0, parts[j], &full[s]);
                } else {
                    tma_load_3d(st, &mapX, kc * kBoxCols, row0, parts[0], &full[s]);
                }
                tma_load_2d(st + kXBytes, &mapWh, kc * kBoxCols, 0, &full[s]);
                tma_load_2d(st + kXBytes + kWBytes, &mapWl, kc * kBoxCols, 0, &full[s]);
                ++issued;
            }
            if (!ok) {
                flags[0] = 1;
                atomicExch(a.status, 1);
                for (int i = issued > S ? issued - S : 0; i < issued; ++i)
                    mbar_wait(&full[i % S], (uint32_t)((i / S) & 1), &flags[1], a.wait_ns);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_tf32(kTileM, kModels, 0, 0);
            bool ok = true;
            for (int kc = 0; kc < a.kchunks; ++kc) {
                const int s = kc % S;
                if (!mbar_wait(&full[s], (uint32_t)((kc / S) & 1), &flags[0], a.wait_ns)) { ok = false; break; }
                tc_fence_after();
                const unsigned char *st = ring + (size_t)s * kStageBytes;
#pragma unroll
                for (int ks = 0; ks < kBoxCols / 8; ++ks) {
                    const uint64_t da = smem_desc(st + ks * 32, 16, 1024, kLayoutSw128);
                    const uint64_t dh = smem_desc(st + kXBytes + ks * 32, 16, 1024, kLayoutSw128);
                    const uint64_t dl = smem_desc(st + kXBytes + kWBytes + ks * 32, 16, 1024, kLayoutSw128);
                    const int g = kc * (kBoxCols / 8) + ks;    // running k-step
                    mma_tf32(tmem_acc + (uint32_t)((g % kHeadAccs) * kModels), da, dh, idesc, g >= kHeadAccs ? 1u : 0u);
                    mma_tf32(tmem_acc + (uint32_t)(kHeadAccs * kModels), da, dl, idesc, g > 0 ? 1u : 0u);
                }
                mma_commit(&empty[s]);       // the stage may be refilled once these MMAs have read it
            }
            if (ok) mma_commit(acc_full);
            else { flags[0] = 1; atomicExch(a.status, 1); }
        }
    } else {
        // epilogue: quarter (warp % 4) of the 128 accumulator lanes, one row per thread
        const int q = warp & 3;
        const int trow = q * 32 + lane;                                  // row of the tile
        const int j = a.ipt > 1 ? trow / a.sub_rows : 0;                 // which item of the group
        const int row = a.ipt > 1 ? trow - j * a.sub_rows : row0 + trow; // row of that item's partition
        const bool mine = j < in_group && (a.ipt == 1 || row < a.sub_rows);
        const int item = mine ? (a.order ? __ldg(&a.order[first + j]) : first + j) : 0;
        const int p = mine ? __ldg(&a.part[item]) : 0;
        const float yv = (mine && row < a.rows) ? __ldg(&a.y[(size_t)p * a.rows + row]) : 0.f;
        const bool ok = __all_sync(0xffffffffu, mbar_wait(acc_full, 0, &flags[0], a.wait_ns) ? 1 : 0) != 0;
        if (ok) {
            tc_fence_after();
            float r[kModels];
            tmem_sum_accs(tmem_acc + ((uint32_t)(q * 32) << 16), a.kchunks * (kBoxCols / 8), r);
            if (mine && row < a.rows_pad) {
                float4 *dh = reinterpret_cast<float4 *>(a.Rh + ((size_t)item * a.rows_pad + row) * kModels);
                float4 *dl = reinterpret_cast<float4 *>(a.Rl + ((size_t)item * a.rows_pad + row) * kModels);
#pragma unroll
                for (int k4 = 0; k4 < kModels / 4; ++k4) {
                    float v[4], h[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int k = k4 * 4 + i;
                        float z = r[k];
                        if (a.loss == 1) z = 1.f / (1.f + expf(-z));
                        v[i] = (k < a.K && row < a.rows) ? z - yv : 0.f;
                        h[i] = tf32_head(v[i]);
                        if (a.R_out && k < a.K && row < a.rows) a.R_out[((size_t)item * a.rows + row) * a.K + k] = v[i];
                    }
                    dh[k4] = make_float4(h[0], h[1], h[2], h[3]);
                    dl[k4] = make_float4(v[0] - h[0], v[1] - h[1], v[2] - h[2], v[3] - h[3]);
                }
            }
        } else if (lane == 0) {
            flags[0] = 1;
            atomicExch(a.status, 1);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_free(tmem_acc, kTmemCols);
}


// ------------------------------------------------------------------------------------------------
// Gradients of K models: G[k][item][col] = sum_rows X_p[row][col] * R[item][row][k]
// ------------------------------------------------------------------------------------------------
//
// grid (column tiles, items), 192 threads, same roles as above.  A stage holds kRowsB rows: four TMA
// boxes of kRowsB rows x 32 columns of X_p (together 128 columns) and kRowsB rows x 32 models of the
// two halves of R.  Seen as an operand with M = columns and K = rows the X boxes are MN-major:
// 32 columns (128 bytes) are contiguous, the next 32 columns lie one box further (the descriptor's
// leading-dimension offset), rows follow at 128 bytes.  MN-major tf32 operands use the 128-byte swizzle
// with 32-byte atoms (TMA and descriptor alike): groups of 4 rows, 512 bytes apart.  Each k-step of 8
// rows is two such groups, so stepping through the rows advances both descriptors by 1024 bytes.

constexpr int kRowsB = 64;

struct TcGradientArgs {
    const int32_t *part;   // [items]
    const int32_t *order;  // [items] or null
    float *G;              // [K][items][d]
    long long d;
    int rows, K, items, stages;
    int *status;
    unsigned long long wait_ns;  // bound of every wait, in nanoseconds
};

__global__ void __launch_bounds__(192, 1)
cr_tc_gradient_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapRh,
                      const __grid_constant__ CUtensorMap mapRl, const TcGradientArgs a) {
    using namespace tc;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr uint32_t kBoxBytes = kRowsB * kBoxCols * 4;          // 8 KB: kRowsB rows of 128 bytes
    constexpr uint32_t kXBytes = (kTileM / kBoxCols) * kBoxBytes;  // 32 KB
    constexpr uint32_t kStageBytes = kXBytes + 2 * kBoxBytes;      // 48 KB
    const int S = a.stages;
    // the swizzled tiles need 1024-byte alignment; the launch reserves 1 KB of slack for this
    unsigned char *ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t *full = reinterpret_cast<uint64_t *>(ring + (size_t)S * kStageBytes);
    uint64_t *empty = full + S;
    uint64_t *acc_full = empty + S;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
    volatile int *flags = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int item = a.order ? __ldg(&a.order[blockIdx.y]) : (int)blockIdx.y;
    const int col0 = blockIdx.x * kTileM;
    const int p = __ldg(&a.part[item]);
    const int chunks = (a.rows + kRowsB - 1) / kRowsB;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_full, 1);
        flags[0] = 0; flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            for (int c = 0; c < chunks; ++c) {
                const int s = c % S;
                if (!mbar_wait(&empty[s], (uint32_t)(((c / S) & 1) ^ 1), &flags[0], a.wait_ns)) { ok = false; break; }
                unsigned char *st = ring + (size_t)s * kStageBytes;
                mbar_expect_tx(&full[s], kStageBytes);
#pragma unroll
                for (int b = 0; b < kTileM / kBoxCols; ++b)
                    tma_load_3d(st + b * kBoxBytes, &mapX, col0 + b * kBoxCols, c * kRowsB, p, &full[s]);
                tma_load_3d(st + kXBytes, &mapRh, 0, c * kRowsB, item, &full[s]);
                tma_load_3d(st + kXBytes + kBoxBytes, &mapRl, 0, c * kRowsB, item, &full[s]);
                ++issued;
            }
            if (!ok) {
                flags[0] = 1;
                atomicExch(a.status, 1);
                for (int i = issued > S ? issued - S : 0; i < issued; ++i)
                    mbar_wait(&full[i % S], (uint32_t)((i / S) & 1), &flags[1], a.wait_ns);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_tf32(kTileM, kModels, 1, 1);
            bool ok = true;
            for (int c = 0; c < chunks; ++c) {
                const int s = c % S;
                if (!mbar_wait(&full[s], (uint32_t)((c / S) & 1), &flags[0], a.wait_ns)) { ok = false; break; }
                tc_fence_after();
                const unsigned char *st = ring + (size_t)s * kStageBytes;
#pragma unroll
                for (int ks = 0; ks < kRowsB / 8; ++ks) {
                    const uint64_t da = smem_desc(st + ks * 1024, kBoxBytes, 512, kLayoutSw128Base32);
                    const uint64_t dh = smem_desc(st + kXBytes + ks * 1024, kBoxBytes, 512, kLayoutSw128Base32);
                    const uint64_t dl = smem_desc(st + kXBytes + kBoxBytes + ks * 1024, kBoxBytes, 512, kLayoutSw128Base32);
                    const int g = c * (kRowsB / 8) + ks;       // running k-step
                    mma_tf32(tmem_acc + (uint32_t)((g % kHeadAccs) * kModels), da, dh, idesc, g >= kHeadAccs ? 1u : 0u);
                    mma_tf32(tmem_acc + (uint32_t)(kHeadAccs * kModels), da, dl, idesc, g > 0 ? 1u : 0u);
                }
                mma_commit(&empty[s]);
            }
            if (ok) mma_commit(acc_full);
            else { flags[0] = 1; atomicExch(a.status, 1); }
        }
    } else {
        const int q = warp & 3;
        const long long col = (long long)col0 + q * 32 + lane;
        const bool ok = __all_sync(0xffffffffu, mbar_wait(acc_full, 0, &flags[0], a.wait_ns) ? 1 : 0) != 0;
        if (ok) {
            tc_fence_after();
            float r[kModels];
            tmem_sum_accs(tmem_acc + ((uint32_t)(q * 32) << 16), chunks * (kRowsB / 8), r);
            if (col < a.d) {
#pragma unroll
                for (int k = 0; k < kModels; ++k)
                    if (k < a.K) a.G[((size_t)k * a.items + item) * a.d + col] = r[k];
            }
        } else if (lane == 0) {
            flags[0] = 1;
            atomicExch(a.status, 1);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_free(tmem_acc, kTmemCols);
}

// The same contraction for partitions of at most kRowsB rows, where the kernel above would be one small MMA
// group between a launch, a tensor-memory allocation and an epilogue per (column tile, item).  Here a CTA
// keeps an item: its residual tiles are fetched once, the column tiles stream through a ring of X stages,
// and two sets of accumulators alternate so that the epilogue of one tile runs under the MMAs of the next.
// With at most eight k-steps the truncation of the tensor core's accumulator is no concern (about 1.5e-8 of
// the sum per addition), so a set is two accumulators only, head products and tail products: the epilogue
// reads 64 columns per tile, not 256 (which made it, not the loads, the pace of the first version: 262 us
// on the logistic shape).  grid (CTAs per item, items), 192 threads, same roles; 128 columns of tensor memory
// and two X stages, so that two CTAs share an SM.
__global__ void __launch_bounds__(192, 2)
cr_tc_gradient_short_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapRh,
                            const __grid_constant__ CUtensorMap mapRl, const TcGradientArgs a) {
    using namespace tc;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr uint32_t kBoxBytes = kRowsB * kBoxCols * 4;          // 8 KB: kRowsB rows of 128 bytes
    constexpr uint32_t kXBytes = (kTileM / kBoxCols) * kBoxBytes;  // 32 KB: one column tile
    constexpr uint32_t kSetCols = 2 * kModels;                     // accumulator columns of one set: head, tail
    const int S = a.stages;
    unsigned char *ring = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char *rtile = ring + (size_t)S * kXBytes;             // residuals: head then tail, 8 KB each
    uint64_t *full = reinterpret_cast<uint64_t *>(rtile + 2 * kBoxBytes);
    uint64_t *empty = full + S;
    uint64_t *r_full = empty + S;
    uint64_t *acc_full = r_full + 1;     // [2]
    uint64_t *acc_empty = acc_full + 2;  // [2]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile int *flags = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int item = a.order ? __ldg(&a.order[blockIdx.y]) : (int)blockIdx.y;
    const int p = __ldg(&a.part[item]);
    const int ntiles = (int)((a.d + kTileM - 1) / kTileM);
    const int my_tiles = (int)blockIdx.x < ntiles ? (ntiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int ksteps = (a.rows + 7) / 8;   // <= kRowsB / 8

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(r_full, 1);
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
        flags[0] = 0; flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, 2 * kSetCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            mbar_expect_tx(r_full, 2 * kBoxBytes);
            tma_load_3d(rtile, &mapRh, 0, 0, item, r_full);
            tma_load_3d(rtile + kBoxBytes, &mapRl, 0, 0, item, r_full);
            for (int i = 0; i < my_tiles; ++i) {
                const int s = i % S;
                const int col0 = ((int)blockIdx.x + i * (int)gridDim.x) * kTileM;
                if (!mbar_wait(&empty[s], (uint32_t)(((i / S) & 1) ^ 1), &flags[0], a.wait_ns)) { ok = false; break; }
                unsigned char *st = ring + (size_t)s * kXBytes;
                mbar_expect_tx(&full[s], kXBytes);
#pragma unroll
                for (int b = 0; b < kTileM / kBoxCols; ++b)
                    tma_load_3d(st + b * kBoxBytes, &mapX, col0 + b * kBoxCols, 0, p, &full[s]);
                ++issued;
            }
            if (!ok) {
                flags[0] = 1;
                atomicExch(a.status, 1);
                mbar_wait(r_full, 0, &flags[1], a.wait_ns);
                for (int i = issued > S ? issued - S : 0; i < issued; ++i)
                    mbar_wait(&full[i % S], (uint32_t)((i / S) & 1), &flags[1], a.wait_ns);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_tf32(kTileM, kModels, 1, 1);
            bool ok = mbar_wait(r_full, 0, &flags[0], a.wait_ns);
            for (int i = 0; i < my_tiles && ok; ++i) {
                const int s = i % S, set = i & 1;
                if (!mbar_wait(&full[s], (uint32_t)((i / S) & 1), &flags[0], a.wait_ns)) { ok = false; break; }
                // the accumulator set must have been read by the epilogue of the tile before last
                if (!mbar_wait(&acc_empty[set], (uint32_t)(((i >> 1) & 1) ^ 1), &flags[0], a.wait_ns)) { ok = false; break; }
                tc_fence_after();
                const unsigned char *st = ring + (size_t)s * kXBytes;
                const uint32_t acc0 = tmem_acc + (uint32_t)set * kSetCols;
                for (int ks = 0; ks < ksteps; ++ks) {
                    const uint64_t da = smem_desc(st + ks * 1024, kBoxBytes, 512, kLayoutSw128Base32);
                    const uint64_t dh = smem_desc(rtile + ks * 1024, kBoxBytes, 512, kLayoutSw128Base32);
                    const uint64_t dl = smem_desc(rtile + kBoxBytes + ks * 1024, kBoxBytes, 512, kLayoutSw128Base32);
                    mma_tf32(acc0, da, dh, idesc, ks > 0 ? 1u : 0u);
                    mma_tf32(acc0 + (uint32_t)kModels, da, dl, idesc, ks > 0 ? 1u : 0u);
                }
                mma_commit(&empty[s]);          // the X stage may be refilled once these MMAs have read it
                mma_commit(&acc_full[set]);     // and the epilogue may read the set
            }
            if (!ok) { flags[0] = 1; atomicExch(a.status, 1); }
        }
    } else {
        const int q = warp & 3;
        bool ok = true;
        for (int i = 0; i < my_tiles; ++i) {
            const int set = i & 1;
            const long long col = (long long)((int)blockIdx.x + i * (int)gridDim.x) * kTileM + q * 32 + lane;
            ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[set], (uint32_t)((i >> 1) & 1), &flags[0], a.wait_ns) ? 1 : 0) != 0;
            if (!ok) break;
            tc_fence_after();
            float r[kModels];
            {
                uint32_t h[32], t[32];
                const uint32_t lane_base = tmem_acc + (uint32_t)set * kSetCols + ((uint32_t)(q * 32) << 16);
                tmem_load_32(lane_base, h);
                tmem_load_32(lane_base + (uint32_t)kModels, t);
#pragma unroll
                for (int k = 0; k < kModels; ++k) r[k] = __uint_as_float(h[k]) + __uint_as_float(t[k]);
            }
            // the set is in registers: hand it back before the stores
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[set]);
            if (col < a.d) {
#pragma unroll
                for (int k = 0; k < kModels; ++k)
                    if (k < a.K) a.G[((size_t)k * a.items + item) * a.d + col] = r[k];
            }
        }
        if (!ok && lane == 0) { flags[0] = 1; atomicExch(a.status, 1); }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_free(tmem_acc, 2 * kSetCols);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------

static CUresult encode_sw128(EncodeTiledFn encode, CUtensorMap *map, const void *base, int rank, const cuuint64_t *dims,
                             const cuuint64_t *strides, const cuuint32_t *box, CUtensorMapSwizzle swizzle) {
    const cuuint32_t estr[3] = {1, 1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

size_t multi_model_workspace_bytes(int items, int rows, int64_t d) {
    const size_t rows_pad = (size_t)(rows + tc::kTileM - 1) / tc::kTileM * tc::kTileM;
    return 2 * (size_t)tc::kModels * (size_t)d * 4 + 2 * (size_t)items * rows_pad * tc::kModels * 4;
}

bool multi_model_eligible(const float *X, const float *G, const void *workspace, int64_t d, int rows, int K, int items) {
    auto al = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    return d % 4 == 0 && d >= tc::kBoxCols && d < (1ll << 31) && K >= 1 && K <= tc::kModels && rows >= 1 && items <= 65535 &&
           al(X) && al(G) && al(workspace);
}

cudaError_t launch_partial_gradients_multi(const float *X, const float *y, const float *W, int K, const int32_t *part,
                                           const int32_t *order, int items, int P, int rows, int64_t d, float *G,
                                           float *R_out, int loss,
                                           void *workspace, int *status, const Tuning &tune, EncodeTiledFn encode,
                                           cudaStream_t stream, int64_t *launches) {
    using namespace tc;
    const int rows_pad = (rows + kTileM - 1) / kTileM * kTileM;
    // partitions of at most kRowsB rows: several items share a 128-row tile of the residual kernel, and the
    // gradient kernel keeps an item per CTA (see the kernels)
    const bool few_rows = rows <= kRowsB;
    const int sub_rows = (rows + 7) / 8 * 8;
    const int ipt = few_rows ? kTileM / sub_rows : 1;
    float *Wh = reinterpret_cast<float *>(workspace);
    float *Wl = Wh + (size_t)kModels * d;
    float *Rh = Wl + (size_t)kModels * d;
    float *Rl = Rh + (size_t)items * rows_pad * kModels;

    {
        const long long n = (long long)kModels * d;
        cr_tc_split_models_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(W, K, d, Wh, Wl);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        ++*launches;
    }

    CUtensorMap mapX, mapXg, mapWh, mapWl, mapRh, mapRl;
    {
        const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)P};
        const cuuint64_t strides[2] = {(cuuint64_t)d * 4, (cuuint64_t)rows * (cuuint64_t)d * 4};
        const cuuint32_t boxA[3] = {kBoxCols, (cuuint32_t)(ipt > 1 ? sub_rows : kTileM), 1};
        const cuuint32_t boxB[3] = {kBoxCols, kRowsB, 1};
        if (encode_sw128(encode, &mapX, X, 3, dims, strides, boxA, CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS) return cudaErrorInvalidValue;
        if (encode_sw128(encode, &mapXg, X, 3, dims, strides, boxB, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    {
        const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)kModels};
        const cuuint64_t strides[1] = {(cuuint64_t)d * 4};
        const cuuint32_t box[2] = {kBoxCols, kModels};
        if (encode_sw128(encode, &mapWh, Wh, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS) return cudaErrorInvalidValue;
        if (encode_sw128(encode, &mapWl, Wl, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    {
        const cuuint64_t dims[3] = {(cuuint64_t)kModels, (cuuint64_t)rows_pad, (cuuint64_t)items};
        const cuuint64_t strides[2] = {(cuuint64_t)kModels * 4, (cuuint64_t)rows_pad * kModels * 4};
        const cuuint32_t box[3] = {kModels, kRowsB, 1};
        if (encode_sw128(encode, &mapRh, Rh, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) != CUDA_SUCCESS) return cudaErrorInvalidValue;
        if (encode_sw128(encode, &mapRl, Rl, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }

    {   // residuals
        TcResidualArgs ra;
        ra.y = y; ra.part = part; ra.order = order; ra.Rh = Rh; ra.Rl = Rl; ra.R_out = R_out; ra.rows = rows; ra.rows_pad = rows_pad;
        ra.items = items; ra.ipt = ipt; ra.sub_rows = sub_rows;
        ra.K = K; ra.loss = loss; ra.stages = 4; ra.kchunks = (int)((d + kBoxCols - 1) / kBoxCols); ra.status = status; ra.wait_ns = tune.wait_limit_ns;
        const size_t smem = (size_t)ra.stages * (kTileM * kBoxCols * 4 + 2 * kModels * kBoxCols * 4) + (2 * ra.stages + 1) * 8 + 16 + 1024;
        cudaError_t e = cudaFuncSetAttribute(cr_tc_residual_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        const dim3 grid = ipt > 1 ? dim3(1, (unsigned)((items + ipt - 1) / ipt)) : dim3((unsigned)(rows_pad / kTileM), (unsigned)items);
        cr_tc_residual_kernel<<<grid, 192, smem, stream>>>(mapX, mapWh, mapWl, ra);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    if (G) {   // gradients
        TcGradientArgs ga;
        ga.part = part; ga.order = order; ga.G = G; ga.d = d; ga.rows = rows; ga.K = K; ga.items = items; ga.stages = tune.tc_stages ? tune.tc_stages : 2; ga.status = status; ga.wait_ns = tune.wait_limit_ns;
        cudaError_t e;
        if (few_rows) {
            ga.stages = tune.tc_stages ? tune.tc_stages : 2;
            const size_t smem = (size_t)ga.stages * (kTileM / kBoxCols) * kRowsB * kBoxCols * 4 + 2 * kRowsB * kBoxCols * 4 +
                                (2 * ga.stages + 5) * 8 + 16 + 1024;
            e = cudaFuncSetAttribute(cr_tc_gradient_short_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            // CTAs per item: enough to give every SM about two CTAs, each with several column tiles
            int dev = 0, sms = 148;
            if (cudaGetDevice(&dev) == cudaSuccess) (void)cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            const int ntiles = (int)((d + kTileM - 1) / kTileM);
            int per_item = (2 * sms + items - 1) / items;
            per_item = std::max(1, std::min(per_item, (ntiles + 3) / 4));
            cr_tc_gradient_short_kernel<<<dim3((unsigned)per_item, (unsigned)items), 192, smem, stream>>>(mapXg, mapRh, mapRl, ga);
            e = cudaGetLastError();
            if (e != cudaSuccess) return e;
            ++*launches;
            return cudaSuccess;
        }
        const size_t smem = (size_t)ga.stages * ((kTileM / kBoxCols + 2) * kRowsB * kBoxCols * 4) + (2 * ga.stages + 1) * 8 + 16 + 1024;
        e = cudaFuncSetAttribute(cr_tc_gradient_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        cr_tc_gradient_kernel<<<dim3((unsigned)((d + kTileM - 1) / kTileM), (unsigned)items), 192, smem, stream>>>(mapXg, mapRh, mapRl, ga);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    return cudaSuccess;
}

}  // namespace cr
