// Plan builder: everything CodedReduce fixes before the first iteration (CR.Allocate of
// Algorithm 2 over CompAlloc of Algorithm 1, plus the gradient-coding matrices of Section II-C).
#include "cr_plan.hpp"

#include <algorithm>
#include <cmath>
#include <cstring>

namespace cr {

// ------------------------------------------------------------------------------------------------
// small dense linear algebra (fp64)
// ------------------------------------------------------------------------------------------------

bool least_squares(std::vector<double> A, int rows, int cols, std::vector<double> b, std::vector<double> &x) {
    // Householder reflections applied column by column to [A | b]; then back substitution on R.
    for (int k = 0; k < cols; ++k) {
        double norm = 0.0;
        for (int i = k; i < rows; ++i) norm += A[(size_t)i * cols + k] * A[(size_t)i * cols + k];
        norm = std::sqrt(norm);
        if (norm == 0.0) return false;
        const double alpha = A[(size_t)k * cols + k] > 0 ? -norm : norm;
        std::vector<double> v(rows, 0.0);
        for (int i = k; i < rows; ++i) v[i] = A[(size_t)i * cols + k];
        v[k] -= alpha;
        double vnorm2 = 0.0;
        for (int i = k; i < rows; ++i) vnorm2 += v[i] * v[i];
        if (vnorm2 == 0.0) continue;
        for (int j = k; j < cols; ++j) {
            double dot = 0.0;
            for (int i = k; i < rows; ++i) dot += v[i] * A[(size_t)i * cols + j];
            const double f = 2.0 * dot / vnorm2;
            for (int i = k; i < rows; ++i) A[(size_t)i * cols + j] -= f * v[i];
        }
        double dot = 0.0;
        for (int i = k; i < rows; ++i) dot += v[i] * b[i];
        const double f = 2.0 * dot / vnorm2;
        for (int i = k; i < rows; ++i) b[i] -= f * v[i];
    }
    x.assign(cols, 0.0);
    for (int k = cols - 1; k >= 0; --k) {
        double acc = b[k];
        for (int j = k + 1; j < cols; ++j) acc -= A[(size_t)k * cols + j] * x[j];
        const double diag = A[(size_t)k * cols + k];
        if (diag == 0.0) return false;
        x[k] = acc / diag;
    }
    return true;
}

// Square solve by Gaussian elimination with partial pivoting; M is q x q row-major.
static bool solve_square(std::vector<double> M, int q, std::vector<double> rhs, std::vector<double> &x) {
    for (int k = 0; k < q; ++k) {
        int piv = k;
        for (int i = k + 1; i < q; ++i)
            if (std::fabs(M[(size_t)i * q + k]) > std::fabs(M[(size_t)piv * q + k])) piv = i;
        if (M[(size_t)piv * q + k] == 0.0) return false;
        if (piv != k) {
            for (int j = 0; j < q; ++j) std::swap(M[(size_t)k * q + j], M[(size_t)piv * q + j]);
            std::swap(rhs[k], rhs[piv]);
        }
        for (int i = k + 1; i < q; ++i) {
            const double f = M[(size_t)i * q + k] / M[(size_t)k * q + k];
            for (int j = k; j < q; ++j) M[(size_t)i * q + j] -= f * M[(size_t)k * q + j];
            rhs[i] -= f * rhs[k];
        }
    }
    x.assign(q, 0.0);
    for (int k = q - 1; k >= 0; --k) {
        double acc = rhs[k];
        for (int j = k + 1; j < q; ++j) acc -= M[(size_t)k * q + j] * x[j];
        x[k] = acc / M[(size_t)k * q + k];
    }
    return true;
}

// ------------------------------------------------------------------------------------------------
// random draws: SplitMix64, counter based
// ------------------------------------------------------------------------------------------------

uint64_t splitmix64_at(uint64_t seed, uint64_t k) {
    uint64_t z = seed + (k + 1) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// Uniform in [-1, 1) from the top 53 bits (exact in fp64).
static double uniform_pm1(uint64_t seed, uint64_t k) {
    const double u = (double)(splitmix64_at(seed, k) >> 11) * (1.0 / 9007199254740992.0);
    return 2.0 * u - 1.0;
}

// ------------------------------------------------------------------------------------------------
// encoding matrices
// ------------------------------------------------------------------------------------------------

// Cyclic-support code: rows of B lie in the null space of a random s x n matrix H whose rows sum to
// zero, so the row space of any n-s independent rows of B is null(H), which contains the all-ones
// vector -- the recoverability condition of Section II-C.
static bool cyclic_code(int n, int s, uint64_t seed, std::vector<double> &B) {
    B.assign((size_t)n * n, 0.0);
    if (s == 0) {
        for (int i = 0; i < n; ++i) B[(size_t)i * n + i] = 1.0;
        return true;
    }
    std::vector<double> H((size_t)s * n, 0.0);
    for (int r = 0; r < s; ++r) {
        double sum = 0.0;
        for (int c = 0; c < n - 1; ++c) {
            const double u = uniform_pm1(seed, (uint64_t)r * (n - 1) + c);
            H[(size_t)r * n + c] = u;
            sum += u;
        }
        H[(size_t)r * n + n - 1] = -sum;
    }
    std::vector<double> M((size_t)s * s), rhs(s), x;
    for (int i = 0; i < n; ++i) {
        for (int r = 0; r < s; ++r) {
            for (int t = 0; t < s; ++t) M[(size_t)r * s + t] = H[(size_t)r * n + (i + 1 + t) % n];
            rhs[r] = -H[(size_t)r * n + i];
        }
        if (!solve_square(M, s, rhs, x)) return false;
        B[(size_t)i * n + i] = 1.0;
        for (int t = 0; t < s; ++t) B[(size_t)i * n + (i + 1 + t) % n] = x[t];
    }
    return true;
}

static void repetition_code(int n, int s, std::vector<double> &B) {
    B.assign((size_t)n * n, 0.0);
    for (int i = 0; i < n; ++i) {
        const int block = i / (s + 1);
        for (int k = block * (s + 1); k < (block + 1) * (s + 1); ++k) B[(size_t)i * n + k] = 1.0;
    }
}

// Eq. (gc3nodes).
static const double kPrintedB[9] = {0.5, 1.0, 0.0, 0.0, 1.0, -1.0, 0.5, 0.0, 1.0};
static const double kPrintedA[9] = {0.0, 1.0, 2.0, 1.0, 0.0, 1.0, 2.0, -1.0, 0.0};

static int popcount32(uint32_t x) { return __builtin_popcount(x); }

// Decode rows of one level for every mask with <= s bits.  Returns false when a row cannot be solved
// or does not reproduce the all-ones vector.
static bool decode_table(int n, int s, int code, const std::vector<double> &B, std::vector<double> &table,
                         double &kappa) {
    const uint32_t nmask = 1u << n;
    table.assign((size_t)nmask * n, 0.0);
    kappa = 0.0;
    std::vector<double> rownorm(n, 0.0);
    for (int i = 0; i < n; ++i)
        for (int k = 0; k < n; ++k) rownorm[i] += std::fabs(B[(size_t)i * n + k]);
    for (uint32_t mask = 0; mask < nmask; ++mask) {
        const int bits = popcount32(mask);
        if (bits > s) continue;
        double *a = &table[(size_t)mask * n];
        if (code == CR_CODE_FRACTIONAL_REPETITION) {
            for (int block = 0; block < n / (s + 1); ++block)
                for (int j = block * (s + 1); j < (block + 1) * (s + 1); ++j)
                    if (!((mask >> j) & 1u)) { a[j] = 1.0; break; }
        } else if (code == CR_CODE_PAPER_3_1) {
            // row f of the printed A serves "child f straggles"; with no straggler the two
            // lowest-indexed children are used, which is the row for f = 2.
            const int f = mask == 1u ? 0 : (mask == 2u ? 1 : 2);
            for (int j = 0; j < 3; ++j) a[j] = kPrintedA[f * 3 + j];
        } else {
            std::vector<int> U;
            for (int j = 0; j < n && (int)U.size() < n - s; ++j)
                if (!((mask >> j) & 1u)) U.push_back(j);
            const int q = (int)U.size();
            // B_U^T a_U = 1 : n equations, q unknowns, consistent when the span property holds.
            std::vector<double> At((size_t)n * q), ones(n, 1.0), sol;
            for (int k = 0; k < n; ++k)
                for (int t = 0; t < q; ++t) At[(size_t)k * q + t] = B[(size_t)U[t] * n + k];
            if (!least_squares(At, n, q, ones, sol)) return false;
            // weights that are pure rounding noise of the solve (a survivor that is not needed) are zero
            double big = 0.0;
            for (int t = 0; t < q; ++t) big = std::max(big, std::fabs(sol[t]));
            for (int t = 0; t < q; ++t) a[U[t]] = std::fabs(sol[t]) <= 1e-13 * big ? 0.0 : sol[t];
        }
        double amp = 0.0;
        for (int j = 0; j < n; ++j) amp += std::fabs(a[j]) * rownorm[j];
        double resid = 0.0;
        for (int k = 0; k < n; ++k) {
            double acc = 0.0;
            for (int j = 0; j < n; ++j) acc += a[j] * B[(size_t)j * n + k];
            resid = std::max(resid, std::fabs(acc - 1.0));
        }
        if (!(resid <= 1e-10 * std::max(1.0, amp))) return false;
        if (bits == s) kappa = std::max(kappa, amp);
    }
    return true;
}

// ------------------------------------------------------------------------------------------------
// HostPlan
// ------------------------------------------------------------------------------------------------

int HostPlan::nodes_in_layer(int l) const {
    int c = 1;
    for (int t = 0; t < l; ++t) c *= n;
    return c;
}

int HostPlan::layer_of(int node) const {
    for (int l = 1; l <= L; ++l)
        if (node < layer_offset[l + 1]) return l;
    return -1;
}

bool HostPlan::mask_ok(uint32_t mask) const { return (mask >> n) == 0 && popcount32(mask) <= s; }

cr_status_t HostPlan::expand(const uint32_t *masks, std::vector<UsedNode> &out) const {
    // Iterative post-order walk.  A frame is a parent (layer, index in layer) and the next child to visit.
    struct Frame { int layer, index, next; double weight; bool first; int seen; };
    std::vector<Frame> stack;
    stack.push_back({0, 0, 0, 0.0, true, 0});
    while (!stack.empty()) {
        Frame &f = stack.back();
        const int group = f.layer == 0 ? 0 : layer_offset[f.layer] + f.index + 1;
        const uint32_t mask = masks[group];
        if ((mask >> n) != 0) return CR_ERR_INVALID_ARG;
        if (popcount32(mask) > s) return CR_ERR_UNDECODABLE_MASK;
        const double *a = decode_row(f.layer, mask);
        int j = f.next;
        while (j < n && a[j] == 0.0) ++j;
        if (j == n) {
            // all used children done: emit this parent itself (not the master)
            if (f.layer > 0) out.push_back({layer_offset[f.layer] + f.index, f.layer, f.weight, f.first});
            stack.pop_back();
            continue;
        }
        f.next = j + 1;
        const bool child_first = f.seen == 0;
        ++f.seen;
        const int cl = f.layer + 1, ci = f.index * n + j;
        if (cl == L) {
            out.push_back({layer_offset[cl] + ci, cl, a[j], child_first});
        } else {
            const double w = a[j];
            stack.push_back({cl, ci, 0, w, child_first, 0});  // invalidates f
        }
    }
    return CR_OK;
}

double HostPlan::latency_masks(const double *compute_time, double t_c, uint32_t *masks_out) const {
    // ready[v] = time at which node v's message is ready for upload.  Layers are handled bottom-up, so
    // the children of a parent are ready before the parent is looked at.
    std::vector<double> ready(N, 0.0);
    for (int v = layer_offset[L]; v < N; ++v) ready[v] = compute_time[v];
    double master_done = 0.0;
    for (int l = L - 1; l >= 0; --l) {
        const int parents = nodes_in_layer(l);
        for (int i = 0; i < parents; ++i) {
            const int first_child = layer_offset[l + 1] + i * n;
            // the parent's single port serves its children in the order in which their messages become
            // ready (ties: lower index first); a transfer takes t_c
            std::vector<int> order(n);
            for (int j = 0; j < n; ++j) order[j] = j;
            std::stable_sort(order.begin(), order.end(),
                             [&](int x, int y) { return ready[first_child + x] < ready[first_child + y]; });
            double port_free = 0.0, got_enough = 0.0;
            uint32_t mask = 0;
            for (int k = 0; k < n; ++k) {
                const int j = order[k];
                if (k < n - s) {
                    const double start = std::max(ready[first_child + j], port_free);
                    port_free = start + t_c;
                    got_enough = port_free;   // arrival of the (k+1)-th message
                } else {
                    mask |= 1u << j;          // the parent no longer waits for these
                }
            }
            const int group = l == 0 ? 0 : layer_offset[l] + i + 1;
            masks_out[group] = mask;
            if (l == 0) master_done = got_enough;
            else ready[layer_offset[l] + i] = std::max(got_enough, compute_time[layer_offset[l] + i]);
        }
    }
    return master_done;
}

cr_status_t build_host_plan(const cr_plan_desc_t &desc, HostPlan &hp) {
    hp = HostPlan();
    const int n = desc.n, L = desc.L, s = desc.s;
    if (n < 2 || n > 16 || L < 1 || L > 8 || s < 0 || s >= n || desc.d < 1 || desc.P < 1 || desc.reserved != 0)
        return CR_ERR_INVALID_ARG;
    if (desc.code < CR_CODE_CYCLIC_RANDOM || desc.code > CR_CODE_EXPLICIT) return CR_ERR_INVALID_ARG;
    if (desc.dtype != CR_F32 && desc.dtype != CR_I32) return CR_ERR_INVALID_ARG;
    if (desc.code == CR_CODE_EXPLICIT && desc.B_explicit == nullptr) return CR_ERR_INVALID_ARG;
    if (desc.code == CR_CODE_FRACTIONAL_REPETITION && n % (s + 1) != 0) return CR_ERR_CODE_UNAVAILABLE;
    if (desc.code == CR_CODE_PAPER_3_1 && !(n == 3 && s == 1)) return CR_ERR_CODE_UNAVAILABLE;
    if (desc.dtype == CR_I32 && desc.code == CR_CODE_CYCLIC_RANDOM && s > 0) return CR_ERR_DTYPE;

    hp.n = n; hp.L = L; hp.s = s; hp.P = desc.P; hp.d = desc.d; hp.code = desc.code; hp.dtype = desc.dtype;

    // tree sizes: N = n + .. + n^L, one group per parent
    hp.layer_offset.assign(L + 2, 0);
    int64_t total = 0, width = 1;
    for (int l = 1; l <= L; ++l) {
        hp.layer_offset[l] = (int)total;
        width *= n;
        total += width;
        if (total > (1 << 22)) return CR_ERR_INVALID_ARG;
    }
    hp.layer_offset[L + 1] = (int)total;
    hp.N = (int)total;
    hp.groups = hp.N / n;

    // load: r_CR = 1 / sum_l (n/(s+1))^l (Theorem 1)  =>  m = r_CR P = c (s+1)^L when
    // P = c * sum_l n^l (s+1)^(L-l); other P would need fractional chunks.
    int64_t quantum = 0, pow_s = 1;
    {
        std::vector<int64_t> np(L + 1, 1), sp(L + 1, 1);
        for (int l = 1; l <= L; ++l) { np[l] = np[l - 1] * n; sp[l] = sp[l - 1] * (s + 1); }
        for (int l = 1; l <= L; ++l) quantum += np[l] * sp[L - l];
        pow_s = sp[L];
    }
    if (desc.P % quantum != 0) return CR_ERR_BAD_PARTITION_COUNT;
    const int64_t m64 = (desc.P / quantum) * pow_s;
    if (m64 * hp.N > (int64_t)1 << 30) return CR_ERR_INVALID_ARG;
    hp.m = (int)m64;

    // encoding matrices and decode tables, per level
    hp.B.assign(L, {});
    hp.decode.assign(L, {});
    hp.kappa.assign(L, 0.0);
    hp.sub_seed.assign(L, 0);
    const double cap = desc.max_kappa > 0 ? desc.max_kappa : 100.0;
    if (desc.code == CR_CODE_EXPLICIT) {
        for (int l = 0; l < L; ++l) {
            hp.B[l].assign(desc.B_explicit + (size_t)l * n * n, desc.B_explicit + (size_t)(l + 1) * n * n);
            if (!decode_table(n, s, desc.code, hp.B[l], hp.decode[l], hp.kappa[l])) return CR_ERR_ILL_CONDITIONED;
        }
    } else {
        std::vector<double> B, table;
        double kappa = 0.0;
        uint64_t used_seed = desc.seed;
        if (desc.code == CR_CODE_CYCLIC_RANDOM) {
            bool found = false;
            for (int t = 0; t < 64 && !found; ++t) {
                used_seed = desc.seed + (uint64_t)t;
                if (!cyclic_code(n, s, used_seed, B)) continue;
                if (!decode_table(n, s, desc.code, B, table, kappa)) continue;
                found = kappa <= cap;
            }
            if (!found) return CR_ERR_ILL_CONDITIONED;
        } else {
            if (desc.code == CR_CODE_FRACTIONAL_REPETITION) repetition_code(n, s, B);
            else B.assign(kPrintedB, kPrintedB + 9);
            if (!decode_table(n, s, desc.code, B, table, kappa)) return CR_ERR_ILL_CONDITIONED;
        }
        for (int l = 0; l < L; ++l) { hp.B[l] = B; hp.decode[l] = table; hp.kappa[l] = kappa; hp.sub_seed[l] = used_seed; }
    }

    // CR.Allocate.  `pass[i]` is the list handed down by parent i of the previous layer.
    hp.slots.assign((size_t)hp.N * hp.m, Slot{0, 0.0});
    std::vector<std::vector<Slot>> pass(1);
    pass[0].resize(desc.P);
    for (int p = 0; p < desc.P; ++p) pass[0][p] = Slot{p, 1.0};
    for (int l = 1; l <= L; ++l) {
        const std::vector<double> &B = hp.B[l - 1];
        std::vector<std::vector<Slot>> next(pass.size() * n);
        for (size_t parent = 0; parent < pass.size(); ++parent) {
            const std::vector<Slot> &Q = pass[parent];
            if (Q.size() % n != 0) return CR_ERR_BAD_PARTITION_COUNT;
            const size_t chunk = Q.size() / n;
            for (int child = 0; child < n; ++child) {
                // CompAlloc: union over kappa of b_{child,kappa} * D_kappa, increasing kappa
                std::vector<Slot> mine;
                for (int k = 0; k < n; ++k) {
                    const double b = B[(size_t)child * n + k];
                    if (b == 0.0) continue;
                    for (size_t t = 0; t < chunk; ++t) mine.push_back(Slot{Q[k * chunk + t].part, Q[k * chunk + t].coeff * b});
                }
                if ((int64_t)mine.size() < hp.m) return CR_ERR_BAD_PARTITION_COUNT;
                const int node = hp.layer_offset[l] + (int)parent * n + child;
                // the node keeps the first m pairs and hands the rest to its own children
                std::copy(mine.begin(), mine.begin() + hp.m, hp.slots.begin() + (size_t)node * hp.m);
                next[parent * n + child].assign(mine.begin() + hp.m, mine.end());
            }
        }
        pass.swap(next);
    }
    for (const auto &rest : pass)
        if (!rest.empty()) return CR_ERR_BAD_PARTITION_COUNT;  // leaves must keep everything

    // integer mode: sigma * B integer at every level, S = sigma^L scales every coefficient to an integer
    if (desc.dtype == CR_I32) {
        int64_t sigma = 1;
        auto integral = [&](int64_t sg) {
            for (const auto &B : hp.B)
                for (double b : B)
                    if (b * (double)sg != std::nearbyint(b * (double)sg)) return false;
            return true;
        };
        while (!integral(sigma)) {
            sigma *= 2;
            if (sigma > (1 << 20)) return CR_ERR_DTYPE;
        }
        int64_t S = 1;
        int shift = 0;
        for (int l = 0; l < L; ++l) S *= sigma;
        for (int64_t t = S; t > 1; t >>= 1) ++shift;
        if (S > ((int64_t)1 << 24)) return CR_ERR_DTYPE;
        for (const Slot &sl : hp.slots) {
            const double v = sl.coeff * (double)S;
            if (v != std::nearbyint(v) || std::fabs(v) > 2147483647.0) return CR_ERR_DTYPE;
        }
        for (int l = 0; l < L; ++l)
            for (uint32_t mask = 0; mask < (1u << n); ++mask) {
                if (popcount32(mask) > s) continue;
                double *a = &hp.decode[l][(size_t)mask * n];
                for (int j = 0; j < n; ++j) {
                    const double r = std::nearbyint(a[j]);
                    if (std::fabs(a[j] - r) > 1e-9) return CR_ERR_DTYPE;
                    a[j] = r;
                }
            }
        hp.int_scale = S;
        hp.int_shift = shift;
    }
    return CR_OK;
}

}  // namespace cr
