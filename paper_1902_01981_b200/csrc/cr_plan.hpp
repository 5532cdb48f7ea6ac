// Host-side plan of the coded tree aggregation: tree indexing, encoding matrices,
// partition allocation and decode tables.  Pure C++ (no CUDA), fp64 + integers.
#pragma once

#include <cstdint>
#include <string>
#include <vector>

#include "codedreduce.h"

namespace cr {

// One entry of a node's local data set D(l,i): a partition and its combining coefficient
// (the "scaled data set" b*D of Section III-A).
struct Slot {
    int32_t part;
    double coeff;
};

// One step of an expanded straggler pattern: a node whose data is consumed, its layer (1..L) and the
// decode weight its message gets at its parent.
struct UsedNode {
    int32_t node;
    int32_t layer;
    double weight;
    bool first;  // first consumed child of its parent (in visiting order)
};

struct HostPlan {
    int n = 0, L = 0, s = 0, P = 0;
    int64_t d = 0;
    int code = 0, dtype = 0;
    int N = 0;       // workers
    int groups = 0;  // sibling groups = parents, master included
    int m = 0;       // slots per node = r_CR * P
    std::vector<int> layer_offset;        // [L+2]: flat index of the first node of layer l (1-based l)
    std::vector<std::vector<double>> B;   // [L] level -> n*n row-major
    std::vector<double> kappa;            // [L]
    std::vector<uint64_t> sub_seed;       // [L]
    std::vector<Slot> slots;              // [N*m]
    std::vector<std::vector<double>> decode;  // [L] level -> (1<<n)*n, rows of undecodable masks unused
    int64_t int_scale = 1;                // S = sigma^L (CR_I32), else 1
    int int_shift = 0;                    // log2(S)

    int layer_of(int node) const;
    int nodes_in_layer(int l) const;  // n^l
    const double *decode_row(int level, uint32_t mask) const { return &decode[level][(size_t)mask * n]; }
    bool mask_ok(uint32_t mask) const;

    // Straggler pattern of one iteration from per-node computation times under the single-port model
    // (Section III-C): see cr_latency_masks in codedreduce.h.  masks_out[groups], returns the time at
    // which the master holds n-s messages.
    double latency_masks(const double *compute_time, double t_c, uint32_t *masks_out) const;

    // Post-order expansion of one pattern.  Returns CR_OK, CR_ERR_UNDECODABLE_MASK or CR_ERR_INVALID_ARG.
    cr_status_t expand(const uint32_t *masks, std::vector<UsedNode> &out) const;
};

// Builds everything from the descriptor.  On failure returns the status and leaves `plan` unspecified.
cr_status_t build_host_plan(const cr_plan_desc_t &desc, HostPlan &plan);

// Least-squares solve min ||A x - b|| for a tall full-column-rank A (rows x cols, row-major) by
// Householder QR.  Returns false if a diagonal of R vanishes.
bool least_squares(std::vector<double> A, int rows, int cols, std::vector<double> b, std::vector<double> &x);

// SplitMix64 (Steele, Lea, Flood 2014): k-th output for a given start state.
uint64_t splitmix64_at(uint64_t seed, uint64_t k);

}  // namespace cr
