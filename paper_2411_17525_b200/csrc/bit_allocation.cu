// Dynamic bit-width assignment (Section 5, Eq. 4): choose one quantisation option j_l per layer so that
//   sum_l alpha_l * t2[l][j_l]   is minimal   subject to   sum_l bits[j_l] * d_l <= b_max * sum_l d_l.
// The objective is separable, so the problem is a multiple-choice knapsack; it is solved exactly on the host by
// dynamic programming over the integer budget.  (The paper hands the same problem to a CP-SAT solver.)
// Costs are made integers without rounding: bits are given in 1/64 bit (the 16-bit scale of a 1024-group is exactly
// 1/64 bit per weight, so 4.02 bits is 257/64), layer sizes are divided by their greatest common divisor.
#include "common.cuh"

#include <cmath>
#include <cstdlib>
#include <limits>
#include <new>
#include <vector>

namespace higgs {

namespace {
int64_t gcd64(int64_t a, int64_t b) { while (b) { const int64_t t = a % b; a = b; b = t; } return a; }
}  // namespace

int allocate_bits(int L, int J, const double* alpha, const double* t2, const int32_t* bits64, const int64_t* sizes,
                  int64_t budget64, int32_t* choice_out, double* objective_out) {
    if (L < 1 || J < 1 || !alpha || !t2 || !bits64 || !sizes || !choice_out) return HIGGS_ERR_INVALID_ARG;
    if (J > 255) return HIGGS_ERR_UNSUPPORTED;                  // the choice table stores one byte per state (255 = unset)
    if (budget64 < 0) return HIGGS_ERR_INVALID_ARG;
    try {
    int64_t g = 0, total = 0;
    for (int l = 0; l < L; ++l) {
        if (sizes[l] <= 0) return HIGGS_ERR_INVALID_ARG;
        g = gcd64(g, sizes[l]);
    }
    for (int j = 0; j < J; ++j)
        if (bits64[j] <= 0) return HIGGS_ERR_INVALID_ARG;
    std::vector<int64_t> unit(L);
    for (int l = 0; l < L; ++l) { unit[l] = sizes[l] / g; total += unit[l]; }
    // budget: sum_l bits64[j_l] * unit_l <= budget64 * total
    if (budget64 > std::numeric_limits<int64_t>::max() / total) return HIGGS_ERR_WORKSPACE;   // the product below would overflow
    const int64_t cap = budget64 * total;
    int64_t min_cost = 0;
    int minb = bits64[0];
    for (int j = 1; j < J; ++j) if (bits64[j] < minb) minb = bits64[j];
    for (int l = 0; l < L; ++l) min_cost += (int64_t)minb * unit[l];
    if (min_cost > cap) return HIGGS_ERR_UNSUPPORTED;           // infeasible: even the smallest option everywhere exceeds the budget
    if ((double)(cap + 1) * (double)L > 2.0e9) return HIGGS_ERR_WORKSPACE;   // table too large for this exact solver
    const size_t W = (size_t)cap + 1;
    const double inf = std::numeric_limits<double>::infinity();
    std::vector<double> cur(W, inf), nxt(W, inf);
    std::vector<uint8_t> pick((size_t)L * W, 255);
    cur[0] = 0.0;
    for (int l = 0; l < L; ++l) {
        std::fill(nxt.begin(), nxt.end(), inf);
        uint8_t* pk = pick.data() + (size_t)l * W;
        for (size_t c = 0; c < W; ++c) {
            if (cur[c] == inf) continue;
            for (int j = 0; j < J; ++j) {
                const int64_t c2 = (int64_t)c + (int64_t)bits64[j] * unit[l];
                if (c2 > cap) continue;
                const double v = cur[c] + alpha[l] * t2[(size_t)l * J + j];
                if (v < nxt[(size_t)c2]) { nxt[(size_t)c2] = v; pk[(size_t)c2] = (uint8_t)j; }   // ties: lowest option index
            }
        }
        cur.swap(nxt);
    }
    size_t best = 0;
    double bv = inf;
    for (size_t c = 0; c < W; ++c)
        if (cur[c] < bv) { bv = cur[c]; best = c; }               // ties: lowest total cost
    if (bv == inf) return HIGGS_ERR_UNSUPPORTED;
    int64_t c = (int64_t)best;
    for (int l = L - 1; l >= 0; --l) {
        const int j = pick[(size_t)l * W + (size_t)c];
        choice_out[l] = j;
        c -= (int64_t)bits64[j] * unit[l];
    }
    if (objective_out) *objective_out = bv;
    return HIGGS_OK;
    } catch (const std::bad_alloc&) {
        return HIGGS_ERR_WORKSPACE;                              // never let an exception cross the C boundary
    }
}

}  // namespace higgs
