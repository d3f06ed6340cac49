// Stage 2 of LExI (paper, Algorithm 2): choose the per-layer numbers of active experts
// k = (k_1..k_L) with sum_j k_j = B and k_min <= k_j <= k_max that minimise the proxy loss
// phi(k) = sum_j D_j(k_j), D being the Stage-1 perturbation table.  Host code only: the paper runs
// this search on the CPU without loading the model.
//
// Two solvers:
//   moe_lexi_allocate_exact         phi is separable, so the constrained minimum is a multiple-choice
//                                   knapsack: dynamic programme over (layer, budget), O(L B k_max).
//   moe_lexi_allocate_evolutionary  Algorithm 2 as printed: feasible initial population, tournament
//                                   selection, uniform crossover, zero-sum +-1 mutation, projection,
//                                   population grown by one child per generation, arg-min at the end.
// What Algorithm 2 leaves open is fixed as follows (the oracle takes the same steps):
//   - random numbers come from a caller-supplied stream of uint32, consumed in program order:
//     below(n) = next % n; coin = next & 1; chance(p) = next / 2^32 < p;
//   - an initial member starts at k_min everywhere and receives the remaining B - L k_min units one
//     at a time, each to below(#layers still under k_max)-th such layer in index order;
//   - a parent is the fittest of `tournament` members drawn with below(|P|) (first drawn wins ties);
//   - crossover: child_j = coin ? p1_j : p2_j for j = 0..L-1;
//   - mutation: with chance(eta_mut): a = below(L), b = below(L-1) skipping a; child_a += 1, child_b -= 1;
//   - projection: clip to [k_min, k_max]; while the sum exceeds B take one unit from the layer where
//     that raises phi least, while it is short add one where that lowers phi most (lowest index on ties);
//   - the result is the first member of P with the smallest phi.
#include <cstdint>
#include <limits>
#include <vector>

#include "moe.h"

namespace {

struct Stream {
    const uint32_t *v;
    int64_t n, pos = 0;
    bool ok = true;
    uint32_t next() {
        if (pos >= n) { ok = false; return 0; }
        return v[pos++];
    }
    int below(int m) { return (int)(next() % (uint32_t)m); }
    bool coin() { return (next() & 1u) != 0; }
    bool chance(double p) { return (double)next() / 4294967296.0 < p; }
};

struct Table {
    const double *D;
    int L, k_max;
    double at(int j, int k) const { return D[(size_t)j * k_max + (k - 1)]; }
    double phi(const int32_t *k) const {
        double s = 0.0;
        for (int j = 0; j < L; ++j) s += at(j, k[j]);
        return s;
    }
};

bool bad_problem(const double *D, int L, int k_max, int k_min, int budget) {
    return !D || L < 1 || k_max < 1 || k_min < 1 || k_min > k_max || budget < (int64_t)L * k_min ||
           budget > (int64_t)L * k_max;
}

void project(const Table &t, int k_min, int k_max, int budget, int32_t *k) {
    int sum = 0;
    for (int j = 0; j < t.L; ++j) {
        if (k[j] < k_min) k[j] = k_min;
        if (k[j] > k_max) k[j] = k_max;
        sum += k[j];
    }
    while (sum > budget) {
        int best = -1;
        double best_cost = 0.0;
        for (int j = 0; j < t.L; ++j) {
            if (k[j] <= k_min) continue;
            const double cost = t.at(j, k[j] - 1) - t.at(j, k[j]);
            if (best < 0 || cost < best_cost) { best = j; best_cost = cost; }
        }
        --k[best];
        --sum;
    }
    while (sum < budget) {
        int best = -1;
        double best_gain = 0.0;
        for (int j = 0; j < t.L; ++j) {
            if (k[j] >= k_max) continue;
            const double gain = t.at(j, k[j]) - t.at(j, k[j] + 1);
            if (best < 0 || gain > best_gain) { best = j; best_gain = gain; }
        }
        ++k[best];
        ++sum;
    }
}

}  // namespace

extern "C" {

int moe_lexi_allocate_exact(const double *D, int32_t L, int32_t k_max, int32_t k_min, int32_t budget,
                            int32_t *k_out, double *phi_out) {
    if (bad_problem(D, L, k_max, k_min, budget) || !k_out) return MOE_ERR_INVALID_ARG;
    const Table t{D, L, k_max};
    const double inf = std::numeric_limits<double>::infinity();
    // f[j][b]: least loss of layers 0..j-1 using exactly b units
    std::vector<double> f((size_t)(L + 1) * (budget + 1), inf);
    std::vector<int32_t> pick((size_t)(L + 1) * (budget + 1), 0);
    f[0] = 0.0;
    for (int j = 1; j <= L; ++j)
        for (int b = 0; b <= budget; ++b) {
            double best = inf;
            int arg = 0;
            for (int k = k_min; k <= k_max && k <= b; ++k) {
                const double prev = f[(size_t)(j - 1) * (budget + 1) + (b - k)];
                if (prev == inf) continue;
                const double v = prev + t.at(j - 1, k);
                if (v < best) { best = v; arg = k; }      // lowest k on ties
            }
            f[(size_t)j * (budget + 1) + b] = best;
            pick[(size_t)j * (budget + 1) + b] = arg;
        }
    if (f[(size_t)L * (budget + 1) + budget] == inf) return MOE_ERR_INVALID_ARG;
    int b = budget;
    for (int j = L; j >= 1; --j) {
        const int k = pick[(size_t)j * (budget + 1) + b];
        k_out[j - 1] = k;
        b -= k;
    }
    if (phi_out) *phi_out = t.phi(k_out);
    return MOE_OK;
}

int moe_lexi_allocate_evolutionary(const double *D, int32_t L, int32_t k_max, int32_t k_min, int32_t budget,
                                   int32_t n_pop, int32_t g_max, double eta_mut, int32_t tournament,
                                   const uint32_t *rnd, int64_t n_rnd, int32_t *k_out, double *phi_out) {
    if (bad_problem(D, L, k_max, k_min, budget) || !k_out || !rnd || n_rnd < 1 || n_pop < 1 || g_max < 0 ||
        tournament < 1 || eta_mut < 0.0 || eta_mut > 1.0)
        return MOE_ERR_INVALID_ARG;
    const Table t{D, L, k_max};
    Stream r{rnd, n_rnd};
    std::vector<int32_t> pop;            // members back to back, L entries each
    std::vector<double> fit;
    pop.reserve((size_t)(n_pop + g_max) * L);
    std::vector<int32_t> open(L), child(L);
    for (int i = 0; i < n_pop; ++i) {
        std::vector<int32_t> k(L, k_min);
        for (int u = budget - L * k_min; u > 0; --u) {
            int n_open = 0;
            for (int j = 0; j < L; ++j)
                if (k[j] < k_max) open[n_open++] = j;
            ++k[open[r.below(n_open)]];
        }
        pop.insert(pop.end(), k.begin(), k.end());
        fit.push_back(t.phi(k.data()));
    }
    for (int g = 0; g < g_max; ++g) {
        int parent[2];
        for (int q = 0; q < 2; ++q) {
            int best = -1;
            for (int c = 0; c < tournament; ++c) {
                const int m = r.below((int)fit.size());
                if (best < 0 || fit[m] < fit[best]) best = m;
            }
            parent[q] = best;
        }
        const int32_t *p1 = &pop[(size_t)parent[0] * L], *p2 = &pop[(size_t)parent[1] * L];
        for (int j = 0; j < L; ++j) child[j] = r.coin() ? p1[j] : p2[j];
        if (L >= 2 && r.chance(eta_mut)) {
            const int a = r.below(L);
            int b = r.below(L - 1);
            if (b >= a) ++b;
            ++child[a];
            --child[b];
        }
        project(t, k_min, k_max, budget, child.data());
        pop.insert(pop.end(), child.begin(), child.end());
        fit.push_back(t.phi(child.data()));
        if (!r.ok) return MOE_ERR_INVALID_ARG;     // the random stream ran out
    }
    if (!r.ok) return MOE_ERR_INVALID_ARG;
    int best = 0;
    for (int m = 1; m < (int)fit.size(); ++m)
        if (fit[m] < fit[best]) best = m;
    for (int j = 0; j < L; ++j) k_out[j] = pop[(size_t)best * L + j];
    if (phi_out) *phi_out = fit[best];
    return MOE_OK;
}

}  // extern "C"
