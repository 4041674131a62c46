// Search-side host code of the ELSA method, data-free parts: the cost model F(alpha) (Sec. 3.2; the
// appendix's settings define F as FLOPs and C_upper as 50 % of the dense model's), the two-step sampling
// of a configuration (Alg. 3: an interval of the cost range drawn uniformly, then a configuration inside
// it drawn from the per-layer level probabilities P_t), and the enumeration of the search space
// (Sec. 2: 3 levels over 48 modules give 3^48 configurations).  No kernel lives here and no GPU is touched.
//
// Alg. 3 draws alpha from P_t restricted to the configurations whose cost lies in the chosen interval.
// Drawing level by level and rejecting until the cost fits does that, but hardly ever accepts in the
// outermost intervals; this file draws from exactly the same conditional distribution without rejection.
// Costs are quantised to integers, suffix[l][c] = probability that layers l.. cost c in total is built
// once by dynamic programming over the layers, and layer l takes level s with probability proportional
// to P[l][s] times the probability that the remaining layers land the total inside the interval.

#include <math.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <vector>

#include "elsa_internal.h"

namespace elsa {
namespace {

constexpr long long kMaxCostUnits = 1 << 22;   // width of the dynamic-programming table

struct CostGrid {
    std::vector<long long> units;   // [L][k] quantised costs
    long long min_total, max_total;
};

elsa_status quantise(const double* cost, int L, int k, double quantum, CostGrid* g)
{
    if (!(quantum > 0)) return fail(ELSA_ERR_SHAPE, "quantum must be positive");
    g->units.resize((size_t)L * k);
    g->min_total = 0;
    g->max_total = 0;
    for (int l = 0; l < L; ++l) {
        long long lo = 0, hi = 0;
        for (int s = 0; s < k; ++s) {
            const double c = cost[(size_t)l * k + s];
            if (!(c >= 0) || !isfinite(c)) return fail(ELSA_ERR_SHAPE, "cost of layer %d at level %d is negative or not finite", l, s);
            const long long u = llround(c / quantum);
            g->units[(size_t)l * k + s] = u;
            if (s == 0 || u < lo) lo = u;
            if (s == 0 || u > hi) hi = u;
        }
        g->min_total += lo;
        g->max_total += hi;
        if (g->max_total > kMaxCostUnits)
            return fail(ELSA_ERR_SHAPE, "cost range of more than %lld quanta: choose a coarser quantum", kMaxCostUnits);
    }
    return ELSA_OK;
}

elsa_status check_table(const double* cost, int L, int k, const double* P)
{
    if (!cost || !P) return fail(ELSA_ERR_NULL, "cost and P must not be NULL");
    if (L < 1 || k < 1) return fail(ELSA_ERR_SHAPE, "need at least one layer and one level (L=%d, k=%d)", L, k);
    for (int l = 0; l < L; ++l) {
        double sum = 0;
        for (int s = 0; s < k; ++s) {
            const double p = P[(size_t)l * k + s];
            if (!(p >= 0) || !isfinite(p)) return fail(ELSA_ERR_SHAPE, "P[%d][%d] is negative or not finite", l, s);
            sum += p;
        }
        if (!(sum > 0)) return fail(ELSA_ERR_SHAPE, "the level probabilities of layer %d are all zero", l);
    }
    return ELSA_OK;
}

// prefix[l][c] = sum over c' < c of the probability that layers l .. L-1 cost c' quanta in total
// (each layer's probabilities normalised to one); row l has width + 1 entries.
void suffix_prefix_sums(const CostGrid& g, int L, int k, const double* P, long long width, std::vector<double>* prefix)
{
    std::vector<double> cur((size_t)width, 0.0), next((size_t)width, 0.0);
    prefix->assign((size_t)(L + 1) * (size_t)(width + 1), 0.0);
    next[0] = 1.0;                                     // no layers left: cost 0 with certainty
    auto store = [&](int l, const std::vector<double>& row) {
        double* out = prefix->data() + (size_t)l * (size_t)(width + 1);
        double acc = 0;
        out[0] = 0;
        for (long long c = 0; c < width; ++c) { acc += row[(size_t)c]; out[c + 1] = acc; }
    };
    store(L, next);
    for (int l = L - 1; l >= 0; --l) {
        double norm = 0;
        for (int s = 0; s < k; ++s) norm += P[(size_t)l * k + s];
        std::fill(cur.begin(), cur.end(), 0.0);
        for (int s = 0; s < k; ++s) {
            const double p = P[(size_t)l * k + s] / norm;
            if (p == 0) continue;
            const long long u = g.units[(size_t)l * k + s];
            for (long long c = 0; c + u < width; ++c) cur[(size_t)(c + u)] += p * next[(size_t)c];
        }
        store(l, cur);
        std::swap(cur, next);
    }
}

double range_mass(const std::vector<double>& prefix, int l, long long width, long long lo, long long hi)   // [lo, hi)
{
    if (lo < 0) lo = 0;
    if (hi > width) hi = width;
    if (hi <= lo) return 0;
    const double* row = prefix.data() + (size_t)l * (size_t)(width + 1);
    return row[hi] - row[lo];
}

// Interval i (0-based, of n_intervals) of the cost range [c_lower, c_upper] in quanta, half open except the last,
// which includes c_upper (Sec. 3.2: configurations with F(alpha) <= C_upper are included).
void interval_bounds(long long lower, long long upper, int n_intervals, int i, long long* lo, long long* hi)
{
    const double w = (double)(upper - lower) / n_intervals;
    *lo = lower + (long long)ceil(i * w - 1e-9);
    *hi = i == n_intervals - 1 ? upper + 1 : lower + (long long)ceil((i + 1) * w - 1e-9);
}

}  // namespace
}  // namespace elsa

using namespace elsa;

extern "C" {

elsa_status elsa_cost_table_macs(const elsa_linear_shape* layers, int n_layers, const elsa_level* levels, int n_levels,
                                 double* cost)
{
    if (!layers || !levels || !cost) return fail(ELSA_ERR_NULL, "layers, levels and cost must not be NULL");
    if (n_layers < 1 || n_levels < 1) return fail(ELSA_ERR_SHAPE, "need at least one layer and one level");
    for (int s = 0; s < n_levels; ++s)
        if (index_bits(levels[s].M) < 0 || levels[s].N < 1 || levels[s].N > levels[s].M)
            return fail(ELSA_ERR_NM, "unsupported level %d:%d", levels[s].N, levels[s].M);
    for (int l = 0; l < n_layers; ++l) {
        const elsa_linear_shape& c = layers[l];
        if (c.rows <= 0 || c.in <= 0 || c.out <= 0) return fail(ELSA_ERR_SHAPE, "layer %d has a non-positive dimension", l);
        for (int s = 0; s < n_levels; ++s)
            cost[(size_t)l * n_levels + s] = (double)c.rows * (double)c.in * (double)c.out * (double)levels[s].N / (double)levels[s].M;
    }
    return ELSA_OK;
}

double elsa_config_cost(const double* cost, int n_layers, int n_levels, const int* choice, double fixed_cost)
{
    if (!cost || !choice || n_layers < 1 || n_levels < 1) return -1.0;
    double total = fixed_cost;
    for (int l = 0; l < n_layers; ++l) {
        if (choice[l] < 0 || choice[l] >= n_levels) return -1.0;
        total += cost[(size_t)l * n_levels + choice[l]];
    }
    return total;
}

elsa_status elsa_interval_masses(const double* cost, int n_layers, int n_levels, const double* P, double fixed_cost,
                                 double c_upper, int n_intervals, double quantum, double* mass)
{
    elsa_status st = check_table(cost, n_layers, n_levels, P);
    if (st != ELSA_OK) return st;
    if (!mass) return fail(ELSA_ERR_NULL, "mass must not be NULL");
    if (n_intervals < 1) return fail(ELSA_ERR_SHAPE, "need at least one interval");
    CostGrid g;
    if ((st = quantise(cost, n_layers, n_levels, quantum, &g)) != ELSA_OK) return st;
    const long long upper = (long long)floor((c_upper - fixed_cost) / quantum + 1e-9);
    if (upper < g.min_total) return fail(ELSA_ERR_SHAPE, "C_upper lies below the cost of the sparsest configuration");
    const long long width = g.max_total + 1;
    std::vector<double> prefix;
    suffix_prefix_sums(g, n_layers, n_levels, P, width, &prefix);
    for (int i = 0; i < n_intervals; ++i) {
        long long lo, hi;
        interval_bounds(g.min_total, upper, n_intervals, i, &lo, &hi);
        mass[i] = range_mass(prefix, 0, width, lo, hi);
    }
    return ELSA_OK;
}

elsa_status elsa_two_step_sample(const double* cost, int n_layers, int n_levels, const double* P, double fixed_cost,
                                 double c_upper, int n_intervals, double quantum, const double* uniforms, int* choice,
                                 int* interval)
{
    elsa_status st = check_table(cost, n_layers, n_levels, P);
    if (st != ELSA_OK) return st;
    if (!uniforms || !choice) return fail(ELSA_ERR_NULL, "uniforms and choice must not be NULL");
    if (n_intervals < 1) return fail(ELSA_ERR_SHAPE, "need at least one interval");
    for (int i = 0; i <= n_layers; ++i)
        if (!(uniforms[i] >= 0.0 && uniforms[i] < 1.0)) return fail(ELSA_ERR_SHAPE, "uniforms[%d] is outside [0, 1)", i);
    CostGrid g;
    if ((st = quantise(cost, n_layers, n_levels, quantum, &g)) != ELSA_OK) return st;
    const long long upper = (long long)floor((c_upper - fixed_cost) / quantum + 1e-9);
    if (upper < g.min_total) return fail(ELSA_ERR_SHAPE, "C_upper lies below the cost of the sparsest configuration");
    const long long width = g.max_total + 1;
    std::vector<double> prefix;
    suffix_prefix_sums(g, n_layers, n_levels, P, width, &prefix);

    // step 1: an interval, uniformly
    int iv = (int)(uniforms[0] * n_intervals);
    if (iv >= n_intervals) iv = n_intervals - 1;
    long long lo, hi;
    interval_bounds(g.min_total, upper, n_intervals, iv, &lo, &hi);
    if (interval) *interval = iv;
    if (!(range_mass(prefix, 0, width, lo, hi) > 0))
        return fail(ELSA_ERR_SHAPE, "no configuration with non-zero probability has its cost in interval %d", iv);

    // step 2: a configuration of that interval, level by level from the conditional distribution
    long long spent = 0;
    std::vector<double> w((size_t)n_levels);
    for (int l = 0; l < n_layers; ++l) {
        double total = 0;
        for (int s = 0; s < n_levels; ++s) {
            const long long u = g.units[(size_t)l * n_levels + s];
            w[(size_t)s] = P[(size_t)l * n_levels + s] * range_mass(prefix, l + 1, width, lo - spent - u, hi - spent - u);
            total += w[(size_t)s];
        }
        // inverse CDF over the levels in their given order
        const double target = uniforms[l + 1] * total;
        double acc = 0;
        int pick = -1;
        for (int s = 0; s < n_levels; ++s) {
            if (w[(size_t)s] <= 0) continue;
            acc += w[(size_t)s];
            pick = s;
            if (target < acc) break;
        }
        if (pick < 0) return fail(ELSA_ERR_SHAPE, "interval %d became unreachable at layer %d", iv, l);
        choice[l] = pick;
        spent += g.units[(size_t)l * n_levels + pick];
    }
    return ELSA_OK;
}

int elsa_search_space_size(int n_layers, int n_levels, char* out, size_t capacity)
{
    if (n_layers < 0 || n_levels < 1 || !out || capacity == 0) return -1;
    std::vector<uint32_t> limbs(1, 1u);              // base 10^9, little endian
    for (int l = 0; l < n_layers; ++l) {
        unsigned long long carry = 0;
        for (size_t i = 0; i < limbs.size(); ++i) {
            const unsigned long long v = (unsigned long long)limbs[i] * (unsigned long long)n_levels + carry;
            limbs[i] = (uint32_t)(v % 1000000000ull);
            carry = v / 1000000000ull;
        }
        while (carry) { limbs.push_back((uint32_t)(carry % 1000000000ull)); carry /= 1000000000ull; }
    }
    std::string text = std::to_string(limbs.back());
    for (size_t i = limbs.size() - 1; i-- > 0;) {
        char part[16];
        snprintf(part, sizeof part, "%09u", limbs[i]);
        text += part;
    }
    if (text.size() + 1 > capacity) return -1;
    memcpy(out, text.c_str(), text.size() + 1);
    return (int)text.size();
}

elsa_status elsa_config_from_index(const char* index_decimal, int n_layers, int n_levels, int* choice)
{
    if (!index_decimal || !choice) return fail(ELSA_ERR_NULL, "index and choice must not be NULL");
    if (n_layers < 1 || n_levels < 1) return fail(ELSA_ERR_SHAPE, "need at least one layer and one level");
    std::vector<uint32_t> limbs;                      // base 10^9, little endian
    const size_t len = strlen(index_decimal);
    if (len == 0) return fail(ELSA_ERR_SHAPE, "empty index");
    for (size_t i = 0; i < len; ++i)
        if (index_decimal[i] < '0' || index_decimal[i] > '9') return fail(ELSA_ERR_SHAPE, "the index is not a decimal number");
    for (size_t end = len; end > 0;) {
        const size_t begin = end >= 9 ? end - 9 : 0;
        uint32_t v = 0;
        for (size_t i = begin; i < end; ++i) v = v * 10u + (uint32_t)(index_decimal[i] - '0');
        limbs.push_back(v);
        end = begin;
    }
    // digit l of the index in base n_levels is the level of layer l (layer 0 = least significant)
    for (int l = 0; l < n_layers; ++l) {
        unsigned long long rem = 0;
        for (size_t i = limbs.size(); i-- > 0;) {
            const unsigned long long v = rem * 1000000000ull + limbs[i];
            limbs[i] = (uint32_t)(v / (unsigned long long)n_levels);
            rem = v % (unsigned long long)n_levels;
        }
        choice[l] = (int)rem;
    }
    for (size_t i = 0; i < limbs.size(); ++i)
        if (limbs[i] != 0) return fail(ELSA_ERR_SHAPE, "the index is not below %d^%d", n_levels, n_layers);
    return ELSA_OK;
}

}  // extern "C"
