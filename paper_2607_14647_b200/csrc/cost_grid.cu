// Start-up cost table C(B, rho) of the paper's deployment mode (Eq. 4-5; Appendix C, "Cost-table profiling protocol"):
// one row per captured batch size, one column per ratio bucket, each cell the median of a few step latencies.  At run
// time the row of the captured batch size nearest to the live one is read.  Host code only: the caller times the steps
// (dummy batches through the real pipeline) and records the samples here; dcut_set_cost_from_grid turns the row into
// the bucket table of dcut_select.
#include <math.h>
#include <stdlib.h>

#include <algorithm>
#include <vector>

#include "dcut_internal.h"

struct dcut_cost_grid {
    std::vector<int> batch;       // captured batch sizes, ascending
    std::vector<int> num, den;    // ratio buckets, ascending
    int gamma;
    std::vector<float> cost;      // [n_batch][n_ratios] ms; 0 = not recorded yet
};

extern "C" {

dcut_status dcut_cost_grid_create(dcut_cost_grid** out, const int* batch_sizes, int n_batch, const int* ratio_num,
                                  const int* ratio_den, int n_ratios, int gamma) {
    if (!out) return DCUT_EINVAL;
    *out = nullptr;
    if (!batch_sizes || !ratio_num || !ratio_den || n_batch < 1 || n_ratios < 1 || n_ratios > DCUT_MAX_BUCKETS || gamma < 1)
        return DCUT_EINVAL;
    for (int b = 0; b < n_batch; ++b)
        if (batch_sizes[b] < 1 || (b > 0 && batch_sizes[b] <= batch_sizes[b - 1])) return DCUT_EINVAL;
    for (int r = 0; r < n_ratios; ++r) {
        if (ratio_den[r] < 1 || ratio_num[r] < 1 || ratio_num[r] > ratio_den[r]) return DCUT_EINVAL;
        // ascending ratios, compared exactly: num[r-1] / den[r-1] < num[r] / den[r]
        if (r > 0 && (long long)ratio_num[r - 1] * ratio_den[r] >= (long long)ratio_num[r] * ratio_den[r - 1]) return DCUT_EINVAL;
    }
    dcut_cost_grid* g = new (std::nothrow) dcut_cost_grid();
    if (!g) return DCUT_EINVAL;
    g->batch.assign(batch_sizes, batch_sizes + n_batch);
    g->num.assign(ratio_num, ratio_num + n_ratios);
    g->den.assign(ratio_den, ratio_den + n_ratios);
    g->gamma = gamma;
    g->cost.assign((size_t)n_batch * n_ratios, 0.0f);
    *out = g;
    return DCUT_OK;
}

dcut_status dcut_cost_grid_destroy(dcut_cost_grid* g) {
    delete g;
    return DCUT_OK;
}

dcut_status dcut_cost_grid_budget(const dcut_cost_grid* g, int B, int r, int* K) {
    if (!g || !K || r < 0 || r >= (int)g->num.size() || B < 1) return DCUT_EINVAL;
    return dcut_budget_from_ratio(B, g->gamma, g->num[r], g->den[r], K);
}

dcut_status dcut_cost_grid_record(dcut_cost_grid* g, int b, int r, const float* samples_ms, int n) {
    if (!g || !samples_ms || n < 1 || b < 0 || b >= (int)g->batch.size() || r < 0 || r >= (int)g->num.size()) return DCUT_EINVAL;
    std::vector<float> v(samples_ms, samples_ms + n);
    for (float x : v)
        if (!(x > 0.0f) || isinf(x)) return DCUT_ECOST;
    std::sort(v.begin(), v.end());
    // median; an even count takes the mean of the two middle samples (in double, rounded once)
    const float med = (n & 1) ? v[n / 2] : (float)(((double)v[n / 2 - 1] + (double)v[n / 2]) * 0.5);
    g->cost[(size_t)b * g->num.size() + r] = med;
    return DCUT_OK;
}

dcut_status dcut_cost_grid_get(const dcut_cost_grid* g, int b, int r, float* cost_ms) {
    if (!g || !cost_ms || b < 0 || b >= (int)g->batch.size() || r < 0 || r >= (int)g->num.size()) return DCUT_EINVAL;
    *cost_ms = g->cost[(size_t)b * g->num.size() + r];
    return DCUT_OK;
}

dcut_status dcut_cost_grid_nearest(const dcut_cost_grid* g, int B, int* b_out) {
    if (!g || !b_out || B < 1) return DCUT_EINVAL;
    int best = 0;
    for (int b = 1; b < (int)g->batch.size(); ++b) {
        const long long d = llabs((long long)g->batch[b] - B), dbest = llabs((long long)g->batch[best] - B);
        if (d <= dbest) best = b;   // ascending sizes: on a tie the larger captured batch wins
    }
    *b_out = best;
    return DCUT_OK;
}

dcut_status dcut_cost_grid_buckets(const dcut_cost_grid* g, int B, int* K_out, float* cost_out, int* n_out) {
    if (!g || !K_out || !cost_out || !n_out || B < 1) return DCUT_EINVAL;
    int b = 0;
    dcut_cost_grid_nearest(g, B, &b);
    const int R = (int)g->num.size();
    int n = 0;
    for (int r = 0; r < R; ++r) {
        const float c = g->cost[(size_t)b * R + r];
        if (!(c > 0.0f)) return DCUT_ECOST;   // the row of the nearest captured batch size has a cell that was never recorded
        int K = 0;
        dcut_budget_from_ratio(B, g->gamma, g->num[r], g->den[r], &K);
        // Eq. 4's clamp and its ceiling can give two ratios the same budget at small B: one bucket, the cheaper latency
        if (n > 0 && K_out[n - 1] == K) {
            if (c < cost_out[n - 1]) cost_out[n - 1] = c;
        } else {
            K_out[n] = K;
            cost_out[n] = c;
            ++n;
        }
    }
    *n_out = n;
    return DCUT_OK;
}

dcut_status dcut_set_cost_from_grid(dcut_ctx* c, const dcut_cost_grid* g, int B) {
    if (!c) return DCUT_EINVAL;
    if (!g || B < 1) return dcut_fail(c, DCUT_EINVAL, "null cost grid or B < 1");
    int K[DCUT_MAX_BUCKETS], n = 0;
    float cost[DCUT_MAX_BUCKETS];
    dcut_status st = dcut_cost_grid_buckets(g, B, K, cost, &n);
    if (st == DCUT_ECOST) return dcut_fail(c, DCUT_ECOST, "the cost grid's row for the batch size nearest to %d is not fully recorded", B);
    if (st != DCUT_OK) return dcut_fail(c, st, "bad cost grid");
    return dcut_set_cost_buckets(c, B, g->gamma, K, cost, n);
}

}  // extern "C"
