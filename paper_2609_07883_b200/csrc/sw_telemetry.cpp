// Telemetry of the serving loop (Table 1 "Telemetry"; Sec. 3.3 "Prediction error"; Sec. 5.1): predicted and observed
// iteration durations feed an empirical high-percentile residual table, which gives the margin delta(n, c) the
// scheduler reserves and the signal for falling back to decode-only iterations.  Host only.
#include <algorithm>
#include <cstdint>
#include <new>
#include <vector>

#include "sw.h"
#include "sw_error.h"

struct sw_telemetry {
    std::vector<int32_t> n_edges, c_edges;
    int32_t window = 0;
    // per bucket: ring of the most recent residuals
    struct Ring {
        std::vector<int64_t> v;
        int32_t next = 0;   // slot the next residual goes to once the ring is full
    };
    std::vector<Ring> rings;  // [n bucket][c bucket]
    sw_telemetry_totals totals{};
};

namespace {

// first bucket whose upper edge is >= value; values beyond the last edge fall into the last bucket
int32_t bucket_of(const std::vector<int32_t>& edges, int64_t value) {
    const auto it = std::lower_bound(edges.begin(), edges.end(), value,
                                     [](int32_t e, int64_t v) { return (int64_t)e < v; });
    return it == edges.end() ? (int32_t)edges.size() - 1 : (int32_t)(it - edges.begin());
}

bool strictly_increasing(const int32_t* e, int32_t k) {
    for (int32_t i = 1; i < k; ++i)
        if (e[i] <= e[i - 1]) return false;
    return true;
}

// nearest rank: the ceil(p * N)-th smallest (at least the first)
int64_t nearest_rank(std::vector<int64_t> v, int32_t percentile_ppm) {
    const int64_t n = (int64_t)v.size();
    int64_t rank = ((int64_t)percentile_ppm * n + 999999) / 1000000;
    rank = std::min(std::max<int64_t>(rank, 1), n);
    std::nth_element(v.begin(), v.begin() + (rank - 1), v.end());
    return v[(size_t)(rank - 1)];
}

int64_t margin_of(const sw_telemetry& t, int64_t n, int64_t c, int32_t percentile_ppm, int32_t min_samples, int64_t floor_ns) {
    const int32_t bi = bucket_of(t.n_edges, n), bj = bucket_of(t.c_edges, c);
    const int32_t need = std::max(min_samples, 1);
    int64_t best = INT64_MIN;
    for (int32_t i = 0; i <= bi; ++i)
        for (int32_t j = 0; j <= bj; ++j) {
            const auto& ring = t.rings[(size_t)i * t.c_edges.size() + j];
            const int64_t v = (int32_t)ring.v.size() >= need ? nearest_rank(ring.v, percentile_ppm) : floor_ns;
            best = std::max(best, v);
        }
    return best;
}

}  // namespace

extern "C" {

sw_status sw_telemetry_create(const int32_t* n_edges, int32_t num_n, const int32_t* c_edges, int32_t num_c, int32_t window,
                              sw_telemetry** out) {
    if (!n_edges || !c_edges || !out || num_n < 1 || num_c < 1 || window < 1)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_telemetry_create: invalid argument");
    if (!strictly_increasing(n_edges, num_n) || !strictly_increasing(c_edges, num_c))
        return sw_fail(SW_ERR_INVALID_ARG, "sw_telemetry_create: bucket edges must be strictly increasing");
    sw_telemetry* t = new (std::nothrow) sw_telemetry();
    if (!t) return sw_fail(SW_ERR_INVALID_ARG, "sw_telemetry_create: out of host memory");
    t->n_edges.assign(n_edges, n_edges + num_n);
    t->c_edges.assign(c_edges, c_edges + num_c);
    t->window = window;
    t->rings.resize((size_t)num_n * num_c);
    *out = t;
    return SW_OK;
}

void sw_telemetry_destroy(sw_telemetry* t) { delete t; }

sw_status sw_telemetry_record(sw_telemetry* t, int32_t n, int32_t c, int64_t predicted_ns, int64_t observed_ns, int64_t slack_ns,
                              int32_t fallback) {
    if (!t || n < 0 || c < 0) return sw_fail(SW_ERR_INVALID_ARG, "sw_telemetry_record: invalid argument");
    auto& ring = t->rings[(size_t)bucket_of(t->n_edges, n) * t->c_edges.size() + bucket_of(t->c_edges, c)];
    const int64_t r = std::max<int64_t>(0, observed_ns - predicted_ns);
    if ((int32_t)ring.v.size() < t->window) {
        ring.v.push_back(r);
    } else {
        ring.v[(size_t)ring.next] = r;   // overwrites the oldest
        ring.next = (ring.next + 1) % t->window;
    }
    t->totals.records += 1;
    t->totals.fallbacks += fallback ? 1 : 0;
    t->totals.deadline_misses += slack_ns < 0 ? 1 : 0;
    t->totals.max_residual_ns = std::max(t->totals.max_residual_ns, r);
    return SW_OK;
}

sw_status sw_telemetry_margin(const sw_telemetry* t, int32_t n, int32_t c, int32_t percentile_ppm, int32_t min_samples,
                              int64_t floor_ns, int64_t* margin_ns) {
    if (!t || !margin_ns || n < 0 || c < 0 || percentile_ppm < 1 || percentile_ppm > 1000000)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_telemetry_margin: invalid argument");
    *margin_ns = margin_of(*t, n, c, percentile_ppm, min_samples, floor_ns);
    return SW_OK;
}

sw_status sw_telemetry_exceeds(const sw_telemetry* t, int32_t n, int32_t c, int32_t percentile_ppm, int32_t min_samples,
                               int64_t configured_margin_ns, int32_t* exceeds) {
    if (!t || !exceeds || n < 0 || c < 0 || percentile_ppm < 1 || percentile_ppm > 1000000)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_telemetry_exceeds: invalid argument");
    *exceeds = margin_of(*t, n, c, percentile_ppm, min_samples, 0) > configured_margin_ns ? 1 : 0;
    return SW_OK;
}

sw_status sw_telemetry_reset(sw_telemetry* t) {
    if (!t) return sw_fail(SW_ERR_INVALID_ARG, "sw_telemetry_reset: null argument");
    for (auto& ring : t->rings) {
        ring.v.clear();
        ring.next = 0;
    }
    return SW_OK;
}

sw_status sw_telemetry_get_totals(const sw_telemetry* t, sw_telemetry_totals* out) {
    if (!t || !out) return sw_fail(SW_ERR_INVALID_ARG, "sw_telemetry_get_totals: invalid argument");
    *out = t->totals;
    return SW_OK;
}

}  // extern "C"
