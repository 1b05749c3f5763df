// Host controller: monotone cost table and the deadline-aware chunk chooser (Algorithm 1).
// Pure host code; integer-nanosecond arithmetic so that ties are exact.
#include <algorithm>
#include <cstdint>
#include <cstdio>
#include <limits>
#include <new>
#include <vector>

#include "sw.h"
#include "sw_error.h"

struct sw_cost_table {
    std::vector<int32_t> n_grid;
    std::vector<int64_t> ctx_grid;
    std::vector<int32_t> prefix_grid;
    std::vector<int32_t> chunk_grid;
    std::vector<int64_t> cost;  // [nn][nc][np][nk]
    bool interp = false;

    size_t at(size_t a, size_t b, size_t c, size_t e) const {
        return ((a * ctx_grid.size() + b) * prefix_grid.size() + c) * chunk_grid.size() + e;
    }
};

namespace {

constexpr int64_t kInf = std::numeric_limits<int64_t>::max();

template <class T>
bool strictly_increasing(const std::vector<T>& g) {
    for (size_t i = 1; i < g.size(); ++i)
        if (!(g[i - 1] < g[i])) return false;
    return true;
}

// Running maximum along one axis of the 4-D table; returns true if anything changed.
bool running_max_axis(sw_cost_table& t, int axis) {
    const size_t dims[4] = {t.n_grid.size(), t.ctx_grid.size(), t.prefix_grid.size(), t.chunk_grid.size()};
    bool changed = false;
    size_t idx[4];
    for (idx[0] = 0; idx[0] < dims[0]; ++idx[0])
        for (idx[1] = 0; idx[1] < dims[1]; ++idx[1])
            for (idx[2] = 0; idx[2] < dims[2]; ++idx[2])
                for (idx[3] = 0; idx[3] < dims[3]; ++idx[3]) {
                    if (idx[axis] == 0) continue;
                    size_t prev[4] = {idx[0], idx[1], idx[2], idx[3]};
                    prev[axis] -= 1;
                    int64_t& cur = t.cost[t.at(idx[0], idx[1], idx[2], idx[3])];
                    const int64_t before = t.cost[t.at(prev[0], prev[1], prev[2], prev[3])];
                    if (cur < before) {
                        cur = before;
                        changed = true;
                    }
                }
    return changed;
}

// delta(T) = margin_abs + ceil(T * ppm / 1e6); infinity stays infinity.
int64_t add_margin(int64_t t, const sw_chooser_params& p) {
    if (t == kInf) return kInf;
    const __int128 rel = ((__int128)t * p.margin_ppm + 999999) / 1000000;
    const __int128 sum = (__int128)t + p.margin_abs_ns + rel;
    return sum >= (__int128)kInf ? kInf : (int64_t)sum;
}

// index of the first grid point >= x, or grid.size() when x lies beyond the grid
template <class T>
size_t round_up_index(const std::vector<T>& grid, int64_t x) {
    return (size_t)(std::lower_bound(grid.begin(), grid.end(), x,
                                     [](const T& g, int64_t v) { return (int64_t)g < v; }) -
                    grid.begin());
}

sw_status lookup(const sw_cost_table& t, int64_t n, int64_t ctx, int64_t prefix, int64_t c, int64_t* out) {
    const size_t a = round_up_index(t.n_grid, n);
    const size_t b = round_up_index(t.ctx_grid, ctx);
    const size_t p = round_up_index(t.prefix_grid, prefix);
    if (a == t.n_grid.size() || b == t.ctx_grid.size() || p == t.prefix_grid.size())
        return sw_fail(SW_ERR_OUT_OF_RANGE, "cost lookup: n=%lld ctx=%lld prefix=%lld beyond the table grid",
                       (long long)n, (long long)ctx, (long long)prefix);
    const size_t e = round_up_index(t.chunk_grid, c);
    if (e == t.chunk_grid.size()) {
        *out = kInf;
        return SW_OK;
    }
    const int64_t hi = t.cost[t.at(a, b, p, e)];
    if (!t.interp || e == 0 || (int64_t)t.chunk_grid[e] == c) {
        *out = hi;
        return SW_OK;
    }
    const int64_t lo = t.cost[t.at(a, b, p, e - 1)];
    const int64_t c_lo = t.chunk_grid[e - 1], c_hi = t.chunk_grid[e];
    const __int128 rise = (__int128)(hi - lo) * (c - c_lo);
    const __int128 span = c_hi - c_lo;
    *out = lo + (int64_t)((rise + span - 1) / span);  // hi >= lo: table is monotone
    return SW_OK;
}

// Largest raw cost t whose margin still fits the budget: t + margin_abs + ceil(t * ppm / 1e6) <= B (-1 if none).
int64_t largest_raw_cost_within(int64_t B, const sw_chooser_params& p) {
    const __int128 room = (__int128)B - p.margin_abs_ns;
    if (room < 0) return -1;
    __int128 t = room * 1000000 / (1000000 + (__int128)p.margin_ppm);  // estimate; the ceiling is settled below
    auto fits = [&](__int128 v) { return v + (v * p.margin_ppm + 999999) / 1000000 <= room; };
    while (t >= 0 && !fits(t)) --t;
    while (fits(t + 1)) ++t;
    return t >= (__int128)kInf ? kInf - 1 : (int64_t)t;
}

// The search of Sec. 3.2 organised around the table instead of around the candidates.  One iteration is asked for
// `offset` prefill tokens already (first fit; 0 for a single prefill) plus c more, c a positive multiple of q with
// c <= K * q.  The predicted cost of offset + c tokens is constant (or, with interpolation, linear) between two
// neighbouring points of the chunk grid, and nondecreasing from point to point.  So: (1) bisect over the grid POINTS
// that the candidates can round up to for the last one whose cost plus margin meets the budget B; (2) every candidate up
// to that point is feasible; with interpolation the stretch towards the next point may hold more, and the last
// feasible token count there follows from one division; (3) the answer is the largest candidate not beyond that.
// Returns c (0 when no candidate is feasible); *predicted is set to the cost plus margin at the answer when c > 0.
// By Proposition 1 this is the maximiser of Eq. (1); the parity tests compare it with the exhaustive scan.
sw_status largest_feasible(const sw_cost_table& t, const sw_chooser_params& params, int64_t n, int64_t ctx, int64_t prefix,
                           int64_t offset, int32_t K, int32_t q, int64_t B, int32_t* c_out, int64_t* predicted,
                           int32_t* queries) {
    *c_out = 0;
    if (K <= 0) return SW_OK;
    const size_t a = round_up_index(t.n_grid, n);
    const size_t b = round_up_index(t.ctx_grid, ctx);
    const size_t p = round_up_index(t.prefix_grid, prefix);
    if (a == t.n_grid.size() || b == t.ctx_grid.size() || p == t.prefix_grid.size())
        return sw_fail(SW_ERR_OUT_OF_RANGE, "cost lookup: n=%lld ctx=%lld prefix=%lld beyond the table grid", (long long)n,
                       (long long)ctx, (long long)prefix);
    const int64_t* row = &t.cost[t.at(a, b, p, 0)];
    const std::vector<int32_t>& grid = t.chunk_grid;
    const int64_t nk = (int64_t)grid.size();
    const int64_t x_first = offset + q, x_last = offset + (int64_t)K * q;   // smallest and largest candidate total
    const int64_t raw_max = largest_raw_cost_within(B, params);            // a raw cost fits iff it is <= raw_max
    // grid points the candidates round up to: [ea, eb]; index nk stands for "beyond the grid" (infinite cost)
    const int64_t ea = (int64_t)round_up_index(grid, x_first), eb = (int64_t)round_up_index(grid, x_last);
    int64_t lo = ea - 1, hi = eb;  // invariant: points <= lo fit (or lo == ea - 1), points > hi do not
    while (lo < hi) {
        const int64_t mid = lo + (hi - lo + 1) / 2;
        *queries += 1;
        if (mid < nk && row[mid] <= raw_max) lo = mid; else hi = mid - 1;
    }
    int64_t x_best = lo >= ea ? (lo == nk ? x_last : std::min<int64_t>(grid[(size_t)lo], x_last)) : 0;  // 0: none so far
    if (lo == eb && lo < nk) x_best = x_last;  // the last candidate itself rounds up to a point that fits
    if (t.interp && x_best < x_last && lo >= 0 && lo + 1 < nk && row[lo] <= raw_max) {
        // between grid[lo] and grid[lo + 1]: cost = row[lo] + ceil((row[lo+1] - row[lo]) * dx / span) <= raw_max
        const int64_t rise = row[lo + 1] - row[lo], span = (int64_t)grid[(size_t)lo + 1] - grid[(size_t)lo];
        const __int128 room = (__int128)raw_max - row[lo];
        const int64_t dx = rise <= 0 ? span : (int64_t)std::min<__int128>(span, room * span / rise);
        x_best = std::max(x_best, std::min<int64_t>(grid[(size_t)lo] + dx, x_last));
    }
    if (x_best < x_first) return SW_OK;
    const int32_t c = (int32_t)((x_best - offset) / q) * q;
    int64_t raw = 0;
    sw_status st = lookup(t, n, ctx, prefix, offset + c, &raw);
    if (st != SW_OK) return st;
    *c_out = c;
    *predicted = add_margin(raw, params);
    return SW_OK;
}

}  // namespace

extern "C" {

sw_status sw_cost_table_create(const int32_t* n_grid, int32_t nn, const int64_t* ctx_grid, int32_t nc,
                               const int32_t* prefix_grid, int32_t np, const int32_t* chunk_grid, int32_t nk,
                               const int64_t* cost_ns, int make_monotone, int interp, sw_cost_table** out) {
    if (!n_grid || !ctx_grid || !prefix_grid || !chunk_grid || !cost_ns || !out)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_cost_table_create: null argument");
    if (nn < 1 || nc < 1 || np < 1 || nk < 1)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_cost_table_create: every axis needs at least one grid point");
    sw_cost_table* t = new (std::nothrow) sw_cost_table();
    if (!t) return sw_fail(SW_ERR_INVALID_ARG, "sw_cost_table_create: out of host memory");
    t->n_grid.assign(n_grid, n_grid + nn);
    t->ctx_grid.assign(ctx_grid, ctx_grid + nc);
    t->prefix_grid.assign(prefix_grid, prefix_grid + np);
    t->chunk_grid.assign(chunk_grid, chunk_grid + nk);
    t->cost.assign(cost_ns, cost_ns + (size_t)nn * nc * np * nk);
    t->interp = interp != 0;
    bool ok = strictly_increasing(t->n_grid) && strictly_increasing(t->ctx_grid) &&
              strictly_increasing(t->prefix_grid) && strictly_increasing(t->chunk_grid) && t->chunk_grid[0] >= 0 &&
              t->n_grid[0] >= 0 && t->ctx_grid[0] >= 0 && t->prefix_grid[0] >= 0;
    for (int64_t v : t->cost) ok = ok && v >= 0 && v < (int64_t(1) << 62);
    if (!ok) {
        delete t;
        return sw_fail(SW_ERR_INVALID_ARG,
                       "sw_cost_table_create: grids must be non-negative and strictly increasing, costs in [0, 2^62)");
    }
    // chunk axis first (the profiler's rule), then prefix, ctx, n; repeat until stable so that the result is
    // nondecreasing along every axis at once.
    bool changed = false;
    for (int round = 0; round < 8; ++round) {
        bool any = false;
        for (int axis = 3; axis >= 0; --axis) any = running_max_axis(*t, axis) || any;
        changed = changed || any;
        if (!any) break;
    }
    if (changed && !make_monotone) {
        delete t;
        return sw_fail(SW_ERR_NOT_MONOTONE, "sw_cost_table_create: table is not nondecreasing and make_monotone == 0");
    }
    *out = t;
    return SW_OK;
}

void sw_cost_table_destroy(sw_cost_table* table) { delete table; }

sw_status sw_cost_table_lookup(const sw_cost_table* table, int64_t n, int64_t ctx, int64_t prefix, int64_t c,
                               int64_t* cost_ns) {
    if (!table || !cost_ns) return sw_fail(SW_ERR_INVALID_ARG, "sw_cost_table_lookup: null argument");
    if (n < 0 || ctx < 0 || prefix < 0 || c < 0)
        return sw_fail(SW_ERR_INVALID_ARG, "sw_cost_table_lookup: negative coordinate");
    return lookup(*table, n, ctx, prefix, c, cost_ns);
}

sw_status sw_choose_chunk(const sw_cost_table* table, const sw_chooser_params* params, int64_t now_ns,
                          const int64_t* deadlines_ns, int32_t n_active, int64_t total_ctx, int32_t prefix_len,
                          int32_t remaining_prefill, sw_choice* out) {
    if (!params || !out) return sw_fail(SW_ERR_INVALID_ARG, "sw_choose_chunk: null argument");
    if (n_active < 0 || remaining_prefill < 0 || prefix_len < 0 || total_ctx < 0 || params->c_max < 0 ||
        params->margin_ppm < 0 || params->margin_abs_ns < 0 || (n_active > 0 && !deadlines_ns))
        return sw_fail(SW_ERR_INVALID_ARG, "sw_choose_chunk: negative size or missing deadlines");
    // Sec. 3.2 / Algorithm 1 as one call of the first-fit routine with a single pending request: nothing pending gives
    // 0, no active decode gives the capped remainder, otherwise the largest chunk whose predicted cost meets the budget.
    int32_t chunk = 0, count = 0;
    return sw_choose_chunks(table, params, now_ns, deadlines_ns, n_active, total_ctx, &prefix_len, &remaining_prefill, 1, &chunk,
                            &count, out);
}

// Several prefills per iteration by first fit (Sec. 3.3): requests oldest first, each admitted whole while the
// prediction for the total still meets the budget; the first one that does not fit whole gets the largest feasible part
// and ends the list.  A decode-only iteration processes no prompt, so its cost (the c = 0 column, which decides
// SW_F_DECODE_INFEASIBLE) is read at prefix 0 whatever the pending requests' prefixes are.
sw_status sw_choose_chunks(const sw_cost_table* table, const sw_chooser_params* params, int64_t now_ns,
                           const int64_t* deadlines_ns, int32_t n_active, int64_t total_ctx, const int32_t* prefix_lens,
                           const int32_t* remaining_prefill, int32_t num_pending, int32_t* chunks, int32_t* num_chunks,
                           sw_choice* out) {
    if (!params || !out || !chunks || !num_chunks || num_pending < 0 || (num_pending > 0 && (!prefix_lens || !remaining_prefill)))
        return sw_fail(SW_ERR_INVALID_ARG, "sw_choose_chunks: null argument");
    if (n_active < 0 || total_ctx < 0 || params->c_max < 0 || params->margin_ppm < 0 || params->margin_abs_ns < 0 ||
        (n_active > 0 && !deadlines_ns))
        return sw_fail(SW_ERR_INVALID_ARG, "sw_choose_chunks: negative size or missing deadlines");
    for (int32_t j = 0; j < num_pending; ++j)
        if (prefix_lens[j] < 0 || remaining_prefill[j] < 0)
            return sw_fail(SW_ERR_INVALID_ARG, "sw_choose_chunks: negative length of pending request %d", j);
    const int32_t q = params->chunk_quantum > 1 ? params->chunk_quantum : 1;
    *out = sw_choice{0, 0, 0, 0, 0};
    *num_chunks = 0;
    if (num_pending == 0 || remaining_prefill[0] == 0) {
        out->flags = SW_F_NO_PREFILL;
        return SW_OK;
    }
    if (params->c_max < remaining_prefill[0]) out->flags |= SW_F_CAPPED;
    int64_t B = 0;
    if (n_active > 0) {
        if (!table) return sw_fail(SW_ERR_INVALID_ARG, "sw_choose_chunks: a cost table is required when decodes are active");
        const int64_t earliest = *std::min_element(deadlines_ns, deadlines_ns + n_active);
        B = earliest > now_ns ? earliest - now_ns : 0;   // the clamp of Sec. 3.1
        out->budget_ns = B;
        int64_t t_raw = 0;
        sw_status st = lookup(*table, n_active, total_ctx, 0, 0, &t_raw);
        if (st != SW_OK) return st;
        const int64_t decode_only = add_margin(t_raw, *params);
        if (decode_only > B) out->flags |= SW_F_DECODE_INFEASIBLE;
        out->predicted_ns = decode_only;
    } else {
        out->flags |= SW_F_NO_DECODE;
    }
    int64_t tokens = 0, prefix_sum = 0;
    const int32_t limit = std::min<int32_t>(num_pending, SW_MAX_CHUNKS);
    for (int32_t j = 0; j < limit; ++j) {
        const int64_t room = (int64_t)params->c_max - tokens;
        const int32_t L = (int32_t)std::min<int64_t>(room, remaining_prefill[j]);
        if (L <= 0) break;
        if (room < remaining_prefill[j]) out->flags |= SW_F_CAPPED;
        int32_t c = 0;
        if (n_active == 0) {
            c = L - L % q;   // no deadline to meet: the table is not consulted
        } else {
            int64_t predicted = 0;
            sw_status st = largest_feasible(*table, *params, n_active, total_ctx, prefix_sum + prefix_lens[j], tokens, L / q, q, B,
                                            &c, &predicted, &out->queries);
            if (st != SW_OK) return st;
            if (c > 0) out->predicted_ns = predicted;
        }
        if (c == 0) break;
        chunks[*num_chunks] = c;
        *num_chunks += 1;
        tokens += c;
        prefix_sum += prefix_lens[j];
        if (c < remaining_prefill[j]) break;
    }
    out->chunk = (int32_t)tokens;
    return SW_OK;
}

}  // extern "C"
