/*
 * CPU oracle for the mixed prefill-chunk + decode attention iteration and the SLOWeave chunk chooser.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64, obviously-correct restatements of what the hot path
 * computes.  Nothing here is shared with, included by, or called from the CUDA library; only the
 * tests, the smoke check and the bench's cpu_baseline / reference legs may execute it.
 *
 * What each function follows:
 *   swo_pool_index, swo_kv_append   the paged KV cache as persistent state whose blocks are filled as
 *                                   each chunk completes (Table 1, "KV manager"; Fig. 1 card 5).  The
 *                                   paper fixes no layout; the one used is [page][K|V][kv head][slot][e].
 *   swo_attend_row, swo_mixed_attention, swo_dense_causal
 *                                   scaled-dot-product attention, whole-row two-pass softmax.  The
 *                                   paper leaves attention kernels untouched (Sec. 1, Sec. 5.1), so
 *                                   the oracle is the textbook definition written out; one iteration
 *                                   = one prefill chunk + one token per active decode (Sec. 4.1).
 *   swo_cost_lookup                 lookup table keyed by decode batch, total cached context and
 *                                   candidate prefill tokens (Sec. 5.1), plus a prefix-length axis.
 *   swo_cummax                      cumulative maximum along the chunk axis (Sec. 5.1, Sec. 6.4).
 *   swo_choose_bruteforce           Eq. (1): the maximum feasible chunk, by linear scan; the budget
 *                                   is the clamped earliest slack of Sec. 3.1; margin as in Sec. 3.3.
 *   swo_analytic_cost_ns            the simulator's analytic cost model (Sec. 4.1), in integer ns.
 *
 * Pins (tests/test_oracle_*.py): softmax rows sum to 1; chunk invariance; paged == dense unpaged ==
 * numpy float64 dense softmax; length-1 rows return V[0]; V==1 -> 1; K==const -> mean of V; causal
 * inclusivity closed form; GQA head mapping; closed-form chunk under the analytic model; the worked
 * cumulative-maximum example; brute force vs an independent python set-definition of Eq. (1).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define SWO_OK 0
#define SWO_ERR_ARG 1
#define SWO_ERR_RANGE 2
#define SWO_INF INT64_MAX

/* ---------------------------------------------------------------------------------------------- */
/* bf16 bits -> double (lossless widening)                                                         */
/* ---------------------------------------------------------------------------------------------- */
static double bf16_to_double(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ---------------------------------------------------------------------------------------------- */
/* paging                                                                                          */
/* ---------------------------------------------------------------------------------------------- */
/* element index of (page, x = 0 for K / 1 for V, kv head, slot in page, element e) */
int64_t swo_pool_index(int64_t page, int x, int kvh, int slot, int e, int Hkv, int S, int d)
{
    return ((((int64_t)page * 2 + x) * Hkv + kvh) * S + slot) * d + e;
}

/* Scatter k_new / v_new rows [C+n][Hkv][d] into the pool.  Chunk row j goes to prompt position P+j;
 * decode row i goes to position L_i - 1 of request i.  Returns SWO_ERR_RANGE on a page id outside the
 * pool or a page list too short for the position. */
int swo_kv_append(uint16_t* pool, int64_t num_pages, int Hkv, int S, int d,
                  const uint16_t* k_new, const uint16_t* v_new,
                  int P, int C, const int32_t* prefill_pages, int num_prefill_pages,
                  int n, const int32_t* decode_kv_len, const int32_t* indptr, const int32_t* decode_pages)
{
    for (int row = 0; row < C + n; ++row) {
        int64_t t;
        const int32_t* pages;
        int npages;
        if (row < C) {
            t = (int64_t)P + row;
            pages = prefill_pages;
            npages = num_prefill_pages;
        } else {
            int i = row - C;
            if (decode_kv_len[i] < 1) return SWO_ERR_ARG;
            t = (int64_t)decode_kv_len[i] - 1;
            pages = decode_pages + indptr[i];
            npages = indptr[i + 1] - indptr[i];
        }
        int64_t pi = t / S;
        int slot = (int)(t % S);
        if (pi >= npages) return SWO_ERR_RANGE;
        int64_t page = pages[pi];
        if (page < 0 || page >= num_pages) return SWO_ERR_RANGE;
        for (int h = 0; h < Hkv; ++h)
            for (int e = 0; e < d; ++e) {
                int64_t src = ((int64_t)row * Hkv + h) * d + e;
                pool[swo_pool_index(page, 0, h, slot, e, Hkv, S, d)] = k_new[src];
                pool[swo_pool_index(page, 1, h, slot, e, Hkv, S, d)] = v_new[src];
            }
    }
    return SWO_OK;
}

/* ---------------------------------------------------------------------------------------------- */
/* attention                                                                                       */
/* ---------------------------------------------------------------------------------------------- */
/* One query row (one q head) attending keys 0..kv_len-1 of a paged sequence, KV head kvh.
 * q: d bf16 values.  out: d doubles.  lse = m + ln Z.  psum = sum of the softmax probabilities.
 * scratch: kv_len doubles. */
static int attend_row(const uint16_t* pool, int64_t num_pages, int Hkv, int S, int d,
                      const int32_t* pages, int npages, int kv_len, const uint16_t* q, int kvh,
                      double scale, double* out, double* lse, double* psum, double* scratch)
{
    if (kv_len < 1) return SWO_ERR_ARG;
    if ((int64_t)(kv_len - 1) / S >= npages) return SWO_ERR_RANGE;
    double m = -INFINITY;
    for (int t = 0; t < kv_len; ++t) {
        int64_t page = pages[t / S];
        if (page < 0 || page >= num_pages) return SWO_ERR_RANGE;
        int slot = t % S;
        double acc = 0.0;
        for (int e = 0; e < d; ++e)
            acc += bf16_to_double(q[e]) * bf16_to_double(pool[swo_pool_index(page, 0, kvh, slot, e, Hkv, S, d)]);
        double s = acc * scale;
        scratch[t] = s;
        if (s > m) m = s;
    }
    double Z = 0.0;
    for (int t = 0; t < kv_len; ++t) {
        scratch[t] = exp(scratch[t] - m);
        Z += scratch[t];
    }
    for (int e = 0; e < d; ++e) out[e] = 0.0;
    double ps = 0.0;
    for (int t = 0; t < kv_len; ++t) {
        double p = scratch[t] / Z;
        ps += p;
        int64_t page = pages[t / S];
        int slot = t % S;
        for (int e = 0; e < d; ++e)
            out[e] += p * bf16_to_double(pool[swo_pool_index(page, 1, kvh, slot, e, Hkv, S, d)]);
    }
    if (lse) *lse = m + log(Z);
    if (psum) *psum = ps;
    return SWO_OK;
}

int swo_attend_row(const uint16_t* pool, int64_t num_pages, int Hkv, int S, int d,
                   const int32_t* pages, int npages, int kv_len, const uint16_t* q, int kvh,
                   double scale, double* out, double* lse, double* psum)
{
    double* scratch = (double*)malloc(sizeof(double) * (size_t)(kv_len > 0 ? kv_len : 1));
    if (!scratch) return SWO_ERR_ARG;
    int rc = attend_row(pool, num_pages, Hkv, S, d, pages, npages, kv_len, q, kvh, scale, out, lse, psum, scratch);
    free(scratch);
    return rc;
}

/* A list of (row, head) pairs of one mixed iteration.  q is [C+n][Hq][d]; out_i (d doubles), lse_i and
 * psum_i are written for pair i.  Row r < C is chunk token r at absolute position P + r, attending keys
 * 0..P+r inclusive of the prompt's pages; row C+i is decode i attending L_i keys.  q head h reads KV
 * head floor(h / (Hq/Hkv)).  scale <= 0 selects 1/sqrt(d).  threads <= 0 selects all cores.
 * If pairs == NULL all (row, head) pairs are evaluated in row-major order (num_pairs must be (C+n)*Hq). */
int swo_mixed_attention(const uint16_t* pool, int64_t num_pages, int Hq, int Hkv, int S, int d, double scale,
                        int P, int C, const int32_t* prefill_pages, int num_prefill_pages,
                        int n, const int32_t* decode_kv_len, const int32_t* indptr, const int32_t* decode_pages,
                        const uint16_t* q, const int32_t* pairs, int64_t num_pairs,
                        double* out, double* lse, double* psum, int threads)
{
    if (Hkv <= 0 || Hq % Hkv != 0 || d <= 0 || S <= 0) return SWO_ERR_ARG;
    if (!pairs && num_pairs != (int64_t)(C + n) * Hq) return SWO_ERR_ARG;
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    int g = Hq / Hkv;
    int rc_all = SWO_OK;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
#pragma omp parallel
    {
        double* scratch = NULL;
        int64_t cap = 0;
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < num_pairs; ++i) {
            int row = pairs ? pairs[2 * i] : (int)(i / Hq);
            int h = pairs ? pairs[2 * i + 1] : (int)(i % Hq);
            int rc = SWO_OK;
            if (row < 0 || row >= C + n || h < 0 || h >= Hq) {
                rc = SWO_ERR_ARG;
            } else {
                const int32_t* pages;
                int npages, kv_len;
                if (row < C) {
                    pages = prefill_pages;
                    npages = num_prefill_pages;
                    kv_len = P + row + 1;
                } else {
                    int r = row - C;
                    pages = decode_pages + indptr[r];
                    npages = indptr[r + 1] - indptr[r];
                    kv_len = decode_kv_len[r];
                }
                if (kv_len > cap) {
                    free(scratch);
                    cap = kv_len;
                    scratch = (double*)malloc(sizeof(double) * (size_t)cap);
                }
                rc = attend_row(pool, num_pages, Hkv, S, d, pages, npages, kv_len,
                                q + ((int64_t)row * Hq + h) * d, h / g, scale,
                                out + i * d, lse ? lse + i : NULL, psum ? psum + i : NULL, scratch);
            }
            if (rc != SWO_OK) {
#pragma omp critical
                rc_all = rc;
            }
        }
        free(scratch);
    }
    return rc_all;
}

int swo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Dense, unpaged causal attention of one prompt: q [T][Hq][d], k,v [T][Hkv][d] (bf16 bits), row t attends
 * keys 0..t.  out [T][Hq][d] doubles.  Same per-row arithmetic as attend_row, on contiguous K/V. */
int swo_dense_causal(const uint16_t* q, const uint16_t* k, const uint16_t* v, int T, int Hq, int Hkv, int d,
                     double scale, double* out, double* lse)
{
    if (Hkv <= 0 || Hq % Hkv != 0) return SWO_ERR_ARG;
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    int g = Hq / Hkv;
    double* w = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
    for (int t = 0; t < T; ++t)
        for (int h = 0; h < Hq; ++h) {
            int kvh = h / g;
            const uint16_t* qr = q + ((int64_t)t * Hq + h) * d;
            double m = -INFINITY;
            for (int u = 0; u <= t; ++u) {
                const uint16_t* kr = k + ((int64_t)u * Hkv + kvh) * d;
                double acc = 0.0;
                for (int e = 0; e < d; ++e) acc += bf16_to_double(qr[e]) * bf16_to_double(kr[e]);
                w[u] = acc * scale;
                if (w[u] > m) m = w[u];
            }
            double Z = 0.0;
            for (int u = 0; u <= t; ++u) {
                w[u] = exp(w[u] - m);
                Z += w[u];
            }
            double* o = out + ((int64_t)t * Hq + h) * d;
            for (int e = 0; e < d; ++e) o[e] = 0.0;
            for (int u = 0; u <= t; ++u) {
                double p = w[u] / Z;
                const uint16_t* vr = v + ((int64_t)u * Hkv + kvh) * d;
                for (int e = 0; e < d; ++e) o[e] += p * bf16_to_double(vr[e]);
            }
            if (lse) lse[(int64_t)t * Hq + h] = m + log(Z);
        }
    free(w);
    return SWO_OK;
}

/* ---------------------------------------------------------------------------------------------- */
/* cost table and chooser                                                                          */
/* ---------------------------------------------------------------------------------------------- */
typedef struct {
    const int32_t* n_grid;      int nn;  /* decode batch sizes, strictly increasing */
    const int64_t* ctx_grid;    int nc;  /* total cached decode context, strictly increasing */
    const int32_t* prefix_grid; int np;  /* cached prefix of the prefilling prompt, strictly increasing */
    const int32_t* chunk_grid;  int nk;  /* candidate prefill tokens, strictly increasing (may start at 0) */
    const int64_t* cost_ns;              /* [nn][nc][np][nk] */
} swo_table;

/* Cumulative maximum along the chunk axis, then along prefix, ctx and n (T is nondecreasing in every
 * argument).  In place. */
void swo_cummax(int64_t* cost, int nn, int nc, int np, int nk)
{
#define AT(a, b, c, e) cost[(((int64_t)(a) * nc + (b)) * np + (c)) * nk + (e)]
    for (int a = 0; a < nn; ++a)
        for (int b = 0; b < nc; ++b)
            for (int c = 0; c < np; ++c)
                for (int e = 1; e < nk; ++e)
                    if (AT(a, b, c, e) < AT(a, b, c, e - 1)) AT(a, b, c, e) = AT(a, b, c, e - 1);
    for (int a = 0; a < nn; ++a)
        for (int b = 0; b < nc; ++b)
            for (int c = 1; c < np; ++c)
                for (int e = 0; e < nk; ++e)
                    if (AT(a, b, c, e) < AT(a, b, c - 1, e)) AT(a, b, c, e) = AT(a, b, c - 1, e);
    for (int a = 0; a < nn; ++a)
        for (int b = 1; b < nc; ++b)
            for (int c = 0; c < np; ++c)
                for (int e = 0; e < nk; ++e)
                    if (AT(a, b, c, e) < AT(a, b - 1, c, e)) AT(a, b, c, e) = AT(a, b - 1, c, e);
    for (int a = 1; a < nn; ++a)
        for (int b = 0; b < nc; ++b)
            for (int c = 0; c < np; ++c)
                for (int e = 0; e < nk; ++e)
                    if (AT(a, b, c, e) < AT(a - 1, b, c, e)) AT(a, b, c, e) = AT(a - 1, b, c, e);
#undef AT
}

/* first index whose grid value is >= x, or -1 */
static int ceil_index_i32(const int32_t* g, int len, int64_t x)
{
    for (int i = 0; i < len; ++i)
        if ((int64_t)g[i] >= x) return i;
    return -1;
}
static int ceil_index_i64(const int64_t* g, int len, int64_t x)
{
    for (int i = 0; i < len; ++i)
        if (g[i] >= x) return i;
    return -1;
}

/* Predicted duration T^(n, ctx, prefix, c) in ns.  Every coordinate is rounded UP to the next grid point
 * (never under-predicts).  interp != 0: along the chunk axis only, integer-linear interpolation between
 * the two neighbouring grid points, rounded up.  A chunk above the last grid point costs SWO_INF;
 * n / ctx / prefix above their last grid point is an error (SWO_ERR_RANGE). */
int swo_cost_lookup(const int32_t* n_grid, int nn, const int64_t* ctx_grid, int nc,
                    const int32_t* prefix_grid, int np, const int32_t* chunk_grid, int nk,
                    const int64_t* cost_ns, int interp,
                    int64_t n, int64_t ctx, int64_t prefix, int64_t c, int64_t* out)
{
    int a = ceil_index_i32(n_grid, nn, n);
    int b = ceil_index_i64(ctx_grid, nc, ctx);
    int p = ceil_index_i32(prefix_grid, np, prefix);
    if (a < 0 || b < 0 || p < 0) return SWO_ERR_RANGE;
    int e = ceil_index_i32(chunk_grid, nk, c);
    if (e < 0) {
        *out = SWO_INF;
        return SWO_OK;
    }
    const int64_t* line = cost_ns + (((int64_t)a * nc + b) * np + p) * nk;
    if (!interp || e == 0 || chunk_grid[e] == c) {
        *out = line[e];
        return SWO_OK;
    }
    int64_t c0 = chunk_grid[e - 1], c1 = chunk_grid[e];
    int64_t t0 = line[e - 1], t1 = line[e];
    int64_t num = (t1 - t0) * (c - c0);
    int64_t den = c1 - c0;
    int64_t q = num / den;
    if (num % den != 0 && num > 0) q += 1; /* ceil for positive slopes */
    *out = t0 + q;
    return SWO_OK;
}

#define SWO_F_NO_PREFILL 1
#define SWO_F_NO_DECODE 2
#define SWO_F_DECODE_INFEASIBLE 4
#define SWO_F_CAPPED 8

static int64_t with_margin(int64_t t, int64_t margin_abs_ns, int32_t margin_ppm)
{
    if (t == SWO_INF) return SWO_INF;
    /* ceil(t * ppm / 1e6) without overflow for t < 2^43 */
    int64_t extra = (t / 1000000) * margin_ppm + (((t % 1000000) * margin_ppm) + 999999) / 1000000;
    return t + margin_abs_ns + extra;
}

/* Eq. (1) by exhaustive scan from the largest candidate down.  quantum q > 1 restricts candidates to
 * positive multiples of q that are <= L.  Returns the chunk; *flags as in the library. */
int swo_choose_bruteforce(const int32_t* n_grid, int nn, const int64_t* ctx_grid, int nc,
                          const int32_t* prefix_grid, int np, const int32_t* chunk_grid, int nk,
                          const int64_t* cost_ns, int interp,
                          int64_t margin_abs_ns, int32_t margin_ppm, int32_t c_max, int32_t quantum,
                          int64_t now_ns, const int64_t* deadlines_ns, int32_t n_active,
                          int64_t total_ctx, int32_t prefix_len, int32_t remaining,
                          int32_t* chunk_out, int32_t* flags_out, int64_t* budget_out)
{
    *flags_out = 0;
    *budget_out = 0;
    if (quantum < 1) quantum = 1;
    if (remaining <= 0) {
        *chunk_out = 0;
        *flags_out = SWO_F_NO_PREFILL;
        return SWO_OK;
    }
    int32_t L = remaining < c_max ? remaining : c_max;
    if (c_max < remaining) *flags_out |= SWO_F_CAPPED;
    if (n_active <= 0) {
        *chunk_out = (L / quantum) * quantum;
        *flags_out |= SWO_F_NO_DECODE;
        return SWO_OK;
    }
    int64_t dmin = deadlines_ns[0];
    for (int i = 1; i < n_active; ++i)
        if (deadlines_ns[i] < dmin) dmin = deadlines_ns[i];
    int64_t B = dmin - now_ns;
    if (B < 0) B = 0;
    *budget_out = B;
    /* cost(0): the decode-only iteration processes no prompt, so it is read at prefix 0 */
    int64_t t0;
    int rc = swo_cost_lookup(n_grid, nn, ctx_grid, nc, prefix_grid, np, chunk_grid, nk, cost_ns, interp,
                             n_active, total_ctx, 0, 0, &t0);
    if (rc != SWO_OK) return rc;
    if (with_margin(t0, margin_abs_ns, margin_ppm) > B) *flags_out |= SWO_F_DECODE_INFEASIBLE;
    for (int32_t c = (L / quantum) * quantum; c >= 1; c -= quantum) {
        int64_t t;
        rc = swo_cost_lookup(n_grid, nn, ctx_grid, nc, prefix_grid, np, chunk_grid, nk, cost_ns, interp,
                             n_active, total_ctx, prefix_len, c, &t);
        if (rc != SWO_OK) return rc;
        if (with_margin(t, margin_abs_ns, margin_ppm) <= B) {
            *chunk_out = c;
            return SWO_OK;
        }
    }
    *chunk_out = 0;
    return SWO_OK;
}

/* T(n,c) = 0.35 + 1[n>0](0.90 + 0.055 n) + 1[c>0](0.40 + 0.006 c) ms, in integer nanoseconds. */
int64_t swo_analytic_cost_ns(int64_t n, int64_t c)
{
    int64_t t = 350000;
    if (n > 0) t += 900000 + 55000 * n;
    if (c > 0) t += 400000 + 6000 * c;
    return t;
}
