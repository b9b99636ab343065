/*
 * CPU oracle for the sparse paged decode-attention step.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, readable
 * restatement of what the decode step computes, used only by the tests, by the
 * smoke check and by the benchmark's CPU-baseline leg.  It shares no code with
 * the CUDA library and includes none of its headers.
 *
 * What each routine follows (sections / equations of the paper):
 *   orc_build_summaries  Sec. 7 step 1 "coarse page summaries k_page"; the paper does
 *                        not define them - here: mean of the page's valid key rows.
 *   orc_route            Sec. 7 step 1 (page routing: score summaries, select P pages).
 *   orc_sparse           Sec. 7 steps 2-4 (token routing to K_c candidates, weights on the
 *                        candidates, gather of values).  The weights are the entropic
 *                        problem of Eq. (5.1) with its quadratic term linearised, i.e. the
 *                        softmax at temperature epsilon restricted to the candidates.
 *                        Diagnostics: Def. 1 (face gap) evaluated with r -> q and
 *                        I -> candidate set; Sec. 8 gap statistic s(1) - s(2); Cor. 1
 *                        leakage bound with c = 1; Sec. 10.3 fallback-to-dense policy.
 *   orc_build_radii,     a certificate for the routing (App. E "screening"; construction not in the
 *   orc_certify          paper): per-page ball around the summary, upper bound on every un-scored
 *                        token, certified gap and leakage bound.
 *   orc_frank_wolfe      App. E: Frank-Wolfe with exact line search on the candidate simplex and its
 *                        duality gap, in mirrored fp32 (the vertex choices are integers).
 *   orc_build_super_summaries, orc_route_two_level
 *                        an approximate pre-filter in front of the page routing (Sec. 7 step 1 says only
 *                        "coarse page summaries"; the two-level construction is not in the paper): one
 *                        representative summary per 16 pages, P_super super-pages kept, exact page scores
 *                        inside them.  Parity unpinned by the paper; pinned here by its special cases.
 *   orc_route_group, orc_sparse_group
 *                        the same steps with the query heads of a GQA group routing as one query
 *                        (summed scores, one page set and one candidate set per KV head); the paper
 *                        has a single query per step, so this is a reading.  Parity unpinned by the
 *                        paper; pinned by its reduction to orc_route / orc_sparse for groups of one.
 *   orc_dense            the plain definition: softmax(<q,k_t>/epsilon) over every token.
 * (The theory objects on tiny dictionaries - Euclidean projection, exact gap, the full
 *  entropic minimiser of Eq. (5.1) - live in theory.py next to this file.)
 *
 * Precision: everything that decides an integer (which pages, which tokens, which units
 * fall back) is computed in fp32 in ONE fixed summation order (orc_canon_dot) because the
 * GPU must reproduce those decisions bit for bit.  Everything else is fp64.
 *
 * Parity status: orc_dense, orc_canon_dot, the selections, the candidate softmax, the
 * leakage identities and the entropic solvers are pinned by the CPU tests.  The choice of
 * "mean key" as the summary, per-query-head routing and the value of the fallback threshold
 * are readings of a silent paper: parity unpinned for those three choices.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC (no -ffast-math).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim, page_size, max_pages_per_seq;
    int64_t num_pool_pages;
    int64_t kv_page_stride, kv_head_stride, kv_token_stride; /* in elements */
} orc_shape;

enum { ORC_DMAX = 256 }; /* head_dim is 64, 128 or 256 */

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ---- bf16 <-> fp32 ------------------------------------------------------- */

float orc_bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round to nearest, ties to even; NaN stays NaN */
uint16_t orc_f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* ---- the one fp32 summation order every discrete decision depends on ------
 * 128 products in 16 chunks of 8 consecutive elements.  Chunk partial: the products of the
 * even elements (0, 2, 4, 6) summed left to right, the products of the odd elements
 * (1, 3, 5, 7) summed left to right, then even sum + odd sum.
 * Then a halving tree over the 16 partials: p[c] += p[c+off], off = 8, 4, 2, 1.
 * A product of two bf16 numbers is exact in fp32, so it does not matter whether a
 * machine fuses the multiply into the add.  (The paper fixes no order; this one is the
 * library's arithmetic contract.)  Other head dimensions keep the chunking: d = 256 has 32 partials and
 * one more tree level (off = 16 first); d = 64 has 8 partials, padded with +0 to 16 for the same tree. */
/* d = 64, 128 or 256: d / 8 chunk partials; the tree runs over max(16, d / 8) partials, the missing ones
 * (d = 64) being +0, off = 16 (d = 256 only), 8, 4, 2, 1. */
static float canon_tree(float *p, int nchunks)
{
    int n = nchunks < 16 ? 16 : nchunks;
    for (int c = nchunks; c < n; ++c) p[c] = 0.0f;
    for (int off = n / 2; off >= 1; off >>= 1)
        for (int c = 0; c < off; ++c) p[c] = p[c] + p[c + off];
    return p[0];
}

float orc_canon_dot_d(const uint16_t *x, const uint16_t *y, int d)
{
    float p[ORC_DMAX / 8];
    for (int c = 0; c < d / 8; ++c) {
        float part[2];
        for (int par = 0; par < 2; ++par) {
            float acc = orc_bf16_to_f32(x[8 * c + par]) * orc_bf16_to_f32(y[8 * c + par]);
            for (int e = 2 + par; e < 8; e += 2) {
                float prod = orc_bf16_to_f32(x[8 * c + e]) * orc_bf16_to_f32(y[8 * c + e]);
                acc = acc + prod;
            }
            part[par] = acc;
        }
        p[c] = part[0] + part[1];
    }
    return canon_tree(p, d / 8);
}

float orc_canon_dot(const uint16_t *x, const uint16_t *y) { return orc_canon_dot_d(x, y, 128); }

static double dot64(const uint16_t *x, const uint16_t *y, int d)
{
    double s = 0.0;
    for (int e = 0; e < d; ++e) s += (double)orc_bf16_to_f32(x[e]) * (double)orc_bf16_to_f32(y[e]);
    return s;
}

static int shape_ok(const orc_shape *s)
{
    return s && (s->head_dim == 64 || s->head_dim == 128 || s->head_dim == 256) && s->page_size > 0 && s->batch > 0 && s->n_kv_heads > 0 &&
           s->n_q_heads > 0 && s->n_q_heads % s->n_kv_heads == 0 && s->max_pages_per_seq > 0;
}

static const uint16_t *kv_row(const orc_shape *s, const uint16_t *pool, int64_t page, int g, int t)
{
    return pool + page * s->kv_page_stride + (int64_t)g * s->kv_head_stride + (int64_t)t * s->kv_token_stride;
}

static int n_pages_of(const orc_shape *s, int T) { return (T + s->page_size - 1) / s->page_size; }

/* ---- step 1a: page summaries ---------------------------------------------
 * k_page[p, g, :] = bf16( (sum over the page's valid rows, fp32, ascending token) / n ). */
int orc_build_summaries(const orc_shape *s, const uint16_t *K, const int32_t *bt, const int32_t *seq_lens,
                        const int32_t *first_page, uint16_t *summaries)
{
    if (!shape_ok(s)) return -1;
    for (int b = 0; b < s->batch; ++b) {
        int T = seq_lens[b];
        int nb = n_pages_of(s, T);
        int l0 = first_page ? first_page[b] : 0;
        for (int l = l0; l < nb; ++l) {
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            int n = T - l * s->page_size;
            if (n > s->page_size) n = s->page_size;
            for (int g = 0; g < s->n_kv_heads; ++g) {
                uint16_t *dst = summaries + (p * s->n_kv_heads + g) * s->head_dim;
                for (int e = 0; e < s->head_dim; ++e) {
                    float acc = 0.0f;
                    for (int t = 0; t < n; ++t) acc = acc + orc_bf16_to_f32(kv_row(s, K, p, g, t)[e]);
                    dst[e] = orc_f32_to_bf16(acc / (float)n);
                }
            }
        }
    }
    return 0;
}

/* ---- ordering used by both selections: score descending, index ascending --- */
typedef struct {
    float s;
    int32_t idx;
} scored;

static int cmp_scored(const void *a, const void *b)
{
    const scored *x = (const scored *)a, *y = (const scored *)b;
    if (x->s > y->s) return -1; /* -0.0f and +0.0f compare equal here */
    if (x->s < y->s) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

/* ---- step 1b: page routing -------------------------------------------------
 * c_l = canon_dot(q[b,h], k_page[bt[b][l], g]); routed = first min(P, n_b) pages in the
 * order above.  routed_pages is [B][Hq][P] padded with -1, listed in that order. */
int orc_route(const orc_shape *s, const uint16_t *q, const uint16_t *summaries, const int32_t *bt,
              const int32_t *seq_lens, int P, int32_t *routed_pages, float *routed_scores, float *all_scores)
{
    if (!shape_ok(s) || P < 1) return -1;
    const int G = s->n_q_heads / s->n_kv_heads;
    const int units = s->batch * s->n_q_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        int b = u / s->n_q_heads, h = u % s->n_q_heads, g = h / G;
        int nb = n_pages_of(s, seq_lens[b]);
        scored *c = (scored *)malloc(sizeof(scored) * (size_t)(nb > 0 ? nb : 1));
        const uint16_t *qv = q + (int64_t)u * s->head_dim;
        for (int l = 0; l < nb; ++l) {
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            c[l].s = orc_canon_dot_d(qv, summaries + (p * s->n_kv_heads + g) * s->head_dim, s->head_dim);
            c[l].idx = l;
            if (all_scores) all_scores[(int64_t)u * s->max_pages_per_seq + l] = c[l].s;
        }
        qsort(c, (size_t)nb, sizeof(scored), cmp_scored);
        int keep = nb < P ? nb : P;
        for (int i = 0; i < P; ++i) {
            routed_pages[(int64_t)u * P + i] = i < keep ? c[i].idx : -1;
            if (routed_scores) routed_scores[(int64_t)u * P + i] = i < keep ? c[i].s : -INFINITY;
        }
        free(c);
    }
    return 0;
}

/* ---- two-level routing (an approximate pre-filter in front of step 1; construction not in the paper) ---
 * A super-page is SUPER consecutive logical pages of a sequence.  Its representative is the page summary
 * with the largest squared norm, the norm taken as canon_dot(row, row) in fp32 (ties: the lowest page);
 * large-norm keys are the ones that can dominate an inner product, so the best score inside a super-page
 * is usually its representative's.  super_summaries is [B][max_supers][Hkv][d] (logical order, per
 * sequence), super_rep [B][max_supers][Hkv] the logical page chosen (-1: super-page past the sequence). */
enum { ORC_SUPER = 16 };

int orc_build_super_summaries(const orc_shape *s, const uint16_t *summaries, const int32_t *bt,
                              const int32_t *seq_lens, int max_supers, uint16_t *super_summaries,
                              int32_t *super_rep)
{
    if (!shape_ok(s) || max_supers < 1) return -1;
    for (int b = 0; b < s->batch; ++b) {
        int nb = n_pages_of(s, seq_lens[b]);
        for (int sp = 0; sp < max_supers; ++sp) {
            for (int g = 0; g < s->n_kv_heads; ++g) {
                int64_t o = ((int64_t)b * max_supers + sp) * s->n_kv_heads + g;
                int best = -1;
                float best_n = 0.0f;
                for (int l = sp * ORC_SUPER; l < (sp + 1) * ORC_SUPER && l < nb; ++l) {
                    int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
                    const uint16_t *row = summaries + (p * s->n_kv_heads + g) * s->head_dim;
                    float n2 = orc_canon_dot_d(row, row, s->head_dim);
                    if (best < 0 || n2 > best_n) {
                        best = l;
                        best_n = n2;
                    }
                }
                super_rep[o] = best;
                if (best >= 0) {
                    int64_t p = bt[(int64_t)b * s->max_pages_per_seq + best];
                    memcpy(super_summaries + o * s->head_dim, summaries + (p * s->n_kv_heads + g) * s->head_dim,
                           sizeof(uint16_t) * s->head_dim);
                } else {
                    memset(super_summaries + o * s->head_dim, 0, sizeof(uint16_t) * s->head_dim);
                }
            }
        }
    }
    return 0;
}

/* Per unit: score the super-pages' representatives, keep the P_super best (score descending, super-page
 * ascending); score every page of the kept super-pages exactly as orc_route does and keep the P best of
 * THOSE (score descending, page ascending).  super_routed is [B][Hq][P_super], -1 padded. */
int orc_route_two_level(const orc_shape *s, const uint16_t *q, const uint16_t *summaries,
                        const uint16_t *super_summaries, int max_supers, const int32_t *bt,
                        const int32_t *seq_lens, int P_super, int P, int32_t *super_routed,
                        int32_t *routed_pages, float *routed_scores)
{
    if (!shape_ok(s) || P < 1 || P_super < 1 || max_supers < 1) return -1;
    const int G = s->n_q_heads / s->n_kv_heads;
    const int units = s->batch * s->n_q_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        int b = u / s->n_q_heads, h = u % s->n_q_heads, g = h / G;
        int nb = n_pages_of(s, seq_lens[b]);
        int ns = (nb + ORC_SUPER - 1) / ORC_SUPER;
        const uint16_t *qv = q + (int64_t)u * s->head_dim;
        scored *c = (scored *)malloc(sizeof(scored) * (size_t)(ns > 0 ? ns : 1));
        for (int sp = 0; sp < ns; ++sp) {
            c[sp].s = orc_canon_dot_d(qv, super_summaries + (((int64_t)b * max_supers + sp) * s->n_kv_heads + g) * s->head_dim, s->head_dim);
            c[sp].idx = sp;
        }
        qsort(c, (size_t)ns, sizeof(scored), cmp_scored);
        int keep_s = ns < P_super ? ns : P_super;
        for (int i = 0; i < P_super; ++i) super_routed[(int64_t)u * P_super + i] = i < keep_s ? c[i].idx : -1;
        scored *pg = (scored *)malloc(sizeof(scored) * (size_t)(keep_s * ORC_SUPER + 1));
        int n = 0;
        for (int i = 0; i < keep_s; ++i) {
            for (int l = c[i].idx * ORC_SUPER; l < (c[i].idx + 1) * ORC_SUPER && l < nb; ++l) {
                int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
                pg[n].s = orc_canon_dot_d(qv, summaries + (p * s->n_kv_heads + g) * s->head_dim, s->head_dim);
                pg[n].idx = l;
                ++n;
            }
        }
        qsort(pg, (size_t)n, sizeof(scored), cmp_scored);
        int keep = n < P ? n : P;
        for (int i = 0; i < P; ++i) {
            routed_pages[(int64_t)u * P + i] = i < keep ? pg[i].idx : -1;
            if (routed_scores) routed_scores[(int64_t)u * P + i] = i < keep ? pg[i].s : -INFINITY;
        }
        free(pg);
        free(c);
    }
    return 0;
}

/* ---- steps 2-4 + diagnostics ------------------------------------------------ */
int orc_sparse(const orc_shape *s, const uint16_t *q, const uint16_t *K, const uint16_t *V, const int32_t *bt,
               const int32_t *seq_lens, const int32_t *routed_pages, int P, int K_c, float epsilon,
               float gap_threshold, double *out, float *delta, float *delta12, float *s_max, double *lse,
               double *leak_bound, int32_t *n_candidates, int32_t *fallback, int32_t *cand_pos,
               double *cand_weight, float *best_rejected)
{
    if (!shape_ok(s) || P < 1 || K_c < 1 || !(epsilon > 0.0f)) return -1;
    const int G = s->n_q_heads / s->n_kv_heads;
    const int units = s->batch * s->n_q_heads;
    const double eps = (double)epsilon;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        int b = u / s->n_q_heads, h = u % s->n_q_heads, g = h / G;
        int T = seq_lens[b];
        const uint16_t *qv = q + (int64_t)u * s->head_dim;
        scored *c = (scored *)malloc(sizeof(scored) * (size_t)P * (size_t)s->page_size);
        int nv = 0;
        /* token routing: exact fp32 score of every valid token of every routed page */
        for (int i = 0; i < P; ++i) {
            int l = routed_pages[(int64_t)u * P + i];
            if (l < 0) continue;
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            for (int t = 0; t < s->page_size; ++t) {
                int pos = l * s->page_size + t;
                if (pos >= T) break;
                c[nv].s = orc_canon_dot_d(qv, kv_row(s, K, p, g, t), s->head_dim);
                c[nv].idx = pos;
                ++nv;
            }
        }
        qsort(c, (size_t)nv, sizeof(scored), cmp_scored);
        int ns = nv < K_c ? nv : K_c; /* |S| */

        /* candidate softmax times V, fp64 */
        double *s64 = (double *)malloc(sizeof(double) * (size_t)(ns > 0 ? ns : 1));
        double m = -INFINITY;
        for (int i = 0; i < ns; ++i) {
            int pos = c[i].idx, l = pos / s->page_size, t = pos % s->page_size;
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            s64[i] = dot64(qv, kv_row(s, K, p, g, t), s->head_dim);
            if (s64[i] > m) m = s64[i];
        }
        double Z = 0.0, acc[ORC_DMAX];
        for (int e = 0; e < s->head_dim; ++e) acc[e] = 0.0;
        for (int i = 0; i < ns; ++i) {
            int pos = c[i].idx, l = pos / s->page_size, t = pos % s->page_size;
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            const uint16_t *vr = kv_row(s, V, p, g, t);
            double w = exp((s64[i] - m) / eps);
            Z += w;
            for (int e = 0; e < s->head_dim; ++e) acc[e] += w * (double)orc_bf16_to_f32(vr[e]);
            if (cand_weight) cand_weight[(int64_t)u * K_c + i] = w;
        }
        for (int e = 0; e < s->head_dim; ++e) out[(int64_t)u * s->head_dim + e] = ns > 0 ? acc[e] / Z : 0.0;
        if (cand_weight)
            for (int i = 0; i < K_c; ++i)
                cand_weight[(int64_t)u * K_c + i] = i < ns ? cand_weight[(int64_t)u * K_c + i] / Z : 0.0;
        if (cand_pos)
            for (int i = 0; i < K_c; ++i) cand_pos[(int64_t)u * K_c + i] = i < ns ? c[i].idx : -1;
        lse[u] = ns > 0 ? m / eps + log(Z) : -INFINITY;

        /* diagnostics, fp32 differences of canonical scores */
        float s1 = ns > 0 ? c[0].s : -INFINITY;
        float s2 = ns > 1 ? c[1].s : -INFINITY;
        float d = nv > ns ? s1 - c[ns].s : INFINITY; /* best rejected scored token */
        float d12 = ns > 0 ? s1 - s2 : INFINITY;
        s_max[u] = s1;
        if (best_rejected) best_rejected[u] = nv > ns ? c[ns].s : -INFINITY;
        delta[u] = d;
        delta12[u] = d12;
        n_candidates[u] = ns;
        double lb = (double)(T - ns) * exp(-(double)d / eps);
        leak_bound[u] = lb < 1.0 ? lb : 1.0;
        fallback[u] = (d < gap_threshold && ns < T) ? 1 : 0;
        free(s64);
        free(c);
    }
    return 0;
}

/* ---- group-shared routing (a variant of Sec. 7 steps 1-4 for grouped-query attention; the paper treats
 * a single query, so how the G query heads that read one KV head route is a reading of this library) ---
 * The G heads of a (sequence, KV head) route as ONE query: a page's score is the sum over the group's
 * heads of their page scores, a token's selection score the sum of their token scores - sums of the
 * per-head fixed-order fp32 scores, added in ascending head order in fp32.  One page set (first min(P,
 * n_b) of score descending, page ascending) and one candidate set (first min(K_c, #valid) of score
 * descending, position ascending) per (sequence, KV head).  Each head then takes the softmax at
 * temperature epsilon of ITS OWN scores over the shared candidates, and its diagnostics are Def. 1 /
 * Sec. 8 / Cor. 1 evaluated with its own scores against the shared set S:
 *   s_max = max_{t in S} s_t,  delta = s_max - max_{t scored, not in S} s_t  (negative when a rejected
 *   token out-scores every kept one for this head; +inf when nothing was rejected),
 *   delta12 = best - second best inside S,  leak_bound = min(1, (T - |S|) exp(-delta / eps)),
 *   fallback = delta < threshold and |S| < T.
 * routed_pages / routed_scores are [B][Hkv][P]; cand_pos is [B][Hkv][K_c]; everything else per unit. */
static float group_sum(const float *per_head, int G)
{
    float acc = per_head[0];
    for (int h = 1; h < G; ++h) acc = acc + per_head[h];
    return acc;
}

int orc_route_group(const orc_shape *s, const uint16_t *q, const uint16_t *summaries, const int32_t *bt,
                    const int32_t *seq_lens, int P, int32_t *routed_pages, float *routed_scores)
{
    if (!shape_ok(s) || P < 1) return -1;
    const int G = s->n_q_heads / s->n_kv_heads;
    const int groups = s->batch * s->n_kv_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int gr = 0; gr < groups; ++gr) {
        int b = gr / s->n_kv_heads, g = gr % s->n_kv_heads;
        int nb = n_pages_of(s, seq_lens[b]);
        scored *c = (scored *)malloc(sizeof(scored) * (size_t)(nb > 0 ? nb : 1));
        float *ph = (float *)malloc(sizeof(float) * (size_t)G);
        for (int l = 0; l < nb; ++l) {
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            for (int h = 0; h < G; ++h)
                ph[h] = orc_canon_dot_d(q + ((int64_t)b * s->n_q_heads + g * G + h) * s->head_dim,
                                      summaries + (p * s->n_kv_heads + g) * s->head_dim, s->head_dim);
            c[l].s = group_sum(ph, G);
            c[l].idx = l;
        }
        qsort(c, (size_t)nb, sizeof(scored), cmp_scored);
        int keep = nb < P ? nb : P;
        for (int i = 0; i < P; ++i) {
            routed_pages[(int64_t)gr * P + i] = i < keep ? c[i].idx : -1;
            if (routed_scores) routed_scores[(int64_t)gr * P + i] = i < keep ? c[i].s : -INFINITY;
        }
        free(ph);
        free(c);
    }
    return 0;
}

/* a scored token of a group: summed score, position, and where its per-head scores are kept */
typedef struct {
    float s;
    int32_t idx;
    int32_t k;
} gscored;

static int cmp_gscored(const void *a, const void *b)
{
    const gscored *x = (const gscored *)a, *y = (const gscored *)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

int orc_sparse_group(const orc_shape *s, const uint16_t *q, const uint16_t *K, const uint16_t *V, const int32_t *bt,
                     const int32_t *seq_lens, const int32_t *routed_pages, int P, int K_c, float epsilon,
                     float gap_threshold, double *out, float *delta, float *delta12, float *s_max, double *lse,
                     double *leak_bound, int32_t *n_candidates, int32_t *fallback, int32_t *cand_pos)
{
    if (!shape_ok(s) || P < 1 || K_c < 1) return -1;
    const int G = s->n_q_heads / s->n_kv_heads;
    const int groups = s->batch * s->n_kv_heads;
    const double eps = (double)epsilon;
#pragma omp parallel for schedule(dynamic, 1)
    for (int gr = 0; gr < groups; ++gr) {
        int b = gr / s->n_kv_heads, g = gr % s->n_kv_heads;
        int T = seq_lens[b];
        size_t cap = (size_t)P * (size_t)s->page_size + 1;
        gscored *c = (gscored *)malloc(sizeof(gscored) * cap);
        float *sh = (float *)malloc(sizeof(float) * cap * (size_t)G); /* per-head scores, [k][h] */
        int nv = 0;
        for (int i = 0; i < P; ++i) {
            int l = routed_pages[(int64_t)gr * P + i];
            if (l < 0) continue;
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            for (int t = 0; t < s->page_size; ++t) {
                int pos = l * s->page_size + t;
                if (pos >= T) break;
                for (int h = 0; h < G; ++h)
                    sh[(size_t)nv * G + h] = orc_canon_dot_d(q + ((int64_t)b * s->n_q_heads + g * G + h) * s->head_dim,
                                                           kv_row(s, K, p, g, t), s->head_dim);
                c[nv].s = group_sum(sh + (size_t)nv * G, G);
                c[nv].idx = pos;
                c[nv].k = nv;
                ++nv;
            }
        }
        qsort(c, (size_t)nv, sizeof(gscored), cmp_gscored);
        int ns = nv < K_c ? nv : K_c; /* |S|, shared by the group */
        for (int i = 0; i < K_c; ++i) cand_pos[(int64_t)gr * K_c + i] = i < ns ? c[i].idx : -1;
        for (int h = 0; h < G; ++h) {
            int64_t u = (int64_t)b * s->n_q_heads + g * G + h;
            const uint16_t *qv = q + u * s->head_dim;
            /* this head's softmax over the shared candidates, fp64 */
            double m = -INFINITY, Z = 0.0, acc[ORC_DMAX];
            double *s64 = (double *)malloc(sizeof(double) * (size_t)(ns > 0 ? ns : 1));
            for (int i = 0; i < ns; ++i) {
                int pos = c[i].idx, l = pos / s->page_size, t = pos % s->page_size;
                int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
                s64[i] = dot64(qv, kv_row(s, K, p, g, t), s->head_dim);
                if (s64[i] > m) m = s64[i];
            }
            for (int e = 0; e < s->head_dim; ++e) acc[e] = 0.0;
            for (int i = 0; i < ns; ++i) {
                int pos = c[i].idx, l = pos / s->page_size, t = pos % s->page_size;
                int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
                const uint16_t *vr = kv_row(s, V, p, g, t);
                double w = exp((s64[i] - m) / eps);
                Z += w;
                for (int e = 0; e < s->head_dim; ++e) acc[e] += w * (double)orc_bf16_to_f32(vr[e]);
            }
            for (int e = 0; e < s->head_dim; ++e) out[u * s->head_dim + e] = ns > 0 ? acc[e] / Z : 0.0;
            lse[u] = ns > 0 ? m / eps + log(Z) : -INFINITY;
            free(s64);
            /* this head's own fp32 scores: best and second best inside S, best outside */
            float s1 = -INFINITY, s2 = -INFINITY, rej = -INFINITY;
            for (int i = 0; i < nv; ++i) {
                float v = sh[(size_t)c[i].k * G + h];
                if (i < ns) {
                    if (v > s1) {
                        s2 = s1;
                        s1 = v;
                    } else if (v > s2) {
                        s2 = v;
                    }
                } else if (v > rej) {
                    rej = v;
                }
            }
            float d = nv > ns ? s1 - rej : INFINITY;
            s_max[u] = s1;
            delta[u] = d;
            delta12[u] = ns > 0 ? s1 - s2 : INFINITY;
            n_candidates[u] = ns;
            double lb = (double)(T - ns) * exp(-(double)d / eps);
            leak_bound[u] = lb < 1.0 ? lb : 1.0;
            fallback[u] = (d < gap_threshold && ns < T) ? 1 : 0;
        }
        free(sh);
        free(c);
    }
    return 0;
}

/* ---- certified routing: an upper bound on every score that was never computed ----------
 * (App. E "screening": a certificate that the candidate set holds the active face.  The paper
 * gives no construction; this is the library's: a ball around each page summary.)
 * For a page with stored summary mu (bf16) every valid key row k satisfies |k - mu| <= r, so for any
 * query  <q, k> <= <q, mu> + |q| r.  The stored radius already carries the slack that covers all
 * fp32 rounding on either side of that inequality:
 *     rhat = r * 1.001 + 2^-12 * |mu|,   r = sqrt(max_t |k_t - mu|^2),
 * with the squared norms summed in the canonical order (products fused into the additions, the
 * first product of a chain rounded on its own - what a packed multiply followed by packed fused
 * multiply-adds computes).  Every operation below is a single correctly rounded fp32 operation,
 * so that a GPU can reproduce the numbers bit for bit. */
static float canon_sumsq(const float *d, int dim)
{
    float p[ORC_DMAX / 8];
    for (int c = 0; c < dim / 8; ++c) {
        float part[2];
        for (int par = 0; par < 2; ++par) {
            float acc = d[8 * c + par] * d[8 * c + par];
            for (int e = 2 + par; e < 8; e += 2) acc = fmaf(d[8 * c + e], d[8 * c + e], acc);
            part[par] = acc;
        }
        p[c] = part[0] + part[1];
    }
    return canon_tree(p, dim / 8);
}

int orc_build_radii(const orc_shape *s, const uint16_t *K, const uint16_t *summaries, const int32_t *bt,
                    const int32_t *seq_lens, const int32_t *first_page, float *radii)
{
    if (!shape_ok(s)) return -1;
    for (int b = 0; b < s->batch; ++b) {
        int T = seq_lens[b];
        int nb = n_pages_of(s, T);
        int l0 = first_page ? first_page[b] : 0;
        for (int l = l0; l < nb; ++l) {
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            int n = T - l * s->page_size;
            if (n > s->page_size) n = s->page_size;
            for (int g = 0; g < s->n_kv_heads; ++g) {
                float mu[ORC_DMAX], diff[ORC_DMAX];
                for (int e = 0; e < s->head_dim; ++e) mu[e] = orc_bf16_to_f32(summaries[(p * s->n_kv_heads + g) * s->head_dim + e]);
                float d2max = 0.0f;
                for (int t = 0; t < n; ++t) {
                    const uint16_t *row = kv_row(s, K, p, g, t);
                    for (int e = 0; e < s->head_dim; ++e) diff[e] = orc_bf16_to_f32(row[e]) - mu[e];
                    float d2 = canon_sumsq(diff, s->head_dim);
                    if (d2 > d2max) d2max = d2;
                }
                float r = sqrtf(d2max), mun = sqrtf(canon_sumsq(mu, s->head_dim));
                float t1 = r * 1.001f, t2 = mun * 0x1p-12f;
                radii[p * s->n_kv_heads + g] = t1 + t2;
            }
        }
    }
    return 0;
}

/* Per unit, from the page scores of orc_route (all_scores), its routed pages, and s(1) / the best
 * rejected scored token of orc_sparse:
 *   ub_unrouted = max over valid un-routed pages of  c_l + qn * rhat_l,  qn = sqrt(|q|^2) * (1 + 2^-20)
 *                 (-INF when every page is routed),
 *   delta_cert  = s(1) - max(best rejected scored token, ub_unrouted)   (+INF when nothing is outside S):
 *                 no token outside S scores above s(1) - delta_cert,
 *   certified   = delta_cert >= gap_threshold,
 *   leak_cert   = min(1, (T - |S|) exp(-delta_cert / eps))  (Cor. 1 with the certified gap). */
int orc_certify(const orc_shape *s, const uint16_t *q, const float *radii, const int32_t *bt,
                const int32_t *seq_lens, const float *all_scores, const int32_t *routed_pages, int P,
                const float *s_max, const float *best_rejected, const int32_t *n_candidates, float epsilon,
                float gap_threshold, float *ub_unrouted, float *delta_cert, int32_t *certified, double *leak_cert)
{
    if (!shape_ok(s) || P < 1) return -1;
    const int G = s->n_q_heads / s->n_kv_heads;
    const int units = s->batch * s->n_q_heads;
    for (int u = 0; u < units; ++u) {
        int b = u / s->n_q_heads, h = u % s->n_q_heads, g = h / G;
        int T = seq_lens[b], nb = n_pages_of(s, T);
        float qf[ORC_DMAX];
        for (int e = 0; e < s->head_dim; ++e) qf[e] = orc_bf16_to_f32(q[(int64_t)u * s->head_dim + e]);
        float qn = sqrtf(canon_sumsq(qf, s->head_dim)) * 1.00000095367431640625f;
        float ub = -INFINITY;
        for (int l = 0; l < nb; ++l) {
            int routed = 0;
            for (int i = 0; i < P; ++i) routed |= routed_pages[(int64_t)u * P + i] == l;
            if (routed) continue;
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            float t = qn * radii[p * s->n_kv_heads + g];
            float v = all_scores[(int64_t)u * s->max_pages_per_seq + l] + t;
            if (v > ub) ub = v;
        }
        float m = best_rejected[u] > ub ? best_rejected[u] : ub;
        float d = m == -INFINITY ? INFINITY : s_max[u] - m;
        ub_unrouted[u] = ub;
        delta_cert[u] = d;
        certified[u] = d >= gap_threshold ? 1 : 0;
        double lb = (double)(T - n_candidates[u]) * exp(-(double)d / (double)epsilon);
        leak_cert[u] = lb < 1.0 ? lb : 1.0;
    }
    return 0;
}

/* ---- Frank-Wolfe on the candidate set (App. E) ------------------------------------------------
 * minimise over the simplex of S   f(a) = 1/2 |sum_i a_i k_i - q|^2   by Frank-Wolfe with exact line
 * search, started at the best-scoring candidate:
 *     g_i = <k_i, y> - <k_i, q>,  j = argmin_i g_i,  d = k_j - y,
 *     gamma = clamp(<q - y, d> / |d|^2, 0, 1),  y <- y + gamma d,  a <- (1 - gamma) a + gamma e_j,
 * and the certificate  g_t = <grad f, a> - min_j grad f_j = <y, y - q> - min_i g_i  >= f(a) - min f.
 * The vertex choices are integers decided by floating point, so all of it is fp32 in one fixed order
 * (canonical dot products, every operation a single rounded one, ties to the lower token position),
 * which a GPU reproduces bit for bit.  The paper fixes neither start, step rule nor tie-break.
 * cand_pos: the candidates' token positions (any order, -1 padded, K_c wide); alpha comes back in
 * the same order. */
static float canon_dot32(const float *a, const float *b, int dim)
{
    float p[ORC_DMAX / 8];
    for (int c = 0; c < dim / 8; ++c) {
        float part[2];
        for (int par = 0; par < 2; ++par) {
            float acc = a[8 * c + par] * b[8 * c + par];
            for (int e = 2 + par; e < 8; e += 2) acc = fmaf(a[8 * c + e], b[8 * c + e], acc);
            part[par] = acc;
        }
        p[c] = part[0] + part[1];
    }
    return canon_tree(p, dim / 8);
}

int orc_frank_wolfe(const orc_shape *s, const uint16_t *q, const uint16_t *K, const int32_t *bt,
                    const int32_t *cand_pos, int K_c, int iters, float *alpha, float *fw_gap, float *objective,
                    float *residual2, float *step)
{
    if (!shape_ok(s) || K_c < 1 || iters < 0) return -1;
    const int G = s->n_q_heads / s->n_kv_heads;
    const int units = s->batch * s->n_q_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        int b = u / s->n_q_heads, h = u % s->n_q_heads, g = h / G;
        const int32_t *cp = cand_pos + (int64_t)u * K_c;
        float *al = alpha + (int64_t)u * K_c;
        int n = 0;
        while (n < K_c && cp[n] >= 0) ++n;
        for (int i = 0; i < K_c; ++i) al[i] = 0.0f;
        fw_gap[u] = objective[u] = residual2[u] = step[u] = 0.0f;
        if (n == 0) continue;
        float *rows = (float *)malloc(sizeof(float) * (size_t)n * s->head_dim);
        float *sc = (float *)malloc(sizeof(float) * (size_t)n);
        float *gr = (float *)malloc(sizeof(float) * (size_t)n);
        float qf[ORC_DMAX], y[ORC_DMAX], d[ORC_DMAX], r[ORC_DMAX];
        for (int e = 0; e < s->head_dim; ++e) qf[e] = orc_bf16_to_f32(q[(int64_t)u * s->head_dim + e]);
        for (int i = 0; i < n; ++i) {
            int l = cp[i] / s->page_size, t = cp[i] % s->page_size;
            const uint16_t *row = kv_row(s, K, bt[(int64_t)b * s->max_pages_per_seq + l], g, t);
            for (int e = 0; e < s->head_dim; ++e) rows[(size_t)i * s->head_dim + e] = orc_bf16_to_f32(row[e]);
            sc[i] = orc_canon_dot_d(q + (int64_t)u * s->head_dim, row, s->head_dim);
        }
        /* start: best score, lower position on ties */
        int j = 0;
        for (int i = 1; i < n; ++i)
            if (sc[i] > sc[j] || (sc[i] == sc[j] && cp[i] < cp[j])) j = i;
        al[j] = 1.0f;
        for (int e = 0; e < s->head_dim; ++e) y[e] = rows[(size_t)j * s->head_dim + e];
        float gamma = 0.0f, gmin = 0.0f;
        for (int it = 0;; ++it) {
            for (int i = 0; i < n; ++i) gr[i] = canon_dot32(y, rows + (size_t)i * s->head_dim, s->head_dim) - sc[i];
            j = 0;
            for (int i = 1; i < n; ++i)
                if (gr[i] < gr[j] || (gr[i] == gr[j] && cp[i] < cp[j])) j = i;
            gmin = gr[j];
            if (it >= iters) break;
            for (int e = 0; e < s->head_dim; ++e) {
                d[e] = rows[(size_t)j * s->head_dim + e] - y[e];
                r[e] = qf[e] - y[e];
            }
            float num = canon_dot32(r, d, s->head_dim), den = canon_dot32(d, d, s->head_dim);
            gamma = den > 0.0f ? num / den : 0.0f;
            gamma = gamma < 0.0f ? 0.0f : (gamma > 1.0f ? 1.0f : gamma);
            for (int e = 0; e < s->head_dim; ++e) y[e] = fmaf(gamma, d[e], y[e]);
            for (int i = 0; i < n; ++i) al[i] = fmaf(-gamma, al[i], al[i]);
            al[j] = al[j] + gamma;
        }
        for (int e = 0; e < s->head_dim; ++e) r[e] = y[e] - qf[e];
        float r2 = canon_dot32(r, r, s->head_dim);
        fw_gap[u] = canon_dot32(y, r, s->head_dim) - gmin;
        residual2[u] = r2;
        objective[u] = 0.5f * r2;
        step[u] = gamma;
        free(rows);
        free(sc);
        free(gr);
    }
    return 0;
}

/* ---- the plain definition: dense softmax attention over every token, fp64 ----
 * Optional extras for one candidate set per unit (cand_pos, -1 padded, K_c wide):
 *   true_leak  = dense softmax mass outside the candidate set,
 *   true_gap   = max_t s_t - max_{j not in S} s_j  (fp64 scores),
 *   y_off      = dense readout renormalised over the complement of S. */
int orc_dense(const orc_shape *s, const uint16_t *q, const uint16_t *K, const uint16_t *V, const int32_t *bt,
              const int32_t *seq_lens, float epsilon, const int32_t *unit_mask, double *out, double *lse,
              const int32_t *cand_pos, int K_c, double *true_leak, double *true_gap, double *y_off)
{
    if (!shape_ok(s) || !(epsilon > 0.0f)) return -1;
    const int G = s->n_q_heads / s->n_kv_heads;
    const int units = s->batch * s->n_q_heads;
    const double eps = (double)epsilon;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < units; ++u) {
        if (unit_mask && !unit_mask[u]) continue;
        int b = u / s->n_q_heads, h = u % s->n_q_heads, g = h / G;
        int T = seq_lens[b];
        const uint16_t *qv = q + (int64_t)u * s->head_dim;
        double *sc = (double *)malloc(sizeof(double) * (size_t)T);
        unsigned char *inS = (unsigned char *)calloc((size_t)T, 1);
        if (cand_pos)
            for (int i = 0; i < K_c; ++i) {
                int pos = cand_pos[(int64_t)u * K_c + i];
                if (pos >= 0 && pos < T) inS[pos] = 1;
            }
        double m = -INFINITY, m_off = -INFINITY;
        for (int pos = 0; pos < T; ++pos) {
            int l = pos / s->page_size, t = pos % s->page_size;
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            sc[pos] = dot64(qv, kv_row(s, K, p, g, t), s->head_dim);
            if (sc[pos] > m) m = sc[pos];
            if (!inS[pos] && sc[pos] > m_off) m_off = sc[pos];
        }
        double Z = 0.0, Zoff = 0.0, acc[ORC_DMAX], accoff[ORC_DMAX];
        for (int e = 0; e < s->head_dim; ++e) acc[e] = accoff[e] = 0.0;
        for (int pos = 0; pos < T; ++pos) {
            int l = pos / s->page_size, t = pos % s->page_size;
            int64_t p = bt[(int64_t)b * s->max_pages_per_seq + l];
            const uint16_t *vr = kv_row(s, V, p, g, t);
            double w = exp((sc[pos] - m) / eps);
            Z += w;
            for (int e = 0; e < s->head_dim; ++e) acc[e] += w * (double)orc_bf16_to_f32(vr[e]);
            if (cand_pos && !inS[pos]) {
                Zoff += w;
                for (int e = 0; e < s->head_dim; ++e) accoff[e] += w * (double)orc_bf16_to_f32(vr[e]);
            }
        }
        for (int e = 0; e < s->head_dim; ++e) out[(int64_t)u * s->head_dim + e] = acc[e] / Z;
        lse[u] = m / eps + log(Z);
        if (cand_pos) {
            if (true_leak) true_leak[u] = Zoff / Z;
            if (true_gap) true_gap[u] = m - m_off; /* +inf when nothing lies outside S */
            if (y_off)
                for (int e = 0; e < s->head_dim; ++e)
                    y_off[(int64_t)u * s->head_dim + e] = Zoff > 0.0 ? accoff[e] / Zoff : 0.0;
        }
        free(inS);
        free(sc);
    }
    return 0;
}
