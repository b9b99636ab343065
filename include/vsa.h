/*
 * vsa.h - C ABI of the sparse paged decode-attention step for NVIDIA B200 (sm_100a).
 *
 * One decode step, per (sequence b, query head h) "unit", over a paged bf16 KV cache (an e4m3 cache
 * through the *_fp8 entry points) (paper Sec. 7, "Paged KV and routing", steps 1-4, and Sec. 10.3 fallback policy):
 *
 *   1. page routing   score one summary vector per page, keep the P best pages
 *   2. token routing  score every token of those pages, keep the K_c best tokens
 *   3. weights        entropic (softmax, temperature epsilon) weights on the K_c candidates
 *   4. fused gather   out = sum_k alpha_k V[page_k, off_k], no candidate list in memory
 *   +  diagnostic     support-gap proxy Delta and the leakage bound exp(-Delta/epsilon)
 *   +  fallback       dense attention for every unit whose gap is below a threshold
 *
 * Conventions for every entry point
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are
 *     ordinary (preferably pinned) host memory.  The library never allocates, frees or keeps
 *     any of them.  All buffers are owned by the caller.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     only enqueue work on that stream and return; they never synchronise.
 *   - Kernels are launched with programmatic stream serialisation: a kernel may become
 *     resident while its predecessor on the stream is still running and then reads
 *     `block_table`, `seq_lens` and (second kernel of a step onwards) `q` before it waits for
 *     that predecessor.  Consequently the KERNEL that immediately precedes a call on the
 *     stream must not be the one that writes `block_table` or `seq_lens` (copies, and
 *     anything enqueued earlier than that kernel, are complete and visible first).
 *   - Return value: 0 on success, a negative VSA_ERR_* code otherwise.  Errors are detected
 *     on the host before anything is launched, so a failed call leaves all buffers untouched.
 *   - Data-dependent anomalies (a block-table entry outside the pool, a sequence longer
 *     than its block-table row, a non-positive length) never trap: the unit's
 *     diag.status becomes non-zero and its output row is zero-filled.
 *   - Inputs are assumed finite (no NaN/Inf in q, K, V).
 *   - v1 shapes: head_dim = 128 (every entry point) or 64 / 256 (page summaries, routing, the closed-form
 *     sparse pass, the dense pass and the steps built from them; the iterative solves, the certificate,
 *     two-level and group-shared routing, vsa_build_page_radii and vsa_append_kv return
 *     VSA_ERR_UNSUPPORTED_SHAPE), page_size = 16 or 32, n_q_heads / n_kv_heads in {1, 2, 4, 8, 16, 32}
 *     (multi-head, grouped-query and multi-query attention; groups of 16 and 32 query heads
 *     are processed as two and four sub-groups of 8 that read the same KV head),
 *     1 <= P <= 128 and P * page_size <= 2048 (the tokens scored per unit), 1 <= K_c <= P * page_size,
 *     max_pages_per_seq <= 32768,
 *     batch * n_kv_heads <= 4096 (batch * n_q_heads / 8 <= 4096 for groups above 8),
 *     num_pool_pages * n_kv_heads * head_dim < 2^34 (the summary pool is addressed in 16-byte units by a
 *     32-bit offset: 2^27 rows at head_dim 128).
 *
 * Native layouts (row-major, last dimension contiguous)
 *   q            bf16 [batch][n_q_heads][head_dim]
 *   k/v cache    bf16 [num_pool_pages][n_kv_heads][page_size][head_dim]  (strides in shape)
 *   summaries    bf16 [num_pool_pages][n_kv_heads][head_dim]
 *   block_table  int32 [batch][max_pages_per_seq]   logical page -> physical page
 *   seq_lens     int32 [batch]                      tokens in each sequence (T_b)
 *   out          fp32 [batch][n_q_heads][head_dim]
 * Query head h reads KV head h / (n_q_heads / n_kv_heads).  A unit id is b * n_q_heads + h.
 * With 32-token pages the summary of a page is the mean of its (up to) 32 valid key rows and a routed
 * page contributes 32 tokens; the token-level steps see the same tokens as with 16-token pages (their
 * results do not depend on where page boundaries fall).  vsa_decode_step_group_shared takes 16-token
 * pages only.
 *
 * Arithmetic contract
 *   Every score that feeds a selection (page scores, token scores) is an fp32 dot product in
 *   one fixed order: 16 chunks of 8 consecutive elements; inside a chunk the even elements'
 *   products and the odd elements' products are each summed left to right and the two sums
 *   added; then the 16 chunk sums are combined by a halving tree (p[c] += p[c+off],
 *   off = 8, 4, 2, 1).  head_dim 256 has 32 chunk sums and one more level (off = 16 first); head_dim 64
 *   has 8, padded with +0 to 16 for the same tree.  Selections
 *   order by (score descending, index ascending), -0 and +0 being equal.  Routed pages,
 *   candidate sets, Delta and the fallback flags are therefore reproducible bit for bit.
 *   Softmax weights and outputs use fp32 accumulation.
 */
#ifndef VSA_H_
#define VSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define VSA_OK 0
#define VSA_ERR_INVALID_ARGUMENT (-1)  /* NULL pointer, size <= 0, bad epsilon/threshold, P/K_c < 1 */
#define VSA_ERR_UNSUPPORTED_SHAPE (-2) /* outside the v1 shapes listed above                          */
#define VSA_ERR_WORKSPACE_TOO_SMALL (-3)
#define VSA_ERR_MISALIGNED (-4)        /* a pointer or stride is not 16-byte aligned                  */
#define VSA_ERR_CUDA (-5)              /* a launch or copy was rejected by the CUDA runtime           */
#define VSA_ERR_STATIC_SCRATCH_EXCEEDED (-6) /* shape too large for the built-in scratch array       */

typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim, page_size;
    int32_t max_pages_per_seq; /* row stride of block_table                                 */
    int64_t num_pool_pages;    /* physical pages in the K/V pools and in `summaries`        */
    int64_t kv_page_stride, kv_head_stride, kv_token_stride; /* elements; 0 = native layout */
} vsa_shape_t;

/* Per-unit diagnostics (paper Sec. 8 and Cor. 1; Def. 1 evaluated with r -> q, I -> candidates). */
typedef struct {
    float delta;          /* s(1) - best rejected scored token; +INF if nothing was rejected */
    float delta12;        /* s(1) - s(2), the paper's gap statistic; +INF with one candidate  */
    float s_max;          /* s(1), raw <q, k> of the best candidate                           */
    float lse;            /* log sum exp(s / epsilon) over the tokens that produced `out`     */
    float leak_bound;     /* min(1, (T_b - |S|) * exp(-delta / epsilon))                      */
    int32_t n_candidates; /* |S| = min(K_c, valid tokens in the routed pages)                 */
    int32_t fallback;     /* 1 if delta < gap_threshold (unit is in the fallback list)        */
    int32_t status;       /* 0 = ok, else VSA_UNIT_*                                          */
} vsa_diag_t;

#define VSA_UNIT_BAD_PAGE 1   /* a needed block-table entry is outside [0, num_pool_pages) */
#define VSA_UNIT_BAD_LENGTH 2 /* seq_len <= 0 or > max_pages_per_seq * page_size           */
#define VSA_UNIT_COPY_TIMEOUT 3 /* a tile copy did not complete within the kernel's poll limit */

/* which_call values of vsa_workspace_bytes */
#define VSA_WS_ROUTE 1
#define VSA_WS_SPARSE 2
#define VSA_WS_DENSE 3
#define VSA_WS_STEP 4
#define VSA_WS_STEP_CERTIFIED 5
#define VSA_WS_STEP_EXPAND 6
#define VSA_WS_ROUTE_TWO_LEVEL 7 /* vsa_workspace_bytes: pass P_super in the P argument */
#define VSA_WS_STEP_TWO_LEVEL 8  /* likewise                                            */
#define VSA_SUPER_PAGES 16       /* logical pages per super-page                        */

/*
 * Page summaries (Sec. 7 step 1: "coarse page summaries k_page"; the paper leaves them
 * undefined - here the mean of the page's valid key rows, per KV head).
 * For every sequence b and logical page l in [first_page[b], ceil(T_b / page_size)):
 *   summaries[block_table[b][l]][g][:] = bf16_rne( (sum_t K[page][g][t][:]) / n ),
 * fp32 sum over the n valid rows in ascending t.  Pages outside that range are not touched.
 *   k_cache, block_table, seq_lens, summaries: device.  first_page: device [batch] or NULL (= 0).
 */
int vsa_build_page_summaries(const vsa_shape_t* shape, const void* k_cache, const int32_t* block_table,
                             const int32_t* seq_lens, const int32_t* first_page, void* summaries,
                             void* stream);

/*
 * Page routing (Sec. 7 step 1).  For every unit: c_l = <q[b][h], summaries[block_table[b][l]][g]>
 * for l < n_b = ceil(T_b / page_size); routed_pages[b][h][0..P) = the min(P, n_b) best logical
 * pages, best first, padded with -1.  routed_scores (optional, may be NULL) receives the scores
 * in the same order, padded with -INF.
 *   All pointers device.  ws: device scratch of vsa_workspace_bytes(shape, P, 0, VSA_WS_ROUTE)
 *   bytes, 16-byte aligned; contents undefined before and after the call.
 */
int vsa_route_pages(const vsa_shape_t* shape, const void* q, const void* summaries,
                    const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                    int32_t* routed_pages, float* routed_scores, void* ws, size_t ws_bytes, void* stream);

/*
 * Token routing + candidate softmax x V + diagnostics (Sec. 7 steps 2-4, Sec. 8, Cor. 1),
 * one fused pass per unit.  Scores every valid token of the unit's routed pages, keeps
 * S = the min(K_c, #valid) best, writes
 *   out[b][h][:] = sum_{i in S} alpha_i V_i,  alpha = softmax over S of <q, k_i> / epsilon,
 * and diag[b][h].  Units with diag.delta < gap_threshold (strict) are appended to
 * fallback_list (unit ids, arbitrary order) and counted in *fallback_count, which this call
 * resets to 0 on the stream first.  gap_threshold = -INF never flags (the "cap-compute"
 * policy of Sec. 10.3); +INF flags every unit that rejected at least one token.
 *   routed_pages: device int32 [batch][n_q_heads][P], distinct logical pages or -1.
 *   fallback_list: device int32 [batch * n_q_heads]; fallback_count: device int32 [1].
 *   ws may be NULL (this call needs no scratch).  All pointers device.
 */
int vsa_sparse_decode(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                      const int32_t* block_table, const int32_t* seq_lens, const int32_t* routed_pages,
                      int32_t P, int32_t K_c, float epsilon, float gap_threshold, float* out,
                      vsa_diag_t* diag, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                      size_t ws_bytes, void* stream);

/*
 * The same pass with the weights of step 3 obtained by an iterative solve (Sec. 7 step 3
 * "convex sparse solve ... small iterations and certificates"; Sec. 5.3 and App. E name entropic
 * mirror descent and the Frank-Wolfe gap; App. F sweeps 2, 4 and 6 iterations).  On the candidate
 * set S of the unit, with k_i its key rows, the problem is Eq. (5.1) restricted to S,
 *     minimise over the simplex  1/2 |sum_i a_i k_i - q|^2 + epsilon * sum_i a_i log a_i,
 * started from the closed form a = softmax(<q, k_i> / epsilon) that vsa_sparse_decode uses and
 * advanced by `solver_iters` entropic mirror-descent steps
 *     g = K_S (K_S^T a) - K_S q,   log a <- (log a - eta * g) / (1 + eta * epsilon) + const,
 * eta = 1 / max_i |k_i|^2 (the paper fixes neither start nor step; with this eta the objective
 * never increases).  out = sum_i a_i V_i with the final weights.  solve[b][h] receives the
 * certificate and the objective at the final weights.  Candidates, diag (lse is that of the
 * closed-form weights) and the fallback list are exactly those of vsa_sparse_decode; units that
 * fall back are later overwritten by plain dense softmax attention, as there.
 *   solver_iters in [0, 64]; 0 returns the closed-form weights together with their certificate.
 *   K_c <= VSA_SOLVER_MAX_CANDIDATES (the candidate keys are held on chip across iterations).
 *   solve: device vsa_solve_t [batch][n_q_heads].  Everything else as for vsa_sparse_decode.
 */
#define VSA_SOLVER_MAX_CANDIDATES 256
#define VSA_SOLVER_MAX_ITERS 64
typedef struct {
    float fw_gap;    /* App. E: <grad f(a), a> - min_j grad f(a)_j >= f(a) - min f,  f = 1/2 |K_S^T a - q|^2 */
    float objective; /* 1/2 |K_S^T a - q|^2 + epsilon * sum_i a_i log a_i                                   */
    float residual2; /* |K_S^T a - q|^2                                                                      */
    float step;      /* eta                                                                                  */
} vsa_solve_t;

int vsa_sparse_decode_entropic(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                               const int32_t* block_table, const int32_t* seq_lens, const int32_t* routed_pages,
                               int32_t P, int32_t K_c, float epsilon, float gap_threshold, int32_t solver_iters,
                               float* out, vsa_diag_t* diag, vsa_solve_t* solve, int32_t* fallback_list,
                               int32_t* fallback_count, void* stream);

/*
 * The same pass with step 3 done by Frank-Wolfe (App. E; "Frank-Wolfe with small iterations and
 * certificates", Sec. 7 step 3) on the unregularised problem over the candidate simplex,
 *     minimise  f(a) = 1/2 |sum_i a_i k_i - q|^2 :
 * start at the best-scoring candidate, then `solver_iters` times
 *     g_i = <k_i, y> - <k_i, q>,  j = argmin_i g_i (ties: lower token position),  d = k_j - y,
 *     gamma = clamp(<q - y, d> / |d|^2, 0, 1),  y <- y + gamma d,  a <- (1 - gamma) a + gamma e_j.
 * At most solver_iters + 1 candidates carry weight.  out = sum_i a_i V_i.  solve[b][h]: fw_gap =
 * <y, y - q> - min_i g_i at the final point, objective = f(a), residual2 = |y - q|^2, step = the last
 * gamma.  The vertex choices are integers decided by floating point: every operation behind them is a
 * single rounded fp32 operation in the library's canonical summation order (start, step rule and
 * tie-break are the library's; the paper fixes none).  epsilon only enters diag (closed-form lse,
 * leakage bound) here.  Candidates, diag, fallback list and all limits as for
 * vsa_sparse_decode_entropic.
 */
int vsa_sparse_decode_frank_wolfe(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                                  const int32_t* block_table, const int32_t* seq_lens, const int32_t* routed_pages,
                                  int32_t P, int32_t K_c, float epsilon, float gap_threshold, int32_t solver_iters,
                                  float* out, vsa_diag_t* diag, vsa_solve_t* solve, int32_t* fallback_list,
                                  int32_t* fallback_count, void* stream);

/*
 * Dense fallback (Sec. 10.3 "fallback-to-dense"): for every unit in fallback_list[0 ..
 * *fallback_count) recompute out[b][h][:] = softmax(<q, k_t> / epsilon over all T_b tokens) V
 * with a split-K pass (K and V of a KV head are read once for all listed heads of its
 * group), overwrite out and diag.lse, and leave every other unit untouched.
 * fallback_count == NULL (then fallback_list is ignored) means every unit: this is the dense
 * decode baseline.  The count is read on the device; nothing synchronises with the host.
 *   diag may be NULL.  ws: device scratch of vsa_workspace_bytes(shape, 0, 0, VSA_WS_DENSE) bytes.
 */
int vsa_dense_decode_fallback(const vsa_shape_t* shape, const void* q, const void* k_cache,
                              const void* v_cache, const int32_t* block_table, const int32_t* seq_lens,
                              const int32_t* fallback_list, const int32_t* fallback_count, float epsilon,
                              float* out, vsa_diag_t* diag, void* ws, size_t ws_bytes, void* stream);

/*
 * The whole step on one stream: vsa_route_pages -> vsa_sparse_decode ->
 * vsa_dense_decode_fallback, same results as the three calls made one after the other.
 *   routed_pages, diag, fallback_list, fallback_count: device outputs as above.
 *   ws: device scratch of vsa_workspace_bytes(shape, P, K_c, VSA_WS_STEP) bytes.
 */
int vsa_decode_step(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                    const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                    int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                    int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                    size_t ws_bytes, void* stream);

/*
 * vsa_decode_step with the iterative solve of vsa_sparse_decode_entropic in place of the closed-form
 * weights: vsa_route_pages -> vsa_sparse_decode_entropic -> vsa_dense_decode_fallback.
 */
int vsa_decode_step_entropic(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                             const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                             int32_t K_c, float epsilon, float gap_threshold, int32_t solver_iters, float* out,
                             vsa_diag_t* diag, vsa_solve_t* solve, int32_t* routed_pages, int32_t* fallback_list,
                             int32_t* fallback_count, void* ws, size_t ws_bytes, void* stream);

/* vsa_route_pages -> vsa_sparse_decode_frank_wolfe -> vsa_dense_decode_fallback. */
int vsa_decode_step_frank_wolfe(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                                const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                                int32_t K_c, float epsilon, float gap_threshold, int32_t solver_iters, float* out,
                                vsa_diag_t* diag, vsa_solve_t* solve, int32_t* routed_pages, int32_t* fallback_list,
                                int32_t* fallback_count, void* ws, size_t ws_bytes, void* stream);

/*
 * Routing certificate (App. E asks for "certificates" that the screened candidate set is the right
 * one and for a fallback when they fail; it gives no construction - this one is the library's).
 * Every page carries the radius of a ball around its stored summary mu that holds all its valid key
 * rows, so no token of the page can score above  <q, mu> + |q| * radius.  The largest such bound
 * over the pages that were NOT routed, together with the best rejected token of the routed pages,
 * bounds every score outside the candidate set S:
 *     delta_cert = s(1) - max(best rejected scored token, ub_unrouted)   (+INF if nothing is outside S),
 * a true lower bound on the gap between s(1) and anything outside S, where diag.delta only sees the
 * routed pages.  Cor. 1 with it gives leak_bound_cert >= the dense softmax mass outside S.
 *
 * vsa_build_page_radii: radii[page][kv_head] (device fp32 [num_pool_pages][n_kv_heads]) for the pages
 * each sequence owns from first_page[b] on (NULL = all), from k_cache and the summaries already
 * built for them: 1.001 * max_t |k_t - mu| + 2^-12 * |mu| in fp32 (the slack covers every rounding
 * in the bound and in the scores it is compared with).  Cache maintenance, like the summaries.
 *
 * vsa_decode_step_certified: vsa_decode_step with the certificate computed in the same pass; the
 * fallback decision becomes  !(delta_cert >= gap_threshold) && |S| < T  (the certified gap instead
 * of diag.delta; diag.fallback and the fallback list follow it), everything else is unchanged.
 *   cert: device vsa_cert_t [batch][n_q_heads].
 *   ws: device scratch of vsa_workspace_bytes(shape, P, K_c, VSA_WS_STEP_CERTIFIED) bytes.
 *   Shapes: max_pages_per_seq <= 8192 (16384 when batch * n_q_heads does not exceed the SM count),
 *   VSA_ERR_UNSUPPORTED_SHAPE beyond.
 */
typedef struct {
    float delta_cert;      /* certified gap, see above                                          */
    float ub_unrouted;     /* best upper bound over the un-routed pages, -INF if all are routed */
    float leak_bound_cert; /* min(1, (T - |S|) exp(-delta_cert / epsilon))                      */
    int32_t certified;     /* delta_cert >= gap_threshold                                       */
} vsa_cert_t;

int vsa_build_page_radii(const vsa_shape_t* shape, const void* k_cache, const void* summaries,
                         const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_page,
                         float* radii, void* stream);

/*
 * Cache maintenance between two decode steps, in one kernel (the paper assumes a paged cache "as in
 * vLLM" and has no counterpart for this call): append one token per sequence and bring the page
 * it lands in up to date.  seq_lens are the lengths AFTER the append: sequence b's new token sits at
 * position seq_lens[b] - 1, i.e. in page block_table[b][(seq_lens[b] - 1) / page_size], which must
 * already be allocated.  Writes the token's key and value rows, then that page's summary and, when
 * radii != NULL, its radius - the same values vsa_build_page_summaries / vsa_build_page_radii would
 * produce for the page.  Sequences with an invalid length or page are skipped.
 *   k_new, v_new: device bf16 [batch][n_kv_heads][head_dim].  k_cache, v_cache, summaries, radii: device,
 *   updated in place.
 */
int vsa_append_kv(const vsa_shape_t* shape, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                  const int32_t* block_table, const int32_t* seq_lens, void* summaries, float* radii,
                  void* stream);

int vsa_decode_step_certified(const vsa_shape_t* shape, const void* q, const void* summaries, const float* radii,
                              const void* k_cache, const void* v_cache, const int32_t* block_table,
                              const int32_t* seq_lens, int32_t P, int32_t K_c, float epsilon, float gap_threshold,
                              float* out, vsa_diag_t* diag, vsa_cert_t* cert, int32_t* routed_pages,
                              int32_t* fallback_list, int32_t* fallback_count, void* ws, size_t ws_bytes,
                              void* stream);

/*
 * The certified step with the "paged expansion" loop (App. E: when the certificate fails, enlarge
 * S until it passes) before anything falls back to the dense pass: every unit is first processed
 * with P routed pages; the units whose certificate fails are processed again with 2P pages, those
 * that still fail with 4P, and so on while the page count stays below P_expand (the last pass uses
 * exactly P_expand), all from the page scores of the same scan and with the same K_c; what the last
 * pass still refuses goes to the dense pass.  The passes are enqueued back to back (ceil(log2(P_expand /
 * P)) extra launches, each over the device-side list its predecessor wrote; an empty list costs a launch
 * whose blocks exit), so the loop is bounded and never synchronises with the host.
 * out, diag and cert of a unit are those of its last sparse pass (dense rows for the final fallback
 * list).  routed_pages: device int32 [batch][n_q_heads][P_expand]; a unit's row holds the pages of its
 * last pass, -1 padded (so a row with more than P entries marks a unit that was retried).
 *   ws: device scratch of vsa_workspace_bytes(shape, P_expand, K_c, VSA_WS_STEP_EXPAND) bytes.
 *   P < P_expand <= 128; K_c <= P * page_size; shapes as for vsa_decode_step_certified.
 */
int vsa_decode_step_certified_expand(const vsa_shape_t* shape, const void* q, const void* summaries,
                                     const float* radii, const void* k_cache, const void* v_cache,
                                     const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                                     int32_t P_expand, int32_t K_c, float epsilon, float gap_threshold, float* out,
                                     vsa_diag_t* diag, vsa_cert_t* cert, int32_t* routed_pages,
                                     int32_t* fallback_list, int32_t* fallback_count, void* ws, size_t ws_bytes,
                                     void* stream);

/*
 * The step with GROUP-SHARED routing (a variant for grouped-query attention; the paper's step has one
 * query, so how a group of query heads routes is this library's reading): the G = n_q_heads / n_kv_heads
 * heads that read one KV head route as ONE query.  A page's routing score is the sum over the group's
 * heads of their page scores, a token's selection score the sum of their token scores - the per-head
 * fixed-order fp32 scores added in ascending head order - so there is one page set (top-P, score
 * descending, page ascending) and one candidate set (top-K_c, score descending, position ascending) per
 * (sequence, KV head): every K and V tile is read once per group and both selections run once per group.
 * Each head then takes the softmax at temperature epsilon of ITS OWN scores over the shared candidates;
 * its diag is Def. 1 / Sec. 8 / Cor. 1 with its own scores against the shared set S: s_max = its best
 * score in S, delta = s_max minus its best score among the scored tokens outside S (negative when a
 * rejected token out-scores every kept one for this head, +inf when nothing was rejected), delta12 = best
 * minus second best inside S, leak_bound and fallback as in vsa_sparse_decode.  Flagged units take the
 * dense pass as in vsa_decode_step.
 *   routed_pages: device int32 [batch][n_kv_heads][P] (one list per group), best first, -1 padded.
 *   everything else as for vsa_decode_step; ws: VSA_WS_STEP bytes.
 *   Needs the native cache layout (kv_token_stride = head_dim, kv_head_stride = page_size * head_dim) and
 *   n_q_heads / n_kv_heads in {1, 2, 4, 8}; otherwise VSA_ERR_UNSUPPORTED_SHAPE.
 */
int vsa_decode_step_group_shared(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                                 const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                                 int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                                 int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                                 size_t ws_bytes, void* stream);

/*
 * Two-level page routing: an approximate pre-filter in front of Sec. 7 step 1 (the paper says only
 * "coarse page summaries"; the construction is this library's).  A super-page is VSA_SUPER_PAGES
 * consecutive LOGICAL pages of a sequence; its representative is the page summary with the largest
 * squared norm among them (fp32 in the library's fixed summation order, ties to the lowest page).
 * Routing scores the representatives (1/16 of the rows the full scan reads), keeps the P_super best
 * super-pages per query head (score descending, super-page ascending), scores the pages inside them
 * exactly - the same numbers the full scan produces - and keeps the P best of those (score
 * descending, page ascending).  With P_super >= the number of super-pages the result equals
 * vsa_route_pages; otherwise a page whose super-page was not kept is lost.
 *
 * vsa_build_super_summaries (cache maintenance, after vsa_build_page_summaries):
 *   summaries: device bf16 [num_pool_pages][n_kv_heads][head_dim].
 *   first_super: device int32 [batch] or NULL: first super-page of each sequence to (re)build, e.g.
 *     (seq_len - 1) / (16 * VSA_SUPER_PAGES) after appending one token.
 *   super_summaries: device bf16 [batch][ceil(max_pages_per_seq / 16)][n_kv_heads][head_dim], in the
 *     sequence's logical order (zero rows past the sequence).
 *   super_rep: device int32 [batch][ceil(max_pages_per_seq / 16)][n_kv_heads] or NULL: the logical page
 *     chosen (-1 past the sequence).
 * vsa_route_pages_two_level: arguments as vsa_route_pages, plus super_summaries, P_super (1..128) and
 *   super_routed: device int32 [batch][n_q_heads][P_super] or NULL, the kept super-pages, -1 padded.
 *   ws: vsa_workspace_bytes(shape, P_super, 0, VSA_WS_ROUTE_TWO_LEVEL) bytes.
 * vsa_decode_step_two_level: vsa_decode_step with the two-level routing in place of the full scan (the
 *   representatives are scanned by one kernel; keeping the super-pages, scoring their pages and routing
 *   happen inside the fused kernel of the step); when ceil(max_pages_per_seq / 16) <= P_super every
 *   super-page would be kept and the call runs vsa_decode_step itself (same results).
 *   ws: vsa_workspace_bytes(shape, P_super, K_c, VSA_WS_STEP_TWO_LEVEL) bytes.
 */
int vsa_build_super_summaries(const vsa_shape_t* shape, const void* summaries, const int32_t* block_table,
                              const int32_t* seq_lens, const int32_t* first_super, void* super_summaries,
                              int32_t* super_rep, void* stream);
int vsa_route_pages_two_level(const vsa_shape_t* shape, const void* q, const void* summaries,
                              const void* super_summaries, const int32_t* block_table, const int32_t* seq_lens,
                              int32_t P_super, int32_t P, int32_t* routed_pages, float* routed_scores,
                              int32_t* super_routed, void* ws, size_t ws_bytes, void* stream);
int vsa_decode_step_two_level(const vsa_shape_t* shape, const void* q, const void* summaries,
                              const void* super_summaries, const void* k_cache, const void* v_cache,
                              const int32_t* block_table, const int32_t* seq_lens, int32_t P_super, int32_t P,
                              int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                              int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                              size_t ws_bytes, void* stream);

/*
 * vsa_decode_step with CUDA events recorded on `stream` between its kernels, for per-kernel
 * timing of exactly the launch sequence the step uses (a measurement aid for the latency
 * breakdown the paper asks for in Sec. 10.4; results are identical to vsa_decode_step).
 *   events: host array of 5 cudaEvent_t created by the caller with timing enabled:
 *   [0] before the page-score scan, [1] after it, [2] recorded right after [1],
 *   [3] after the fused sparse pass, [4] after the dense fallback pass.
 * The top-P selection runs inside the fused sparse kernel, so the interval [1] -> [2] brackets no
 * kernel: it reads what a pair of event records costs on the stream, which every other interval
 * also contains.
 */
int vsa_decode_step_timed(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                          const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                          int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                          int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                          size_t ws_bytes, void* stream, void* const* events);

/*
 * The same step for a caller whose per-step tensors live in host memory: copies q_host
 * (bf16 [batch][n_q_heads][head_dim]) to q_dev, runs vsa_decode_step, and copies the results
 * back into out_host (fp32 [batch][n_q_heads][head_dim]) and diag_host ([batch][n_q_heads],
 * may be NULL).  The KV cache, summaries, block table and lengths stay device-resident: they
 * are the decode state, not per-step inputs.  Everything is asynchronous on `stream`; the host
 * buffers must stay valid, and hold the results, once the stream has been synchronised by the
 * caller.
 *   q_host, out_host, diag_host: host.  q is brought into q_dev on the stream (by a kernel
 *   that reads it across the bus when it is page-locked, by a copy otherwise).  A page-locked
 *   (cudaHostAlloc / cudaHostRegister) out_host or diag_host is written IN PLACE by the kernels,
 *   with no copy and without touching its staging buffer; a pageable one is staged through
 *   out_dev / diag_dev with a copy on the stream.
 *   q_dev, out_dev, diag_dev, routed_pages, fallback_list, fallback_count, ws: device staging
 *   and scratch buffers of the sizes given for vsa_decode_step; the contents of the three staging
 *   buffers after the call are unspecified.
 */
int vsa_decode_step_host(const vsa_shape_t* shape, const void* q_host, void* q_dev, const void* summaries,
                         const void* k_cache, const void* v_cache, const int32_t* block_table,
                         const int32_t* seq_lens, int32_t P, int32_t K_c, float epsilon,
                         float gap_threshold, float* out_host, float* out_dev, vsa_diag_t* diag_host,
                         vsa_diag_t* diag_dev, int32_t* routed_pages, int32_t* fallback_list,
                         int32_t* fallback_count, void* ws, size_t ws_bytes, void* stream);

/*
 * Page routing without a caller-provided workspace (no counterpart in the paper: this is a
 * deployment convenience of the library).  Same inputs, outputs and results as vsa_route_pages,
 * but the page-score scratch lives in a fixed array inside the library's device image, so the
 * call needs no device memory from the caller and performs no allocation of any kind.  It is
 * meant for callers that cannot obtain device memory at call time: an attention backend inside a
 * serving engine whose KV-cache pool already owns all free HBM (a later cudaMalloc would fail
 * or stall the device), or code in a decode loop where allocation calls are forbidden.
 *   Limit: batch * n_q_heads * max_pages_per_seq <= VSA_STATIC_ROUTE_SCORES (one fp32 score per
 *   unit and logical page; the array occupies 4 MiB on every GPU that loads the library, until
 *   the process exits).  Larger shapes are rejected with VSA_ERR_STATIC_SCRATCH_EXCEEDED before
 *   anything is launched.
 *   The first call on each device looks up the array's device address (with that device
 *   current); make that first call outside any stream capture.
 *   All calls share the one array, which keeps the scores of the last call; nothing in it has to
 *   be cleared, because the selection only reads scores that the scan of the same call wrote.
 *   Two calls that overlap on the GPU (different streams, or host threads) race on it: serialise
 *   them, or use vsa_route_pages with separate workspaces.
 */
#define VSA_STATIC_ROUTE_SCORES (1 << 20)
int vsa_route_pages_static(const vsa_shape_t* shape, const void* q, const void* summaries,
                           const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                           int32_t* routed_pages, float* routed_scores, void* stream);

/*
 * fp8 KV cache (the paper's system sketch, Sec. 7, fixes no storage format; this is a deployment option of
 * the library).  k_cache / v_cache hold e4m3 bytes (OCP e4m3fn, no NaN encodings expected) in the native
 * layout [num_pool_pages][n_kv_heads][page_size][head_dim] with the shape's strides counted in BYTES (each
 * a multiple of 16); k_scale / v_scale, device fp32 [num_pool_pages][n_kv_heads], give the value a byte
 * stands for: value = e4m3(byte) * scale[page][kv head].  Summaries stay bf16, so routing is unchanged.
 * Token scores are the fixed-order dot of q with the decoded bytes, multiplied by the page's key scale;
 * the readout multiplies each candidate's weight by its page's value scale.  With POWER-OF-TWO scales every
 * one of those multiplications is exact, and all results equal - discrete ones bit for bit - those of
 * the bf16 entry points on a bf16 cache that holds the same values; with other scales the score carries
 * one more rounding.  head_dim 128; page_size 16 or 32; closed-form weights only.  Otherwise the four entry
 * points take the arguments, workspaces and error rules of the entry points they are named after.
 */
int vsa_build_page_summaries_fp8(const vsa_shape_t* shape, const void* k_cache, const float* k_scale,
                                 const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_page,
                                 void* summaries, void* stream);
int vsa_sparse_decode_fp8(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                          const float* k_scale, const float* v_scale, const int32_t* block_table,
                          const int32_t* seq_lens, const int32_t* routed_pages, int32_t P, int32_t K_c, float epsilon,
                          float gap_threshold, float* out, vsa_diag_t* diag, int32_t* fallback_list,
                          int32_t* fallback_count, void* stream);
int vsa_dense_decode_fallback_fp8(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                                  const float* k_scale, const float* v_scale, const int32_t* block_table,
                                  const int32_t* seq_lens, const int32_t* fallback_list,
                                  const int32_t* fallback_count, float epsilon, float* out, vsa_diag_t* diag,
                                  void* ws, size_t ws_bytes, void* stream);
int vsa_decode_step_fp8(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                        const void* v_cache, const float* k_scale, const float* v_scale, const int32_t* block_table,
                        const int32_t* seq_lens, int32_t P, int32_t K_c, float epsilon, float gap_threshold,
                        float* out, vsa_diag_t* diag, int32_t* routed_pages, int32_t* fallback_list,
                        int32_t* fallback_count, void* ws, size_t ws_bytes, void* stream);

/*
 * Per-rank steps of the sequence-sharded (context-parallel) decode step.  One sequence's pages may be
 * spread over several ranks: every rank passes a block table of the full width in which only the entries
 * of the pages IT holds are valid (every other entry negative), and the global seq_lens.  Because page
 * scores, token scores and the readout do not depend on where a page lives (Sec. 7), three small
 * exchanges between the ranks reproduce the single-rank step:
 *   1. every rank calls vsa_route_pages (pages it does not hold score -inf: drop them) and the local
 *      top-P proposals are merged under the total order into the global routed pages;
 *   2. vsa_cp_token_candidates scores the tokens of the globally routed pages the rank holds and returns
 *      its best K_out = K_c + 1 of them; merged, the first K_c are the candidate set and the next one is
 *      the best rejected token of the gap statistic;
 *   3. vsa_cp_partial_readout forms the rank's softmax readout over its own members of the global
 *      candidate set; the partial readouts combine with weights exp(lse_r - lse).
 * The exchanges themselves are not part of this library's C ABI (paper_2602_13804_b200/context_parallel.py
 * runs them over torch.distributed).  head_dim 128; page_size 16 or 32.
 *   vsa_cp_token_candidates: q device bf16 [batch][n_q_heads][128]; routed_pages device int32
 *     [batch][n_q_heads][P] (global logical pages, any order, -1 padded); 1 <= K_out <= P * page_size + 1;
 *     cand_pos device int32 / cand_score device fp32 [batch][n_q_heads][K_out]: the rank's best tokens in
 *     position order, (-1, -inf) padded.  Routed pages the rank does not hold are skipped, not an error.
 *   vsa_cp_partial_readout: cand_pos / cand_score device [batch][n_q_heads][K_c]: the global candidate set
 *     with its scores (-1 padded, the same on every rank); out_partial device fp32 [batch][n_q_heads][128]:
 *     the readout over the rank's own members, normalised by their weight sum (zeros if it holds none);
 *     lse_partial device fp32 [batch][n_q_heads]: log of their sum of exp(score / epsilon) (-inf if none).
 * Units with an invalid length get empty lists / zero rows.  Nothing is allocated; both calls are
 * asynchronous on `stream`.
 */
int vsa_cp_token_candidates(const vsa_shape_t* shape, const void* q, const void* k_cache,
                            const int32_t* block_table, const int32_t* seq_lens, const int32_t* routed_pages,
                            int32_t P, int32_t K_out, int32_t* cand_pos, float* cand_score, void* stream);
int vsa_cp_partial_readout(const vsa_shape_t* shape, const void* v_cache, const int32_t* block_table,
                           const int32_t* seq_lens, const int32_t* cand_pos, const float* cand_score,
                           int32_t K_c, float epsilon, float* out_partial, float* lse_partial, void* stream);

/* Scratch bytes needed by one call kind for this shape (0 if the shape is invalid). */
size_t vsa_workspace_bytes(const vsa_shape_t* shape, int32_t P, int32_t K_c, int which_call);

/* Static, human-readable text for a return code. */
const char* vsa_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* VSA_H_ */
