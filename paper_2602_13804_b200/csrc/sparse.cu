// Host side of the fused sparse pass (paper Sec. 7 steps 2-4): shared-memory sizing, the choice of the
// block size and of the kernel family.  The kernel itself is in sparse_kernel.cuh; each family of its
// variants is instantiated in a translation unit of its own (sparse_plain.cu, sparse_solve.cu,
// sparse_cert.cu) so that they compile in parallel.
#include "sparse_kernel.cuh"

namespace vsa {


namespace {

size_t sparse_smem_bytes(const Geometry& g, int P, int K_c, bool fused, int threads, bool solve, int P_super = 0)
{
    if (P_super > 0)   // two-level front end
        return (size_t)two_level_smem_words(g.max_pages, P, P << g.tile_shift, K_c, P_super) * 4 + 16;
    // the register variants of the fused kernel (PAGE_KPT > 0) keep a copy of the block-table row
    const bool staged = fused && g.max_pages <= 32 * threads;
    const int PT = P << g.tile_shift;   // routed tiles of 16 tokens
    if (solve)
        return (size_t)solve_tile_offset_words(g.max_pages, P, PT, K_c, fused, staged) * 4 +
               (size_t)solve_tile_rows(K_c) * kRowBytes + 16;
    size_t words = (size_t)bt_stage_offset_words(g.max_pages, P, PT, K_c, fused, g.head_dim);
    if (staged) words += (size_t)g.max_pages;
    return words * 4 + 16;
}

int sm_count() { return device_sm_count(); }

// thread-block size of the per-unit kernel for a launch
int sparse_block_threads(const Geometry& g, int P, bool solve, bool cert, bool listed, bool two_level = false,
                         int P_super = 0)
{
    const long long units = (long long)g.batch * g.n_q_heads;
    int threads = (!solve && units <= sm_count()) ? 512 : 256;
    // two-level front end: every thread holds 8 representative scores and 8 of the 16 * P_super exact scores
    if (two_level) {
        const int max_supers = (g.max_pages + 15) / 16;
        if (units > 2 * sm_count() && (P << g.tile_shift) <= 64 && max_supers <= 8 * 128 && P_super <= 64) threads = 128;
        return threads;
    }
    // Tables wider than 32 scores per thread: the 128-thread shape selects from shared memory, which loses
    // to the 256-thread register selection when every sequence is long (99 against 88 us per layer at
    // batch 16, T = 128k) and wins when most are short (410 against 445 us on the ragged config 4).  The
    // lengths are not known here; what is known is the pool: when batch * max_pages exceeds it, the
    // sequences cannot all be long.
    const bool narrow = g.max_pages <= 32 * 128;
    const bool cannot_all_be_long = (long long)g.batch * g.max_pages > (long long)g.pool_pages;
    if (!solve && !listed && units > 2 * sm_count() && (P << g.tile_shift) <= 64 && (narrow || (!cert && cannot_all_be_long)))
        threads = 128;
    return threads;
}

}  // namespace

bool sparse_shared_memory_fits(const Geometry& g, int P, int K_c, bool fused, bool solve, bool cert, int P_super)
{
    const int threads = sparse_block_threads(g, P, solve, cert, false, P_super > 0, P_super);
    return sparse_smem_bytes(g, P, K_c, fused, threads, solve, P_super) <= (size_t)227 * 1024;
}

int sparse_register_select_max_pages(long long units) { return 32 * (units <= sm_count() ? 512 : 256); }

cudaError_t launch_sparse(const Geometry& g, const void* q, const void* k_cache, const void* v_cache,
                          const int32_t* block_table, const int32_t* seq_lens, int32_t* routed_pages,
                          const float* page_scores, int P, int K_c, float epsilon, float gap_threshold, float* out,
                          vsa_diag_t* diag, int32_t* fallback_list, int32_t* fallback_count, cudaStream_t stream,
                          int solver_iters, vsa_solve_t* solve, const float* rad_logical, vsa_cert_t* cert,
                          int solver_kind, const int32_t* unit_list, const int32_t* unit_count, int routed_stride,
                          const void* tl_summaries, int P_super, const float* k_scale, const float* v_scale)
{
    SparseArgs a;
    a.g = g;
    // no more units than SMs: one larger block per unit (latency shape); otherwise two blocks per SM.
    // The iterative solve exists in the 256-thread shape only.
    // More units than two blocks per SM hold: 128 threads, four blocks per SM.  A unit is a chain of
    // dependent phases, so twice as many units in flight per SM gain more than each loses by having half
    // the threads (measured 1.26x per unit): 512 units take one wave instead of two (25 against 30 us per
    // layer at batch 16, T = 4k), 2048 units 80 against 101 us (batch 64, T = 8k).  Closed-form variants
    // (with or without the certificate) only; fused ones with the page scores in registers (32 per thread at most).
    const int threads = sparse_block_threads(g, P, solve != nullptr, cert != nullptr, unit_list != nullptr,
                                             tl_summaries != nullptr, P_super);
    a.smem = sparse_smem_bytes(g, P, K_c, page_scores != nullptr, threads, solve != nullptr,
                               tl_summaries ? P_super : 0);
    a.tl_summaries = (const uint16_t*)tl_summaries;
    a.P_super = P_super;
    a.k_scale = k_scale;
    a.v_scale = v_scale;
    a.solver_iters = solver_iters;
    a.solver_kind = solver_kind;
    a.solve = solve;
    a.rad_logical = rad_logical;
    a.cert = cert;
    a.unit_list = unit_list;
    a.unit_count = unit_count;
    a.routed_stride = routed_stride > 0 ? routed_stride : P;
    a.q = (const uint16_t*)q;
    a.k = (const uint16_t*)k_cache;
    a.v = (const uint16_t*)v_cache;
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.routed_pages = routed_pages;
    a.page_scores = page_scores;
    a.P = P;
    a.K_c = K_c;
    a.epsilon = epsilon;
    a.gap_threshold = gap_threshold;
    a.out = out;
    a.diag = diag;
    a.fallback_list = fallback_list;
    a.fallback_count = fallback_count;
    a.stream = stream;
    if (k_scale || v_scale) {   // fp8 cache
        if (!k_scale || !v_scale || solve || cert || tl_summaries || g.head_dim != kHeadDim) return cudaErrorInvalidValue;
        return launch_sparse_plain_fp8(a, threads);
    }
    if (g.head_dim != kHeadDim) {
        if (solve || cert || tl_summaries) return cudaErrorInvalidValue;   // (refused by the entry points)
        return g.head_dim == 64 ? launch_sparse_plain_d64(a, threads) : launch_sparse_plain_d256(a, threads);
    }
    if (tl_summaries) return (solve || cert || !page_scores) ? cudaErrorInvalidValue : launch_sparse_two_level(a, threads);
    if (solve) return launch_sparse_solve(a);
    if (cert) return page_scores ? launch_sparse_cert(a, threads) : cudaErrorInvalidValue;
    return launch_sparse_plain(a, threads);
}

}  // namespace vsa
