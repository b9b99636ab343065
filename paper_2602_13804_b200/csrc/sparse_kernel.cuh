// Fused sparse pass (kernel template and its launch dispatch; included by the translation units that
// instantiate one family of variants each, see sparse_plain.cu, sparse_solve.cu, sparse_cert.cu).
// Fused sparse pass for one (sequence, query head) unit per thread block (paper Sec. 7 steps 2-4,
// Sec. 8 gap statistic, Cor. 1 leakage bound, Sec. 10.3 fallback flag):
//   [top-P page selection from the page scores, when fused with routing] ->
//   score every valid token of the routed pages -> exact top-K_c -> softmax weights at temperature
//   epsilon -> weighted sum of the candidates' value rows -> diagnostics.
// The candidate list and the weights live in shared memory and registers only.
#pragma once

#include <limits.h>
#include <math.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"
#include "vsa_select.cuh"

namespace vsa {

namespace {


constexpr int kMaxSparseWarps = 16;

// token-phase shared memory, in 4-byte words, after the two tile arrays (PT = routed tiles of 16 tokens)
__host__ __device__ constexpr int token_phase_words(int PT, int K_c, int D = kHeadDim)
{
    return PT * 16 /*keys*/ + (PT * 16 + 3) / 4 /*take*/ + 2 * K_c + 2 /*voff*/ + K_c /*wgt*/ +
           K_c /*score*/ + 256 + 16 + 72 + kTopkList + kMaxSparseWarps * D + kMaxSparseWarps + 4;
}

// first word of the block-table copy: after the two tile arrays and the larger of the two phases
__host__ __device__ inline int bt_stage_offset_words(int max_pages, int P, int PT, int K_c, bool fused,
                                                     int D = kHeadDim)
{
    int words = token_phase_words(PT, K_c, D);
    if (fused && select_pages_words(max_pages, P) > words) words = select_pages_words(max_pages, P);
    return 2 * PT + words;
}

// Two-level front end (PAGE_KPT == -2): [selection over the super-pages | exact keys of the pages inside the
// kept super-pages, 16 per super-page | selection over those], all dead before the token phase
__host__ __device__ inline int two_level_words(int max_pages, int P, int P_super)
{
    const int max_supers = (max_pages + 15) / 16;
    return select_pages_words(max_supers, P_super) + 16 * P_super + select_pages_words(16 * P_super, P);
}
__host__ __device__ inline int two_level_smem_words(int max_pages, int P, int PT, int K_c, int P_super)
{
    const int a = token_phase_words(PT, K_c), b = two_level_words(max_pages, P, P_super);
    return 2 * PT + (a > b ? a : b);
}

// rows of the candidate key tile of the iterative solve: K_c rounded up to whole half-warps of
// sixteen, plus sixteen rows of zeros for the half-warps that own no candidate
__host__ __device__ constexpr int solve_tile_rows(int K_c) { return ((K_c + 15) & ~15) + 16; }

// first word of that tile ([rows][128] bf16, 16-byte aligned): after the block-table copy when there
// is one
__host__ __device__ inline int solve_tile_offset_words(int max_pages, int P, int PT, int K_c, bool fused, bool staged)
{
    const int w = bt_stage_offset_words(max_pages, P, PT, K_c, fused) + (staged ? max_pages : 0);
    return (w + 3) & ~3;
}

struct TokenSmem {
    uint32_t* keys;   // [PT * 16] token score keys, array index = 16 * slot + token (position order)
    uint8_t* take;    // [PT * 16] scratch of the selection's slow path
    long long* voff;  // [K_c] element offset of each candidate's value row, candidates in position order
    float* wgt;       // [K_c] unnormalised softmax weight of each candidate
    float* score;     // [K_c] score of each candidate (read by the iterative solve only)
    TopkScratch ts;
    float* red;       // [warps][D]
    float* zred;      // [warps]
};

__device__ __forceinline__ TokenSmem carve_tokens(uint32_t* base, int PT, int K_c, int D = kHeadDim)
{
    TokenSmem s;
    const int N = PT * 16;
    s.keys = base;
    s.take = (uint8_t*)(s.keys + N);
    uint32_t* after_take = s.keys + N + (N + 3) / 4;
    after_take += ((uintptr_t)after_take & 4u) ? 1 : 0;   // 8-byte alignment of the offsets
    s.voff = (long long*)after_take;
    s.wgt = (float*)(s.voff + K_c);
    s.score = s.wgt + K_c;
    s.ts.hist = (uint32_t*)(s.score + K_c);
    s.ts.misc = s.ts.hist + 256;
    s.ts.wred = s.ts.misc + 16;
    s.ts.list = (int32_t*)(s.ts.wred + 72);
    s.red = (float*)(s.ts.list + kTopkList);
    s.zred = s.red + kMaxSparseWarps * D;
    return s;
}

__device__ __forceinline__ void write_failed_unit(float* out, vsa_diag_t* diag, long long unit, int status,
                                                  int D = kHeadDim)
{
    for (int e = threadIdx.x; e < D; e += blockDim.x) out[unit * D + e] = 0.0f;
    if (threadIdx.x == 0) {
        vsa_diag_t d;
        d.delta = d.delta12 = d.s_max = d.lse = d.leak_bound = 0.0f;
        d.n_candidates = 0;
        d.fallback = 0;
        d.status = status;
        diag[unit] = d;
    }
}

// THREADS: 256 (two blocks per SM; the throughput shape), 512 (one block per SM; used when there
//   are no more units than SMs, so that one unit gets twice the loads in flight and half the passes)
//   or 128 (four blocks per SM; used when there are more units than two blocks per SM hold: more
//   units in flight, fewer waves).
// PAGE_KPT ==  0: routed_pages is an input.
// PAGE_KPT == -1: fused with routing; page scores staged in shared memory (any block-table width).
// PAGE_KPT == -2: fused with two-level routing; page_scores holds the unit's scores of the super-pages'
//   representatives [unit][ceil(max_pages / 16)]; the P_super best super-pages are kept, the pages inside
//   them scored exactly from tl_summaries, and the top-P of those routed.
// PAGE_KPT  >  0: fused with routing; each thread keeps PAGE_KPT page scores in registers.
//   In both fused forms the unit's top-P pages are selected here from page_scores[unit][0..n_b) and
//   written to routed_pages (best first, -1 padded).
// TOK_KPT: token scores per thread, P * 16 <= TOK_KPT * THREADS.
// SOLVE 1: the weights on the candidates come from `solver_iters` entropic mirror-descent iterations;
// SOLVE 2: from `solver_iters` Frank-Wolfe iterations with exact line search on the unregularised
//   problem (256 threads only: every lane owns one candidate, every half-warp sixteen candidate rows).
// CERT (fused register variants only): the certified gap of the unit - an upper bound on every score
//   of the pages that were not routed, from the pages' radii (rad_logical, written by the scan) -
//   is computed, reported in cert[] and used for the fallback decision in place of the proxy gap.
// D: head dimension.  A row is spread over the 16 lanes of a half-warp in pieces of 8 elements: lane c holds
//   elements 8c .. 8c+7 and, at D = 256, 128 + 8c .. 128 + 8c + 7 as well (its partial is the sum of the two
//   pieces' partials: the first level of the 32-partial tree); at D = 64 only lanes 0 .. 7 hold data, the
//   others contribute +0.  Iterative solves, certificate and the two-level front end exist at D = 128 only.
// FP8: k_cache / v_cache hold e4m3 bytes, value = byte * scale with one scale per (pool page, KV head) in
//   k_scale / v_scale (fp32 [pool pages][n_kv_heads]); strides are in elements (= bytes).  The decoded bytes go
//   through the same fixed-order dot and the score is multiplied by the scale afterwards; with power-of-two
//   scales that is exact and every discrete result equals that of a bf16 cache holding the same values.  Closed-form family, D = 128.
template <int THREADS, int PAGE_KPT, int TOK_KPT, int SOLVE = 0, bool CERT = false, int D = kHeadDim, bool FP8 = false>
__global__ void __launch_bounds__(THREADS, 512 / THREADS)
sparse_decode_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_cache,
                     const uint16_t* __restrict__ v_cache, const int32_t* __restrict__ block_table,
                     const int32_t* __restrict__ seq_lens, int32_t* __restrict__ routed_pages,
                     const float* __restrict__ page_scores, int P, int K_c, float epsilon, float gap_threshold,
                     float* __restrict__ out, vsa_diag_t* __restrict__ diag, int32_t* __restrict__ fallback_list,
                     int32_t* __restrict__ fallback_count, int solver_iters, vsa_solve_t* __restrict__ solve,
                     const float* __restrict__ rad_logical, vsa_cert_t* __restrict__ cert,
                     const int32_t* __restrict__ unit_list, const int32_t* __restrict__ unit_count,
                     int routed_stride,
                     const uint16_t* __restrict__ tl_summaries, int P_super,
                     const float* __restrict__ k_scale, const float* __restrict__ v_scale)
{
    constexpr int WARPS = THREADS / 32, GROUPS = 2 * WARPS;
    static_assert(PAGE_KPT != -2 || (SOLVE == 0 && !CERT), "two-level front end: plain family only");
    static_assert(D == 128 || ((D == 64 || D == 256) && SOLVE == 0 && !CERT && PAGE_KPT != -2), "other head dimensions: plain family");
    static_assert(!FP8 || (D == 128 && SOLVE == 0 && !CERT && PAGE_KPT != -2), "fp8 cache: closed-form family, D = 128");
    constexpr int PIECES = D == 256 ? 2 : 1;
    static_assert(SOLVE == 0 || THREADS == 256, "the solve maps one candidate to each of 256 lanes");
    static_assert(!CERT || PAGE_KPT > 0, "the certificate needs every page score of the unit in registers");
    static_assert(TOK_KPT * WARPS <= 64 && 4 * WARPS <= 72, "wred capacity");
    extern __shared__ uint32_t smem_raw[];
    // The token phases work on tiles of 16 rows: a routed page is 1 << tile_shift of them (one at 16 tokens
    // per page, two at 32).  Tile v of the sequence holds tokens 16 v .. 16 v + 15.
    const int tsh = geo.tile_shift, PT = P << tsh;
    int32_t* page_l = (int32_t*)smem_raw;   // [PT] tiles of the routed pages, ascending, invalid entries last
    int32_t* page_phys = page_l + PT;       // [PT] pool page of each tile
    uint32_t* region = smem_raw + 2 * PT;   // page-selection scratch first, token-phase arrays afterwards
    const int N = PT * 16;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, c = lane & 15, gi = lane >> 4;
    // unit_list != nullptr: block i handles unit_list[i] for i < *unit_count (a retry pass over the units
    // an earlier pass of the same step listed); the list is that pass's product, so it is read after
    // the wait
    long long unit = blockIdx.x;
    if (unit_list) {
        pdl_wait();
        if ((int)blockIdx.x >= __ldcg(unit_count)) {
            pdl_launch_dependents();
            return;
        }
        unit = __ldcg(unit_list + blockIdx.x);
    }
    const int b = (int)(unit / geo.n_q_heads), h = (int)(unit % geo.n_q_heads), g = h / geo.group;
    // Loads that depend on nothing computed in this step go out before the wait on the preceding
    // kernel: the sequence length, the query row (the routing kernel that precedes this one in a step
    // has read it already) and a copy of the block-table row for the page lookups that follow the
    // selection.  The page scores, which that kernel writes, are fetched right after the wait (the
    // sequence length, asked for before it, has arrived by then).
    const int32_t* bt = block_table + (long long)b * geo.max_pages;
    const int T = ld_ca_s32(seq_lens + b);
    const bool lane_has = D != 64 || c < 8;   // this lane holds a piece of every row
    const uint4 qraw = lane_has ? ld_nc_16B(q + unit * D + c * 8) : make_uint4(0u, 0u, 0u, 0u);
    const uint4 qraw1 = PIECES == 2 ? ld_nc_16B(q + unit * D + 128 + c * 8) : make_uint4(0u, 0u, 0u, 0u);
    int32_t* bt_s = (int32_t*)(smem_raw + bt_stage_offset_words(geo.max_pages, P, PT, K_c, PAGE_KPT > 0, D));
    if constexpr (PAGE_KPT > 0) {
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(bt_s);
        for (int i = tid; i < geo.max_pages; i += THREADS) cp_async_4(dst + 4u * (uint32_t)i, bt + i);
        cp_async_commit_group();
    }
    pdl_wait();
    pdl_launch_dependents();
    // Only the scores of the sequence's own pages are fetched: the rest of the scratch row was not
    // written in this step (in a ragged batch it is most of the row, and it would come from DRAM).
    const int nb_fetch = geo.length_ok(T) ? geo.pages_of(T) : 0;
    float praw[PAGE_KPT > 0 ? PAGE_KPT : 1];
    if constexpr (PAGE_KPT > 0) {
#pragma unroll
        for (int j = 0; j < PAGE_KPT; ++j) {
            const int i = tid + j * THREADS;
            praw[j] = i < nb_fetch ? ld_cg_f32(page_scores + unit * geo.max_pages + i) : 0.0f;
        }
    }
    float prad[CERT ? PAGE_KPT : 1];
    if constexpr (CERT) {
#pragma unroll
        for (int j = 0; j < PAGE_KPT; ++j) {
            const int i = tid + j * THREADS;
            prad[j] = i < nb_fetch
                          ? ld_cg_f32(rad_logical + ((long long)b * geo.n_kv_heads + g) * geo.max_pages + i)
                          : 0.0f;
        }
    }
    if (!geo.length_ok(T)) {
        cp_async_wait_all();
        write_failed_unit(out, diag, unit, VSA_UNIT_BAD_LENGTH, D);
        if (SOLVE && tid == 0) solve[unit] = vsa_solve_t{0.0f, 0.0f, 0.0f, 0.0f};
        if (CERT && tid == 0) cert[unit] = vsa_cert_t{0.0f, 0.0f, 0.0f, 0};
        if (PAGE_KPT != 0)
            for (int t = tid; t < routed_stride; t += THREADS) routed_pages[unit * routed_stride + t] = -1;
        return;
    }
    const int nb = geo.pages_of(T);

    // ---- routed pages -> page_l[] sorted by logical page, so that array order = position order ----
    int np;
    int bad = 0;
    if constexpr (PAGE_KPT != 0) {
        const PageSelectSmem ps =
            PAGE_KPT == -2 ? carve_page_select(region + select_pages_words((geo.max_pages + 15) >> 4, P_super) + 16 * P_super,
                                               16 * P_super, P)
                           : carve_page_select(region, geo.max_pages, P);
        if constexpr (PAGE_KPT > 0) {
            uint32_t pkey[PAGE_KPT];
#pragma unroll
            for (int j = 0; j < PAGE_KPT; ++j)
                pkey[j] = tid + j * THREADS < nb ? float_to_key(praw[j]) : 0u;
            cp_async_wait_all();   // this thread's part of the block-table copy; the selection's barriers publish it
            np = select_top_pages_keys<PAGE_KPT>(pkey, nb, P, ps);
            if constexpr (CERT) {
                // |q| (rounded up a little), every lane of a half-warp computing the same value
                float qe[8];
                unpack8(qraw, qe);
                float q2 = chunk_partial(qe, qe);
#pragma unroll
                for (int off = 8; off; off >>= 1) q2 = q2 + __shfl_xor_sync(kFullMask, q2, off);
                const float qn = __fmul_rn(__fsqrt_rn(q2), 1.00000095367431640625f);
                // a page is un-routed iff it is ordered after the last winner (score descending, index
                // ascending); its tokens score at most  c + |q| * radius
                const uint32_t k_last = ps.win_key[np - 1];
                const int i_last = ps.win_idx[np - 1];
                uint32_t ub_key = 0u;
#pragma unroll
                for (int j = 0; j < PAGE_KPT; ++j) {
                    const int i = tid + j * THREADS;
                    const bool unrouted = pkey[j] != 0u && ((pkey[j] < k_last) | ((pkey[j] == k_last) & (i > i_last)));
                    if (unrouted)
                        ub_key = max(ub_key, float_to_key(__fadd_rn(key_to_float(pkey[j]), __fmul_rn(qn, prad[j]))));
                }
                ub_key = __reduce_max_sync(kFullMask, ub_key);
                if (lane == 0) ps.ts.wred[warp] = ub_key;   // published by the barrier below, read right after it
            }
        } else if constexpr (PAGE_KPT == -1) {
            np = select_top_pages(page_scores + unit * geo.max_pages, nb, P, ps);
        }
        // position -> logical page of a winner (two-level: position 16 j + c is page c of the j-th kept
        // super-page in ascending order)
        const int32_t* asc_super = nullptr;
        if constexpr (PAGE_KPT == -2) {
            const int max_supers = (geo.max_pages + 15) >> 4, ns = (nb + 15) >> 4;
            const PageSelectSmem ps1 = carve_page_select(region, max_supers, P_super);
            uint32_t* exact = region + select_pages_words(max_supers, P_super);
            uint32_t skey[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = tid + j * THREADS;
                skey[j] = i < ns ? float_to_key(ld_cg_f32(page_scores + unit * max_supers + i)) : 0u;
            }
            if (tid == 0) ps1.ts.misc[12] = 0u;   // pages that get a score (a word the selection does not use)
            const int Ks = select_top_pages_keys<8>(skey, ns, P_super, ps1);   // ends with a barrier
            asc_super = ps1.asc_idx;
            float qe[8];
            unpack8(qraw, qe);
            // one kept super-page = 16 summary rows = one 16-value reduction per half-warp; lane c ends with
            // the exact score of page 16 s + c
            for (int j0 = warp * 2; j0 < Ks; j0 += GROUPS) {
                const int j = j0 + gi;
                const bool have = j < Ks;
                const int l = have ? asc_super[j] * 16 + c : nb;
                long long phys = -1;
                if (l < nb) {
                    phys = bt[l];
                    if (phys < 0 || phys >= geo.pool_pages) phys = -1;
                }
                uint4 srows[16];
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    const long long pr = __shfl_sync(kFullMask, phys, (lane & 16) | r);
                    srows[r] = pr >= 0 ? ld_nc_16B(tl_summaries + (pr * geo.n_kv_heads + g) * kHeadDim + c * 8)
                                       : make_uint4(0u, 0u, 0u, 0u);
                }
                float vals[16];
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    float kf[8];
                    unpack8(srows[r], kf);
                    vals[r] = chunk_partial(qe, kf);
                }
                const float sc = reduce_scatter16(vals, c);
                const bool scored = have && phys >= 0;
                if (have) exact[j * 16 + c] = scored ? float_to_key(sc) : 0u;
                const int n_ok = __popc(__ballot_sync(kFullMask, scored));
                if (lane == 0 && n_ok) atomicAdd(&ps1.ts.misc[12], (uint32_t)n_ok);
            }
            __syncthreads();
            const int n2 = Ks * 16, P2 = min(P, (int)ps1.ts.misc[12]);
            uint32_t pkey2[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = tid + j * THREADS;
                pkey2[j] = i < n2 ? exact[i] : 0u;
            }
            np = P2 > 0 ? select_top_pages_keys<8>(pkey2, n2, P2, ps) : 0;
        }
        auto page_of = [&](int pos) { return PAGE_KPT == -2 ? asc_super[pos >> 4] * 16 + (pos & 15) : pos; };
        for (int t = P + tid; t < routed_stride; t += THREADS) routed_pages[unit * routed_stride + t] = -1;
        for (int t = tid; t < P; t += THREADS) {
            routed_pages[unit * routed_stride + t] = t < np ? page_of(ps.win_idx[t]) : -1;
            int l = INT_MAX, phys = -1;
            if (t < np) {
                l = page_of(ps.asc_idx[t]);
                phys = PAGE_KPT > 0 ? bt_s[l] : bt[l];
                if (phys < 0 || phys >= geo.pool_pages) {
                    phys = -1;
                    bad = 1;
                }
            }
            for (int hf = 0; hf < (1 << tsh); ++hf) {
                page_l[(t << tsh) + hf] = l == INT_MAX ? INT_MAX : (l << tsh) + hf;
                page_phys[(t << tsh) + hf] = phys;
            }
        }
    } else {
        int32_t* raw = (int32_t*)region;   // staging; dead before the token phase reuses the region
        for (int t = tid; t < P; t += THREADS) {
            const int l = routed_pages[unit * routed_stride + t];
            raw[t] = (l >= 0 && l < nb) ? l : INT_MAX;
        }
        __syncthreads();
        for (int t = tid; t < P; t += THREADS) {
            const int l = raw[t];
            int rank = 0;
#pragma unroll 8
            for (int j = 0; j < P; ++j) rank += (int)((raw[j] < l) | ((raw[j] == l) & (j < t)));
            int phys = -1;
            if (l != INT_MAX) {
                phys = bt[l];
                if (phys < 0 || phys >= geo.pool_pages) {
                    phys = -1;
                    bad = 1;
                }
            }
            for (int hf = 0; hf < (1 << tsh); ++hf) {
                page_l[(rank << tsh) + hf] = l == INT_MAX ? INT_MAX : (l << tsh) + hf;
                page_phys[(rank << tsh) + hf] = phys;
            }
        }
        // (P <= 128 < THREADS: thread t < P owns slot t in the count)
        np = __syncthreads_count(tid < P && raw[tid < P ? tid : 0] != INT_MAX);
    }
    const int any_bad = __syncthreads_or(bad);
    uint32_t ub_unrouted_key = 0u;   // CERT: key of the best upper bound over the un-routed pages, 0 = none
    if constexpr (CERT) {
        const PageSelectSmem ps = carve_page_select(region, geo.max_pages, P);
#pragma unroll
        for (int w = 0; w < WARPS; ++w) ub_unrouted_key = max(ub_unrouted_key, ps.ts.wred[w]);
        __syncthreads();   // the selection scratch is rewritten by the token phase
    }
    if (any_bad) {
        write_failed_unit(out, diag, unit, VSA_UNIT_BAD_PAGE, D);
        if (SOLVE && tid == 0) solve[unit] = vsa_solve_t{0.0f, 0.0f, 0.0f, 0.0f};
        if (CERT && tid == 0) cert[unit] = vsa_cert_t{0.0f, 0.0f, 0.0f, 0};
        return;
    }
    const TokenSmem sm = carve_tokens(region, PT, K_c, D);
    const int nt = np << tsh;   // tiles of the routed pages
#pragma unroll
    for (int j = 0; j < TOK_KPT; ++j)
        if (tid + j * THREADS < N) sm.keys[tid + j * THREADS] = 0u;
    __syncthreads();

    // ---- token routing: score all 16 tokens of a page per half-warp ----
    float qf[8];
    unpack8(qraw, qf);
    float qf1[8];
    unpack8(qraw1, qf1);
    for (int pp = warp; pp * 2 < nt; pp += WARPS) {
        const int slot = pp * 2 + gi;
        const bool active = slot < nt;
        float vals[16];
        float kscale = 1.0f;
        if constexpr (FP8) {
            uint2 rows[16];
            if (active) {
                const uint8_t* src = reinterpret_cast<const uint8_t*>(k_cache) + (long long)page_phys[slot] * geo.page_stride +
                                     (long long)g * geo.head_stride + c * 8 +
                                     (long long)((page_l[slot] & ((1 << tsh) - 1)) * 16) * geo.token_stride;
                kscale = __ldg(k_scale + (long long)page_phys[slot] * geo.n_kv_heads + g);
#pragma unroll
                for (int t = 0; t < 16; ++t) rows[t] = ld_nc_8B(src + (long long)t * geo.token_stride);
            } else {
#pragma unroll
                for (int t = 0; t < 16; ++t) rows[t] = make_uint2(0u, 0u);
            }
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                float kf[8];
                unpack8_e4m3(rows[t], kf);
                vals[t] = chunk_partial(qf, kf);
            }
        } else {
#pragma unroll
        for (int pc = 0; pc < PIECES; ++pc) {
            uint4 rows[16];
            if (active && lane_has) {
                const uint16_t* src = k_cache + (long long)page_phys[slot] * geo.page_stride +
                                      (long long)g * geo.head_stride + c * 8 + pc * 128 +
                                      (long long)((page_l[slot] & ((1 << tsh) - 1)) * 16) * geo.token_stride;
#pragma unroll
                for (int t = 0; t < 16; ++t) rows[t] = ld_nc_16B(src + (long long)t * geo.token_stride);
            } else {
#pragma unroll
                for (int t = 0; t < 16; ++t) rows[t] = make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                float kf[8];
                unpack8(rows[t], kf);
                const float part = chunk_partial(pc == 0 ? qf : qf1, kf);
                vals[t] = pc == 0 ? part : vals[t] + part;
            }
        }
        }
        float s = reduce_scatter16(vals, c);   // lane c: score of token c of the page
        if constexpr (FP8) s = __fmul_rn(s, kscale);   // exact: a power of two
        if (active && page_l[slot] * 16 + c < T) sm.keys[slot * 16 + c] = float_to_key(s);
    }
    __syncthreads();

    // ---- every thread takes its TOK_KPT token keys into registers ----
    uint32_t key[TOK_KPT];
    int present = 0;
    uint32_t a1 = 0u, a2 = 0u;   // best and second-best key (multiset order statistics)
    uint32_t amin = 0xffffffffu;  // smallest present key
#pragma unroll
    for (int j = 0; j < TOK_KPT; ++j) {
        const int i = tid + j * THREADS;
        key[j] = i < N ? sm.keys[i] : 0u;
        present += key[j] != 0u;
        if (key[j] != 0u) amin = min(amin, key[j]);
        if (key[j] > a1) {
            a2 = a1;
            a1 = key[j];
        } else if (key[j] > a2) {
            a2 = key[j];
        }
    }
    // number of valid scored tokens, the two best keys and the smallest key: per warp with the
    // single-instruction warp reductions, then across the warps through shared memory.  Each warp
    // also publishes its best key: the smallest of those (hi_r) and the largest of the warps' smallest
    // keys (lo_r) bracket the bulk of the scores and serve as the histogram range of the selection.
    {
        present = __reduce_add_sync(kFullMask, present);
        amin = __reduce_min_sync(kFullMask, amin);
        const uint32_t wmax = __reduce_max_sync(kFullMask, a1);
        const int holder = __ffs(__ballot_sync(kFullMask, a1 == wmax)) - 1;
        const uint32_t wsecond = __reduce_max_sync(kFullMask, lane == holder ? a2 : a1);
        a1 = wmax;
        a2 = wsecond;
    }
    if (lane == 0) {
        sm.ts.wred[4 * warp] = a1;
        sm.ts.wred[4 * warp + 1] = a2;
        sm.ts.wred[4 * warp + 2] = (uint32_t)present;
        sm.ts.wred[4 * warp + 3] = amin;
    }
    // the selection below starts from a cleared histogram and list counter
    for (int i = tid; i < 256; i += THREADS) sm.ts.hist[i] = 0u;
    if (tid == 0) sm.ts.misc[4] = 0u;
    __syncthreads();
    uint32_t key1 = 0u, key2 = 0u, kmin = 0xffffffffu, hi_r = 0xffffffffu, lo_r = 0u;
    int n_valid = 0;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) {
        const uint32_t b1 = sm.ts.wred[4 * w], b2 = sm.ts.wred[4 * w + 1], bmin = sm.ts.wred[4 * w + 3];
        const uint32_t n1 = max(key1, b1), n2 = max(min(key1, b1), max(key2, b2));
        key1 = n1;
        key2 = n2;
        n_valid += (int)sm.ts.wred[4 * w + 2];
        kmin = min(kmin, bmin);
        if (b1 != 0u) hi_r = min(hi_r, b1);                 // warps without a valid token do not count
        if (bmin != 0xffffffffu) lo_r = max(lo_r, bmin);
    }
    const int ns = min(K_c, n_valid);

    // ---- exact top-(ns+1): its last element is the best rejected token, the rest are the candidates ----
    uint32_t out_key = 0u, mask = 0u;
    const bool has_rejected = n_valid > ns;
    if (has_rejected) {
        // token scores are finite, so the smallest and largest keys are the range of the finite scores
        // (when the bracket is empty or inverted the selection falls back to the full range itself)
        const TopkRegResult r = block_topk_reg<TOK_KPT, true>(key, N, ns + 1, sm.ts, sm.keys, sm.take,
                                                             key_to_float(lo_r), key_to_float(hi_r),
                                                             key_to_float(kmin), key_to_float(key1));
        out_key = r.kth_key;
        mask = r.mask;
#pragma unroll
        for (int j = 0; j < TOK_KPT; ++j)
            if (tid + j * THREADS == r.kth_idx) mask &= ~(1u << j);
    } else {
#pragma unroll
        for (int j = 0; j < TOK_KPT; ++j)
            if (key[j] != 0u) mask |= 1u << j;
        __syncthreads();   // wred is rewritten by the compaction
    }

    // ---- ordered compaction of the candidates (position order); the thread that holds a candidate's
    //      key writes the address of its value row and its softmax weight ----
    const float s1 = ns > 0 ? key_to_float(key1) : -INFINITY;
    const float scale = 1.4426950408889634f / epsilon;   // log2(e) / epsilon
    {
        int before[TOK_KPT];
#pragma unroll
        for (int j = 0; j < TOK_KPT; ++j) {
            const unsigned bal = __ballot_sync(kFullMask, (mask >> j) & 1u);
            before[j] = __popc(bal & ((1u << lane) - 1u));
            if (lane == 0) sm.ts.wred[j * WARPS + warp] = (uint32_t)__popc(bal);
        }
        __syncthreads();
        int base = 0;
#pragma unroll
        for (int j = 0; j < TOK_KPT; ++j) {
            // elements of row j (indices j * THREADS + tid) come after all of rows < j
            int mine = base;
#pragma unroll
            for (int w = 0; w < WARPS; ++w) {
                const int cw = (int)sm.ts.wred[j * WARPS + w];
                if (w < warp) mine += cw;
                base += cw;
            }
            if ((mask >> j) & 1u) {
                const int i = tid + j * THREADS, pos = mine + before[j];
                sm.voff[pos] = (long long)page_phys[i >> 4] * geo.page_stride +
                               (long long)((page_l[i >> 4] & ((1 << tsh) - 1)) * 16 + (i & 15)) * geo.token_stride;
                sm.wgt[pos] = exp2f((key_to_float(key[j]) - s1) * scale);
                if constexpr (SOLVE != 0) sm.score[pos] = key_to_float(key[j]);
                // fp8: the scale of the candidate's value row (the score array is free in the closed-form family)
                if constexpr (FP8) sm.score[pos] = __ldg(v_scale + (long long)page_phys[i >> 4] * geo.n_kv_heads + g);
            }
        }
    }
    __syncthreads();

    float lse_closed = 0.0f;   // log-sum-exp of the closed-form weights (SOLVE only)
    if constexpr (SOLVE != 0) {
        if (ns > 0) {
            // ---- iterative entropic solve on the candidates (Eq. (5.1) restricted to S) ----
            // Lane (half-warp hw, column c) owns candidate j = 16 * hw + c: its score, log-weight and
            // gradient entry live in registers.  Half-warp hw keeps the key rows of its sixteen
            // candidates in shared memory, lane c reading column c of each.
            const int hw = warp * 2 + gi, j_own = hw * 16 + c;
            const bool have = j_own < ns;
            uint8_t* ktile = (uint8_t*)(smem_raw + solve_tile_offset_words(geo.max_pages, P, PT, K_c, PAGE_KPT != 0,
                                                                           PAGE_KPT > 0));
            // a half-warp without candidates works on the block of sixteen zero rows behind the tile
            const int my_first = hw * 16 < ns ? hw * 16 : solve_tile_rows(K_c) - 16;
            uint8_t* my_rows = ktile + (size_t)my_first * kRowBytes + c * 16;   // row r at + r * kRowBytes
            {
                const uint32_t dst = (uint32_t)__cvta_generic_to_shared(my_rows);
                const uint16_t* kbase = k_cache + (long long)g * geo.head_stride + c * 8;
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    if (hw * 16 + r < ns)
                        cp_async_16B(dst + r * kRowBytes, kbase + sm.voff[hw * 16 + r]);
                    else
                        *reinterpret_cast<uint4*>(my_rows + r * kRowBytes) = make_uint4(0u, 0u, 0u, 0u);
                }
                cp_async_commit_group();
                cp_async_wait_all();
                __syncwarp();
            }
            const float s_own = have ? sm.score[j_own] : 0.0f;
            float vals[16];
            if constexpr (SOLVE == 2) {
                // ---- Frank-Wolfe with exact line search on f(a) = 1/2 |sum a_i k_i - q|^2 (App. E) ----
                // Vertex choices are integers, so everything that feeds them is single-rounded fp32 in the
                // canonical order (mirrored by the oracle): the readout y = sum a_i k_i is kept incrementally
                // (lane c holds elements 8c .. 8c+7, every half-warp the same copy), g_i = <k_i, y> - s_i by
                // the fixed-order dot, argmin with ties to the lower position, gamma by an IEEE division.
                __syncthreads();   // rows staged by other half-warps are read below
                // block-wide best (largest key, then smallest candidate index); `slot` alternates so that a
                // fast warp cannot overwrite statistics that a slow one still reads
                auto arg_best = [&](uint32_t key, int slot, uint32_t& best_key, int& best_j) {
                    const uint32_t wk = __reduce_max_sync(kFullMask, key);
                    const int wj = __reduce_min_sync(kFullMask, (key == wk && key != 0u) ? j_own : INT_MAX);
                    if (lane == 0) {
                        sm.ts.wred[slot * 16 + warp] = wk;
                        sm.ts.wred[slot * 16 + 8 + warp] = (uint32_t)wj;
                    }
                    __syncthreads();
                    best_key = 0u;
                    best_j = INT_MAX;
#pragma unroll
                    for (int w = 0; w < WARPS; ++w) {
                        const uint32_t k = sm.ts.wred[slot * 16 + w];
                        const int j = (int)sm.ts.wred[slot * 16 + 8 + w];
                        if (k > best_key || (k == best_key && j < best_j)) {
                            best_key = k;
                            best_j = j;
                        }
                    }
                };
                // closed-form log-sum-exp for diag (the weights written at the compaction), and the start
                {
                    float w0 = have ? sm.wgt[j_own] : 0.0f;
#pragma unroll
                    for (int off = 16; off; off >>= 1) w0 += __shfl_xor_sync(kFullMask, w0, off);
                    if (lane == 0) sm.ts.wred[56 + warp] = __float_as_uint(w0);
                }
                uint32_t bk;
                int jb;
                arg_best(have ? float_to_key(s_own) : 0u, 0, bk, jb);
                {
                    float z0 = 0.0f;
#pragma unroll
                    for (int w = 0; w < WARPS; ++w) z0 += __uint_as_float(sm.ts.wred[56 + w]);
                    lse_closed = s1 / epsilon + logf(z0);
                }
                float yv[8];
                unpack8(*reinterpret_cast<const uint4*>(ktile + (size_t)jb * kRowBytes + c * 16), yv);
                float a_own = (have && j_own == jb) ? 1.0f : 0.0f;
                float gamma = 0.0f, gmin = 0.0f;
                auto tree16 = [&](float p) {   // canonical halving tree over the half-warp, result in every lane
#pragma unroll
                    for (int off = 8; off; off >>= 1) p = p + __shfl_xor_sync(kFullMask, p, off);
                    return p;
                };
                for (int it = 0;; ++it) {
#pragma unroll
                    for (int r = 0; r < 16; ++r) {
                        float uf[8];
                        unpack8(*reinterpret_cast<const uint4*>(my_rows + r * kRowBytes), uf);
                        vals[r] = chunk_partial(yv, uf);
                    }
                    const float g_own = reduce_scatter16(vals, c) - s_own;
                    arg_best(have ? float_to_key(-g_own) : 0u, 1 + (it & 1), bk, jb);
                    gmin = -key_to_float(bk);
                    if (it >= solver_iters) break;
                    float uj[8], dv[8], rv[8];
                    unpack8(*reinterpret_cast<const uint4*>(ktile + (size_t)jb * kRowBytes + c * 16), uj);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        dv[e] = __fsub_rn(uj[e], yv[e]);
                        rv[e] = __fsub_rn(qf[e], yv[e]);
                    }
                    const float num = tree16(chunk_partial(rv, dv)), den = tree16(chunk_partial(dv, dv));
                    gamma = den > 0.0f ? __fdiv_rn(num, den) : 0.0f;
                    gamma = gamma < 0.0f ? 0.0f : (gamma > 1.0f ? 1.0f : gamma);
#pragma unroll
                    for (int e = 0; e < 8; ++e) yv[e] = __fmaf_rn(gamma, dv[e], yv[e]);
                    a_own = __fmaf_rn(-gamma, a_own, a_own);
                    if (have && j_own == jb) a_own = __fadd_rn(a_own, gamma);
                }
                {
                    float rv[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) rv[e] = __fsub_rn(yv[e], qf[e]);
                    const float r2 = tree16(chunk_partial(rv, rv)), yr = tree16(chunk_partial(yv, rv));
                    if (tid == 0) {
                        vsa_solve_t sv;
                        sv.fw_gap = __fsub_rn(yr, gmin);
                        sv.objective = __fmul_rn(0.5f, r2);
                        sv.residual2 = r2;
                        sv.step = gamma;
                        solve[unit] = sv;
                    }
                }
                if (have) sm.wgt[j_own] = a_own;
                __syncthreads();
            } else {
            // step: eta = 1 / max_i |k_i|^2
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                float uf[8];
                unpack8(*reinterpret_cast<const uint4*>(my_rows + r * kRowBytes), uf);
                vals[r] = chunk_partial(uf, uf);
            }
            {
                const float nrm = reduce_scatter16(vals, c);
                const uint32_t wmax = __reduce_max_sync(kFullMask, have ? float_to_key(nrm) : 0u);
                if (lane == 0) sm.ts.wred[warp] = wmax;
            }
            __syncthreads();
            uint32_t lkey = 0u;
#pragma unroll
            for (int w = 0; w < WARPS; ++w) lkey = max(lkey, sm.ts.wred[w]);
            const float Lmax = lkey != 0u ? key_to_float(lkey) : 0.0f;
            const float eta = Lmax > 0.0f ? 1.0f / Lmax : 0.0f;
            const float shrink = 1.0f / (1.0f + eta * epsilon);
            float l_own = have ? s_own / epsilon : -INFINITY;
            float m = 0.0f, Z = 1.0f, a_own = 0.0f, g_own = 0.0f;
            float yq[8];
            __syncthreads();   // wred is rewritten below
            // One block barrier per pass: every warp exponentiates against its own maximum and publishes
            // (partial readout, partial sum, maximum); after the barrier every lane rebuilds the block-wide
            // readout for its own eight columns.  The buffers alternate between passes.
            for (int it = 0;; ++it) {
                const float mw = key_to_float(__reduce_max_sync(kFullMask, float_to_key(l_own)));
                const float e_own = have ? __expf(l_own - mw) : 0.0f;
                // sum_i e_i k_i over this half-warp's sixteen rows, then over the warp
                float ya[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) ya[e] = 0.0f;
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    const float e_r = __shfl_sync(kFullMask, e_own, (lane & 16) | r);
                    float uf[8];
                    unpack8(*reinterpret_cast<const uint4*>(my_rows + r * kRowBytes), uf);
#pragma unroll
                    for (int e = 0; e < 8; e += 2) fma2(ya[e], ya[e + 1], e_r, e_r, uf[e], uf[e + 1]);
                }
                float zw = e_own;
#pragma unroll
                for (int off = 16; off; off >>= 1) zw += __shfl_xor_sync(kFullMask, zw, off);
#pragma unroll
                for (int e = 0; e < 8; ++e) ya[e] += __shfl_xor_sync(kFullMask, ya[e], 16);
                float* redb = sm.red + (it & 1) * (WARPS * kHeadDim);
                uint32_t* statb = sm.ts.wred + (it & 1) * 16;   // [0..8) partial sums, [8..16) maxima
                if (gi == 0) {
                    // layout [warp][element pair][column]: the sixteen lanes of a half-warp touch 128
                    // consecutive bytes (the area is 8-byte aligned, not more)
#pragma unroll
                    for (int e = 0; e < 8; e += 2)
                        *reinterpret_cast<float2*>(redb + ((warp * 4 + e / 2) * 16 + c) * 2) = make_float2(ya[e], ya[e + 1]);
                    if (c == 0) {
                        statb[warp] = __float_as_uint(zw);
                        statb[8 + warp] = __float_as_uint(mw);
                    }
                }
                __syncthreads();
                m = -INFINITY;
#pragma unroll
                for (int w = 0; w < WARPS; ++w) m = fmaxf(m, __uint_as_float(statb[8 + w]));
                Z = 0.0f;
#pragma unroll
                for (int e = 0; e < 8; ++e) yq[e] = 0.0f;
#pragma unroll
                for (int w = 0; w < WARPS; ++w) {
                    const float mwv = __uint_as_float(statb[8 + w]);
                    const float f = mwv > -INFINITY ? __expf(mwv - m) : 0.0f;
                    Z = fmaf(__uint_as_float(statb[w]), f, Z);
#pragma unroll
                    for (int e = 0; e < 8; e += 2) {
                        const float2 p = *reinterpret_cast<const float2*>(redb + ((w * 4 + e / 2) * 16 + c) * 2);
                        yq[e] = fmaf(f, p.x, yq[e]);
                        yq[e + 1] = fmaf(f, p.y, yq[e + 1]);
                    }
                }
                {
                    const float rz = 1.0f / Z;
#pragma unroll
                    for (int e = 0; e < 8; ++e) yq[e] *= rz;
                }
                a_own = have ? e_own * __expf(mw - m) : 0.0f;   // exp(l_own - m)
                // gradient of the quadratic part: g_i = <k_i, y> - <k_i, q>
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    float uf[8];
                    unpack8(*reinterpret_cast<const uint4*>(my_rows + r * kRowBytes), uf);
                    vals[r] = chunk_partial(yq, uf);
                }
                g_own = reduce_scatter16(vals, c) - s_own;
                if (it == 0) lse_closed = m + logf(Z);
                if (it >= solver_iters) break;
                l_own = have ? ((l_own - m) - eta * g_own) * shrink : -INFINITY;
            }
            // certificate and objective at the final weights a_i = a_own / Z
            {
                const float alpha = a_own / Z;
                float sum_ag = have ? alpha * g_own : 0.0f;
                float ent = (have && alpha > 0.0f) ? alpha * ((l_own - m) - logf(Z)) : 0.0f;
                float r2 = 0.0f;
#pragma unroll
                for (int e = 0; e < 8; ++e) r2 += (yq[e] - qf[e]) * (yq[e] - qf[e]);
#pragma unroll
                for (int off = 8; off; off >>= 1) r2 += __shfl_xor_sync(kFullMask, r2, off);
#pragma unroll
                for (int off = 16; off; off >>= 1) {
                    sum_ag += __shfl_xor_sync(kFullMask, sum_ag, off);
                    ent += __shfl_xor_sync(kFullMask, ent, off);
                }
                // (-g) as a key: the largest key is the smallest gradient entry
                const uint32_t wmin = __reduce_max_sync(kFullMask, have ? float_to_key(-g_own) : 0u);
                if (lane == 0) {
                    sm.ts.wred[32 + warp] = wmin;
                    sm.ts.wred[40 + warp] = __float_as_uint(sum_ag);
                    sm.ts.wred[48 + warp] = __float_as_uint(ent);
                }
                if (have) sm.wgt[j_own] = a_own;
                __syncthreads();
                if (tid == 0) {
                    uint32_t gk = 0u;
                    float sag = 0.0f, en = 0.0f;
                    for (int w = 0; w < WARPS; ++w) {
                        gk = max(gk, sm.ts.wred[32 + w]);
                        sag += __uint_as_float(sm.ts.wred[40 + w]);
                        en += __uint_as_float(sm.ts.wred[48 + w]);
                    }
                    vsa_solve_t sv;
                    sv.fw_gap = sag + key_to_float(gk);   // <g, a> - min_j g_j
                    sv.objective = 0.5f * r2 + epsilon * en;
                    sv.residual2 = r2;
                    sv.step = eta;
                    solve[unit] = sv;
                }
            }
            }   // SOLVE == 1
        } else if (tid == 0) {
            solve[unit] = vsa_solve_t{0.0f, 0.0f, 0.0f, 0.0f};
        }
    }
    // ---- value gather ----
    float acc[PIECES][8], z = 0.0f;
#pragma unroll
    for (int pc = 0; pc < PIECES; ++pc)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[pc][e] = 0.0f;
    const int gidx = warp * 2 + gi;
    constexpr int UNR = THREADS == 512 ? 8 : 16;   // 256 threads, K_c = 256: every half-warp's rows in one batch
    if constexpr (FP8) {
        const uint8_t* vbase = reinterpret_cast<const uint8_t*>(v_cache) + (long long)g * geo.head_stride + c * 8;
        for (int j0 = gidx; j0 < ns; j0 += GROUPS * UNR) {
            uint2 rows[UNR];
            float w[UNR], ws[UNR];
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                const int j = j0 + u * GROUPS, jc = min(j, ns - 1);
                rows[u] = ld_nc_8B(vbase + sm.voff[jc]);
                w[u] = j < ns ? sm.wgt[jc] : 0.0f;
                ws[u] = w[u] * sm.score[jc];   // weight times the row's power-of-two scale
            }
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                float vf[8];
                unpack8_e4m3(rows[u], vf);
#pragma unroll
                for (int e = 0; e < 8; e += 2) fma2(acc[0][e], acc[0][e + 1], ws[u], ws[u], vf[e], vf[e + 1]);
                z += w[u];
            }
        }
    } else {
#pragma unroll
    for (int pc = 0; pc < PIECES; ++pc) {
        const uint16_t* vbase = v_cache + (long long)g * geo.head_stride + c * 8 + pc * 128;
        for (int j0 = gidx; j0 < ns; j0 += GROUPS * UNR) {
            // all value rows of the batch at once; slots past the candidate count re-read the last
            // candidate with weight 0
            uint4 rows[UNR];
            float w[UNR];
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                const int j = j0 + u * GROUPS, jc = min(j, ns - 1);
                rows[u] = lane_has ? ld_nc_16B(vbase + sm.voff[jc]) : make_uint4(0u, 0u, 0u, 0u);
                w[u] = j < ns ? sm.wgt[jc] : 0.0f;
            }
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                float vf[8];
                unpack8(rows[u], vf);
#pragma unroll
                for (int e = 0; e < 8; e += 2) fma2(acc[pc][e], acc[pc][e + 1], w[u], w[u], vf[e], vf[e + 1]);
                if (pc == 0) z += w[u];
            }
        }
    }
    }
#pragma unroll
    for (int pc = 0; pc < PIECES; ++pc)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[pc][e] += __shfl_xor_sync(kFullMask, acc[pc][e], 16);
    z += __shfl_xor_sync(kFullMask, z, 16);
    if (gi == 0) {
        if (lane_has) {
#pragma unroll
            for (int pc = 0; pc < PIECES; ++pc)
#pragma unroll
                for (int e = 0; e < 8; ++e) sm.red[warp * D + pc * 128 + c * 8 + e] = acc[pc][e];
        }
        if (c == 0) sm.zred[warp] = z;
    }
    __syncthreads();
    float Z = 0.0f;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) Z += sm.zred[w];
    for (int e = tid; e < D; e += THREADS) {
        float a = 0.0f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) a += sm.red[w * D + e];
        out[unit * D + e] = ns > 0 ? a / Z : 0.0f;
    }

    // ---- diagnostics and fallback flag ----
    if (tid == 0) {
        const float s2 = ns > 1 ? key_to_float(key2) : -INFINITY;
        const float delta = has_rejected ? s1 - key_to_float(out_key) : INFINITY;
        vsa_diag_t d;
        d.delta = delta;
        d.delta12 = ns > 0 ? s1 - s2 : INFINITY;
        d.s_max = s1;
        d.lse = ns > 0 ? (SOLVE ? lse_closed : s1 / epsilon + logf(Z)) : -INFINITY;
        d.leak_bound = fminf(1.0f, (float)(T - ns) * expf(-delta / epsilon));
        d.n_candidates = ns;
        d.fallback = (delta < gap_threshold && ns < T) ? 1 : 0;
        if constexpr (CERT) {
            const float ub = ub_unrouted_key != 0u ? key_to_float(ub_unrouted_key) : -INFINITY;
            const float rej = has_rejected ? key_to_float(out_key) : -INFINITY;
            const float m = fmaxf(rej, ub);
            vsa_cert_t ce;
            ce.ub_unrouted = ub;
            ce.delta_cert = m == -INFINITY ? INFINITY : s1 - m;
            ce.certified = ce.delta_cert >= gap_threshold ? 1 : 0;
            ce.leak_bound_cert = fminf(1.0f, (float)(T - ns) * expf(-ce.delta_cert / epsilon));
            cert[unit] = ce;
            d.fallback = (!ce.certified && ns < T) ? 1 : 0;   // the certified gap decides
        }
        d.status = 0;
        diag[unit] = d;
        if (d.fallback) fallback_list[atomicAdd(fallback_count, 1)] = (int32_t)unit;
    }
}

}  // namespace

// everything one launch of the fused kernel needs
struct SparseArgs {
    Geometry g;
    size_t smem;
    const uint16_t *q, *k, *v;
    const int32_t *block_table, *seq_lens;
    int32_t* routed_pages;
    const float* page_scores;
    int P, K_c;
    float epsilon, gap_threshold;
    float* out;
    vsa_diag_t* diag;
    int32_t *fallback_list, *fallback_count;
    int solver_iters, solver_kind;   // kind 1: entropic mirror descent, 2: Frank-Wolfe
    vsa_solve_t* solve;   // non-null: an iterative-solve variant of the kernel
    const float* rad_logical;
    vsa_cert_t* cert;     // non-null: the certificate variant (fused register variants only)
    const int32_t *unit_list, *unit_count;   // non-null: only the listed units (blocks beyond the count exit)
    int routed_stride;                       // row stride of routed_pages (>= P)
    const uint16_t* tl_summaries;            // non-null: two-level front end (page_scores = representative scores)
    int P_super;
    const float *k_scale, *v_scale;          // non-null: fp8 cache (one scale per pool page and KV head)
    cudaStream_t stream;
};


namespace {

template <int THREADS, int PAGE_KPT, int TOK_KPT, int SOLVE, bool CERT, int D = kHeadDim, bool FP8 = false>
cudaError_t launch_variant(const SparseArgs& a)
{
    static bool attr_done[kMaxDevices] = {};   // per template instance
    if (a.smem > 48 * 1024) {
        const cudaError_t e =
            allow_large_dynamic_smem(sparse_decode_kernel<THREADS, PAGE_KPT, TOK_KPT, SOLVE, CERT, D, FP8>, attr_done);
        if (e != cudaSuccess) return e;
    }
    const unsigned units = (unsigned)(a.g.batch * a.g.n_q_heads);
    return launch_pdl(sparse_decode_kernel<THREADS, PAGE_KPT, TOK_KPT, SOLVE, CERT, D, FP8>, dim3(units), dim3(THREADS),
                      a.smem, a.stream, a.g, a.q, a.k, a.v, a.block_table, a.seq_lens, a.routed_pages, a.page_scores,
                      a.P, a.K_c, a.epsilon, a.gap_threshold, a.out, a.diag, a.fallback_list, a.fallback_count,
                      a.solver_iters, a.solve, a.rad_logical, a.cert, a.unit_list, a.unit_count, a.routed_stride,
                      a.tl_summaries, a.P_super, a.k_scale, a.v_scale);
}

// token-score registers per thread from the number of routed tokens
template <int THREADS, int PAGE_KPT, int SOLVE, bool CERT, int D = kHeadDim, bool FP8 = false>
cudaError_t launch_tok(const SparseArgs& a)
{
    const int N = a.P * a.g.page_size;
    if (N <= 2 * THREADS) return launch_variant<THREADS, PAGE_KPT, 2, SOLVE, CERT, D, FP8>(a);
    if (N <= 4 * THREADS) return launch_variant<THREADS, PAGE_KPT, 4, SOLVE, CERT, D, FP8>(a);
    if constexpr (THREADS <= 256)
        return N <= 8 * THREADS ? launch_variant<THREADS, PAGE_KPT, 8, SOLVE, CERT, D, FP8>(a) : cudaErrorInvalidValue;
    else
        return cudaErrorInvalidValue;   // 128 pages * 16 tokens = 4 * 512: never reached
}

// page-score registers per thread from the block-table width (CERT: register variants only)
template <int THREADS, int SOLVE, bool CERT, int D = kHeadDim, bool FP8 = false>
cudaError_t launch_threads(const SparseArgs& a)
{
    if constexpr (!CERT) {
        if (!a.page_scores) return launch_tok<THREADS, 0, SOLVE, CERT, D, FP8>(a);
    }
    if (a.g.max_pages <= 8 * THREADS) return launch_tok<THREADS, 8, SOLVE, CERT, D, FP8>(a);
    if (a.g.max_pages <= 16 * THREADS) return launch_tok<THREADS, 16, SOLVE, CERT, D, FP8>(a);
    if (a.g.max_pages <= 32 * THREADS) return launch_tok<THREADS, 32, SOLVE, CERT, D, FP8>(a);
    if constexpr (!CERT)
        return launch_tok<THREADS, -1, SOLVE, CERT, D, FP8>(a);
    else
        return cudaErrorInvalidValue;   // (refused by the entry point before any launch)
}

// the 128-thread shape (P <= 64, the caller checks): routed pages given, or selected from scores held
// in registers (max_pages <= 4096) or staged in shared memory (wider tables)
template <int D = kHeadDim, bool FP8 = false>
inline cudaError_t launch_threads_128(const SparseArgs& a)
{
    if (!a.page_scores) return launch_tok<128, 0, 0, false, D, FP8>(a);
    if (a.g.max_pages <= 8 * 128) return launch_tok<128, 8, 0, false, D, FP8>(a);
    if (a.g.max_pages <= 16 * 128) return launch_tok<128, 16, 0, false, D, FP8>(a);
    if (a.g.max_pages <= 32 * 128) return launch_tok<128, 32, 0, false, D, FP8>(a);
    return launch_tok<128, -1, 0, false, D, FP8>(a);   // wider tables: selection staged in shared memory
}

}  // namespace

// one family of kernel variants per translation unit
cudaError_t launch_sparse_plain(const SparseArgs& a, int threads);   // closed-form weights
cudaError_t launch_sparse_plain_d64(const SparseArgs& a, int threads);    // the same at head dimension 64
cudaError_t launch_sparse_plain_d256(const SparseArgs& a, int threads);   // and 256
cudaError_t launch_sparse_plain_fp8(const SparseArgs& a, int threads);    // closed-form weights on an fp8 cache
cudaError_t launch_sparse_solve(const SparseArgs& a);                // iterative solves (256 threads)
cudaError_t launch_sparse_cert(const SparseArgs& a, int threads);    // routing certificate
cudaError_t launch_sparse_two_level(const SparseArgs& a, int threads);   // two-level front end

}  // namespace vsa
