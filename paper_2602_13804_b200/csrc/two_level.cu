// Two-level page routing: an approximate pre-filter in front of the exact page scoring (paper Sec. 7
// step 1 speaks only of "coarse page summaries"; this construction is the library's).
//
// A super-page is 16 consecutive logical pages of a sequence.  Its representative is the page summary
// with the largest squared norm among its pages (fp32, the library's fixed summation order; ties go to
// the lowest page): keys of large norm are the ones that can dominate an inner product, so the best
// page score inside a super-page is usually its representative's.  Routing then takes three short
// steps instead of one scan over every page: score the representatives (1/16 of the rows), keep the
// P_super best super-pages per query head, score the pages inside those exactly.  The page scores
// are the same numbers the full scan would produce, so whatever is routed is routed in the exact
// order; what the pre-filter can lose is a page whose super-page was not kept.
//
//   super_summaries_kernel  cache maintenance: representative (and its logical page) per super-page
//   (the page-routing scan, run on the representatives with a geometry whose pages are super-pages)
//   inner_scan_kernel       per unit: top-P_super super-pages, -inf over the unit's score row, exact scores
//                           of the pages inside the kept super-pages
#include <math.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"
#include "vsa_select.cuh"

namespace vsa {

namespace {

constexpr int kSuper = 16;   // logical pages per super-page

// One half-warp per (sequence, super-page, KV head): lane c holds columns 8c .. 8c+7 of each of the
// super-page's summary rows.
__global__ void __launch_bounds__(256)
super_summaries_kernel(Geometry geo, const uint16_t* __restrict__ summaries, const int32_t* __restrict__ block_table,
                       const int32_t* __restrict__ seq_lens, const int32_t* __restrict__ first_super, int max_supers,
                       uint16_t* __restrict__ super_summaries, int32_t* __restrict__ super_rep)
{
    const int b = blockIdx.y;
    const long long hw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 4;   // (super-page, KV head)
    const int lane = threadIdx.x & 31, c = lane & 15;
    const unsigned hmask = 0xffffu << (lane & 16);
    const int g = (int)(hw % geo.n_kv_heads);
    const long long sp = hw / geo.n_kv_heads;
    if (sp >= max_supers) return;
    const int T = seq_lens[b];
    const bool okT = geo.length_ok(T);
    const int nb = okT ? geo.pages_of(T) : 0;
    if (first_super && sp < first_super[b]) return;
    const long long o = ((long long)b * max_supers + sp) * geo.n_kv_heads + g;
    int best = -1;
    float best_n = 0.0f;
    uint4 best_row = make_uint4(0u, 0u, 0u, 0u);
    for (int l = (int)sp * kSuper; l < ((int)sp + 1) * kSuper && l < nb; ++l) {
        const long long p = block_table[(long long)b * geo.max_pages + l];
        if (p < 0 || p >= geo.pool_pages) continue;   // an entry outside the pool is no candidate
        const uint4 row = ld_nc_16B(summaries + (p * geo.n_kv_heads + g) * kHeadDim + c * 8);
        float f[8];
        unpack8(row, f);
        float n2 = chunk_partial(f, f);
#pragma unroll
        for (int off = 8; off; off >>= 1) n2 = n2 + __shfl_xor_sync(hmask, n2, off);
        if (best < 0 || n2 > best_n) {
            best = l;
            best_n = n2;
            best_row = row;
        }
    }
    *reinterpret_cast<uint4*>(super_summaries + o * kHeadDim + c * 8) = best_row;
    if (super_rep && c == 0) super_rep[o] = best;
}

// One block (256 or 512 threads) per (sequence, query head): exact top-P_super of the unit's representative scores (score
// descending, super-page ascending); the unit's score row [0, n_b) is set to -inf; then every page of the
// kept super-pages gets its exact score (one super-page = 16 summary rows = one 16-value reduction per
// half-warp, lane c ending with the score of page 16 s + c).  page_budget[unit] = pages scored.
__global__ void __launch_bounds__(512)
inner_scan_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ summaries,
                  const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_lens,
                  const float* __restrict__ super_scores, int max_supers, int P_super,
                  int32_t* __restrict__ super_routed_out, float* __restrict__ scores,
                  int32_t* __restrict__ page_budget)
{
    extern __shared__ uint32_t inner_smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, c = lane & 15, gi = lane >> 4;
    const unsigned hmask = 0xffffu << (lane & 16);
    const long long unit = blockIdx.x;
    const int b = (int)(unit / geo.n_q_heads), h = (int)(unit % geo.n_q_heads), g = h / geo.group;
    const int T = ld_ca_s32(seq_lens + b);
    const uint4 qraw = ld_nc_16B(q + unit * kHeadDim + c * 8);
    pdl_wait();
    pdl_launch_dependents();
    if (!geo.length_ok(T)) {
        if (super_routed_out)
            for (int t = tid; t < P_super; t += blockDim.x) super_routed_out[unit * P_super + t] = -1;
        return;
    }
    const int nb = geo.pages_of(T), ns = (nb + kSuper - 1) / kSuper;
    const PageSelectSmem ps = carve_page_select(inner_smem, max_supers, P_super);
    const int K = select_top_pages_reg<8>(super_scores + unit * max_supers, ns, P_super, ps);   // ends with a barrier
    if (super_routed_out)
        for (int t = tid; t < P_super; t += blockDim.x) super_routed_out[unit * P_super + t] = t < K ? ps.win_idx[t] : -1;
    int* scored = (int*)ps.ts.misc;   // pages that get a score (selection scratch, free after its last barrier)
    if (tid == 0) *scored = 0;
    float* row = scores + unit * geo.max_pages;
    for (int i = tid; i < nb; i += blockDim.x) row[i] = -INFINITY;
    __syncthreads();
    float qf[8];
    unpack8(qraw, qf);
    const int32_t* bt = block_table + (long long)b * geo.max_pages;
    for (int j = warp * 2 + gi; j < K; j += (int)(blockDim.x >> 4)) {
        const int sp = ps.win_idx[j];
        const int l = sp * kSuper + c;
        long long phys = -1;
        if (l < nb) {
            phys = bt[l];
            if (phys < 0 || phys >= geo.pool_pages) phys = -1;
        }
        uint4 rows[kSuper];
#pragma unroll
        for (int r = 0; r < kSuper; ++r) {
            const long long pr = __shfl_sync(hmask, phys, (lane & 16) | r);
            rows[r] = pr >= 0 ? ld_nc_16B(summaries + (pr * geo.n_kv_heads + g) * kHeadDim + c * 8)
                              : make_uint4(0u, 0u, 0u, 0u);
        }
        float vals[16];
#pragma unroll
        for (int r = 0; r < kSuper; ++r) {
            float kf[8];
            unpack8(rows[r], kf);
            vals[r] = chunk_partial(qf, kf);
        }
        const float s = reduce_scatter16(vals, c, hmask);
        if (l < nb && phys >= 0) row[l] = s;
        const int n_ok = __popc(__ballot_sync(hmask, l < nb && phys >= 0));
        if (c == 0) atomicAdd(scored, n_ok);
    }
    __syncthreads();
    // no more than the scored pages may be routed (every other entry of the row holds -inf)
    if (tid == 0) page_budget[unit] = *scored;
}

}  // namespace

int two_level_max_supers(const Geometry& g) { return (g.max_pages + kSuper - 1) / kSuper; }

// geometry of the representative scan: one "page" per super-page, representatives in logical order
Geometry two_level_super_geometry(const Geometry& g)
{
    Geometry s = g;
    s.max_pages = two_level_max_supers(g);
    s.pool_pages = (long long)g.batch * s.max_pages;
    s.super_pages = kSuper;
    return s;
}

cudaError_t launch_build_super_summaries(const Geometry& g, const void* summaries, const int32_t* block_table,
                                         const int32_t* seq_lens, const int32_t* first_super, void* super_summaries,
                                         int32_t* super_rep, cudaStream_t stream)
{
    const int ms = two_level_max_supers(g);
    const long long halfwarps = (long long)ms * g.n_kv_heads;
    const dim3 grid((unsigned)((halfwarps * 16 + 255) / 256), (unsigned)g.batch);
    super_summaries_kernel<<<grid, 256, 0, stream>>>(g, (const uint16_t*)summaries, block_table, seq_lens,
                                                     first_super, ms, (uint16_t*)super_summaries, super_rep);
    return cudaGetLastError();
}

cudaError_t launch_inner_scan(const Geometry& g, const void* q, const void* summaries, const int32_t* block_table,
                              const int32_t* seq_lens, const float* super_scores, int P_super,
                              int32_t* super_routed_out, float* scores, int32_t* page_budget, cudaStream_t stream)
{
    const int ms = two_level_max_supers(g);   // <= 2048: the selection keeps 8 scores per thread in registers
    const size_t smem = (size_t)select_pages_words(ms, P_super) * 4;
    // 512 threads when that lets every kept super-page have a half-warp of its own (one round of loads)
    const long long units = (long long)g.batch * g.n_q_heads;
    const unsigned threads = (P_super > 16 && units <= 2LL * device_sm_count()) ? 512u : 256u;
    return launch_pdl(inner_scan_kernel, dim3((unsigned)units), dim3(threads), smem, stream, g,
                      (const uint16_t*)q, (const uint16_t*)summaries, block_table, seq_lens, super_scores, ms, P_super,
                      super_routed_out, scores, page_budget);
}

}  // namespace vsa
