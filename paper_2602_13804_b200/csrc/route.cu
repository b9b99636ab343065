// Page routing (paper Sec. 7 step 1): score one summary row per page against every query head that
// reads its KV head, then keep the P best pages per query head.
//
//   route_scan_kernel    streams the summary rows (the only part of the step whose traffic grows
//                        with the context length) and writes all page scores to scratch.
//   route_select_kernel  one block per (sequence, query head): exact top-P selection.
#include <math.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"
#include "vsa_select.cuh"

namespace vsa {

namespace {

constexpr int kScanThreads = 256;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kBlockPages = 32;   // pages whose block-table entries one warp holds in a register

// Warp w of the grid row of sequence b handles KV head (w % n_kv) and the 32-page blocks
// [slice * blocks_per_warp, (slice + 1) * blocks_per_warp), slice = w / n_kv, so the warps of a
// thread block read the summaries of all KV heads of the same pages (2 KB contiguous per page).
// A half-warp reads one 256-byte row per load instruction; the G query heads of the row's group
// share each unpacked element; 16 (row, head) partials are reduced at once.  The loads of the next
// round are issued before the current round is reduced (two register buffers), and the block-table
// entries of the block after next are fetched while the current block is processed.
template <int G>
__global__ void __launch_bounds__(kScanThreads, 2)
route_scan_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ summaries,
                  const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_lens,
                  float* __restrict__ scores, int blocks_per_warp, int32_t* zero_word, int32_t* zero_words,
                  int zero_count)
{
    constexpr int ROWS = G == 1 ? 8 : 16 / G;      // rows per half-warp per round
    constexpr int VALS = ROWS * G;                 // (row, head) partials per lane per round (8 or 16)
    constexpr int ROUND_PAGES = 2 * ROWS;          // pages per warp per round
    constexpr int ROUNDS = kBlockPages / ROUND_PAGES;   // rounds per 32-page block (even)
    static_assert(ROUNDS % 2 == 0, "the round loop is unrolled by two");

    // housekeeping for the kernels that follow in a step: clear the fallback counter and the
    // per-group tickets of the dense pass
    if (blockIdx.y == 0) {
        if (zero_word && blockIdx.x == 0 && threadIdx.x == 0) *zero_word = 0;
        if (zero_words)
            for (int i = blockIdx.x * kScanThreads + threadIdx.x; i < zero_count; i += gridDim.x * kScanThreads)
                zero_words[i] = 0;
    }

    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31, c = lane & 15, gi = lane >> 4;
    const int w = blockIdx.x * kScanWarps + (threadIdx.x >> 5);
    const int g = w % geo.n_kv_heads;
    const int slice = w / geo.n_kv_heads;
    const int T = seq_lens[b];
    if (T <= 0 || T > geo.max_pages * kPageSize) return;
    const int nb = (T + kPageSize - 1) / kPageSize;
    const int first_block = slice * blocks_per_warp;
    if (first_block * kBlockPages >= nb) return;
    const int n_blocks = min(blocks_per_warp, (nb - first_block * kBlockPages + kBlockPages - 1) / kBlockPages);

    const int32_t* bt = block_table + (long long)b * geo.max_pages;
    auto load_bt = [&](int blk) -> int {   // physical page of this lane's page in block `blk`, -1 if none
        const int l = blk * kBlockPages + lane;
        if (blk >= first_block + n_blocks || l >= nb) return -1;
        const int p = bt[l];
        return (p >= 0 && p < geo.pool_pages) ? p : -1;
    };
    int phys_even = load_bt(first_block);       // blocks first_block + 0, 2, 4, ...
    int phys_odd = load_bt(first_block + 1);    // blocks first_block + 1, 3, 5, ...

    float qf[G][8];
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
        const uint4 v = *reinterpret_cast<const uint4*>(
            q + ((long long)b * geo.n_q_heads + g * G + hh) * kHeadDim + c * 8);
        unpack8(v, qf[hh]);
    }
    const uint16_t* srow = summaries + (long long)g * kHeadDim + c * 8;
    const long long page_elems = (long long)geo.n_kv_heads * kHeadDim;
    // after the reduction this lane owns (row own_r, head own_h) of its half-warp's ROWS rows
    const int own_r = VALS == 16 ? c / G : (c & 7) / G, own_h = c % G;
    float* out_lane = scores + ((long long)b * geo.n_q_heads + g * G + own_h) * geo.max_pages + gi * ROWS + own_r;

    // rows of round `rnd` (0 .. ROUNDS-1) of a block whose block-table entries sit in `phys_reg`;
    // rows without a valid page read row 0 of the pool instead (their result is never stored)
    auto issue = [&](uint4 (&buf)[ROWS], int phys_reg, int rnd) {
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const int phys = __shfl_sync(kFullMask, phys_reg, rnd * ROUND_PAGES + gi * ROWS + r);
            buf[r] = ld_nc_16B(srow + max(phys, 0) * page_elems);
        }
    };
    auto reduce_store = [&](const uint4 (&buf)[ROWS], int phys_reg, int blk, int rnd) {
        float vals[16];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            float kf[8];
            unpack8(buf[r], kf);
#pragma unroll
            for (int hh = 0; hh < G; ++hh) vals[r * G + hh] = chunk_partial(qf[hh], kf);
        }
        if (VALS < 16) {
#pragma unroll
            for (int i = VALS; i < 16; ++i) vals[i] = 0.0f;
        }
        const float s = reduce_scatter16(vals, c);
        const int pl = rnd * ROUND_PAGES + gi * ROWS + own_r;
        const int phys = __shfl_sync(kFullMask, phys_reg, pl);
        const int l = blk * kBlockPages + pl;
        if (l < nb && (VALS == 16 || c < 8)) out_lane[blk * kBlockPages + rnd * ROUND_PAGES] = phys >= 0 ? s : -INFINITY;
    };

    uint4 buf_a[ROWS], buf_b[ROWS];
    issue(buf_a, phys_even, 0);
    for (int k = 0; k < n_blocks; ++k) {
        const int blk = first_block + k;
        const bool even = (k & 1) == 0;
        const int phys_cur = even ? phys_even : phys_odd;
        const int phys_nxt = even ? phys_odd : phys_even;
#pragma unroll
        for (int rnd = 0; rnd < ROUNDS; rnd += 2) {
            issue(buf_b, phys_cur, rnd + 1);
            reduce_store(buf_a, phys_cur, blk, rnd);
            if (rnd + 2 < ROUNDS)
                issue(buf_a, phys_cur, rnd + 2);
            else if (k + 1 < n_blocks)
                issue(buf_a, phys_nxt, 0);
            reduce_store(buf_b, phys_cur, blk, rnd + 1);
        }
        // this block's register is free: fetch the entries of the block after next into it
        const int refill = load_bt(blk + 2);
        if (even)
            phys_even = refill;
        else
            phys_odd = refill;
    }
}

// Exact top-P of one unit's page scores, order (score descending, page ascending).
// KPT > 0: every thread keeps its KPT scores in registers (max_pages <= KPT * blockDim.x);
// KPT == 0: scores staged in shared memory, any size.
template <int KPT>
__global__ void route_select_kernel(Geometry geo, const float* __restrict__ scores,
                                    const int32_t* __restrict__ seq_lens, int P,
                                    int32_t* __restrict__ routed_pages, float* __restrict__ routed_scores)
{
    extern __shared__ uint32_t smem[];
    const PageSelectSmem s = carve_page_select(smem, geo.max_pages, P);
    const int h = blockIdx.x, b = blockIdx.y;
    const long long unit = (long long)b * geo.n_q_heads + h;
    const int T = seq_lens[b];
    const bool ok = T > 0 && T <= geo.max_pages * kPageSize;
    const int n = ok ? (T + kPageSize - 1) / kPageSize : 0;
    int K;
    if constexpr (KPT > 0)
        K = select_top_pages_reg<KPT>(scores + unit * geo.max_pages, n, P, s);
    else
        K = select_top_pages(scores + unit * geo.max_pages, n, P, s);
    for (int t = threadIdx.x; t < P; t += blockDim.x) {
        routed_pages[unit * P + t] = t < K ? s.win_idx[t] : -1;
        if (routed_scores) routed_scores[unit * P + t] = t < K ? key_to_float(s.win_key[t]) : -INFINITY;
    }
}

size_t select_smem_bytes(const Geometry& g, int P) { return (size_t)select_pages_words(g.max_pages, P) * 4; }

int scan_blocks_per_warp(const Geometry& g)
{
    // 32-page blocks per warp: about one resident wave of warps (2 thread blocks of 8 warps per SM
    // on 148 SMs) when the problem is large enough, never more than 16 blocks per warp
    const long long blocks = (long long)g.batch * g.n_kv_heads * ((g.max_pages + kBlockPages - 1) / kBlockPages);
    long long k = (blocks + 2367) / 2368;
    if (k < 1) k = 1;
    if (k > 16) k = 16;
    return (int)k;
}

}  // namespace

size_t route_workspace_bytes(const Geometry& g)
{
    return (size_t)g.batch * g.n_q_heads * g.max_pages * sizeof(float);
}

cudaError_t launch_route_scan(const Geometry& g, const void* q, const void* summaries, const int32_t* block_table,
                              const int32_t* seq_lens, void* ws, int32_t* zero_word, int32_t* zero_words,
                              int zero_count, cudaStream_t stream)
{
    float* scores = (float*)ws;
    const int bpw = scan_blocks_per_warp(g);
    const int slices = ((g.max_pages + kBlockPages - 1) / kBlockPages + bpw - 1) / bpw;
    const int warps = slices * g.n_kv_heads;
    dim3 grid((unsigned)((warps + kScanWarps - 1) / kScanWarps), (unsigned)g.batch);
    const uint16_t* qq = (const uint16_t*)q;
    const uint16_t* ss = (const uint16_t*)summaries;
#define VSA_SCAN_LAUNCH(GG)                                                                                      \
    route_scan_kernel<GG><<<grid, kScanThreads, 0, stream>>>(g, qq, ss, block_table, seq_lens, scores, bpw,      \
                                                             zero_word, zero_words, zero_count)
    switch (g.group) {
        case 1: VSA_SCAN_LAUNCH(1); break;
        case 2: VSA_SCAN_LAUNCH(2); break;
        case 4: VSA_SCAN_LAUNCH(4); break;
        case 8: VSA_SCAN_LAUNCH(8); break;
        default: return cudaErrorInvalidValue;
    }
#undef VSA_SCAN_LAUNCH
    return cudaGetLastError();
}

cudaError_t launch_route_select(const Geometry& g, const void* ws, const int32_t* seq_lens, int P,
                                int32_t* routed_pages, float* routed_scores, cudaStream_t stream)
{
    const size_t smem = select_smem_bytes(g, P);
    const dim3 grid((unsigned)g.n_q_heads, (unsigned)g.batch);
#define VSA_SELECT_LAUNCH(KPT, THREADS)                                                                          \
    {                                                                                                            \
        if (smem > 48 * 1024) {                                                                                  \
            cudaError_t e = cudaFuncSetAttribute(route_select_kernel<KPT>,                                       \
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);        \
            if (e != cudaSuccess) return e;                                                                      \
        }                                                                                                        \
        route_select_kernel<KPT><<<grid, THREADS, smem, stream>>>(g, (const float*)ws, seq_lens, P, routed_pages, \
                                                                 routed_scores);                                \
    }
    if (g.max_pages <= 2048) VSA_SELECT_LAUNCH(8, 256)
    else if (g.max_pages <= 4096) VSA_SELECT_LAUNCH(16, 256)
    else if (g.max_pages <= 8192) VSA_SELECT_LAUNCH(32, 256)
    else VSA_SELECT_LAUNCH(0, 512)
#undef VSA_SELECT_LAUNCH
    return cudaGetLastError();
}

}  // namespace vsa
