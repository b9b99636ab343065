// Page routing (paper Sec. 7 step 1): score one summary row per page against every query head that
// reads its KV head, then keep the P best pages per query head.
//
//   route_scan_kernel    streams the summary rows (the only part of the step whose traffic grows
//                        with the context length) and writes all page scores to scratch.
//   route_select_kernel  one block per (sequence, query head): exact top-P by radix select.
#include <math.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"
#include "vsa_select.cuh"

namespace vsa {

namespace {

constexpr int kScanThreads = 256;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kBlockPages = 32;   // pages whose block-table entries one warp holds in registers

// Warp w of the grid row of sequence b handles KV head (w % n_kv) and page blocks
// [slice * blocks_per_warp, (slice + 1) * blocks_per_warp) of 32 pages, slice = w / n_kv, so the
// 8 warps of a block read the summaries of all KV heads of the same pages (2 KB contiguous
// per page).  A half-warp reads one 256-byte row per load; the G query heads of the row's
// group share each unpacked element; 16 (row, head) partials are reduced at once.
template <int G>
__global__ void __launch_bounds__(kScanThreads)
route_scan_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ summaries,
                  const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_lens,
                  float* __restrict__ scores, int blocks_per_warp, int32_t* zero_word)
{
    constexpr int ROWS = 16 / G;                 // rows per half-warp per round
    constexpr int ROUND_PAGES = 2 * ROWS;        // pages per warp per round
    constexpr int ROUNDS = kBlockPages / ROUND_PAGES;
    constexpr int U = (8 / ROWS) < 1 ? 1 : ((8 / ROWS) > ROUNDS ? ROUNDS : (8 / ROWS));   // rounds in flight

    if (zero_word && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) *zero_word = 0;

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

    float qf[G][8];
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
        const uint4 v = *reinterpret_cast<const uint4*>(
            q + ((long long)b * geo.n_q_heads + g * G + hh) * kHeadDim + c * 8);
        unpack8(v, qf[hh]);
    }
    const int32_t* bt = block_table + (long long)b * geo.max_pages;
    const uint16_t* srow = summaries + (long long)g * kHeadDim + c * 8;
    const long long page_elems = (long long)geo.n_kv_heads * kHeadDim;
    float* out_base = scores + ((long long)b * geo.n_q_heads + g * G) * geo.max_pages;

    for (int blk = first_block; blk < first_block + blocks_per_warp; ++blk) {
        const int l0 = blk * kBlockPages;
        if (l0 >= nb) break;
        int phys_reg = -1;
        if (l0 + lane < nb) {
            const int p = bt[l0 + lane];
            phys_reg = (p >= 0 && p < geo.pool_pages) ? p : -1;
        }
#pragma unroll 1
        for (int round = 0; round < ROUNDS; round += U) {
            if (l0 + round * ROUND_PAGES >= nb) break;
            uint4 data[U][ROWS];
#pragma unroll
            for (int u = 0; u < U; ++u) {
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    const int pl = (round + u) * ROUND_PAGES + gi * ROWS + r;
                    const int phys = __shfl_sync(kFullMask, phys_reg, pl);
                    data[u][r] = make_uint4(0u, 0u, 0u, 0u);
                    if (phys >= 0) data[u][r] = ld_nc_16B(srow + phys * page_elems);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float vals[16];
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    float kf[8];
                    unpack8(data[u][r], kf);
#pragma unroll
                    for (int hh = 0; hh < G; ++hh) vals[r * G + hh] = chunk_partial(qf[hh], kf);
                }
                const float s = reduce_scatter16(vals, c);
                // this lane now owns (row c / G, head c % G) of its half-warp's ROWS rows
                const int pl = (round + u) * ROUND_PAGES + gi * ROWS + c / G;
                const int phys = __shfl_sync(kFullMask, phys_reg, pl);
                const int l = l0 + pl;
                if (l < nb) out_base[(long long)(c % G) * geo.max_pages + l] = phys >= 0 ? s : -INFINITY;
            }
        }
    }
}

// Exact top-P of one unit's page scores, order (score descending, page ascending).
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
    const int K = select_top_pages(scores + unit * geo.max_pages, n, P, s);
    for (int t = threadIdx.x; t < P; t += blockDim.x) {
        routed_pages[unit * P + t] = t < K ? s.win_idx[t] : -1;
        if (routed_scores) routed_scores[unit * P + t] = t < K ? key_to_float(s.win_key[t]) : -INFINITY;
    }
}

size_t select_smem_bytes(const Geometry& g, int P) { return (size_t)select_pages_words(g.max_pages, P) * 4; }

int scan_blocks_per_warp(const Geometry& g)
{
    // 32-page blocks per warp: keep at least ~4k warps in the grid when the problem is large
    const long long blocks = (long long)g.batch * g.n_kv_heads * ((g.max_pages + kBlockPages - 1) / kBlockPages);
    long long k = blocks / 4096;
    if (k < 1) k = 1;
    if (k > 8) k = 8;
    return (int)k;
}

}  // namespace

size_t route_workspace_bytes(const Geometry& g)
{
    return (size_t)g.batch * g.n_q_heads * g.max_pages * sizeof(float);
}

cudaError_t launch_route_scan(const Geometry& g, const void* q, const void* summaries, const int32_t* block_table,
                              const int32_t* seq_lens, void* ws, int32_t* zero_word, cudaStream_t stream)
{
    float* scores = (float*)ws;
    const int bpw = scan_blocks_per_warp(g);
    const int slices = ((g.max_pages + kBlockPages - 1) / kBlockPages + bpw - 1) / bpw;
    const int warps = slices * g.n_kv_heads;
    dim3 grid((unsigned)((warps + kScanWarps - 1) / kScanWarps), (unsigned)g.batch);
    const uint16_t* qq = (const uint16_t*)q;
    const uint16_t* ss = (const uint16_t*)summaries;
    switch (g.group) {
        case 1: route_scan_kernel<1><<<grid, kScanThreads, 0, stream>>>(g, qq, ss, block_table, seq_lens, scores, bpw, zero_word); break;
        case 2: route_scan_kernel<2><<<grid, kScanThreads, 0, stream>>>(g, qq, ss, block_table, seq_lens, scores, bpw, zero_word); break;
        case 4: route_scan_kernel<4><<<grid, kScanThreads, 0, stream>>>(g, qq, ss, block_table, seq_lens, scores, bpw, zero_word); break;
        case 8: route_scan_kernel<8><<<grid, kScanThreads, 0, stream>>>(g, qq, ss, block_table, seq_lens, scores, bpw, zero_word); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_route_select(const Geometry& g, const void* ws, const int32_t* seq_lens, int P,
                                int32_t* routed_pages, float* routed_scores, cudaStream_t stream)
{
    const size_t smem = select_smem_bytes(g, P);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(route_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const int threads = g.max_pages <= 4096 ? 256 : 512;
    route_select_kernel<<<dim3((unsigned)g.n_q_heads, (unsigned)g.batch), threads, smem, stream>>>(
        g, (const float*)ws, seq_lens, P, routed_pages, routed_scores);
    return cudaGetLastError();
}

}  // namespace vsa
