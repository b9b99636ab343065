// Page routing (paper Sec. 7 step 1): score one summary row per page against every query head that
// reads its KV head, then keep the P best pages per query head.
//
//   route_scan_kernel    streams the summary rows (the only part of the step whose traffic grows
//                        with the context length) and writes all page scores to scratch.
//   route_select_kernel  one block per (sequence, query head): exact top-P by radix select.
#include <math.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"

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
    const int max_pages = geo.max_pages;
    uint32_t* keys = smem;                                  // [max_pages]
    uint32_t* hist = keys + max_pages;                      // [256]
    uint32_t* scratch = hist + 256;                         // [8]
    uint32_t* warp_counts = scratch + 8;                    // [40]
    uint32_t* win_key = warp_counts + 40;                   // [P]
    int32_t* win_idx = (int32_t*)(win_key + P);             // [P]
    uint8_t* take = (uint8_t*)(win_idx + P);                // [max_pages]

    const int h = blockIdx.x, b = blockIdx.y;
    const long long unit = (long long)b * geo.n_q_heads + h;
    const int T = seq_lens[b];
    const bool ok = T > 0 && T <= max_pages * kPageSize;
    const int n = ok ? (T + kPageSize - 1) / kPageSize : 0;
    const int K = min(P, n);
    const float* sc = scores + unit * max_pages;

    for (int i = threadIdx.x; i < n; i += blockDim.x) keys[i] = float_to_key(sc[i]);
    if (threadIdx.x == 0) scratch[4] = 0;   // winner counter
    __syncthreads();

    if (n > P) {
        const SelectResult r = block_select_kth(keys, n, K, hist, scratch);
        const int need = K - r.n_greater;
        const bool straddle = r.n_equal > need;
        if (straddle) {
            for (int i = threadIdx.x; i < n; i += blockDim.x) take[i] = 0;
            __syncthreads();
            block_mark_first_equal(keys, n, r.kth, need, take, warp_counts);
            __syncthreads();
        }
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const uint32_t key = keys[i];
            if (key > r.kth || (key == r.kth && (!straddle || take[i]))) {
                const int slot = (int)atomicAdd(&scratch[4], 1u);
                win_key[slot] = key;
                win_idx[slot] = i;
            }
        }
    } else {
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            win_key[i] = keys[i];
            win_idx[i] = i;
        }
    }
    __syncthreads();

    // order the K winners (all (key, index) pairs are distinct) and write them best first
    for (int t = threadIdx.x; t < P; t += blockDim.x) {
        if (t < K) {
            const uint32_t key = win_key[t];
            const int idx = win_idx[t];
            int rank = 0;
            for (int j = 0; j < K; ++j) {
                const uint32_t kj = win_key[j];
                rank += (kj > key) || (kj == key && win_idx[j] < idx);
            }
            routed_pages[unit * P + rank] = idx;
            if (routed_scores) routed_scores[unit * P + rank] = key_to_float(key);
        } else {
            routed_pages[unit * P + t] = -1;
            if (routed_scores) routed_scores[unit * P + t] = -INFINITY;
        }
    }
}

size_t select_smem_bytes(const Geometry& g, int P)
{
    return (size_t)g.max_pages * 4 + 256 * 4 + 8 * 4 + 40 * 4 + (size_t)P * 8 + (size_t)g.max_pages + 16;
}

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

cudaError_t launch_route(const Geometry& g, const void* q, const void* summaries, const int32_t* block_table,
                         const int32_t* seq_lens, int P, int32_t* routed_pages, float* routed_scores,
                         void* ws, int32_t* zero_word, cudaStream_t stream, cudaEvent_t after_scan)
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
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (after_scan && (e = cudaEventRecord(after_scan, stream)) != cudaSuccess) return e;

    const size_t smem = select_smem_bytes(g, P);
    if (smem > 48 * 1024) {
        e = cudaFuncSetAttribute(route_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const int threads = g.max_pages <= 1024 ? 256 : 1024;
    route_select_kernel<<<dim3((unsigned)g.n_q_heads, (unsigned)g.batch), threads, smem, stream>>>(
        g, scores, seq_lens, P, routed_pages, routed_scores);
    return cudaGetLastError();
}

}  // namespace vsa
