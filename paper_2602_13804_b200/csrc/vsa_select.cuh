// Top-P page selection of one (sequence, query head) unit from its page scores, shared by the
// stand-alone routing kernel and by the fused step kernel (paper Sec. 7 step 1, "select P pages").
#pragma once

#include <math.h>

#include "vsa_device.cuh"

namespace vsa {

// Shared-memory needs of the page selection for n_max scores and P pages, in 4-byte words.
__host__ __device__ constexpr int select_pages_words(int n_max, int P)
{
    return n_max /*keys*/ + (n_max + 3) / 4 /*take*/ + 256 + 16 + 72 + kTopkList /*scratch*/ + 5 * P /*lists*/;
}

struct PageSelectSmem {
    uint32_t* keys;      // [n_max]  (register variant: only the slow path stores keys here)
    uint8_t* take;       // [n_max]
    TopkScratch ts;
    uint32_t* tmp_key;   // [P] winners, unordered
    int32_t* tmp_idx;    // [P]
    uint32_t* win_key;   // [P] winners, best first
    int32_t* win_idx;    // [P]
    int32_t* asc_idx;    // [P] winners by ascending page index
};

__device__ __forceinline__ PageSelectSmem carve_page_select(uint32_t* base, int n_max, int P)
{
    PageSelectSmem s;
    s.keys = base;
    s.take = (uint8_t*)(s.keys + n_max);
    s.ts.hist = s.keys + n_max + (n_max + 3) / 4;
    s.ts.misc = s.ts.hist + 256;
    s.ts.wred = s.ts.misc + 16;
    s.ts.list = (int32_t*)(s.ts.wred + 72);
    s.tmp_key = (uint32_t*)(s.ts.list + kTopkList);
    s.tmp_idx = (int32_t*)(s.tmp_key + P);
    s.win_key = (uint32_t*)(s.tmp_idx + P);
    s.win_idx = (int32_t*)(s.win_key + P);
    s.asc_idx = s.win_idx + P;
    return s;
}

// Orders the K unordered winners in tmp_key/tmp_idx: win_* best first (key descending, index
// ascending), asc_idx by ascending index.  Ends with a block barrier.
__device__ __forceinline__ void order_winners(int K, const PageSelectSmem& s)
{
    for (int t = threadIdx.x; t < K; t += blockDim.x) {
        const uint32_t key = s.tmp_key[t];
        const int idx = s.tmp_idx[t];
        int rank = 0, rank_asc = 0;
#pragma unroll 8
        for (int j = 0; j < K; ++j) {
            const uint32_t kj = s.tmp_key[j];
            const int ij = s.tmp_idx[j];
            rank += (int)((kj > key) | ((kj == key) & (ij < idx)));
            rank_asc += ij < idx;
        }
        s.win_key[rank] = key;
        s.win_idx[rank] = idx;
        s.asc_idx[rank_asc] = idx;
    }
    __syncthreads();
}

// Exact top-min(P, n) of sc[0..n) under (score descending, page ascending), keys staged in shared
// memory (any n up to the carve size).  Returns K; winners in s.win_* / s.asc_idx.
// sparse_row: scores of -inf mark pages that were never scored (two-level routing); they are treated as
// absent, and the caller guarantees P <= the number of scored pages.
__device__ __forceinline__ int select_top_pages(const float* __restrict__ sc, int n, int P, const PageSelectSmem& s,
                                                bool sparse_row = false)
{
    const int K = min(P, n);
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const float v = __ldcg(sc + i);
        s.keys[i] = (sparse_row && v == -INFINITY) ? 0u : float_to_key(v);
        s.take[i] = 0;
    }
    if (threadIdx.x == 0) s.ts.misc[8] = 0u;
    __syncthreads();
    if (n > P) {
        block_topk_mark(s.keys, n, K, s.take, s.ts);
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            if (s.take[i]) {
                const int slot = (int)atomicAdd(&s.ts.misc[8], 1u);
                s.tmp_key[slot] = s.keys[i];
                s.tmp_idx[slot] = i;
            }
        }
    } else {
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            s.tmp_key[i] = s.keys[i];
            s.tmp_idx[i] = i;
        }
    }
    __syncthreads();
    order_winners(K, s);
    return K;
}

// The same with each thread holding its KPT scores in registers (n <= KPT * blockDim.x):
// key[j] is the key of score tid + j * blockDim.x, 0 for indices at or beyond n.
template <int KPT>
__device__ __forceinline__ int select_top_pages_keys(const uint32_t (&key)[KPT], int n, int P,
                                                     const PageSelectSmem& s)
{
    const int K = min(P, n);
    const int tid = threadIdx.x, stride = blockDim.x;
    if (tid == 0) s.ts.misc[8] = 0u;
    uint32_t mask = 0u;
    if (n > P) {
        // Filter first: take each thread's best score; in every warp find the r-th largest of these
        // (r = ceil(K / warps)); the smallest such value over the warps, theta, has at least K scores
        // at or above it, so the top K are among the scores >= theta - typically only a few more than
        // K of them - which are then ranked exactly against each other.
        const int lane = tid & 31, warp = tid >> 5, nwarps = stride >> 5;
        // only warps whose 32 threads all own a score take part (short sequences fill fewer warps)
        const int nw_full = min(nwarps, n >> 5);
        const int r = nw_full > 0 ? (K + nw_full - 1) / nw_full : 33;
        uint32_t tmax = 0u;
#pragma unroll
        for (int j = 0; j < KPT; ++j) tmax = max(tmax, key[j]);
        uint32_t v = tmax, thr = 0u;
        for (int i = 0; i < r && r <= 32; ++i) {
            thr = __reduce_max_sync(kFullMask, v);
            const unsigned holders = __ballot_sync(kFullMask, v == thr);
            if (lane == __ffs(holders) - 1) v = 0u;   // remove one holder of the maximum
        }
        if (lane == 0) s.ts.wred[warp] = thr;
        if (tid == 0) s.ts.misc[4] = 0u;
        __syncthreads();
        // (a warp with fewer than r present scores publishes 0 and does not count: with a sparse row of
        // scores only the warps that vouch for r scores each may set the threshold)
        uint32_t theta = 0xffffffffu;
        int vouching = 0;
        for (int w = 0; w < nw_full; ++w) {
            const uint32_t tw = s.ts.wred[w];
            if (tw != 0u) {
                theta = min(theta, tw);
                ++vouching;
            }
        }
        if (r > 32 || vouching * r < K) theta = 0u;   // too few scores to filter: every score is a candidate
        {
            uint32_t keep = 0u;
#pragma unroll
            for (int j = 0; j < KPT; ++j)
                if (key[j] != 0u && key[j] >= theta) keep |= 1u << j;
            int slot = warp_append_slots(__popc(keep), &s.ts.misc[4]);
#pragma unroll
            for (int j = 0; j < KPT; ++j) {
                if ((keep >> j) & 1u) {
                    if (slot < kTopkList) {
                        s.ts.list[slot] = tid + j * stride;
                        s.ts.hist[slot] = key[j];
                    }
                    ++slot;
                }
            }
        }
        __syncthreads();
        const int m = (int)s.ts.misc[4];
        if (m <= kTopkList) {
            for (int t = tid; t < m; t += stride) {
                const int idx = s.ts.list[t];
                const uint32_t kt = s.ts.hist[t];
                int rank = 0;
#pragma unroll 8
                for (int u = 0; u < m; ++u) {
                    const uint32_t ku = s.ts.hist[u];
                    const int iu = s.ts.list[u];
                    rank += (int)((ku > kt) | ((ku == kt) & (iu < idx)));
                }
                if (rank < K) {   // ranks are distinct: the K winners land best first
                    s.win_key[rank] = kt;
                    s.win_idx[rank] = idx;
                }
            }
            __syncthreads();
            for (int t = tid; t < K; t += stride) {
                const int idx = s.win_idx[t];
                int rank_asc = 0;
#pragma unroll 8
                for (int u = 0; u < K; ++u) rank_asc += s.win_idx[u] < idx;
                s.asc_idx[rank_asc] = idx;
            }
            __syncthreads();
            return K;
        }
        // crowded (many equal scores): the general selection decides
        __syncthreads();
        mask = block_topk_reg<KPT>(key, n, K, s.ts, s.keys, s.take).mask;   // barriers inside order misc[8]
    } else {
#pragma unroll
        for (int j = 0; j < KPT; ++j)
            if (key[j] != 0u) mask |= 1u << j;
        __syncthreads();
    }
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        if ((mask >> j) & 1u) {
            const int slot = (int)atomicAdd(&s.ts.misc[8], 1u);
            s.tmp_key[slot] = key[j];
            s.tmp_idx[slot] = tid + j * stride;
        }
    }
    __syncthreads();
    order_winners(K, s);
    return K;
}

// The register variant fed from the scores in global memory.
template <int KPT>
__device__ __forceinline__ int select_top_pages_reg(const float* __restrict__ sc, int n, int P,
                                                    const PageSelectSmem& s, bool sparse_row = false)
{
    uint32_t key[KPT];
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        const int i = threadIdx.x + j * blockDim.x;
        const float v = i < n ? __ldcg(sc + i) : 0.0f;
        key[j] = (i < n && !(sparse_row && v == -INFINITY)) ? float_to_key(v) : 0u;
    }
    return select_top_pages_keys<KPT>(key, n, P, s);
}

}  // namespace vsa
