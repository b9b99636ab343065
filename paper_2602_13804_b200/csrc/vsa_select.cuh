// Top-P page selection of one (sequence, query head) unit from its page scores, shared by the
// stand-alone routing kernel and by the fused step kernel (paper Sec. 7 step 1, "select P pages").
#pragma once

#include <math.h>

#include "vsa_device.cuh"

namespace vsa {

// Shared-memory needs of select_top_pages for n_max scores and P pages, in 4-byte words.
__host__ __device__ constexpr int select_pages_words(int n_max, int P)
{
    return n_max /*keys*/ + (n_max + 3) / 4 /*take*/ + 256 + 16 + 72 + kTopkList /*scratch*/ + 4 * P /*tmp + winners*/;
}

struct PageSelectSmem {
    uint32_t* keys;      // [n_max]
    uint8_t* take;       // [n_max]
    TopkScratch ts;
    uint32_t* tmp_key;   // [P] winners, unordered
    int32_t* tmp_idx;    // [P]
    uint32_t* win_key;   // [P] winners, best first
    int32_t* win_idx;    // [P]
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
    return s;
}

// Exact top-min(P, n) of sc[0..n) under (score descending, page ascending).  On return (after a
// block barrier) s.win_idx[0..K) / s.win_key[0..K) hold the winners best first; returns K.
// All threads of the block call it.
__device__ __forceinline__ int select_top_pages(const float* __restrict__ sc, int n, int P, const PageSelectSmem& s)
{
    const int K = min(P, n);
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        s.keys[i] = float_to_key(__ldcg(sc + i));
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
    for (int t = threadIdx.x; t < K; t += blockDim.x) {
        const uint32_t key = s.tmp_key[t];
        const int idx = s.tmp_idx[t];
        int rank = 0;
        for (int j = 0; j < K; ++j) {
            const uint32_t kj = s.tmp_key[j];
            rank += (kj > key) || (kj == key && s.tmp_idx[j] < idx);
        }
        s.win_key[rank] = key;
        s.win_idx[rank] = idx;
    }
    __syncthreads();
    return K;
}

}  // namespace vsa
