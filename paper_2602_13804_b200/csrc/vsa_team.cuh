// Exact selections run by a TEAM: a fixed set of whole warps of a thread block that synchronise on a
// named barrier of their own (the whole block is a team too).  Used by the group-shared kernel
// (sparse_shared.cuh), whose one selection per (sequence, KV head) spans all 512 threads of the block.
// The order is the library's: (key descending, index ascending), key 0 = absent.
#pragma once

#include "vsa_device.cuh"

namespace vsa {

struct Team {
    int tid;    // index of this thread inside its team
    int size;   // threads in the team (a multiple of 32)
    int bar;    // named barrier of the team (1..15; 0 is the block barrier)
    __device__ __forceinline__ void sync() const
    {
        asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(size) : "memory");
    }
};

// Exact top-K of key(0..n) for any multiplicity of equal keys: MSB-first radix select (8 bits per pass)
// for the K-th key, then every index with a larger key and the first K - n_greater indices of the equal
// keys, in index order, are passed to emit().  key(i) is evaluated several times per element (it may
// re-read memory): this is the path for crowded ties only.  Returns the key and the index of the K-th
// element.  hist: 256 words, misc: 16 words, wred: one word per warp of the team.  Needs 1 <= K <= number
// of present keys.  All threads of the team call it; ends with a team barrier.
template <class KeyFn, class EmitFn>
__device__ __forceinline__ TopkResult team_exact_topk_slow(const Team& tm, KeyFn key, int n, int K, uint32_t* hist,
                                                           uint32_t* misc, uint32_t* wred, EmitFn emit)
{
    const int tid = tm.tid, stride = tm.size, lane = tid & 31, warp = tid >> 5, nwarps = stride >> 5;
    uint32_t prefix = 0u, prefix_mask = 0u;
    int remaining = K, greater = 0;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += stride) hist[i] = 0u;
        tm.sync();
        for (int i = tid; i < n; i += stride) {
            const uint32_t k = key(i);
            if (k != 0u && (k & prefix_mask) == prefix) atomicAdd(&hist[(k >> shift) & 0xffu], 1u);
        }
        tm.sync();
        if (warp == 0) {
            // lane j owns digits 8j .. 8j+7; find the digit where the count from the top reaches `remaining`
            uint32_t c[8], mine = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                c[j] = hist[lane * 8 + j];
                mine += c[j];
            }
            uint32_t incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t o = __shfl_down_sync(kFullMask, incl, off);
                if (lane + off < 32) incl += o;
            }
            uint32_t above = incl - mine;
            if (above < (uint32_t)remaining && (uint32_t)remaining <= incl) {
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (above < (uint32_t)remaining && (uint32_t)remaining <= above + c[j]) {
                        misc[0] = (uint32_t)(lane * 8 + j);
                        misc[1] = above;
                        misc[2] = c[j];
                    }
                    above += c[j];
                }
            }
        }
        tm.sync();
        const uint32_t digit = misc[0];
        greater += (int)misc[1];
        remaining -= (int)misc[1];
        prefix |= digit << shift;
        prefix_mask |= 0xffu << shift;
        tm.sync();
    }
    const uint32_t kth = prefix;
    const int need_eq = K - greater;
    for (int i = tid; i < n; i += stride)
        if (key(i) > kth) emit(i);
    int base = 0;
    for (int start = 0; start < n; start += stride) {
        const int i = start + tid;
        const bool eq = i < n && key(i) == kth;
        const unsigned b = __ballot_sync(kFullMask, eq);
        if (lane == 0) wred[warp] = (uint32_t)__popc(b);
        tm.sync();
        int before = base, total = 0;
        for (int w = 0; w < nwarps; ++w) {
            const int cw = (int)wred[w];
            if (w < warp) before += cw;
            total += cw;
        }
        if (eq) {
            const int rank = before + __popc(b & ((1u << lane) - 1u));
            if (rank < need_eq) emit(i);
            if (rank == need_eq - 1) misc[6] = (uint32_t)i;
        }
        base += total;
        tm.sync();
        if (base >= need_eq) break;
    }
    if (tid == 0) misc[5] = kth;
    tm.sync();
    TopkResult r;
    r.kth_key = misc[5];
    r.kth_idx = (int)misc[6];
    return r;
}

// Orders the K unordered winners in tmp_key / tmp_idx: win_* best first, asc_idx by ascending index.
// Ends with a team barrier.
__device__ __forceinline__ void team_order_winners(const Team& tm, int K, const uint32_t* tmp_key,
                                                   const int32_t* tmp_idx, uint32_t* win_key, int32_t* win_idx,
                                                   int32_t* asc_idx)
{
    for (int t = tm.tid; t < K; t += tm.size) {
        const uint32_t key = tmp_key[t];
        const int idx = tmp_idx[t];
        int rank = 0, rank_asc = 0;
#pragma unroll 8
        for (int j = 0; j < K; ++j) {
            const uint32_t kj = tmp_key[j];
            const int ij = tmp_idx[j];
            rank += (int)((kj > key) | ((kj == key) & (ij < idx)));
            rank_asc += ij < idx;
        }
        win_key[rank] = key;
        win_idx[rank] = idx;
        asc_idx[rank_asc] = idx;
    }
    tm.sync();
}

// Exact top-min(P, n) of n page scores by one team.  key_at(i) returns the key of score i (it may read
// memory); kc[j] must hold key_at(tm.tid + j * tm.size) for j < KC (0 at or beyond n): scores past those
// cached ones are re-evaluated in each of the two passes.  Filter: every thread's best score;
// per warp the r-th largest of these (r = ceil(K / warps)); the smallest such value over the warps has
// at least K scores at or above it, so the winners are among the scores at or above it - usually a few
// more than K - which are ranked exactly against each other.  Crowded ties take the radix select.
// Returns K; winners in win_* (best first) and asc_idx (ascending page).  Ends with a team barrier.
template <int KC, class KeyAt>
__device__ __forceinline__ int team_top_pages(const Team& tm, KeyAt key_at, const uint32_t (&kc)[KC],
                                              int n, int P, const TopkScratch& s, uint32_t* tmp_key, int32_t* tmp_idx,
                                              uint32_t* win_key, int32_t* win_idx, int32_t* asc_idx)
{
    const int K = min(P, n);
    const int tid = tm.tid, stride = tm.size, lane = tid & 31, warp = tid >> 5, nwarps = stride >> 5;
    if (tid == 0) {
        s.misc[4] = 0u;
        s.misc[8] = 0u;
    }
    if (n > P) {
        // only warps whose 32 threads all own a score take part (short sequences fill fewer warps)
        const int nw_full = min(nwarps, n >> 5);
        const int r = nw_full > 0 ? (K + nw_full - 1) / nw_full : 33;
        uint32_t tmax = 0u;
#pragma unroll
        for (int j = 0; j < KC; ++j) tmax = max(tmax, kc[j]);
#pragma unroll 8
        for (int i = tid + KC * stride; i < n; i += stride) tmax = max(tmax, key_at(i));
        uint32_t v = tmax, thr = 0u;
        for (int i = 0; i < r && r <= 32; ++i) {
            thr = __reduce_max_sync(kFullMask, v);
            const unsigned holders = __ballot_sync(kFullMask, v == thr);
            if (lane == __ffs(holders) - 1) v = 0u;   // remove one holder of the maximum
        }
        if (lane == 0) s.wred[warp] = thr;
        tm.sync();
        uint32_t theta = 0xffffffffu;
        for (int w = 0; w < nw_full; ++w) theta = min(theta, s.wred[w]);
        if (r > 32) theta = 0u;   // too few scores to filter: every score is a candidate
        {
            uint32_t keep = 0u;
#pragma unroll
            for (int j = 0; j < KC; ++j)
                if (kc[j] != 0u && kc[j] >= theta) keep |= 1u << j;
            int slot = warp_append_slots(__popc(keep), &s.misc[4]);
#pragma unroll
            for (int j = 0; j < KC; ++j) {
                if ((keep >> j) & 1u) {
                    if (slot < kTopkList) {
                        s.list[slot] = tid + j * stride;
                        s.hist[slot] = kc[j];
                    }
                    ++slot;
                }
            }
            // scores past the cached ones, a warp-uniform number of rounds
            for (int i0 = KC * stride + warp * 32; i0 < n; i0 += stride) {
                const int i = i0 + lane;
                const uint32_t k = i < n ? key_at(i) : 0u;
                const bool kp = k != 0u && k >= theta;
                const unsigned bal = __ballot_sync(kFullMask, kp);
                if (bal) {
                    int base = 0;
                    if (lane == 0) base = (int)atomicAdd(&s.misc[4], (uint32_t)__popc(bal));
                    base = __shfl_sync(kFullMask, base, 0);
                    const int sl = base + __popc(bal & ((1u << lane) - 1u));
                    if (kp && sl < kTopkList) {
                        s.list[sl] = i;
                        s.hist[sl] = k;
                    }
                }
            }
        }
        tm.sync();
        const int m = (int)s.misc[4];
        if (m <= kTopkList) {
            for (int t = tid; t < m; t += stride) {
                const int idx = s.list[t];
                const uint32_t kt = s.hist[t];
                int rank = 0;
#pragma unroll 8
                for (int u = 0; u < m; ++u) {
                    const uint32_t ku = s.hist[u];
                    const int iu = s.list[u];
                    rank += (int)((ku > kt) | ((ku == kt) & (iu < idx)));
                }
                if (rank < K) {   // ranks are distinct: the K winners land best first
                    win_key[rank] = kt;
                    win_idx[rank] = idx;
                }
            }
            tm.sync();
            for (int t = tid; t < K; t += stride) {
                const int idx = win_idx[t];
                int rank_asc = 0;
#pragma unroll 8
                for (int u = 0; u < K; ++u) rank_asc += win_idx[u] < idx;
                asc_idx[rank_asc] = idx;
            }
            tm.sync();
            return K;
        }
        // crowded (many equal scores): the radix select decides, re-reading the scores
        tm.sync();
        team_exact_topk_slow(tm, key_at, n, K, s.hist, s.misc, s.wred, [&](int i) {
            const int slot = (int)atomicAdd(&s.misc[8], 1u);
            tmp_key[slot] = key_at(i);
            tmp_idx[slot] = i;
        });
    } else {
        for (int i = tid; i < n; i += stride) {
            tmp_key[i] = key_at(i);
            tmp_idx[i] = i;
        }
        tm.sync();
    }
    team_order_winners(tm, K, tmp_key, tmp_idx, win_key, win_idx, asc_idx);
    return K;
}

// Exact top-K of the token keys a team holds in registers: thread t owns elements t, t + size, ...,
// t + (KPT-1) * size (key 0 = absent).  Bit j of the result's mask is set iff element t + j * size is among
// the K best; kth_key / kth_idx describe the K-th element.  One pass over a 256-bin histogram that is
// LINEAR in the score over [lo, hi] (monotone: a higher score never lands in a lower bin; scores outside
// the bracket fall into the first or last bin) isolates the bin that holds the cut; bins above it are
// taken whole, the few elements of the cut bin are ranked exactly.  The caller supplies the bracket
// (lo_in, hi_in) - any bracket of the bulk of the scores - and the full range, used when the bracket is
// empty, and has zeroed s.hist[0..256) and s.misc[4] before the team's last barrier.  A crowded cut bin
// or a degenerate range spills the keys to `spill` ([n] words, `spill_take` [n] bytes) and runs the
// radix select.  Needs 1 <= K <= number of present keys.  Ends with a team barrier.
template <int KPT>
__device__ __forceinline__ TopkRegResult team_topk_reg(const Team& tm, const uint32_t (&key)[KPT], int n, int K,
                                                       const TopkScratch& s, uint32_t* spill, uint8_t* spill_take,
                                                       float lo_in, float hi_in, float lo_full, float hi_full)
{
    static_assert(KPT <= 32, "one mask bit per owned element");
    const int tid = tm.tid, lane = tid & 31, warp = tid >> 5, stride = tm.size;
    float f[KPT];
#pragma unroll
    for (int j = 0; j < KPT; ++j) f[j] = key_to_float(key[j]);
    const bool bracket = hi_in > lo_in;
    const float lo = bracket ? lo_in : lo_full, hi = bracket ? hi_in : hi_full;
    const float scale = 256.0f / (hi - lo);
    const bool fast = hi > lo && isfinite(scale) && isfinite(hi - lo);
    int cut = -1, need = K;
    int bucket[KPT];
    if (fast) {
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            bucket[j] = f[j] > -INFINITY ? (int)fminf(fmaxf((f[j] - lo) * scale, 0.0f), 255.0f) : 0;
            if (key[j] != 0u) atomicAdd(&s.hist[bucket[j]], 1u);
        }
        tm.sync();
        if (warp == 0) {
            // one warp scans the histogram and publishes the cut through the barrier that follows
            uint32_t c[8], mine = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                c[j] = s.hist[lane * 8 + j];
                mine += c[j];
            }
            uint32_t incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const uint32_t o = __shfl_down_sync(kFullMask, incl, off);
                if (lane + off < 32) incl += o;
            }
            uint32_t above = incl - mine;
            int my_cut = -1, my_above = 0, my_count = 0;
            if (above < (uint32_t)K && (uint32_t)K <= incl) {
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (above < (uint32_t)K && (uint32_t)K <= above + c[j]) {
                        my_cut = lane * 8 + j;
                        my_above = (int)above;
                        my_count = (int)c[j];
                    }
                    above += c[j];
                }
            }
            const unsigned found = __ballot_sync(kFullMask, my_cut >= 0);
            const int src = __ffs(found) - 1;   // exactly one lane owns the cut bin
            my_cut = __shfl_sync(kFullMask, my_cut, src);
            my_above = __shfl_sync(kFullMask, my_above, src);
            my_count = __shfl_sync(kFullMask, my_count, src);
            if (lane == 0) {
                s.misc[9] = my_count <= kTopkList ? (uint32_t)my_cut : 0xffffffffu;
                s.misc[10] = (uint32_t)(K - my_above);
            }
        }
        tm.sync();   // the histogram has been read: its words are reused for the cut bin's keys
        if (s.misc[9] != 0xffffffffu) {
            cut = (int)s.misc[9];
            need = (int)s.misc[10];
        }
    }
    TopkRegResult out;
    out.mask = 0u;
    if (cut >= 0) {
        uint32_t in_cut = 0u;
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            if (key[j] != 0u) {
                if (bucket[j] > cut) out.mask |= 1u << j;
                if (bucket[j] == cut) in_cut |= 1u << j;
            }
        }
        {
            int slot = warp_append_slots(__popc(in_cut), &s.misc[4]);
#pragma unroll
            for (int j = 0; j < KPT; ++j) {
                if ((in_cut >> j) & 1u) {
                    s.list[slot] = tid + j * stride;
                    s.hist[slot] = key[j];
                    ++slot;
                }
            }
        }
        tm.sync();
        const int m = (int)s.misc[4];
        for (int t = tid; t < m; t += stride) {
            const int idx = s.list[t];
            const uint32_t kt = s.hist[t];
            int rank = 0;
#pragma unroll 8
            for (int u = 0; u < m; ++u) {
                const uint32_t ku = s.hist[u];
                const int iu = s.list[u];
                rank += (int)((ku > kt) | ((ku == kt) & (iu < idx)));
            }
            spill_take[idx] = rank < need ? 1 : 0;   // read back by the element's owner below
            if (rank == need - 1) {
                s.misc[5] = kt;
                s.misc[6] = (uint32_t)idx;
            }
        }
        tm.sync();
#pragma unroll
        for (int j = 0; j < KPT; ++j)
            if (((in_cut >> j) & 1u) && spill_take[tid + j * stride]) out.mask |= 1u << j;
    } else {
        tm.sync();
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            const int i = tid + j * stride;
            if (i < n) {
                spill[i] = key[j];
                spill_take[i] = 0;
            }
        }
        tm.sync();
        team_exact_topk_slow(tm, [&](int i) { return spill[i]; }, n, K, s.hist, s.misc, s.wred,
                             [&](int i) { spill_take[i] = 1; });
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            const int i = tid + j * stride;
            if (i < n && spill_take[i]) out.mask |= 1u << j;
        }
    }
    out.kth_key = s.misc[5];
    out.kth_idx = (int)s.misc[6];
    tm.sync();   // scratch may be reused by the caller right away
    return out;
}

}  // namespace vsa
