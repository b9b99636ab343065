// Group-shared sparse pass: the G query heads that read one KV head route as ONE query (a reading of
// paper Sec. 7 steps 1-4 for grouped-query attention, where the paper has a single query per step).
// One thread block of 512 threads per (sequence, KV head):
//
//   top-P pages of the SUMMED page scores (sum over the group's heads of the scan's per-head fp32 scores,
//     ascending head order)                                         - one selection per group, not per head
//   per warp: K tile of a routed page -> shared memory by ONE bulk copy (4 KB, mbarrier), scored for all G
//     heads with the fixed-order dot product; the slot is then refilled with the warp's next K tile or,
//     once its K tiles are done, with the page's V tile (in flight during the selection)
//   exact top-(K_c + 1) of the SUMMED token scores                  - one selection per group
//   per head: best / second best inside the candidate set, best outside it, softmax weights of its own
//     scores over the shared candidates (written over the scores)
//   per warp: V tile x the weights of every head at once; block reduction; out / diag / fallback list
//
// Every K and V tile is read once per group, the two selections run once per group, and the candidate
// math is a G x (P * 16) x 128 score block and a G x K_c x 128 readout per group.  The scores that decide
// the selections stay on the CUDA cores in the fixed summation order (the sets are bit-exact against the
// CPU oracle); nothing but the routed pages' tiles is staged.  Needs the native cache layout (a (page, KV
// head) tile is 4 KB contiguous).
#pragma once

#include <limits.h>
#include <math.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"
#include "vsa_team.cuh"

namespace vsa {

namespace {

constexpr int kSharedThreads = 512;
constexpr int kSharedWarps = kSharedThreads / 32;
constexpr int kTileBytes = kPageSize * kRowBytes;     // 4096: one (page, KV head) tile of K or of V
constexpr int kSlotsPerWarp = 2;
constexpr int kSharedSlots = kSharedWarps * kSlotsPerWarp;
constexpr int kPageKeysCached = 16;                   // summed page scores per thread kept in registers
constexpr int kTeamScratchWords = 256 + 16 + 72 + kTopkList;
constexpr uint32_t kWaitLimit = 1u << 22;             // polls of a tile's barrier before the group is failed

// ---- bulk copies global -> shared with completion on an mbarrier -------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t addr, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(addr), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t addr, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(__cvta_generic_to_global(src)), "r"(bytes), "r"(mbar)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t addr, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok)
                 : "r"(addr), "r"(parity)
                 : "memory");
    return ok != 0u;
}
// bounded wait: false when the copy has not landed after kWaitLimit polls
__device__ __forceinline__ bool mbar_wait(uint32_t addr, uint32_t parity)
{
    for (uint32_t it = 0; it < kWaitLimit; ++it)
        if (mbar_try_wait(addr, parity)) return true;
    return false;
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- shared-memory layout, in 4-byte words from the start of dynamic shared memory ---------------------
struct SharedLayout {
    int tiles, mbar, q32, sc, keys, take, scratch, lists, upage, uphys, hwarp, hfin, ctl, total;
};

__host__ __device__ inline SharedLayout shared_layout(int G, int P)
{
    const int N = P * kPageSize;
    SharedLayout l;
    int w = 0;
    l.tiles = w;    w += kSharedSlots * kTileBytes / 4;
    l.mbar = w;     w += kSharedSlots * 2;
    l.q32 = w;      w += G * kHeadDim;
    l.sc = w;       w += G * N;                 // per-head token scores, later the weights
    l.keys = w;     w += N;                     // keys of the summed scores (slow path of the selection)
    l.take = w;     w += (N + 3) / 4;
    l.scratch = w;  w += kTeamScratchWords;
    l.lists = w;    w += 5 * P;
    l.upage = w;    w += P;
    l.uphys = w;    w += P;
    l.hwarp = w;    w += G * kSharedWarps * 4;  // per (head, warp): best, second best, best rejected, sum
    l.hfin = w;     w += G * 8;                 // per head: s1, s2, rejected, Z
    l.ctl = w;      w += 16;
    l.total = w;
    return l;
}

// G: query heads per KV head.  TOK_KPT: summed token scores per thread, P * 16 <= TOK_KPT * 512.
// routed_pages is [batch][n_kv_heads][P], written here (best first, -1 padded).
template <int G, int TOK_KPT>
__global__ void __launch_bounds__(kSharedThreads, 1)
sparse_shared_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_cache,
                     const uint16_t* __restrict__ v_cache, const int32_t* __restrict__ block_table,
                     const int32_t* __restrict__ seq_lens, int32_t* __restrict__ routed_pages,
                     const float* __restrict__ page_scores, int P, int K_c, float epsilon, float gap_threshold,
                     float* __restrict__ out, vsa_diag_t* __restrict__ diag, int32_t* __restrict__ fallback_list,
                     int32_t* __restrict__ fallback_count)
{
    extern __shared__ __align__(128) uint32_t ssm[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, c = lane & 15, gi = lane >> 4;
    const int N = P * kPageSize;
    const SharedLayout L = shared_layout(G, P);
    uint8_t* tiles = (uint8_t*)(ssm + L.tiles);
    float* q32 = (float*)(ssm + L.q32);
    float* sc = (float*)(ssm + L.sc);
    uint32_t* keys = ssm + L.keys;
    uint8_t* take = (uint8_t*)(ssm + L.take);
    int32_t* upage = (int32_t*)(ssm + L.upage);
    int32_t* uphys = (int32_t*)(ssm + L.uphys);
    uint32_t* hwarp = ssm + L.hwarp;
    float* hfin = (float*)(ssm + L.hfin);
    uint32_t* ctl = ssm + L.ctl;   // [0] a routed page is outside the pool, [1] a copy timed out
    const uint32_t tiles_s = (uint32_t)__cvta_generic_to_shared(tiles);
    const uint32_t mbar_s = (uint32_t)__cvta_generic_to_shared(ssm + L.mbar);
    const Team tm{tid, kSharedThreads, 1};
    TopkScratch ts;
    ts.hist = ssm + L.scratch;
    ts.misc = ts.hist + 256;
    ts.wred = ts.misc + 16;
    ts.list = (int32_t*)(ts.wred + 72);
    uint32_t* tmp_key = ssm + L.lists;
    int32_t* tmp_idx = (int32_t*)(tmp_key + P);
    uint32_t* win_key = (uint32_t*)(tmp_idx + P);
    int32_t* win_idx = (int32_t*)(win_key + P);
    int32_t* asc_idx = win_idx + P;

    const int b = blockIdx.x / geo.n_kv_heads, g = blockIdx.x % geo.n_kv_heads;
    const long long group_id = blockIdx.x;
    const long long unit0 = (long long)b * geo.n_q_heads + (long long)g * G;

    // ---- before the wait on the preceding kernel: what no kernel of the step produces ----
    const int T = ld_ca_s32(seq_lens + b);
    if (tid < G * 16) {
        const uint4 raw = ld_nc_16B(q + (unit0 + tid / 16) * kHeadDim + (tid % 16) * 8);
        float f[8];
        unpack8(raw, f);
#pragma unroll
        for (int e = 0; e < 8; ++e) q32[(tid / 16) * kHeadDim + (tid % 16) * 8 + e] = f[e];
    }
    if (tid < 16) ctl[tid] = 0u;
    if (tid < kSharedSlots) mbar_init(mbar_s + 8u * (uint32_t)tid, 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    pdl_wait();
    pdl_launch_dependents();

    const bool okT = T > 0 && T <= geo.max_pages * kPageSize;
    const int nb = okT ? (T + kPageSize - 1) / kPageSize : 0;
    // summed page score: the group's per-head scores added in ascending head order
    const float* sc_rows = page_scores + unit0 * geo.max_pages;
    auto page_key = [&](int i) {
        float acc = __ldcg(sc_rows + i);
#pragma unroll
        for (int hh = 1; hh < G; ++hh) acc = __fadd_rn(acc, __ldcg(sc_rows + (long long)hh * geo.max_pages + i));
        return float_to_key(acc);
    };
    uint32_t kc[kPageKeysCached];
#pragma unroll
    for (int j = 0; j < kPageKeysCached; ++j) {
        const int i = tid + j * kSharedThreads;
        kc[j] = i < nb ? page_key(i) : 0u;
    }
    if (!okT) {
        for (int o = tid; o < G * kHeadDim; o += kSharedThreads) out[unit0 * kHeadDim + o] = 0.0f;
        if (tid < G) {
            vsa_diag_t d;
            d.delta = d.delta12 = d.s_max = d.lse = d.leak_bound = 0.0f;
            d.n_candidates = 0;
            d.fallback = 0;
            d.status = VSA_UNIT_BAD_LENGTH;
            diag[unit0 + tid] = d;
        }
        for (int t = tid; t < P; t += kSharedThreads) routed_pages[group_id * P + t] = -1;
        return;
    }
    __syncthreads();

    // ---- the group's routed pages ----
    const int np = team_top_pages<kPageKeysCached>(tm, page_key, kc, nb, P, ts, tmp_key, tmp_idx, win_key, win_idx,
                                                   asc_idx);
    for (int t = tid; t < P; t += kSharedThreads) {
        routed_pages[group_id * P + t] = t < np ? win_idx[t] : -1;
        int l = -1, phys = -1;
        if (t < np) {
            l = asc_idx[t];
            phys = __ldg(block_table + (long long)b * geo.max_pages + l);
            if (phys < 0 || phys >= geo.pool_pages) {
                phys = -1;
                ctl[0] = 1u;
            }
        }
        upage[t] = l;
        uphys[t] = phys;
    }
    __syncthreads();

    // ---- tiles: warp w takes the routed pages w, w + 16, ... (ascending page order); two slots per warp ----
    const int nK = np > warp ? (np - warp + kSharedWarps - 1) / kSharedWarps : 0;
    const uint32_t my_slot = tiles_s + (uint32_t)(warp * kSlotsPerWarp * kTileBytes);
    const uint32_t my_bar = mbar_s + 8u * (uint32_t)(warp * kSlotsPerWarp);
    uint32_t par = 0u;     // phase parity of the warp's two barriers
    bool wait_failed = false;
    auto page_of = [&](int i) { return warp + kSharedWarps * i; };
    auto issue = [&](const uint16_t* cache, int i, int slot) {   // lane 0 only
        const long long phys = uphys[page_of(i)];
        mbar_expect_tx(my_bar + 8u * (uint32_t)slot, (uint32_t)kTileBytes);
        bulk_load(my_slot + (uint32_t)(slot * kTileBytes),
                  cache + phys * geo.page_stride + (long long)g * geo.head_stride, (uint32_t)kTileBytes,
                  my_bar + 8u * (uint32_t)slot);
    };
    if (lane == 0) {
        if (nK > 0 && uphys[page_of(0)] >= 0) issue(k_cache, 0, 0);
        if (nK > 1 && uphys[page_of(1)] >= 0) issue(k_cache, 1, 1);
    }
    for (int i = 0; i < nK; ++i) {
        const int u = page_of(i), slot = i & 1;
        const bool ok = uphys[u] >= 0;
        uint4 rows[8];
        if (ok) {
            if (!mbar_wait(my_bar + 8u * (uint32_t)slot, (par >> slot) & 1u)) wait_failed = true;
            par ^= 1u << slot;
            const uint8_t* src = tiles + (warp * kSlotsPerWarp + slot) * kTileBytes + gi * 8 * kRowBytes + c * 16;
#pragma unroll
            for (int r = 0; r < 8; ++r) rows[r] = *reinterpret_cast<const uint4*>(src + r * kRowBytes);
        }
        __syncwarp();
        if (lane == 0) {
            // the slot's rows are in registers: refill it with the warp's next K tile or, when there is
            // none, with the V tile of the warp's first (second) page, which the readout will need
            fence_async_proxy();
            if (i + 2 < nK) {
                if (uphys[page_of(i + 2)] >= 0) issue(k_cache, i + 2, slot);
            } else if (uphys[page_of(slot)] >= 0) {
                issue(v_cache, slot, slot);
            }
        }
        if (!ok) continue;
        // scores of the page's sixteen tokens for every head, two heads per reduction: this half-warp holds
        // rows gi * 8 .. gi * 8 + 7; value v of the sixteen reduced at once is (head ha if v < 8 else ha + 1,
        // row v & 7)
        const int l = upage[u];
#pragma unroll
        for (int ha = 0; ha < G; ha += 2) {
            const int hb = ha + 1 < G ? ha + 1 : ha;
            float qa[8], qb[8];
            {
                const float4 a0 = *reinterpret_cast<const float4*>(q32 + ha * kHeadDim + c * 8);
                const float4 a1 = *reinterpret_cast<const float4*>(q32 + ha * kHeadDim + c * 8 + 4);
                qa[0] = a0.x; qa[1] = a0.y; qa[2] = a0.z; qa[3] = a0.w;
                qa[4] = a1.x; qa[5] = a1.y; qa[6] = a1.z; qa[7] = a1.w;
                const float4 b0 = *reinterpret_cast<const float4*>(q32 + hb * kHeadDim + c * 8);
                const float4 b1 = *reinterpret_cast<const float4*>(q32 + hb * kHeadDim + c * 8 + 4);
                qb[0] = b0.x; qb[1] = b0.y; qb[2] = b0.z; qb[3] = b0.w;
                qb[4] = b1.x; qb[5] = b1.y; qb[6] = b1.z; qb[7] = b1.w;
            }
            float vals[16];
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                float kf[8];
                unpack8(rows[r], kf);
                vals[r] = chunk_partial(qa, kf);
                vals[8 + r] = chunk_partial(qb, kf);
            }
            const float s = reduce_scatter16(vals, c);
            const int hd = c < 8 ? ha : ha + 1, t = gi * 8 + (c & 7);
            if (hd < G && l * kPageSize + t < T) sc[hd * N + u * kPageSize + t] = s;
        }
    }
    __syncthreads();
    const bool bad_page = ctl[0] != 0u;

    // ---- one exact top-(K_c + 1) of the summed token scores ----
    int ns;
    bool has_rejected;
    uint32_t mask = 0u;
    {
        uint32_t key[TOK_KPT];
        int present = 0;
        uint32_t a1 = 0u, amin = 0xffffffffu;
#pragma unroll
        for (int j = 0; j < TOK_KPT; ++j) {
            const int i = tid + j * kSharedThreads;
            key[j] = 0u;
            if (i < N) {
                const int slot = i >> 4;
                if (slot < np && uphys[slot] >= 0 && upage[slot] * kPageSize + (i & 15) < T) {
                    float acc = sc[i];
#pragma unroll
                    for (int hh = 1; hh < G; ++hh) acc = __fadd_rn(acc, sc[hh * N + i]);
                    key[j] = float_to_key(acc);
                }
            }
            present += key[j] != 0u;
            if (key[j] != 0u) amin = min(amin, key[j]);
            a1 = max(a1, key[j]);
        }
        present = __reduce_add_sync(kFullMask, present);
        amin = __reduce_min_sync(kFullMask, amin);
        a1 = __reduce_max_sync(kFullMask, a1);
        if (lane == 0) {
            ts.wred[4 * warp] = a1;
            ts.wred[4 * warp + 2] = (uint32_t)present;
            ts.wred[4 * warp + 3] = amin;
        }
        for (int i = tid; i < 256; i += kSharedThreads) ts.hist[i] = 0u;
        if (tid == 0) ts.misc[4] = 0u;
        __syncthreads();
        // each warp's best key: the smallest of those (hi_r) and the largest of the warps' smallest keys
        // (lo_r) bracket the bulk of the scores and serve as the histogram range of the selection
        uint32_t key1 = 0u, kmin = 0xffffffffu, hi_r = 0xffffffffu, lo_r = 0u;
        int n_valid = 0;
#pragma unroll
        for (int w = 0; w < kSharedWarps; ++w) {
            const uint32_t b1 = ts.wred[4 * w], bmin = ts.wred[4 * w + 3];
            key1 = max(key1, b1);
            n_valid += (int)ts.wred[4 * w + 2];
            kmin = min(kmin, bmin);
            if (b1 != 0u) hi_r = min(hi_r, b1);
            if (bmin != 0xffffffffu) lo_r = max(lo_r, bmin);
        }
        ns = min(K_c, n_valid);
        has_rejected = n_valid > ns;
        if (has_rejected) {
            const TopkRegResult r = team_topk_reg<TOK_KPT>(tm, key, N, ns + 1, ts, keys, take, key_to_float(lo_r),
                                                           key_to_float(hi_r), key_to_float(kmin), key_to_float(key1));
            mask = r.mask;
#pragma unroll
            for (int j = 0; j < TOK_KPT; ++j)
                if (tid + j * kSharedThreads == r.kth_idx) mask &= ~(1u << j);
        } else {
#pragma unroll
            for (int j = 0; j < TOK_KPT; ++j)
                if (key[j] != 0u) mask |= 1u << j;
        }
        // per head: best and second best of its own scores inside the set, best outside it
        uint32_t valid = 0u;
#pragma unroll
        for (int j = 0; j < TOK_KPT; ++j)
            if (key[j] != 0u) valid |= 1u << j;
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
            uint32_t m1 = 0u, m2 = 0u, rj = 0u;
#pragma unroll
            for (int j = 0; j < TOK_KPT; ++j) {
                if ((valid >> j) & 1u) {
                    const uint32_t k = float_to_key(sc[hh * N + tid + j * kSharedThreads]);
                    if ((mask >> j) & 1u) {
                        if (k > m1) {
                            m2 = m1;
                            m1 = k;
                        } else if (k > m2) {
                            m2 = k;
                        }
                    } else {
                        rj = max(rj, k);
                    }
                }
            }
            const uint32_t wmax = __reduce_max_sync(kFullMask, m1);
            const int holder = __ffs(__ballot_sync(kFullMask, m1 == wmax)) - 1;
            const uint32_t wsecond = __reduce_max_sync(kFullMask, lane == holder ? m2 : m1);
            const uint32_t wrej = __reduce_max_sync(kFullMask, rj);
            if (lane == 0) {
                hwarp[(hh * kSharedWarps + warp) * 4] = wmax;
                hwarp[(hh * kSharedWarps + warp) * 4 + 1] = wsecond;
                hwarp[(hh * kSharedWarps + warp) * 4 + 2] = wrej;
            }
        }
        __syncthreads();
        if (tid < G) {
            uint32_t k1 = 0u, k2 = 0u, kr = 0u;
            for (int w = 0; w < kSharedWarps; ++w) {
                const uint32_t b1 = hwarp[(tid * kSharedWarps + w) * 4], b2 = hwarp[(tid * kSharedWarps + w) * 4 + 1];
                const uint32_t n1 = max(k1, b1), n2 = max(min(k1, b1), max(k2, b2));
                k1 = n1;
                k2 = n2;
                kr = max(kr, hwarp[(tid * kSharedWarps + w) * 4 + 2]);
            }
            hfin[tid * 8] = ns > 0 ? key_to_float(k1) : -INFINITY;
            hfin[tid * 8 + 1] = ns > 1 ? key_to_float(k2) : -INFINITY;
            hfin[tid * 8 + 2] = has_rejected ? key_to_float(kr) : -INFINITY;
        }
        __syncthreads();
        // weights of every head over the shared candidates, written over the scores; their sums
        const float scale = 1.4426950408889634f / epsilon;   // log2(e) / epsilon
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
            const float s1 = hfin[hh * 8];
            float z = 0.0f;
#pragma unroll
            for (int j = 0; j < TOK_KPT; ++j) {
                const int i = tid + j * kSharedThreads;
                if (i < N) {
                    const float w = ((mask >> j) & 1u) ? exp2f((sc[hh * N + i] - s1) * scale) : 0.0f;
                    sc[hh * N + i] = w;
                    z += w;
                }
            }
#pragma unroll
            for (int off = 16; off; off >>= 1) z += __shfl_xor_sync(kFullMask, z, off);
            if (lane == 0) hwarp[(hh * kSharedWarps + warp) * 4 + 3] = __float_as_uint(z);
        }
    }
    __syncthreads();
    if (tid < G) {
        float Z = 0.0f;
        for (int w = 0; w < kSharedWarps; ++w) Z += __uint_as_float(hwarp[(tid * kSharedWarps + w) * 4 + 3]);
        hfin[tid * 8 + 3] = Z;
        if (!bad_page) {
            const float s1 = hfin[tid * 8], s2 = hfin[tid * 8 + 1], rej = hfin[tid * 8 + 2];
            const float delta = has_rejected ? s1 - rej : INFINITY;
            vsa_diag_t d;
            d.delta = delta;
            d.delta12 = ns > 0 ? s1 - s2 : INFINITY;
            d.s_max = s1;
            d.lse = ns > 0 ? s1 / epsilon + logf(Z) : -INFINITY;
            d.leak_bound = fminf(1.0f, (float)(T - ns) * expf(-delta / epsilon));
            d.n_candidates = ns;
            d.fallback = (delta < gap_threshold && ns < T) ? 1 : 0;
            d.status = 0;
            diag[unit0 + tid] = d;
            if (d.fallback) fallback_list[atomicAdd(fallback_count, 1)] = (int32_t)(unit0 + tid);
        }
    }

    // ---- V tiles x the weights of every head (a page none of whose tokens was kept is skipped) ----
    float acc[G][8];
#pragma unroll
    for (int hh = 0; hh < G; ++hh)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[hh][e] = 0.0f;
    auto page_needed = [&](int u) {   // a warp-wide result
        bool nz = false;
        if (lane < kPageSize) {
#pragma unroll
            for (int hh = 0; hh < G; ++hh) nz |= sc[hh * N + u * kPageSize + lane] != 0.0f;
        }
        return __ballot_sync(kFullMask, nz) != 0u && !bad_page;
    };
    for (int j = 0; j < nK; ++j) {
        const int u = page_of(j), slot = j & 1;
        const bool ok = uphys[u] >= 0;
        const bool need = page_needed(u);
        const bool issued = ok && (j < 2 || need);
        if (issued) {
            if (!mbar_wait(my_bar + 8u * (uint32_t)slot, (par >> slot) & 1u)) wait_failed = true;
            par ^= 1u << slot;
        }
        if (issued && need) {
            const uint8_t* src = tiles + (warp * kSlotsPerWarp + slot) * kTileBytes + gi * 8 * kRowBytes + c * 16;
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                float vf[8];
                unpack8(*reinterpret_cast<const uint4*>(src + r * kRowBytes), vf);
#pragma unroll
                for (int hh = 0; hh < G; ++hh) {
                    const float w = sc[hh * N + u * kPageSize + gi * 8 + r];
#pragma unroll
                    for (int e = 0; e < 8; e += 2) fma2(acc[hh][e], acc[hh][e + 1], w, w, vf[e], vf[e + 1]);
                }
            }
        }
        const int nxt = j + 2;
        const bool need_next = nxt < nK ? page_needed(page_of(nxt)) : false;
        __syncwarp();
        if (lane == 0 && need_next && uphys[page_of(nxt)] >= 0) {
            fence_async_proxy();
            issue(v_cache, nxt, slot);
        }
    }
    if (wait_failed) atomicOr(&ctl[1], 1u);
    __syncthreads();   // every tile has been consumed: the tile area takes the warps' partial sums

    float* part = (float*)tiles;   // [warp][G][128]
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[hh][e] += __shfl_xor_sync(kFullMask, acc[hh][e], 16);
        if (gi == 0) {
            float* dst = part + (warp * G + hh) * kHeadDim + c * 8;
            *reinterpret_cast<float4*>(dst) = make_float4(acc[hh][0], acc[hh][1], acc[hh][2], acc[hh][3]);
            *reinterpret_cast<float4*>(dst + 4) = make_float4(acc[hh][4], acc[hh][5], acc[hh][6], acc[hh][7]);
        }
    }
    __syncthreads();
    const bool failed = bad_page || ctl[1] != 0u;
    for (int o = tid; o < G * kHeadDim; o += kSharedThreads) {
        const int hh = o / kHeadDim, col = o - hh * kHeadDim;
        float a = 0.0f;
#pragma unroll
        for (int w = 0; w < kSharedWarps; ++w) a += part[(w * G + hh) * kHeadDim + col];
        out[(unit0 + hh) * kHeadDim + col] = (!failed && ns > 0) ? a / hfin[hh * 8 + 3] : 0.0f;
    }
    if (tid < G && failed) {
        vsa_diag_t d;
        d.delta = d.delta12 = d.s_max = d.lse = d.leak_bound = 0.0f;
        d.n_candidates = 0;
        d.fallback = 0;
        d.status = bad_page ? VSA_UNIT_BAD_PAGE : VSA_UNIT_COPY_TIMEOUT;
        diag[unit0 + tid] = d;
    }
}

template <int G, int TOK_KPT>
cudaError_t launch_shared_variant(const GroupSharedArgs& a)
{
    const size_t smem = (size_t)shared_layout(G, a.P).total * 4;
    static bool attr_done[kMaxDevices] = {};   // per template instance
    const cudaError_t e = allow_large_dynamic_smem(sparse_shared_kernel<G, TOK_KPT>, attr_done);
    if (e != cudaSuccess) return e;
    const unsigned blocks = (unsigned)(a.g.batch * a.g.n_kv_heads);
    return launch_pdl(sparse_shared_kernel<G, TOK_KPT>, dim3(blocks), dim3(kSharedThreads), smem, a.stream, a.g, a.q,
                      a.k, a.v, a.block_table, a.seq_lens, a.routed_pages, a.page_scores, a.P, a.K_c, a.epsilon,
                      a.gap_threshold, a.out, a.diag, a.fallback_list, a.fallback_count);
}

template <int G>
cudaError_t launch_shared_tok(const GroupSharedArgs& a)
{
    const int per_thread = (a.P * kPageSize + kSharedThreads - 1) / kSharedThreads;
    if (per_thread <= 1) return launch_shared_variant<G, 1>(a);
    if (per_thread <= 2) return launch_shared_variant<G, 2>(a);
    if (per_thread <= 4) return launch_shared_variant<G, 4>(a);
    return cudaErrorInvalidValue;
}

}  // namespace

}  // namespace vsa
