// Dense fallback (paper Sec. 10.3, "fallback-to-dense"): plain softmax attention over every token of
// the flagged units, as a split-K pass over the paged cache.  A work item is one (sequence, KV head,
// token range): K and V are read once for all query heads of the group, every half-warp keeps an
// online-softmax state over its own pages, and the partial (max, sum, acc) triples are merged by the
// last block that finishes an item of a (sequence, KV head).  The grid is persistent: a fixed number
// of blocks walk the item list, so a step without any flagged unit costs one nearly empty launch.
#include <math.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"

namespace vsa {

namespace {

constexpr int kDenseThreads = 256;
constexpr int kDenseWarps = kDenseThreads / 32;
constexpr int kDenseGroups = 2 * kDenseWarps;

// partial record per (unit, split): [0] = running max (log2 domain), [1] = sum, [2..130) = acc
constexpr int kPartialFloats = 2 + kHeadDim;

template <int G>
__global__ void __launch_bounds__(kDenseThreads)
dense_split_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_cache,
                   const uint16_t* __restrict__ v_cache, const int32_t* __restrict__ block_table,
                   const int32_t* __restrict__ seq_lens, const int32_t* __restrict__ fallback_list,
                   const int32_t* __restrict__ fallback_count, float epsilon, float* __restrict__ partials,
                   int32_t* __restrict__ counters, float* __restrict__ out, vsa_diag_t* __restrict__ diag,
                   int pages_per_split, int n_splits)
{
    constexpr int ROWS = 16 / G;   // token rows per half-warp per step
    __shared__ float sm_m[kDenseWarps][G], sm_l[kDenseWarps][G];
    __shared__ float sm_acc[kDenseWarps][G][kHeadDim];
    __shared__ int sm_last;
    extern __shared__ uint8_t sm_group_mask[];   // [batch * n_kv_heads] heads of each group that are listed

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, c = lane & 15, gi = lane >> 4;
    const int n_groups = geo.batch * geo.n_kv_heads;
    pdl_wait();
    pdl_launch_dependents();

    // ---- which heads of which groups are listed? ----
    if (fallback_count) {
        const int count = *fallback_count;
        if (count <= 0) return;
        for (int i = tid; i < n_groups; i += kDenseThreads) sm_group_mask[i] = 0;
        __syncthreads();
        for (int i = tid; i < count; i += kDenseThreads) {
            const int u = fallback_list[i];
            const int ub = u / geo.n_q_heads, uh = u % geo.n_q_heads;
            // byte-wide OR through the aligned 32-bit word that holds the group's byte
            const int grp = ub * geo.n_kv_heads + uh / G;
            atomicOr(reinterpret_cast<unsigned int*>(sm_group_mask) + (grp >> 2), (1u << (uh % G)) << (8 * (grp & 3)));
        }
    } else {
        for (int i = tid; i < n_groups; i += kDenseThreads) sm_group_mask[i] = (uint8_t)((1u << G) - 1u);
    }
    __syncthreads();

    const float scale = 1.4426950408889634f / epsilon;   // scores are kept in the log2 domain
    const long long n_items = (long long)n_groups * n_splits;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int grp = (int)(item / n_splits), split = (int)(item % n_splits);
        const uint32_t mask = sm_group_mask[grp];
        if (mask == 0u) continue;
        const int b = grp / geo.n_kv_heads, g = grp % geo.n_kv_heads;
        const int T = seq_lens[b];
        if (T <= 0 || T > geo.max_pages * kPageSize) continue;
        const int nb = (T + kPageSize - 1) / kPageSize;
        const int first_page = split * pages_per_split;
        if (first_page >= nb) continue;
        const int end_page = min(nb, first_page + pages_per_split);
        const int active_splits = (nb + pages_per_split - 1) / pages_per_split;

        float qf[G][8];
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
            const uint4 v = *reinterpret_cast<const uint4*>(
                q + ((long long)b * geo.n_q_heads + g * G + hh) * kHeadDim + c * 8);
            unpack8(v, qf[hh]);
        }
        float m[G], l[G], acc[G][8];
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
            m[hh] = -INFINITY;
            l[hh] = 0.0f;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[hh][e] = 0.0f;
        }

        const int32_t* bt = block_table + (long long)b * geo.max_pages;
        // both half-warps of a warp run the same number of iterations (shuffles need all 32 lanes)
        for (int pl0 = first_page + warp * 2; pl0 < end_page; pl0 += kDenseGroups) {
            const int pl = pl0 + gi;
            bool page_ok = pl < end_page;
            long long phys = 0;
            if (page_ok) {
                phys = bt[pl];
                page_ok = phys >= 0 && phys < geo.pool_pages;
                if (!page_ok) phys = 0;
            }
            const uint16_t* kp = k_cache + phys * geo.page_stride + (long long)g * geo.head_stride + c * 8;
            const uint16_t* vp = v_cache + phys * geo.page_stride + (long long)g * geo.head_stride + c * 8;
#pragma unroll 1
            for (int step = 0; step < G; ++step) {
                uint4 kr[ROWS], vr[ROWS];
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    const int t = step * ROWS + r;
                    const bool ok = page_ok && pl * kPageSize + t < T;
                    kr[r] = make_uint4(0u, 0u, 0u, 0u);
                    vr[r] = make_uint4(0u, 0u, 0u, 0u);
                    if (ok) {
                        kr[r] = ld_nc_16B(kp + (long long)t * geo.token_stride);
                        vr[r] = ld_nc_16B(vp + (long long)t * geo.token_stride);
                    }
                }
                float vals[16];
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    float kf[8];
                    unpack8(kr[r], kf);
#pragma unroll
                    for (int hh = 0; hh < G; ++hh) vals[r * G + hh] = chunk_partial(qf[hh], kf);
                }
                const float s_own = reduce_scatter16(vals, c);   // lane c: (row c / G, head c % G)
                const bool own_ok = page_ok && pl * kPageSize + step * ROWS + c / G < T;
                const float t_own = own_ok ? s_own * scale : -INFINITY;
                float sv[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) sv[i] = __shfl_sync(kFullMask, t_own, (lane & 16) | i);
                float vf[ROWS][8];
#pragma unroll
                for (int r = 0; r < ROWS; ++r) unpack8(vr[r], vf[r]);
#pragma unroll
                for (int hh = 0; hh < G; ++hh) {
                    float mx = sv[hh];
#pragma unroll
                    for (int r = 1; r < ROWS; ++r) mx = fmaxf(mx, sv[r * G + hh]);
                    const float m_new = fmaxf(m[hh], mx);
                    if (m_new == -INFINITY) continue;   // nothing valid seen yet
                    const float corr = exp2f(m[hh] - m_new);
                    m[hh] = m_new;
                    float p[ROWS], psum = 0.0f;
#pragma unroll
                    for (int r = 0; r < ROWS; ++r) {
                        p[r] = exp2f(sv[r * G + hh] - m_new);
                        psum += p[r];
                    }
                    l[hh] = fmaf(l[hh], corr, psum);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        float a = acc[hh][e] * corr;
#pragma unroll
                        for (int r = 0; r < ROWS; ++r) a = fmaf(p[r], vf[r][e], a);
                        acc[hh][e] = a;
                    }
                }
            }
        }

        // ---- merge the two half-warps of each warp, then the warps, into one partial per head ----
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
            const float m2 = __shfl_xor_sync(kFullMask, m[hh], 16);
            const float l2 = __shfl_xor_sync(kFullMask, l[hh], 16);
            const float M = fmaxf(m[hh], m2);
            const float f1 = M == -INFINITY ? 0.0f : exp2f(m[hh] - M);
            const float f2 = M == -INFINITY ? 0.0f : exp2f(m2 - M);
            // lower half-warp first, so that both halves compute the same bits
            const float la = gi == 0 ? l[hh] * f1 : l2 * f2;
            const float lb = gi == 0 ? l2 * f2 : l[hh] * f1;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float a2 = __shfl_xor_sync(kFullMask, acc[hh][e], 16);
                const float xa = gi == 0 ? acc[hh][e] * f1 : a2 * f2;
                const float xb = gi == 0 ? a2 * f2 : acc[hh][e] * f1;
                acc[hh][e] = xa + xb;
            }
            if (gi == 0) {
#pragma unroll
                for (int e = 0; e < 8; ++e) sm_acc[warp][hh][c * 8 + e] = acc[hh][e];
                if (c == 0) {
                    sm_m[warp][hh] = M;
                    sm_l[warp][hh] = la + lb;
                }
            }
        }
        __syncthreads();
        for (int idx = tid; idx < G * kHeadDim; idx += kDenseThreads) {
            const int hh = idx / kHeadDim, e = idx % kHeadDim;
            if (!((mask >> hh) & 1u)) continue;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kDenseWarps; ++w) M = fmaxf(M, sm_m[w][hh]);
            float a = 0.0f, L = 0.0f;
#pragma unroll
            for (int w = 0; w < kDenseWarps; ++w) {
                const float f = sm_m[w][hh] == -INFINITY ? 0.0f : exp2f(sm_m[w][hh] - M);
                a = fmaf(sm_acc[w][hh][e], f, a);
                L = fmaf(sm_l[w][hh], f, L);
            }
            const long long unit = (long long)b * geo.n_q_heads + g * G + hh;
            float* rec = partials + (unit * n_splits + split) * kPartialFloats;
            rec[2 + e] = a;
            if (e == 0) {
                rec[0] = M;
                rec[1] = L;
            }
        }

        // ---- the block that finishes the last split of this (sequence, KV head) combines them ----
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int ticket = atomicAdd(&counters[grp], 1);
            sm_last = ticket == active_splits - 1;
        }
        __syncthreads();
        if (sm_last) {
            __threadfence();
            for (int idx = tid; idx < G * kHeadDim; idx += kDenseThreads) {
                const int hh = idx / kHeadDim, e = idx % kHeadDim;
                if (!((mask >> hh) & 1u)) continue;
                const long long unit = (long long)b * geo.n_q_heads + g * G + hh;
                const float* rec0 = partials + unit * n_splits * kPartialFloats;
                float M = -INFINITY;
                for (int s = 0; s < active_splits; ++s) M = fmaxf(M, __ldcg(rec0 + s * kPartialFloats));
                float a = 0.0f, L = 0.0f;
                for (int s = 0; s < active_splits; ++s) {
                    const float* rec = rec0 + s * kPartialFloats;
                    const float ms = __ldcg(rec);
                    const float f = ms == -INFINITY ? 0.0f : exp2f(ms - M);
                    a = fmaf(__ldcg(rec + 2 + e), f, a);
                    L = fmaf(__ldcg(rec + 1), f, L);
                }
                out[unit * kHeadDim + e] = a / L;
                if (e == 0 && diag) diag[unit].lse = (M + log2f(L)) * 0.6931471805599453f;
            }
        }
        __syncthreads();   // sm_* are reused by the next item
    }
}

int g_num_sms = 0;

int num_sms()
{
    if (g_num_sms == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            g_num_sms = n;
        else
            return 148;
    }
    return g_num_sms;
}

}  // namespace

int dense_pages_per_split(const Geometry& g)
{
    // aim for a few thousand items when every unit is listed; a split is a multiple of 16 pages
    const long long total_pages = (long long)g.batch * g.n_kv_heads * g.max_pages;
    long long pps = (total_pages / 2048 + 15) / 16 * 16;
    if (pps < 16) pps = 16;
    if (pps > 256) pps = 256;
    return (int)pps;
}

static int dense_n_splits(const Geometry& g)
{
    const int pps = dense_pages_per_split(g);
    return (g.max_pages + pps - 1) / pps;
}

static size_t dense_counter_bytes(const Geometry& g)
{
    return (((size_t)g.batch * g.n_kv_heads * sizeof(int32_t)) + 255) / 256 * 256;
}

int32_t* dense_tickets(void* ws_dense) { return (int32_t*)ws_dense; }

int dense_ticket_count(const Geometry& g) { return g.batch * g.n_kv_heads; }

size_t dense_workspace_bytes(const Geometry& g)
{
    return dense_counter_bytes(g) +
           (size_t)g.batch * g.n_q_heads * dense_n_splits(g) * kPartialFloats * sizeof(float);
}

cudaError_t launch_dense(const Geometry& g, const void* q, const void* k_cache, const void* v_cache,
                         const int32_t* block_table, const int32_t* seq_lens, const int32_t* fallback_list,
                         const int32_t* fallback_count, float epsilon, float* out, vsa_diag_t* diag, void* ws,
                         cudaStream_t stream, bool tickets_cleared)
{
    int32_t* counters = (int32_t*)ws;
    float* partials = (float*)((char*)ws + dense_counter_bytes(g));
    cudaError_t e = cudaSuccess;
    if (!tickets_cleared) {
        e = cudaMemsetAsync(counters, 0, dense_counter_bytes(g), stream);
        if (e != cudaSuccess) return e;
    }
    const int pps = dense_pages_per_split(g), ns = dense_n_splits(g);
    const long long n_items = (long long)g.batch * g.n_kv_heads * ns;
    const size_t mask_bytes = ((size_t)g.batch * g.n_kv_heads + 15) / 16 * 16;
    const uint16_t *qq = (const uint16_t*)q, *kk = (const uint16_t*)k_cache, *vv = (const uint16_t*)v_cache;
    // persistent grid: exactly as many blocks as can be resident at once
#define VSA_DENSE_LAUNCH(GG)                                                                                     \
    {                                                                                                            \
        int per_sm = 0;                                                                                          \
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dense_split_kernel<GG>, kDenseThreads,        \
                                                          mask_bytes);                                           \
        if (e != cudaSuccess) return e;                                                                          \
        if (per_sm < 1) per_sm = 1;                                                                              \
        long long blocks = (long long)num_sms() * per_sm;                                                        \
        if (blocks > n_items) blocks = n_items;                                                                  \
        e = launch_pdl(dense_split_kernel<GG>, dim3((unsigned)blocks), dim3(kDenseThreads), mask_bytes, stream, \
                       g, qq, kk, vv, block_table, seq_lens, fallback_list, fallback_count, epsilon, partials,   \
                       counters, out, diag, pps, ns);                                                            \
        if (e != cudaSuccess) return e;                                                                          \
    }
    switch (g.group) {
        case 1: VSA_DENSE_LAUNCH(1); break;
        case 2: VSA_DENSE_LAUNCH(2); break;
        case 4: VSA_DENSE_LAUNCH(4); break;
        case 8: VSA_DENSE_LAUNCH(8); break;
        default: return cudaErrorInvalidValue;
    }
#undef VSA_DENSE_LAUNCH
    return cudaGetLastError();
}

}  // namespace vsa
