// Dense fallback (paper Sec. 10.3, "fallback-to-dense"): plain softmax attention over every token of
// the flagged units, as a split-K pass over the paged cache.
//
// This is the one place of the step where the arithmetic is a real dense contraction - the G query
// heads of a GQA group against the same K and V tiles - and where only the output (not a discrete
// decision) depends on it, so it runs on the tensor cores: per 16-token page and warp,
//   S[heads x 16]  = Q[heads x 128] . K_page^T      (16 mma.m16n8k16, bf16 in, fp32 accumulate)
//   O[heads x 128] += P[heads x 16] . V_page        (16 mma.m16n8k16)
// with the heads padded to the 16-row MMA tile and an online softmax in between.  K and V tiles
// stream through a per-warp cp.async ring (three pages deep, XOR-swizzled for ldmatrix).
//
// Work decomposition: an item is (sequence, KV head, range of pages); K and V are read once for all
// listed heads of the group.  The number of pages per item is chosen ON THE DEVICE from how much
// was flagged, so that one flagged head of a 128k-token sequence is spread over the whole chip
// while a full dense pass uses long items.  A persistent grid (one block per SM) walks the items;
// the block that finishes the last item of a (sequence, KV head) combines its partials.
#include <math.h>

#include <cuda_fp8.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"

namespace vsa {

namespace {

constexpr int kStages = 3;                         // pages in flight per warp
constexpr int kTileRows = 16;                      // the pass walks tiles of 16 tokens: one per 16-token page, two per 32-token page
constexpr int kPagesPerItemGoal = 128;             // pages per item and block from which a second round pays
constexpr int kMaxRounds = 2;
constexpr int kMaxRoundsRagged = 8;

// Sizes that depend on the head dimension D (64, 128 or 256).  The ring of a block holds three stages of a
// K tile and a V tile per warp: 192 KB with eight warps at D = 128; D = 256 runs four warps per block so
// that the same ring fits.
// FP8 (D = 128): the unit of work is 32 tokens (two tiles); a stage holds their e4m3 rows as they are (4 KB of
// K, 4 KB of V, the four scales) and the tensor cores consume them directly (m16n8k32 e4m3 MMAs).
template <int D, bool FP8 = false>
struct DenseCfg {
    static constexpr int kDenseThreads = D == 256 ? 128 : 256;
    static constexpr int kDenseWarps = kDenseThreads / 32;
    static constexpr int kRowBytes = 2 * D;
    static constexpr int kTileBytes = kTileRows * kRowBytes;   // K (or V) rows of one tile and KV head (4 KB at D = 128)
    static constexpr int kUnitRows = FP8 ? 32 : kTileRows;     // tokens per unit of work of a warp
    static constexpr int kRawBytes = 32 * D;                   // FP8: K (or V) rows of a unit as e4m3 bytes
    static constexpr int kStageBytes = FP8 ? 2 * kRawBytes + 16 : 2 * kTileBytes;   // K + V (+ scales)
    static constexpr int kWarpBytes = kStages * kStageBytes;
    static constexpr int kRingBytes = kDenseWarps * kWarpBytes;
    static constexpr int kPartialFloats = 2 + D;               // per (item, head): max (log2 domain), sum, acc[D]
    static constexpr int kMinPagesPerItem = 2 * kDenseWarps;   // at least two pages per warp: one would expose the DRAM latency
};

__device__ __forceinline__ void cp_async_16_zfill(uint32_t smem_addr, const void* gptr, bool valid)
{
    const int n = valid ? 16 : 0;   // src-size 0: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_addr), "l"(gptr), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col); rows 8..15 of A are zero here
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    const uint32_t zero = 0u;
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                 "{%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(zero), "r"(a2), "r"(zero), "r"(b0), "r"(b1));
}
// D (16x8, fp32) += A (16x32, e4m3, row) * B (32x8, e4m3, col).  The (at most eight) heads occupy rows 0..7 of
// A with the high e4m3 term of each operand value and rows 8..15 with the low term (a1, a3), so that one MMA
// forms both partial products: d[0], d[1] (row g) and d[2], d[3] (row g + 8) are added by the caller.
__device__ __forceinline__ void mma_e4m3(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                 "{%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// 16 x 16 bytes, transposed: lane (g = lane / 4, t = lane % 4) receives rows 4t .. 4t+3 of column g (first
// register) and of column g + 8 (second); .x2 loads a second matrix (addresses from lanes 16 .. 31) into r2, r3
__device__ __forceinline__ void ldmatrix_x2_trans_b8(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m16n16.x2.trans.shared.b8 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// x = hi + lo with hi, lo e4m3 (x of up to eight significant bits inside the e4m3 range splits exactly)
__device__ __forceinline__ void split_e4m3x2(float x0, float x1, uint32_t& hi, uint32_t& lo)
{
    const __nv_fp8x2_storage_t h = __nv_cvt_float2_to_fp8x2(make_float2(x0, x1), __NV_SATFINITE, __NV_E4M3);
    const __half2_raw hr = __nv_cvt_fp8x2_to_halfraw2(h, __NV_E4M3);
    const float2 hf = __half22float2(*reinterpret_cast<const __half2*>(&hr));
    const __nv_fp8x2_storage_t l = __nv_cvt_float2_to_fp8x2(make_float2(x0 - hf.x, x1 - hf.y), __NV_SATFINITE, __NV_E4M3);
    hi = h;
    lo = l;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

struct DenseSmem {
    uint8_t* ring;         // [warps][stages][K tile | V tile]; reused for the cross-warp merge
    int32_t* item_base;    // [n_groups + 1] first item of every group (exclusive scan)
    uint8_t* group_mask;   // [n_groups] listed heads of the group
    int32_t* misc;         // [16]
};

template <int G, int D = vsa::kHeadDim, bool FP8 = false>
__global__ void __launch_bounds__(DenseCfg<D>::kDenseThreads, 1)
dense_split_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_cache,
                   const uint16_t* __restrict__ v_cache, const int32_t* __restrict__ block_table,
                   const int32_t* __restrict__ seq_lens, const int32_t* __restrict__ fallback_list,
                   const int32_t* __restrict__ fallback_count, float epsilon, float* __restrict__ partials,
                   int32_t* __restrict__ counters, float* __restrict__ out, vsa_diag_t* __restrict__ diag,
                   int max_items, const float* __restrict__ k_scale, const float* __restrict__ v_scale)
{
    static_assert(!FP8 || D == 128, "fp8 cache: head dimension 128");
    using Cfg = DenseCfg<D, FP8>;
    constexpr int kDenseThreads = Cfg::kDenseThreads, kDenseWarps = Cfg::kDenseWarps, kRowBytes = Cfg::kRowBytes,
                  kTileBytes = Cfg::kTileBytes, kStageBytes = Cfg::kStageBytes, kRingBytes = Cfg::kRingBytes,
                  kPartialFloats = Cfg::kPartialFloats, kMinPagesPerItem = Cfg::kMinPagesPerItem, kHeadDim = D;
    constexpr int kUnit = Cfg::kUnitRows;
    constexpr int KS = D / 16;    // 16-element steps of the Q K^T contraction = 16-column steps of P V
    constexpr int NT = D / 8;     // 8-column output tiles
    constexpr int CPR = D / 8;    // 16-byte chunks per row
    constexpr int RPI = 32 / (CPR < 32 ? CPR : 32);   // rows one copy instruction of a warp covers
    extern __shared__ __align__(128) uint8_t dense_smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_groups = geo.batch * geo.n_kv_heads;
    DenseSmem sm;
    sm.ring = dense_smem;
    sm.item_base = (int32_t*)(dense_smem + kRingBytes);
    sm.misc = sm.item_base + n_groups + 1;
    sm.group_mask = (uint8_t*)(sm.misc + 16);
    pdl_wait();
    pdl_launch_dependents();

    // ---- which heads of which groups are listed? ----
    if (fallback_count) {
        const int count = *fallback_count;
        if (count <= 0) return;
        for (int i = tid; i < n_groups; i += kDenseThreads) sm.group_mask[i] = 0;
        __syncthreads();
        for (int i = tid; i < count; i += kDenseThreads) {
            const int u = fallback_list[i];
            const int ub = u / geo.n_q_heads, uh = u % geo.n_q_heads;
            const int grp = ub * geo.n_kv_heads + uh / G;
            // byte-wide OR through the aligned 32-bit word that holds the group's byte
            atomicOr(reinterpret_cast<unsigned int*>(sm.group_mask) + (grp >> 2), (1u << (uh % G)) << (8 * (grp & 3)));
        }
    } else {
        for (int i = tid; i < n_groups; i += kDenseThreads) sm.group_mask[i] = (uint8_t)((1u << G) - 1u);
    }
    if (tid < 16) sm.misc[tid] = 0;
    __syncthreads();

    // ---- pages per item from the amount of flagged work, then the item table ----
    auto pages_of = [&](int grp) -> int {
        if (!sm.group_mask[grp]) return 0;
        const int T = seq_lens[grp / geo.n_kv_heads];
        if (!geo.length_ok(T)) return 0;
        return (T + kUnit - 1) / kUnit;
    };
    {
        int pages = 0, groups = 0, longest = 0;
        for (int i = tid; i < n_groups; i += kDenseThreads) {
            const int p = pages_of(i);
            pages += p;
            groups += p > 0;
            longest = max(longest, p);
        }
#pragma unroll
        for (int off = 16; off; off >>= 1) {
            pages += __shfl_xor_sync(kFullMask, pages, off);
            groups += __shfl_xor_sync(kFullMask, groups, off);
            longest = max(longest, __shfl_xor_sync(kFullMask, longest, off));
        }
        if (lane == 0) {
            atomicAdd(&sm.misc[0], pages);
            atomicAdd(&sm.misc[1], groups);
            atomicMax(&sm.misc[2], longest);
        }
    }
    __syncthreads();
    const int total_pages = sm.misc[0], flagged_groups = sm.misc[1], longest_group = sm.misc[2];
    if (total_pages == 0) return;
    int ppi;   // pages per item, a multiple of the warp count
    {
        // Whole rounds: at most `rounds` items per block - one when the work is small (an item costs a few
        // microseconds of fixed overhead: query fragments, pipeline fill, merge, ticket), two when items
        // stay long.  Every group may add one ragged item, so sizing for (target - groups) full items
        // keeps the count within the target and no block starts a round the others do not have.
        long long rounds = total_pages / ((long long)gridDim.x * kPagesPerItemGoal);
        rounds = rounds < 1 ? 1 : (rounds > kMaxRounds ? kMaxRounds : rounds);   // 1 or 2
        // many flagged groups of uneven length (the longest more than twice the mean): about four items
        // per group, so that short and long groups mix over the blocks
        if ((long long)longest_group * flagged_groups > 2LL * total_pages) {
            const long long by_groups = (4LL * flagged_groups + gridDim.x - 1) / gridDim.x;
            if (rounds < by_groups) rounds = by_groups < kMaxRoundsRagged ? by_groups : kMaxRoundsRagged;
        }
        const long long target = (long long)gridDim.x * rounds;
        long long want = target > 2LL * flagged_groups ? (total_pages + (target - flagged_groups) - 1) / (target - flagged_groups)
                                                       : (total_pages + target - 1) / target;
        const long long room = max_items - flagged_groups;
        const long long need = (total_pages + room - 1) / room;
        if (want < need) want = need;
        ppi = (int)((want + kDenseWarps - 1) / kDenseWarps) * kDenseWarps;
        if (ppi < kMinPagesPerItem) ppi = kMinPagesPerItem;
    }
    {
        // exclusive scan of items per group: contiguous ranges per thread, then across threads
        const int per = (n_groups + kDenseThreads - 1) / kDenseThreads;
        const int lo = tid * per, hi = min(n_groups, lo + per);
        int mine = 0;
        for (int i = lo; i < hi; ++i) mine += (pages_of(i) + ppi - 1) / ppi;
        int incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(kFullMask, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) sm.misc[4 + warp] = incl;
        __syncthreads();
        int base = incl - mine;
        for (int w = 0; w < warp; ++w) base += sm.misc[4 + w];
        for (int i = lo; i < hi; ++i) {
            sm.item_base[i] = base;
            base += (pages_of(i) + ppi - 1) / ppi;
        }
        if (tid == kDenseThreads - 1) sm.item_base[n_groups] = base;
    }
    __syncthreads();
    const int n_items = sm.item_base[n_groups];

    const float scale = 1.4426950408889634f / epsilon;   // scores are kept in the log2 domain
    const int head = lane >> 2;                          // MMA row of this lane = query head in the group
    const int quad = lane & 3;
    uint8_t* my_ring = sm.ring + warp * Cfg::kWarpBytes;
    const uint32_t ring_addr = (uint32_t)__cvta_generic_to_shared(my_ring);
    // copy mapping: lane covers 16-byte chunk lane % CPR of rows lane / CPR + RPI i, i = 0 .. 16 / RPI - 1
    const int cp_chunk = lane % CPR, cp_row0 = lane / CPR;

    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        // group of this item: last g with item_base[g] <= item
        int glo = 0, ghi = n_groups;
        while (ghi - glo > 1) {
            const int mid = (glo + ghi) >> 1;
            if (sm.item_base[mid] <= item) glo = mid; else ghi = mid;
        }
        const int grp = glo;
        const uint32_t mask = sm.group_mask[grp];
        const int b = grp / geo.n_kv_heads, g = grp % geo.n_kv_heads;
        const int T = seq_lens[b];
        const int nb = (T + kUnit - 1) / kUnit;   // units (tiles of 16 tokens; fp8: pairs of tiles) of the sequence
        const int chunk = item - sm.item_base[grp];
        const int items_of_group = sm.item_base[grp + 1] - sm.item_base[grp];
        // the group's pages are split evenly over its items (whole multiples of the warp count)
        const int even = ((nb + items_of_group - 1) / items_of_group + kDenseWarps - 1) / kDenseWarps * kDenseWarps;
        const int first_page = min(nb, chunk * even);
        const int end_page = min(nb, first_page + even);
        const int32_t* bt = block_table + (long long)b * geo.max_pages;

        // Q fragments of the group: bf16 pairs straight from memory, rows >= G are zero
        uint32_t qa0[KS], qa2[KS];
        float q_unscale = 1.0f;
        if constexpr (FP8) {
            // q as e4m3 operands: scaled by a power of two into the top of the e4m3 range, split into hi + lo
            // (qa0 / qa2 hold, per 32-column step, {hi, lo} of columns 4 quad .. + 3 and of 16 + the same)
            const uint16_t* qrow = q + ((long long)b * geo.n_q_heads + g * G + (head < G ? head : 0)) * kHeadDim;
            float qv[4][8];
            float amax = 0.0f;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
                for (int part = 0; part < 2; ++part) {
                    const uint2 raw = *reinterpret_cast<const uint2*>(qrow + ks * 32 + part * 16 + quad * 4);
                    qv[ks][part * 4 + 0] = __uint_as_float(raw.x << 16);
                    qv[ks][part * 4 + 1] = __uint_as_float(raw.x & 0xffff0000u);
                    qv[ks][part * 4 + 2] = __uint_as_float(raw.y << 16);
                    qv[ks][part * 4 + 3] = __uint_as_float(raw.y & 0xffff0000u);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(qv[ks][i]));
            }
            amax = fmaxf(amax, __shfl_xor_sync(kFullMask, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(kFullMask, amax, 2));
            const int sq = amax > 0.0f ? 7 - ilogbf(amax) : 0;   // largest |q| of the head lands in [128, 256)
            q_unscale = ldexpf(1.0f, -sq);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint32_t h01, l01, h23, l23, h45, l45, h67, l67;
                split_e4m3x2(ldexpf(qv[ks][0], sq), ldexpf(qv[ks][1], sq), h01, l01);
                split_e4m3x2(ldexpf(qv[ks][2], sq), ldexpf(qv[ks][3], sq), h23, l23);
                split_e4m3x2(ldexpf(qv[ks][4], sq), ldexpf(qv[ks][5], sq), h45, l45);
                split_e4m3x2(ldexpf(qv[ks][6], sq), ldexpf(qv[ks][7], sq), h67, l67);
                const bool on = head < G;
                qa0[2 * ks] = on ? (h01 | (h23 << 16)) : 0u;       // hi: columns 4 quad .. + 3
                qa0[2 * ks + 1] = on ? (h45 | (h67 << 16)) : 0u;   // hi: columns 16 + 4 quad .. + 3
                qa2[2 * ks] = on ? (l01 | (l23 << 16)) : 0u;       // lo, likewise
                qa2[2 * ks + 1] = on ? (l45 | (l67 << 16)) : 0u;
            }
        } else {
            const uint16_t* qrow = q + ((long long)b * geo.n_q_heads + g * G + (head < G ? head : 0)) * kHeadDim;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const uint32_t v0 = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + quad * 2);
                const uint32_t v2 = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + quad * 2);
                qa0[ks] = head < G ? v0 : 0u;
                qa2[ks] = head < G ? v2 : 0u;
            }
        }
        float m_run = -INFINITY, l_run = 0.0f;   // per lane: head `head`, partial over this lane's columns
        float o[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) o[n][i] = 0.0f;

        // pages of this warp: first_page + warp, + 8, ...
        const int my_first = first_page + warp;
        const int my_count = my_first < end_page ? (end_page - my_first + kDenseWarps - 1) / kDenseWarps : 0;
        auto issue = [&](int k) {   // k-th unit of this warp into stage k % kStages
            const int pl = my_first + k * kDenseWarps;
            const uint32_t dst = ring_addr + (uint32_t)((k % kStages) * kStageBytes);
            if constexpr (FP8) {
                // 32 rows of 128 bytes per cache: lane covers 16-byte chunk lane % 8 of rows lane / 8 + 4 i; the two
                // halves of the unit are tiles 2 pl and 2 pl + 1 (one page, or two pages with their own scales)
                const int ch = lane & 7, r0 = lane >> 3;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int tile = 2 * pl + hf;
                    const int rows_here = min(kTileRows, T - tile * kTileRows);   // <= 0: the half lies past the sequence
                    long long phys = rows_here > 0 ? bt[tile >> geo.tile_shift] : -1;
                    const bool page_ok = phys >= 0 && phys < geo.pool_pages;
                    if (!page_ok) phys = 0;
                    const int valid_rows = page_ok ? rows_here : 0;
                    const long long off8 = phys * geo.page_stride + (long long)(g / geo.kv_div) * geo.head_stride + ch * 16 +
                                           (long long)((tile & ((1 << geo.tile_shift) - 1)) * kTileRows) * geo.token_stride;
                    const uint8_t* kp = reinterpret_cast<const uint8_t*>(k_cache) + off8;
                    const uint8_t* vp = reinterpret_cast<const uint8_t*>(v_cache) + off8;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int r = r0 + 4 * i, row = hf * 16 + r;
                        const uint32_t off = (uint32_t)(row * 128 + ((ch ^ (row & 7)) << 4));
                        const bool ok = r < valid_rows;
                        cp_async_16_zfill(dst + off, kp + (long long)r * geo.token_stride, ok);
                        cp_async_16_zfill(dst + Cfg::kRawBytes + off, vp + (long long)r * geo.token_stride, ok);
                    }
                    if (lane < 2) {   // the half's two scales ride the same stage: [k0, k1, v0, v1]
                        const float* sp = (lane == 0 ? k_scale : v_scale) + phys * geo.kv_heads_stored + g / geo.kv_div;
                        cp_async_4(dst + 2 * Cfg::kRawBytes + 8 * lane + 4 * hf, sp);
                    }
                }
            } else {
            long long phys = bt[pl >> geo.tile_shift];
            const bool page_ok = phys >= 0 && phys < geo.pool_pages;
            if (!page_ok) phys = 0;
            const int valid_rows = page_ok ? min(kTileRows, T - pl * kTileRows) : 0;
            const long long head_off = (long long)(g / geo.kv_div) * geo.head_stride + cp_chunk * 8 +
                                       (long long)((pl & ((1 << geo.tile_shift) - 1)) * kTileRows) * geo.token_stride;
            const uint16_t* kp = k_cache + phys * geo.page_stride + head_off;
            const uint16_t* vp = v_cache + phys * geo.page_stride + head_off;
#pragma unroll
            for (int i = 0; i < kTileRows / RPI; ++i) {
                const int r = cp_row0 + RPI * i;
                const uint32_t off = (uint32_t)(r * kRowBytes + ((cp_chunk ^ (r & 7)) << 4));
                const bool ok = r < valid_rows;
                cp_async_16_zfill(dst + off, kp + (long long)r * geo.token_stride, ok);
                cp_async_16_zfill(dst + kTileBytes + off, vp + (long long)r * geo.token_stride, ok);
            }
            }
        };
#pragma unroll
        for (int s = 0; s < kStages - 1; ++s) {
            if (s < my_count) issue(s);
            cp_async_commit();
        }
        for (int k = 0; k < my_count; ++k) {
            if (k + kStages - 1 < my_count) issue(k + kStages - 1);
            cp_async_commit();
            cp_async_wait<kStages - 1>();
            __syncwarp();
            if constexpr (FP8) {
            const int pl = my_first + k * kDenseWarps;
            const int valid = min(kUnit, T - pl * kUnit);   // > 0
            {
                // a page outside the pool: the group's listed heads fail
                const long long ph0 = bt[(2 * pl) >> geo.tile_shift];
                const long long ph1 = valid > kTileRows ? bt[(2 * pl + 1) >> geo.tile_shift] : ph0;
                if (ph0 < 0 || ph0 >= geo.pool_pages || ph1 < 0 || ph1 >= geo.pool_pages) {
                    if (lane == 0) sm.misc[13] = 1;   // (cleared at the end of the previous item)
                    __syncwarp();
                    continue;
                }
            }
            const uint32_t kbase = ring_addr + (uint32_t)((k % kStages) * kStageBytes);
            const uint32_t vbase = kbase + Cfg::kRawBytes;
            const float* scales = reinterpret_cast<const float*>(my_ring + (k % kStages) * kStageBytes + 2 * Cfg::kRawBytes);
            const float ks0 = scales[0], ks1 = scales[1], vs0 = scales[2], vs1 = scales[3];

            // S = Q K^T for the 32 tokens of the unit (four 8-token column tiles), q = hi + lo
            float sc4[4][4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int i = 0; i < 4; ++i) sc4[j][i] = 0.0f;
            {
                // ldmatrix.x4 on byte rows: matrix mi = lane / 8 is (tokens 8 (mi / 2) .. + 7) x (16-byte chunk 2 ks + mi % 2);
                // a lane receives 4 consecutive columns of one token: the B fragment of an m16n8k32 MMA
                const int mi = lane >> 3, rr = lane & 7;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const int tok = hf * 16 + (mi >> 1) * 8 + rr;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const int ch = 2 * ks + (mi & 1);
                        uint32_t r[4];
                        ldmatrix_x4(r, kbase + (uint32_t)(tok * 128 + ((ch ^ (tok & 7)) << 4)));
                        mma_e4m3(sc4[2 * hf], qa0[2 * ks], qa2[2 * ks], qa0[2 * ks + 1], qa2[2 * ks + 1], r[0], r[1]);
                        mma_e4m3(sc4[2 * hf + 1], qa0[2 * ks], qa2[2 * ks], qa0[2 * ks + 1], qa2[2 * ks + 1], r[2], r[3]);
                    }
                }
            }
            // this lane: head `head`, tokens 8 j + 2 quad, + 1 of column tile j = 0 .. 3
            float t[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float ts = scale * q_unscale * (j < 2 ? ks0 : ks1);   // the page's key scale folded in
                t[2 * j] = (8 * j + 2 * quad < valid) ? (sc4[j][0] + sc4[j][2]) * ts : -INFINITY;   // hi + lo rows
                t[2 * j + 1] = (8 * j + 2 * quad + 1 < valid) ? (sc4[j][1] + sc4[j][3]) * ts : -INFINITY;
            }
            float pm = fmaxf(fmaxf(fmaxf(t[0], t[1]), fmaxf(t[2], t[3])), fmaxf(fmaxf(t[4], t[5]), fmaxf(t[6], t[7])));
            pm = fmaxf(pm, __shfl_xor_sync(kFullMask, pm, 1));
            pm = fmaxf(pm, __shfl_xor_sync(kFullMask, pm, 2));
            const float m_new = fmaxf(m_run, pm);       // finite: token 0 of a unit is always valid
            const float corr = exp2f(m_run - m_new);    // 0 on the first unit
            float p[8], psum = 0.0f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                p[i] = exp2f(t[i] - m_new);
                psum += p[i];
            }
            l_run = fmaf(l_run, corr, psum);
            if (__any_sync(kFullMask, m_new > m_run)) {
#pragma unroll
                for (int n = 0; n < NT; ++n) {
                    o[n][0] *= corr;
                    o[n][1] *= corr;
                }
            }
            m_run = m_new;
            // P as e4m3 operands: p * (value scale of its page / the larger of the two scales) * 2^8 = hi + lo.
            // The 8 tokens of this lane take the lane's 8 slots of the contraction index: slots 4 quad .. + 3 are
            // tokens 2 quad, 2 quad + 1, 8 + 2 quad, 9 + 2 quad, slots 16 + 4 quad .. + 3 the same + 16; the V rows
            // are fetched in the matching order below.
            const float vref = fmaxf(vs0, vs1);
            const float w0 = vref > 0.0f ? 256.0f * (vs0 / vref) : 0.0f, w1 = vref > 0.0f ? 256.0f * (vs1 / vref) : 0.0f;
            uint32_t h01, l01, h23, l23, h45, l45, h67, l67;
            split_e4m3x2(p[0] * w0, p[1] * w0, h01, l01);
            split_e4m3x2(p[2] * w0, p[3] * w0, h23, l23);
            split_e4m3x2(p[4] * w1, p[5] * w1, h45, l45);
            split_e4m3x2(p[6] * w1, p[7] * w1, h67, l67);
            const uint32_t ph0 = h01 | (h23 << 16), ph2 = h45 | (h67 << 16), pl0 = l01 | (l23 << 16), pl2 = l45 | (l67 << 16);
            const float oscale = vref * (1.0f / 256.0f);

            // O += P V, 16 columns at a time: one transposing byte load per 32 tokens x 16 columns
            {
                const int rrow = lane & 15, qd = rrow >> 2, ii = rrow & 3;
                const int tokp = (lane >> 4) * 16 + ((ii < 2) ? 0 : 8) + 2 * qd + (ii & 1);
                const uint32_t vrow = vbase + (uint32_t)(tokp * 128);
#pragma unroll
                for (int dp = 0; dp < 8; ++dp) {
                    uint32_t r[4];
                    ldmatrix_x2_trans_b8(r, vrow + (uint32_t)((dp ^ (tokp & 7)) << 4));
                    float ta[4] = {0.f, 0.f, 0.f, 0.f}, tb[4] = {0.f, 0.f, 0.f, 0.f};
                    mma_e4m3(ta, ph0, pl0, ph2, pl2, r[0], r[2]);
                    mma_e4m3(tb, ph0, pl0, ph2, pl2, r[1], r[3]);
                    o[2 * dp][0] = fmaf(ta[0] + ta[2], oscale, o[2 * dp][0]);
                    o[2 * dp][1] = fmaf(ta[1] + ta[3], oscale, o[2 * dp][1]);
                    o[2 * dp + 1][0] = fmaf(tb[0] + tb[2], oscale, o[2 * dp + 1][0]);
                    o[2 * dp + 1][1] = fmaf(tb[1] + tb[3], oscale, o[2 * dp + 1][1]);
                }
            }
            } else {
            const int pl = my_first + k * kDenseWarps;
            const int valid = min(kTileRows, T - pl * kTileRows);   // > 0
            {
                const long long phys = bt[pl >> geo.tile_shift];   // a page outside the pool: the group's listed heads fail
                if (phys < 0 || phys >= geo.pool_pages) {
                    if (lane == 0) sm.misc[13] = 1;   // (cleared at the end of the previous item)
                    __syncwarp();
                    continue;
                }
            }
            const uint32_t kbase = ring_addr + (uint32_t)((k % kStages) * kStageBytes);
            const uint32_t vbase = kbase + kTileBytes;

            // S = Q K^T for the 16 tokens of the page (two 8-token column tiles)
            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
            {
                const int mi = lane >> 3, tok = (mi >> 1) * 8 + (lane & 7);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int ch = 2 * ks + (mi & 1);
                    uint32_t r[4];
                    ldmatrix_x4(r, kbase + (uint32_t)(tok * kRowBytes + ((ch ^ (tok & 7)) << 4)));
                    mma_bf16(s0, qa0[ks], qa2[ks], r[0], r[1]);
                    mma_bf16(s1, qa0[ks], qa2[ks], r[2], r[3]);
                }
            }
            // this lane: head `head`, tokens 2 quad, 2 quad + 1 (tile 0) and 8 + the same (tile 1)
            const float tscale = scale;
            float t[4];
            t[0] = (2 * quad < valid) ? s0[0] * tscale : -INFINITY;
            t[1] = (2 * quad + 1 < valid) ? s0[1] * tscale : -INFINITY;
            t[2] = (8 + 2 * quad < valid) ? s1[0] * tscale : -INFINITY;
            t[3] = (8 + 2 * quad + 1 < valid) ? s1[1] * tscale : -INFINITY;
            float pm = fmaxf(fmaxf(t[0], t[1]), fmaxf(t[2], t[3]));
            pm = fmaxf(pm, __shfl_xor_sync(kFullMask, pm, 1));
            pm = fmaxf(pm, __shfl_xor_sync(kFullMask, pm, 2));
            const float m_new = fmaxf(m_run, pm);       // finite: token 0 of a page is always valid
            const float corr = exp2f(m_run - m_new);    // 0 on the first page
            float p[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) p[i] = exp2f(t[i] - m_new);
            l_run = fmaf(l_run, corr, (p[0] + p[1]) + (p[2] + p[3]));
            if (__any_sync(kFullMask, m_new > m_run)) {
#pragma unroll
                for (int n = 0; n < NT; ++n) {
                    o[n][0] *= corr;
                    o[n][1] *= corr;
                }
            }
            m_run = m_new;
            const uint32_t pa0 = pack_bf16x2(p[0], p[1]), pa2 = pack_bf16x2(p[2], p[3]);

            // O += P V
            {
                const int mi = lane >> 3, tok = (mi & 1) * 8 + (lane & 7);
#pragma unroll
                for (int dp = 0; dp < KS; ++dp) {
                    const int ch = 2 * dp + (mi >> 1);
                    uint32_t r[4];
                    ldmatrix_x4_trans(r, vbase + (uint32_t)(tok * kRowBytes + ((ch ^ (tok & 7)) << 4)));
                    mma_bf16(o[2 * dp], pa0, pa2, r[0], r[1]);
                    mma_bf16(o[2 * dp + 1], pa0, pa2, r[2], r[3]);
                }
            }
            }
            __syncwarp();   // the stage is overwritten by a later issue
        }
        cp_async_wait<0>();

        // ---- merge: quad lanes share a head (sum l), then the warps, into one partial per head ----
        l_run += __shfl_xor_sync(kFullMask, l_run, 1);
        l_run += __shfl_xor_sync(kFullMask, l_run, 2);
        __syncthreads();   // every warp is done with its ring: reuse it for the merge
        float* mg = reinterpret_cast<float*>(sm.ring);   // [warps][G][2 + 128]
        if (head < G) {
            float* rec = mg + (warp * G + head) * kPartialFloats;
            if (quad == 0) {
                rec[0] = m_run;
                rec[1] = l_run;
            }
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                rec[2 + n * 8 + quad * 2] = o[n][0];
                rec[2 + n * 8 + quad * 2 + 1] = o[n][1];
            }
        }
        __syncthreads();
        for (int idx = tid; idx < G * kHeadDim; idx += kDenseThreads) {
            const int hh = idx / kHeadDim, e = idx % kHeadDim;
            if (!((mask >> hh) & 1u)) continue;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kDenseWarps; ++w) M = fmaxf(M, mg[(w * G + hh) * kPartialFloats]);
            float a = 0.0f, L = 0.0f;
#pragma unroll
            for (int w = 0; w < kDenseWarps; ++w) {
                const float* rec = mg + (w * G + hh) * kPartialFloats;
                const float f = rec[0] == -INFINITY ? 0.0f : exp2f(rec[0] - M);
                a = fmaf(rec[2 + e], f, a);
                L = fmaf(rec[1], f, L);
            }
            float* dst = partials + ((long long)item * G + hh) * kPartialFloats;
            dst[2 + e] = a;
            if (e == 0) {
                dst[0] = M;
                dst[1] = sm.misc[13] ? -1.0f : L;   // sums are never negative: -1 marks a page outside the pool
            }
        }

        // ---- the block that finishes the last item of this (sequence, KV head) combines them ----
        __threadfence();
        __syncthreads();
        if (tid == 0) sm.misc[12] = atomicAdd(&counters[grp], 1) == items_of_group - 1;
        __syncthreads();
        if (sm.misc[12]) {
            __threadfence();
            const float* gp = partials + (long long)sm.item_base[grp] * G * kPartialFloats;
            // Stage every item's (max, sum) of every head in shared memory first: the weighted sums below
            // then consist of independent loads only (a running maximum would make each load wait for the
            // previous item's, which costs a memory round trip per item).
            float* ms_s = reinterpret_cast<float*>(sm.ring);          // [items][G]
            float* ls_s = ms_s + (size_t)items_of_group * G;           // [items][G]
            for (int i = tid; i < items_of_group * G; i += kDenseThreads) {
                const float* rec = gp + (long long)i * kPartialFloats;
                ms_s[i] = __ldcg(rec);
                ls_s[i] = __ldcg(rec + 1);
            }
            __syncthreads();
            for (int idx = tid; idx < G * kHeadDim; idx += kDenseThreads) {
                const int hh = idx / kHeadDim, e = idx % kHeadDim;
                if (!((mask >> hh) & 1u)) continue;
                float M = -INFINITY;
                bool bad_page = false;
                for (int it = 0; it < items_of_group; ++it) {
                    M = fmaxf(M, ms_s[it * G + hh]);
                    bad_page |= ls_s[it * G + hh] < 0.0f;
                }
                const long long unit = (long long)b * geo.n_q_heads + g * G + hh;
                if (bad_page) {
                    // a block-table entry of the sequence is outside the pool: no dense result exists
                    out[unit * kHeadDim + e] = 0.0f;
                    if (e == 0 && diag) {
                        diag[unit].lse = 0.0f;
                        diag[unit].status = VSA_UNIT_BAD_PAGE;
                    }
                    continue;
                }
                // one pass in item order
                float acc = 0.0f, L = 0.0f;
#pragma unroll 8
                for (int it = 0; it < items_of_group; ++it) {
                    const float ms = ms_s[it * G + hh];
                    const float f = ms == -INFINITY ? 0.0f : exp2f(ms - M);
                    acc = fmaf(__ldcg(gp + ((long long)it * G + hh) * kPartialFloats + 2 + e), f, acc);
                    L = fmaf(ls_s[it * G + hh], f, L);
                }
                out[unit * kHeadDim + e] = L > 0.0f ? acc / L : 0.0f;
                if (e == 0 && diag) diag[unit].lse = (M + log2f(L)) * 0.6931471805599453f;
            }
        }
        if (tid == 0) sm.misc[13] = 0;
        __syncthreads();   // the ring (merge buffer) and misc are reused by the next item
    }
}

int num_sms() { return device_sm_count(); }

// room for the items the kernel may create: one ragged item per group plus the balancing target
int dense_max_items(const Geometry& g) { return g.batch * g.n_kv_heads + 2048; }

size_t dense_smem_bytes(const Geometry& g, bool fp8 = false)
{
    const size_t n_groups = (size_t)g.batch * g.n_kv_heads;
    const size_t ring = fp8 ? DenseCfg<128, true>::kRingBytes
                            : g.head_dim == 64 ? DenseCfg<64>::kRingBytes
                                               : (g.head_dim == 256 ? DenseCfg<256>::kRingBytes : DenseCfg<128>::kRingBytes);
    return ring + (n_groups + 1) * 4 + 16 * 4 + (n_groups + 15) / 16 * 16;
}

}  // namespace

static size_t dense_counter_bytes(const Geometry& g_in)
{
    const Geometry g = with_virtual_kv_heads(g_in);
    return (((size_t)g.batch * g.n_kv_heads * sizeof(int32_t)) + 255) / 256 * 256;
}

int32_t* dense_tickets(void* ws_dense) { return (int32_t*)ws_dense; }

int dense_ticket_count(const Geometry& g_in)
{
    const Geometry g = with_virtual_kv_heads(g_in);
    return g.batch * g.n_kv_heads;
}

size_t dense_workspace_bytes(const Geometry& g_in)
{
    const Geometry g = with_virtual_kv_heads(g_in);
    return dense_counter_bytes(g) + (size_t)dense_max_items(g) * g.group * (2 + g.head_dim) * sizeof(float);
}

template <int G, int D, bool FP8 = false>
static cudaError_t launch_dense_gd(const Geometry& g, const uint16_t* q, const uint16_t* k, const uint16_t* v,
                                   const int32_t* block_table, const int32_t* seq_lens, const int32_t* fallback_list,
                                   const int32_t* fallback_count, float epsilon, float* partials, int32_t* counters,
                                   float* out, vsa_diag_t* diag, cudaStream_t stream, const float* k_scale = nullptr,
                                   const float* v_scale = nullptr)
{
    const size_t smem = dense_smem_bytes(g, FP8);
    static bool attr_done[kMaxDevices] = {};   // per template instance
    const cudaError_t e = allow_large_dynamic_smem(dense_split_kernel<G, D, FP8>, attr_done);
    if (e != cudaSuccess) return e;
    // persistent grid: one block per SM (the ring fills the shared memory)
    return launch_pdl(dense_split_kernel<G, D, FP8>, dim3((unsigned)num_sms()), dim3(DenseCfg<D>::kDenseThreads), smem,
                      stream, g, q, k, v, block_table, seq_lens, fallback_list, fallback_count, epsilon, partials,
                      counters, out, diag, dense_max_items(g), k_scale, v_scale);
}

template <int G>
static cudaError_t launch_dense_g(const Geometry& g, const uint16_t* q, const uint16_t* k, const uint16_t* v,
                                  const int32_t* block_table, const int32_t* seq_lens, const int32_t* fallback_list,
                                  const int32_t* fallback_count, float epsilon, float* partials, int32_t* counters,
                                  float* out, vsa_diag_t* diag, cudaStream_t stream, const float* k_scale,
                                  const float* v_scale)
{
    if (k_scale)
        return launch_dense_gd<G, 128, true>(g, q, k, v, block_table, seq_lens, fallback_list, fallback_count, epsilon,
                                             partials, counters, out, diag, stream, k_scale, v_scale);
    if (g.head_dim == 64)
        return launch_dense_gd<G, 64>(g, q, k, v, block_table, seq_lens, fallback_list, fallback_count, epsilon,
                                      partials, counters, out, diag, stream);
    if (g.head_dim == 256)
        return launch_dense_gd<G, 256>(g, q, k, v, block_table, seq_lens, fallback_list, fallback_count, epsilon,
                                       partials, counters, out, diag, stream);
    return launch_dense_gd<G, 128>(g, q, k, v, block_table, seq_lens, fallback_list, fallback_count, epsilon, partials,
                                   counters, out, diag, stream);
}

cudaError_t launch_dense(const Geometry& g_in, const void* q, const void* k_cache, const void* v_cache,
                         const int32_t* block_table, const int32_t* seq_lens, const int32_t* fallback_list,
                         const int32_t* fallback_count, float epsilon, float* out, vsa_diag_t* diag, void* ws,
                         cudaStream_t stream, bool tickets_cleared, const float* k_scale, const float* v_scale)
{
    if ((k_scale || v_scale) && (!k_scale || !v_scale || g_in.head_dim != kHeadDim)) return cudaErrorInvalidValue;
    const Geometry g = with_virtual_kv_heads(g_in);
    int32_t* counters = (int32_t*)ws;
    float* partials = (float*)((char*)ws + dense_counter_bytes(g));
    if (!tickets_cleared) {
        cudaError_t e = cudaMemsetAsync(counters, 0, dense_counter_bytes(g), stream);
        if (e != cudaSuccess) return e;
    }
    const uint16_t *qq = (const uint16_t*)q, *kk = (const uint16_t*)k_cache, *vv = (const uint16_t*)v_cache;
    switch (g.group) {
        case 1: return launch_dense_g<1>(g, qq, kk, vv, block_table, seq_lens, fallback_list, fallback_count, epsilon, partials, counters, out, diag, stream, k_scale, v_scale);
        case 2: return launch_dense_g<2>(g, qq, kk, vv, block_table, seq_lens, fallback_list, fallback_count, epsilon, partials, counters, out, diag, stream, k_scale, v_scale);
        case 4: return launch_dense_g<4>(g, qq, kk, vv, block_table, seq_lens, fallback_list, fallback_count, epsilon, partials, counters, out, diag, stream, k_scale, v_scale);
        case 8: return launch_dense_g<8>(g, qq, kk, vv, block_table, seq_lens, fallback_list, fallback_count, epsilon, partials, counters, out, diag, stream, k_scale, v_scale);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace vsa
