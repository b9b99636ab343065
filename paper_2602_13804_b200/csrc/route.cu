// Page routing (paper Sec. 7 step 1): score one summary row per page against every query head that
// reads its KV head, then keep the P best pages per query head.
//
//   route_scan_kernel    streams the summary rows (the only part of the step whose traffic grows
//                        with the context length) and writes all page scores to scratch.
//   route_select_kernel  one block per (sequence, query head): exact top-P selection.
#include <math.h>

#include <algorithm>

#include "vsa_device.cuh"
#include "vsa_launch.h"
#include "vsa_select.cuh"

namespace vsa {

namespace {

constexpr int kScanThreads = 256;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kBlockPages = 32;      // pages per block-table block (one coalesced 128-byte load per warp)
// Blocks of 32 pages one warp takes at most.  More per warp would amortise its start-up further, but
// the launch then has fewer, longer warps and a ragged batch (whose short sequences leave most of a
// grid sized for the longest one idle) ends on a long tail: 4 measured best from batch 16, T = 128k
// (87.7 against 93.6 us per layer with 16) to a 64-sequence log-uniform batch (455 against 482 us).
constexpr int kMaxBlocksPerWarp = 4;

template <int G, int D = kHeadDim>
struct ScanCfg {
    static constexpr int kRowBytes = 2 * D;               // one summary row
    static constexpr int ROWS = G == 1 ? 8 : 16 / G;      // rows per half-warp per round
    static constexpr int VALS = ROWS * G;                 // (row, head) partials per lane per round (8 or 16)
    static constexpr int ROUND_PAGES = 2 * ROWS;          // pages (rows of one KV head) per warp per round
    // ring slots per warp: a power of two (cheap slot index), about 8 KB of rows
    static constexpr int STAGES = 8192 / (ROUND_PAGES * kRowBytes) < 2 ? 2 : 8192 / (ROUND_PAGES * kRowBytes);
    static_assert((STAGES & (STAGES - 1)) == 0, "slot index is R & (STAGES - 1)");
    static constexpr int RING_BYTES = STAGES * ROUND_PAGES * kRowBytes;
    static constexpr int TAB_BYTES = kMaxBlocksPerWarp * kBlockPages * 4;
    static constexpr int RAD_BYTES = STAGES * ROUND_PAGES * 4;   // page radii of the rounds in flight (CERT)
    static constexpr int WARP_BYTES = RING_BYTES + TAB_BYTES + RAD_BYTES;
};

__device__ __forceinline__ void cp_async_16(uint32_t smem_addr, const void* gptr)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Warp w of the grid row of sequence b handles KV head (w % n_kv) and the 32-page blocks
// [slice * blocks_per_warp, (slice + 1) * blocks_per_warp), slice = w / n_kv, so the warps of a
// thread block read the summaries of all KV heads of the same pages (2 KB contiguous per page).
// Every lane streams its own 16-byte column of the rows through a private ring in shared memory
// with cp.async (several rounds in flight, no registers held by loads in flight, and no
// cross-thread synchronisation: a lane only ever reads back what it copied itself).  A half-warp
// covers one 256-byte row per copy instruction; the G query heads of the row's group share each
// unpacked element; 16 (row, head) partials are reduced at once.  For G >= 2 lane c takes the
// rows and the heads of a round in the order (r ^ c / G, h ^ c % G), which is what lets the
// reduction run without per-lane selects (reduce_scatter16_xor).
// CERT: the radius of every page (radii[page][kv head], see radii_kernel) is copied into logical page
// order, rad_logical[b][kv head][page], for the certificate that the fused kernel computes.
// D: head dimension (see sparse_kernel.cuh for how a row of 64 or 256 elements maps to the half-warp's lanes).
template <int G, bool CERT, int D = kHeadDim>
__global__ void __launch_bounds__(kScanThreads, 2)
route_scan_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ summaries,
                  const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_lens,
                  float* __restrict__ scores, int blocks_per_warp, int32_t* zero_word, int32_t* zero_words,
                  int zero_count, const float* __restrict__ radii, float* __restrict__ rad_logical)
{
    using Cfg = ScanCfg<G, D>;
    constexpr int ROWS = Cfg::ROWS, VALS = Cfg::VALS, ROUND_PAGES = Cfg::ROUND_PAGES, STAGES = Cfg::STAGES;
    constexpr int kRowBytes = Cfg::kRowBytes, PIECES = D == 256 ? 2 : 1;
    static_assert(D == 128 || ((D == 64 || D == 256) && !CERT), "certificate: head dimension 128 only");
    constexpr bool XOR_MAP = VALS == 16;
    // block-table blocks fetched before the sequence length is known: the warp's whole range
    constexpr int kFirstBlocks = kMaxBlocksPerWarp;
    extern __shared__ __align__(16) uint8_t scan_smem[];
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, c = lane & 15, gi = lane >> 4;
    const int w = blockIdx.x * (blockDim.x >> 5) + warp;
    const int g = w % geo.n_kv_heads;
    const int slice = w / geo.n_kv_heads;
    const int first_page = slice * blocks_per_warp * kBlockPages;
    const bool has_range = first_page < geo.max_pages;
    const int kr = XOR_MAP ? c / G : 0, kh = XOR_MAP ? c % G : 0;

    // The sequence length and the block-table entries of the first blocks of this warp's range are
    // fetched before the wait on the preceding kernel (they are scheduler state, not the product of a
    // kernel that signals early completion) so that their latency overlaps that kernel's tail.
    // Every index below max_pages is inside the table's row, whatever the sequence length is.
    const int32_t* bt = block_table + (long long)b * geo.max_pages + first_page;
    const int span = min(blocks_per_warp * kBlockPages, geo.max_pages - first_page);
    int T = 0;
    int first_entries[kFirstBlocks];
    if (has_range) {
        T = ld_ca_s32(seq_lens + b);
#pragma unroll
        for (int k = 0; k < kFirstBlocks; ++k) {
            const int i = k * kBlockPages + lane;
            first_entries[k] = i >= span ? -1 : geo.super_pages ? b * geo.max_pages + first_page + i : ld_ca_s32(bt + i);
        }
    }

    pdl_wait();                 // the score scratch may still be read by the previous step's kernels
    pdl_launch_dependents();

    // housekeeping for the kernels that follow in a step: clear the fallback counter and the
    // per-group tickets of the dense pass
    if (blockIdx.y == 0) {
        if (zero_word && blockIdx.x == 0 && threadIdx.x == 0) *zero_word = 0;
        if (zero_words)
            for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < zero_count; i += gridDim.x * blockDim.x)
                zero_words[i] = 0;
    }
    if (!has_range) return;

    const bool lane_has = D != 64 || c < 8;   // this lane holds a piece of every row
    uint4 qraw[G][PIECES];
#pragma unroll
    for (int hh = 0; hh < G; ++hh)
#pragma unroll
        for (int pc = 0; pc < PIECES; ++pc)
            qraw[hh][pc] = lane_has ? ld_nc_16B(q + ((long long)b * geo.n_q_heads + g * G + (hh ^ kh)) * D + pc * 128 + c * 8)
                                    : make_uint4(0u, 0u, 0u, 0u);

    if (geo.super_pages) {
        // the length in super-pages, expressed as a token count so that the page arithmetic below applies
        const int ns = (geo.pages_of(T) + geo.super_pages - 1) / geo.super_pages;
        T = (T > 0 && ns <= geo.max_pages) ? ns * geo.page_size : 0;
    }
    if (!geo.length_ok(T)) return;
    const int nb = geo.pages_of(T);
    if (first_page >= nb) return;
    const int n_pages = min(blocks_per_warp * kBlockPages, nb - first_page);
    const int n_blocks = (n_pages + kBlockPages - 1) / kBlockPages;
    const int n_rounds = (n_pages + ROUND_PAGES - 1) / ROUND_PAGES;

    uint8_t* my_smem = scan_smem + warp * Cfg::WARP_BYTES;
    // [n_blocks * 32] offset of the page's summary row in 16-byte units, -1 = no valid page
    int32_t* off_tab = (int32_t*)(my_smem + Cfg::RING_BYTES);
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(my_smem);
    const int page_units = geo.kv_heads_stored * (kRowBytes / 16);
    auto encode = [&](int p, int i) { return (i < n_pages && p >= 0 && p < geo.pool_pages) ? p * page_units : -1; };
#pragma unroll
    for (int k = 0; k < kFirstBlocks; ++k)
        if (k < n_blocks) off_tab[k * kBlockPages + lane] = encode(first_entries[k], k * kBlockPages + lane);
    float qf[G][PIECES][8];
#pragma unroll
    for (int hh = 0; hh < G; ++hh)
#pragma unroll
        for (int pc = 0; pc < PIECES; ++pc) unpack8(qraw[hh][pc], qf[hh][pc]);
    __syncwarp();

    const int g_stored = g / geo.kv_div;   // the KV head whose summaries this (possibly virtual) head reads
    const uint8_t* srow = reinterpret_cast<const uint8_t*>(summaries) + (long long)g_stored * kRowBytes + c * 16;
    const uint32_t lane_off = (uint32_t)(gi * ROWS * kRowBytes + c * 16);
    int tab_row[ROWS];   // the table entry of this lane's r-th row of a round
#pragma unroll
    for (int r = 0; r < ROWS; ++r) tab_row[r] = gi * ROWS + (r ^ kr);
    // after the reduction this lane owns (row own_r, head own_h) of its half-warp's ROWS rows
    const int own_r = VALS == 16 ? c / G : (c & 7) / G, own_h = c % G;
    const bool owns = VALS == 16 || c < 8;
    float* out_lane = scores + ((long long)b * geo.n_q_heads + g * G + own_h) * geo.max_pages + first_page +
                      gi * ROWS + own_r;
    // CERT: the lane that owns (row, head 0) also moves the row's radius
    const bool rad_lane = CERT && owns && own_h == 0;
    float* rad_ring = (float*)(my_smem + Cfg::RING_BYTES + Cfg::TAB_BYTES);
    const uint32_t rad_ring_s = (uint32_t)__cvta_generic_to_shared(rad_ring);
    float* rad_out = nullptr;
    if constexpr (CERT)
        rad_out = rad_logical + ((long long)b * geo.kv_heads_stored + g / geo.kv_div) * geo.max_pages + first_page +
                  gi * ROWS + own_r;

    // rows without a valid page read row 0 of the pool instead (their result is never stored)
    auto issue = [&](int R) {
        const uint32_t dst = ring + (uint32_t)((R & (STAGES - 1)) * ROUND_PAGES * kRowBytes) + lane_off;
        const int* tab = off_tab + R * ROUND_PAGES;
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const uint8_t* from = srow + (long long)max(tab[tab_row[r]], 0) * 16;
#pragma unroll
            for (int pc = 0; pc < PIECES; ++pc)
                if (lane_has) cp_async_16(dst + r * kRowBytes + pc * 256, from + pc * 256);
        }
        if constexpr (CERT) {
            if (rad_lane) {
                // off / 16 = page * n_kv_heads: the row of this page in radii[][n_kv_heads]
                const int off = max(tab[gi * ROWS + own_r], 0);
                cp_async_4(rad_ring_s + 4u * (uint32_t)((R & (STAGES - 1)) * ROUND_PAGES + gi * ROWS + own_r),
                           radii + (off >> 4) + g / geo.kv_div);
            }
        }
    };

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < n_rounds) issue(s);
        cp_async_commit();
    }
    for (int R = 0; R < n_rounds; ++R) {
        if (R + STAGES - 1 < n_rounds) issue(R + STAGES - 1);
        cp_async_commit();
        cp_async_wait<STAGES - 1>();   // this lane's copies of round R have landed
        const uint8_t* src = my_smem + (R & (STAGES - 1)) * ROUND_PAGES * kRowBytes + lane_off;
        float vals[16];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
#pragma unroll
            for (int pc = 0; pc < PIECES; ++pc) {
                const uint4 v = lane_has ? *reinterpret_cast<const uint4*>(src + r * kRowBytes + pc * 256)
                                         : make_uint4(0u, 0u, 0u, 0u);
                float kf[8];
                unpack8(v, kf);
#pragma unroll
                for (int hh = 0; hh < G; ++hh) {
                    const float part = chunk_partial(qf[hh][pc], kf);
                    vals[r * G + hh] = pc == 0 ? part : vals[r * G + hh] + part;
                }
            }
        }
        float s;
        if constexpr (XOR_MAP) {
            s = reduce_scatter16_xor(vals);
        } else {
#pragma unroll
            for (int i = VALS; i < 16; ++i) vals[i] = 0.0f;
            s = reduce_scatter16(vals, c);
        }
        const int pl = R * ROUND_PAGES + gi * ROWS + own_r;
        if (owns && pl < n_pages) out_lane[R * ROUND_PAGES] = off_tab[pl] >= 0 ? s : -INFINITY;
        if constexpr (CERT) {
            if (rad_lane && pl < n_pages)
                rad_out[R * ROUND_PAGES] =
                    off_tab[pl] >= 0 ? rad_ring[(R & (STAGES - 1)) * ROUND_PAGES + gi * ROWS + own_r] : 0.0f;
        }
    }
}

// Exact top-P of one unit's page scores, order (score descending, page ascending).
// KPT > 0: every thread keeps its KPT scores in registers (max_pages <= KPT * blockDim.x);
// KPT == 0: scores staged in shared memory, any size.
template <int KPT>
__global__ void route_select_kernel(Geometry geo, const float* __restrict__ scores,
                                    const int32_t* __restrict__ seq_lens, int P,
                                    int32_t* __restrict__ routed_pages, float* __restrict__ routed_scores,
                                    const int32_t* __restrict__ page_budget)
{
    extern __shared__ uint32_t smem[];
    pdl_wait();
    pdl_launch_dependents();
    const PageSelectSmem s = carve_page_select(smem, geo.max_pages, P);
    const int h = blockIdx.x, b = blockIdx.y;
    const long long unit = (long long)b * geo.n_q_heads + h;
    const int T = seq_lens[b];
    const bool ok = geo.length_ok(T);
    const int n = ok ? geo.pages_of(T) : 0;
    const int P_sel = page_budget ? min(P, __ldcg(page_budget + unit)) : P;   // scored pages only (two-level routing)
    int K;
    if constexpr (KPT > 0)
        K = select_top_pages_reg<KPT>(scores + unit * geo.max_pages, n, P_sel, s, page_budget != nullptr);
    else
        K = select_top_pages(scores + unit * geo.max_pages, n, P_sel, s, page_budget != nullptr);
    for (int t = threadIdx.x; t < P; t += blockDim.x) {
        routed_pages[unit * P + t] = t < K ? s.win_idx[t] : -1;
        if (routed_scores) routed_scores[unit * P + t] = t < K ? key_to_float(s.win_key[t]) : -INFINITY;
    }
}


size_t select_smem_bytes(const Geometry& g, int P) { return (size_t)select_pages_words(g.max_pages, P) * 4; }

int scan_blocks_per_warp(const Geometry& g)
{
    // 32-page blocks per warp: about one resident wave of warps (2 thread blocks of 8 warps per SM)
    // while that takes no more than kMaxBlocksPerWarp
    const long long blocks = (long long)g.batch * g.n_kv_heads * ((g.max_pages + kBlockPages - 1) / kBlockPages);
    const long long resident_warps = 2LL * kScanWarps * device_sm_count();
    long long k = (blocks + resident_warps - 1) / resident_warps;
    if (k < 1) k = 1;
    if (k > kMaxBlocksPerWarp) k = kMaxBlocksPerWarp;
    return (int)k;
}

// Warps per thread block (8 at most).  When the whole launch is resident at once (two blocks per SM)
// the busiest SM sets the time, so smaller blocks that spread the warps over more SMs
// win: the 64 warps of one 4k-token sequence run as 64 blocks of one warp instead of 8 blocks of 8
// (0.6 us per layer at batch 1); 2048 warps as 296 blocks of 7 instead of 256 of 8.
int scan_warps_per_block(int warps_per_seq, int batch)
{
    const int sms = device_sm_count();
    int best = kScanWarps, best_load = 1 << 30;
    for (int wpb = kScanWarps; wpb >= 1; --wpb) {
        const long long blocks = (long long)batch * ((warps_per_seq + wpb - 1) / wpb);
        if (blocks > 2 * sms) continue;
        const int load = blocks <= sms ? wpb : 2 * wpb;   // warps on the busiest SM
        if (load < best_load) best = wpb, best_load = load;
    }
    return best;
}

template <int G, bool CERT, int D = kHeadDim>
cudaError_t launch_scan_g(const Geometry& g, const uint16_t* q, const uint16_t* summaries, const int32_t* block_table,
                          const int32_t* seq_lens, float* scores, int32_t* zero_word, int32_t* zero_words,
                          int zero_count, const float* radii, float* rad_logical, cudaStream_t stream)
{
    const int bpw = scan_blocks_per_warp(g);
    const int slices = ((g.max_pages + kBlockPages - 1) / kBlockPages + bpw - 1) / bpw;
    const int warps = slices * g.n_kv_heads;
    const int wpb = scan_warps_per_block(warps, g.batch);
    const dim3 grid((unsigned)((warps + wpb - 1) / wpb), (unsigned)g.batch);
    // The request is padded to 81 KB so that exactly two blocks are resident per SM: with a third one
    // fewer blocks of the kernel that follows fit beside the scan's to start early, and the step gets
    // slower although the scan does not (measured: 30.0 against 24.8 us per layer at batch 8, T = 32k).
    const size_t smem = std::max((size_t)kScanWarps * ScanCfg<G, D>::WARP_BYTES, (size_t)81 * 1024);
    static bool attr_done[kMaxDevices] = {};   // per template instance
    const cudaError_t e = allow_large_dynamic_smem(route_scan_kernel<G, CERT, D>, attr_done);
    if (e != cudaSuccess) return e;
    return launch_pdl(route_scan_kernel<G, CERT, D>, grid, dim3(wpb * 32), smem, stream, g, q, summaries,
                      block_table, seq_lens, scores, bpw, zero_word, zero_words, zero_count, radii, rad_logical);
}

}  // namespace

size_t route_workspace_bytes(const Geometry& g)
{
    return (size_t)g.batch * g.n_q_heads * g.max_pages * sizeof(float);
}

cudaError_t launch_route_scan(const Geometry& g_in, const void* q, const void* summaries, const int32_t* block_table,
                              const int32_t* seq_lens, void* ws, int32_t* zero_word, int32_t* zero_words,
                              int zero_count, cudaStream_t stream, const float* radii, float* rad_logical)
{
    const Geometry g = with_virtual_kv_heads(g_in);
    float* scores = (float*)ws;
    const uint16_t* qq = (const uint16_t*)q;
    const uint16_t* ss = (const uint16_t*)summaries;
#define VSA_SCAN_CASE(G)                                                                                       \
    case G:                                                                                                    \
        if (g.head_dim == 64)                                                                                  \
            return launch_scan_g<G, false, 64>(g, qq, ss, block_table, seq_lens, scores, zero_word, zero_words, \
                                               zero_count, nullptr, nullptr, stream);                          \
        if (g.head_dim == 256)                                                                                 \
            return launch_scan_g<G, false, 256>(g, qq, ss, block_table, seq_lens, scores, zero_word, zero_words, \
                                                zero_count, nullptr, nullptr, stream);                         \
        return radii ? launch_scan_g<G, true>(g, qq, ss, block_table, seq_lens, scores, zero_word, zero_words, \
                                              zero_count, radii, rad_logical, stream)                          \
                     : launch_scan_g<G, false>(g, qq, ss, block_table, seq_lens, scores, zero_word, zero_words, \
                                               zero_count, nullptr, nullptr, stream);
    if (g.head_dim != kHeadDim && radii) return cudaErrorInvalidValue;   // (refused by the entry points)
    switch (g.group) {
        VSA_SCAN_CASE(1)
        VSA_SCAN_CASE(2)
        VSA_SCAN_CASE(4)
        VSA_SCAN_CASE(8)
        default: return cudaErrorInvalidValue;
    }
#undef VSA_SCAN_CASE
}

cudaError_t launch_route_select(const Geometry& g, const void* ws, const int32_t* seq_lens, int P,
                                int32_t* routed_pages, float* routed_scores, cudaStream_t stream,
                                const int32_t* page_budget)
{
    const size_t smem = select_smem_bytes(g, P);
    const dim3 grid((unsigned)g.n_q_heads, (unsigned)g.batch);
#define VSA_SELECT_LAUNCH(KPT, THREADS)                                                                          \
    {                                                                                                            \
        static bool attr_done[kMaxDevices] = {};                                                                 \
        if (smem > 48 * 1024) {                                                                                  \
            const cudaError_t e = allow_large_dynamic_smem(route_select_kernel<KPT>, attr_done);                 \
            if (e != cudaSuccess) return e;                                                                      \
        }                                                                                                        \
        cudaError_t e2 = launch_pdl(route_select_kernel<KPT>, grid, dim3(THREADS), smem, stream, g,            \
                                    (const float*)ws, seq_lens, P, routed_pages, routed_scores, page_budget);  \
        if (e2 != cudaSuccess) return e2;                                                                       \
    }
    if (g.max_pages <= 2048) VSA_SELECT_LAUNCH(8, 256)
    else if (g.max_pages <= 4096) VSA_SELECT_LAUNCH(16, 256)
    else if (g.max_pages <= 8192) VSA_SELECT_LAUNCH(32, 256)
    else VSA_SELECT_LAUNCH(0, 512)
#undef VSA_SELECT_LAUNCH
    return cudaGetLastError();
}

}  // namespace vsa
