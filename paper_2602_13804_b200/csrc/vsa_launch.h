// Host-side launch interface between the C ABI (api.cu) and the kernel files.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/vsa.h"

namespace vsa {

// Kernel launch with programmatic stream serialization allowed: the kernel may be scheduled
// before its predecessor in the stream has drained (it synchronises itself with pdl_wait()).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- per-device facts, looked up once per device ordinal ---------------------------------------------
constexpr int kMaxDevices = 64;

// ordinal of the current device when it can index the per-device tables below, else -1
inline int device_slot()
{
    int d = -1;
    if (cudaGetDevice(&d) != cudaSuccess) return -1;
    return (d >= 0 && d < kMaxDevices) ? d : -1;
}

// number of SMs of the current device (148 on a B200); 1 if the query fails
inline int device_sm_count()
{
    static int cached[kMaxDevices] = {};
    const int d = device_slot();
    if (d >= 0 && cached[d] > 0) return cached[d];
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        return 1;
    if (d >= 0) cached[d] = n;
    return n;
}

// Lets `kernel` request up to the device's opt-in maximum of dynamic shared memory (227 KB).  The attribute
// belongs to the (kernel, device) pair and is set on the first launch on each device: `done` is the
// caller's table for this kernel (a function-local static, one entry per device ordinal).
template <typename... KArgs>
inline cudaError_t allow_large_dynamic_smem(void (*kernel)(KArgs...), bool (&done)[kMaxDevices])
{
    const int d = device_slot();
    if (d >= 0 && done[d]) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess && d >= 0) done[d] = true;
    return e;
}

struct Geometry {
    int batch, n_q_heads, n_kv_heads, group, max_pages;
    long long pool_pages;
    long long page_stride, head_stride, token_stride;   // elements
    // Groups of more than 8 query heads per KV head (multi-query attention) reach the page scan and the
    // dense pass as "virtual" KV heads of 8 query heads each: there n_kv_heads and group describe the
    // virtual heads, virtual head g reads the cache of KV head g / kv_div, and kv_heads_stored is the
    // number of KV heads the pools and the summaries are laid out with.  Elsewhere kv_div = 1.
    int kv_div = 1;
    int kv_heads_stored = 0;
    // Non-zero (two-level routing, the scan over the super-pages' representatives): a "page" of this
    // geometry is a super-page of that many pages - lengths are still token counts of the sequence, and
    // logical super-page s of sequence b is stored at row b * max_pages + s (no block table).
    int super_pages = 0;
    // Tokens per page, 16 or 32.  The token-level kernels work on tiles of 16 rows; a page holds
    // 1 << tile_shift of them, and tile v of a sequence (tokens 16 v .. 16 v + 15) lies in logical page
    // v >> tile_shift at row offset 16 * (v & ((1 << tile_shift) - 1)).
    int page_size = 16;
    int tile_shift = 0;
    // Elements per head: 128, or 64 / 256 (closed-form step, routing, summaries and the dense pass only).
    int head_dim = 128;
    // pages a sequence of T tokens occupies / whether T is a length the block table can hold
    __host__ __device__ int pages_of(int T) const { return (T + page_size - 1) >> (4 + tile_shift); }
    __host__ __device__ bool length_ok(int T) const { return T > 0 && T <= max_pages * page_size; }
};

// the geometry the page scan and the dense pass work with (see kv_div above)
inline Geometry with_virtual_kv_heads(const Geometry& g)
{
    Geometry v = g;
    v.kv_heads_stored = g.n_kv_heads;
    if (g.group > 8) {
        v.kv_div = g.group / 8;
        v.group = 8;
        v.n_kv_heads = g.n_q_heads / 8;
    }
    return v;
}

// ---- page summaries -----------------------------------------------------------------------
cudaError_t launch_build_summaries(const Geometry& g, const void* k_cache, const int32_t* block_table,
                                   const int32_t* seq_lens, const int32_t* first_page, void* summaries,
                                   cudaStream_t stream);

cudaError_t launch_build_summaries_fp8(const Geometry& g, const void* k_cache, const float* k_scale,
                                       const int32_t* block_table, const int32_t* seq_lens,
                                       const int32_t* first_page, void* summaries, cudaStream_t stream);

cudaError_t launch_build_radii(const Geometry& g, const void* k_cache, const void* summaries,
                               const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_page,
                               float* radii, cudaStream_t stream);

cudaError_t launch_append(const Geometry& g, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                          const int32_t* block_table, const int32_t* seq_lens, void* summaries, float* radii,
                          cudaStream_t stream);

// ---- page routing ---------------------------------------------------------------------------
size_t route_workspace_bytes(const Geometry& g);
// zero_word (one int) and zero_words[0..zero_count) are cleared by the scan kernel when not null
// radii != nullptr: the pages' radii are also copied into logical page order, rad_logical[b][kv head][page]
cudaError_t launch_route_scan(const Geometry& g, const void* q, const void* summaries, const int32_t* block_table,
                              const int32_t* seq_lens, void* ws, int32_t* zero_word, int32_t* zero_words,
                              int zero_count, cudaStream_t stream, const float* radii = nullptr,
                              float* rad_logical = nullptr);
// page_budget (device, per unit, or nullptr): at most that many pages of a unit are routed (two-level
// routing: the pages that were scored; the rest of the unit's score row is -inf)
cudaError_t launch_route_select(const Geometry& g, const void* ws, const int32_t* seq_lens, int P,
                                int32_t* routed_pages, float* routed_scores, cudaStream_t stream,
                                const int32_t* page_budget = nullptr);

// ---- two-level routing (two_level.cu) -----------------------------------------------------------
int two_level_max_supers(const Geometry& g);
Geometry two_level_super_geometry(const Geometry& g);
cudaError_t launch_build_super_summaries(const Geometry& g, const void* summaries, const int32_t* block_table,
                                         const int32_t* seq_lens, const int32_t* first_super, void* super_summaries,
                                         int32_t* super_rep, cudaStream_t stream);
// selects the P_super best super-pages of every unit from super_scores (the representative scan's output)
// and writes the exact scores of the pages inside them (everything else -inf) and the number of scored
// pages per unit; super_routed_out (nullable) receives the kept super-pages
cudaError_t launch_inner_scan(const Geometry& g, const void* q, const void* summaries, const int32_t* block_table,
                              const int32_t* seq_lens, const float* super_scores, int P_super,
                              int32_t* super_routed_out, float* scores, int32_t* page_budget, cudaStream_t stream);

// ---- fused sparse pass ------------------------------------------------------------------------
// page_scores == nullptr: routed_pages is read; otherwise the top-P selection runs inside the kernel on
// page_scores (the scan's output) and routed_pages is written.  solve != nullptr: the weights on the
// candidates come from solver_iters iterations of entropic mirror descent (solver_kind 1) or of
// Frank-Wolfe with exact line search (solver_kind 2), K_c <= 256.  cert != nullptr
// (with page_scores and rad_logical): the certified gap is computed and decides the fallback.
// unit_list / unit_count (device): only the listed units are processed; routed_stride: row stride of
// routed_pages when it is wider than P (0 = P), the tail of a row is filled with -1.
cudaError_t launch_sparse(const Geometry& g, const void* q, const void* k_cache, const void* v_cache,
                          const int32_t* block_table, const int32_t* seq_lens, int32_t* routed_pages,
                          const float* page_scores, int P, int K_c, float epsilon, float gap_threshold, float* out,
                          vsa_diag_t* diag, int32_t* fallback_list, int32_t* fallback_count, cudaStream_t stream,
                          int solver_iters = 0, vsa_solve_t* solve = nullptr, const float* rad_logical = nullptr,
                          vsa_cert_t* cert = nullptr, int solver_kind = 1, const int32_t* unit_list = nullptr,
                          const int32_t* unit_count = nullptr, int routed_stride = 0,
                          const void* tl_summaries = nullptr, int P_super = 0, const float* k_scale = nullptr,
                          const float* v_scale = nullptr);
// k_scale / v_scale != nullptr: k_cache / v_cache hold e4m3 bytes, value = byte * scale[pool page][KV head]
// (closed-form family, head dimension 128).
// tl_summaries != nullptr: the two-level front end - page_scores then holds the scores of the super-pages'
// representatives, fp32 [batch][n_q_heads][two_level_max_supers], and the kernel keeps the P_super best
// super-pages, scores their pages from tl_summaries and routes the best P of those.
// ---- group-shared sparse pass (sparse_shared.cuh) -------------------------------------------------
// One thread block per (sequence, KV head); the group's heads share one page set and one candidate set
// selected on summed scores.  page_scores: the scan's per-head scores; routed_pages [batch][n_kv][P] out.
struct GroupSharedArgs {
    Geometry g;
    const uint16_t *q, *k, *v;
    const int32_t *block_table, *seq_lens;
    int32_t* routed_pages;
    const float* page_scores;
    int P, K_c;
    float epsilon, gap_threshold;
    float* out;
    vsa_diag_t* diag;
    int32_t *fallback_list, *fallback_count;
    cudaStream_t stream;
};
// native cache layout, groups of 1, 2, 4 or 8 heads, shared memory within the limit
bool sparse_shared_supported(const Geometry& g, int P);
cudaError_t launch_sparse_shared(const GroupSharedArgs& a);

// false when the kernel variant a launch would take needs more dynamic shared memory than a thread block
// can have (227 KB): wide block tables together with the iterative solve's key tile
bool sparse_shared_memory_fits(const Geometry& g, int P, int K_c, bool fused, bool solve, bool cert,
                               int P_super = 0);
// widest block table for which the fused kernel keeps every page score of a unit in registers (the
// certificate variant exists for those shapes only); `units` = batch * n_q_heads
int sparse_register_select_max_pages(long long units);

// ---- dense split-K pass -------------------------------------------------------------------------
size_t dense_workspace_bytes(const Geometry& g);
cudaError_t launch_dense(const Geometry& g, const void* q, const void* k_cache, const void* v_cache,
                         const int32_t* block_table, const int32_t* seq_lens, const int32_t* fallback_list,
                         const int32_t* fallback_count, float epsilon, float* out, vsa_diag_t* diag, void* ws,
                         cudaStream_t stream, bool tickets_cleared = false, const float* k_scale = nullptr,
                         const float* v_scale = nullptr);
// the per-(sequence, KV head) tickets at the start of the dense workspace, and how many there are
int32_t* dense_tickets(void* ws_dense);
int dense_ticket_count(const Geometry& g);

// ---- per-rank kernels of the context-parallel step (context_parallel.cu) ---------------------------
cudaError_t launch_cp_token_candidates(const Geometry& g, const void* q, const void* k_cache,
                                       const int32_t* block_table, const int32_t* seq_lens,
                                       const int32_t* routed_pages, int P, int K_out, int32_t* cand_pos,
                                       float* cand_score, cudaStream_t stream);
cudaError_t launch_cp_partial_readout(const Geometry& g, const void* v_cache, const int32_t* block_table,
                                      const int32_t* seq_lens, const int32_t* cand_pos, const float* cand_score,
                                      int K_c, float epsilon, float* out_partial, float* lse_partial,
                                      cudaStream_t stream);

}  // namespace vsa
