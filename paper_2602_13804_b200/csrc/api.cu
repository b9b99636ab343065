// C ABI of libvsa: argument validation (everything is checked on the host before any launch),
// workspace layout, and the composition of the kernels into the entry points of vsa.h.
#include <math.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"

namespace {

using vsa::Geometry;

constexpr int kMaxP = 128;
constexpr int kMaxPagesPerSeq = 32768;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// device-side address of a page-locked (pinned or registered) host buffer, NULL for anything else
const void* mapped_device_pointer(const void* host)
{
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    if (attr.type != cudaMemoryTypeHost || !attr.devicePointer) return nullptr;
    return attr.devicePointer;
}

// Brings the step's queries from page-locked host memory into the device staging buffer with plain
// 16-byte loads across the bus: one short kernel in the stream's launch chain instead of a copy
// operation, which would serialise fully against the kernels before and after it.
__global__ void fetch_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int n16)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (i < n16) v = vsa::ld_nc_16B(src + i);   // host memory is stable: fetched before the wait
    vsa::pdl_wait();                            // the previous step's kernels may still read dst
    vsa::pdl_launch_dependents();
    if (i < n16) dst[i] = v;
}

// shape checks shared by every entry point; fills the kernel-side geometry
int make_geometry(const vsa_shape_t* s, Geometry* g)
{
    if (!s) return VSA_ERR_INVALID_ARGUMENT;
    if (s->batch <= 0 || s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->head_dim <= 0 || s->page_size <= 0 ||
        s->max_pages_per_seq <= 0 || s->num_pool_pages <= 0)
        return VSA_ERR_INVALID_ARGUMENT;
    if (s->n_q_heads % s->n_kv_heads != 0) return VSA_ERR_INVALID_ARGUMENT;
    if (s->kv_page_stride < 0 || s->kv_head_stride < 0 || s->kv_token_stride < 0) return VSA_ERR_INVALID_ARGUMENT;
    const int group = s->n_q_heads / s->n_kv_heads;
    if ((s->head_dim != 64 && s->head_dim != 128 && s->head_dim != 256) || (s->page_size != 16 && s->page_size != 32))
        return VSA_ERR_UNSUPPORTED_SHAPE;
    if (group != 1 && group != 2 && group != 4 && group != 8 && group != 16 && group != 32)
        return VSA_ERR_UNSUPPORTED_SHAPE;
    if (s->max_pages_per_seq > kMaxPagesPerSeq) return VSA_ERR_UNSUPPORTED_SHAPE;
    if (s->num_pool_pages > 0x7fffffffLL) return VSA_ERR_UNSUPPORTED_SHAPE;
    if ((long long)s->batch * s->n_q_heads > 0x3fffffffLL) return VSA_ERR_UNSUPPORTED_SHAPE;
    // (sequence, KV head) pairs the dense pass tracks; groups above 8 count as n_q_heads / 8 heads there
    if ((long long)s->batch * (group > 8 ? s->n_q_heads / 8 : s->n_kv_heads) > 4096) return VSA_ERR_UNSUPPORTED_SHAPE;
    // (the summary pool is addressed in 16-byte units by a 32-bit offset: 2^27 rows of 256 bytes)
    if (s->num_pool_pages * s->n_kv_heads * (s->head_dim / 8) >= (1LL << 31)) return VSA_ERR_UNSUPPORTED_SHAPE;
    g->batch = s->batch;
    g->n_q_heads = s->n_q_heads;
    g->n_kv_heads = s->n_kv_heads;
    g->group = group;
    g->kv_div = 1;
    g->kv_heads_stored = s->n_kv_heads;
    g->max_pages = s->max_pages_per_seq;
    g->page_size = s->page_size;
    g->head_dim = s->head_dim;
    g->tile_shift = s->page_size == 32 ? 1 : 0;
    g->super_pages = 0;
    g->pool_pages = s->num_pool_pages;
    g->token_stride = s->kv_token_stride ? s->kv_token_stride : s->head_dim;
    g->head_stride = s->kv_head_stride ? s->kv_head_stride : (long long)s->page_size * g->token_stride;
    g->page_stride = s->kv_page_stride ? s->kv_page_stride : (long long)s->n_kv_heads * g->head_stride;
    if (g->token_stride < s->head_dim) return VSA_ERR_INVALID_ARGUMENT;
    if ((g->token_stride % 8) || (g->head_stride % 8) || (g->page_stride % 8)) return VSA_ERR_MISALIGNED;
    return VSA_OK;
}

// an fp8 cache: head dimension 128, rows copied in 16-byte pieces (strides are in bytes there)
int check_fp8_cache(const Geometry& g, const void* k_scale, const void* v_scale)
{
    if (!k_scale || !v_scale) return VSA_ERR_INVALID_ARGUMENT;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;
    if ((g.token_stride % 16) || (g.head_stride % 16) || (g.page_stride % 16)) return VSA_ERR_MISALIGNED;
    return VSA_OK;
}

int check_routing_sizes(const Geometry& g, int P, int K_c, bool need_kc)
{
    if (P < 1) return VSA_ERR_INVALID_ARGUMENT;
    if (P > kMaxP) return VSA_ERR_UNSUPPORTED_SHAPE;
    if (need_kc) {
        if (K_c < 1) return VSA_ERR_INVALID_ARGUMENT;
        if (K_c > P * g.page_size) return VSA_ERR_UNSUPPORTED_SHAPE;
        if (P * g.page_size > kMaxP * 16) return VSA_ERR_UNSUPPORTED_SHAPE;   // candidate tokens before the top-K_c
    }
    return VSA_OK;
}

int check_solver_sizes(int K_c, int solver_iters)
{
    if (solver_iters < 0 || solver_iters > VSA_SOLVER_MAX_ITERS) return VSA_ERR_INVALID_ARGUMENT;
    if (K_c > VSA_SOLVER_MAX_CANDIDATES) return VSA_ERR_UNSUPPORTED_SHAPE;
    return VSA_OK;
}

int check_epsilon(float epsilon)
{
    if (!(epsilon > 0.0f) || isinf(epsilon)) return VSA_ERR_INVALID_ARGUMENT;
    return VSA_OK;
}

// step workspace = [ route scores | dense scratch ], each part 256-byte aligned
size_t step_route_part(const Geometry& g) { return align_up(vsa::route_workspace_bytes(g), 256); }

// certified step: [ route scores | dense scratch | page radii in logical order, fp32 [batch][n_kv_heads][max_pages] ]
size_t step_rad_offset(const Geometry& g) { return step_route_part(g) + align_up(vsa::dense_workspace_bytes(g), 256); }
size_t step_rad_bytes(const Geometry& g) { return (size_t)g.batch * g.n_kv_heads * g.max_pages * sizeof(float); }

// expanding step: the certified layout followed by the retry lists - kMaxExpandRounds counters, then one
// list of one int per unit for every round (P doubles per round and P <= 128, so seven rounds at most)
constexpr int kMaxExpandRounds = 8;
size_t step_retry_offset(const Geometry& g) { return align_up(step_rad_offset(g) + step_rad_bytes(g), 256); }
size_t step_retry_bytes(const Geometry& g)
{
    return ((size_t)kMaxExpandRounds * ((size_t)g.batch * g.n_q_heads + 1)) * sizeof(int32_t);
}

int cuda_rc(cudaError_t e) { return e == cudaSuccess ? VSA_OK : VSA_ERR_CUDA; }

// two-level routing scratch: [ page scores | representative scores | scored pages per unit ], each part
// 256-byte aligned; the step adds the dense scratch
struct TwoLevelWs {
    size_t super_scores, budget, dense, total_route;
};
TwoLevelWs two_level_layout(const Geometry& g)
{
    const Geometry gs = vsa::two_level_super_geometry(g);
    TwoLevelWs w;
    size_t o = step_route_part(g);
    w.super_scores = o;
    o += align_up(vsa::route_workspace_bytes(gs), 256);
    w.budget = o;
    o += align_up((size_t)g.batch * g.n_q_heads * sizeof(int32_t), 256);
    w.dense = o;
    w.total_route = o;
    return w;
}

// representative scan -> per unit: top-P_super super-pages and the exact scores inside them (into the
// page-score scratch at the start of ws).  zero_word / tickets: cleared by the representative scan.
int two_level_scores(const Geometry& g, const void* q, const void* summaries, const void* super_summaries,
                     const int32_t* block_table, const int32_t* seq_lens, int P_super, int32_t* super_routed_out,
                     void* ws, int32_t* zero_word, int32_t* zero_words, int zero_count, cudaStream_t st)
{
    const TwoLevelWs w = two_level_layout(g);
    const Geometry gs = vsa::two_level_super_geometry(g);
    char* base = (char*)ws;
    // (the block-table argument is not read in a geometry whose pages are super-pages)
    if (vsa::launch_route_scan(gs, q, super_summaries, block_table, seq_lens, base + w.super_scores, zero_word,
                               zero_words, zero_count, st) != cudaSuccess)
        return VSA_ERR_CUDA;
    return cuda_rc(vsa::launch_inner_scan(g, q, summaries, block_table, seq_lens, (const float*)(base + w.super_scores),
                                          P_super, super_routed_out, (float*)ws, (int32_t*)(base + w.budget), st));
}

}  // namespace

extern "C" {

const char* vsa_strerror(int code)
{
    switch (code) {
        case VSA_OK: return "ok";
        case VSA_ERR_INVALID_ARGUMENT: return "invalid argument";
        case VSA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case VSA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case VSA_ERR_MISALIGNED: return "pointer or stride not 16-byte aligned";
        case VSA_ERR_CUDA: return "CUDA runtime error";
        case VSA_ERR_STATIC_SCRATCH_EXCEEDED:
            return "shape exceeds the built-in scratch array (batch * n_q_heads * max_pages_per_seq > 2^20)";
        default: return "unknown error code";
    }
}

size_t vsa_workspace_bytes(const vsa_shape_t* shape, int32_t P, int32_t K_c, int which_call)
{
    Geometry g;
    if (make_geometry(shape, &g) != VSA_OK) return 0;
    (void)K_c;
    switch (which_call) {
        case VSA_WS_ROUTE: return vsa::route_workspace_bytes(g);
        case VSA_WS_SPARSE: return 0;
        case VSA_WS_DENSE: return vsa::dense_workspace_bytes(g);
        case VSA_WS_STEP: return step_route_part(g) + vsa::dense_workspace_bytes(g);
        case VSA_WS_STEP_CERTIFIED: return step_rad_offset(g) + step_rad_bytes(g);
        case VSA_WS_STEP_EXPAND: return step_retry_offset(g) + step_retry_bytes(g);
        // (for the two-level kinds the P argument is P_super, the number of super-pages kept per unit)
        case VSA_WS_ROUTE_TWO_LEVEL: return P >= 1 ? two_level_layout(g).total_route : 0;
        case VSA_WS_STEP_TWO_LEVEL: return P >= 1 ? two_level_layout(g).dense + vsa::dense_workspace_bytes(g) : 0;
        default: return 0;
    }
}

int vsa_build_page_summaries(const vsa_shape_t* shape, const void* k_cache, const int32_t* block_table,
                             const int32_t* seq_lens, const int32_t* first_page, void* summaries, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (!k_cache || !block_table || !seq_lens || !summaries) return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(k_cache) || !aligned16(summaries)) return VSA_ERR_MISALIGNED;
    return cuda_rc(vsa::launch_build_summaries(g, k_cache, block_table, seq_lens, first_page, summaries,
                                               (cudaStream_t)stream));
}

int vsa_build_page_summaries_fp8(const vsa_shape_t* shape, const void* k_cache, const float* k_scale,
                                 const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_page,
                                 void* summaries, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (!k_cache || !k_scale || !block_table || !seq_lens || !summaries) return VSA_ERR_INVALID_ARGUMENT;
    if ((rc = check_fp8_cache(g, k_scale, k_scale))) return rc;
    if (!aligned16(k_cache) || !aligned16(summaries)) return VSA_ERR_MISALIGNED;
    return cuda_rc(vsa::launch_build_summaries_fp8(g, k_cache, k_scale, block_table, seq_lens, first_page, summaries,
                                                   (cudaStream_t)stream));
}

int vsa_build_page_radii(const vsa_shape_t* shape, const void* k_cache, const void* summaries,
                         const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_page,
                         float* radii, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;   // this entry point: head_dim 128 only
    if (!k_cache || !summaries || !block_table || !seq_lens || !radii) return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(k_cache) || !aligned16(summaries)) return VSA_ERR_MISALIGNED;
    return cuda_rc(vsa::launch_build_radii(g, k_cache, summaries, block_table, seq_lens, first_page, radii,
                                           (cudaStream_t)stream));
}

int vsa_append_kv(const vsa_shape_t* shape, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                  const int32_t* block_table, const int32_t* seq_lens, void* summaries, float* radii, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;   // this entry point: head_dim 128 only
    if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !seq_lens || !summaries)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(summaries))
        return VSA_ERR_MISALIGNED;
    return cuda_rc(vsa::launch_append(g, k_new, v_new, k_cache, v_cache, block_table, seq_lens, summaries, radii,
                                      (cudaStream_t)stream));
}

int vsa_route_pages(const vsa_shape_t* shape, const void* q, const void* summaries, const int32_t* block_table,
                    const int32_t* seq_lens, int32_t P, int32_t* routed_pages, float* routed_scores, void* ws,
                    size_t ws_bytes, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if ((rc = check_routing_sizes(g, P, 0, false))) return rc;
    if (!q || !summaries || !block_table || !seq_lens || !routed_pages || !ws) return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(summaries) || !aligned16(ws)) return VSA_ERR_MISALIGNED;
    if (ws_bytes < vsa::route_workspace_bytes(g)) return VSA_ERR_WORKSPACE_TOO_SMALL;
    cudaError_t e = vsa::launch_route_scan(g, q, summaries, block_table, seq_lens, ws, nullptr, nullptr, 0,
                                           (cudaStream_t)stream);
    if (e != cudaSuccess) return VSA_ERR_CUDA;
    return cuda_rc(vsa::launch_route_select(g, ws, seq_lens, P, routed_pages, routed_scores, (cudaStream_t)stream));
}

int vsa_build_super_summaries(const vsa_shape_t* shape, const void* summaries, const int32_t* block_table,
                              const int32_t* seq_lens, const int32_t* first_super, void* super_summaries,
                              int32_t* super_rep, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;   // this entry point: head_dim 128 only
    if (!summaries || !block_table || !seq_lens || !super_summaries) return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(summaries) || !aligned16(super_summaries)) return VSA_ERR_MISALIGNED;
    return cuda_rc(vsa::launch_build_super_summaries(g, summaries, block_table, seq_lens, first_super,
                                                     super_summaries, super_rep, (cudaStream_t)stream));
}

int vsa_route_pages_two_level(const vsa_shape_t* shape, const void* q, const void* summaries,
                              const void* super_summaries, const int32_t* block_table, const int32_t* seq_lens,
                              int32_t P_super, int32_t P, int32_t* routed_pages, float* routed_scores,
                              int32_t* super_routed, void* ws, size_t ws_bytes, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;   // this entry point: head_dim 128 only
    if ((rc = check_routing_sizes(g, P, 0, false))) return rc;
    if ((rc = check_routing_sizes(g, P_super, 0, false))) return rc;
    if (!q || !summaries || !super_summaries || !block_table || !seq_lens || !routed_pages || !ws)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(summaries) || !aligned16(super_summaries) || !aligned16(ws))
        return VSA_ERR_MISALIGNED;
    if (ws_bytes < two_level_layout(g).total_route) return VSA_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    if ((rc = two_level_scores(g, q, summaries, super_summaries, block_table, seq_lens, P_super, super_routed, ws,
                               nullptr, nullptr, 0, st)))
        return rc;
    return cuda_rc(vsa::launch_route_select(g, ws, seq_lens, P, routed_pages, routed_scores, st,
                                            (const int32_t*)((char*)ws + two_level_layout(g).budget)));
}

int vsa_decode_step_two_level(const vsa_shape_t* shape, const void* q, const void* summaries,
                              const void* super_summaries, const void* k_cache, const void* v_cache,
                              const int32_t* block_table, const int32_t* seq_lens, int32_t P_super, int32_t P,
                              int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                              int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                              size_t ws_bytes, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;   // this entry point: head_dim 128 only
    if ((rc = check_routing_sizes(g, P, K_c, true))) return rc;
    if ((rc = check_routing_sizes(g, P_super, 0, false))) return rc;
    if ((rc = check_epsilon(epsilon))) return rc;
    if (isnan(gap_threshold)) return VSA_ERR_INVALID_ARGUMENT;
    if (!q || !summaries || !super_summaries || !k_cache || !v_cache || !block_table || !seq_lens || !out || !diag ||
        !routed_pages || !fallback_list || !fallback_count || !ws)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(summaries) || !aligned16(super_summaries) || !aligned16(k_cache) ||
        !aligned16(v_cache) || !aligned16(ws))
        return VSA_ERR_MISALIGNED;
    const TwoLevelWs w = two_level_layout(g);
    if (ws_bytes < w.dense + vsa::dense_workspace_bytes(g)) return VSA_ERR_WORKSPACE_TOO_SMALL;
    if (!vsa::sparse_shared_memory_fits(g, P, K_c, true, false, false, P_super)) return VSA_ERR_UNSUPPORTED_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    void* ws_dense = (char*)ws + w.dense;
    // Every super-page of every sequence would be kept: the routing is the exact one, which the full scan
    // computes with less work per unit (same routed pages, same order)
    if (vsa::two_level_max_supers(g) <= P_super) {
        if (ws_bytes < step_route_part(g) + vsa::dense_workspace_bytes(g)) return VSA_ERR_WORKSPACE_TOO_SMALL;
        return vsa_decode_step(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                               gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws, ws_bytes,
                               stream);
    }
    // Three launches: the scan over the representatives (1/16 of the full scan's rows; it also clears the
    // fallback counter and the dense tickets), the fused kernel whose front end keeps the P_super best
    // super-pages of its unit, scores their pages exactly and routes the best P, and the dense pass.
    const Geometry gs = vsa::two_level_super_geometry(g);
    const float* super_scores = (const float*)((char*)ws + w.super_scores);
    if (vsa::launch_route_scan(gs, q, super_summaries, block_table, seq_lens, (void*)super_scores, fallback_count,
                               vsa::dense_tickets(ws_dense), vsa::dense_ticket_count(g), st) != cudaSuccess)
        return VSA_ERR_CUDA;
    cudaError_t e = vsa::launch_sparse(g, q, k_cache, v_cache, block_table, seq_lens, routed_pages, super_scores, P,
                                       K_c, epsilon, gap_threshold, out, diag, fallback_list, fallback_count, st, 0,
                                       nullptr, nullptr, nullptr, 1, nullptr, nullptr, 0, summaries, P_super);
    if (e != cudaSuccess) return VSA_ERR_CUDA;
    return cuda_rc(vsa::launch_dense(g, q, k_cache, v_cache, block_table, seq_lens, fallback_list, fallback_count,
                                     epsilon, out, diag, ws_dense, st, /*tickets_cleared=*/true));
}

static int sparse_decode_impl(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                              const float* k_scale, const float* v_scale, bool fp8, const int32_t* block_table,
                              const int32_t* seq_lens, const int32_t* routed_pages, int32_t P, int32_t K_c,
                              float epsilon, float gap_threshold, float* out, vsa_diag_t* diag, int32_t* fallback_list,
                              int32_t* fallback_count, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (fp8 && (rc = check_fp8_cache(g, k_scale, v_scale))) return rc;
    if ((rc = check_routing_sizes(g, P, K_c, true))) return rc;
    if ((rc = check_epsilon(epsilon))) return rc;
    if (isnan(gap_threshold)) return VSA_ERR_INVALID_ARGUMENT;
    if (!q || !k_cache || !v_cache || !block_table || !seq_lens || !routed_pages || !out || !diag ||
        !fallback_list || !fallback_count)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache)) return VSA_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaMemsetAsync(fallback_count, 0, sizeof(int32_t), st);
    if (e != cudaSuccess) return VSA_ERR_CUDA;
    return cuda_rc(vsa::launch_sparse(g, q, k_cache, v_cache, block_table, seq_lens, (int32_t*)routed_pages, nullptr,
                                      P, K_c, epsilon, gap_threshold, out, diag, fallback_list, fallback_count, st, 0,
                                      nullptr, nullptr, nullptr, 1, nullptr, nullptr, 0, nullptr, 0, k_scale, v_scale));
}

int vsa_sparse_decode(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                      const int32_t* block_table, const int32_t* seq_lens, const int32_t* routed_pages,
                      int32_t P, int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                      int32_t* fallback_list, int32_t* fallback_count, void* ws, size_t ws_bytes, void* stream)
{
    (void)ws;
    (void)ws_bytes;
    return sparse_decode_impl(shape, q, k_cache, v_cache, nullptr, nullptr, false, block_table, seq_lens, routed_pages,
                              P, K_c, epsilon, gap_threshold, out, diag, fallback_list, fallback_count, stream);
}

int vsa_sparse_decode_fp8(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                          const float* k_scale, const float* v_scale, const int32_t* block_table,
                          const int32_t* seq_lens, const int32_t* routed_pages, int32_t P, int32_t K_c, float epsilon,
                          float gap_threshold, float* out, vsa_diag_t* diag, int32_t* fallback_list,
                          int32_t* fallback_count, void* stream)
{
    return sparse_decode_impl(shape, q, k_cache, v_cache, k_scale, v_scale, true, block_table, seq_lens, routed_pages,
                              P, K_c, epsilon, gap_threshold, out, diag, fallback_list, fallback_count, stream);
}

static int sparse_solver_impl(int solver_kind, const vsa_shape_t* shape, const void* q, const void* k_cache,
                              const void* v_cache, const int32_t* block_table, const int32_t* seq_lens,
                              const int32_t* routed_pages, int32_t P, int32_t K_c, float epsilon, float gap_threshold,
                              int32_t solver_iters, float* out, vsa_diag_t* diag, vsa_solve_t* solve,
                              int32_t* fallback_list, int32_t* fallback_count, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;   // this entry point: head_dim 128 only
    if ((rc = check_routing_sizes(g, P, K_c, true))) return rc;
    if ((rc = check_solver_sizes(K_c, solver_iters))) return rc;
    if ((rc = check_epsilon(epsilon))) return rc;
    if (isnan(gap_threshold)) return VSA_ERR_INVALID_ARGUMENT;
    if (!q || !k_cache || !v_cache || !block_table || !seq_lens || !routed_pages || !out || !diag || !solve ||
        !fallback_list || !fallback_count)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache)) return VSA_ERR_MISALIGNED;
    if (!vsa::sparse_shared_memory_fits(g, P, K_c, false, true, false)) return VSA_ERR_UNSUPPORTED_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(fallback_count, 0, sizeof(int32_t), st) != cudaSuccess) return VSA_ERR_CUDA;
    return cuda_rc(vsa::launch_sparse(g, q, k_cache, v_cache, block_table, seq_lens, (int32_t*)routed_pages, nullptr,
                                      P, K_c, epsilon, gap_threshold, out, diag, fallback_list, fallback_count, st,
                                      solver_iters, solve, nullptr, nullptr, solver_kind));
}

int vsa_sparse_decode_entropic(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                               const int32_t* block_table, const int32_t* seq_lens, const int32_t* routed_pages,
                               int32_t P, int32_t K_c, float epsilon, float gap_threshold, int32_t solver_iters,
                               float* out, vsa_diag_t* diag, vsa_solve_t* solve, int32_t* fallback_list,
                               int32_t* fallback_count, void* stream)
{
    return sparse_solver_impl(1, shape, q, k_cache, v_cache, block_table, seq_lens, routed_pages, P, K_c, epsilon,
                              gap_threshold, solver_iters, out, diag, solve, fallback_list, fallback_count, stream);
}

int vsa_sparse_decode_frank_wolfe(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                                  const int32_t* block_table, const int32_t* seq_lens, const int32_t* routed_pages,
                                  int32_t P, int32_t K_c, float epsilon, float gap_threshold, int32_t solver_iters,
                                  float* out, vsa_diag_t* diag, vsa_solve_t* solve, int32_t* fallback_list,
                                  int32_t* fallback_count, void* stream)
{
    return sparse_solver_impl(2, shape, q, k_cache, v_cache, block_table, seq_lens, routed_pages, P, K_c, epsilon,
                              gap_threshold, solver_iters, out, diag, solve, fallback_list, fallback_count, stream);
}

static int dense_impl(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                      const float* k_scale, const float* v_scale, bool fp8, const int32_t* block_table,
                      const int32_t* seq_lens, const int32_t* fallback_list, const int32_t* fallback_count,
                      float epsilon, float* out, vsa_diag_t* diag, void* ws, size_t ws_bytes, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (fp8 && (rc = check_fp8_cache(g, k_scale, v_scale))) return rc;
    if ((rc = check_epsilon(epsilon))) return rc;
    if (!q || !k_cache || !v_cache || !block_table || !seq_lens || !out || !ws) return VSA_ERR_INVALID_ARGUMENT;
    if (fallback_count && !fallback_list) return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(ws)) return VSA_ERR_MISALIGNED;
    if (ws_bytes < vsa::dense_workspace_bytes(g)) return VSA_ERR_WORKSPACE_TOO_SMALL;
    return cuda_rc(vsa::launch_dense(g, q, k_cache, v_cache, block_table, seq_lens, fallback_list, fallback_count,
                                     epsilon, out, diag, ws, (cudaStream_t)stream, false, k_scale, v_scale));
}

int vsa_dense_decode_fallback(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                              const int32_t* block_table, const int32_t* seq_lens, const int32_t* fallback_list,
                              const int32_t* fallback_count, float epsilon, float* out, vsa_diag_t* diag,
                              void* ws, size_t ws_bytes, void* stream)
{
    return dense_impl(shape, q, k_cache, v_cache, nullptr, nullptr, false, block_table, seq_lens, fallback_list,
                      fallback_count, epsilon, out, diag, ws, ws_bytes, stream);
}

int vsa_dense_decode_fallback_fp8(const vsa_shape_t* shape, const void* q, const void* k_cache, const void* v_cache,
                                  const float* k_scale, const float* v_scale, const int32_t* block_table,
                                  const int32_t* seq_lens, const int32_t* fallback_list,
                                  const int32_t* fallback_count, float epsilon, float* out, vsa_diag_t* diag,
                                  void* ws, size_t ws_bytes, void* stream)
{
    return dense_impl(shape, q, k_cache, v_cache, k_scale, v_scale, true, block_table, seq_lens, fallback_list,
                      fallback_count, epsilon, out, diag, ws, ws_bytes, stream);
}

static int decode_step_impl(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                            const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                            int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                            int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                            size_t ws_bytes, void* stream, void* const* events, int solver_iters = 0,
                            vsa_solve_t* solve = nullptr, const float* radii = nullptr, vsa_cert_t* cert = nullptr,
                            int solver_kind = 1, bool fp8 = false, const float* k_scale = nullptr,
                            const float* v_scale = nullptr)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (fp8 && (rc = check_fp8_cache(g, k_scale, v_scale))) return rc;
    if (g.head_dim != vsa::kHeadDim && (solve || cert)) return VSA_ERR_UNSUPPORTED_SHAPE;   // closed form only
    if ((rc = check_routing_sizes(g, P, K_c, true))) return rc;
    if (solve && (rc = check_solver_sizes(K_c, solver_iters))) return rc;
    if ((rc = check_epsilon(epsilon))) return rc;
    if (isnan(gap_threshold)) return VSA_ERR_INVALID_ARGUMENT;
    if (!q || !summaries || !k_cache || !v_cache || !block_table || !seq_lens || !out || !diag ||
        !routed_pages || !fallback_list || !fallback_count || !ws)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(summaries) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(ws))
        return VSA_ERR_MISALIGNED;
    if (ws_bytes < step_route_part(g) + vsa::dense_workspace_bytes(g)) return VSA_ERR_WORKSPACE_TOO_SMALL;
    if (!vsa::sparse_shared_memory_fits(g, P, K_c, true, solve != nullptr, cert != nullptr))
        return VSA_ERR_UNSUPPORTED_SHAPE;
    float* rad_logical = nullptr;
    if (cert) {
        if (!radii) return VSA_ERR_INVALID_ARGUMENT;
        if (g.max_pages > vsa::sparse_register_select_max_pages((long long)g.batch * g.n_q_heads))
            return VSA_ERR_UNSUPPORTED_SHAPE;
        if (ws_bytes < step_rad_offset(g) + step_rad_bytes(g)) return VSA_ERR_WORKSPACE_TOO_SMALL;
        rad_logical = (float*)((char*)ws + step_rad_offset(g));
    }
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    if (events)
        for (int i = 0; i < 5; ++i) {
            if (!events[i]) return VSA_ERR_INVALID_ARGUMENT;
            ev[i] = (cudaEvent_t)events[i];
        }
    void* ws_dense = (char*)ws + step_route_part(g);
    if (ev[0] && cudaEventRecord(ev[0], st) != cudaSuccess) return VSA_ERR_CUDA;
    // the scan kernel clears fallback_count and the dense pass's tickets: the step enqueues no memset
    cudaError_t e = vsa::launch_route_scan(g, q, summaries, block_table, seq_lens, ws, fallback_count,
                                           vsa::dense_tickets(ws_dense), vsa::dense_ticket_count(g), st,
                                           cert ? radii : nullptr, rad_logical);
    if (e != cudaSuccess) return VSA_ERR_CUDA;
    if (ev[1] && cudaEventRecord(ev[1], st) != cudaSuccess) return VSA_ERR_CUDA;
    // the top-P selection runs inside the fused kernel, on the scores the scan left in ws
    if (ev[2] && cudaEventRecord(ev[2], st) != cudaSuccess) return VSA_ERR_CUDA;
    e = vsa::launch_sparse(g, q, k_cache, v_cache, block_table, seq_lens, routed_pages, (const float*)ws, P, K_c,
                           epsilon, gap_threshold, out, diag, fallback_list, fallback_count, st, solver_iters, solve,
                           rad_logical, cert, solver_kind, nullptr, nullptr, 0, nullptr, 0, k_scale, v_scale);
    if (e != cudaSuccess) return VSA_ERR_CUDA;
    if (ev[3] && cudaEventRecord(ev[3], st) != cudaSuccess) return VSA_ERR_CUDA;
    e = vsa::launch_dense(g, q, k_cache, v_cache, block_table, seq_lens, fallback_list, fallback_count, epsilon,
                          out, diag, ws_dense, st, /*tickets_cleared=*/true, k_scale, v_scale);
    if (e != cudaSuccess) return VSA_ERR_CUDA;
    if (ev[4] && cudaEventRecord(ev[4], st) != cudaSuccess) return VSA_ERR_CUDA;
    return VSA_OK;
}

int vsa_decode_step(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                    const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                    int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                    int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                    size_t ws_bytes, void* stream)
{
    return decode_step_impl(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                            gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws, ws_bytes,
                            stream, nullptr);
}

int vsa_decode_step_fp8(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                        const void* v_cache, const float* k_scale, const float* v_scale, const int32_t* block_table,
                        const int32_t* seq_lens, int32_t P, int32_t K_c, float epsilon, float gap_threshold,
                        float* out, vsa_diag_t* diag, int32_t* routed_pages, int32_t* fallback_list,
                        int32_t* fallback_count, void* ws, size_t ws_bytes, void* stream)
{
    return decode_step_impl(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                            gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws, ws_bytes,
                            stream, nullptr, 0, nullptr, nullptr, nullptr, 1, true, k_scale, v_scale);
}

int vsa_decode_step_group_shared(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                                 const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                                 int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                                 int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                                 size_t ws_bytes, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;   // this entry point: head_dim 128 only
    if ((rc = check_routing_sizes(g, P, K_c, true))) return rc;
    if ((rc = check_epsilon(epsilon))) return rc;
    if (isnan(gap_threshold)) return VSA_ERR_INVALID_ARGUMENT;
    if (!q || !summaries || !k_cache || !v_cache || !block_table || !seq_lens || !out || !diag || !routed_pages ||
        !fallback_list || !fallback_count || !ws)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(summaries) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(ws))
        return VSA_ERR_MISALIGNED;
    if (!vsa::sparse_shared_supported(g, P)) return VSA_ERR_UNSUPPORTED_SHAPE;
    if (ws_bytes < step_route_part(g) + vsa::dense_workspace_bytes(g)) return VSA_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    void* ws_dense = (char*)ws + step_route_part(g);
    cudaError_t e = vsa::launch_route_scan(g, q, summaries, block_table, seq_lens, ws, fallback_count,
                                           vsa::dense_tickets(ws_dense), vsa::dense_ticket_count(g), st);
    if (e != cudaSuccess) return VSA_ERR_CUDA;
    vsa::GroupSharedArgs a;
    a.g = g;
    a.q = (const uint16_t*)q;
    a.k = (const uint16_t*)k_cache;
    a.v = (const uint16_t*)v_cache;
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.routed_pages = routed_pages;
    a.page_scores = (const float*)ws;
    a.P = P;
    a.K_c = K_c;
    a.epsilon = epsilon;
    a.gap_threshold = gap_threshold;
    a.out = out;
    a.diag = diag;
    a.fallback_list = fallback_list;
    a.fallback_count = fallback_count;
    a.stream = st;
    if (vsa::launch_sparse_shared(a) != cudaSuccess) return VSA_ERR_CUDA;
    return cuda_rc(vsa::launch_dense(g, q, k_cache, v_cache, block_table, seq_lens, fallback_list, fallback_count,
                                     epsilon, out, diag, ws_dense, st, /*tickets_cleared=*/true));
}

int vsa_decode_step_entropic(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                             const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                             int32_t K_c, float epsilon, float gap_threshold, int32_t solver_iters, float* out,
                             vsa_diag_t* diag, vsa_solve_t* solve, int32_t* routed_pages, int32_t* fallback_list,
                             int32_t* fallback_count, void* ws, size_t ws_bytes, void* stream)
{
    if (!solve) return VSA_ERR_INVALID_ARGUMENT;
    return decode_step_impl(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                            gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws, ws_bytes,
                            stream, nullptr, solver_iters, solve);
}

int vsa_decode_step_frank_wolfe(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                                const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                                int32_t K_c, float epsilon, float gap_threshold, int32_t solver_iters, float* out,
                                vsa_diag_t* diag, vsa_solve_t* solve, int32_t* routed_pages, int32_t* fallback_list,
                                int32_t* fallback_count, void* ws, size_t ws_bytes, void* stream)
{
    if (!solve) return VSA_ERR_INVALID_ARGUMENT;
    return decode_step_impl(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                            gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws, ws_bytes,
                            stream, nullptr, solver_iters, solve, nullptr, nullptr, 2);
}

int vsa_decode_step_certified(const vsa_shape_t* shape, const void* q, const void* summaries, const float* radii,
                              const void* k_cache, const void* v_cache, const int32_t* block_table,
                              const int32_t* seq_lens, int32_t P, int32_t K_c, float epsilon, float gap_threshold,
                              float* out, vsa_diag_t* diag, vsa_cert_t* cert, int32_t* routed_pages,
                              int32_t* fallback_list, int32_t* fallback_count, void* ws, size_t ws_bytes,
                              void* stream)
{
    if (!cert || !radii) return VSA_ERR_INVALID_ARGUMENT;
    return decode_step_impl(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                            gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws, ws_bytes,
                            stream, nullptr, 0, nullptr, radii, cert);
}

int vsa_decode_step_certified_expand(const vsa_shape_t* shape, const void* q, const void* summaries,
                                     const float* radii, const void* k_cache, const void* v_cache,
                                     const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                                     int32_t P_expand, int32_t K_c, float epsilon, float gap_threshold, float* out,
                                     vsa_diag_t* diag, vsa_cert_t* cert, int32_t* routed_pages,
                                     int32_t* fallback_list, int32_t* fallback_count, void* ws, size_t ws_bytes,
                                     void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;   // this entry point: head_dim 128 only
    if ((rc = check_routing_sizes(g, P, K_c, true))) return rc;
    if ((rc = check_routing_sizes(g, P_expand, K_c, true))) return rc;
    if (P_expand <= P) return VSA_ERR_INVALID_ARGUMENT;
    if ((rc = check_epsilon(epsilon))) return rc;
    if (isnan(gap_threshold)) return VSA_ERR_INVALID_ARGUMENT;
    if (!q || !summaries || !radii || !k_cache || !v_cache || !block_table || !seq_lens || !out || !diag || !cert ||
        !routed_pages || !fallback_list || !fallback_count || !ws)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(summaries) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(ws))
        return VSA_ERR_MISALIGNED;
    if (g.max_pages > vsa::sparse_register_select_max_pages((long long)g.batch * g.n_q_heads))
        return VSA_ERR_UNSUPPORTED_SHAPE;
    if (ws_bytes < step_retry_offset(g) + step_retry_bytes(g)) return VSA_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    void* ws_dense = (char*)ws + step_route_part(g);
    float* rad_logical = (float*)((char*)ws + step_rad_offset(g));
    const size_t units = (size_t)g.batch * g.n_q_heads;
    int32_t* retry_counts = (int32_t*)((char*)ws + step_retry_offset(g));   // [kMaxExpandRounds]
    int32_t* retry_lists = retry_counts + kMaxExpandRounds;                  // [round][units]
    if (cudaMemsetAsync(retry_counts, 0, kMaxExpandRounds * sizeof(int32_t), st) != cudaSuccess) return VSA_ERR_CUDA;
    // the scan clears the final fallback counter and the dense tickets
    cudaError_t e = vsa::launch_route_scan(g, q, summaries, block_table, seq_lens, ws, fallback_count,
                                           vsa::dense_tickets(ws_dense), vsa::dense_ticket_count(g), st, radii,
                                           rad_logical);
    if (e != cudaSuccess) return VSA_ERR_CUDA;
    // Pass 0 over every unit with P pages; then, while the page budget allows, the units the previous pass
    // could not certify are run again with twice the pages (at most P_expand) from the same page scores.
    // Every pass is enqueued unconditionally - a pass whose list is empty costs blocks that read the count
    // and exit - so the loop is bounded on the host and needs no synchronisation.  What the last pass still
    // refuses goes to the dense pass.
    int P_round = P, round = 0;
    const int32_t *in_list = nullptr, *in_count = nullptr;
    for (;;) {
        const bool last = P_round >= P_expand;
        int32_t* out_list = last ? fallback_list : retry_lists + (size_t)round * units;
        int32_t* out_count = last ? fallback_count : retry_counts + round;
        e = vsa::launch_sparse(g, q, k_cache, v_cache, block_table, seq_lens, routed_pages, (const float*)ws, P_round,
                               K_c, epsilon, gap_threshold, out, diag, out_list, out_count, st, 0, nullptr,
                               rad_logical, cert, 1, in_list, in_count, P_expand);
        if (e != cudaSuccess) return VSA_ERR_CUDA;
        if (last) break;
        in_list = out_list;
        in_count = out_count;
        P_round = P_round * 2 < P_expand ? P_round * 2 : P_expand;
        if (++round >= kMaxExpandRounds) return VSA_ERR_INVALID_ARGUMENT;   // (P >= 1, P_expand <= 128: not reached)
    }
    e = vsa::launch_dense(g, q, k_cache, v_cache, block_table, seq_lens, fallback_list, fallback_count, epsilon,
                          out, diag, ws_dense, st, /*tickets_cleared=*/true);
    return cuda_rc(e);
}

int vsa_decode_step_timed(const vsa_shape_t* shape, const void* q, const void* summaries, const void* k_cache,
                          const void* v_cache, const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                          int32_t K_c, float epsilon, float gap_threshold, float* out, vsa_diag_t* diag,
                          int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                          size_t ws_bytes, void* stream, void* const* events)
{
    if (!events) return VSA_ERR_INVALID_ARGUMENT;
    return decode_step_impl(shape, q, summaries, k_cache, v_cache, block_table, seq_lens, P, K_c, epsilon,
                            gap_threshold, out, diag, routed_pages, fallback_list, fallback_count, ws, ws_bytes,
                            stream, events);
}

int vsa_decode_step_host(const vsa_shape_t* shape, const void* q_host, void* q_dev, const void* summaries,
                         const void* k_cache, const void* v_cache, const int32_t* block_table,
                         const int32_t* seq_lens, int32_t P, int32_t K_c, float epsilon, float gap_threshold,
                         float* out_host, float* out_dev, vsa_diag_t* diag_host, vsa_diag_t* diag_dev,
                         int32_t* routed_pages, int32_t* fallback_list, int32_t* fallback_count, void* ws,
                         size_t ws_bytes, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (!q_host || !q_dev || !out_host || !out_dev || !diag_dev) return VSA_ERR_INVALID_ARGUMENT;
    // validate everything else before the first copy is enqueued
    if ((rc = check_routing_sizes(g, P, K_c, true))) return rc;
    if ((rc = check_epsilon(epsilon))) return rc;
    if (isnan(gap_threshold)) return VSA_ERR_INVALID_ARGUMENT;
    if (!summaries || !k_cache || !v_cache || !block_table || !seq_lens || !routed_pages || !fallback_list ||
        !fallback_count || !ws)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q_dev) || !aligned16(summaries) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(ws))
        return VSA_ERR_MISALIGNED;
    if (ws_bytes < step_route_part(g) + vsa::dense_workspace_bytes(g)) return VSA_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t units = (size_t)g.batch * g.n_q_heads;
    // Page-locked result buffers are written in place by the kernels (posted stores across the bus,
    // overlapped with the rest of the step); pageable ones go through the device staging buffers
    // with a copy on the stream.  q is always staged (every warp of the routing scan re-reads it, which
    // only the device's caches serve well): by a fetch kernel when page-locked, by a copy otherwise.
    float* out_direct = (float*)mapped_device_pointer(out_host);
    vsa_diag_t* diag_direct = diag_host ? (vsa_diag_t*)mapped_device_pointer(diag_host) : nullptr;
    const void* q_mapped = mapped_device_pointer(q_host);
    if (q_mapped && aligned16(q_mapped)) {
        const int n16 = (int)(units * g.head_dim * 2 / 16);
        if (vsa::launch_pdl(fetch_rows_kernel, dim3((unsigned)((n16 + 255) / 256)), dim3(256), 0, st,
                            (const uint4*)q_mapped, (uint4*)q_dev, n16) != cudaSuccess)
            return VSA_ERR_CUDA;
    } else if (cudaMemcpyAsync(q_dev, q_host, units * g.head_dim * 2, cudaMemcpyHostToDevice, st) !=
               cudaSuccess) {
        return VSA_ERR_CUDA;
    }
    rc = vsa_decode_step(shape, q_dev, summaries, k_cache, v_cache, block_table, seq_lens, P,
                         K_c, epsilon, gap_threshold, out_direct ? out_direct : out_dev,
                         diag_direct ? diag_direct : diag_dev, routed_pages, fallback_list, fallback_count, ws,
                         ws_bytes, stream);
    if (rc) return rc;
    if (!out_direct && cudaMemcpyAsync(out_host, out_dev, units * g.head_dim * sizeof(float),
                                       cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return VSA_ERR_CUDA;
    if (diag_host && !diag_direct &&
        cudaMemcpyAsync(diag_host, diag_dev, units * sizeof(vsa_diag_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return VSA_ERR_CUDA;
    return VSA_OK;
}

}  // extern "C"

// ---- routing for callers that cannot allocate ------------------------------------------------------
// The page-score scratch of vsa_route_pages_static: part of the library's device image, so every GPU
// that loads the library holds these 4 MiB until the process exits.  In host code the symbol's name
// is only a handle - it is not a device address and must never be handed to a kernel; the device
// address is looked up once per device with cudaGetSymbolAddress and cached below.
static __device__ __align__(256) float vsa_static_route_scratch[VSA_STATIC_ROUTE_SCORES];

namespace {

constexpr int kMaxDevices = 64;
float* g_static_scratch_addr[kMaxDevices];   // per device ordinal; nullptr = not looked up yet

// Device address of the scratch array on the current device.  The first call on a device performs
// the lookup (it may initialise the device's copy of the module, so it belongs outside stream
// capture); later calls only read the cached pointer.  Concurrent first calls store the same value.
int static_scratch_address(float** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VSA_ERR_CUDA;
    float* p = g_static_scratch_addr[dev];
    if (!p) {
        void* sym = nullptr;
        if (cudaGetSymbolAddress(&sym, vsa_static_route_scratch) != cudaSuccess || !sym) return VSA_ERR_CUDA;
        p = static_cast<float*>(sym);
        g_static_scratch_addr[dev] = p;
    }
    *out = p;
    return VSA_OK;
}

}  // namespace

extern "C" int vsa_route_pages_static(const vsa_shape_t* shape, const void* q, const void* summaries,
                                      const int32_t* block_table, const int32_t* seq_lens, int32_t P,
                                      int32_t* routed_pages, float* routed_scores, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if ((rc = check_routing_sizes(g, P, 0, false))) return rc;
    if (!q || !summaries || !block_table || !seq_lens || !routed_pages) return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(summaries)) return VSA_ERR_MISALIGNED;
    // one fp32 score per (unit, logical page) must fit the fixed array
    if ((unsigned long long)g.batch * g.n_q_heads * g.max_pages > (unsigned long long)VSA_STATIC_ROUTE_SCORES)
        return VSA_ERR_STATIC_SCRATCH_EXCEEDED;
    float* scratch = nullptr;
    if ((rc = static_scratch_address(&scratch))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // nothing in the array needs clearing: the selection reads scores [0, n_b) of every unit, all of
    // which the scan below writes first; whatever an earlier call left beyond n_b is never read
    cudaError_t e = vsa::launch_route_scan(g, q, summaries, block_table, seq_lens, scratch, nullptr, nullptr, 0, st);
    if (e != cudaSuccess) return VSA_ERR_CUDA;
    return cuda_rc(vsa::launch_route_select(g, scratch, seq_lens, P, routed_pages, routed_scores, st));
}

extern "C" int vsa_cp_token_candidates(const vsa_shape_t* shape, const void* q, const void* k_cache,
                                       const int32_t* block_table, const int32_t* seq_lens,
                                       const int32_t* routed_pages, int32_t P, int32_t K_out, int32_t* cand_pos,
                                       float* cand_score, void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;
    if ((rc = check_routing_sizes(g, P, 1, true))) return rc;
    if (K_out < 1) return VSA_ERR_INVALID_ARGUMENT;
    if (K_out > P * g.page_size + 1) return VSA_ERR_UNSUPPORTED_SHAPE;
    if (!q || !k_cache || !block_table || !seq_lens || !routed_pages || !cand_pos || !cand_score)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(q) || !aligned16(k_cache)) return VSA_ERR_MISALIGNED;
    return cuda_rc(vsa::launch_cp_token_candidates(g, q, k_cache, block_table, seq_lens, routed_pages, P, K_out,
                                                   cand_pos, cand_score, (cudaStream_t)stream));
}

extern "C" int vsa_cp_partial_readout(const vsa_shape_t* shape, const void* v_cache, const int32_t* block_table,
                                      const int32_t* seq_lens, const int32_t* cand_pos, const float* cand_score,
                                      int32_t K_c, float epsilon, float* out_partial, float* lse_partial,
                                      void* stream)
{
    Geometry g;
    int rc = make_geometry(shape, &g);
    if (rc) return rc;
    if (g.head_dim != vsa::kHeadDim) return VSA_ERR_UNSUPPORTED_SHAPE;
    if (K_c < 1) return VSA_ERR_INVALID_ARGUMENT;
    if (K_c > kMaxP * 16) return VSA_ERR_UNSUPPORTED_SHAPE;
    if ((rc = check_epsilon(epsilon))) return rc;
    if (!v_cache || !block_table || !seq_lens || !cand_pos || !cand_score || !out_partial || !lse_partial)
        return VSA_ERR_INVALID_ARGUMENT;
    if (!aligned16(v_cache)) return VSA_ERR_MISALIGNED;
    return cuda_rc(vsa::launch_cp_partial_readout(g, v_cache, block_table, seq_lens, cand_pos, cand_score, K_c,
                                                  epsilon, out_partial, lse_partial, (cudaStream_t)stream));
}
