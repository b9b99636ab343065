// Per-rank kernels of the sequence-sharded (context-parallel) decode step: one sequence's pages are spread
// over several ranks, each rank holding the pages whose block-table entries are valid in ITS table (every
// other entry is negative).  The routed page set, the candidate set and the readout are functions of
// per-page / per-token scores that do not depend on where a page lives (paper Sec. 7), so a rank
//   1. scores its own pages (the ordinary page scan: entries outside the pool score -inf) and proposes its
//      local top-P,
//   2. scores the tokens of the GLOBALLY routed pages it owns and proposes its local top-(K_c + 1)
//      (cp_token_candidates_kernel),
//   3. forms the softmax readout over its own members of the GLOBAL candidate set, with its log-sum-exp
//      (cp_partial_readout_kernel);
// the exchanges between the steps (merge of proposals under the library's total order, log-sum-exp
// combine) run on the host side through torch.distributed.  head_dim 128 only.
#include <limits.h>
#include <math.h>

#include "vsa_device.cuh"
#include "vsa_launch.h"

namespace vsa {

namespace {

constexpr int kCpThreads = 256;

__host__ __device__ constexpr int cp_candidates_words(int PT)
{
    return 2 * PT /*tiles*/ + PT * 16 /*keys*/ + (PT * 16 + 3) / 4 /*take*/ + 256 + 16 + 72 + kTopkList + 16;
}

// One block per (sequence, query head).  routed_pages [unit][P]: the unit's routed logical pages (any order,
// -1 padded).  Output: the rank's best min(K_out, scored tokens) tokens of the routed pages it owns, as
// (position, score) pairs in position order, (-1, -inf) padded to K_out.
__global__ void __launch_bounds__(kCpThreads)
cp_token_candidates_kernel(Geometry geo, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_cache,
                           const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_lens,
                           const int32_t* __restrict__ routed_pages, int P, int K_out,
                           int32_t* __restrict__ cand_pos, float* __restrict__ cand_score)
{
    extern __shared__ uint32_t cp_smem[];
    constexpr int WARPS = kCpThreads / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, c = lane & 15, gi = lane >> 4;
    const long long unit = blockIdx.x;
    const int b = (int)(unit / geo.n_q_heads), h = (int)(unit % geo.n_q_heads), g = h / geo.group;
    const int tsh = geo.tile_shift, PT = P << tsh, N = PT * 16;
    int32_t* tile_l = (int32_t*)cp_smem;        // [PT] owned routed tiles, ascending, INT_MAX = none
    int32_t* tile_phys = tile_l + PT;           // [PT]
    uint32_t* keys = cp_smem + 2 * PT;          // [N]
    uint8_t* take = (uint8_t*)(keys + N);       // [N]
    TopkScratch ts;
    ts.hist = keys + N + (N + 3) / 4;
    ts.misc = ts.hist + 256;
    ts.wred = ts.misc + 16;
    ts.list = (int32_t*)(ts.wred + 72);
    int32_t* raw = ts.list + kTopkList;         // [16] scratch words; the page staging below reuses keys[]

    const int T = seq_lens[b];
    const uint4 qraw = ld_nc_16B(q + unit * kHeadDim + c * 8);
    pdl_wait();
    pdl_launch_dependents();
    for (int t = tid; t < K_out; t += kCpThreads) {
        cand_pos[unit * K_out + t] = -1;
        cand_score[unit * K_out + t] = -INFINITY;
    }
    if (!geo.length_ok(T)) return;
    const int nb = geo.pages_of(T);
    const int32_t* bt = block_table + (long long)b * geo.max_pages;

    // routed pages this rank owns, sorted by logical page (array order = position order)
    int32_t* stage = (int32_t*)keys;   // [P] staging; dead before the keys are written
    for (int t = tid; t < P; t += kCpThreads) {
        const int l = routed_pages[unit * P + t];
        int v = INT_MAX;
        if (l >= 0 && l < nb) {
            const int phys = bt[l];
            if (phys >= 0 && phys < geo.pool_pages) v = l;
        }
        stage[t] = v;
    }
    __syncthreads();
    int my_l = INT_MAX, my_rank = 0;
    if (tid < P) {   // P <= 128 < kCpThreads
        my_l = stage[tid];
        for (int j = 0; j < P; ++j) my_rank += (int)((stage[j] < my_l) | ((stage[j] == my_l) & (j < tid)));
    }
    const int np = __syncthreads_count(tid < P && my_l != INT_MAX);   // also: every thread has read the staging
    if (tid < P) {
        for (int hf = 0; hf < (1 << tsh); ++hf) {
            tile_l[(my_rank << tsh) + hf] = my_l == INT_MAX ? INT_MAX : (my_l << tsh) + hf;
            tile_phys[(my_rank << tsh) + hf] = my_l == INT_MAX ? -1 : bt[my_l];
        }
    }
    for (int i = tid; i < N; i += kCpThreads) {
        keys[i] = 0u;
        take[i] = 0;
    }
    if (tid == 0) raw[0] = 0;
    __syncthreads();

    // token scores of the owned tiles: 16 rows per half-warp, lane c ends with the score of token c
    float qf[8];
    unpack8(qraw, qf);
    const int nt = np << tsh;
    int scored = 0;
    for (int pp = warp; pp * 2 < nt; pp += WARPS) {
        const int slot = pp * 2 + gi;
        const bool active = slot < nt;
        uint4 rows[16];
        if (active) {
            const uint16_t* src = k_cache + (long long)tile_phys[slot] * geo.page_stride + (long long)g * geo.head_stride +
                                  c * 8 + (long long)((tile_l[slot] & ((1 << tsh) - 1)) * 16) * geo.token_stride;
#pragma unroll
            for (int t = 0; t < 16; ++t) rows[t] = ld_nc_16B(src + (long long)t * geo.token_stride);
        } else {
#pragma unroll
            for (int t = 0; t < 16; ++t) rows[t] = make_uint4(0u, 0u, 0u, 0u);
        }
        float vals[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
            float kf[8];
            unpack8(rows[t], kf);
            vals[t] = chunk_partial(qf, kf);
        }
        const float s = reduce_scatter16(vals, c);
        const bool valid = active && tile_l[slot] * 16 + c < T;
        if (valid) keys[slot * 16 + c] = float_to_key(s);
        scored += (int)valid;
    }
    scored = __reduce_add_sync(kFullMask, scored);
    if (lane == 0 && scored) atomicAdd(&raw[0], scored);
    __syncthreads();
    const int n_valid = raw[0];
    const int K = min(K_out, n_valid);
    if (K == 0) return;
    if (K < n_valid) {
        block_topk_mark(keys, N, K, take, ts);
    } else {
        for (int i = tid; i < N; i += kCpThreads) take[i] = keys[i] != 0u;
    }
    __syncthreads();

    // ordered compaction: thread t owns the contiguous entries [t * per, (t + 1) * per)
    const int per = (N + kCpThreads - 1) / kCpThreads;
    const int lo = tid * per, hi = min(N, lo + per);
    int mine = 0;
    for (int i = lo; i < hi; ++i) mine += take[i];
    int incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(kFullMask, incl, off);
        if (lane >= off) incl += o;
    }
    if (lane == 31) ts.wred[warp] = (uint32_t)incl;
    __syncthreads();
    int base = incl - mine;
    for (int w = 0; w < warp; ++w) base += (int)ts.wred[w];
    for (int i = lo; i < hi; ++i) {
        if (take[i]) {
            cand_pos[unit * K_out + base] = tile_l[i >> 4] * 16 + (i & 15);
            cand_score[unit * K_out + base] = key_to_float(keys[i]);
            ++base;
        }
    }
}

// One block (128 threads, eight half-warps) per (sequence, query head).  cand_pos / cand_score [unit][K_c]: the
// GLOBAL candidate set with its scores (-1 padded).  The rank sums exp((s - s1) / epsilon) v over the
// candidates whose page it owns, s1 = the largest score of the list; out_partial = that sum normalised by the
// rank's own weight sum (zeros when it owns none), lse_partial = log of the rank's sum of exp(s / epsilon)
// (-inf when it owns none).
__global__ void __launch_bounds__(128)
cp_partial_readout_kernel(Geometry geo, const uint16_t* __restrict__ v_cache, const int32_t* __restrict__ block_table,
                          const int32_t* __restrict__ seq_lens, const int32_t* __restrict__ cand_pos,
                          const float* __restrict__ cand_score, int K_c, float epsilon,
                          float* __restrict__ out_partial, float* __restrict__ lse_partial)
{
    __shared__ float red[8][kHeadDim];
    __shared__ float zred[8];
    __shared__ float smax[4];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, c = lane & 15, hw = tid >> 4;
    const long long unit = blockIdx.x;
    const int b = (int)(unit / geo.n_q_heads), h = (int)(unit % geo.n_q_heads), g = h / geo.group;
    const int T = seq_lens[b];
    pdl_wait();
    pdl_launch_dependents();
    const bool ok = geo.length_ok(T);
    // the largest score of the list (every rank sees the same list, so the same reference)
    float m = -INFINITY;
    for (int j = tid; j < K_c; j += 128)
        if (cand_pos[unit * K_c + j] >= 0) m = fmaxf(m, cand_score[unit * K_c + j]);
#pragma unroll
    for (int off = 16; off; off >>= 1) m = fmaxf(m, __shfl_xor_sync(kFullMask, m, off));
    if (lane == 0) smax[warp] = m;
    __syncthreads();
    const float s1 = fmaxf(fmaxf(smax[0], smax[1]), fmaxf(smax[2], smax[3]));
    const float scale = 1.4426950408889634f / epsilon;
    const int32_t* bt = block_table + (long long)b * geo.max_pages;
    const int page_shift = 4 + geo.tile_shift;
    float acc[8], z = 0.0f;
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
    for (int j = hw; j < K_c && ok; j += 8) {
        const int pos = cand_pos[unit * K_c + j];
        if (pos < 0 || pos >= T) continue;
        const int phys = bt[pos >> page_shift];
        if (phys < 0 || phys >= geo.pool_pages) continue;   // another rank's page
        const float w = exp2f((cand_score[unit * K_c + j] - s1) * scale);
        const uint4 row = ld_nc_16B(v_cache + (long long)phys * geo.page_stride + (long long)g * geo.head_stride +
                                    (long long)(pos & (geo.page_size - 1)) * geo.token_stride + c * 8);
        float vf[8];
        unpack8(row, vf);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = fmaf(w, vf[e], acc[e]);
        z += w;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) red[hw][c * 8 + e] = acc[e];
    if (c == 0) zred[hw] = z;
    __syncthreads();
    float Z = 0.0f;
#pragma unroll
    for (int w = 0; w < 8; ++w) Z += zred[w];
    float a = 0.0f;
#pragma unroll
    for (int w = 0; w < 8; ++w) a += red[w][tid];
    out_partial[unit * kHeadDim + tid] = Z > 0.0f ? a / Z : 0.0f;
    if (tid == 0) lse_partial[unit] = Z > 0.0f ? s1 / epsilon + logf(Z) : -INFINITY;
}

}  // namespace

cudaError_t launch_cp_token_candidates(const Geometry& g, const void* q, const void* k_cache,
                                       const int32_t* block_table, const int32_t* seq_lens,
                                       const int32_t* routed_pages, int P, int K_out, int32_t* cand_pos,
                                       float* cand_score, cudaStream_t stream)
{
    const size_t smem = (size_t)cp_candidates_words(P << g.tile_shift) * 4;
    static bool attr_done[kMaxDevices] = {};
    if (smem > 48 * 1024) {
        const cudaError_t e = allow_large_dynamic_smem(cp_token_candidates_kernel, attr_done);
        if (e != cudaSuccess) return e;
    }
    return launch_pdl(cp_token_candidates_kernel, dim3((unsigned)(g.batch * g.n_q_heads)), dim3(kCpThreads), smem, stream,
                      g, (const uint16_t*)q, (const uint16_t*)k_cache, block_table, seq_lens, routed_pages, P, K_out,
                      cand_pos, cand_score);
}

cudaError_t launch_cp_partial_readout(const Geometry& g, const void* v_cache, const int32_t* block_table,
                                      const int32_t* seq_lens, const int32_t* cand_pos, const float* cand_score,
                                      int K_c, float epsilon, float* out_partial, float* lse_partial,
                                      cudaStream_t stream)
{
    return launch_pdl(cp_partial_readout_kernel, dim3((unsigned)(g.batch * g.n_q_heads)), dim3(128), 0, stream, g,
                      (const uint16_t*)v_cache, block_table, seq_lens, cand_pos, cand_score, K_c, epsilon, out_partial,
                      lse_partial);
}

}  // namespace vsa
