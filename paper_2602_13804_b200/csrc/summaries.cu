// Page summaries: mean of the valid key rows of each page, per KV head (paper Sec. 7 step 1 names
// "coarse page summaries k_page" without defining them; the mean key is this library's reading).
#include "vsa_device.cuh"
#include "vsa_launch.h"

namespace vsa {

// Mean of the first n rows (this thread's 8 columns of each): fp32 sum in ascending token order, IEEE
// division by n, round-to-nearest-even to bf16, packed.
template <int PS>
__device__ __forceinline__ uint4 mean_of_rows(const uint4 (&rows)[PS], int n)
{
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
#pragma unroll
    for (int t = 0; t < PS; ++t) {
        if (t < n) {
            float f[8];
            unpack8(rows[t], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = acc[e] + f[e];
        }
    }
    const float fn = (float)n;
    uint32_t h[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) h[e] = bf16_bits_rne(__fdiv_rn(acc[e], fn));
    uint4 o;
    o.x = h[0] | (h[1] << 16);
    o.y = h[2] | (h[3] << 16);
    o.z = h[4] | (h[5] << 16);
    o.w = h[6] | (h[7] << 16);
    return o;
}

// Radius of the first n rows around mu (see radii_kernel), computed by the 16 lanes of a half-warp
// (lane c = columns 8c .. 8c+7, `hmask` = the half-warp's lanes); every lane returns the value.
template <int PS>
__device__ __forceinline__ float radius_of_rows(const uint4 (&rows)[PS], int n, const uint4& mu_bits, int c,
                                                unsigned hmask)
{
    float mu[8];
    unpack8(mu_bits, mu);
    float d2 = 0.0f;   // lane t: the largest |k_t' - mu|^2 over its rows t' = t, t + 16, ...; 0 for absent rows
#pragma unroll
    for (int t0 = 0; t0 < PS; t0 += 16) {
        float vals[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
            float f[8], d[8];
            unpack8(rows[t0 + t], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) d[e] = __fsub_rn(f[e], mu[e]);
            vals[t] = t0 + t < n ? chunk_partial(d, d) : 0.0f;
        }
        d2 = fmaxf(d2, reduce_scatter16(vals, c, hmask));
    }
#pragma unroll
    for (int off = 8; off; off >>= 1) d2 = fmaxf(d2, __shfl_xor_sync(hmask, d2, off));
    float m2 = chunk_partial(mu, mu);
#pragma unroll
    for (int off = 8; off; off >>= 1) m2 = m2 + __shfl_xor_sync(hmask, m2, off);
    return __fadd_rn(__fmul_rn(__fsqrt_rn(d2), 1.001f), __fmul_rn(__fsqrt_rn(m2), 0x1p-12f));
}

// One thread per (logical page, kv head, 16-byte slice of the head dimension): the D / 8 threads of a
// (page, head) read one contiguous key row per iteration.  fp32 sum in ascending token
// order, IEEE division by the number of valid rows, round-to-nearest-even to bf16.
template <int PS, int D>
__global__ void __launch_bounds__(256) summaries_kernel(Geometry geo, const uint16_t* __restrict__ k_cache,
                                                        const int32_t* __restrict__ block_table,
                                                        const int32_t* __restrict__ seq_lens,
                                                        const int32_t* __restrict__ first_page,
                                                        uint16_t* __restrict__ summaries)
{
    constexpr int SL = D / 8;   // slices per row
    const int b = blockIdx.y;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int c = (int)(idx % SL);
    const int g = (int)((idx / SL) % geo.n_kv_heads);
    const long long l = (idx / SL) / geo.n_kv_heads;
    const int T = seq_lens[b];
    if (T <= 0 || T > geo.max_pages * PS) return;
    const int nb = (T + PS - 1) / PS;
    const int l0 = first_page ? first_page[b] : 0;
    if (l < l0 || l >= nb) return;
    const long long p = block_table[(long long)b * geo.max_pages + l];
    if (p < 0 || p >= geo.pool_pages) return;
    const int n = min(PS, T - (int)l * PS);

    const uint16_t* src = k_cache + p * geo.page_stride + (long long)g * geo.head_stride + c * 8;
    uint4 rows[PS];
#pragma unroll
    for (int t = 0; t < PS; ++t)
        if (t < n) rows[t] = ld_nc_16B(src + (long long)t * geo.token_stride);
    *reinterpret_cast<uint4*>(summaries + (p * geo.n_kv_heads + g) * D + c * 8) = mean_of_rows<PS>(rows, n);
}

// The same for an fp8 cache (e4m3 bytes, value = byte * scale with one scale per page and KV head): the
// decoded bytes are summed in fp32 in ascending token order, multiplied by the scale, divided by the number of
// valid rows and rounded to bf16 - with power-of-two scales bit for bit the summary of the bf16 cache that
// holds the same values.
// One thread per (logical page, kv head, 8-byte slice); head dimension 128.
template <int PS>
__global__ void __launch_bounds__(256) summaries_fp8_kernel(Geometry geo, const uint8_t* __restrict__ k_cache,
                                                            const float* __restrict__ k_scale,
                                                            const int32_t* __restrict__ block_table,
                                                            const int32_t* __restrict__ seq_lens,
                                                            const int32_t* __restrict__ first_page,
                                                            uint16_t* __restrict__ summaries)
{
    const int b = blockIdx.y;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int c = (int)(idx & 15);
    const int g = (int)((idx >> 4) % geo.n_kv_heads);
    const long long l = (idx >> 4) / geo.n_kv_heads;
    const int T = seq_lens[b];
    if (T <= 0 || T > geo.max_pages * PS) return;
    const int nb = (T + PS - 1) / PS;
    const int l0 = first_page ? first_page[b] : 0;
    if (l < l0 || l >= nb) return;
    const long long p = block_table[(long long)b * geo.max_pages + l];
    if (p < 0 || p >= geo.pool_pages) return;
    const int n = min(PS, T - (int)l * PS);
    const uint8_t* src = k_cache + p * geo.page_stride + (long long)g * geo.head_stride + c * 8;
    uint2 rows[PS];
#pragma unroll
    for (int t = 0; t < PS; ++t)
        if (t < n) rows[t] = ld_nc_8B(src + (long long)t * geo.token_stride);
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
#pragma unroll
    for (int t = 0; t < PS; ++t) {
        if (t < n) {
            float f[8];
            unpack8_e4m3(rows[t], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = acc[e] + f[e];
        }
    }
    const float scale = k_scale[p * geo.n_kv_heads + g], fn = (float)n;
    uint32_t h[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) h[e] = bf16_bits_rne(__fdiv_rn(__fmul_rn(acc[e], scale), fn));
    uint4 o;
    o.x = h[0] | (h[1] << 16);
    o.y = h[2] | (h[3] << 16);
    o.z = h[4] | (h[5] << 16);
    o.w = h[6] | (h[7] << 16);
    *reinterpret_cast<uint4*>(summaries + (p * geo.n_kv_heads + g) * kHeadDim + c * 8) = o;
}

// Radius of each page around its stored summary (the ball bound of the routing certificate):
//   rhat = 1.001 * sqrt(max_t |k_t - mu|^2) + 2^-12 * |mu|,
// squared norms summed in the library's canonical order, every operation a single rounded fp32
// operation so that the CPU oracle reproduces the value bit for bit.  Same thread mapping as the
// summaries kernel; the 16 threads of a (page, head) form a half-warp and only talk to each other.
template <int PS>
__global__ void __launch_bounds__(256) radii_kernel(Geometry geo, const uint16_t* __restrict__ k_cache,
                                                    const uint16_t* __restrict__ summaries,
                                                    const int32_t* __restrict__ block_table,
                                                    const int32_t* __restrict__ seq_lens,
                                                    const int32_t* __restrict__ first_page,
                                                    float* __restrict__ radii)
{
    const int b = blockIdx.y;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int c = (int)(idx & 15);
    const int g = (int)((idx >> 4) % geo.n_kv_heads);
    const long long l = (idx >> 4) / geo.n_kv_heads;
    const int T = seq_lens[b];
    if (T <= 0 || T > geo.max_pages * PS) return;
    const int nb = (T + PS - 1) / PS;
    const int l0 = first_page ? first_page[b] : 0;
    if (l < l0 || l >= nb) return;
    const long long p = block_table[(long long)b * geo.max_pages + l];
    if (p < 0 || p >= geo.pool_pages) return;
    const int n = min(PS, T - (int)l * PS);
    const unsigned hmask = 0xffffu << (threadIdx.x & 16);   // this half-warp (the other may have returned)

    const uint4 mu_bits = *reinterpret_cast<const uint4*>(summaries + (p * geo.n_kv_heads + g) * kHeadDim + c * 8);
    const uint16_t* src = k_cache + p * geo.page_stride + (long long)g * geo.head_stride + c * 8;
    uint4 rows[PS];
#pragma unroll
    for (int t = 0; t < PS; ++t)
        rows[t] = t < n ? ld_nc_16B(src + (long long)t * geo.token_stride) : make_uint4(0u, 0u, 0u, 0u);
    const float rhat = radius_of_rows<PS>(rows, n, mu_bits, c, hmask);
    if (c == 0) radii[p * geo.n_kv_heads + g] = rhat;
}

// Appends one token per sequence to the paged cache and brings the page it lands in up to date: its
// key and value rows, the page's summary and (when asked for) its radius.  A half-warp per
// (sequence, kv head); seq_lens are the lengths AFTER the append.
template <int PS>
__global__ void __launch_bounds__(256) append_kernel(Geometry geo, const uint16_t* __restrict__ k_new,
                                                     const uint16_t* __restrict__ v_new, uint16_t* __restrict__ k_cache,
                                                     uint16_t* __restrict__ v_cache,
                                                     const int32_t* __restrict__ block_table,
                                                     const int32_t* __restrict__ seq_lens,
                                                     uint16_t* __restrict__ summaries, float* __restrict__ radii)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int c = (int)(idx & 15);
    const long long pair = idx >> 4;
    if (pair >= (long long)geo.batch * geo.n_kv_heads) return;
    const int b = (int)(pair / geo.n_kv_heads), g = (int)(pair % geo.n_kv_heads);
    const int T = seq_lens[b];
    if (T <= 0 || T > geo.max_pages * PS) return;
    const int l = (T - 1) / PS, n = (T - 1) % PS + 1;   // page of the new token, rows it holds now
    const long long p = block_table[(long long)b * geo.max_pages + l];
    if (p < 0 || p >= geo.pool_pages) return;
    const unsigned hmask = 0xffffu << (threadIdx.x & 16);

    const long long row0 = p * geo.page_stride + (long long)g * geo.head_stride + c * 8;
    const uint4 kn = *reinterpret_cast<const uint4*>(k_new + pair * kHeadDim + c * 8);
    const uint4 vn = *reinterpret_cast<const uint4*>(v_new + pair * kHeadDim + c * 8);
    *reinterpret_cast<uint4*>(k_cache + row0 + (long long)(n - 1) * geo.token_stride) = kn;
    *reinterpret_cast<uint4*>(v_cache + row0 + (long long)(n - 1) * geo.token_stride) = vn;
    uint4 rows[PS];
#pragma unroll
    for (int t = 0; t < PS; ++t)
        rows[t] = t < n - 1 ? *reinterpret_cast<const uint4*>(k_cache + row0 + (long long)t * geo.token_stride)
                            : (t == n - 1 ? kn : make_uint4(0u, 0u, 0u, 0u));
    const uint4 mu_bits = mean_of_rows<PS>(rows, n);
    *reinterpret_cast<uint4*>(summaries + (p * geo.n_kv_heads + g) * kHeadDim + c * 8) = mu_bits;
    if (radii) {
        const float rhat = radius_of_rows<PS>(rows, n, mu_bits, c, hmask);
        if (c == 0) radii[p * geo.n_kv_heads + g] = rhat;
    }
}

cudaError_t launch_append(const Geometry& g, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                          const int32_t* block_table, const int32_t* seq_lens, void* summaries, float* radii,
                          cudaStream_t stream)
{
    const long long threads = (long long)g.batch * g.n_kv_heads * 16;
    auto* kernel = g.page_size == 32 ? append_kernel<32> : append_kernel<16>;
    kernel<<<(unsigned)((threads + 255) / 256), 256, 0, stream>>>(
        g, (const uint16_t*)k_new, (const uint16_t*)v_new, (uint16_t*)k_cache, (uint16_t*)v_cache, block_table,
        seq_lens, (uint16_t*)summaries, radii);
    return cudaGetLastError();
}

cudaError_t launch_build_radii(const Geometry& g, const void* k_cache, const void* summaries,
                               const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_page,
                               float* radii, cudaStream_t stream)
{
    const long long threads = (long long)g.max_pages * g.n_kv_heads * 16;
    dim3 grid((unsigned)((threads + 255) / 256), (unsigned)g.batch);
    auto* kernel = g.page_size == 32 ? radii_kernel<32> : radii_kernel<16>;
    kernel<<<grid, 256, 0, stream>>>(g, (const uint16_t*)k_cache, (const uint16_t*)summaries, block_table,
                                           seq_lens, first_page, radii);
    return cudaGetLastError();
}

cudaError_t launch_build_summaries(const Geometry& g, const void* k_cache, const int32_t* block_table,
                                   const int32_t* seq_lens, const int32_t* first_page, void* summaries,
                                   cudaStream_t stream)
{
    const long long threads = (long long)g.max_pages * g.n_kv_heads * (g.head_dim / 8);
    dim3 grid((unsigned)((threads + 255) / 256), (unsigned)g.batch);
    auto* kernel = g.page_size == 32 ? summaries_kernel<32, 128> : summaries_kernel<16, 128>;
    if (g.head_dim == 64) kernel = g.page_size == 32 ? summaries_kernel<32, 64> : summaries_kernel<16, 64>;
    if (g.head_dim == 256) kernel = g.page_size == 32 ? summaries_kernel<32, 256> : summaries_kernel<16, 256>;
    kernel<<<grid, 256, 0, stream>>>(g, (const uint16_t*)k_cache, block_table, seq_lens, first_page,
                                     (uint16_t*)summaries);
    return cudaGetLastError();
}

cudaError_t launch_build_summaries_fp8(const Geometry& g, const void* k_cache, const float* k_scale,
                                       const int32_t* block_table, const int32_t* seq_lens,
                                       const int32_t* first_page, void* summaries, cudaStream_t stream)
{
    const long long threads = (long long)g.max_pages * g.n_kv_heads * 16;
    dim3 grid((unsigned)((threads + 255) / 256), (unsigned)g.batch);
    auto* kernel = g.page_size == 32 ? summaries_fp8_kernel<32> : summaries_fp8_kernel<16>;
    kernel<<<grid, 256, 0, stream>>>(g, (const uint8_t*)k_cache, k_scale, block_table, seq_lens, first_page,
                                     (uint16_t*)summaries);
    return cudaGetLastError();
}

}  // namespace vsa
