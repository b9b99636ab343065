// Device-side building blocks shared by the kernels of libvsa: bf16 unpacking, the fixed-order
// fp32 dot product, order-preserving keys and block-wide exact top-k selection.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace vsa {

constexpr int kHeadDim = 128;   // elements per head
constexpr int kPageSize = 16;   // tokens per page
constexpr int kRowBytes = kHeadDim * 2;
constexpr unsigned kFullMask = 0xffffffffu;

// ---- programmatic dependent launch ----------------------------------------------------------
// Every kernel of the step is launched with programmatic stream serialization: it may be
// scheduled while its predecessor in the stream is still running.  pdl_wait() blocks until the
// predecessor grid has completed and its memory is visible (a no-op for ordinary launches), so
// it precedes the first access to anything another kernel writes or reads;
// pdl_launch_dependents() lets the successor start being scheduled.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- bf16 ------------------------------------------------------------------------------
// A 16-byte vector holds 8 consecutive bf16 values, element 0 in the low half of .x
__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8])
{
    f[0] = __uint_as_float(v.x << 16);
    f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16);
    f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16);
    f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16);
    f[7] = __uint_as_float(v.w & 0xffff0000u);
}

// ---- fp8 (e4m3) -----------------------------------------------------------------------------
// An 8-byte vector holds 8 consecutive e4m3 values, element 0 in the low byte of .x.  The conversion is
// exact (every e4m3 value is an fp16 value).  A cache stores value = byte * scale with one fp32 scale per
// (pool page, KV head); multiplying by a power-of-two scale is exact.
__device__ __forceinline__ void unpack8_e4m3(const uint2& v, float (&f)[8])
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const unsigned short pair = (unsigned short)(((i < 2) ? v.x : v.y) >> (16 * (i & 1)));
        unsigned int h2;
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(pair));
        asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tcvt.f32.f16 %0, lo;\n\tcvt.f32.f16 %1, hi;\n\t}"
            : "=f"(f[2 * i]), "=f"(f[2 * i + 1])
            : "r"(h2));
    }
}

// Four e4m3 bytes of a 32-bit word -> two packed bf16 pairs (bytes 0, 1 -> lo; bytes 2, 3 -> hi) with integer
// operations and one packed multiply (the conversion instructions run at a fraction of that rate): the seven
// exponent and mantissa bits of a byte, placed at the top of a bf16's exponent and mantissa fields, read as
// 2^(e - 127) (1 + m / 8) - or, for e = 0, as the bf16 subnormal (m / 8) 2^-126 - and the product with 2^120
// is the e4m3 value in both cases, exactly.
__device__ __forceinline__ void e4m3x4_to_bf16x2x2(uint32_t w, uint32_t& lo, uint32_t& hi)
{
    const uint32_t a = __byte_perm(w, 0u, 0x4140), b = __byte_perm(w, 0u, 0x4342);   // 0x00b1'00b0, 0x00b3'00b2
    const uint32_t xa = ((a << 8) & 0x80008000u) | ((a << 4) & 0x07f007f0u);
    const uint32_t xb = ((b << 8) & 0x80008000u) | ((b << 4) & 0x07f007f0u);
    const uint32_t two120 = 0x7b807b80u;   // bf16 2^120, twice
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(lo) : "r"(xa), "r"(two120));
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(hi) : "r"(xb), "r"(two120));
}

__device__ __forceinline__ uint2 ld_nc_8B(const void* p)
{
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

// round-to-nearest-even fp32 -> bf16 bits (finite inputs)
__device__ __forceinline__ uint32_t bf16_bits_rne(float f)
{
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (u >> 16) | 0x0040u;
    u += 0x7fffu + ((u >> 16) & 1u);
    return u >> 16;
}

__device__ __forceinline__ uint4 ld_nc_16B(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// global load that the compiler keeps where it is written (used to issue independent loads
// ahead of the first branch that needs any of them)
__device__ __forceinline__ float ld_cg_f32(const float* p)
{
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

__device__ __forceinline__ int ld_ca_s32(const int32_t* p)
{
    int v;
    asm volatile("ld.global.ca.s32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// 4-byte asynchronous copies into shared memory (sources with no 16-byte alignment guarantee)
__device__ __forceinline__ void cp_async_4(uint32_t smem_addr, const void* gptr)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_addr), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_16B(uint32_t smem_addr, const void* gptr)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_commit_group() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// ---- the fixed-order dot product ---------------------------------------------------------
// A row of 128 elements is spread over 16 lanes, lane c holding elements 8c .. 8c+7.
// chunk_partial() sums the lane's 8 products as two interleaved chains,
//     (((x0 y0 + x2 y2) + x4 y4) + x6 y6)  +  (((x1 y1 + x3 y3) + x5 y5) + x7 y7),
// which is exactly what one packed mul.f32x2 followed by three packed fma.rn.f32x2 compute on the
// (even, odd) element pairs that unpacking a 32-bit word yields (bf16 x bf16 products are exact in
// fp32, so fusing the multiply into the add changes nothing).
__device__ __forceinline__ void mul2(float& d0, float& d1, float a0, float a1, float b0, float b1)
{
    asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "mul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b0, float b1)
{
    asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rd, {%0, %1};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rd;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "+f"(d0), "+f"(d1)
        : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

__device__ __forceinline__ float chunk_partial(const float (&x)[8], const float (&y)[8])
{
    float even, odd;
    mul2(even, odd, x[0], x[1], y[0], y[1]);
    fma2(even, odd, x[2], x[3], y[2], y[3]);
    fma2(even, odd, x[4], x[5], y[4], y[5]);
    fma2(even, odd, x[6], x[7], y[6], y[7]);
    return even + odd;
}

// The same tree without any per-lane selection: on entry slot i of lane c holds this lane's partial
// of value (i ^ c) - the caller arranges that through which data each lane loads - so that at
// every level the slot a lane sends and the slot it adds into are fixed.  On return lane c holds
// the complete sum of value c.  Per value the additions are again p[c] += p[c+off], off = 8, 4, 2, 1.
__device__ __forceinline__ float reduce_scatter16_xor(float (&v)[16])
{
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] += __shfl_xor_sync(kFullMask, v[i + 8], 8);
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] += __shfl_xor_sync(kFullMask, v[i + 4], 4);
#pragma unroll
    for (int i = 0; i < 2; ++i) v[i] += __shfl_xor_sync(kFullMask, v[i + 2], 2);
    return v[0] + __shfl_xor_sync(kFullMask, v[1], 1);
}

// Halving tree over the 16 lanes of a half-warp for 16 independent values at once
// ("reduce-scatter"): on entry v[i] is this lane's partial of value i, on return lane c
// (0..15 within its half-warp) holds the complete sum of value c.  For each value the
// additions are exactly p[c] += p[c+off] for off = 8, 4, 2, 1 (addition is commutative, so
// which lane of a pair performs it does not change a bit).  15 shuffles for 16 values.  `mask` names
// the lanes that take part (the whole warp, or one half-warp when the other may have exited).
__device__ __forceinline__ float reduce_scatter16(float (&v)[16], int c, unsigned mask = kFullMask)
{
    {
        const bool hi = c & 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float send = hi ? v[i] : v[i + 8];
            const float keep = hi ? v[i + 8] : v[i];
            v[i] = keep + __shfl_xor_sync(mask, send, 8);
        }
    }
    {
        const bool hi = c & 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float send = hi ? v[i] : v[i + 4];
            const float keep = hi ? v[i + 4] : v[i];
            v[i] = keep + __shfl_xor_sync(mask, send, 4);
        }
    }
    {
        const bool hi = c & 2;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const float send = hi ? v[i] : v[i + 2];
            const float keep = hi ? v[i + 2] : v[i];
            v[i] = keep + __shfl_xor_sync(mask, send, 2);
        }
    }
    {
        const bool hi = c & 1;
        const float send = hi ? v[0] : v[1];
        const float keep = hi ? v[1] : v[0];
        v[0] = keep + __shfl_xor_sync(mask, send, 1);
    }
    return v[0];
}

// ---- order-preserving keys -----------------------------------------------------------------
// key(a) > key(b)  <=>  a > b for finite floats and infinities; -0 and +0 map to one key.
// Key 0 is never produced by a non-NaN float and serves as "no element".
__device__ __forceinline__ uint32_t float_to_key(float f)
{
    uint32_t u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float key_to_float(uint32_t k)
{
    const uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(u);
}

// ---- exact block-wide top-k ------------------------------------------------------------------
// Elements are keys[0..n) in shared memory (key 0 = absent).  The order is (key descending,
// array index ascending).  After the call, for k >= 1 and at least k present elements:
//   *kth       = key of the k-th element in that order,
//   *n_greater = number of elements with key > *kth  (all of them belong to the top k),
//   *n_equal   = number of elements with key == *kth; the top k takes the first
//                k - *n_greater of them in array-index order.
// MSB-first radix select, 8 bits per pass.  hist: 256 counters in shared memory.
// All threads of the block must call it; results are valid for all threads on return.
struct SelectResult {
    uint32_t kth;
    int n_greater;
    int n_equal;
};

__device__ __forceinline__ SelectResult block_select_kth(const uint32_t* keys, int n, int k, uint32_t* hist,
                                                         uint32_t* scratch /* >= 4 words */)
{
    uint32_t prefix = 0, prefix_mask = 0;
    int remaining = k;   // rank still to find inside the current prefix bucket
    int greater = 0;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const uint32_t key = keys[i];
            if (key != 0u && (key & prefix_mask) == prefix) atomicAdd(&hist[(key >> shift) & 0xffu], 1u);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane j owns digits 8j .. 8j+7; find the digit where the count from the top reaches `remaining`
            const int lane = threadIdx.x;
            uint32_t c[8], mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                c[j] = hist[lane * 8 + j];
                mine += c[j];
            }
            // suffix sum over lanes: above = total count in digits of higher lanes
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
                        scratch[0] = (uint32_t)(lane * 8 + j);
                        scratch[1] = above;   // elements of this bucket set that rank strictly higher
                        scratch[2] = c[j];
                    }
                    above += c[j];
                }
            }
        }
        __syncthreads();
        const uint32_t digit = scratch[0];
        greater += (int)scratch[1];
        remaining -= (int)scratch[1];
        prefix |= digit << shift;
        prefix_mask |= 0xffu << shift;
        const int bucket = (int)scratch[2];
        __syncthreads();
        if (shift == 0) {
            SelectResult r;
            r.kth = prefix;
            r.n_greater = greater;
            r.n_equal = bucket;
            return r;
        }
    }
    SelectResult r = {0u, 0, 0};
    return r;
}

// Rank, in array-index order, of element i among the elements with keys[j] == kth, for every
// i at once: marks take[i] = 1 for the first `need` of them.  Runs tile by tile; only called when
// a tie straddles the cut.  warp_counts: >= blockDim.x / 32 + 1 words of shared memory.
__device__ __forceinline__ void block_mark_first_equal(const uint32_t* keys, int n, uint32_t kth, int need,
                                                       uint8_t* take, uint32_t* warp_counts,
                                                       uint32_t* last_taken = nullptr)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    int base = 0;
    for (int start = 0; start < n; start += blockDim.x) {
        const int i = start + threadIdx.x;
        const bool eq = i < n && keys[i] == kth;
        const unsigned b = __ballot_sync(kFullMask, eq);
        if (lane == 0) warp_counts[warp] = __popc(b);
        __syncthreads();
        int before = base;
        for (int w = 0; w < warp; ++w) before += warp_counts[w];
        int total = 0;
        for (int w = 0; w < nwarps; ++w) total += warp_counts[w];
        if (eq) {
            const int rank = before + __popc(b & ((1u << lane) - 1u));
            if (rank < need) take[i] = 1;
            if (last_taken && rank == need - 1) *last_taken = (uint32_t)i;
        }
        base += total;
        __syncthreads();
        if (base >= need) break;
    }
}

// ---- exact block-wide top-K, one histogram pass in the common case --------------------------------
// Marks take[i] = 1 for exactly the K best of keys[0..n) under (key descending, index ascending);
// key 0 = absent; take[] must be zero on entry; needs 1 <= K <= number of present keys.  Returns (to
// every thread) the key and array index of the K-th = worst selected element.
//
// Fast path: keys are bucketed LINEARLY in score between the smallest and largest finite score
// (monotone: a higher score never lands in a lower bucket), so one 256-bin histogram isolates the
// bucket that contains the cut; buckets above it are taken whole and the few elements of the cut
// bucket are ranked exactly against each other.  If the cut bucket is crowded (> kTopkList
// elements) or the score range is degenerate, the MSB radix select above decides instead.
constexpr int kTopkList = 256;

struct TopkScratch {
    uint32_t* hist;    // [256]
    uint32_t* misc;    // [16]
    uint32_t* wred;    // [72]  per-warp partials (up to 32 warps, two values each) + warp counts
    int32_t* list;     // [kTopkList]
};

struct TopkResult {
    uint32_t kth_key;
    int kth_idx;
};

__device__ __forceinline__ TopkResult block_topk_mark(const uint32_t* keys, int n, int K, uint8_t* take,
                                                      const TopkScratch& s)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    // ---- range of the finite scores ----
    float lo = INFINITY, hi = -INFINITY;
    for (int i = tid; i < n; i += blockDim.x) {
        const uint32_t key = keys[i];
        if (key != 0u) {
            const float f = key_to_float(key);
            if (f > -INFINITY) lo = fminf(lo, f);
            hi = fmaxf(hi, f);
        }
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(kFullMask, lo, off));
        hi = fmaxf(hi, __shfl_xor_sync(kFullMask, hi, off));
    }
    if (lane == 0) {
        s.wred[2 * warp] = __float_as_uint(lo);
        s.wred[2 * warp + 1] = __float_as_uint(hi);
    }
    for (int i = tid; i < 256; i += blockDim.x) s.hist[i] = 0u;
    if (tid == 0) s.misc[4] = 0u;   // list length
    __syncthreads();
    lo = INFINITY;
    hi = -INFINITY;
    for (int w = 0; w < nwarps; ++w) {
        lo = fminf(lo, __uint_as_float(s.wred[2 * w]));
        hi = fmaxf(hi, __uint_as_float(s.wred[2 * w + 1]));
    }
    const float scale = 256.0f / (hi - lo);
    const bool fast = hi > lo && isfinite(scale) && isfinite(hi - lo);
    int cut = -1, need = K;
    if (fast) {
        for (int i = tid; i < n; i += blockDim.x) {
            const uint32_t key = keys[i];
            if (key != 0u) {
                const float f = key_to_float(key);
                const int b = f > -INFINITY ? min(255, (int)((f - lo) * scale)) : 0;
                atomicAdd(&s.hist[b], 1u);
            }
        }
        __syncthreads();
        if (tid < 32) {
            uint32_t c[8], mine = 0;
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
            if (above < (uint32_t)K && (uint32_t)K <= incl) {
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (above < (uint32_t)K && (uint32_t)K <= above + c[j]) {
                        s.misc[0] = (uint32_t)(lane * 8 + j);
                        s.misc[1] = above;
                        s.misc[2] = c[j];
                    }
                    above += c[j];
                }
            }
        }
        __syncthreads();
        if ((int)s.misc[2] <= kTopkList) {
            cut = (int)s.misc[0];
            need = K - (int)s.misc[1];
        }
    }
    if (cut >= 0) {
        for (int i = tid; i < n; i += blockDim.x) {
            const uint32_t key = keys[i];
            if (key != 0u) {
                const float f = key_to_float(key);
                const int b = f > -INFINITY ? min(255, (int)((f - lo) * scale)) : 0;
                if (b > cut) take[i] = 1;
                if (b == cut) s.list[atomicAdd(&s.misc[4], 1u)] = i;
            }
        }
        __syncthreads();
        const int m = (int)s.misc[4];
        for (int t = tid; t < m; t += blockDim.x) {
            const int idx = s.list[t];
            const uint32_t key = keys[idx];
            int rank = 0;
            for (int j = 0; j < m; ++j) {
                const int ij = s.list[j];
                const uint32_t kj = keys[ij];
                rank += (int)((kj > key) | ((kj == key) & (ij < idx)));
            }
            if (rank < need) take[idx] = 1;
            if (rank == need - 1) {
                s.misc[5] = key;
                s.misc[6] = (uint32_t)idx;
            }
        }
        __syncthreads();
    } else {
        __syncthreads();   // everyone has read misc[] of the fast attempt
        const SelectResult r = block_select_kth(keys, n, K, s.hist, s.misc);
        const int need_eq = K - r.n_greater;
        for (int i = tid; i < n; i += blockDim.x)
            if (keys[i] > r.kth) take[i] = 1;
        block_mark_first_equal(keys, n, r.kth, need_eq, take, s.wred, &s.misc[6]);
        if (tid == 0) s.misc[5] = r.kth;
        __syncthreads();
    }
    TopkResult out;
    out.kth_key = s.misc[5];
    out.kth_idx = (int)s.misc[6];
    return out;
}

// Block-wide list append without one atomic per entry: every thread of a (converged) warp passes
// the number of entries it wants to add and gets the first of its consecutive slots; the warp
// takes its range with a single atomic on `counter`.
__device__ __forceinline__ int warp_append_slots(int cnt, uint32_t* counter)
{
    const int lane = threadIdx.x & 31;
    int incl = cnt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(kFullMask, incl, off);
        if (lane >= off) incl += o;
    }
    const int total = __shfl_sync(kFullMask, incl, 31);
    int base = 0;
    if (lane == 31 && total > 0) base = (int)atomicAdd(counter, (uint32_t)total);
    base = __shfl_sync(kFullMask, base, 31);
    return base + incl - cnt;
}

// ---- the same selection with the keys held in registers -------------------------------------------
// Thread t owns elements t, t + blockDim, ..., t + (KPT-1) * blockDim (key[j] = 0 where the element is
// absent or past n).  On return bit j of the result's `mask` is set iff element t + j * blockDim is
// among the K best, for every thread; kth_key / kth_idx describe the K-th (worst selected) element.
// No pass re-reads shared memory for the keys, so the per-thread work of a pass is KPT independent
// register operations.  `spill` ([n] words) and `spill_take` ([n] bytes) are only touched on the slow
// path (crowded cut bucket or degenerate range), which stores the keys and runs the routine above.
struct TopkRegResult {
    uint32_t mask;
    uint32_t kth_key;
    int kth_idx;
};

// HAVE_RANGE: the caller supplies the histogram range and has zeroed hist[0..256) and misc[4] before
// its last barrier, which saves the range reduction and one barrier here.  (lo_in, hi_in) may be any
// bracket of the bulk of the scores - scores outside it fall into the first or the last bucket, which
// keeps the buckets fine where the cut is when a few outliers stretch the full range - and
// (lo_full, hi_full), the smallest finite and the largest score, is used when that bracket is empty.
template <int KPT, bool HAVE_RANGE = false>
__device__ __forceinline__ TopkRegResult block_topk_reg(const uint32_t (&key)[KPT], int n, int K,
                                                        const TopkScratch& s, uint32_t* spill, uint8_t* spill_take,
                                                        float lo_in = 0.0f, float hi_in = 0.0f, float lo_full = 0.0f,
                                                        float hi_full = 0.0f)
{
    static_assert(KPT <= 32, "one mask bit per owned element");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const int stride = blockDim.x;
    float f[KPT];
    float lo = INFINITY, hi = -INFINITY;
#pragma unroll
    for (int j = 0; j < KPT; ++j) {
        f[j] = key_to_float(key[j]);
        if (!HAVE_RANGE && key[j] != 0u) {
            if (f[j] > -INFINITY) lo = fminf(lo, f[j]);
            hi = fmaxf(hi, f[j]);
        }
    }
    if constexpr (HAVE_RANGE) {
        const bool bracket = hi_in > lo_in;
        lo = bracket ? lo_in : lo_full;
        hi = bracket ? hi_in : hi_full;
    } else {
#pragma unroll
        for (int off = 16; off; off >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(kFullMask, lo, off));
            hi = fmaxf(hi, __shfl_xor_sync(kFullMask, hi, off));
        }
        if (lane == 0) {
            s.wred[2 * warp] = __float_as_uint(lo);
            s.wred[2 * warp + 1] = __float_as_uint(hi);
        }
        for (int i = tid; i < 256; i += stride) s.hist[i] = 0u;
        if (tid == 0) s.misc[4] = 0u;   // list length
        __syncthreads();
        lo = INFINITY;
        hi = -INFINITY;
        for (int w = 0; w < nwarps; ++w) {
            lo = fminf(lo, __uint_as_float(s.wred[2 * w]));
            hi = fmaxf(hi, __uint_as_float(s.wred[2 * w + 1]));
        }
    }
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
        __syncthreads();
        if (warp == 0) {
            // one warp scans the histogram and publishes the cut through the barrier that follows
            uint32_t c[8], mine = 0;
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
            const int src = __ffs(found) - 1;   // exactly one lane owns the cut bucket
            my_cut = __shfl_sync(kFullMask, my_cut, src);
            my_above = __shfl_sync(kFullMask, my_above, src);
            my_count = __shfl_sync(kFullMask, my_count, src);
            if (lane == 0) {
                s.misc[9] = my_count <= kTopkList ? (uint32_t)my_cut : 0xffffffffu;
                s.misc[10] = (uint32_t)(K - my_above);
            }
        }
        __syncthreads();   // the histogram has been read: its words are reused for the cut bucket's keys
        if (s.misc[9] != 0xffffffffu) {
            cut = (int)s.misc[9];
            need = (int)s.misc[10];
        }
    }
    TopkRegResult out;
    out.mask = 0u;
    if (cut >= 0) {
        // list entries: element index in list[], its key in hist[] (the histogram is dead by now)
        uint32_t in_cut = 0u;
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            if (key[j] != 0u) {
                if (bucket[j] > cut) out.mask |= 1u << j;
                if (bucket[j] == cut) in_cut |= 1u << j;
            }
        }
        {
            // the histogram is dead (read before the last barrier): its words take the listed keys
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
        __syncthreads();
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
        __syncthreads();
#pragma unroll
        for (int j = 0; j < KPT; ++j)
            if (((in_cut >> j) & 1u) && spill_take[tid + j * stride]) out.mask |= 1u << j;
    } else {
        __syncthreads();
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            const int i = tid + j * stride;
            if (i < n) {
                spill[i] = key[j];
                spill_take[i] = 0;
            }
        }
        __syncthreads();
        block_topk_mark(spill, n, K, spill_take, s);
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            const int i = tid + j * stride;
            if (i < n && spill_take[i]) out.mask |= 1u << j;
        }
    }
    out.kth_key = s.misc[5];
    out.kth_idx = (int)s.misc[6];
    __syncthreads();   // scratch may be reused by the caller right away
    return out;
}

}  // namespace vsa
