// Device-side helpers shared by the kernels of libw2v: the counter-based
// generator, warp/block scans, row loads and vector reductions into global memory.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace w2v {

constexpr uint32_t kFullMask = 0xFFFFFFFFu;

// Purposes in counter word c2 (low byte); see counter layout in w2v_internal.h.
enum : uint32_t { kPurInit = 0, kPurSubsample = 1, kPurRadius = 2, kPurNegative = 3 };

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies and
// xors; the key is bumped by the Weyl constants after each round.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1,
                                               uint32_t c2, uint32_t c3)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Inclusive scan of one value per lane.
template <typename T>
__device__ __forceinline__ T warp_inclusive_scan(T x, uint32_t lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        T y = __shfl_up_sync(kFullMask, x, o);
        if (lane >= (uint32_t)o) x += y;
    }
    return x;
}

template <typename T>
__device__ __forceinline__ T warp_sum(T x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(kFullMask, x, o);
    return x;
}

// Exclusive scan over the threads of a block (blockDim.x a multiple of 32, <= 1024).
// `warp_tot` is shared memory for 32 values of T.  Returns the exclusive prefix of
// this thread and, in `total`, the sum over the block.
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T x, T *warp_tot, T &total)
{
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const T incl = warp_inclusive_scan(x, lane);
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        T t = lane < nw ? warp_tot[lane] : T(0);
        T ti = warp_inclusive_scan(t, lane);
        warp_tot[lane] = ti - t;                       // exclusive prefix of each warp
        if (lane == 31) warp_tot[32] = ti;             // block total
    }
    __syncthreads();
    const T base = warp_tot[wid];
    total = warp_tot[32];
    __syncthreads();
    return base + incl - x;
}

// One table row spread over a warp: lane l holds float4 number l, l+32, ... of the row,
// i.e. a fixed column slice of every vector (the role a shard has in the paper).
template <int VPL>
struct Row {
    float4 x[VPL];
};

template <int VPL>
__device__ __forceinline__ void row_zero(Row<VPL> &r)
{
#pragma unroll
    for (int v = 0; v < VPL; ++v) r.x[v] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// Loads go to L2 only (ld.global.cg): each row is used once by this warp and other
// SMs may be adding to it, so there is nothing to gain from L1.
template <int VPL>
__device__ __forceinline__ void row_load(Row<VPL> &r, const float4 *base, uint32_t d4, uint32_t lane)
{
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const uint32_t idx = lane + 32u * v;
        r.x[v] = idx < d4 ? __ldcg(base + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

// Row touch: one 4-byte load per 64-byte DRAM burst of a row brings the whole row into L2 at
// the price of one register per 2 KB of row (a full gather costs one per 16 bytes), so many
// more rows can be in flight per warp.  NCH = touches per lane.  The last touch is the row's
// last word: a row that does not start on a 64-byte boundary spans one burst more.
template <int NCH>
__device__ __forceinline__ void row_touch(uint32_t (&x)[NCH], const float4 *base, uint32_t d4, uint32_t lane)
{
    const char *b = reinterpret_cast<const char *>(base);
    const uint32_t bytes = d4 * 16u, n = (bytes + 63u) / 64u + 1u;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        const uint32_t idx = lane + 32u * c;
        x[c] = 0u;
        if (idx < n) {
            const uint32_t off = idx * 64u < bytes ? idx * 64u : bytes - 4u;
            asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(x[c]) : "l"(b + off));
        }
    }
}

// An offset that is always zero (`zero` is a kernel argument equal to 0) but that the hardware
// can only compute once the touches have landed: added to the address of the additions that
// follow, it makes them wait for the row to be in L2.
template <int NCH>
__device__ __forceinline__ uint32_t touch_fence(const uint32_t (&x)[NCH], uint32_t zero)
{
    uint32_t a = x[0];
#pragma unroll
    for (int c = 1; c < NCH; ++c) a |= x[c];
    return a & zero;
}

template <int VPL>
__device__ __forceinline__ float row_dot_partial(const Row<VPL> &a, const Row<VPL> &b)
{
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        s = fmaf(a.x[v].x, b.x[v].x, s);
        s = fmaf(a.x[v].y, b.x[v].y, s);
        s = fmaf(a.x[v].z, b.x[v].z, s);
        s = fmaf(a.x[v].w, b.x[v].w, s);
    }
    return s;
}

// acc += g * r
template <int VPL>
__device__ __forceinline__ void row_axpy(Row<VPL> &acc, float g, const Row<VPL> &r)
{
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        acc.x[v].x = fmaf(g, r.x[v].x, acc.x[v].x);
        acc.x[v].y = fmaf(g, r.x[v].y, acc.x[v].y);
        acc.x[v].z = fmaf(g, r.x[v].z, acc.x[v].z);
        acc.x[v].w = fmaf(g, r.x[v].w, acc.x[v].w);
    }
}

template <int VPL>
__device__ __forceinline__ void row_add(Row<VPL> &acc, const Row<VPL> &r)
{
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        acc.x[v].x += r.x[v].x;
        acc.x[v].y += r.x[v].y;
        acc.x[v].z += r.x[v].z;
        acc.x[v].w += r.x[v].w;
    }
}

// Fire-and-forget 16-byte floating point add into global memory (resolved in L2).
__device__ __forceinline__ void red_add_f32x4(float4 *addr, float a, float b, float c, float d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 :
                 : "l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

// dst_row += g * r
template <int VPL>
__device__ __forceinline__ void row_red_scaled(float4 *dst, float g, const Row<VPL> &r, uint32_t d4, uint32_t lane)
{
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const uint32_t idx = lane + 32u * v;
        if (idx < d4) red_add_f32x4(dst + idx, g * r.x[v].x, g * r.x[v].y, g * r.x[v].z, g * r.x[v].w);
    }
}

// dst_row (double precision sums, d consecutive doubles) += g * r
template <int VPL>
__device__ __forceinline__ void row_add_scaled_f64(double *dst, float g, const Row<VPL> &r, uint32_t d4, uint32_t lane)
{
    const double gd = (double)g;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
        const uint32_t idx = lane + 32u * v;
        if (idx < d4) {
            double *a = dst + 4u * idx;
            atomicAdd(a + 0, gd * (double)r.x[v].x);
            atomicAdd(a + 1, gd * (double)r.x[v].y);
            atomicAdd(a + 2, gd * (double)r.x[v].z);
            atomicAdd(a + 3, gd * (double)r.x[v].w);
        }
    }
}

__device__ __forceinline__ float sigmoidf_exact(float x)
{
    return 1.0f / (1.0f + expf(-x));
}

}  // namespace w2v
