// Table-level kernels: initialisation (Section 5.1: the same initial values as the word2vec program),
// row export/import (Section 6.1, vector export) and the column-slice partial dot
// products of Algorithm 1 for caller-given index pairs.
#include <math_constants.h>

#include "w2v_device.cuh"
#include "w2v_internal.h"

namespace w2v {

// U[w][4 j4 .. 4 j4 + 3] = ((r >> 8) 2^-24 - 0.5) / d, r the four words of
// Philox(seed; w, j4, 0, 0).  Padding columns between d and the row stride are zeroed.
// A column shard stores columns col4_off*4 .. of vectors of d_full columns: the value of a
// column does not depend on which shard holds it.
__global__ void __launch_bounds__(256)
init_u_kernel(float4 *__restrict__ U4, uint64_t total4, uint32_t d4, uint32_t ld4, uint32_t col4_off, float d,
              uint32_t k0, uint32_t k1)
{
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t idx = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total4; idx += stride) {
        const uint32_t row = (uint32_t)(idx / ld4), j4 = (uint32_t)(idx % ld4);
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j4 < d4) {
            const uint4 r = philox4x32_10(k0, k1, row, j4 + col4_off, kPurInit, 0);
            const float s = 1.0f / 16777216.0f;
            o.x = ((float)(r.x >> 8) * s - 0.5f) / d;
            o.y = ((float)(r.y >> 8) * s - 0.5f) / d;
            o.z = ((float)(r.z >> 8) * s - 0.5f) / d;
            o.w = ((float)(r.w >> 8) * s - 0.5f) / d;
        }
        U4[idx] = o;
    }
}

int launch_init_tables(float *U, float *V, uint64_t vocab, uint32_t d, uint32_t ld, uint32_t d_full,
                       uint32_t col_lo, uint64_t seed, cudaStream_t s)
{
    const uint64_t total4 = vocab * (ld / 4);
    const uint64_t want = (total4 + 255) / 256;
    const int grid = (int)(want < 148ull * 32 ? (want ? want : 1) : 148ull * 32);
    init_u_kernel<<<grid, 256, 0, s>>>(reinterpret_cast<float4 *>(U), total4, d / 4, ld / 4, col_lo / 4,
                                       (float)d_full, (uint32_t)seed, (uint32_t)(seed >> 32));
    if (cudaGetLastError() != cudaSuccess) return -1;
    if (cudaMemsetAsync(V, 0, vocab * (uint64_t)ld * sizeof(float), s) != cudaSuccess) return -1;
    return 1;
}

// One warp per pair; lanes stride over the columns of the slice.  The 16-byte aligned
// middle of the slice is read as float4, the ragged ends as scalars.
__global__ void __launch_bounds__(kBlock)
partial_dots_kernel(const float *__restrict__ U, const float *__restrict__ V, uint32_t vocab, uint32_t ld,
                    const int32_t *__restrict__ pairs, uint64_t m, uint32_t col_lo, uint32_t col_hi,
                    float *__restrict__ out, DevState *st)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t a0 = (col_lo + 3u) & ~3u;            // first aligned column
    const uint32_t a1 = col_hi & ~3u;                   // end of the aligned part
    for (uint64_t i = warp; i < m; i += nwarps) {
        const int32_t wi = pairs[2 * i], wo = pairs[2 * i + 1];
        if (wi < 0 || (uint32_t)wi >= vocab || wo < 0 || (uint32_t)wo >= vocab) {
            if (lane == 0) { out[i] = CUDART_NAN_F; atomicOr(&st->status, 1u); }
            continue;
        }
        const float *u = U + (size_t)wi * ld, *v = V + (size_t)wo * ld;
        float s = 0.f;
        if (a0 < a1) {
            for (uint32_t j = col_lo + lane; j < a0; j += 32) s = fmaf(__ldcg(u + j), __ldcg(v + j), s);
            const float4 *u4 = reinterpret_cast<const float4 *>(u), *v4 = reinterpret_cast<const float4 *>(v);
            for (uint32_t j4 = a0 / 4 + lane; j4 < a1 / 4; j4 += 32) {
                const float4 x = __ldcg(u4 + j4), y = __ldcg(v4 + j4);
                s = fmaf(x.x, y.x, s); s = fmaf(x.y, y.y, s); s = fmaf(x.z, y.z, s); s = fmaf(x.w, y.w, s);
            }
            for (uint32_t j = a1 + lane; j < col_hi; j += 32) s = fmaf(__ldcg(u + j), __ldcg(v + j), s);
        } else {
            for (uint32_t j = col_lo + lane; j < col_hi; j += 32) s = fmaf(__ldcg(u + j), __ldcg(v + j), s);
        }
        s = warp_sum(s);
        if (lane == 0) out[i] = s;
    }
}

int launch_partial_dots(const float *U, const float *V, uint32_t vocab, uint32_t ld, const int32_t *pairs,
                        uint64_t m, uint32_t col_lo, uint32_t col_hi, float *out, DevState *st, int sms,
                        cudaStream_t s)
{
    if (m == 0) return 0;
    const uint64_t want = (m + (kBlock / 32) - 1) / (kBlock / 32);
    const uint64_t cap = (uint64_t)sms * 8;
    const int grid = (int)(want < cap ? want : cap);
    partial_dots_kernel<<<grid, kBlock, 0, s>>>(U, V, vocab, ld, pairs, m, col_lo, col_hi, out, st);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

// One warp per row, 16 bytes per lane per trip.
__global__ void __launch_bounds__(kBlock)
copy_rows_kernel(float4 *__restrict__ table, uint32_t vocab, uint32_t d4, uint32_t ld4,
                 const int64_t *__restrict__ ids,
                 uint64_t m, float4 *__restrict__ buf, bool to_table)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t warp = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint64_t nwarps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t i = warp; i < m; i += nwarps) {
        const int64_t w = ids[i];
        if (w < 0 || (uint64_t)w >= vocab) continue;
        float4 *row = table + (size_t)w * ld4, *b = buf + (size_t)i * d4;
        for (uint32_t j = lane; j < d4; j += 32) {
            if (to_table) row[j] = b[j];
            else b[j] = __ldcg(row + j);
        }
    }
}

int launch_copy_rows(float *table, uint32_t vocab, uint32_t d, uint32_t ld, const int64_t *ids, uint64_t m,
                     float *buf, bool to_table, int sms, cudaStream_t s)
{
    if (m == 0) return 0;
    const uint64_t want = (m + (kBlock / 32) - 1) / (kBlock / 32);
    const uint64_t cap = (uint64_t)sms * 8;
    const int grid = (int)(want < cap ? want : cap);
    copy_rows_kernel<<<grid, kBlock, 0, s>>>(reinterpret_cast<float4 *>(table), vocab, d / 4, ld / 4, ids, m,
                                             reinterpret_cast<float4 *>(buf), to_table);
    if (cudaGetLastError() != cudaSuccess) return -1;
    return 1;
}

}  // namespace w2v
