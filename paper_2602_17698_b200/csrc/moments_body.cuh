// The streaming column reduction both moments entry points run: one CTA adds the squares of
// its 256 columns over its split of the rows and writes one partial sum per column.
#pragma once
#include "common.cuh"

constexpr int MOM_TX = 32;            // lanes across columns, 8 bf16 (16 B) each
constexpr int MOM_TY = 8;             // warps across rows
constexpr int MOM_COLS = MOM_TX * 8;  // 256 columns per CTA
constexpr int MOM_UNROLL = 8;         // 16-byte loads in flight per thread

// blockIdx.x = column chunk of 256, blockIdx.y = row split, block = (MOM_TX, MOM_TY);
// writes partial[blockIdx.y][column] for every column of the chunk below K (so a reader never
// sees what an earlier call left there).  Ends after a __syncthreads(), all stores issued.
__device__ __forceinline__ void moments_split_partial(const __nv_bfloat16* __restrict__ X, int64_t T,
                                                      int64_t K, int64_t ldx, int64_t rows_per_split,
                                                      float* __restrict__ partial) {
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int64_t col = (int64_t)blockIdx.x * MOM_COLS + tx * 8;
    const int64_t t0 = (int64_t)blockIdx.y * rows_per_split;
    const int64_t t1 = min(T, t0 + rows_per_split);
    float acc[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = 0.f;
    if (col < K) {
        const __nv_bfloat16* base = X + col;
        int64_t t = t0 + ty;
        // main loop: MOM_UNROLL independent loads, then the FMAs
        for (; t + (MOM_UNROLL - 1) * MOM_TY < t1; t += MOM_UNROLL * MOM_TY) {
            uint4 v[MOM_UNROLL];
#pragma unroll
            for (int u = 0; u < MOM_UNROLL; ++u) v[u] = ld_stream16(base + (t + u * MOM_TY) * ldx);
#pragma unroll
            for (int u = 0; u < MOM_UNROLL; ++u) {
                const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float a = bf16lo(w[k]), b = bf16hi(w[k]);
                    acc[2 * k] = fmaf(a, a, acc[2 * k]);
                    acc[2 * k + 1] = fmaf(b, b, acc[2 * k + 1]);
                }
            }
        }
        for (; t < t1; t += MOM_TY) {
            uint4 v = ld_stream16(base + t * ldx);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float a = bf16lo(w[k]), b = bf16hi(w[k]);
                acc[2 * k] = fmaf(a, a, acc[2 * k]);
                acc[2 * k + 1] = fmaf(b, b, acc[2 * k + 1]);
            }
        }
    }
    // fixed-order reduction over the 8 row-warps
    __shared__ float red[MOM_TY][MOM_COLS + 8];
#pragma unroll
    for (int k = 0; k < 8; ++k) red[ty][tx * 8 + k] = acc[k];
    __syncthreads();
    const int c = ty * MOM_TX + tx;   // 256 threads, one column each
    const int64_t gc = (int64_t)blockIdx.x * MOM_COLS + c;
    if (gc < K) {
        float s = 0.f;
#pragma unroll
        for (int y = 0; y < MOM_TY; ++y) s += red[y][c];
        partial[(int64_t)blockIdx.y * K + gc] = s;
    }
}
