// Calibration second moments: sumsq[j] (+)= scale * sum_t X[t][j]^2.
// HBM-bound streaming column reduction: 2 bytes and one FMA per activation; one kernel (the
// last CTA of a column chunk adds the row splits' partial sums).
#include "common.cuh"

namespace {

constexpr int MOM_TX = 32;            // lanes across columns, 8 bf16 (16 B) each
constexpr int MOM_TY = 8;             // warps across rows
constexpr int MOM_COLS = MOM_TX * 8;  // 256 columns per CTA
constexpr int MOM_UNROLL = 8;         // 16-byte loads in flight per thread

// grid.x = column chunks of 256, grid.y = row splits; partial[split][K]
__global__ void __launch_bounds__(MOM_TX * MOM_TY)
moments_partial_kernel(const __nv_bfloat16* __restrict__ X, int64_t T, int64_t K, int64_t ldx,
                       int64_t rows_per_split, float* __restrict__ partial,
                       unsigned* __restrict__ chunk_done, float scale, int accumulate,
                       float* __restrict__ out) {
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
    // The last CTA of this column chunk to finish adds the splits' partial sums in split order
    // (a fixed order whichever CTA does it: bit-identical reruns) and clears the counter.
    __shared__ bool last_sh;
    __threadfence();
    __syncthreads();
    if (c == 0) last_sh = atomicAdd(chunk_done + blockIdx.x, 1u) == gridDim.y - 1;
    __syncthreads();
    if (last_sh) {
        __threadfence();
        if (gc < K) {
            float s = 0.f;
            for (unsigned p = 0; p < gridDim.y; ++p) s += __ldcg(partial + (int64_t)p * K + gc);
            s *= scale;
            out[gc] = accumulate ? out[gc] + s : s;
        }
        if (c == 0) chunk_done[blockIdx.x] = 0u;
    }
}

}  // namespace

extern "C" sb_status sb_calib_moments(sb_ctx* ctx, const void* X, int64_t T, int64_t K,
                                      int64_t ldx, float* sumsq, int accumulate, float scale) {
    if (!ctx) return SB_ERR_INVALID;
    if ((!X && T > 0) || !sumsq || T < 0 || K <= 0) return sb_fail(ctx, SB_ERR_INVALID, "moments: null or empty");
    if (K % 8 || ldx % 8 || ldx < K || (reinterpret_cast<uintptr_t>(X) & 15))
        return sb_fail(ctx, SB_ERR_SHAPE, "moments: K, ldx must be multiples of 8 and X 16-byte aligned");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const int col_chunks = (int)((K + MOM_COLS - 1) / MOM_COLS);
    // about 8 CTAs of 256 threads per SM in flight
    int splits = (ctx->sm_count * 8 + col_chunks - 1) / col_chunks;
    const int64_t min_rows = MOM_TY * MOM_UNROLL;
    if ((int64_t)splits * min_rows > T) splits = (int)((T + min_rows - 1) / min_rows);
    if (splits < 1) splits = 1;
    int64_t rows_per_split = (T + splits - 1) / splits;
    rows_per_split = (rows_per_split + min_rows - 1) / min_rows * min_rows;
    if (rows_per_split < min_rows) rows_per_split = min_rows;
    splits = (int)((T + rows_per_split - 1) / rows_per_split);
    if (splits < 1) splits = 1;
    void* arena;
    sb_status st = sb_scratch(ctx, Carver::need({(size_t)splits * K * sizeof(float)}), &arena);
    if (st != SB_OK) return st;
    Carver cv(arena);
    float* partial = cv.take<float>((size_t)splits * K);
    if (col_chunks > SB_MOMENT_CHUNKS)
        return sb_fail(ctx, SB_ERR_SHAPE, "moments: K above %d not supported", SB_MOMENT_CHUNKS * MOM_COLS);
    dim3 grid(col_chunks, splits), block(MOM_TX, MOM_TY);
    moments_partial_kernel<<<grid, block, 0, ctx->stream>>>(
        static_cast<const __nv_bfloat16*>(X), T, K, ldx, rows_per_split, partial, ctx->moment_done, scale,
        accumulate, sumsq);
    SB_LAUNCHED(ctx);
    return SB_OK;
}
