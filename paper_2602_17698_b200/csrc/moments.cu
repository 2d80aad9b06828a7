// Calibration second moments: sumsq[j] (+)= scale * sum_t X[t][j]^2.
// HBM-bound streaming column reduction: 2 bytes and one FMA per activation; one kernel (the
// last CTA of a column chunk adds the row splits' partial sums).
#include "common.cuh"
#include "moments_body.cuh"

namespace {

// grid.x = column chunks of 256, grid.y = row splits; partial[split][K]
__global__ void __launch_bounds__(MOM_TX * MOM_TY)
moments_partial_kernel(const __nv_bfloat16* __restrict__ X, int64_t T, int64_t K, int64_t ldx,
                       int64_t rows_per_split, float* __restrict__ partial,
                       unsigned* __restrict__ chunk_done, float scale, int accumulate,
                       float* __restrict__ out) {
    moments_split_partial(X, T, K, ldx, rows_per_split, partial);
    const int c = threadIdx.y * MOM_TX + threadIdx.x;   // 256 threads, one column each
    const int64_t gc = (int64_t)blockIdx.x * MOM_COLS + c;
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
    // One wave: as many CTAs as are resident at once, not more (each CTA has the same share of the
    // rows, so a second, partly filled wave would leave SMs idle at the end: measured 0.538 ms for
    // the four inputs of an 8B layer with a third of a wave left over against 0.502 ms without).
    if (ctx->moments_ctas_per_sm == 0) {
        int occ = 0;
        SB_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, moments_partial_kernel, MOM_TX * MOM_TY, 0));
        ctx->moments_ctas_per_sm = occ > 0 ? occ : 1;
    }
    int splits = (ctx->sm_count * ctx->moments_ctas_per_sm) / col_chunks;
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
