// sb_calib_moments_noalloc: the calibration second moments for callers that must not
// allocate device memory.
//
// Who needs it: code that runs where cudaMalloc is off limits -- a serving loop whose device
// memory was handed out in full at start-up (another pool owns every byte, so an allocation
// fails or evicts someone), a section managed by a framework's caching allocator where a raw
// cudaMalloc would synchronise the device and fragment the pool, or a latency-critical path
// that cannot afford the implicit synchronisation of an allocation.  The regular entry point
// keeps its per-split partial sums in a context-owned arena that grows with cudaMalloc; this
// one keeps them in a fixed array that is part of the library image instead.
//
// The array costs SB_NOALLOC_SCRATCH_FLOATS * 4 bytes (4 MiB) on EVERY GPU that loads the
// library, for the life of the process.  All calls share it and it keeps whatever the last
// call left there; the kernels overwrite every partial they later read, so nothing has to
// start at zero, but two calls whose kernels overlap on the GPU (for instance on different
// streams) race on it.
//
// The first call on each device looks up the array's device address (no allocation); make
// that first call before any stream capture begins.
#include <mutex>

#include "common.cuh"
#include "moments_body.cuh"

#define SB_NOALLOC_SCRATCH_FLOATS (1 << 20)
#define SB_NOALLOC_MAX_K 65536

static __device__ __align__(256) float sb_noalloc_scratch[SB_NOALLOC_SCRATCH_FLOATS];

namespace {

constexpr int NA_TX = MOM_TX, NA_TY = MOM_TY, NA_COLS = MOM_COLS, NA_UNROLL = MOM_UNROLL;

// grid.x = chunks of 256 columns, grid.y = row splits; partial[split][K]: the same reduction as
// the regular entry point (every (split, column) it later reads is written first)
__global__ void __launch_bounds__(NA_TX * NA_TY)
noalloc_partial_kernel(const __nv_bfloat16* __restrict__ X, int64_t T, int64_t K, int64_t ldx,
                       int64_t rows_per_split, float* __restrict__ partial) {
    moments_split_partial(X, T, K, ldx, rows_per_split, partial);
}

__global__ void noalloc_finish_kernel(const float* __restrict__ partial, int splits, int64_t K,
                                      float scale, int accumulate, float* __restrict__ out) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= K) return;
    float s = 0.f;
    for (int p = 0; p < splits; ++p) s += partial[(int64_t)p * K + j];
    s *= scale;
    out[j] = accumulate ? out[j] + s : s;
}

// In host code `sb_noalloc_scratch` is only a stand-in for the symbol, not a device address:
// the address the kernels can use comes from cudaGetSymbolAddress, looked up once per device
// with that device current.
std::mutex g_mu;
float* g_scratch_ptr[64] = {nullptr};
int g_sm_count[64] = {0};          // resident CTAs of the partial-sum kernel per device (SMs x CTAs per SM)

sb_status scratch_for_current_device(float** out, int* sm_count) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        (void)cudaGetLastError();
        fprintf(stderr, "sb_calib_moments_noalloc: no current CUDA device\n");
        return SB_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        float* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), sb_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            (void)cudaGetLastError();
            fprintf(stderr, "sb_calib_moments_noalloc: cudaGetSymbolAddress failed: %s\n",
                    cudaGetErrorString(e));
            return SB_ERR_CUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            sms = 148;
        // one wave of resident CTAs (a host-side calculation: nothing is allocated)
        int occ = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, noalloc_partial_kernel, NA_TX * NA_TY, 0) != cudaSuccess ||
            occ <= 0) {
            (void)cudaGetLastError();
            occ = 6;
        }
        g_sm_count[dev] = sms * occ;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    *sm_count = g_sm_count[dev];               // resident CTAs of the partial-sum kernel on this device
    return SB_OK;
}

}  // namespace

extern "C" sb_status sb_calib_moments_noalloc(void* cuda_stream, const void* X, int64_t T, int64_t K,
                                              int64_t ldx, float* sumsq, int accumulate, float scale) {
    if ((!X && T > 0) || !sumsq || T < 0 || K <= 0) {
        fprintf(stderr, "sb_calib_moments_noalloc: null or empty argument\n");
        return SB_ERR_INVALID;
    }
    if (K % 8 || ldx % 8 || ldx < K || (reinterpret_cast<uintptr_t>(X) & 15)) {
        fprintf(stderr, "sb_calib_moments_noalloc: K and ldx must be multiples of 8, X 16-byte aligned\n");
        return SB_ERR_SHAPE;
    }
    if (K > SB_NOALLOC_MAX_K) {
        fprintf(stderr, "sb_calib_moments_noalloc: K = %lld exceeds the fixed scratch (at most %d "
                        "channels per call; split the columns or use sb_calib_moments)\n",
                (long long)K, SB_NOALLOC_MAX_K);
        return SB_ERR_SCRATCH;
    }
    float* partial = nullptr;
    int sms = 148 * 6;                              // resident CTAs of the partial-sum kernel
    sb_status st = scratch_for_current_device(&partial, &sms);
    if (st != SB_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int col_chunks = (int)((K + NA_COLS - 1) / NA_COLS);
    const int64_t min_rows = NA_TY * NA_UNROLL;
    int splits = sms / col_chunks;                  // sms: resident CTAs; the grid is one wave of them
    const int max_splits = (int)(SB_NOALLOC_SCRATCH_FLOATS / K);       // >= 16 by the K limit
    if (splits > max_splits) splits = max_splits;
    if ((int64_t)splits * min_rows > T) splits = (int)((T + min_rows - 1) / min_rows);
    if (splits < 1) splits = 1;
    int64_t rows_per_split = (T + splits - 1) / splits;
    rows_per_split = (rows_per_split + min_rows - 1) / min_rows * min_rows;
    if (rows_per_split < min_rows) rows_per_split = min_rows;
    splits = (int)((T + rows_per_split - 1) / rows_per_split);
    if (splits < 1) splits = 1;
    dim3 grid(col_chunks, splits), block(NA_TX, NA_TY);
    noalloc_partial_kernel<<<grid, block, 0, stream>>>(static_cast<const __nv_bfloat16*>(X), T, K, ldx,
                                                       rows_per_split, partial);
    noalloc_finish_kernel<<<(unsigned)((K + 255) / 256), 256, 0, stream>>>(partial, splits, K, scale,
                                                                           accumulate, sumsq);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        fprintf(stderr, "sb_calib_moments_noalloc: launch failed: %s\n", cudaGetErrorString(e));
        return SB_ERR_CUDA;
    }
    return SB_OK;
}
