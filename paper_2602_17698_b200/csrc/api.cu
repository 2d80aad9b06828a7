// Context management of the C-ABI library: device, stream, scratch arena, status word.
#include <stdarg.h>
#include <string.h>

#include "common.cuh"

sb_status sb_fail(sb_ctx* ctx, sb_status st, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof ctx->err, fmt, ap);
        va_end(ap);
    }
    return st;
}

bool sb_check_bits(const int* bits, int n_bits) {
    if (!bits || n_bits < 1 || n_bits > 8) return false;
    for (int l = 0; l < n_bits; ++l) {
        if (bits[l] < 1 || bits[l] > 8) return false;
        if (l > 0 && bits[l] <= bits[l - 1]) return false;
    }
    return true;
}

sb_status sb_scratch(sb_ctx* ctx, size_t bytes, void** out) {
    if (bytes > ctx->scratch_bytes) {
        // Growth is rare (first call of a shape).  The old arena is retired, not freed: launches
        // already enqueued, or captured in a CUDA graph by the caller, keep valid pointers until
        // the context is destroyed.  Doubling bounds the retired arenas by the live one.
        size_t want = bytes + bytes / 8 + (1u << 20);
        if (want < 2 * ctx->scratch_bytes) want = 2 * ctx->scratch_bytes;
        void* fresh = nullptr;
        cudaError_t e = cudaMalloc(&fresh, want);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return sb_fail(ctx, SB_ERR_SCRATCH, "scratch arena of %zu bytes: %s", want,
                           cudaGetErrorString(e));
        }
        if (ctx->scratch) ctx->retired.push_back(ctx->scratch);
        ctx->scratch = fresh;
        ctx->scratch_bytes = want;
    }
    *out = ctx->scratch;
    return SB_OK;
}

extern "C" {

sb_status sb_create(sb_ctx** out, int device, void* cuda_stream) {
    if (!out) return SB_ERR_INVALID;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) {
        (void)cudaGetLastError();
        return SB_ERR_CUDA;   // no usable CUDA device: this library has no CPU path
    }
    sb_ctx* ctx = new sb_ctx();
    ctx->device = device;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    cudaDeviceProp prop;
    if (cudaSetDevice(device) != cudaSuccess ||
        cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
        delete ctx;
        return SB_ERR_CUDA;
    }
    if (prop.major != 10) {   // built for sm_100a only
        delete ctx;
        return SB_ERR_CUDA;
    }
    ctx->sm_count = prop.multiProcessorCount;
    SbDeviceState init{};
    init.lb_wait_ns = 250ull * 1000 * 1000;
    init.lb_mute_tile = 0xffffffffu;
    if (cudaMalloc(&ctx->dstate, sizeof(SbDeviceState)) != cudaSuccess ||
        cudaMemcpy(ctx->dstate, &init, sizeof(SbDeviceState), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMalloc(&ctx->moment_done, SB_MOMENT_CHUNKS * sizeof(unsigned)) != cudaSuccess ||
        cudaMemset(ctx->moment_done, 0, SB_MOMENT_CHUNKS * sizeof(unsigned)) != cudaSuccess ||
        cudaMalloc(&ctx->stats_done, 2 * SB_STATS_TILES * sizeof(unsigned)) != cudaSuccess ||
        cudaMemset(ctx->stats_done, 0, 2 * SB_STATS_TILES * sizeof(unsigned)) != cudaSuccess ||
        cudaMallocHost(&ctx->pinned, 4096) != cudaSuccess) {
        (void)cudaGetLastError();
        sb_destroy(ctx);      // frees whatever was allocated before the failure
        return SB_ERR_CUDA;
    }
    ctx->pinned_bytes = 4096;
    *out = ctx;
    return SB_OK;
}

sb_status sb_destroy(sb_ctx* ctx) {
    if (!ctx) return SB_OK;
    cudaSetDevice(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    if (ctx->scratch) cudaFree(ctx->scratch);
    for (void* p : ctx->retired) cudaFree(p);
    if (ctx->dstate) cudaFree(ctx->dstate);
    if (ctx->lb_mem) cudaFree(ctx->lb_mem);
    if (ctx->moment_done) cudaFree(ctx->moment_done);
    if (ctx->stats_done) cudaFree(ctx->stats_done);
    if (ctx->pinned) cudaFreeHost(ctx->pinned);
    delete ctx;
    return SB_OK;
}

sb_status sb_sync(sb_ctx* ctx) {
    if (!ctx) return SB_ERR_INVALID;
    SbDeviceState* h = static_cast<SbDeviceState*>(ctx->pinned);
    SB_CUDA(ctx, cudaMemcpyAsync(h, ctx->dstate, sizeof(SbDeviceState), cudaMemcpyDeviceToHost,
                                 ctx->stream));
    SB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (h->status != 0) {
        sb_status st = static_cast<sb_status>(h->status);
        int where = h->where;
        SB_CUDA(ctx, cudaMemsetAsync(ctx->dstate, 0, 2 * sizeof(int), ctx->stream));
        SB_CUDA(ctx, cudaMemsetAsync(&ctx->dstate->bad_index, 0, 2 * sizeof(long long), ctx->stream));
        if (h->bad_limit != 0)
            return sb_fail(ctx, st, "device-side status %d latched by kernel family %d: index %lld outside [0, %lld)",
                           (int)st, where, h->bad_index, h->bad_limit);
        return sb_fail(ctx, st, "device-side status %d latched by kernel family %d", (int)st, where);
    }
    return SB_OK;
}

sb_status sb_debug_lookback(sb_ctx* ctx, int64_t wait_ns, int64_t mute_tile) {
    if (!ctx) return SB_ERR_INVALID;
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const unsigned long long w = wait_ns < 0 ? 250ull * 1000 * 1000 : (unsigned long long)wait_ns;
    const unsigned m = mute_tile < 0 ? 0xffffffffu : (unsigned)mute_tile;
    SB_CUDA(ctx, cudaMemcpyAsync(&ctx->dstate->lb_wait_ns, &w, sizeof w, cudaMemcpyHostToDevice, ctx->stream));
    SB_CUDA(ctx, cudaMemcpyAsync(&ctx->dstate->lb_mute_tile, &m, sizeof m, cudaMemcpyHostToDevice, ctx->stream));
    SB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));     // the two host words are on this stack
    return SB_OK;
}

const char* sb_last_error(const sb_ctx* ctx) { return ctx ? ctx->err : "null context"; }

int64_t sb_kernel_launches(const sb_ctx* ctx) { return ctx ? ctx->launches : 0; }

int sb_checked_build(void) {
#ifdef SB_CHECKED
    return 1;
#else
    return 0;
#endif
}

}  // extern "C"
