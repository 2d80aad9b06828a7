// Shared host/device helpers of the CUDA library (sm_100a only).
#pragma once
#include <set>
#include <vector>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "scalebits.h"

// ---- context ---------------------------------------------------------------------
struct SbDeviceState {           // lives in device memory, one per context
    int status;                  // latched sb_status detected on the device
    int where;                   // kernel id that latched it
    unsigned int ticket;         // dynamic tile ids of the look-back scans
    unsigned int pad;            // CTAs of the current look-back launch that have finished
    unsigned long long lb_wait_ns;   // how long a look-back wait may last (default 250 ms)
    unsigned int lb_mute_tile;       // test hook: this tile of a look-back launch publishes nothing
    unsigned int pad2;               //   (0xffffffff: none)
    long long bad_index, bad_limit;  // checked build: the first index that failed its bounds check
};

struct sb_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    int sm_count = 148;
    void* scratch = nullptr;     // arena, grown on demand
    size_t scratch_bytes = 0;
    std::vector<void*> retired;  // outgrown arenas and descriptor buffers, freed with the context
    std::set<const void*> configured;   // kernels whose launch attributes this context has set
    SbDeviceState* dstate = nullptr;
    void* pinned = nullptr;      // small pinned host buffer for read-backs
    size_t pinned_bytes = 0;
    unsigned int* moment_done = nullptr;   // per column chunk: row splits finished (zero between calls)
    int moments_ctas_per_sm = 0;           // resident CTAs per SM of the moments kernel (asked once)
    unsigned int* stats_done = nullptr;    // per tile row / tile column: tiles finished (zero between calls)
    void* lb_mem = nullptr;      // look-back descriptors (context-owned, never in the arena)
    unsigned int lb_max_tiles = 0;
    int64_t launches = 0;
    char err[256] = {0};
};

sb_status sb_fail(sb_ctx* ctx, sb_status st, const char* fmt, ...);
sb_status sb_scratch(sb_ctx* ctx, size_t bytes, void** out);   // whole arena, >= bytes

#define SB_CUDA(ctx, call)                                                              \
    do {                                                                                \
        cudaError_t e__ = (call);                                                       \
        if (e__ != cudaSuccess)                                                         \
            return sb_fail((ctx), SB_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e__)); \
    } while (0)

// one-time launch attribute of a kernel, per context (so per device), not per process
#define SB_FUNC_ATTR(ctx, func, attr, value)                                            \
    do {                                                                                \
        const void* f__ = reinterpret_cast<const void*>(func);                          \
        if (!(ctx)->configured.count(f__)) {                                            \
            SB_CUDA((ctx), cudaFuncSetAttribute(f__, (attr), (value)));                 \
            (ctx)->configured.insert(f__);                                              \
        }                                                                               \
    } while (0)

#define SB_LAUNCHED(ctx)                                                                \
    do {                                                                                \
        (ctx)->launches++;                                                              \
        cudaError_t e__ = cudaGetLastError();                                           \
        if (e__ != cudaSuccess)                                                         \
            return sb_fail((ctx), SB_ERR_CUDA, "launch failed at %s:%d: %s", __FILE__,  \
                           __LINE__, cudaGetErrorString(e__));                          \
    } while (0)

// carve aligned sub-buffers out of the arena
struct Carver {
    char* base; size_t off = 0;
    explicit Carver(void* p) : base(static_cast<char*>(p)) {}
    template <typename T> T* take(size_t n) {
        off = (off + 255) & ~size_t(255);
        T* p = reinterpret_cast<T*>(base + off);
        off += n * sizeof(T);
        return p;
    }
    static size_t need(std::initializer_list<size_t> bytes) {
        size_t t = 0;
        for (size_t b : bytes) t = ((t + 255) & ~size_t(255)) + b;
        return t + 256;
    }
};

bool sb_check_bits(const int* bits, int n_bits);
constexpr int SB_STATS_TILES = 8192;     // 128-wide tiles per axis a reorder call may have
constexpr int SB_MOMENT_CHUNKS = 4096;   // column chunks of 256 a moments call may have (K <= 1M)

enum SbKernelId { SBK_MOMENTS = 1, SBK_STATS, SBK_SCORES, SBK_GATHER, SBK_ARGSORT, SBK_SCAN,
                  SBK_SORT, SBK_ALLOC, SBK_PACK, SBK_GEMM };

// ---- device helpers ----------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ void sb_latch(SbDeviceState* st, int status, int where) {
    if (atomicCAS(&st->status, 0, status) == 0) st->where = where;
}

// Checked build (-DSB_CHECKED, the stand-in for a memory checker): SB_IN_BOUNDS guards the
// accesses whose index comes from data (permutations, sorted lists, prefix sums, record numbers).
// A failing index is latched with the kernel family into the device state (SB_ERR_INVALID,
// surfaced by sb_sync) and the access is skipped; nothing traps.  In the regular build the macro
// is the constant true and costs nothing.
#ifdef SB_CHECKED
__device__ __forceinline__ bool sb_in_bounds(SbDeviceState* st, int where, long long idx, long long limit) {
    if (idx >= 0 && idx < limit) return true;
    if (atomicCAS(&st->status, 0, (int)SB_ERR_INVALID) == 0) { st->where = where; st->bad_index = idx; st->bad_limit = limit; }
    return false;
}
#define SB_IN_BOUNDS(st, where, idx, limit) sb_in_bounds((st), (where), (long long)(idx), (long long)(limit))
#else
#define SB_IN_BOUNDS(st, where, idx, limit) true
#endif

// two bf16 packed in a 32-bit word -> two fp32 (exact)
__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// 128-bit read-only streaming load (weights / activations are read exactly once)
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ld_stream8(const void* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];"
                 : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(unsigned* p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// sm_100a executes fma / add / mul on two fp32 values held in one 64-bit register.  The FP32
// pipe does the same number of lane-operations per clock either way, but the packed form needs
// half the issue slots, which leaves room for the integer, shuffle and load instructions.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk2(float a, float b) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void upk2(f32x2 v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

__device__ __forceinline__ uint32_t u32(__nv_bfloat162 v) { return *reinterpret_cast<uint32_t*>(&v); }
__device__ __forceinline__ __nv_bfloat162 b162(uint32_t v) { return *reinterpret_cast<__nv_bfloat162*>(&v); }

// min and max of a group: NW packed words per lane, `team` lanes (a power of two, aligned)
// per group.  Exact: bf16 min/max, the pair (min, -max) rides one register through the
// shuffles.
template <int NW, int TEAM = 0>
__device__ __forceinline__ void group_minmax(const uint32_t (&w)[NW], int team, float& lo, float& hi) {
    __nv_bfloat162 mn = b162(w[0]), mx = mn;
#pragma unroll
    for (int k = 1; k < NW; ++k) {
        mn = __hmin2(mn, b162(w[k]));
        mx = __hmax2(mx, b162(w[k]));
    }
    const uint32_t mnu = u32(mn), mxu = u32(mx);
    const uint32_t a = u32(__hmin2(mn, b162(__byte_perm(mnu, mnu, 0x1032))));
    const uint32_t b = u32(__hmax2(mx, b162(__byte_perm(mxu, mxu, 0x1032)))) ^ 0x80008000u;
    uint32_t p = (a & 0x0000ffffu) | (b & 0xffff0000u);
    if (TEAM > 0) {
#pragma unroll
        for (int o = TEAM >> 1; o > 0; o >>= 1)
            p = u32(__hmin2(b162(p), b162(__shfl_xor_sync(0xffffffffu, p, o))));
    } else {
        for (int o = team >> 1; o > 0; o >>= 1)
            p = u32(__hmin2(b162(p), b162(__shfl_xor_sync(0xffffffffu, p, o))));
    }
    lo = bf16lo(p);
    hi = -bf16hi(p);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
#endif
