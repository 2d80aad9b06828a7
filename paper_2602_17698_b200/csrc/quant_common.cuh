// Pieces the weight-tile kernels share (reorder statistics, gather, block scores): the constants
// of the fp32 round-to-nearest quantiser, the per-candidate constants passed by value, asynchronous
// 16-byte copies.
#pragma once
#include "common.cuh"

constexpr int TILE_COLS = 128;
constexpr float RNE_MAGIC = 12582912.f;        // 1.5 * 2^23: fma(x, s, MAGIC) - MAGIC = rint(x*s)
constexpr float MIN_RANGE = 7.52316385e-37f;   // 2^-120: below this a group counts as constant

struct __align__(8) BitsArg {
    float2 q2[8];        // (qmax, qmax), qmax = 2^b - 1, as a packed fp32 pair
    float2 niq2[8];      // (-1/qmax, -1/qmax)
    float qmax[8];
    float inv_qmax[8];
    int bits[8];
};

__device__ __forceinline__ float rcp_approx(float x) {
    float r;
    asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// ---- asynchronous 16-byte copies global -> shared (L2 only, no register staging) -----------
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }


inline BitsArg make_bits(const int* bits, int n) {
    BitsArg ba{};
    for (int l = 0; l < 8; ++l) {
        const int b = l < n ? bits[l] : 1;
        ba.bits[l] = b;
        ba.qmax[l] = (float)((1 << b) - 1);
        ba.inv_qmax[l] = 1.0f / (float)((1 << b) - 1);
        ba.q2[l] = make_float2(ba.qmax[l], ba.qmax[l]);
        ba.niq2[l] = make_float2(-ba.inv_qmax[l], -ba.inv_qmax[l]);
    }
    return ba;
}

inline bool valid_group(int g) { return g == 16 || g == 32 || g == 64 || g == 128; }

