// Block error table with the FULL calibration second-moment matrix (Section 3.2 with the cross
// terms between input channels kept): for block i with columns J and candidate b_l,
//     E[i][l] = sum_r d_r H'_JJ d_r^T = < H'_JJ , D^T D >,     D = (W' - Q_{b_l}(W'))[rows of i, J],
// where H' is H = X^T X / T in the permuted column order.  The 128 x 128 Gram matrix D^T D of
// every (block, candidate) is a tensor-core contraction over the block's 128 rows; the inner
// product with H'_JJ is the epilogue.  bf16 alone is too coarse for D, so D is split into two
// bf16 terms D = D0 + D1 and G = D0^T D0 + D0^T D1 + (D0^T D1)^T (the D1^T D1 term is 2^-16 of
// G); with H symmetric, E = <H, D0^T D0> + 2 <H, D0^T D1>: two accumulators per candidate.
//
// One persistent CTA per SM, warp-specialised:
//   warps 4-11 (256 threads, one half row of the block each): quantise the block at candidate l
//     (codes by the binary64 sequence, residual in fp32 with a two-float grid step), split it into
//     two bf16 terms and write them into a shared-memory stage in the MN-major 128-byte-swizzle
//     layout the tensor cores read (the layout a TMA load of the tile would produce);
//   warp 12 (one thread): 2 x 8 tcgen05.mma (M = N = 128, K = 16, bf16 -> fp32) per candidate
//     into one of two TMEM stages of 2 x 128 columns, tcgen05.commit to free the shared-memory
//     stage and to publish the accumulators;
//   warps 0-3: tcgen05.ld of a row of both accumulators, inner product with the row of H'_JJ,
//     sum over the 128 rows in a fixed order, err / gain.
// Two shared-memory stages and two TMEM stages keep the three roles one candidate apart.  Every
// mbarrier wait is bounded; on a time-out the kernel latches SB_ERR_TIMEOUT and all roles leave.
#include "common.cuh"

sb_status sb_gather_bf16(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                         const int32_t* rp, const int32_t* cp, void* out);

namespace {

constexpr int FS_N = 128;                              // block rows = block columns = 128
constexpr int FS_ATOM_BYTES = FS_N * 128;              // 128 rows x 64 columns of bf16
constexpr int FS_TILE_BYTES = 2 * FS_ATOM_BYTES;       // one 128 x 128 bf16 operand
constexpr int FS_STAGE_BYTES = 2 * FS_TILE_BYTES;      // D0 and D1
constexpr int FS_STAGES = 2;
constexpr int FS_EPI_WARPS = 4, FS_PROD_WARPS = 8;
constexpr int FS_PROD_THREADS = FS_PROD_WARPS * 32;
constexpr int FS_THREADS = (FS_EPI_WARPS + FS_PROD_WARPS + 1) * 32;
constexpr int FS_TMEM_COLS = 512;                      // 2 stages x 2 accumulators x 128 columns
constexpr int FS_SMEM = FS_STAGES * FS_STAGE_BYTES + 1024 /* alignment */ + 512 /* barriers, sums */;
constexpr unsigned long long FS_WAIT_NS = 2000ull * 1000 * 1000;
constexpr double FS_MAGIC64 = 6755399441055744.0;      // 1.5 * 2^52: low word of (t + MAGIC) = rint(t)
constexpr unsigned FS_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                              ((FS_N >> 3) << 17) | ((FS_N >> 4) << 24);

struct FsBits { float qmax[8]; float inv_qmax[8]; int bits[8]; };

__device__ __forceinline__ unsigned fs_smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long fs_now_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void fs_mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fs_mbar_arrive(unsigned bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool fs_mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool fs_mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag) {
    unsigned long long t0 = 0;
    for (unsigned spins = 0;; ++spins) {
        if (fs_mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((spins & 255u) == 255u) {
            const unsigned long long now = fs_now_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > FS_WAIT_NS) { *abort_flag = 1; return false; }
        }
    }
}
// MN-major operand, 128-byte swizzle: rows of 128 bytes (64 columns), 8-row groups 1024 bytes
// apart, the other 64 columns FS_ATOM_BYTES further
__device__ __forceinline__ unsigned long long fs_desc(unsigned addr) {
    unsigned long long d = 0;
    d |= (unsigned long long)((addr >> 4) & 0x3fffu);
    d |= (unsigned long long)((FS_ATOM_BYTES >> 4) & 0x3fff) << 16;
    d |= (unsigned long long)((1024 >> 4) & 0x3fff) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
__device__ __forceinline__ void fs_mma(unsigned tmem_d, unsigned long long a, unsigned long long b, unsigned acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a), "l"(b), "r"(FS_IDESC), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void fs_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fs_tmem_ld32(unsigned taddr, float (&v)[32]) {
    unsigned r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int k = 0; k < 32; ++k) v[k] = __uint_as_float(r[k]);
}

// H'_JJ of every block column: hblk[bj][a][b] = H[cp[J0 + a]][cp[J0 + b]]
__global__ void gather_hblocks_kernel(const float* __restrict__ H, int64_t C, const int32_t* __restrict__ cp,
                                      float* __restrict__ hblk) {
    const int64_t j0 = (int64_t)blockIdx.x * FS_N;
    for (int idx = threadIdx.x; idx < FS_N * FS_N; idx += blockDim.x) {
        const int a = idx / FS_N, b = idx % FS_N;
        const int64_t ja = cp ? cp[j0 + a] : j0 + a, jb = cp ? cp[j0 + b] : j0 + b;
        hblk[((int64_t)blockIdx.x * FS_N + a) * FS_N + b] = H[ja * C + jb];
    }
}

__global__ void __launch_bounds__(FS_THREADS, 1)
full_scores_kernel(const __nv_bfloat16* __restrict__ W, int64_t ldw, const float* __restrict__ hblk,
                   int group, FsBits fb, int L, int64_t n_blocks, int64_t n_block_cols,
                   float* __restrict__ err, float* __restrict__ gain, SbDeviceState* ds) {
    extern __shared__ unsigned char fs_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(fs_smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + FS_STAGES * FS_STAGE_BYTES);
    unsigned long long* smem_full = bars;             // [2] producers -> MMA
    unsigned long long* smem_empty = bars + 2;        // [2] MMA -> producers
    unsigned long long* tmem_full = bars + 4;         // [2] MMA -> epilogue
    unsigned long long* tmem_empty = bars + 6;        // [2] epilogue -> MMA
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(bars + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* red = reinterpret_cast<float*>(tmem_slot + 4);          // [2][4] warp sums of the epilogue
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            fs_mbar_init(fs_smem_u32(smem_full + s), FS_PROD_THREADS);
            fs_mbar_init(fs_smem_u32(smem_empty + s), 1);
            fs_mbar_init(fs_smem_u32(tmem_full + s), 1);
            fs_mbar_init(fs_smem_u32(tmem_empty + s), FS_EPI_WARPS);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == FS_EPI_WARPS + FS_PROD_WARPS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(fs_smem_u32(tmem_slot)),
                     "r"(FS_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_base = *tmem_slot;

    if (warp >= FS_EPI_WARPS && warp < FS_EPI_WARPS + FS_PROD_WARPS) {
        // ---- producers: thread p owns columns [64 half, 64 half + 64) of row p / 2 -----------------
        const int p = threadIdx.x - FS_EPI_WARPS * 32;
        const int r = p >> 1, half = p & 1;
        const int gpc = group >> 3;                          // 16-byte chunks (8 columns) per group
        long long item = 0;
        bool ok = true;
        for (int64_t blk = blockIdx.x; blk < n_blocks && ok; blk += gridDim.x) {
            const int64_t bi = blk / n_block_cols, bj = blk - bi * n_block_cols;
            const uint4* src = reinterpret_cast<const uint4*>(W + (bi * FS_N + r) * ldw + bj * FS_N + half * 64);
            uint32_t wv[32];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 x = __ldg(src + c);
                wv[4 * c] = x.x; wv[4 * c + 1] = x.y; wv[4 * c + 2] = x.z; wv[4 * c + 3] = x.w;
            }
            // group minimum and maximum per 8-column chunk (exact bf16 min / max); crange holds the
            // maximum: the range is taken in binary64, where the difference is exact
            float clo[8], crange[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                __nv_bfloat162 mn = b162(wv[4 * c]), mx = mn;
#pragma unroll
                for (int k = 1; k < 4; ++k) { mn = __hmin2(mn, b162(wv[4 * c + k])); mx = __hmax2(mx, b162(wv[4 * c + k])); }
                clo[c] = fminf(bf16lo(u32(mn)), bf16hi(u32(mn)));
                crange[c] = fmaxf(bf16lo(u32(mx)), bf16hi(u32(mx)));      // the maximum for now
            }
            // combine the chunks of a group (2, 4 or 8 of them; 16 with the partner thread)
#pragma unroll
            for (int span = 1; span < 8; span <<= 1) {
                if (span < gpc) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float l2 = clo[c ^ span], h2 = crange[c ^ span];
                        clo[c] = fminf(clo[c], l2);            // pairs exchange symmetrically: order is irrelevant
                        crange[c] = fmaxf(crange[c], h2);
                    }
                }
            }
            if (gpc == 16) {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    clo[c] = fminf(clo[c], __shfl_xor_sync(0xffffffffu, clo[c], 1));
                    crange[c] = fmaxf(crange[c], __shfl_xor_sync(0xffffffffu, crange[c], 1));
                }
            }
            for (int l = 0; l < L && ok; ++l, ++item) {
                const int s = (int)(item & 1);
                // uniform per warp: the shuffles of the next block need all lanes
                ok = __all_sync(0xffffffffu, fs_mbar_wait(fs_smem_u32(smem_empty + s),
                                                          ((unsigned)(item >> 1) & 1u) ^ 1u, abort_flag));
                if (!ok) break;
                unsigned char* d0 = smem + s * FS_STAGE_BYTES + half * FS_ATOM_BYTES + r * 128;
                unsigned char* d1 = d0 + FS_TILE_BYTES;
                // The quadratic form has cross terms, so it jumps where a code flips, and exact
                // rounding ties are common for bf16 weights: the codes follow the binary64 sequence
                //   inv = qmax / range; q = rint((v - lo) * inv)
                // literally (one division per group), the residual is taken in fp32 with the grid
                // step as a two-float sum.
                const float qmax = fb.qmax[l], inv_qmax = fb.inv_qmax[l];
                const int cpg = gpc < 8 ? gpc : 8;               // chunks of this thread per group
                double dlo = 0.0, inv64 = 0.0;
                float lo = 0.f, ns = 0.f, ns_lo = 0.f;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    if ((c & (cpg - 1)) == 0) {                   // first chunk of a group
                        lo = clo[c];
                        dlo = (double)lo;
                        const double range64 = __dsub_rn((double)crange[c], dlo);      // exact
                        const float range = (float)range64;
                        const bool live = range64 != 0.0;
                        inv64 = live ? __ddiv_rn((double)qmax, range64) : 0.0;
                        ns = live ? -(range * inv_qmax) : 0.f;
                        ns_lo = live ? -(fmaf(ns, qmax, range) * inv_qmax) : 0.f;
                    }
                    uint32_t h[4], lw[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float w0 = bf16lo(wv[4 * c + k]), w1 = bf16hi(wv[4 * c + k]);
                        const double t0 = __dmul_rn(__dsub_rn((double)w0, dlo), inv64);
                        const double t1 = __dmul_rn(__dsub_rn((double)w1, dlo), inv64);
                        const unsigned qi0 = (unsigned)__double2loint(__dadd_rn(t0, FS_MAGIC64));
                        const unsigned qi1 = (unsigned)__double2loint(__dadd_rn(t1, FS_MAGIC64));
                        const float q0 = __uint_as_float(0x4B000000u | qi0) - 8388608.f;     // exact int -> float
                        const float q1 = __uint_as_float(0x4B000000u | qi1) - 8388608.f;
                        const float v0 = w0 - lo, v1 = w1 - lo;
                        const float e0 = fmaf(q0, ns_lo, fmaf(q0, ns, v0)), e1 = fmaf(q1, ns_lo, fmaf(q1, ns, v1));
                        const __nv_bfloat162 hi2 = __floats2bfloat162_rn(e0, e1);
                        const float2 hf = __bfloat1622float2(hi2);
                        const __nv_bfloat162 lo2 = __floats2bfloat162_rn(e0 - hf.x, e1 - hf.y);
                        h[k] = u32(hi2); lw[k] = u32(lo2);
                    }
                    const int sw = (c ^ (r & 7)) * 16;            // the 128-byte swizzle of the layout
                    *reinterpret_cast<uint4*>(d0 + sw) = make_uint4(h[0], h[1], h[2], h[3]);
                    *reinterpret_cast<uint4*>(d1 + sw) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                }
                // the tensor cores read shared memory through the async proxy
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                fs_mbar_arrive(fs_smem_u32(smem_full + s));
            }
        }
    } else if (warp == FS_EPI_WARPS + FS_PROD_WARPS) {
        if (lane == 0) {
            // ---- MMA issue ---------------------------------------------------------------------------
            long long item = 0;
            bool ok = true;
            for (int64_t blk = blockIdx.x; blk < n_blocks && ok; blk += gridDim.x) {
                for (int l = 0; l < L && ok; ++l, ++item) {
                    const int s = (int)(item & 1);
                    const unsigned ph = (unsigned)(item >> 1) & 1u;
                    ok = fs_mbar_wait(fs_smem_u32(smem_full + s), ph, abort_flag) &&
                         fs_mbar_wait(fs_smem_u32(tmem_empty + s), ph ^ 1u, abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const unsigned a0 = fs_smem_u32(smem + s * FS_STAGE_BYTES), a1 = a0 + FS_TILE_BYTES;
                    const unsigned acc00 = tmem_base + (unsigned)(s * 2 * FS_N), acc01 = acc00 + FS_N;
#pragma unroll
                    for (int ks = 0; ks < FS_N / 16; ++ks) {
                        const unsigned long long d0 = fs_desc(a0 + ks * 2048), d1 = fs_desc(a1 + ks * 2048);
                        fs_mma(acc00, d0, d0, ks > 0 ? 1u : 0u);      // D0^T D0
                        fs_mma(acc01, d0, d1, ks > 0 ? 1u : 0u);      // D0^T D1
                    }
                    fs_commit(fs_smem_u32(smem_empty + s));
                    fs_commit(fs_smem_u32(tmem_full + s));
                }
            }
        }
    } else {
        // ---- epilogue: thread j holds row j of both accumulators ------------------------------------
        const int q = warp, j = q * 32 + lane;
        long long item = 0;
        bool ok = true;
        float e_prev = 0.f;
        for (int64_t blk = blockIdx.x; blk < n_blocks && ok; blk += gridDim.x) {
            const int64_t bj = blk % n_block_cols;
            const float4* hrow = reinterpret_cast<const float4*>(hblk + (bj * FS_N + j) * FS_N);
            for (int l = 0; l < L && ok; ++l, ++item) {
                const int s = (int)(item & 1);
                // a warp that gives up still meets the others at this item's barrier; everybody
                // leaves together right after it
                const bool got = __all_sync(0xffffffffu,
                                            fs_mbar_wait(fs_smem_u32(tmem_full + s), (unsigned)(item >> 1) & 1u, abort_flag));
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                float acc = 0.f;
#pragma unroll 1
                for (int c0 = 0; got && c0 < FS_N; c0 += 32) {
                    float g00[32], g01[32];
                    const unsigned t = tmem_base + ((unsigned)(q * 32) << 16) + (unsigned)(s * 2 * FS_N + c0);
                    fs_tmem_ld32(t, g00);
                    fs_tmem_ld32(t + FS_N, g01);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const float4 hv = __ldg(hrow + (c0 >> 2) + k);
                        acc = fmaf(hv.x, fmaf(2.f, g01[4 * k], g00[4 * k]), acc);
                        acc = fmaf(hv.y, fmaf(2.f, g01[4 * k + 1], g00[4 * k + 1]), acc);
                        acc = fmaf(hv.z, fmaf(2.f, g01[4 * k + 2], g00[4 * k + 2]), acc);
                        acc = fmaf(hv.w, fmaf(2.f, g01[4 * k + 3], g00[4 * k + 3]), acc);
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) fs_mbar_arrive(fs_smem_u32(tmem_empty + s));
                // the 128 rows, in a fixed order
                acc = warp_sum(acc);
                if (lane == 0) red[(item & 1) * 4 + q] = acc;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (*abort_flag) { ok = false; break; }
                if (threadIdx.x == 0) {
                    const float* rr = red + (item & 1) * 4;
                    const float e = (rr[0] + rr[1]) + (rr[2] + rr[3]);
                    if (!isfinite(e)) sb_latch(ds, SB_ERR_NONFINITE, SBK_SCORES);
                    err[blk * L + l] = e;
                    if (gain && l > 0)
                        gain[blk * (L - 1) + l - 1] =
                            (e_prev - e) / ((float)(fb.bits[l] - fb.bits[l - 1]) * (float)(FS_N * FS_N));
                    e_prev = e;
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == FS_EPI_WARPS + FS_PROD_WARPS)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(FS_TMEM_COLS) : "memory");
    if (threadIdx.x == 0 && *abort_flag) sb_latch(ds, SB_ERR_TIMEOUT, SBK_SCORES);
}

}  // namespace

extern "C" sb_status sb_block_scores_full(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                                          const int32_t* row_perm, const int32_t* col_perm, const float* H,
                                          int br, int bc, int group, const int* bits, int n_bits, float* err,
                                          float* gain, void* W_perm_out) {
    if (!ctx) return SB_ERR_INVALID;
    if (!W || !H || !err || R <= 0 || C <= 0) return sb_fail(ctx, SB_ERR_INVALID, "full scores: null or empty");
    if (!sb_check_bits(bits, n_bits)) return sb_fail(ctx, SB_ERR_INVALID, "full scores: bits must be ascending in 1..8");
    const bool g_ok = group == 16 || group == 32 || group == 64 || group == 128;
    if (br != FS_N || bc != FS_N || !g_ok || R % FS_N || C % FS_N || ldw % 8 || ldw < C ||
        (reinterpret_cast<uintptr_t>(W) & 15))
        return sb_fail(ctx, SB_ERR_SHAPE, "full scores: blocks of 128 x 128 tiling the matrix, group in {16,32,64,128}");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const int64_t nbc = C / FS_N, n_blocks = (R / FS_N) * nbc;
    const bool need_copy = row_perm || col_perm || W_perm_out;
    void* arena;
    sb_status st = sb_scratch(ctx, Carver::need({(size_t)nbc * FS_N * FS_N * 4,
                                                 (need_copy && !W_perm_out) ? (size_t)R * C * 2 : 0}), &arena);
    if (st != SB_OK) return st;
    Carver cv(arena);
    float* hblk = cv.take<float>((size_t)nbc * FS_N * FS_N);
    const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(W);
    int64_t ld = ldw;
    if (need_copy) {
        void* dst = W_perm_out ? W_perm_out : static_cast<void*>(cv.take<unsigned char>((size_t)R * C * 2));
        st = sb_gather_bf16(ctx, W, R, C, ldw, row_perm, col_perm, dst);
        if (st != SB_OK) return st;
        src = static_cast<const __nv_bfloat16*>(dst);
        ld = C;
    }
    gather_hblocks_kernel<<<(unsigned)nbc, 256, 0, ctx->stream>>>(H, C, col_perm, hblk);
    SB_LAUNCHED(ctx);
    FsBits fb{};
    for (int l = 0; l < 8; ++l) {
        const int b = l < n_bits ? bits[l] : 1;
        fb.bits[l] = b;
        fb.qmax[l] = (float)((1 << b) - 1);
        fb.inv_qmax[l] = 1.0f / (float)((1 << b) - 1);
    }
    SB_FUNC_ATTR(ctx, full_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FS_SMEM);
    const int64_t grid = n_blocks < ctx->sm_count ? n_blocks : ctx->sm_count;
    full_scores_kernel<<<(unsigned)grid, FS_THREADS, FS_SMEM, ctx->stream>>>(src, ld, hblk, group, fb, n_bits,
                                                                            n_blocks, nbc, err, gain, ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}
