// Full calibration second-moment matrix H = scale * X^T X (bf16 inputs, fp32 accumulation) on
// the 5th-generation tensor cores: the one dense contraction next to this path (Section 3.2: the
// column factor of the sensitivity is the diagonal of this matrix; a sensitivity that keeps the
// cross terms between input channels needs all of it).
//
// One CTA per tile of the upper triangle of H; a tile is 128 rows x 256 columns (a 128 x 128
// tile on every second diagonal position).  D[i][j] = sum_t X[t][i0+i] X[t][j0+j]: both operands
// are slices of X with the CHANNEL index contiguous ("MN-major" operands), so the same tensor map
// serves A and B, and a tile whose 128 rows lie inside its 256 columns loads one slice only.  The
// kernel is bound by the operand traffic from L2 to the SMs (64 tokens of 128 + 256 channels per
// 128 x 256 x 64 contraction; with square 128 x 128 tiles it was 4/3 of that per flop).  Warp 0
// issues TMA loads (cp.async.bulk.tensor, 128-byte swizzle) of 64 tokens x 64 channels into a
// 4-stage shared-memory ring; warp 1 issues tcgen05.mma (M = 128, N = 256, K = 16, kind::f16,
// bf16 -> fp32) into one of two 256-column TMEM accumulators and releases ring stages with
// tcgen05.commit.  The tensor cores' fp32 accumulation drifts on long sums of same-sign terms (the
// diagonal: about 4e-9 per token, relative), so an accumulator only ever takes 512 tokens: warps
// 2-9 drain it with tcgen05.ld into true fp32 registers (128 per thread: half a row of the tile)
// while the other accumulator takes the next 512 tokens, and at the end apply scale / accumulate
// and store the tile and its mirror image.  Every mbarrier wait is bounded: on a time-out the
// kernel latches SB_ERR_TIMEOUT, all roles leave their loops, TMEM is freed and the kernel returns.
#include <cuda.h>

#include "common.cuh"

namespace {

constexpr int GM_TILE = 128;            // rows of a tile (M); a wide tile has 2 * GM_TILE columns (N)
constexpr int GM_BK = 64;               // tokens per ring stage
constexpr int GM_STAGES = 4;
constexpr int GM_CHUNK_KB = 8;          // ring stages (512 tokens) per TMEM accumulator pass
constexpr int GM_TMEM_COLS = 4 * GM_TILE;           // two accumulators of 256 columns
constexpr int GM_ATOM_BYTES = GM_BK * 128;          // 64 tokens x 64 channels of bf16
constexpr int GM_OPERAND_BYTES = 2 * GM_ATOM_BYTES; // 128 channels
constexpr int GM_STAGE_BYTES = 3 * GM_OPERAND_BYTES; // B: 256 channels, then A: 128 channels
constexpr int GM_EPI_WARPS = 8;         // (TMEM lane quarter) x (column half)
constexpr int GM_THREADS = (2 + GM_EPI_WARPS) * 32; // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue
constexpr int GM_SMEM = GM_STAGES * GM_STAGE_BYTES + 1024 /* alignment */ + 256 /* barriers */;
static_assert((2 * GM_STAGES + 4) * 8 + 8 <= 256, "barrier block");
constexpr unsigned long long GM_WAIT_NS = 2000ull * 1000 * 1000;   // give up after 2 s

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long gm_now_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
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
// bounded wait: false (and the abort flag set) if the phase does not complete in time or another
// role has already given up
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag) {
    unsigned long long t0 = 0;
    for (unsigned spins = 0;; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((spins & 255u) == 255u) {
            const unsigned long long now = gm_now_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > GM_WAIT_NS) { *abort_flag = 1; return false; }
        }
    }
}
__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap* map, int x, int y, unsigned bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
// shared-memory matrix descriptor of an MN-major operand in the 128-byte-swizzle layout:
// 8 tokens x 128 bytes per swizzle atom, consecutive 8-token groups 1024 bytes apart (stride
// offset), the next 64 channels GM_ATOM_BYTES further (leading offset)
__device__ __forceinline__ unsigned long long umma_desc_mn_sw128(unsigned addr) {
    unsigned long long d = 0;
    d |= (unsigned long long)((addr >> 4) & 0x3fffu);
    d |= (unsigned long long)((GM_ATOM_BYTES >> 4) & 0x3fff) << 16;
    d |= (unsigned long long)((1024 >> 4) & 0x3fff) << 32;
    d |= 1ull << 46;                       // descriptor version of this architecture
    d |= 2ull << 61;                       // 128-byte swizzle
    return d;
}
// instruction descriptor: fp32 accumulator, bf16 x bf16, both operands MN-major, M = 128, N = n
__host__ __device__ constexpr unsigned gm_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((unsigned)(n >> 3) << 17) |
           ((unsigned)(GM_TILE >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(unsigned tmem_d, unsigned long long a, unsigned long long b,
                                          unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__global__ void __launch_bounds__(GM_THREADS, 1)
gram_kernel(const __grid_constant__ CUtensorMap xmap, int64_t T, int64_t K, int n_tiles, float scale,
            int accumulate, float* __restrict__ H, SbDeviceState* ds) {
    extern __shared__ unsigned char gm_smem_raw[];
    // 1024-byte alignment for the 128-byte swizzle
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(gm_smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + GM_STAGES * GM_STAGE_BYTES);
    // bars[0..S): full, bars[S..2S): empty, then accumulator full[2], accumulator empty[2]
    unsigned long long* acc_full = bars + 2 * GM_STAGES;
    unsigned long long* acc_empty = acc_full + 2;
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // Tiles in units of 128 x 128 blocks (n_tiles per side).  Column pair J = block columns 2J and
    // 2J + 1.  The first n_pairs^2 CTAs take the wide tiles (block row ti <= 2J, pair J), J^2 +
    // ti in the order of the launch; a wide tile with ti == 2J holds the diagonal block (2J, 2J)
    // and its 128 rows are the first half of its columns.  The remaining CTAs take the diagonal
    // blocks (2J + 1, 2J + 1) as narrow tiles of 128 columns: half the work, so they come last.
    const int n_pairs = (n_tiles + 1) / 2;
    const bool wide = (int)blockIdx.x < n_pairs * n_pairs;
    int ti, tj;                         // block row, first block column
    if (wide) {
        int J = (int)sqrtf((float)blockIdx.x);
        while (J * J > (int)blockIdx.x) --J;
        while ((J + 1) * (J + 1) <= (int)blockIdx.x) ++J;
        ti = (int)blockIdx.x - J * J;
        tj = 2 * J;
    } else {
        ti = tj = 2 * ((int)blockIdx.x - n_pairs * n_pairs) + 1;
    }
    const bool a_in_b = ti == tj;       // the rows are the first 128 columns: one slice serves both
    const int num_kb = (int)((T + GM_BK - 1) / GM_BK);
    const int num_chunks = (num_kb + GM_CHUNK_KB - 1) / GM_CHUNK_KB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < GM_STAGES; ++s) {
            mbar_init(smem_u32(bars + s), 1);
            mbar_init(smem_u32(bars + GM_STAGES + s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(acc_full + b), 1);
            mbar_init(smem_u32(acc_empty + b), wide ? GM_EPI_WARPS : GM_EPI_WARPS / 2);   // one arrival per draining warp
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        // 512 TMEM columns: two fp32 accumulators of 128 lanes x 256 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(GM_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_d = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---- producer: TMA loads of the channel slices (out-of-range channels and tokens read as
            // zero), 64 tokens per stage ------------------------------------------------------------
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % GM_STAGES;
                const unsigned ph = (unsigned)(kb / GM_STAGES) & 1u;
                if (!mbar_wait(smem_u32(bars + GM_STAGES + s), ph ^ 1u, abort_flag)) break;
                const unsigned full = smem_u32(bars + s);
                const int b_atoms = wide ? 4 : 2, a_atoms = a_in_b ? 0 : 2;
                mbar_expect_tx(full, (unsigned)((b_atoms + a_atoms) * GM_ATOM_BYTES));
                const unsigned b = smem_u32(smem + s * GM_STAGE_BYTES);
                const int t0 = kb * GM_BK;
                for (int u = 0; u < b_atoms; ++u)
                    tma_load_2d(b + u * GM_ATOM_BYTES, &xmap, tj * GM_TILE + 64 * u, t0, full);
                for (int u = 0; u < a_atoms; ++u)
                    tma_load_2d(b + 2 * GM_OPERAND_BYTES + u * GM_ATOM_BYTES, &xmap, ti * GM_TILE + 64 * u, t0, full);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issue: 4 instructions of K = 16 tokens per stage, 8 stages per accumulator ---
            bool ok = true;
            const unsigned idesc = gm_idesc(wide ? 2 * GM_TILE : GM_TILE);
            for (int c = 0; c < num_chunks && ok; ++c) {
                const int ab = c & 1;
                // the epilogue has drained this accumulator's previous pass
                ok = mbar_wait(smem_u32(acc_empty + ab), ((unsigned)(c >> 1) & 1u) ^ 1u, abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const unsigned acc = tmem_d + (unsigned)(ab * 2 * GM_TILE);
                const int kb_end = min(num_kb, (c + 1) * GM_CHUNK_KB);
                for (int kb = c * GM_CHUNK_KB; kb < kb_end; ++kb) {
                    const int s = kb % GM_STAGES;
                    const unsigned ph = (unsigned)(kb / GM_STAGES) & 1u;
                    ok = mbar_wait(smem_u32(bars + s), ph, abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const unsigned b = smem_u32(smem + s * GM_STAGE_BYTES);
                    const unsigned a = a_in_b ? b : b + 2 * GM_OPERAND_BYTES;
#pragma unroll
                    for (int ks = 0; ks < GM_BK / 16; ++ks) {
                        // 16 tokens = two 8-token groups = 2048 bytes further along K
                        const unsigned long long da = umma_desc_mn_sw128(a + ks * 2048);
                        const unsigned long long db = umma_desc_mn_sw128(b + ks * 2048);
                        umma_bf16(acc, da, db, idesc, (kb > c * GM_CHUNK_KB || ks > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(bars + GM_STAGES + s));    // the stage is free when these MMAs are done
                }
                umma_commit(smem_u32(acc_full + ab));                // this pass of the accumulator is complete
            }
        }
    } else {
        // ---- epilogue: warp w reads TMEM lanes 32 (w % 4) .. + 31 of column half (w - 2) / 4; a
        // thread keeps half a row of the tile (128 columns) in fp32 registers across the accumulator
        // passes.  A narrow tile has no second half: those four warps have nothing to do. ---------
        const int q = warp & 3, half = (warp - 2) >> 2;
        if (wide || half == 0) {
            float row[GM_TILE];
#pragma unroll
            for (int c = 0; c < GM_TILE; ++c) row[c] = 0.f;
            bool ok = true;
            for (int c = 0; c < num_chunks && ok; ++c) {
                const int ab = c & 1;
                // the loads below are warp-collective: the outcome of the wait must be uniform
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(acc_full + ab), (unsigned)(c >> 1) & 1u, abort_flag));
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (int c0 = 0; c0 < GM_TILE; c0 += 32) {
                    unsigned r[32];
                    const unsigned taddr = tmem_d + ((unsigned)(q * 32) << 16) +
                                           (unsigned)(ab * 2 * GM_TILE + half * GM_TILE + c0);
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
                          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
                          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]),
                          "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
                          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                        : "r"(taddr)
                        : "memory");
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int k = 0; k < 32; ++k) row[c0 + k] += __uint_as_float(r[k]);
                }
                // this accumulator may take its next pass
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0)
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(acc_empty + ab)) : "memory");
            }
            if (ok) {
                const int bc = tj + half;                                      // block column of this half
                const bool diagonal = bc == ti;
                const int64_t i = (int64_t)ti * GM_TILE + q * 32 + lane;       // row of H held by this thread
                // K % 8 == 0: four consecutive columns are inside the matrix or outside together
#pragma unroll
                for (int c = 0; c < GM_TILE; c += 4) {
                    const int64_t j = (int64_t)bc * GM_TILE + c;
                    if (i < K && j < K) {
                        float4 v = make_float4(scale * row[c], scale * row[c + 1], scale * row[c + 2], scale * row[c + 3]);
                        float4* dst = reinterpret_cast<float4*>(H + i * K + j);
                        if (accumulate) {
                            const float4 o = *dst;
                            v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                        }
                        *dst = v;
                        if (!diagonal) {                      // mirror image; lanes = consecutive i: coalesced
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                float* md = H + (j + u) * K + i;
                                const float m = scale * row[c + u];
                                *md = accumulate ? *md + m : m;
                            }
                        }
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(GM_TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag) sb_latch(ds, SB_ERR_TIMEOUT, SBK_MOMENTS);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

}  // namespace

extern "C" sb_status sb_calib_gram(sb_ctx* ctx, const void* X, int64_t T, int64_t K, int64_t ldx, float* H,
                                   int accumulate, float scale) {
    if (!ctx) return SB_ERR_INVALID;
    if (!H || T < 0 || K <= 0 || (T > 0 && !X)) return sb_fail(ctx, SB_ERR_INVALID, "gram: null or empty");
    if (K % 8 || ldx % 8 || ldx < K || (reinterpret_cast<uintptr_t>(X) & 15))
        return sb_fail(ctx, SB_ERR_SHAPE, "gram: K %% 8 == 0, ldx %% 8 == 0, ldx >= K and a 16-byte aligned base");
    if (T >= (1ll << 31) || K >= (1ll << 31)) return sb_fail(ctx, SB_ERR_SHAPE, "gram: T and K must fit 31 bits");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    if (T == 0) {
        if (!accumulate) SB_CUDA(ctx, cudaMemsetAsync(H, 0, sizeof(float) * (size_t)K * K, ctx->stream));
        return SB_OK;
    }
    static EncodeTiledFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        SB_CUDA(ctx, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (!fn || qres != cudaDriverEntryPointSuccess)
            return sb_fail(ctx, SB_ERR_CUDA, "gram: the driver does not export cuTensorMapEncodeTiled");
        encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    // X as a 2-D tensor (channels innermost); boxes of 64 channels x 64 tokens, 128-byte swizzle,
    // out-of-range channels and tokens read as zero
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)T};
    const cuuint64_t strides[1] = {(cuuint64_t)ldx * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)GM_BK};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(X), dims, strides, box,
                              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return sb_fail(ctx, SB_ERR_CUDA, "gram: cuTensorMapEncodeTiled failed (%d)", (int)r);
    // wide tiles (block row ti <= 2J, column pair J), then the diagonal blocks at odd positions
    const int n_tiles = (int)((K + GM_TILE - 1) / GM_TILE);
    const long long n_pairs = (n_tiles + 1) / 2;
    const long long n_ctas = n_pairs * n_pairs + n_tiles / 2;
    if (n_ctas >= (1ll << 31)) return sb_fail(ctx, SB_ERR_SHAPE, "gram: too many tiles");
    SB_FUNC_ATTR(ctx, gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GM_SMEM);
    gram_kernel<<<(unsigned)n_ctas, GM_THREADS, GM_SMEM, ctx->stream>>>(map, T, K, n_tiles, scale, accumulate, H,
                                                                       ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}
