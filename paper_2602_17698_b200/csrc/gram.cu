// Full calibration second-moment matrix H = scale * X^T X (bf16 inputs, fp32 accumulation) on
// the 5th-generation tensor cores: the one dense contraction next to this path (Section 3.2: the
// column factor of the sensitivity is the diagonal of this matrix; a sensitivity that keeps the
// cross terms between input channels needs all of it).
//
// One pair of CTAs (a cluster of two, on the two SMs of a TPC) per 256 x 256 tile of the upper
// triangle of H, contracted by tcgen05.mma.cta_group::2 (M = 256 over the pair, N = 256, K = 16,
// kind::f16, bf16 -> fp32).  D[i][j] = sum_t X[t][i0+i] X[t][j0+j]: both operands are slices of X
// with the CHANNEL index contiguous ("MN-major" operands), so one tensor map serves A and B.  The
// kernel is bound by the operand traffic from L2 to the SMs; with the pair, CTA r loads only its
// 128 rows of A and its 128 columns of B (64 tokens x 256 channels per 128 x 256 x 64 of work:
// half of what square 128 x 128 tiles of single CTAs need per flop), and a diagonal tile loads
// one slice for both.  In each CTA warp 0 issues the TMA loads (cp.async.bulk.tensor, 128-byte
// swizzle, 64 tokens x 64 channels) into its own 6-stage shared-memory ring; their bytes are
// counted on the LEADER's (rank 0) "full" barrier.  Warp 1 of the leader issues the contractions
// into one of two 256-column TMEM accumulators (each CTA holds its 128 rows) and releases ring
// stages / publishes accumulators in both CTAs with tcgen05.commit to both barriers.  The tensor
// cores' fp32 accumulation drifts on long sums of same-sign terms (the diagonal: about 4e-9 per
// token, relative), so an accumulator only ever takes 512 tokens: warps 2-9 of either CTA drain
// it with tcgen05.ld into true fp32 registers (128 per thread: half a row) while the other
// accumulator takes the next 512 tokens (they report to the leader's "accumulator empty"
// barrier, the peer through its cluster address), and at the end apply scale / accumulate and
// store the tile and its mirror image.  Every mbarrier wait is bounded: on a time-out the kernel
// latches SB_ERR_TIMEOUT, all roles leave their loops, the pair meets at the cluster barrier,
// TMEM is freed and the kernel returns.
#include <cuda.h>

#include "common.cuh"

namespace {

constexpr int GM_TILE = 128;            // rows of H per CTA; the pair's tile is 256 x 256
constexpr int GM_BK = 64;               // tokens per ring stage
constexpr int GM_STAGES = 6;
constexpr int GM_CHUNK_KB = 8;          // ring stages (512 tokens) per TMEM accumulator pass
constexpr int GM_TMEM_COLS = 4 * GM_TILE;           // two accumulators of 256 columns
constexpr int GM_ATOM_BYTES = GM_BK * 128;          // 64 tokens x 64 channels of bf16
constexpr int GM_OPERAND_BYTES = 2 * GM_ATOM_BYTES; // 128 channels
constexpr int GM_STAGE_BYTES = 2 * GM_OPERAND_BYTES; // this CTA's 128 columns of B, then its 128 rows of A
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
// Load into this CTA's shared memory; the bytes are counted on the barrier `bar`, which may be
// the pair leader's (cluster address).
__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap* map, int x, int y, unsigned bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
// cluster address of the same shared-memory offset in the CTA of rank `rank`
__device__ __forceinline__ unsigned cluster_addr(unsigned own, unsigned rank) {
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(own), "r"(rank));
    return r;
}
__device__ __forceinline__ unsigned cluster_ctarank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
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
// instruction descriptor: fp32 accumulator, bf16 x bf16, both operands MN-major, M = 256 over the
// pair, N = 256
constexpr unsigned GM_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                              ((unsigned)((2 * GM_TILE) >> 3) << 17) | ((unsigned)((2 * GM_TILE) >> 4) << 24);

// issued by one thread of the leader; reads A and B at the same offsets of both CTAs' shared memory
__device__ __forceinline__ void umma_bf16(unsigned tmem_d, unsigned long long a, unsigned long long b,
                                          unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a), "l"(b), "r"(GM_IDESC), "r"(accumulate)
        : "memory");
}
// arrives on the barrier at this offset in BOTH CTAs once the contractions issued so far are done
__device__ __forceinline__ void umma_commit_pair(unsigned bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((unsigned short)3) : "memory");
}

__global__ void __launch_bounds__(GM_THREADS, 1)
gram_kernel(const __grid_constant__ CUtensorMap xmap, int64_t T, int64_t K, float scale, int accumulate,
            float* __restrict__ H, SbDeviceState* ds) {
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

    // Tile (I <= J) of the upper triangle in units of 256 channels from the cluster's number:
    // column by column, J (J + 1) / 2 + I.
    const unsigned rank = cluster_ctarank();           // 0: leader
    const int cl = (int)(blockIdx.x >> 1);
    int J = (int)((sqrtf(8.f * (float)cl + 1.f) - 1.f) * 0.5f);
    while (J * (J + 1) / 2 > cl) --J;
    while ((J + 1) * (J + 2) / 2 <= cl) ++J;
    const int I = cl - J * (J + 1) / 2;
    const bool a_in_b = I == J;                        // diagonal tile: this CTA's rows are its columns
    const int row0 = (2 * I + (int)rank) * GM_TILE;    // this CTA's 128 rows of H = its channels of A
    const int col0 = (2 * J + (int)rank) * GM_TILE;    // its 128 channels of B (tile columns 128 rank ...)
    const int num_kb = (int)((T + GM_BK - 1) / GM_BK);
    const int num_chunks = (num_kb + GM_CHUNK_KB - 1) / GM_CHUNK_KB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < GM_STAGES; ++s) {
            mbar_init(smem_u32(bars + s), 1);                      // full: the leader's expect_tx arrival
            mbar_init(smem_u32(bars + GM_STAGES + s), 1);          // empty: the leader's commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(acc_full + b), 1);
            mbar_init(smem_u32(acc_empty + b), 2 * GM_EPI_WARPS); // one arrival per draining warp of the pair
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        // 512 TMEM columns in each CTA: two fp32 accumulators of 128 lanes x 256 columns
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(GM_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    cluster_sync_all();                 // barriers of both CTAs exist before anything arrives on them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_d = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---- producer: TMA loads of this CTA's channel slices (out-of-range channels and tokens
            // read as zero), 64 tokens per stage; bytes of both CTAs are counted by the leader ------
            const unsigned stage_bytes = (unsigned)(a_in_b ? GM_OPERAND_BYTES : GM_STAGE_BYTES);
            for (int kb = 0; kb < num_kb; ++kb) {
                const int s = kb % GM_STAGES;
                const unsigned ph = (unsigned)(kb / GM_STAGES) & 1u;
                if (!mbar_wait(smem_u32(bars + GM_STAGES + s), ph ^ 1u, abort_flag)) break;
                const unsigned full_leader = cluster_addr(smem_u32(bars + s), 0);
                if (rank == 0) mbar_expect_tx(smem_u32(bars + s), 2 * stage_bytes);
                const unsigned b = smem_u32(smem + s * GM_STAGE_BYTES);
                const int t0 = kb * GM_BK;
                tma_load_2d(b, &xmap, col0, t0, full_leader);
                tma_load_2d(b + GM_ATOM_BYTES, &xmap, col0 + 64, t0, full_leader);
                if (!a_in_b) {
                    tma_load_2d(b + GM_OPERAND_BYTES, &xmap, row0, t0, full_leader);
                    tma_load_2d(b + GM_OPERAND_BYTES + GM_ATOM_BYTES, &xmap, row0 + 64, t0, full_leader);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ---- MMA issue (leader): 4 instructions of K = 16 tokens per stage, 8 stages per
            // accumulator pass -------------------------------------------------------------------
            bool ok = true;
            for (int c = 0; c < num_chunks && ok; ++c) {
                const int ab = c & 1;
                // both CTAs have drained this accumulator's previous pass
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
                    const unsigned a = a_in_b ? b : b + GM_OPERAND_BYTES;
#pragma unroll
                    for (int ks = 0; ks < GM_BK / 16; ++ks) {
                        // 16 tokens = two 8-token groups = 2048 bytes further along K
                        const unsigned long long da = umma_desc_mn_sw128(a + ks * 2048);
                        const unsigned long long db = umma_desc_mn_sw128(b + ks * 2048);
                        umma_bf16(acc, da, db, (kb > c * GM_CHUNK_KB || ks > 0) ? 1u : 0u);
                    }
                    umma_commit_pair(smem_u32(bars + GM_STAGES + s));  // the stage is free in both CTAs
                }
                umma_commit_pair(smem_u32(acc_full + ab));              // this pass of the accumulator is complete
            }
        }
    } else {
        // ---- epilogue: warp w reads TMEM lanes 32 (w % 4) .. + 31 of column half (w - 2) / 4; a
        // thread keeps half a row of its CTA's part of the tile (128 columns) in fp32 registers
        // across the accumulator passes -----------------------------------------------------------
        const int q = warp & 3, half = (warp - 2) >> 2;
        // the leader's "accumulator empty" barriers, as cluster addresses
        unsigned empty_leader[2];
#pragma unroll
        for (int b = 0; b < 2; ++b)
            empty_leader[b] = cluster_addr(smem_u32(acc_empty + b), 0);
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
                asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(empty_leader[ab]) : "memory");
        }
        // 128 x 128 block (br, bc) of H: above the diagonal it is stored with its mirror image, on
        // the diagonal alone, and the one below it (second CTA, first half of a diagonal tile) is
        // the mirror image of what the leader stores
        const int br = 2 * I + (int)rank, bc = 2 * J + half;
        if (ok && br <= bc) {
            const bool diagonal = bc == br;
            const int64_t i = (int64_t)br * GM_TILE + q * 32 + lane;       // row of H held by this thread
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
    // nobody leaves while its partner may still read its shared memory or signal its barriers
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    cluster_sync_all();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(GM_TMEM_COLS) : "memory");
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
    // one pair of CTAs per 256 x 256 tile of the upper triangle
    const long long n256 = (K + 2 * GM_TILE - 1) / (2 * GM_TILE);
    const long long n_ctas = n256 * (n256 + 1);
    if (n_ctas >= (1ll << 31)) return sb_fail(ctx, SB_ERR_SHAPE, "gram: too many tiles");
    SB_FUNC_ATTR(ctx, gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GM_SMEM);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)n_ctas);
    cfg.blockDim = dim3(GM_THREADS);
    cfg.dynamicSmemBytes = GM_SMEM;
    cfg.stream = ctx->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    SB_CUDA(ctx, cudaLaunchKernelEx(&cfg, gram_kernel, map, T, K, scale, accumulate, H, ctx->dstate));
    SB_LAUNCHED(ctx);
    return SB_OK;
}
