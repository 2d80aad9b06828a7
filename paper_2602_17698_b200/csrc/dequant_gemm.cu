// Fused mixed-precision dequantisation + matrix product on the packed format (Section 5.3,
// Table 4: dequantise tile by tile, one bitwidth per tile, feed the tensor cores):
//     Y[t][r] = sum_c X[t][c] * (lo[r][g(c)] + scale[r][g(c)] * q[r][c])
// for a few tokens t (decode batches) against a packed R x C matrix.  The codes are small
// integers, exactly representable in bf16, so the contraction runs on the CODES:
//     Y[t][r] = sum over column blocks j of  scale[r][j] * (sum_c X[t][c] q[r][c]) + lo[r][j] * (sum_c X[t][c])
// with one tcgen05 contraction (M = 128 weight rows, N = tokens, K = the block's 128 columns,
// bf16 x bf16 -> fp32) per 128 x 128 block, scaled per row in the drain; nothing is rounded
// but the fp32 accumulation.  The packed codes are read once from HBM; what costs time is
// turning them into operands, so the unpacking is kept to about 1.4 operations per code:
// for b in {1, 2, 4, 8} a 32-bit word of codes is split by ONE mask per pair,
//     (w >> (b s)) & (2^b - 1) * 0x00010001     ->  codes s and s + 16 / b of the word as two 16-bit halves,
// which OR 0x4300 turns into the bf16 pair (128 + q_lo, 128 + q_hi); subtracting 128 is exact.
// That visits the columns of a word in the order s, s + n/2, s + 1, ... (n = 32 / b); the
// contraction does not care about the order of K as long as X uses the same one, so a small
// kernel first writes X in each of those column orders (and the per-block column sums of X).
//
// The unpacked codes never touch shared memory: bf16 codes are four times the packed bytes at
// 4 bits, and writing them to a shared-memory operand tile and reading them back by the tensor
// cores made shared-memory bandwidth the bound.  They go from registers to TENSOR MEMORY
// (tcgen05.st, thread = weight row = TMEM lane) and the contraction takes its A operand from
// there; only the few-token slice of X is a shared-memory operand.
//
// Grid: (R / 128 row tiles) x (S column segments), two CTAs per SM.  Per CTA:
//   warp 13 (one thread): per block two bulk copies (cp.async.bulk, mbarrier complete_tx) into a
//     four-stage ring, three blocks ahead: the block's packed codes as they lie in memory, and its
//     slice of X, which the preparation kernel has already laid out as the K-major
//     128-byte-swizzle operand image;
//   warps 4-11 (thread = 2 x 32 columns of a weight row): unpack the block into registers,
//     tcgen05.st into one of three 64-column TMEM operand buffers, tcgen05.wait::st, fences,
//     mbarrier arrives (operand ready; code stage free);
//   warp 12 (one thread): 8 tcgen05.mma (K = 16, A from TMEM, B = X slice from shared memory) per
//     block into one of two TMEM accumulators of N columns, one tcgen05.commit per block, which
//     frees the operand buffer and the X slice and publishes the accumulator;
//   warps 0-3 (thread = weight row = TMEM lane): tcgen05.ld of the block's accumulator,
//     y += scale * acc + lo * colsum(X) in fp32 registers; at the end the segment's partial
//     sums go to scratch (or to Y when there is one segment) and a second kernel adds the
//     segments in order.
// Every mbarrier wait is bounded; on a time-out the kernel latches SB_ERR_TIMEOUT and all
// roles leave.
#include "common.cuh"

namespace {

constexpr int DQ_M = 128;                   // weight rows per CTA = block rows
constexpr int DQ_KB = 128;                  // block columns
constexpr int DQ_RING = 4;                  // blocks in flight (codes + X slice)
constexpr int DQ_CODE_STAGE = 2048 * 8;     // bytes of codes of one block at 8 bits
constexpr int DQ_A_COLS = DQ_KB / 2;         // TMEM columns of a block's codes: two bf16 per 32-bit column
constexpr int DQ_ABUF = 3;                  // TMEM operand buffers: the unpackers run up to two blocks ahead of the contraction
constexpr int DQ_MAX_T = 32;
constexpr int DQ_X_STAGE = DQ_MAX_T * DQ_KB * 2;        // X slice of a block: tokens x 128 bf16
constexpr int DQ_CONV_WARPS = 8, DQ_EPI_WARPS = 4;    // unpacking thread = 32 columns of a weight row
constexpr int DQ_THREADS = (DQ_EPI_WARPS + DQ_CONV_WARPS + 2) * 32;   // + MMA warp + loader warp
constexpr int DQ_MAX_SEG_BLOCKS = 32;       // column blocks per segment (their column sums sit in shared memory)
constexpr int DQ_ORDERS = 5;                // column orders of X: identity, b = 1, 2, 4, 8
constexpr int DQ_SMEM = DQ_RING * (DQ_CODE_STAGE + DQ_X_STAGE) + DQ_MAX_SEG_BLOCKS * DQ_MAX_T * 4 +
                        1024 /* alignment */ + 512 /* barriers, block table */;
constexpr int DQ_TMEM_COLS = 256;           // accumulators in columns [0, 64), operand buffers at 64, 128 and 192
constexpr unsigned long long DQ_WAIT_NS = 2000ull * 1000 * 1000;

// candidate bitwidths, four bits each
struct DqBits { unsigned packed; };
__device__ __forceinline__ int dq_bits(DqBits b, int l) { return (int)((b.packed >> (4 * l)) & 15u); }
// column order of X that the unpacking of b-bit codes produces
__host__ __device__ inline int dq_order(int b) { return b == 1 ? 1 : b == 2 ? 2 : b == 4 ? 3 : b == 8 ? 4 : 0; }

__device__ __forceinline__ unsigned dq_smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long dq_now_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void dq_mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void dq_mbar_arrive(unsigned bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool dq_mbar_try_wait(unsigned bar, unsigned parity) {
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
__device__ __forceinline__ bool dq_mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag) {
    unsigned long long t0 = 0;
    for (unsigned spins = 0;; ++spins) {
        if (dq_mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((spins & 255u) == 255u) {
            const unsigned long long now = dq_now_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > DQ_WAIT_NS) { *abort_flag = 1; return false; }
        }
    }
}
__device__ __forceinline__ void dq_mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// contiguous bytes (a multiple of 16, both addresses 16-byte aligned) into shared memory; the
// bytes are counted on the mbarrier
__device__ __forceinline__ void dq_bulk_load(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// K-major operand in the 128-byte-swizzle layout: rows of 128 bytes (64 bf16 along K), 8-row
// groups 1024 bytes apart; the leading offset is not used by swizzled K-major layouts
__device__ __forceinline__ unsigned long long dq_desc(unsigned addr) {
    unsigned long long d = 0;
    d |= (unsigned long long)((addr >> 4) & 0x3fffu);
    d |= 1ull << 16;
    d |= (unsigned long long)((1024 >> 4) & 0x3fff) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
// fp32 accumulator, bf16 x bf16, both operands K-major, M = 128, N = n
__device__ __forceinline__ unsigned dq_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(DQ_M >> 4) << 24);
}
// A (128 rows x 16 columns of bf16 = 8 TMEM columns, row = lane) from tensor memory, B from shared memory
__device__ __forceinline__ void dq_mma(unsigned tmem_d, unsigned tmem_a, unsigned long long b, unsigned idesc,
                                       unsigned acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(b), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void dq_tmem_st16(unsigned taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void dq_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void dq_tmem_ld16(unsigned taddr, float (&v)[16]) {
    unsigned r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int k = 0; k < 16; ++k) v[k] = __uint_as_float(r[k]);
}

// ---- X in the column orders of the unpacking, and its per-block column sums ------------------
// order o > 0 (codes of b bits, n = 32 / b per word): position n m + 2 s + h holds column
// n m + s + (n / 2) h.  xp: [DQ_ORDERS][C / 128] images of T x 128 bf16, each laid out as the
// shared-memory operand (two K halves of T rows x 128 bytes, 16-byte chunks XOR-swizzled with the
// row), so that one contiguous copy brings a block's slice in; xsum: [C / 128][T] fp32.
__device__ __forceinline__ int dq_image_index(int T, int t, int p) {
    const int panel = p >> 6, pp = p & 63;
    return panel * (T * 64) + t * 64 + (((pp >> 3) ^ (t & 7)) << 3) + (pp & 7);
}
__global__ void dq_prepare_x_kernel(const __nv_bfloat16* __restrict__ X, int64_t ldx, int T, int64_t nbc,
                                    __nv_bfloat16* __restrict__ xp, float* __restrict__ xsum) {
    const int64_t jb = blockIdx.x;                       // column block
    const int t = blockIdx.y;
    const int p = threadIdx.x;                           // position inside the block, 0..127
    const __nv_bfloat16* xrow = X + (int64_t)t * ldx + jb * DQ_KB;
    const float v = __bfloat162float(xrow[p]);
    // column sum of the block in a fixed order: pairwise inside the warp, then the four warps
    __shared__ float ws[4];
    const float s = warp_sum(v);
    if ((p & 31) == 0) ws[p >> 5] = s;
    __syncthreads();
    if (p == 0) xsum[jb * T + t] = (ws[0] + ws[1]) + (ws[2] + ws[3]);
    const int64_t image = (int64_t)T * DQ_KB;
    __nv_bfloat16* out = xp + jb * image + dq_image_index(T, t, p);
    out[0] = xrow[p];
#pragma unroll
    for (int o = 1; o < DQ_ORDERS; ++o) {
        const int n = 32 >> (o - 1);                     // codes per word: 32, 16, 8, 4
        const int m = p / n, w = p % n, s2 = w >> 1, h = w & 1;
        out[(int64_t)o * nbc * image] = xrow[n * m + s2 + (n >> 1) * h];
    }
}

// ---- unpacking ---------------------------------------------------------------------------------
// 32 codes (B words) of one weight row, b in {1, 2, 4, 8}, from shared memory into 16 registers of
// bf16 pairs.  `src` points at the row's codes (16 B bytes), `qi` = which 32 codes of the row (0..3).
template <int B>
__device__ __forceinline__ void dq_unpack32(const unsigned char* src, int qi, uint32_t (&out)[16]) {
    constexpr int N = 32 / B;                            // codes per word
    constexpr unsigned MASK = ((1u << B) - 1u) * 0x00010001u;
    const __nv_bfloat162 c128 = __float2bfloat162_rn(128.f);
    uint32_t w[B];
    if constexpr (B == 1) {
        w[0] = *reinterpret_cast<const uint32_t*>(src + 4 * qi);
    } else if constexpr (B == 2) {
        const uint2 v = *reinterpret_cast<const uint2*>(src + 8 * qi);
        w[0] = v.x; w[1] = v.y;
    } else {
#pragma unroll
        for (int k = 0; k < B / 4; ++k) {
            const int chunk = qi * (B / 4) + k;          // 16-byte chunk of the row
            const uint4 v = *reinterpret_cast<const uint4*>(src + (chunk << 4));
            w[4 * k] = v.x; w[4 * k + 1] = v.y; w[4 * k + 2] = v.z; w[4 * k + 3] = v.w;
        }
    }
#pragma unroll
    for (int m = 0; m < B; ++m) {
#pragma unroll
        for (int s = 0; s < N / 2; ++s) {
            const uint32_t v = (w[m] >> (B * s)) & MASK;
            uint32_t bits;
            if constexpr (B < 8) {
                bits = u32(__hsub2(b162(v | 0x43004300u), c128));
            } else {
                // 8 significant bits: the low seven through the exponent trick, the top one added
                const __nv_bfloat162 lo7 = __hsub2(b162((v & 0x007f007fu) | 0x43004300u), c128);
                const uint32_t top = ((v >> 7) & 0x00010001u) * 0x4300u;     // 128.0 or 0 per half
                bits = u32(__hadd2(lo7, b162(top)));
            }
            out[(N / 2) * m + s] = bits;
        }
    }
}

// any other bitwidth below 8: code k of the row at bit k b of its stream, columns in their own order
__device__ __forceinline__ void dq_unpack32_generic(const unsigned char* src, int b, int qi, uint32_t (&out)[16]) {
    const uint32_t* words = reinterpret_cast<const uint32_t*>(src);
    const uint32_t mask = (1u << b) - 1u;
    const __nv_bfloat162 c128 = __float2bfloat162_rn(128.f);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t pair = 0;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int bit = (32 * qi + 8 * c + 2 * k + h) * b;
                const int wi = bit >> 5;
                // the row's stream is 4 b words long; the funnel shift may look one word past a code
                // that ends at the stream's end, so that word is clamped to the last one
                const uint32_t w0 = words[wi], w1 = words[min(wi + 1, 4 * b - 1)];
                pair |= (__funnelshift_r(w0, w1, bit & 31) & mask) << (16 * h);
            }
            out[4 * c + k] = u32(__hsub2(b162(pair | 0x43004300u), c128));
        }
    }
}

struct DqArgs {
    const uint32_t* packed;
    const int64_t* block_off;       // [nb + 1], words
    const float2* meta;             // [(r * nbc + j)] = (scale, lo), group == block width
    const uint8_t* level;           // [nb]
    const __nv_bfloat16* xp;        // [DQ_ORDERS][nbc] operand images of T x 128
    const float* xsum;              // [nbc][T]
    float* out;                     // partial sums [S][T][R] (or Y when S == 1)
    int64_t out_t_stride;           // R for the partial sums, ldy for Y
    int64_t out_seg_stride;
    int64_t R, C;
    int nbc, seg_blocks, T;
    DqBits bits;
    SbDeviceState* ds;
};

template <int NT>
__global__ void __launch_bounds__(DQ_THREADS, 2) dequant_gemm_kernel(const DqArgs a) {
    extern __shared__ unsigned char dq_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(dq_smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* x_ring = smem;                                         // DQ_RING x 8 KB slices of X
    unsigned char* code_ring = x_ring + DQ_RING * DQ_X_STAGE;             // DQ_RING x 16 KB packed codes
    float* xs = reinterpret_cast<float*>(code_ring + DQ_RING * DQ_CODE_STAGE);   // [seg_blocks][NT] column sums
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(xs + DQ_MAX_SEG_BLOCKS * DQ_MAX_T);
    unsigned long long* a_full = bars;              // [DQ_ABUF] unpackers (TMEM operand buffer written) -> MMA
    // [DQ_RING] the contraction of block j is complete (one commit per block, at j % DQ_RING): the
    // drain may read its accumulator, the unpackers may rewrite the operand buffer two blocks
    // later, the loader may refill the stage DQ_RING blocks later
    unsigned long long* done = bars + DQ_ABUF;
    unsigned long long* d_empty = done + DQ_RING;          // [2] drained -> MMA
    unsigned long long* ld_full = d_empty + 2;             // [DQ_RING] both copies of a block landed
    unsigned long long* code_empty = ld_full + DQ_RING;    // [DQ_RING] all unpackers have read the codes -> loader
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(code_empty + DQ_RING);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    // per block of the segment: first word of its codes (blocks are below 2^32 words apart from the
    // segment's first) and its bitwidth, so that the loop below has no dependent global loads
    unsigned* blk_word = tmem_slot + 4;                 // [DQ_MAX_SEG_BLOCKS]
    unsigned char* blk_bits = reinterpret_cast<unsigned char*>(blk_word + DQ_MAX_SEG_BLOCKS);   // [DQ_MAX_SEG_BLOCKS]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int TMEM_COLS = DQ_TMEM_COLS;
    static_assert(2 * NT <= 64, "accumulators below the operand buffers");

    const int bi = blockIdx.x;                                  // row tile
    const int j0 = blockIdx.y * a.seg_blocks;                   // first column block of the segment
    const int nblk = min(a.seg_blocks, a.nbc - j0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            dq_mbar_init(dq_smem_u32(d_empty + s), DQ_EPI_WARPS);
        }
        for (int s = 0; s < DQ_ABUF; ++s) dq_mbar_init(dq_smem_u32(a_full + s), DQ_CONV_WARPS * 32);
        for (int s = 0; s < DQ_RING; ++s) {
            dq_mbar_init(dq_smem_u32(done + s), 1);
            dq_mbar_init(dq_smem_u32(ld_full + s), 1);
            dq_mbar_init(dq_smem_u32(code_empty + s), DQ_CONV_WARPS * 32);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == DQ_EPI_WARPS + DQ_CONV_WARPS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dq_smem_u32(tmem_slot)),
                     "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // the segment's column sums of X and its block table
    for (int i = threadIdx.x; i < nblk * NT; i += DQ_THREADS) xs[i] = a.xsum[(int64_t)j0 * NT + i];
    const int64_t blk0 = (int64_t)bi * a.nbc + j0;
    const int64_t word0 = a.block_off[blk0];
    if (threadIdx.x < nblk) {
        blk_word[threadIdx.x] = (unsigned)(a.block_off[blk0 + threadIdx.x] - word0);
        blk_bits[threadIdx.x] = (unsigned char)dq_bits(a.bits, a.level[blk0 + threadIdx.x]);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_base = *tmem_slot;

    if (warp >= DQ_EPI_WARPS && warp < DQ_EPI_WARPS + DQ_CONV_WARPS) {
        // ---- unpackers: thread = columns 32 hq ... and 64 + 32 hq ... of weight row r of the tile ------
        const int ct = threadIdx.x - DQ_EPI_WARPS * 32;
        const int r = ct & (DQ_M - 1), hq = ct >> 7;
        // TMEM lanes 32 (warp % 4) ... + 31 belong to this warp: lane = weight row
        const unsigned a_lane = (unsigned)((r >> 5) * 32) << 16;
        bool ok = true;
        for (int j = 0; j < nblk && ok; ++j) {
            const int st = j % DQ_RING, buf = j % DQ_ABUF;
            const int b = blk_bits[j];
            // the block has landed, and the contraction of block j - DQ_ABUF no longer reads the operand buffer
            ok = __all_sync(0xffffffffu, dq_mbar_wait(dq_smem_u32(ld_full + st), (unsigned)(j / DQ_RING) & 1u, abort_flag) &&
                                         (j < DQ_ABUF || dq_mbar_wait(dq_smem_u32(done + (j - DQ_ABUF) % DQ_RING),
                                                                      (unsigned)((j - DQ_ABUF) / DQ_RING) & 1u, abort_flag)));
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const unsigned char* src = code_ring + st * DQ_CODE_STAGE + r * 16 * b;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int qi = 2 * h + hq;
                uint32_t v[16];
                switch (b) {                                  // uniform over the CTA
                    case 1: dq_unpack32<1>(src, qi, v); break;
                    case 2: dq_unpack32<2>(src, qi, v); break;
                    case 4: dq_unpack32<4>(src, qi, v); break;
                    case 8: dq_unpack32<8>(src, qi, v); break;
                    default: dq_unpack32_generic(src, b, qi, v); break;
                }
                dq_tmem_st16(tmem_base + a_lane + (unsigned)(64 + buf * DQ_A_COLS + 16 * qi), v);
            }
            dq_mbar_arrive(dq_smem_u32(code_empty + st));     // the codes are in registers: the stage may be refilled
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            dq_mbar_arrive(dq_smem_u32(a_full + buf));
        }
    } else if (warp == DQ_EPI_WARPS + DQ_CONV_WARPS) {
        if (lane == 0) {
            // ---- MMA issue -----------------------------------------------------------------------------
            const unsigned idesc = dq_idesc(NT);
            bool ok = true;
            for (int j = 0; j < nblk && ok; ++j) {
                const int ds_ = j & 1, st = j % DQ_RING, buf = j % DQ_ABUF;
                ok = dq_mbar_wait(dq_smem_u32(d_empty + ds_), ((unsigned)(j >> 1) & 1u) ^ 1u, abort_flag) &&
                     dq_mbar_wait(dq_smem_u32(ld_full + st), (unsigned)(j / DQ_RING) & 1u, abort_flag) &&
                     dq_mbar_wait(dq_smem_u32(a_full + buf), (unsigned)(j / DQ_ABUF) & 1u, abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const unsigned at = tmem_base + (unsigned)(64 + buf * DQ_A_COLS);
                const unsigned xt = dq_smem_u32(x_ring + st * DQ_X_STAGE);
#pragma unroll
                for (int ks = 0; ks < DQ_KB / 16; ++ks)             // 16 columns: 8 TMEM columns of A, 32 bytes of X along K
                    dq_mma(tmem_base + (unsigned)(ds_ * NT), at + ks * 8,
                           dq_desc(xt + (ks >> 2) * (NT * 128) + (ks & 3) * 32), idesc, ks > 0 ? 1u : 0u);
                dq_commit(dq_smem_u32(done + st));
            }
        }
    } else if (warp == DQ_EPI_WARPS + DQ_CONV_WARPS + 1) {
        if (lane == 0) {
            // ---- loader: the codes of block j as they lie in memory and its slice of X (an operand
            // image) into ring stage j % DQ_RING, as soon as the unpackers and the contraction of block
            // j - DQ_RING have let go of it ----------------------------------------------------------------
            bool ok = true;
            const unsigned x_bytes = (unsigned)(NT * DQ_KB * 2);
            for (int j = 0; j < nblk && ok; ++j) {
                const int st = j % DQ_RING;
                // block j - DQ_RING used this stage: its codes have been read and its contraction is complete
                if (j >= DQ_RING) {
                    const unsigned ph = (unsigned)(j / DQ_RING - 1) & 1u;
                    ok = dq_mbar_wait(dq_smem_u32(code_empty + st), ph, abort_flag) &&
                         dq_mbar_wait(dq_smem_u32(done + st), ph, abort_flag);
                }
                if (!ok) break;
                const int b = blk_bits[j];
                const unsigned code_bytes = (unsigned)(2048 * b);
                const unsigned full = dq_smem_u32(ld_full + st);
                dq_mbar_expect_tx(full, code_bytes + x_bytes);
                dq_bulk_load(dq_smem_u32(code_ring + st * DQ_CODE_STAGE), a.packed + word0 + blk_word[j], code_bytes, full);
                dq_bulk_load(dq_smem_u32(x_ring + st * DQ_X_STAGE),
                             a.xp + ((int64_t)dq_order(b) * a.nbc + j0 + j) * (NT * DQ_KB), x_bytes, full);
            }
        }
    } else {
        // ---- drain: thread = weight row = TMEM lane -----------------------------------------------------
        const int r = threadIdx.x;
        const int64_t row = (int64_t)bi * DQ_M + r;
        float y[NT];
#pragma unroll
        for (int t = 0; t < NT; ++t) y[t] = 0.f;
        bool ok = true;
        float2 sl = a.meta[row * a.nbc + j0];
        for (int j = 0; j < nblk && ok; ++j) {
            const float2 cur = sl;
            if (j + 1 < nblk) sl = a.meta[row * a.nbc + j0 + j + 1];
            const int ds_ = j & 1;
            ok = __all_sync(0xffffffffu, dq_mbar_wait(dq_smem_u32(done + j % DQ_RING), (unsigned)(j / DQ_RING) & 1u, abort_flag));
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int c0 = 0; c0 < NT; c0 += 16) {
                float d[16];
                dq_tmem_ld16(tmem_base + ((unsigned)(warp * 32) << 16) + (unsigned)(ds_ * NT + c0), d);
#pragma unroll
                for (int k = 0; k < 16; ++k)
                    y[c0 + k] = fmaf(cur.x, d[k], fmaf(cur.y, xs[j * NT + c0 + k], y[c0 + k]));
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) dq_mbar_arrive(dq_smem_u32(d_empty + ds_));
        }
        if (ok) {
            float* out = a.out + (int64_t)blockIdx.y * a.out_seg_stride + row;
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                if (!isfinite(y[t])) sb_latch(a.ds, SB_ERR_NONFINITE, SBK_GEMM);
                if (t < a.T) out[(int64_t)t * a.out_t_stride] = y[t];
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == DQ_EPI_WARPS + DQ_CONV_WARPS)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    if (threadIdx.x == 0 && *abort_flag) sb_latch(a.ds, SB_ERR_TIMEOUT, SBK_GEMM);
}

// Y[t][r] = sum over segments, in order
__global__ void dq_reduce_kernel(const float* __restrict__ part, int S, int T, int64_t R, float* __restrict__ Y,
                                 int64_t ldy) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int t = blockIdx.y;
    if (r >= R) return;
    float acc = 0.f;
    for (int s = 0; s < S; ++s) acc += part[((int64_t)s * T + t) * R + r];
    Y[(int64_t)t * ldy + r] = acc;
}

}  // namespace

extern "C" sb_status sb_dequant_gemm(sb_ctx* ctx, const void* X, int64_t T, int64_t ldx, const uint32_t* packed,
                                     const int64_t* block_off_words, const float* meta, const uint8_t* level,
                                     int64_t R, int64_t C, int br, int bc, int group, const int* bits, int n_bits,
                                     float* Y, int64_t ldy) {
    if (!ctx) return SB_ERR_INVALID;
    if (!X || !packed || !block_off_words || !meta || !level || !Y || T <= 0 || R <= 0 || C <= 0)
        return sb_fail(ctx, SB_ERR_INVALID, "dequant gemm: null or empty");
    if (!sb_check_bits(bits, n_bits)) return sb_fail(ctx, SB_ERR_INVALID, "dequant gemm: bits must be ascending in 1..8");
    if (br != DQ_M || bc != DQ_KB || group != DQ_KB || R % DQ_M || C % DQ_KB || ldx < C || ldy < R ||
        (reinterpret_cast<uintptr_t>(packed) & 15))
        return sb_fail(ctx, SB_ERR_SHAPE, "dequant gemm: blocks of 128 x 128 with group 128 tiling the matrix, 16-byte aligned codes");
    if (R >= (1ll << 31) || C >= (1ll << 31)) return sb_fail(ctx, SB_ERR_SHAPE, "dequant gemm: R and C must fit 31 bits");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const int nbc = (int)(C / DQ_KB);
    const int64_t nbr = R / DQ_M;
    // column segments: enough CTAs for two per SM, at most DQ_MAX_SEG_BLOCKS blocks each
    int S = (int)((2 * (int64_t)ctx->sm_count) / nbr);
    if (S < 1) S = 1;
    if (S > nbc) S = nbc;
    int seg_blocks = (nbc + S - 1) / S;
    if (seg_blocks > DQ_MAX_SEG_BLOCKS) seg_blocks = DQ_MAX_SEG_BLOCKS;
    S = (nbc + seg_blocks - 1) / seg_blocks;
    if (S > 65535) return sb_fail(ctx, SB_ERR_SHAPE, "dequant gemm: too many column segments");
    DqBits db{};
    for (int l = 0; l < n_bits; ++l) db.packed |= (unsigned)bits[l] << (4 * l);
    // tokens in slices of at most DQ_MAX_T (padded to 16 or 32 with zero rows)
    for (int64_t t0 = 0; t0 < T; t0 += DQ_MAX_T) {
        const int Tn = (int)((T - t0) < DQ_MAX_T ? (T - t0) : DQ_MAX_T);
        const int NT = Tn <= 16 ? 16 : 32;
        void* arena;
        sb_status st = sb_scratch(ctx, Carver::need({(size_t)DQ_ORDERS * NT * C * 2, (size_t)nbc * NT * 4,
                                                     S > 1 ? (size_t)S * Tn * R * 4 : 0}), &arena);
        if (st != SB_OK) return st;
        Carver cv(arena);
        __nv_bfloat16* xp = cv.take<__nv_bfloat16>((size_t)DQ_ORDERS * NT * C);
        float* xsum = cv.take<float>((size_t)nbc * NT);
        float* part = S > 1 ? cv.take<float>((size_t)S * Tn * R) : nullptr;
        const __nv_bfloat16* Xs = static_cast<const __nv_bfloat16*>(X) + t0 * ldx;
        if (Tn < NT) {      // zero rows for the padding tokens
            SB_CUDA(ctx, cudaMemsetAsync(xp, 0, (size_t)DQ_ORDERS * NT * C * 2, ctx->stream));
            SB_CUDA(ctx, cudaMemsetAsync(xsum, 0, (size_t)nbc * NT * 4, ctx->stream));
        }
        dq_prepare_x_kernel<<<dim3((unsigned)nbc, (unsigned)Tn), 128, 0, ctx->stream>>>(Xs, ldx, NT, nbc, xp, xsum);
        SB_LAUNCHED(ctx);
        DqArgs a{};
        a.packed = packed; a.block_off = block_off_words; a.meta = reinterpret_cast<const float2*>(meta);
        a.level = level; a.xp = xp; a.xsum = xsum;
        a.out = S > 1 ? part : Y + t0 * ldy;
        a.out_t_stride = S > 1 ? R : ldy;
        a.out_seg_stride = S > 1 ? (int64_t)Tn * R : 0;
        a.R = R; a.C = C; a.nbc = nbc; a.seg_blocks = seg_blocks; a.T = Tn; a.bits = db; a.ds = ctx->dstate;
        const dim3 grid((unsigned)nbr, (unsigned)S);
        if (NT == 16) {
            SB_FUNC_ATTR(ctx, dequant_gemm_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, DQ_SMEM);
            dequant_gemm_kernel<16><<<grid, DQ_THREADS, DQ_SMEM, ctx->stream>>>(a);
        } else {
            SB_FUNC_ATTR(ctx, dequant_gemm_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, DQ_SMEM);
            dequant_gemm_kernel<32><<<grid, DQ_THREADS, DQ_SMEM, ctx->stream>>>(a);
        }
        SB_LAUNCHED(ctx);
        if (S > 1) {
            dq_reduce_kernel<<<dim3((unsigned)((R + 255) / 256), (unsigned)Tn), 256, 0, ctx->stream>>>(part, S, Tn, R,
                                                                                                       Y + t0 * ldy, ldy);
            SB_LAUNCHED(ctx);
        }
    }
    return SB_OK;
}
