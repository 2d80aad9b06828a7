// Block error table with the FULL calibration second-moment matrix (Section 3.2 with the cross
// terms between input channels kept): for block i with columns J and candidate b_l,
//     E[i][l] = sum_r d_r H'_JJ d_r^T = < H'_JJ , D^T D >,     D = (W' - Q_{b_l}(W'))[rows of i, J],
// where H' is H = X^T X / T in the permuted column order.  The 128 x 128 Gram matrix D^T D of
// every (block, candidate) is a tensor-core contraction over the block's 128 rows; the inner
// product with H'_JJ is the epilogue.  bf16 alone is too coarse for D, so D is split into two
// bf16 terms D = D0 + D1 and G = D0^T D0 + D0^T D1 + (D0^T D1)^T (the D1^T D1 term is 2^-16 of
// G); with H symmetric, E = <H, D0^T D0> + 2 <H, D0^T D1>: two accumulators per candidate.
//
// One persistent CTA of 16 identical warps per SM.  The quantisation arithmetic of the operands
// (one division, three binary64 and about ten fp32 / integer operations per weight and
// candidate) is what bounds the kernel, not the tensor pipe, so every warp spends most of its
// time there and the contraction runs beside it.  Work items are (block, candidate) pairs; in
// iteration i every thread
//   1. quantises its quarter row of the block at the candidate of item i (codes by the binary64
//      sequence, residual in fp32 with a two-float grid step), splits it into two bf16 terms and
//      writes them into shared-memory stage i & 1 in the MN-major 128-byte-swizzle layout the
//      tensor cores read (the layout a TMA load of the tile would produce);
//   2. drains item i - 1: tcgen05.ld of its 32 columns of one row of both accumulators, inner
//      product with the same 32 entries of H'_JJ, which the thread keeps in registers for the
//      whole block column; warp sums go to shared memory and thread 0 adds the 16 of them in a
//      fixed order one iteration later;
//   3. (thread 0) once all 512 threads have arrived, issues 8 tcgen05.mma (M = 128, N = 256,
//      K = 16, bf16 -> fp32: D0^T [D0 | D1]) for item i into TMEM stage i & 1 of 2 x 128 columns, and commits to
//      free the shared-memory stage and to publish the accumulators: the contraction of item i
//      runs while the warps quantise item i + 1.
// Two shared-memory stages and two TMEM stages: nobody waits for the tensor pipe.  Every mbarrier wait is bounded; on a time-out the kernel
// latches SB_ERR_TIMEOUT and all warps leave.
#include "common.cuh"

sb_status sb_gather_bf16(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                         const int32_t* rp, const int32_t* cp, void* out);

namespace {

constexpr int FS_N = 128;                              // block rows = block columns = 128
constexpr int FS_ATOM_BYTES = FS_N * 128;              // 128 rows x 64 columns of bf16
constexpr int FS_TILE_BYTES = 2 * FS_ATOM_BYTES;       // one 128 x 128 bf16 operand
constexpr int FS_STAGE_BYTES = 2 * FS_TILE_BYTES;      // D0 and D1
constexpr int FS_STAGES = 2;
constexpr int FS_WARPS = 16;
constexpr int FS_THREADS = FS_WARPS * 32;              // thread = quarter row of the block
constexpr int FS_TMEM_COLS = 512;                      // 2 stages x 2 accumulators x 128 columns
constexpr int FS_SMEM = FS_STAGES * FS_STAGE_BYTES + 1024 /* alignment */ + 512 /* barriers, sums */;
constexpr unsigned long long FS_WAIT_NS = 2000ull * 1000 * 1000;
// 1.5 * 2^52 + 0x4B000000: the low word of (t + MAGIC) is 0x4B000000 + rint(t), the bits of the
// float 2^23 + rint(t) (codes are below 2^23; MAGIC is even, so ties still go to even)
constexpr double FS_MAGIC64 = 6755399441055744.0 + 1258291200.0;
// bf16 x bf16 -> fp32, both operands MN-major, M = 128, N = 256: D0^T [D0 | D1] in one instruction
constexpr unsigned FS_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                              (((2 * FS_N) >> 3) << 17) | ((FS_N >> 4) << 24);

// candidate bitwidths, four bits each (a dynamically indexed parameter array would live on the stack)
struct FsBits { unsigned packed; };
__device__ __forceinline__ int fs_bits(FsBits fb, int l) { return (int)((fb.packed >> (4 * l)) & 15u); }

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
__device__ __forceinline__ void fs_tmem_ld16(unsigned taddr, float (&v)[16]) {
    unsigned r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int k = 0; k < 16; ++k) v[k] = __uint_as_float(r[k]);
}
__device__ __forceinline__ void fs_tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

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

// PLAIN: units of 128 rows and no row weights (both known at compile time: the common case keeps
// its instruction stream)
template <int GROUP, bool PLAIN>
__global__ void __launch_bounds__(FS_THREADS, 1)
full_scores_kernel(const __nv_bfloat16* __restrict__ W, int64_t ldw, const float* __restrict__ hblk,
                   FsBits fb, int L, int64_t n_blocks, int64_t n_block_cols, int unit_rows,
                   const float* __restrict__ row_weight, const int32_t* __restrict__ a_perm, float gain_elems, int halves,
                   float* __restrict__ err, float* __restrict__ gain, SbDeviceState* ds) {
    // A work unit is `unit_rows` (64 or 128) rows x 128 columns; the contraction always runs over 128
    // rows, the rows past unit_rows of a 64-row unit are written as zeros (they add nothing).
    // n_blocks / n_block_cols count UNITS here; the host adds the two units of a 256-row block.
    // this CTA's blocks: a contiguous range of the COLUMN-major block sequence, so that consecutive
    // blocks share their columns J (and every thread keeps its entries of H'_JJ in registers)
    const int64_t n_block_rows = n_blocks / n_block_cols;
    const int64_t seq_lo = n_blocks * blockIdx.x / gridDim.x, seq_hi = n_blocks * (blockIdx.x + 1) / gridDim.x;
    const long long n_items = (long long)(seq_hi - seq_lo) * L;
    extern __shared__ unsigned char fs_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(fs_smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + FS_STAGES * FS_STAGE_BYTES);
    unsigned long long* smem_full = bars;             // [2] all threads -> MMA issue
    unsigned long long* smem_empty = bars + 2;        // [2] MMA done reading -> all threads
    unsigned long long* tmem_full = bars + 4;         // [2] MMA done -> drain
    unsigned long long* tmem_empty = bars + 6;        // [2] 16 warps drained -> MMA issue
    unsigned long long* red_full = bars + 8;          // [2] 16 warp sums written -> thread 0
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(bars + 10);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* red = reinterpret_cast<float*>(tmem_slot + 4);          // [2][16] warp sums
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            fs_mbar_init(fs_smem_u32(smem_full + s), FS_THREADS);
            fs_mbar_init(fs_smem_u32(smem_empty + s), 1);
            fs_mbar_init(fs_smem_u32(tmem_full + s), 1);
            fs_mbar_init(fs_smem_u32(tmem_empty + s), FS_WARPS);
            fs_mbar_init(fs_smem_u32(red_full + s), FS_WARPS);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(fs_smem_u32(tmem_slot)),
                     "r"(FS_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_base = *tmem_slot;

    // quantisation: thread owns 32 columns (quarter qd) of row r.  Register slot c holds the
    // 8-column chunk (c ^ 2 (qd >> 1)) of the quarter, so that the eight lanes of one shared-memory
    // store phase (2 rows x 4 quarters) hit eight different 16-byte bank groups of the swizzled layout.
    const int r = threadIdx.x >> 2, qd = threadIdx.x & 3;
    const int cflip = (qd >> 1) * 2;
    constexpr int GPC = GROUP / 8;                       // 16-byte chunks (8 columns) per group
    constexpr int CPG = GPC < 4 ? GPC : 4;               // chunks of this thread per group
    constexpr int NG = 4 / CPG;                          // groups (or parts of one) of this thread
    // drain: TMEM lanes 32 (warp & 3) ... + 31 belong to this warp; thread = row j of the Gram
    // matrix, columns [32 cq, 32 cq + 32)
    const int j = (warp & 3) * 32 + lane, cq = warp >> 2;

    if (PLAIN) unit_rows = FS_N;
    const bool row_live = PLAIN || r < unit_rows;
    float sa = 1.f;                                   // sqrt of the row weight: scales the row's residual
    uint32_t wv[16];
    float glo[NG], hreg[32];
    double dlo[NG], range64[NG];
    // (block row, block column) of the item quantised last, and of the item thread 0 finishes
    // next; both advance down the block column (64-bit divisions only here)
    int64_t bj_q = seq_lo / n_block_rows, bi_q = seq_lo - bj_q * n_block_rows - 1;
    int64_t bj_f = bj_q, bi_f = bi_q + 1, bj_h = -1, blocks_left = seq_hi - seq_lo;
    int l = L - 1, l_f = 0;
    float e_prev = 0.f;
    bool ok = true;

    // thread 0: the warp sums of item `it` are complete; add them in a fixed order, write err / gain
    auto finish_item = [&](long long it) -> bool {
        const int s = (int)(it & 1);
        if (!fs_mbar_wait(fs_smem_u32(red_full + s), (unsigned)(it >> 1) & 1u, abort_flag)) return false;
        const float* rr = red + s * FS_WARPS;
        float e = 0.f;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) e += (rr[4 * q4] + rr[4 * q4 + 1]) + (rr[4 * q4 + 2] + rr[4 * q4 + 3]);
        const int64_t blk = bi_f * n_block_cols + bj_f;
        if (!isfinite(e)) sb_latch(ds, SB_ERR_NONFINITE, SBK_SCORES);
        if (!PLAIN && halves == 2) {
            // blocks of 64 columns: the unit holds two of them side by side; each takes the diagonal
            // quadrant of the 128 x 128 Gram matrix that belongs to its own columns (warps 0, 1, 4, 5 hold
            // rows and columns 0..63, warps 10, 11, 14, 15 rows and columns 64..127), the cross
            // quadrants belong to no block
            err[(blk * 2) * L + l_f] = (rr[0] + rr[1]) + (rr[4] + rr[5]);
            err[(blk * 2 + 1) * L + l_f] = (rr[10] + rr[11]) + (rr[14] + rr[15]);
        } else {
            err[blk * L + l_f] = e;
        }
        if (gain && l_f > 0)
            gain[blk * (L - 1) + l_f - 1] =
                (e_prev - e) / ((float)(fs_bits(fb, l_f) - fs_bits(fb, l_f - 1)) * gain_elems);
        e_prev = e;
        if (++l_f == L) {
            l_f = 0;
            if (++bi_f == n_block_rows) { bi_f = 0; ++bj_f; }
        }
        return true;
    };

    for (long long i = 0; i <= n_items && ok; ++i) {
        const int s = (int)(i & 1);
        const int64_t bj_d = bj_q;                               // block column of item i - 1
        if (i < n_items) {
            if (++l == L) {
                // ---- a new block: its weights, group minima and ranges ------------------------------
                l = 0;
                if (++bi_q == n_block_rows) { bi_q = 0; ++bj_q; }
                --blocks_left;
                const uint4* src = reinterpret_cast<const uint4*>(W + (bi_q * unit_rows + r) * ldw + bj_q * FS_N + qd * 32);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 x = row_live ? __ldg(src + (c ^ cflip)) : make_uint4(0u, 0u, 0u, 0u);
                    wv[4 * c] = x.x; wv[4 * c + 1] = x.y; wv[4 * c + 2] = x.z; wv[4 * c + 3] = x.w;
                }
                if (!PLAIN && row_weight) {
                    const int64_t row = bi_q * unit_rows + r;
                    sa = row_live ? sqrtf(__ldg(row_weight + (a_perm ? a_perm[row] : row))) : 0.f;
                }
                if (blocks_left > 0 && row_live) {           // the next block's 64 bytes of this thread towards L2
                    const bool wrap = bi_q + 1 == n_block_rows;
                    const int64_t bi1 = wrap ? 0 : bi_q + 1, bj1 = wrap ? bj_q + 1 : bj_q;
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(W + (bi1 * unit_rows + r) * ldw + bj1 * FS_N + qd * 32));
                }
                // group minimum and maximum per 8-column chunk (exact bf16 min / max)
                float clo[4], chi[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    __nv_bfloat162 mn = b162(wv[4 * c]), mx = mn;
#pragma unroll
                    for (int k = 1; k < 4; ++k) { mn = __hmin2(mn, b162(wv[4 * c + k])); mx = __hmax2(mx, b162(wv[4 * c + k])); }
                    clo[c] = fminf(bf16lo(u32(mn)), bf16hi(u32(mn)));
                    chi[c] = fmaxf(bf16lo(u32(mx)), bf16hi(u32(mx)));
                }
                // combine the chunks of a group: 2 or 4 of this thread (slots c, c ^ 1 hold chunks of
                // one pair whatever the flip), then the 2 or 4 threads of the row
#pragma unroll
                for (int span = 1; span < CPG; span <<= 1) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const float l2 = clo[c ^ span], h2 = chi[c ^ span];
                        clo[c] = fminf(clo[c], l2);           // pairs exchange symmetrically: order is irrelevant
                        chi[c] = fmaxf(chi[c], h2);
                    }
                }
#pragma unroll
                for (int m = 1; m < GPC / 4; m <<= 1) {       // group 64 joins 2 threads, 128 all 4
                    clo[0] = fminf(clo[0], __shfl_xor_sync(0xffffffffu, clo[0], m));
                    chi[0] = fmaxf(chi[0], __shfl_xor_sync(0xffffffffu, chi[0], m));
                }
                // minimum and range in binary64 (the difference of two bf16 values is exact there)
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                    glo[g] = clo[g * CPG];
                    dlo[g] = (double)glo[g];
                    range64[g] = __dsub_rn((double)chi[g * CPG], dlo[g]);
                }
            }
            // ---- quantise at candidate l into shared-memory stage s --------------------------------
            // The quadratic form has cross terms, so it jumps where a code flips, and exact rounding
            // ties are common for bf16 weights: the codes follow the binary64 sequence
            //   inv = qmax / range; q = rint((v - lo) * inv)
            // literally (one division per group), the residual is taken in fp32 with the grid step
            // as a two-float sum.
            const float qmax = (float)((1 << fs_bits(fb, l)) - 1), inv_qmax = __fdiv_rn(1.0f, qmax);
            double inv64[NG];
            float ns[NG], ns_lo[NG];
#pragma unroll
            for (int g = 0; g < NG; ++g) {
                const float range = (float)range64[g];
                const bool live = range64[g] != 0.0;
                inv64[g] = live ? __ddiv_rn((double)qmax, range64[g]) : 0.0;
                ns[g] = live ? -(range * inv_qmax) : 0.f;
                ns_lo[g] = live ? -(fmaf(ns[g], qmax, range) * inv_qmax) : 0.f;
            }
            ok = __all_sync(0xffffffffu, fs_mbar_wait(fs_smem_u32(smem_empty + s), ((unsigned)(i >> 1) & 1u) ^ 1u, abort_flag));
            if (!ok) break;
            unsigned char* d0 = smem + s * FS_STAGE_BYTES + (qd >> 1) * FS_ATOM_BYTES + r * 128;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int g = c / CPG;
                uint32_t h[4], lw[4];
                float w8[8];
                double t8[8];
#pragma unroll
                for (int k = 0; k < 4; ++k) { w8[2 * k] = bf16lo(wv[4 * c + k]); w8[2 * k + 1] = bf16hi(wv[4 * c + k]); }
#pragma unroll
                for (int k = 0; k < 8; ++k) t8[k] = __dsub_rn((double)w8[k], dlo[g]);
#pragma unroll
                for (int k = 0; k < 8; ++k) t8[k] = __dadd_rn(__dmul_rn(t8[k], inv64[g]), FS_MAGIC64);
                // the fp32 part on packed pairs (half the issue slots)
                const f32x2 ns2 = pk2(ns[g], ns[g]), ns_lo2 = pk2(ns_lo[g], ns_lo[g]), nlo2 = pk2(-glo[g], -glo[g]);
                const f32x2 sa2 = pk2(sa, sa);
                const bool weighted = !PLAIN && row_weight != nullptr;
                const f32x2 nmagic2 = pk2(-8388608.f, -8388608.f), none2 = pk2(-1.f, -1.f);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    // exact int -> float: 2^23 + q as bits, minus 2^23
                    const f32x2 q2 = add2(pk2(__int_as_float(__double2loint(t8[2 * k])),
                                              __int_as_float(__double2loint(t8[2 * k + 1]))), nmagic2);
                    f32x2 e2 = fma2(q2, ns_lo2, fma2(q2, ns2, add2(pk2(w8[2 * k], w8[2 * k + 1]), nlo2)));
                    if (weighted) e2 = mul2(e2, sa2);
                    float e0, e1;
                    upk2(e2, e0, e1);
                    const __nv_bfloat162 hi2 = __floats2bfloat162_rn(e0, e1);
                    const f32x2 d2 = fma2(pk2(bf16lo(u32(hi2)), bf16hi(u32(hi2))), none2, e2);    // e - hi, exact
                    float d0f, d1f;
                    upk2(d2, d0f, d1f);
                    h[k] = u32(hi2);
                    lw[k] = u32(__floats2bfloat162_rn(d0f, d1f));
                }
                // chunk of the 128-byte row, then the 128-byte swizzle of the layout
                const int sw = (((qd & 1) * 4 + (c ^ cflip)) ^ (r & 7)) * 16;
                *reinterpret_cast<uint4*>(d0 + sw) = make_uint4(h[0], h[1], h[2], h[3]);
                *reinterpret_cast<uint4*>(d0 + FS_TILE_BYTES + sw) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
            }
            // the tensor cores read shared memory through the async proxy
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            fs_mbar_arrive(fs_smem_u32(smem_full + s));
        }
        if (i >= 1) {
            // ---- drain item i - 1 ---------------------------------------------------------------------
            const long long it = i - 1;
            const int sd = (int)(it & 1);
            if (bj_d != bj_h) {                                  // this thread's 32 entries of H'_JJ
                const float4* hsrc = reinterpret_cast<const float4*>(hblk + (bj_d * FS_N + j) * FS_N + cq * 32);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float4 v = __ldg(hsrc + k);
                    hreg[4 * k] = v.x; hreg[4 * k + 1] = v.y; hreg[4 * k + 2] = v.z; hreg[4 * k + 3] = v.w;
                }
                bj_h = bj_d;
            }
            ok = __all_sync(0xffffffffu, fs_mbar_wait(fs_smem_u32(tmem_full + sd), (unsigned)(it >> 1) & 1u, abort_flag));
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float a4[4] = {0.f, 0.f, 0.f, 0.f};                  // four chains, joined in a fixed order
#pragma unroll
            for (int c0 = 0; c0 < 32; c0 += 16) {
                float g00[16], g01[16];
                const unsigned t = tmem_base + ((unsigned)((warp & 3) * 32) << 16) + (unsigned)(sd * 2 * FS_N + cq * 32 + c0);
                fs_tmem_ld16(t, g00);
                fs_tmem_ld16(t + FS_N, g01);
                fs_tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 16; ++k) a4[k & 3] = fmaf(hreg[c0 + k], fmaf(2.f, g01[k], g00[k]), a4[k & 3]);
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            const float acc = warp_sum((a4[0] + a4[1]) + (a4[2] + a4[3]));
            if (lane == 0) {
                fs_mbar_arrive(fs_smem_u32(tmem_empty + sd));
                red[sd * FS_WARPS + warp] = acc;
                fs_mbar_arrive(fs_smem_u32(red_full + sd));     // release: orders the store before it
            }
        }
        if (threadIdx.x == 0) {
            // Issued after this thread's drain, so that the contraction runs beside the quantisation
            // of the next item instead of delaying the TMEM loads of the drain.  The sums of item
            // i - 2 first: their slot is rewritten by the drain of item i, which cannot start before
            // the contraction issued below has completed
            bool ok0 = i < 2 || finish_item(i - 2);
            if (ok0 && i < n_items) {
                // ---- contraction of item i ----------------------------------------------------------
                const unsigned ph = (unsigned)(i >> 1) & 1u;
                ok0 = fs_mbar_wait(fs_smem_u32(smem_full + s), ph, abort_flag) &&
                      fs_mbar_wait(fs_smem_u32(tmem_empty + s), ph ^ 1u, abort_flag);
                if (ok0) {
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    // The four 64-column atoms of a stage (D0, D0, D1, D1) lie FS_ATOM_BYTES apart, which
                    // is the descriptor's stride between atoms: as the N = 256 operand the stage is
                    // [D0 | D1], and the 256 accumulator columns are D0^T D0 | D0^T D1.  D0 is read once.
                    const unsigned a0 = fs_smem_u32(smem + s * FS_STAGE_BYTES);
                    const unsigned acc = tmem_base + (unsigned)(s * 2 * FS_N);
#pragma unroll
                    for (int ks = 0; ks < FS_N / 16; ++ks) {
                        const unsigned long long dsc = fs_desc(a0 + ks * 2048);
                        fs_mma(acc, dsc, dsc, ks > 0 ? 1u : 0u);
                    }
                    fs_commit(fs_smem_u32(smem_empty + s));
                    fs_commit(fs_smem_u32(tmem_full + s));
                }
            }
        }
        __syncwarp();
    }
    if (threadIdx.x == 0 && !*abort_flag) {
        finish_item(n_items - 1);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(FS_TMEM_COLS) : "memory");
    if (threadIdx.x == 0 && *abort_flag) sb_latch(ds, SB_ERR_TIMEOUT, SBK_SCORES);
}

// blocks that are not one contraction unit: err[blk][l] = the sum over the block's units (two for
// 256-row blocks) of the unit's entry for the block's half (two halves per unit for 64-column
// blocks); gains
__global__ void full_combine_kernel(const float* __restrict__ unit_err, int64_t n_blocks, int64_t nbc_blocks,
                                    int64_t nbc_units, int units_per_block, int halves, int L, FsBits fb,
                                    float gain_elems, float* __restrict__ err, float* __restrict__ gain) {
    const int64_t blk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (blk >= n_blocks) return;
    const int64_t bi = blk / nbc_blocks, bjb = blk - bi * nbc_blocks;
    const int64_t bj = bjb / halves, half = bjb - bj * halves;
    float prev = 0.f;
    for (int l = 0; l < L; ++l) {
        float e = 0.f;
        for (int u = 0; u < units_per_block; ++u)
            e += unit_err[(((bi * units_per_block + u) * nbc_units + bj) * halves + half) * L + l];
        err[blk * L + l] = e;
        if (gain && l > 0) gain[blk * (L - 1) + l - 1] = (prev - e) / ((float)(fs_bits(fb, l) - fs_bits(fb, l - 1)) * gain_elems);
        prev = e;
    }
}

}  // namespace

extern "C" sb_status sb_block_scores_full(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                                          const int32_t* row_perm, const int32_t* col_perm, const float* H,
                                          const float* row_weight, int br, int bc, int group, const int* bits,
                                          int n_bits, float* err, float* gain, void* W_perm_out) {
    if (!ctx) return SB_ERR_INVALID;
    if (!W || !H || !err || R <= 0 || C <= 0) return sb_fail(ctx, SB_ERR_INVALID, "full scores: null or empty");
    if (!sb_check_bits(bits, n_bits)) return sb_fail(ctx, SB_ERR_INVALID, "full scores: bits must be ascending in 1..8");
    const bool g_ok = group == 16 || group == 32 || group == 64 || group == 128;
    if (!(br == 64 || br == 128 || br == 256) || !(bc == 64 || bc == FS_N) || !g_ok || group > bc || R % br || C % FS_N ||
        ldw % 8 || ldw < C || (reinterpret_cast<uintptr_t>(W) & 15))
        return sb_fail(ctx, SB_ERR_SHAPE, "full scores: blocks of 64, 128 or 256 rows x 64 or 128 columns tiling the "
                                          "matrix (C a multiple of 128), group in {16,32,64,128} and at most the block width");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const int unit_rows = br < FS_N ? br : FS_N;                 // rows of one contraction
    const int units_per_block = br / unit_rows;                  // 1, or 2 for 256-row blocks
    const int halves = FS_N / bc;                                // 64-column blocks: two side by side in a unit
    const int64_t nbc = C / FS_N, n_units = (R / unit_rows) * nbc, n_blocks = (R / br) * (C / bc);
    const bool combine = units_per_block > 1 || halves > 1;
    const bool need_copy = row_perm || col_perm || W_perm_out;
    void* arena;
    sb_status st = sb_scratch(ctx, Carver::need({(size_t)nbc * FS_N * FS_N * 4,
                                                 (need_copy && !W_perm_out) ? (size_t)R * C * 2 : 0,
                                                 combine ? (size_t)n_units * halves * n_bits * 4 : 0}), &arena);
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
    float* unit_err = combine ? cv.take<float>((size_t)n_units * halves * n_bits) : err;
    gather_hblocks_kernel<<<(unsigned)nbc, 256, 0, ctx->stream>>>(H, C, col_perm, hblk);
    SB_LAUNCHED(ctx);
    FsBits fb{};
    for (int l = 0; l < n_bits; ++l) fb.packed |= (unsigned)bits[l] << (4 * l);
    const int64_t grid = n_units < ctx->sm_count ? n_units : ctx->sm_count;
    const float gain_elems = (float)br * (float)bc;
    float* kernel_gain = combine ? nullptr : gain;
    const bool plain = unit_rows == FS_N && !row_weight && halves == 1;
#define FS_LAUNCH_P(G, P)                                                                                         \
    do {                                                                                                          \
        SB_FUNC_ATTR(ctx, (full_scores_kernel<G, P>), cudaFuncAttributeMaxDynamicSharedMemorySize, FS_SMEM);      \
        full_scores_kernel<G, P><<<(unsigned)grid, FS_THREADS, FS_SMEM, ctx->stream>>>(                           \
            src, ld, hblk, fb, n_bits, n_units, nbc, unit_rows, row_weight, row_perm, gain_elems, halves, unit_err, \
            kernel_gain, ctx->dstate);                                                                            \
    } while (0)
#define FS_LAUNCH(G)                                                                                              \
    do {                                                                                                          \
        if (plain) FS_LAUNCH_P(G, true); else FS_LAUNCH_P(G, false);                                              \
    } while (0)
    switch (group) {
        case 16: FS_LAUNCH(16); break;
        case 32: FS_LAUNCH(32); break;
        case 64: FS_LAUNCH(64); break;
        default: FS_LAUNCH(128); break;
    }
#undef FS_LAUNCH
#undef FS_LAUNCH_P
    SB_LAUNCHED(ctx);
    if (combine) {
        full_combine_kernel<<<(unsigned)((n_blocks + 255) / 256), 256, 0, ctx->stream>>>(
            unit_err, n_blocks, C / bc, nbc, units_per_block, halves, n_bits, fb, gain_elems, err, gain);
        SB_LAUNCHED(ctx);
    }
    return SB_OK;
}
