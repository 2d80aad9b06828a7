// Fused mixed-precision dequantisation + matrix product on the packed format (Section 5.3,
// Table 4: dequantise tile by tile, one bitwidth per tile, feed the tensor cores):
//     Y[t][r] = sum_c X[t][c] * (lo[r][g(c)] + scale[r][g(c)] * q[r][c])
// for a few tokens t (decode batches) against a packed R x C matrix.  The codes are small
// integers, exactly representable in bf16, so the contraction runs on the CODES:
//     Y[t][r] = sum over column blocks j of  scale[r][j] * (sum_c X[t][c] q[r][c]) + lo[r][j] * (sum_c X[t][c])
// bf16 x bf16 -> fp32 per block, scaled per row when the block is done; nothing is rounded but
// the fp32 accumulation.
//
// A decode batch is at most 32 tokens against 4 bits per weight on average: the packed bytes
// are what must move, and what costs time is turning codes into tensor-core operands.  A warp
// owns 32 weight rows of a block and feeds the tensor cores from REGISTERS (mma.sync m16n8k16:
// weight rows on M, tokens on N): the unpacked codes are the A fragment where the unpacking
// leaves them, with no trip through shared or tensor memory, no second thread to hand them to
// and no accumulator to fetch back.  (A tcgen05 form of this kernel -- codes stored to tensor
// memory as the A operand of M = 128, N = tokens instructions issued by one thread -- needed the
// same number of instructions per code for the hand-overs between its unpacking, issuing and
// draining warps and was bound by those chains; with so few tokens the contraction is a
// microsecond or two of tensor work on either path.)
//
// Unpacking, one shift and one three-input logic operation per PAIR of codes: lane (g, t) of a
// warp holds the 32 codes 32 t .. 32 t + 31 of rows g and g + 8 of each of its 16-row tiles.
// For b in {1, 2, 4} a 32-bit word of codes gives
//     ((w >> (b s - (7 - b))) & MASK) | 0x43004300  ->  bf16 pair (128 + 2^(7-b) q_s, 128 + 2^(7-b) q_(s + 16/b)):
// the code lands in the top bits of the bf16 mantissa under the exponent of 128.  The offset and
// the power of two are taken out again when the block is scaled (they fold into scale and lo), so
// no subtraction is spent per code.  Codes of 8 bits go through as their two nibbles, the low one
// under the exponent of 128 and the high one under the exponent of 2048 (sixteen times the
// weight), both against the same fragment of X; 3, 5, 6 and 7 bits are cut out of the bit stream
// one by one.  The contraction does not care in which order it visits the columns of a block as
// long as X uses the same one, so a small kernel first writes X in the column order each
// unpacking produces (and the per-block column sums of X).
//
// Grid: (R / block_rows row tiles) x (S column segments); block_rows / 32 contraction warps and
// a loader warp per CTA, two CTAs per SM for 128-row blocks.  The loader warp brings each block
// into a ring in shared memory whose entries are as large as their block (image of X, codes at
// their own bitwidth, the rows' scale and minimum): lane 0 issues two bulk copies (cp.async.bulk,
// mbarrier complete_tx) for the block's packed codes as they lie in memory and for its slice of X
// as the image ldmatrix reads without bank conflicts, all lanes fetch the rows' (scale, minimum)
// with 8-byte asynchronous copies counted on the same barrier.  Each contraction warp: wait for
// the block, read its rows' codes, eight steps of {ldmatrix the next step's tokens, unpack four
// registers per tile, one mma.sync per tile and eight tokens}, release the entry, then
// y += scale' * acc + lo' * colsum(X) in fp32 registers.  With 2 to 8 segments the segments of a
// row tile are the CTAs of one cluster and are added in segment order through distributed shared
// memory; with more, partial sums go to scratch and a second kernel adds them in order.  Every
// mbarrier wait is bounded; on a time-out the kernel latches SB_ERR_TIMEOUT and all roles leave.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int DQ_KB = 128;                  // block columns = quantisation group
constexpr int DQ_MAX_T = 32;                // tokens per pass
constexpr int DQ_MAX_SEG_BLOCKS = 16;       // column blocks per segment (their column sums sit in shared memory)
constexpr int DQ_MT = 2;                    // tiles of 16 rows per contraction warp
constexpr int DQ_MAX_CTAS = 4;              // resident CTAs per SM the launch bounds ask for at most
constexpr int DQ_ORDERS = 5;                // column orders of X: one by one, b = 1, 2, 4, and 8 as byte pairs
constexpr unsigned long long DQ_WAIT_NS = 2000ull * 1000 * 1000;

// candidate bitwidths, four bits each
struct DqBits { unsigned packed; };
__device__ __forceinline__ int dq_bits(DqBits b, int l) { return (int)((b.packed >> (4 * l)) & 15u); }
// column order of X that the unpacking of b-bit codes produces, and the columns its image has
__host__ __device__ inline int dq_order(int b) { return b == 1 ? 1 : b == 2 ? 2 : b == 4 ? 3 : b == 8 ? 4 : 0; }
// first element of order o's images: nbc images of NT x 128 per order
__host__ __device__ inline int64_t dq_order_base(int o, int64_t nbc, int NT) { return (int64_t)o * nbc * NT * DQ_KB; }

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
// one try: the thread may sleep inside the instruction for up to hint_ns before it answers
__device__ __forceinline__ bool dq_mbar_try_wait(unsigned bar, unsigned parity, unsigned hint_ns = 2000u) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
__device__ __noinline__ bool dq_mbar_wait_slow(unsigned bar, unsigned parity, volatile int* abort_flag) {
    unsigned long long t0 = 0;
    for (unsigned spins = 0;; ++spins) {
        if (dq_mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((spins & 15u) == 15u) {
            const unsigned long long now = dq_now_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > DQ_WAIT_NS) { *abort_flag = 1; return false; }
        }
    }
}
// bounded wait: the first try is inline, the rest (with the clock and the abort flag) out of line
__device__ __forceinline__ bool dq_mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag) {
    if (dq_mbar_try_wait(bar, parity)) return true;
    return dq_mbar_wait_slow(bar, parity, abort_flag);
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
__device__ __forceinline__ uint32_t dq_lds32(unsigned addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 dq_lds64(unsigned addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 dq_lds128(unsigned addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
// four 8 x 8 matrices of 16-bit elements: lane L gives the address of row L % 8 of matrix L / 8
// and receives elements 2 (L % 4), 2 (L % 4) + 1 of row L / 4 of each matrix
__device__ __forceinline__ void dq_ldmatrix4(unsigned addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16 weight rows x 8 tokens, fp32) = or += A (16 x 16 codes, from registers) * B (16 x 8, X)
__device__ __forceinline__ void dq_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1, bool first) {
    if (first) {
        asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
            "{%10, %10, %10, %10};"
            : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
    } else {
        asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
            "{%0, %1, %2, %3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
}

// ---- the column order of each unpacking ------------------------------------------------------
// Position p of a block's image = 16 (step) + kappa, kappa = the column index inside one
// m16n8k16: lane t of a quad holds kappa = 2 t, 2 t + 1 (first A register of a row, low and high
// half) and 2 t + 8, 2 t + 9 (second register).  Register i = 2 step + (kappa >> 3) of lane t is
// pair i of that lane's unpacking.  Returns the block column (0..127) that position p holds.
__host__ __device__ inline int dq_source(int o, int p) {
    const int step = p >> 4, kap = p & 15;
    const int t = (kap & 7) >> 1, half = kap & 1, i = 2 * step + (kap >> 3);
    int col;
    if (o == 0) {
        col = 32 * t + 2 * i + half;                       // codes cut out one by one: pair i = codes 2 i, 2 i + 1
    } else if (o <= 3) {
        const int b = 1 << (o - 1), n = 32 / b, hp = n / 2; // pair (m, s) of word m: fields s and s + n / 2
        const int m = i / hp, s = i % hp;
        col = 32 * t + n * m + s + hp * half;
    } else {
        // 8 bits: the lane's words are chunk t (codes 16 t ..) and chunk t + 4 (codes 64 + 16 t ..) of the row;
        // pair i = bytes beta and beta + 2 of word i / 2 (beta = i % 2), whose low and high nibbles go
        // through as two registers against the same columns of X
        const int vw = i >> 1, beta = i & 1;
        col = 16 * (vw < 4 ? t : t + 4) + 4 * (vw & 3) + beta + 2 * half;
    }
    return col;
}

// ---- X in the column orders of the unpacking, and its per-block column sums ------------------
// xp: per order and column block an image of NT rows (tokens) x 128 bf16, laid out as the
// contraction warps read it: 16-byte chunks of a row XOR-swizzled with the token index so that
// the eight rows of an ldmatrix hit different banks; one contiguous copy brings a block's slice
// in.  xsum: [C / 128][NT] fp32.
__device__ __forceinline__ int dq_image_index(int n, int p) {
    return n * DQ_KB + ((((p >> 3) ^ (n & 7))) << 3) + (p & 7);
}
__global__ void __launch_bounds__(DQ_KB)
dq_prepare_x_kernel(const __nv_bfloat16* __restrict__ X, int64_t ldx, int NT, int64_t nbc,
                    __nv_bfloat16* __restrict__ xp, float* __restrict__ xsum) {
    const int64_t jb = blockIdx.x;                       // column block
    const int n = blockIdx.y;                            // token
    const int p = threadIdx.x;                           // position inside an image row, 0..127
    const __nv_bfloat16* xrow = X + (int64_t)n * ldx + jb * DQ_KB;
    // column sum of the block in a fixed order: pairwise inside the warp, then the four warps
    __shared__ float ws[4];
    const float s = warp_sum(__bfloat162float(xrow[p]));
    if ((p & 31) == 0) ws[p >> 5] = s;
    __syncthreads();
    if (p == 0) xsum[jb * NT + n] = (ws[0] + ws[1]) + (ws[2] + ws[3]);
    const int64_t image = (int64_t)NT * DQ_KB;
#pragma unroll
    for (int o = 0; o < DQ_ORDERS; ++o)
        xp[dq_order_base(o, nbc, NT) + jb * image + dq_image_index(n, p)] = xrow[dq_source(o, p)];
}

// ---- unpacking ---------------------------------------------------------------------------------
// Pair i of a row's codes held by this lane (w: the lane's words of the row) as two bf16
// 128 + 2^(7-B) q in one register.
// (x & mask) | c in one instruction; mask and c come in registers so that neither is split off
__device__ __forceinline__ uint32_t dq_and_or(uint32_t x, uint32_t mask, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(x), "r"(mask), "r"(c));
    return d;
}
template <int B>
__device__ __forceinline__ uint32_t dq_pair(const uint32_t* w, int i, uint32_t mask, uint32_t c43) {
    if constexpr (B == 1 || B == 2 || B == 4 || B == 8) {
        // 8 bits: "pair" 2 i' + h is the low (h = 0) or high (h = 1) nibbles of bytes beta, beta + 2 of
        // word i' / 2 (beta = i' % 2), i.e. nibbles s and s + 4 of the word with s = 2 beta + h: the same
        // arithmetic as 4-bit fields, the caller passes 128's exponent for the low and 2048's for the high nibbles
        constexpr int F = B == 8 ? 4 : B;                   // field width
        constexpr int HP = 16 / F;                          // pairs per word
        constexpr int P = 7 - F;                            // the field's lowest bit inside the bf16 mantissa
        const int m = i / HP, s = i % HP;
        const int sh = F * s - P;
        const uint32_t v = sh >= 0 ? (w[m] >> (sh & 31)) : (w[m] << ((-sh) & 31));
        return dq_and_or(v, mask, c43);
    } else {
        // codes 2 i and 2 i + 1 of the lane's 32, code k at bit k B of the lane's B words
        constexpr int P = 7 - B;
        constexpr uint32_t M1 = (1u << B) - 1u;
        uint32_t out = 0x43004300u;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int bit = (2 * i + h) * B, wi = bit >> 5, off = bit & 31;
            uint32_t e;
            if (off + B <= 32) e = w[wi] >> off;
            else e = __funnelshift_r(w[wi], w[wi + 1], off);
            out |= (e & M1) << (P + 16 * h);
        }
        return out;
    }
}
// the mask of dq_pair's fields for B bits, kept in a register across the block
template <int B>
__device__ __forceinline__ uint32_t dq_pair_mask() {
    constexpr int F = B == 8 ? 4 : B;
    constexpr int P = 7 - F;
    return (((1u << F) - 1u) << P) * 0x00010001u;
}

// The lane's words of one weight row.  rowaddr: shared address of the row's codes (16 B bytes);
// t: the lane's place in its quad.
template <int B>
__device__ __forceinline__ void dq_load_row(unsigned rowaddr, int t, uint32_t* w) {
    if constexpr (B == 8) {
        const uint4 a = dq_lds128(rowaddr + 16 * t), b = dq_lds128(rowaddr + 64 + 16 * t);
        w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
    } else if constexpr (B == 4) {
        const uint4 a = dq_lds128(rowaddr + 16 * t);
        w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
    } else if constexpr (B == 2) {
        const uint2 a = dq_lds64(rowaddr + 8 * t);
        w[0] = a.x; w[1] = a.y;
    } else {
#pragma unroll
        for (int k = 0; k < B; ++k) w[k] = dq_lds32(rowaddr + 4 * B * t + 4 * k);
    }
}

// One block for one warp: acc[m][nt][.] = sum over the block's columns of codes x X for the warp's
// 16 MT rows (MT tiles of 16) and tokens 8 nt .. 8 nt + 7; every fragment of X that is fetched
// serves all MT tiles.  codes: shared address of the warp's first row in the stage; xlane: the
// lane's ldmatrix row address(es) in the stage's image, before the step is XOR-ed in; meta[m][h]:
// (scale, minimum) of row 16 m + 8 h + g.
template <int B, int NT, int MT>
__device__ __forceinline__ void dq_block(unsigned codes, const unsigned (&xlane)[2], int g, int t,
                                         unsigned empty_bar, int lane, const float2 (&meta)[MT][2], unsigned xs_addr,
                                         float (&y)[MT][NT / 8][4]) {
    float acc[MT][NT / 8][4];
    constexpr int VW = B == 8 ? 8 : B;
    constexpr int STEPS = 8;
    constexpr int SUB = B == 8 ? 2 : 1;         // 8 bits: low and high nibbles against the same columns of X
    uint32_t w[MT][2][VW];
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        dq_load_row<B>(codes + (unsigned)((16 * m + g) * 16 * B), t, w[m][0]);
        dq_load_row<B>(codes + (unsigned)((16 * m + g + 8) * 16 * B), t, w[m][1]);
    }
    // the constants of the unpacking live in registers (an immediate would split the operation in
    // two): the field mask and the exponent under which the field sits, 128 (x 16 for high nibbles)
    uint32_t mask = dq_pair_mask<B>(), c43 = 0x43004300u, c45 = 0x45004500u;
    asm volatile("" : "+r"(mask), "+r"(c43), "+r"(c45));
    // registers 2 ks and 2 ks + 1 of step ks (8 bits: of its low, then of its high nibbles)
    auto a_regs = [&](int m, int ks, int sub, uint32_t (&a)[4]) {
        const int i0 = SUB * (2 * ks) + sub, i1 = SUB * (2 * ks + 1) + sub;
        const uint32_t c = sub ? c45 : c43;
        a[0] = dq_pair<B>(w[m][0], i0, mask, c);
        a[1] = dq_pair<B>(w[m][1], i0, mask, c);
        a[2] = dq_pair<B>(w[m][0], i1, mask, c);
        a[3] = dq_pair<B>(w[m][1], i1, mask, c);
    };
    if constexpr (NT == 8) {
        // one ldmatrix brings the fragments of two steps; the next pair of steps is fetched a pair ahead
        uint32_t bf[2][4];
        dq_ldmatrix4(xlane[0], bf[0]);
#pragma unroll
        for (int ks = 0; ks < STEPS; ++ks) {
            if ((ks & 1) == 0 && ks + 2 < STEPS) dq_ldmatrix4(xlane[0] ^ (unsigned)((ks + 2) << 5), bf[((ks >> 1) + 1) & 1]);
            const uint32_t(&cur)[4] = bf[(ks >> 1) & 1];
#pragma unroll
            for (int sub = 0; sub < SUB; ++sub) {
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    uint32_t a[4];
                    a_regs(m, ks, sub, a);
                    dq_mma(acc[m][0], a, cur[2 * (ks & 1)], cur[2 * (ks & 1) + 1], ks == 0 && sub == 0);
                }
            }
        }
    } else {
        // the tokens' fragments of step ks + 1 are fetched before the products of step ks are issued
        constexpr int NQ = NT / 16;
        uint32_t bf[2][NQ][4];
#pragma unroll
        for (int q = 0; q < NQ; ++q) dq_ldmatrix4(xlane[q], bf[0][q]);
#pragma unroll
        for (int ks = 0; ks < STEPS; ++ks) {
            if (ks + 1 < STEPS) {
#pragma unroll
                for (int q = 0; q < NQ; ++q) dq_ldmatrix4(xlane[q] ^ (unsigned)((ks + 1) << 5), bf[(ks + 1) & 1][q]);
            }
#pragma unroll
            for (int sub = 0; sub < SUB; ++sub) {
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    uint32_t a[4];
                    a_regs(m, ks, sub, a);
#pragma unroll
                    for (int q = 0; q < NQ; ++q) {
                        dq_mma(acc[m][2 * q], a, bf[ks & 1][q][0], bf[ks & 1][q][1], ks == 0 && sub == 0);
                        dq_mma(acc[m][2 * q + 1], a, bf[ks & 1][q][2], bf[ks & 1][q][3], ks == 0 && sub == 0);
                    }
                }
            }
        }
    }
    __syncwarp();
    if (lane == 0) dq_mbar_arrive(empty_bar);            // codes and image are in registers
    // codes went in as 128 + 2^P q (P = 7 - B; 8 bits: low nibbles as 128 + 8 n, high nibbles as
    // 2048 + 128 n, offset 128 * 17): sum_c x q = (acc - OFF colsum) / 2^P, folded into the row's
    // scale and minimum
    constexpr float INV = B == 8 ? 0.125f : 1.f / (float)(1 << (7 - B));
    constexpr float OFF = B == 8 ? 2176.f : 128.f;
    float sc[MT][2], lo[MT][2];
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            sc[m][h] = meta[m][h].x * INV;
            lo[m][h] = fmaf(-sc[m][h], OFF, meta[m][h].y);
        }
    }
#pragma unroll
    for (int nt = 0; nt < NT / 8; ++nt) {
        const uint2 cu = dq_lds64(xs_addr + 32 * nt);
        const float cx = __uint_as_float(cu.x), cy = __uint_as_float(cu.y);
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            y[m][nt][0] = fmaf(sc[m][0], acc[m][nt][0], fmaf(lo[m][0], cx, y[m][nt][0]));
            y[m][nt][1] = fmaf(sc[m][0], acc[m][nt][1], fmaf(lo[m][0], cy, y[m][nt][1]));
            y[m][nt][2] = fmaf(sc[m][1], acc[m][nt][2], fmaf(lo[m][1], cx, y[m][nt][2]));
            y[m][nt][3] = fmaf(sc[m][1], acc[m][nt][3], fmaf(lo[m][1], cy, y[m][nt][3]));
        }
    }
}

struct DqArgs {
    const uint32_t* packed;
    const int64_t* block_off;       // [nb + 1], words
    const float2* meta;             // [(r * nbc + j)] = (scale, lo), group == block width
    const uint8_t* level;           // [nb]
    const __nv_bfloat16* xp;        // per order, per column block: image of NT x 128
    const float* xsum;              // [nbc][NT]
    float* out;                     // partial sums [S][T][R] (or Y when S == 1)
    int64_t out_t_stride;           // R for the partial sums, ldy for Y
    int64_t out_seg_stride;
    int64_t R, C;
    int nbc, seg_blocks, T;
    int cluster_sum;                // the segments of a row tile are one cluster: summed through shared memory, out = Y
    DqBits bits;
    SbDeviceState* ds;
};

// WARPS contraction warps of MT tiles of 16 rows each.  A block's entry in the CTA's ring is its
// image of X, its codes at their own bitwidth and its rows' (scale, minimum): entries are as large
// as their block, so that low-bit blocks leave room for more blocks in flight.
template <int NT, int WARPS, int MT> struct DqShape {
    static constexpr int ROWS = 16 * MT * WARPS;                    // block rows
    static constexpr int X_BYTES = NT * DQ_KB * 2;                  // an image: NT x 128 bf16
    static constexpr int META_BYTES = ROWS * 8;                     // (scale, minimum) of the block's rows
    static constexpr int RING_BYTES = WARPS >= 4 ? 104 * 1024 : 46 * 1024;
    static constexpr int THREADS = (WARPS + 1) * 32;                // + loader warp
    static constexpr int SMEM = RING_BYTES + DQ_MAX_SEG_BLOCKS * NT * 4 + 256 /* alignment */ +
                                512 /* barriers, block table */;
    // resident CTAs per SM by shared memory (227 KB, 1 KB reserved per CTA), at most DQ_MAX_CTAS
    static constexpr int FIT = (227 * 1024) / (SMEM + 1024);
    static constexpr int CTAS_PER_SM = FIT > DQ_MAX_CTAS ? DQ_MAX_CTAS : FIT;
    __host__ __device__ static constexpr int entry_bytes(int b) { return X_BYTES + ROWS * 16 * b + META_BYTES; }
    static_assert(X_BYTES + ROWS * 16 * 8 + META_BYTES <= RING_BYTES, "the largest entry fits the ring");
};

template <int NT, int WARPS, int MT>
__global__ void __launch_bounds__(DqShape<NT, WARPS, MT>::THREADS, DqShape<NT, WARPS, MT>::CTAS_PER_SM)
dequant_gemm_kernel(const DqArgs a) {
    using S = DqShape<NT, WARPS, MT>;
    extern __shared__ unsigned char dq_smem_raw[];
    // the ring (256-byte aligned in the shared window: entries are multiples of 256 bytes and start
    // with the image, whose swizzle is an XOR on the address bits below a row's 256 bytes)
    unsigned char* smem = dq_smem_raw + ((256u - (dq_smem_u32(dq_smem_raw) & 255u)) & 255u);
    float* xs = reinterpret_cast<float*>(smem + S::RING_BYTES);             // [seg_blocks][NT] column sums
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(xs + DQ_MAX_SEG_BLOCKS * NT);
    // one pair of barriers per block of the segment, each used once
    unsigned long long* full = bars;                        // [j] the block's copies have landed
    unsigned long long* empty = bars + DQ_MAX_SEG_BLOCKS;   // [j] every contraction warp has read the block
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty + DQ_MAX_SEG_BLOCKS);
    // per block of the segment: first word of its codes (blocks are below 2^32 words apart from the
    // segment's first), where its entry starts in the ring (written by the loader before the
    // block's barrier is armed) and its bitwidth
    unsigned* blk_word = reinterpret_cast<unsigned*>(const_cast<int*>(abort_flag) + 4);   // [DQ_MAX_SEG_BLOCKS]
    unsigned* blk_at = blk_word + DQ_MAX_SEG_BLOCKS;
    unsigned char* blk_bits = reinterpret_cast<unsigned char*>(blk_at + DQ_MAX_SEG_BLOCKS);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int bi = blockIdx.x;                                  // row tile
    const int j0 = blockIdx.y * a.seg_blocks;                   // first column block of the segment
    const int nblk = min(a.seg_blocks, a.nbc - j0);

    // Set-up is the loader warp's: it arms the barriers, reads the segment's block table (one load of
    // the offsets, one of the levels) and starts the first copies without waiting for the other
    // warps, which meanwhile fetch the segment's column sums of X; they meet it at a named barrier on
    // which the loader only arrives.
    const int64_t blk0 = (int64_t)bi * a.nbc + j0;
    int64_t word0 = 0;
    if (warp == WARPS) {
        if (lane < nblk) {
            dq_mbar_init(dq_smem_u32(full + lane), 1 + 32);     // the bulk copies' expect_tx and the loader lanes' row copies
            dq_mbar_init(dq_smem_u32(empty + lane), WARPS);
        }
        if (lane == 0) *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const int64_t off = lane <= nblk ? a.block_off[blk0 + lane] : 0;
        const int lv = lane < nblk ? (int)a.level[blk0 + lane] : 0;
        word0 = __shfl_sync(0xffffffffu, off, 0);
        if (lane < nblk) {
            blk_word[lane] = (unsigned)(off - word0);
            blk_bits[lane] = (unsigned char)dq_bits(a.bits, lv);
        }
        __syncwarp();
        asm volatile("bar.arrive 2, %0;" ::"r"(S::THREADS) : "memory");
    } else {
        for (int i = threadIdx.x; i < nblk * NT; i += WARPS * 32) xs[i] = a.xsum[(int64_t)j0 * NT + i];
        asm volatile("bar.sync 2, %0;" ::"r"(S::THREADS) : "memory");
    }
    const float2* mbase = a.meta + ((int64_t)bi * S::ROWS) * a.nbc + j0;
    // what the loader does for block j
    auto load_codes_meta = [&](int j, unsigned at) {
        const unsigned bar = dq_smem_u32(full + j);
        const unsigned code_bytes = (unsigned)(S::ROWS * 16 * blk_bits[j]);
        if (lane == 0) {
            blk_at[j] = at;
            dq_mbar_expect_tx(bar, code_bytes + (unsigned)S::X_BYTES);
            dq_bulk_load(dq_smem_u32(smem + at + S::X_BYTES), a.packed + word0 + blk_word[j], code_bytes, bar);   // word0: the loader's
        }
        const unsigned mdst = dq_smem_u32(smem + at + S::X_BYTES) + code_bytes;
#pragma unroll
        for (int r = lane; r < S::ROWS; r += 32)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(mdst + 8u * r), "l"(mbase + (int64_t)r * a.nbc + j)
                         : "memory");
        // counted on the block's barrier when this lane's copies have landed
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
    };
    auto load_image = [&](int j, unsigned at) {
        if (lane == 0)
            dq_bulk_load(dq_smem_u32(smem + at),
                         a.xp + dq_order_base(dq_order(blk_bits[j]), a.nbc, NT) + (int64_t)(j0 + j) * (NT * DQ_KB),
                         (unsigned)S::X_BYTES, dq_smem_u32(full + j));
    };
    // The ring: entries in order of the blocks, each where the one before it ends, back to the
    // start when the end is reached; `head` = where the next entry goes, `tail` = the oldest block
    // not yet known to be released (its entry is the first thing `head` would run into).
    unsigned head = 0;
    int tail = 0, jl = 0;
    bool lok = true;
    // place block j: returns its offset, waiting for older blocks to be released where it must
    auto place = [&](int j, bool may_wait, unsigned& at) -> bool {
        const unsigned sz = (unsigned)S::entry_bytes(blk_bits[j]);
        for (;;) {
            if (tail == j) { head = 0; break; }                          // nothing in flight: start over
            const unsigned ta = blk_at[tail];
            if (head > ta) {                                             // in flight: [ta, head)
                if (head + sz <= (unsigned)S::RING_BYTES) break;
                if (sz <= ta) { head = 0; break; }
            } else if (head + sz <= ta) {                                // in flight: [ta, end) and [0, head)
                break;
            }
            if (!may_wait) return false;
            lok = dq_mbar_wait(dq_smem_u32(empty + tail), 0u, abort_flag);
            lok = __all_sync(0xffffffffu, lok);
            if (!lok) return false;
            ++tail;
        }
        at = head;
        head += sz;
        return true;
    };

    if (warp == WARPS) {
        // ---- loader warp: the codes of block j as they lie in memory and its slice of X (an image in
        // the order of the block's bitwidth) by two bulk copies of lane 0, the rows' (scale, minimum) by
        // 8-byte asynchronous copies of all lanes, into the ring as soon as the blocks whose entries are
        // in the way have been let go of by every contraction warp ------------------------------------
        for (jl = 0; jl < nblk && lok; ++jl) {
            unsigned at;
            if (!place(jl, true, at)) break;
            __syncwarp();
            load_codes_meta(jl, at);
            load_image(jl, at);
            __syncwarp();
        }
    } else {
        // ---- contraction warps: 16 MT weight rows each --------------------------------------------------
        const int g = lane >> 2, t = lane & 3;
        const int64_t row_lo = (int64_t)bi * S::ROWS + warp * (16 * MT) + g;   // rows row_lo + 16 m + 8 h
        // the lane's ldmatrix row inside an image, without the stage: matrix mi = lane / 8, row r8 = lane % 8
        const int mi = lane >> 3, r8 = lane & 7;
        constexpr unsigned pitch = 2u * DQ_KB;                          // bytes of an image row
        unsigned xoff[2];
        if constexpr (NT == 8) {
            // matrices: (step, low half), (step, high half), (step + 1, low), (step + 1, high) of tokens 0..7
            xoff[0] = ((unsigned)r8 * pitch + (unsigned)((((mi & 1) ^ r8) << 4))) ^ (unsigned)((mi >> 1) << 5);
            xoff[1] = 0;
        } else {
            // matrices: tokens 16 q + 8 (mi / 2) .., low (mi even) or high (mi odd) half of the step
#pragma unroll
            for (int q = 0; q < 2; ++q)
                xoff[q] = (unsigned)(16 * q + 8 * (mi >> 1) + r8) * pitch + (unsigned)(((mi & 1) ^ r8) << 4);
        }
        float y[MT][NT / 8][4];
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int nt = 0; nt < NT / 8; ++nt) y[m][nt][0] = y[m][nt][1] = y[m][nt][2] = y[m][nt][3] = 0.f;
        bool ok = true;
        for (int j = 0; j < nblk && ok; ++j) {
            ok = dq_mbar_wait(dq_smem_u32(full + j), 0u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int b = blk_bits[j];                       // uniform over the CTA
            const unsigned stage = dq_smem_u32(smem) + blk_at[j];
            const unsigned codes = stage + S::X_BYTES + (unsigned)(warp * (16 * MT) * 16 * b);
            const unsigned metas = stage + S::X_BYTES + (unsigned)(S::ROWS * 16 * b);
            const unsigned xlane[2] = {stage + xoff[0], stage + xoff[1]};
            const unsigned eb = dq_smem_u32(empty + j);
            const unsigned xa = dq_smem_u32(xs + j * NT + 2 * t);
            // (scale, minimum) of rows 16 m + 8 h + g of the warp
            float2 cur[MT][2];
#pragma unroll
            for (int m = 0; m < MT; ++m)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint2 v = dq_lds64(metas + 8u * (unsigned)(warp * (16 * MT) + 16 * m + 8 * h + g));
                    cur[m][h] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
                }
            switch (b) {
                case 1: dq_block<1, NT, MT>(codes, xlane, g, t, eb, lane, cur, xa, y); break;
                case 2: dq_block<2, NT, MT>(codes, xlane, g, t, eb, lane, cur, xa, y); break;
                case 3: dq_block<3, NT, MT>(codes, xlane, g, t, eb, lane, cur, xa, y); break;
                case 4: dq_block<4, NT, MT>(codes, xlane, g, t, eb, lane, cur, xa, y); break;
                case 5: dq_block<5, NT, MT>(codes, xlane, g, t, eb, lane, cur, xa, y); break;
                case 6: dq_block<6, NT, MT>(codes, xlane, g, t, eb, lane, cur, xa, y); break;
                case 7: dq_block<7, NT, MT>(codes, xlane, g, t, eb, lane, cur, xa, y); break;
                default: dq_block<8, NT, MT>(codes, xlane, g, t, eb, lane, cur, xa, y); break;
            }
        }
        if (a.cluster_sum) {
            // all of the CTA's warps are past their last block before the ring's memory is reused
            asm volatile("bar.sync 1, %0;" ::"r"(WARPS * 32) : "memory");
            float* ysm = reinterpret_cast<float*>(smem);                 // [NT][ROWS] partial sums of the segment
#pragma unroll
            for (int m = 0; m < MT; ++m)
#pragma unroll
                for (int nt = 0; nt < NT / 8; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        ysm[(8 * nt + 2 * t + (e & 1)) * S::ROWS + warp * (16 * MT) + 16 * m + 8 * (e >> 1) + g] =
                            ok ? y[m][nt][e] : 0.f;
        } else if (ok) {
            float* out = a.out + (int64_t)blockIdx.y * a.out_seg_stride;
#pragma unroll
            for (int m = 0; m < MT; ++m) {
#pragma unroll
                for (int nt = 0; nt < NT / 8; ++nt) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int tok = 8 * nt + 2 * t + (e & 1);
                        if (!isfinite(y[m][nt][e])) sb_latch(a.ds, SB_ERR_NONFINITE, SBK_GEMM);
                        if (tok < a.T) out[(int64_t)tok * a.out_t_stride + row_lo + 16 * m + 8 * (e >> 1)] = y[m][nt][e];
                    }
                }
            }
        }
    }
    if (a.cluster_sum) {
        // the segments of this row tile are the CTAs of one cluster, rank = segment: every CTA adds a
        // slice of the tile's outputs over all segments, in segment order, out of their shared memory
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();
        const float* ysm = reinterpret_cast<const float*>(smem);
        const int nseg = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
        const int total = a.T * S::ROWS, chunk = (total + nseg - 1) / nseg;
        const int end = min(total, (rank + 1) * chunk);
        // the remote reads of an output are issued together (up to 8 segments), then added in order
        const float* seg[8];
#pragma unroll
        for (int sgm = 0; sgm < 8; ++sgm) seg[sgm] = cluster.map_shared_rank(ysm, sgm < nseg ? sgm : 0);
        // four outputs per thread at a time, so that up to 32 remote reads are in flight
        constexpr int OU = 4;
        for (int base = rank * chunk + (int)threadIdx.x; base < end; base += OU * S::THREADS) {
            float v[OU][8];
#pragma unroll
            for (int u = 0; u < OU; ++u) {
                const int idx = base + u * S::THREADS;
#pragma unroll
                for (int sgm = 0; sgm < 8; ++sgm) v[u][sgm] = (sgm < nseg && idx < end) ? seg[sgm][idx] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < OU; ++u) {
                const int idx = base + u * S::THREADS;
                float acc = 0.f;
#pragma unroll
                for (int sgm = 0; sgm < 8; ++sgm) acc += v[u][sgm];
                if (!isfinite(acc)) sb_latch(a.ds, SB_ERR_NONFINITE, SBK_GEMM);
                if (idx < end)
                    a.out[(int64_t)(idx / S::ROWS) * a.out_t_stride + (int64_t)bi * S::ROWS + idx % S::ROWS] = acc;
            }
        }
        cluster.sync();                     // nobody leaves while its shared memory may still be read
    }
    __syncthreads();
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

template <int NT, int WARPS>
sb_status dq_launch(sb_ctx* ctx, const DqArgs& a, dim3 grid) {
    using S = DqShape<NT, WARPS, DQ_MT>;
    SB_FUNC_ATTR(ctx, (dequant_gemm_kernel<NT, WARPS, DQ_MT>), cudaFuncAttributeMaxDynamicSharedMemorySize, S::SMEM);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(S::THREADS);
    cfg.dynamicSmemBytes = S::SMEM;
    cfg.stream = ctx->stream;
    cudaLaunchAttribute attr[1];
    cfg.numAttrs = 0;
    if (a.cluster_sum) {
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 1;
        attr[0].val.clusterDim.y = grid.y;
        attr[0].val.clusterDim.z = 1;
        cfg.numAttrs = 1;
    }
    cfg.attrs = attr;
    SB_CUDA(ctx, cudaLaunchKernelEx(&cfg, dequant_gemm_kernel<NT, WARPS, DQ_MT>, a));
    SB_LAUNCHED(ctx);
    return SB_OK;
}
// Can a cluster of `segments` CTAs of this instance be resident at all (it can on a whole B200; a
// partition with fewer SMs per GPC may not hold one)?  Asked from the occupancy calculator.
template <int NT, int WARPS>
bool dq_cluster_fits(sb_ctx* ctx, int segments) {
    using S = DqShape<NT, WARPS, DQ_MT>;
    const void* f = reinterpret_cast<const void*>(dequant_gemm_kernel<NT, WARPS, DQ_MT>);
    if (!ctx->configured.count(f)) {
        if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, S::SMEM) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        ctx->configured.insert(f);
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(1, (unsigned)segments);
    cfg.blockDim = dim3(S::THREADS);
    cfg.dynamicSmemBytes = S::SMEM;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = (unsigned)segments;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, dequant_gemm_kernel<NT, WARPS, DQ_MT>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return n >= 1;
}
// contraction warps of a CTA for blocks of br rows; resident CTAs per SM of the instance that
// serves (tokens padded to NT, block rows)
constexpr int dq_warps(int br) { return br / (16 * DQ_MT); }
bool dq_cluster_ok(sb_ctx* ctx, int NT, int br, int segments) {
    if (br == 128)
        return NT == 8 ? dq_cluster_fits<8, dq_warps(128)>(ctx, segments)
                       : NT == 16 ? dq_cluster_fits<16, dq_warps(128)>(ctx, segments) : dq_cluster_fits<32, dq_warps(128)>(ctx, segments);
    return NT == 8 ? dq_cluster_fits<8, dq_warps(64)>(ctx, segments)
                   : NT == 16 ? dq_cluster_fits<16, dq_warps(64)>(ctx, segments) : dq_cluster_fits<32, dq_warps(64)>(ctx, segments);
}
int dq_ctas_per_sm(int NT, int br) {
    if (br == 128)
        return NT == 8 ? DqShape<8, dq_warps(128), DQ_MT>::CTAS_PER_SM
                       : NT == 16 ? DqShape<16, dq_warps(128), DQ_MT>::CTAS_PER_SM : DqShape<32, dq_warps(128), DQ_MT>::CTAS_PER_SM;
    return NT == 8 ? DqShape<8, dq_warps(64), DQ_MT>::CTAS_PER_SM
                   : NT == 16 ? DqShape<16, dq_warps(64), DQ_MT>::CTAS_PER_SM : DqShape<32, dq_warps(64), DQ_MT>::CTAS_PER_SM;
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
    if ((br != 64 && br != 128) || bc != DQ_KB || group != DQ_KB || R % br || C % DQ_KB || ldx < C || ldy < R ||
        (reinterpret_cast<uintptr_t>(packed) & 15))
        return sb_fail(ctx, SB_ERR_SHAPE,
                       "dequant gemm: blocks of 64 x 128 or 128 x 128 with group 128 tiling the matrix, 16-byte aligned codes");
    if (R >= (1ll << 31) || C >= (1ll << 31)) return sb_fail(ctx, SB_ERR_SHAPE, "dequant gemm: R and C must fit 31 bits");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const int nbc = (int)(C / DQ_KB);
    const int64_t nbr = R / br;
    // column segments: enough CTAs to fill every SM's slots once, at most DQ_MAX_SEG_BLOCKS blocks each
    const int NT0 = T <= 8 ? 8 : T <= 16 ? 16 : 32;            // the first (largest) slice decides the segments
    int S = (int)((dq_ctas_per_sm(NT0, br) * (int64_t)ctx->sm_count) / nbr);
    if (S < 1) S = 1;
    if (S > nbc) S = nbc;
    int seg_blocks = (nbc + S - 1) / S;
    if (seg_blocks > DQ_MAX_SEG_BLOCKS) seg_blocks = DQ_MAX_SEG_BLOCKS;
    S = (nbc + seg_blocks - 1) / seg_blocks;
    if (S > 65535) return sb_fail(ctx, SB_ERR_SHAPE, "dequant gemm: too many column segments");
    DqBits db{};
    for (int l = 0; l < n_bits; ++l) db.packed |= (unsigned)bits[l] << (4 * l);
    // how the segments of a row tile are added: as one (portable) cluster through shared memory, or by
    // a second kernel over partial sums in scratch
    const bool cluster_sum = S >= 2 && S <= 8 && dq_cluster_ok(ctx, NT0, br, S);
    const bool two_pass = S > 1 && !cluster_sum;
    // tokens in slices of at most DQ_MAX_T (padded to 8, 16 or 32 with zero rows)
    for (int64_t t0 = 0; t0 < T; t0 += DQ_MAX_T) {
        const int Tn = (int)((T - t0) < DQ_MAX_T ? (T - t0) : DQ_MAX_T);
        const int NT = Tn <= 8 ? 8 : Tn <= 16 ? 16 : 32;
        const size_t image_elems = (size_t)DQ_ORDERS * NT * C;
        void* arena;
        sb_status st = sb_scratch(ctx, Carver::need({image_elems * 2, (size_t)nbc * NT * 4,
                                                     two_pass ? (size_t)S * Tn * R * 4 : 0}), &arena);
        if (st != SB_OK) return st;
        Carver cv(arena);
        __nv_bfloat16* xp = cv.take<__nv_bfloat16>(image_elems);
        float* xsum = cv.take<float>((size_t)nbc * NT);
        float* part = two_pass ? cv.take<float>((size_t)S * Tn * R) : nullptr;
        const __nv_bfloat16* Xs = static_cast<const __nv_bfloat16*>(X) + t0 * ldx;
        if (Tn < NT) {      // zero rows for the padding tokens
            SB_CUDA(ctx, cudaMemsetAsync(xp, 0, image_elems * 2, ctx->stream));
            SB_CUDA(ctx, cudaMemsetAsync(xsum, 0, (size_t)nbc * NT * 4, ctx->stream));
        }
        dq_prepare_x_kernel<<<dim3((unsigned)nbc, (unsigned)Tn), DQ_KB, 0, ctx->stream>>>(Xs, ldx, NT, nbc, xp, xsum);
        SB_LAUNCHED(ctx);
        DqArgs a{};
        a.packed = packed; a.block_off = block_off_words; a.meta = reinterpret_cast<const float2*>(meta);
        a.level = level; a.xp = xp; a.xsum = xsum;
        a.cluster_sum = cluster_sum ? 1 : 0;
        a.out = two_pass ? part : Y + t0 * ldy;
        a.out_t_stride = two_pass ? R : ldy;
        a.out_seg_stride = two_pass ? (int64_t)Tn * R : 0;
        a.R = R; a.C = C; a.nbc = nbc; a.seg_blocks = seg_blocks; a.T = Tn; a.bits = db; a.ds = ctx->dstate;
        const dim3 grid((unsigned)nbr, (unsigned)S);
        if (br == 128) {
            constexpr int W = dq_warps(128);
            st = NT == 8 ? dq_launch<8, W>(ctx, a, grid) : NT == 16 ? dq_launch<16, W>(ctx, a, grid)
                                                                    : dq_launch<32, W>(ctx, a, grid);
        } else {
            constexpr int W = dq_warps(64);
            st = NT == 8 ? dq_launch<8, W>(ctx, a, grid) : NT == 16 ? dq_launch<16, W>(ctx, a, grid)
                                                                    : dq_launch<32, W>(ctx, a, grid);
        }
        if (st != SB_OK) return st;
        if (two_pass) {
            dq_reduce_kernel<<<dim3((unsigned)((R + 255) / 256), (unsigned)Tn), 256, 0, ctx->stream>>>(part, S, Tn, R,
                                                                                                       Y + t0 * ldy, ldy);
            SB_LAUNCHED(ctx);
        }
    }
    return SB_OK;
}
