// Pack: integer codes of every block at its assigned bitwidth, bit-packed, plus per-group
// (scale, min).  The code arithmetic is IEEE binary64 in a fixed operation order so that the
// integers are reproducible bit for bit:
//   range = hi - lo; inv = qmax / range; q = rint((v - lo) * inv); scale = range / qmax.
#include "lookback.cuh"

sb_status sb_gather_bf16(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                         const int32_t* rp, const int32_t* cp, void* out);

namespace {

constexpr int PK_THREADS = 128;
constexpr int PK_WARPS = PK_THREADS / 32;

struct PackBits { int bits[8]; };

// block_off[i] = first 32-bit word of block i = exclusive prefix sum of the block sizes
// (block_rows*block_cols*bits[level] / 32), block_off[nb] = total; one look-back scan.
constexpr int PO_THREADS = 256, PO_ITEMS = 8, PO_TILE = PO_THREADS * PO_ITEMS;
__global__ void __launch_bounds__(PO_THREADS)
pack_offsets_kernel(const unsigned char* __restrict__ level, int64_t nb, int n_bits, PackBits pb,
                    unsigned long long words_per_bit, unsigned long long* __restrict__ block_off,
                    LookbackBuf lb, SbDeviceState* ds) {
    const unsigned tile = lookback_tile_id(ds);
    const int64_t base = (int64_t)tile * PO_TILE + (int64_t)threadIdx.x * PO_ITEMS;
    unsigned long long v[PO_ITEMS], sum = 0ull;
#pragma unroll
    for (int k = 0; k < PO_ITEMS; ++k) {
        v[k] = 0ull;
        if (base + k < nb) {
            int l = level[base + k];
            if (l >= n_bits) { sb_latch(ds, SB_ERR_INVALID, SBK_PACK); l = n_bits - 1; }
            int b = pb.bits[0];
#pragma unroll
            for (int j = 1; j < 8; ++j) b = (l == j) ? pb.bits[j] : b;
            v[k] = words_per_bit * (unsigned long long)b;
        }
        sum += v[k];
    }
    unsigned long long tile_total;
    const unsigned long long ex = block_exclusive_scan<unsigned long long, PO_THREADS>(sum, tile_total);
    const unsigned long long prefix = lookback_prefix<unsigned long long>(tile_total, tile, lb, ds);
    unsigned long long run = prefix + ex;
#pragma unroll
    for (int k = 0; k < PO_ITEMS; ++k) {
        if (base + k < nb) block_off[base + k] = run;
        run += v[k];
    }
    if (tile == gridDim.x - 1 && threadIdx.x == PO_THREADS - 1) block_off[nb] = run;
    lookback_finish(ds, lb);
}

// The same for a matrix whose blocks fit one CTA (up to 1024 x PO1_ITEMS): a plain CTA scan,
// no descriptors, no ticket.
constexpr int PO1_THREADS = 1024, PO1_ITEMS = 8;
__global__ void __launch_bounds__(PO1_THREADS)
pack_offsets_small_kernel(const unsigned char* __restrict__ level, int nb, int n_bits, PackBits pb,
                          unsigned long long words_per_bit, unsigned long long* __restrict__ block_off,
                          SbDeviceState* ds) {
    const int base = (int)threadIdx.x * PO1_ITEMS;
    unsigned long long v[PO1_ITEMS], sum = 0ull;
#pragma unroll
    for (int k = 0; k < PO1_ITEMS; ++k) {
        v[k] = 0ull;
        if (base + k < nb) {
            int l = level[base + k];
            if (l >= n_bits) { sb_latch(ds, SB_ERR_INVALID, SBK_PACK); l = n_bits - 1; }
            int b = pb.bits[0];
#pragma unroll
            for (int j = 1; j < 8; ++j) b = (l == j) ? pb.bits[j] : b;
            v[k] = words_per_bit * (unsigned long long)b;
        }
        sum += v[k];
    }
    unsigned long long total;
    unsigned long long run = block_exclusive_scan<unsigned long long, PO1_THREADS>(sum, total);
#pragma unroll
    for (int k = 0; k < PO1_ITEMS; ++k) {
        if (base + k < nb) block_off[base + k] = run;
        run += v[k];
    }
    if (threadIdx.x == 0) block_off[nb] = total;
}



constexpr double PK_MAGIC64 = 6755399441055744.0;     // 1.5 * 2^52: low word of (t + MAGIC) = rint(t)

// 16 codes of B bits -> 16*B bits in w[0..3] (little-endian bit stream).  All positions are
// compile-time constants; the fields are disjoint, so adding is the same as or-ing.
template <int B>
__device__ __forceinline__ void pack16(const unsigned (&code)[16], unsigned (&w)[4]) {
    w[0] = w[1] = w[2] = w[3] = 0u;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const int bit = k * B, j = bit >> 5, sh = bit & 31;
        w[j] += code[k] << sh;
        if (sh + B > 32) w[j + 1] += code[k] >> (32 - sh);
    }
}

// What a lane needs to know about its place in the CTA's chunk.
struct PackLane {
    const __nv_bfloat16* colp;   // W + first column of the lane
    const int32_t* rp;           // row permutation applied at load time, or null
    int64_t ldw, row0;           // leading dimension, first row of the block row
    int br, team;                // block rows; lanes per quantisation group
    float2* meta;                // metadata of the lane's group in row row0
    int64_t meta_ld;             // groups per matrix row
    unsigned* dst;               // first word of the lane in row row0 of its block
    unsigned row_words;          // words per block row
    bool meta_lane, odd_lane;
    const unsigned* packed;      // the packed buffer and its capacity in words (checked build)
    long long capacity;
    SbDeviceState* ds;
};

// One (row, 16 columns) per lane and step: binary64 codes of the lane's 16 weights.
// Returns the stored scale; code[] is all zero for a constant group.
template <typename QMAX>
__device__ __forceinline__ float encode16(const uint32_t (&wv)[8], float lo, float hi, QMAX qmax,
                                          unsigned (&code)[16]) {
    const double dlo = (double)lo;
    const double range64 = __dsub_rn((double)hi, dlo);            // exact
    const float range = (float)range64;
    float scale = 0.f;
    if (range64 != 0.0) {
        const float qmaxf = (float)qmax;
        const double inv = __ddiv_rn((double)qmaxf, range64);
        scale = (double)range == range64 ? __fdiv_rn(range, qmaxf)
                                         : (float)__ddiv_rn(range64, (double)qmaxf);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const double t0 = __dmul_rn(__dsub_rn((double)bf16lo(wv[k]), dlo), inv);
            const double t1 = __dmul_rn(__dsub_rn((double)bf16hi(wv[k]), dlo), inv);
            // 0 <= t <= qmax, so no clamp and no mask: the low word of t + 1.5 * 2^52 is rint(t)
            code[2 * k] = (unsigned)__double2loint(__dadd_rn(t0, PK_MAGIC64));
            code[2 * k + 1] = (unsigned)__double2loint(__dadd_rn(t1, PK_MAGIC64));
        }
    } else {
#pragma unroll
        for (int k = 0; k < 16; ++k) code[k] = 0u;
    }
    return scale;
}

// The whole chunk has one bitwidth B and fits the packed buffer: no per-word checks, all bit
// positions constant.  A lane's 16 codes are 16*B bits: whole words for even B; for odd B a
// pair of lanes makes whole words (the even lane completes its last word with the low
// half-word of its neighbour, the odd lane drops that half-word).
template <int B>
__device__ __forceinline__ void pack_rows(const PackLane& pl) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int rr = warp * 4 + (lane >> 3);
    auto row_ptr = [&](int r_in) {
        const int64_t r = pl.row0 + r_in;
        return reinterpret_cast<const uint4*>(pl.colp + (pl.rp ? (int64_t)pl.rp[r] : r) * pl.ldw);
    };
    uint4 n0 = make_uint4(0, 0, 0, 0), n1 = n0;
    if (rr < pl.br) { const uint4* p = row_ptr(rr); n0 = __ldg(p); n1 = __ldg(p + 1); }
    unsigned* dst = pl.dst + (size_t)rr * pl.row_words;
    float2* mp = pl.meta + (int64_t)rr * pl.meta_ld;
    const unsigned dst_step = PK_WARPS * 4 * pl.row_words;
    const int64_t meta_step = (int64_t)PK_WARPS * 4 * pl.meta_ld;
    for (; rr < pl.br; rr += PK_WARPS * 4, dst += dst_step, mp += meta_step) {   // br % 4 == 0
        const uint32_t wv[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
        if (rr + PK_WARPS * 4 < pl.br) { const uint4* p = row_ptr(rr + PK_WARPS * 4); n0 = __ldg(p); n1 = __ldg(p + 1); }
        float lo, hi;
        group_minmax<8>(wv, pl.team, lo, hi);
        unsigned code[16], w[4];
        const float scale = encode16(wv, lo, hi, (1 << B) - 1, code);
        if (pl.meta_lane) *mp = make_float2(scale, lo);
        pack16<B>(code, w);
        if constexpr (B & 1) {
            const unsigned nb_low = __shfl_down_sync(0xffffffffu, w[0], 1);
            if (!pl.odd_lane) {
                w[B >> 1] |= nb_low << 16;
#pragma unroll
                for (int i = 0; i <= (B >> 1); ++i)
                    if (SB_IN_BOUNDS(pl.ds, SBK_PACK, (dst - pl.packed) + i, pl.capacity)) dst[i] = w[i];
            } else {
#pragma unroll
                for (int i = 0; i < (B >> 1); ++i)
                    if (SB_IN_BOUNDS(pl.ds, SBK_PACK, (dst - pl.packed) + i, pl.capacity))
                        dst[i] = (w[i] >> 16) | (w[i + 1] << 16);
            }
        } else {
#pragma unroll
            for (int i = 0; i < (B >> 1); ++i)
                if (SB_IN_BOUNDS(pl.ds, SBK_PACK, (dst - pl.packed) + i, pl.capacity)) dst[i] = w[i];
        }
    }
}

// Chunks that hold blocks of different bitwidths (blocks narrower than 128 columns) or that
// reach past the packed buffer: bitwidth per lane at run time, every word checked.
__device__ __noinline__ void pack_rows_generic(PackLane pl, int b, long long lane_word,
                                               long long capacity, unsigned* packed, SbDeviceState* ds) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool odd_b = b & 1;
    for (int rr = warp * 4 + (lane >> 3); rr < pl.br; rr += PK_WARPS * 4) {
        const int64_t r = pl.row0 + rr;
        const uint4* p = reinterpret_cast<const uint4*>(pl.colp + (pl.rp ? (int64_t)pl.rp[r] : r) * pl.ldw);
        const uint4 n0 = __ldg(p), n1 = __ldg(p + 1);
        const uint32_t wv[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
        float lo, hi;
        group_minmax<8>(wv, pl.team, lo, hi);
        unsigned code[16], w[4];
        const float scale = encode16(wv, lo, hi, (1 << b) - 1, code);
        if (pl.meta_lane) pl.meta[(int64_t)rr * pl.meta_ld] = make_float2(scale, lo);
        switch (b) {
            case 1: pack16<1>(code, w); break;
            case 2: pack16<2>(code, w); break;
            case 3: pack16<3>(code, w); break;
            case 4: pack16<4>(code, w); break;
            case 5: pack16<5>(code, w); break;
            case 6: pack16<6>(code, w); break;
            case 7: pack16<7>(code, w); break;
            default: pack16<8>(code, w); break;
        }
        const unsigned nb_low = __shfl_down_sync(0xffffffffu, w[0], 1);
        int nwords = b >> 1;                                  // even b: b/2 whole words
        if (odd_b) {
            if (!pl.odd_lane) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (i == (b >> 1)) w[i] |= nb_low << 16;
                nwords = (b >> 1) + 1;
            } else {
#pragma unroll
                for (int i = 0; i < 3; ++i) w[i] = (w[i] >> 16) | (w[i + 1] << 16);
                w[3] >>= 16;
            }
        }
        const long long dst = lane_word + (long long)rr * pl.row_words;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (i < nwords) {
                if (dst + i < capacity) packed[dst + i] = w[i];
                else sb_latch(ds, SB_ERR_SCRATCH, SBK_PACK);
            }
        }
    }
}

// CTA = one block row x one 128-column chunk.  A lane owns 16 consecutive columns (two
// 16-byte loads), 8 lanes cover a row of the chunk, a warp covers 4 rows per step; the next
// step's loads are issued before the current rows are encoded.
//
// Codes follow the binary64 sequence
//   range = hi - lo; inv = qmax / range; q = rint((v - lo) * inv)
// literally: one fp64 division per lane and row, then a subtract, a multiply and the magic-number
// add per element (its low word is the rounded integer, ties to even).  B200 issues fp64 at half
// the fp32 rate, so this costs less than an fp32 path with a tie test and a divergent fp64 redo.
// The stored scale is fl32(range / qmax): with range exact in fp32 (checked) one correctly
// rounded fp32 division equals the rounded fp64 quotient (a 24-bit integer over 2^b - 1 has a
// binary expansion of period <= 8, never within 2^-53 of an fp32 rounding boundary).
__global__ void __launch_bounds__(PK_THREADS)
pack_kernel(const __nv_bfloat16* __restrict__ W, int64_t ldw, const int32_t* __restrict__ rp,
            int br, int bc, int group, PackBits pb, int n_bits,
            const unsigned char* __restrict__ level, const unsigned long long* __restrict__ off,
            unsigned* __restrict__ packed, long long capacity, float2* __restrict__ meta,
            int64_t n_block_cols, int64_t groups_per_row, SbDeviceState* ds) {
    __shared__ int s_bits[4];
    __shared__ long long s_base[4];
    const int lane = threadIdx.x & 31;
    const int cl = lane & 7;
    const int piece = bc < 128 ? bc : 128;               // columns of one block inside the chunk
    const int lpp = piece >> 4;                           // lanes per piece
    const int64_t bi = blockIdx.y;
    const int64_t col0 = (int64_t)blockIdx.x * 128;
    bool fits = true;
    if (threadIdx.x < 128 / piece) {
        const int64_t c0 = col0 + (int64_t)threadIdx.x * piece;
        const int64_t bj = c0 / bc;
        const int64_t blk = bi * n_block_cols + bj;
        int lv = level[blk];
        if (lv >= n_bits) { sb_latch(ds, SB_ERR_INVALID, SBK_PACK); lv = n_bits - 1; }
        const int b = pb.bits[lv];
        const long long base = (long long)off[blk] + ((c0 - bj * bc) * b) / 32;
        s_bits[threadIdx.x] = b;
        s_base[threadIdx.x] = base;
        // last word this piece writes
        fits = base + (long long)(br - 1) * ((long long)bc * b / 32) + (long long)piece * b / 32 <= capacity;
    }
    const bool all_fit = __syncthreads_and(fits);
    const int pc = cl / lpp, lp = cl - pc * lpp;
    const int b = s_bits[pc];
    bool uniform = true;
    for (int q = 1; q < 128 / piece; ++q) uniform = uniform && s_bits[q] == s_bits[0];

    PackLane pl;
    pl.colp = W + col0 + cl * 16;
    pl.rp = rp;
    pl.ldw = ldw;
    pl.row0 = bi * br;
    pl.br = br;
    pl.team = group >> 4;                                 // lanes per quantisation group (16 columns each)
    pl.meta_ld = groups_per_row;
    pl.meta = meta + pl.row0 * groups_per_row + (col0 + cl * 16) / group;
    pl.meta_lane = (cl % pl.team) == 0;
    pl.odd_lane = lp & 1;
    pl.row_words = (unsigned)((long long)bc * b / 32);
    // word offset of this lane's bits inside its row piece; odd b: the odd lane starts 16 bits in
    const long long lane_word = s_base[pc] + (lp * 16 * b) / 32 + (((b & 1) && pl.odd_lane) ? 1 : 0);
    pl.dst = packed + lane_word;
    pl.packed = packed; pl.capacity = capacity; pl.ds = ds;

    if (uniform && all_fit) {
        switch (b) {
            case 1: pack_rows<1>(pl); break;
            case 2: pack_rows<2>(pl); break;
            case 3: pack_rows<3>(pl); break;
            case 4: pack_rows<4>(pl); break;
            case 5: pack_rows<5>(pl); break;
            case 6: pack_rows<6>(pl); break;
            case 7: pack_rows<7>(pl); break;
            default: pack_rows<8>(pl); break;
        }
    } else {
        pack_rows_generic(pl, b, lane_word, capacity, packed, ds);
    }
}

}  // namespace

extern "C" sb_status sb_pack_blocks(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                                    const int32_t* row_perm, const int32_t* col_perm, int br, int bc,
                                    int group, const int* bits, int n_bits, const uint8_t* level,
                                    uint32_t* packed, int64_t capacity_words, int64_t* block_off_words,
                                    float* meta) {
    if (!ctx) return SB_ERR_INVALID;
    if (!W || !level || !packed || !block_off_words || !meta || R <= 0 || C <= 0 || capacity_words < 0)
        return sb_fail(ctx, SB_ERR_INVALID, "pack: null or empty");
    if (!sb_check_bits(bits, n_bits)) return sb_fail(ctx, SB_ERR_INVALID, "pack: bits must be ascending in 1..8");
    const bool g_ok = group == 16 || group == 32 || group == 64 || group == 128;
    if (br <= 0 || bc <= 0 || br % 4 || R % br || C % bc || !g_ok || bc % group || bc % 32 || C % 128 ||
        !(bc == 32 || bc == 64 || bc % 128 == 0) || ldw % 8 || ldw < C ||
        (reinterpret_cast<uintptr_t>(W) & 15) || (reinterpret_cast<uintptr_t>(meta) & 7))
        return sb_fail(ctx, SB_ERR_SHAPE, "pack: block %dx%d group %d does not tile %lldx%lld", br, bc,
                       group, (long long)R, (long long)C);
    for (int l = 0; l < n_bits; ++l)
        if (((long long)br * bc * bits[l]) % 32) return sb_fail(ctx, SB_ERR_SHAPE, "pack: block bits not a multiple of 32");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const int64_t nb = (R / br) * (C / bc);
    const size_t gather_bytes = col_perm ? (size_t)R * C * 2 : 0;
    const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(W);
    int64_t ld = ldw;
    const int32_t* load_rp = row_perm;
    if (col_perm) {
        void* arena;
        sb_status st = sb_scratch(ctx, Carver::need({gather_bytes}), &arena);
        if (st != SB_OK) return st;
        Carver cv(arena);
        void* g = cv.take<unsigned char>(gather_bytes);
        st = sb_gather_bf16(ctx, W, R, C, ldw, row_perm, col_perm, g);
        if (st != SB_OK) return st;
        src = static_cast<const __nv_bfloat16*>(g);
        ld = C;
        load_rp = nullptr;
    }
    PackBits pb{};
    for (int l = 0; l < 8; ++l) pb.bits[l] = l < n_bits ? bits[l] : bits[n_bits - 1];
    if (nb <= PO1_THREADS * PO1_ITEMS) {
        pack_offsets_small_kernel<<<1, PO1_THREADS, 0, ctx->stream>>>(
            level, (int)nb, n_bits, pb, (unsigned long long)br * bc / 32,
            reinterpret_cast<unsigned long long*>(block_off_words), ctx->dstate);
        SB_LAUNCHED(ctx);
    } else {
        const unsigned tiles = (unsigned)((nb + PO_TILE - 1) / PO_TILE);
        sb_status st;
        LookbackBuf lb = sb_lookback(ctx, tiles, &st);
        if (st != SB_OK) return st;
        pack_offsets_kernel<<<tiles, PO_THREADS, 0, ctx->stream>>>(
            level, nb, n_bits, pb, (unsigned long long)br * bc / 32,
            reinterpret_cast<unsigned long long*>(block_off_words), lb, ctx->dstate);
        SB_LAUNCHED(ctx);
    }
    dim3 grid((unsigned)(C / 128), (unsigned)(R / br));
    pack_kernel<<<grid, PK_THREADS, 0, ctx->stream>>>(
        src, ld, load_rp, br, bc, group, pb, n_bits, level,
        reinterpret_cast<const unsigned long long*>(block_off_words), packed, capacity_words,
        reinterpret_cast<float2*>(meta), C / bc, C / group, ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}
