// Pack: integer codes of every block at its assigned bitwidth, bit-packed, plus per-group
// (scale, min).  The code arithmetic is IEEE binary64 in a fixed operation order so that the
// integers are reproducible bit for bit:
//   range = hi - lo; inv = qmax / range; q = rint((v - lo) * inv); scale = range / qmax.
#include "lookback.cuh"

sb_status sb_gather_bf16(sb_ctx* ctx, const void* W, int64_t R, int64_t C, int64_t ldw,
                         const int32_t* rp, const int32_t* cp, void* out);

namespace {

constexpr int PK_THREADS = 256;
constexpr int PK_WARPS = PK_THREADS / 32;

__global__ void block_words_kernel(const unsigned char* __restrict__ level, int64_t nb, int n_bits,
                                   long long words_per_bit, const int* __restrict__ bits_dev,
                                   unsigned long long* __restrict__ words, SbDeviceState* ds) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nb) return;
    int l = level[i];
    if (l >= n_bits) { sb_latch(ds, SB_ERR_INVALID, SBK_PACK); l = n_bits - 1; }
    words[i] = (unsigned long long)(words_per_bit * bits_dev[l]);
}

struct PackBits { int bits[8]; };

constexpr float PK_MAGIC = 12582912.f;          // 1.5 * 2^23
constexpr float PK_TIE_BAND = 0.5f - 1.0f / 4096.0f;

// CTA = one block row x one 128-column chunk; a warp takes one row of the chunk at a time, a
// lane 4 consecutive columns.  Codes are DEFINED by the binary64 sequence
//   range = hi - lo; inv = qmax / range; q = rint((v - lo) * inv)
// but computed in fp32 wherever that provably gives the same integer: the fp32 value of t is
// within 2^-13 of the fp64 one (t <= 255), so an element farther than 2^-12 from a rounding
// tie keeps its fp32 code, and only rows that contain an element inside that band (exact
// ties are common with bf16 data) redo those elements in fp64.  The stored scale is
// fl32(range / qmax): with range exact in fp32 (checked) one correctly rounded fp32 division
// equals the rounded fp64 quotient (a 24-bit integer over 2^b - 1 has a binary expansion of
// period <= 8, never within 2^-53 of an fp32 rounding boundary).
__global__ void __launch_bounds__(PK_THREADS)
pack_kernel(const __nv_bfloat16* __restrict__ W, int64_t ldw, const int32_t* __restrict__ rp,
            int br, int bc, int group, PackBits pb, int n_bits,
            const unsigned char* __restrict__ level, const unsigned long long* __restrict__ off,
            unsigned* __restrict__ packed, long long capacity, float2* __restrict__ meta,
            int64_t n_block_cols, int64_t groups_per_row, SbDeviceState* ds) {
    __shared__ unsigned stage[PK_WARPS][32];
    __shared__ int s_bits[4];
    __shared__ long long s_base[4];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int piece = bc < 128 ? bc : 128;               // columns of one block inside the chunk
    const int lpp = piece >> 2;                           // lanes (and stage words) per piece
    const int64_t bi = blockIdx.y;
    const int64_t col0 = (int64_t)blockIdx.x * 128;
    if (threadIdx.x < 128 / piece) {
        const int64_t c0 = col0 + (int64_t)threadIdx.x * piece;
        const int64_t bj = c0 / bc;
        const int64_t blk = bi * n_block_cols + bj;
        int lv = level[blk];
        if (lv >= n_bits) { sb_latch(ds, SB_ERR_INVALID, SBK_PACK); lv = n_bits - 1; }
        const int b = pb.bits[lv];
        s_bits[threadIdx.x] = b;
        s_base[threadIdx.x] = (long long)off[blk] + ((c0 - bj * bc) * b) / 32;
    }
    __syncthreads();
    const int pc = lane / lpp, lp = lane - pc * lpp;
    const int b = s_bits[pc];
    const long long base = s_base[pc];
    const long long row_words = (long long)bc * b / 32;
    const float qmaxf = (float)((1 << b) - 1);
    const int team = group >> 2;                          // lanes per quantisation group
    const int64_t gcol = (col0 + lane * 4) / group;
    const bool meta_lane = (lane % team) == 0;
    const int words = piece * b / 32;                     // words per row of one piece
    const int bit0 = lp * 4 * b;
    unsigned* st = &stage[warp][pc * lpp];

    int rr = warp;
    uint2 raw = make_uint2(0u, 0u);
    if (rr < br) {
        const int64_t r = bi * br + rr;
        raw = ld_stream8(W + (rp ? (int64_t)rp[r] : r) * ldw + col0 + lane * 4);
    }
    for (; rr < br; rr += PK_WARPS) {
        const int64_t r = bi * br + rr;
        const uint2 cur = raw;
        if (rr + PK_WARPS < br) {                         // prefetch the next row of this warp
            const int64_t rn = r + PK_WARPS;
            raw = ld_stream8(W + (rp ? (int64_t)rp[rn] : rn) * ldw + col0 + lane * 4);
        }
        const float v[4] = {bf16lo(cur.x), bf16hi(cur.x), bf16lo(cur.y), bf16hi(cur.y)};
        float lo = fminf(fminf(v[0], v[1]), fminf(v[2], v[3]));
        float hi = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
        for (int o = team >> 1; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        }
        const double range64 = __dsub_rn((double)hi, (double)lo);     // exact
        const float range = (float)range64;
        const bool exact = (double)range == range64;
        unsigned code[4] = {0u, 0u, 0u, 0u};
        float scale = 0.f;
        bool redo = false;
        unsigned near = 0u;
        if (range64 != 0.0) {
            // fp32 fast path (a denormal range overflows the reciprocal: let fp64 handle it)
            const bool fast = range >= 1e-30f;
            const float inv = fast ? qmaxf / range : 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float t = (v[k] - lo) * inv;
                const float q = (t + PK_MAGIC) - PK_MAGIC;
                code[k] = (unsigned)fminf(fmaxf(q, 0.f), qmaxf);
                if (!fast || fabsf(t - q) >= PK_TIE_BAND) near |= 1u << k;
            }
            scale = __fdiv_rn(range, qmaxf);
            redo = near != 0u || !exact;
        }
        if (__any_sync(0xffffffffu, redo)) {
            if (redo) {
                const double qmax = (double)qmaxf, dlo = (double)lo;
                const double inv = __ddiv_rn(qmax, range64);
                if (!exact) scale = (float)__ddiv_rn(range64, qmax);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (near & (1u << k)) {
                        const double t = __dmul_rn(__dsub_rn((double)v[k], dlo), inv);
                        double q = rint(t);                          // round half to even
                        q = fmin(fmax(q, 0.0), qmax);
                        code[k] = (unsigned)q;
                    }
                }
            }
        }
        if (meta_lane) meta[r * groups_per_row + gcol] = make_float2(scale, lo);
        // a lane's 4 codes go to bit lp*4*b of its piece of the warp's stage
        stage[warp][lane] = 0;
        __syncwarp();
        const unsigned long long chunk = (unsigned long long)code[0] | ((unsigned long long)code[1] << b) |
                                         ((unsigned long long)code[2] << (2 * b)) |
                                         ((unsigned long long)code[3] << (3 * b));
        const unsigned long long sh = chunk << (bit0 & 31);
        atomicOr(&st[bit0 >> 5], (unsigned)sh);
        if ((unsigned)(sh >> 32)) atomicOr(&st[(bit0 >> 5) + 1], (unsigned)(sh >> 32));
        __syncwarp();
        if (lp < words) {
            const long long dst = base + (long long)rr * row_words + lp;
            if (dst < capacity) packed[dst] = st[lp];
            else sb_latch(ds, SB_ERR_SCRATCH, SBK_PACK);
        }
        __syncwarp();
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
    const bool g_ok = group == 4 || group == 8 || group == 16 || group == 32 || group == 64 || group == 128;
    if (br <= 0 || bc <= 0 || R % br || C % bc || !g_ok || bc % group || bc % 32 || C % 128 ||
        !(bc == 32 || bc == 64 || bc % 128 == 0) || ldw % 8 || ldw < C ||
        (reinterpret_cast<uintptr_t>(W) & 15) || (reinterpret_cast<uintptr_t>(meta) & 7))
        return sb_fail(ctx, SB_ERR_SHAPE, "pack: block %dx%d group %d does not tile %lldx%lld", br, bc,
                       group, (long long)R, (long long)C);
    for (int l = 0; l < n_bits; ++l)
        if (((long long)br * bc * bits[l]) % 32) return sb_fail(ctx, SB_ERR_SHAPE, "pack: block bits not a multiple of 32");
    SB_CUDA(ctx, cudaSetDevice(ctx->device));
    const int64_t nb = (R / br) * (C / bc);
    const size_t gather_bytes = col_perm ? (size_t)R * C * 2 : 0;
    void* arena;
    sb_status st = sb_scratch(ctx, Carver::need({(size_t)nb * 8, 64, gather_bytes}), &arena);
    if (st != SB_OK) return st;
    Carver cv(arena);
    unsigned long long* words = cv.take<unsigned long long>((size_t)nb);
    int* bits_dev = cv.take<int>(8);
    const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(W);
    int64_t ld = ldw;
    const int32_t* load_rp = row_perm;
    if (col_perm) {
        void* g = cv.take<unsigned char>(gather_bytes);
        st = sb_gather_bf16(ctx, W, R, C, ldw, row_perm, col_perm, g);
        if (st != SB_OK) return st;
        src = static_cast<const __nv_bfloat16*>(g);
        ld = C;
        load_rp = nullptr;
    }
    PackBits pb{};
    for (int l = 0; l < 8; ++l) pb.bits[l] = l < n_bits ? bits[l] : bits[n_bits - 1];
    int* hb = reinterpret_cast<int*>(static_cast<char*>(ctx->pinned) + 3072);
    for (int l = 0; l < 8; ++l) hb[l] = pb.bits[l];
    SB_CUDA(ctx, cudaMemcpyAsync(bits_dev, hb, 8 * sizeof(int), cudaMemcpyHostToDevice, ctx->stream));
    block_words_kernel<<<(unsigned)((nb + 255) / 256), 256, 0, ctx->stream>>>(
        level, nb, n_bits, (long long)br * bc / 32, bits_dev, words, ctx->dstate);
    SB_LAUNCHED(ctx);
    st = sb_scan_exclusive_u64(ctx, words, reinterpret_cast<unsigned long long*>(block_off_words), nb);
    if (st != SB_OK) return st;
    dim3 grid((unsigned)(C / 128), (unsigned)(R / br));
    pack_kernel<<<grid, PK_THREADS, 0, ctx->stream>>>(
        src, ld, load_rp, br, bc, group, pb, n_bits, level,
        reinterpret_cast<const unsigned long long*>(block_off_words), packed, capacity_words,
        reinterpret_cast<float2*>(meta), C / bc, C / group, ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}
