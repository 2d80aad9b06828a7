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

// One warp handles one row of a 128-column chunk: a lane owns 4 consecutive columns.
// grid.x = C / 128 chunks, grid.y = row groups of PK_WARPS rows.
__global__ void __launch_bounds__(PK_THREADS)
pack_kernel(const __nv_bfloat16* __restrict__ W, int64_t R, int64_t C, int64_t ldw,
            const int32_t* __restrict__ rp, int br, int bc, int group, PackBits pb, int n_bits,
            const unsigned char* __restrict__ level, const unsigned long long* __restrict__ off,
            unsigned* __restrict__ packed, long long capacity, float2* __restrict__ meta,
            int64_t n_block_cols, SbDeviceState* ds) {
    __shared__ unsigned stage[PK_WARPS][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t r = (int64_t)blockIdx.y * PK_WARPS + warp;
    if (r >= R) return;
    const int64_t col = (int64_t)blockIdx.x * 128 + lane * 4;
    const int64_t rs = rp ? rp[r] : r;
    const uint2 raw = ld_stream8(W + rs * ldw + col);
    float v[4] = {bf16lo(raw.x), bf16hi(raw.x), bf16lo(raw.y), bf16hi(raw.y)};
    float lo = fminf(fminf(v[0], v[1]), fminf(v[2], v[3]));
    float hi = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
    const int team = group / 4;                       // lanes per group (4..32)
    for (int o = team >> 1; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    const int64_t bi = r / br, bj = col / bc;
    const int64_t blk = bi * n_block_cols + bj;
    const int b = pb.bits[min((int)level[blk], n_bits - 1)];
    const double qmax = (double)((1 << b) - 1);
    const double dlo = (double)lo;
    const double range = __dsub_rn((double)hi, dlo);
    double scale = 0.0;
    unsigned code[4] = {0u, 0u, 0u, 0u};
    if (range != 0.0) {
        const double inv = __ddiv_rn(qmax, range);
        scale = __ddiv_rn(range, qmax);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const double t = __dmul_rn(__dsub_rn((double)v[k], dlo), inv);
            double q = rint(t);                         // round half to even
            q = fmin(fmax(q, 0.0), qmax);
            code[k] = (unsigned)q;
        }
    }
    if ((lane % team) == 0) {
        const int64_t gi = r * (C / group) + col / group;
        meta[gi] = make_float2((float)scale, (float)dlo);
    }
    // The 128-column chunk is cut into pieces of min(bc, 128) columns, one per block it
    // touches; each piece has its block's bitwidth and owns piece/4 words of the stage
    // (enough for 8 bits).  A lane's 4 codes go to bit lp*4*b of its piece.
    const int piece = bc < 128 ? bc : 128;
    const int lpp = piece / 4;                          // lanes (and stage words) per piece
    const int pc = lane / lpp, lp = lane % lpp;
    stage[warp][lane] = 0;
    __syncwarp();
    const unsigned long long chunk = (unsigned long long)code[0] | ((unsigned long long)code[1] << b) |
                                     ((unsigned long long)code[2] << (2 * b)) |
                                     ((unsigned long long)code[3] << (3 * b));
    const int bit0 = lp * 4 * b;
    const unsigned long long sh = chunk << (bit0 & 31);
    atomicOr(&stage[warp][pc * lpp + (bit0 >> 5)], (unsigned)sh);
    if ((unsigned)(sh >> 32)) atomicOr(&stage[warp][pc * lpp + (bit0 >> 5) + 1], (unsigned)(sh >> 32));
    __syncwarp();
    if (lp < piece * b / 32) {                          // lane lp writes word lp of its piece
        const int64_t c0 = (int64_t)blockIdx.x * 128 + (int64_t)pc * piece;   // first column of the piece
        const long long e0 = (long long)(r - bi * br) * bc + (c0 - bj * bc);  // element index in the block
        const long long dst = (long long)off[blk] + (e0 * b) / 32 + lp;
        if (dst < capacity) packed[dst] = stage[warp][pc * lpp + lp];
        else sb_latch(ds, SB_ERR_SCRATCH, SBK_PACK);
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
    dim3 grid((unsigned)(C / 128), (unsigned)((R + PK_WARPS - 1) / PK_WARPS));
    pack_kernel<<<grid, PK_THREADS, 0, ctx->stream>>>(
        src, R, C, ld, load_rp, br, bc, group, pb, n_bits, level,
        reinterpret_cast<const unsigned long long*>(block_off_words), packed, capacity_words,
        reinterpret_cast<float2*>(meta), C / bc, ctx->dstate);
    SB_LAUNCHED(ctx);
    return SB_OK;
}
