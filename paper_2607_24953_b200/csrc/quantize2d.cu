// fp4q_quantize2d: 2D-block (32x32) FP4 quantization with dual-layout pack, sm_100a.
//
// One pass over HBM: 2 B/element read, 0.5 + 0.5 B/element written, 1 B per 1024 elements of scale.
// A CTA of 4 warps owns a 128x128 element block; a warp owns 32 rows x 128 columns (four 32x32
// blocks side by side); 8 lanes own one 32x32 block, each lane 8 rows x 16 consecutive columns
// (one 256-bit load per row, all eight issued before anything else).  While the loads are in flight
// the lane draws its Philox bytes (they do not depend on the data) and parks them in shared memory.
// The block maximum is reduced with warp shuffles over the 8 lanes, the E2M1 codes come from the
// hardware converts, the row-major payload goes straight to global memory (8 B per lane and row,
// 64 B contiguous per row and warp) and the transposed payload is built with an in-register 8x8
// nibble transpose, staged through 8 KB of shared memory and written as 64 B contiguous segments.
// CTAs whose tile lies fully inside an aligned tensor run a check-free body; ragged edges, unaligned
// inputs, cols % 16 != 0 and the transposed index take a general body with the same arithmetic.
//
// Rounding: x 2^-e (exact in FP32) goes through the hardware converts cvt.rn.satfinite.e2m1x2.f32
// (nearest even) or cvt.rs.satfinite.e2m1x4.f32 (stochastic).  The stochastic convert adds 16 random bits
// below the kept mantissa bit and truncates; the elements that land in nibbles 0 and 2 take the upper 8
// of their 16 bits from rbits[23:16] and rbits[31:24] and the lower 8 from rbits[7:0] and rbits[15:8]
// (the other two inputs reuse the same bits in reversed order).  With the lower bytes zero and only
// those two inputs used, the instruction computes exactly "up iff floor(256 p) + r8 >= 256" for two
// elements at a time: the element's random byte is routed into place with one PRMT.  Blocks that
// contain non-finite values take a scalar path that rounds on the fp16 bit pattern of |x| 2^(-e-14)
// (magnitude code in bits 11..9, position between neighbours in bits 8..0).
#include <cuda_bf16.h>

#include "common.cuh"
#include "quant_device.cuh"

namespace fp4q {

struct Quant2dParams {
    const uint16_t *x;
    int64_t rows, cols, ld_x;
    uint8_t *q_rm;
    int64_t ld_rm;
    uint8_t *q_t;
    int64_t ld_t;
    uint8_t *scale;
    int64_t ld_s;
    int64_t grid_x;           // CTAs along the column direction
    uint32_t tensor_id;
    uint32_t flags;
    int x_vec_ok;             // 2: x 32-byte aligned, ld_x % 16 == 0 (256-bit loads); 1: 16-byte aligned, ld_x % 8 == 0
    int rng_aligned;          // cols % 16 == 0 and index not transposed: one Philox block per 16-element segment
    PhiloxRoundKeys keys;
};

__device__ __noinline__ uint32_t philox_byte(const Quant2dParams &p, uint64_t idx)
{
    uint32_t o[4];
    const uint64_t blk = idx >> 4;
    philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), p.tensor_id, 0u, p.keys, o);
    const uint32_t w = (idx >> 2) & 3;
    const uint32_t word = w == 0 ? o[0] : w == 1 ? o[1] : w == 2 ? o[2] : o[3];
    return (word >> (8 * (idx & 3))) & 0xFFu;
}

// In-register transpose of an 8x8 matrix of nibbles: a[r] holds row r (nibble c = column c);
// on return a[c] holds column c (nibble r = row r).
__device__ __forceinline__ void transpose8x8_nibbles(uint32_t a[8])
{
#pragma unroll
    for (int r = 0; r < 4; r++) {   // swap 4x4 quadrants (16-bit halves between rows r and r+4)
        const uint32_t lo = __byte_perm(a[r], a[r + 4], 0x5410), hi = __byte_perm(a[r], a[r + 4], 0x7632);
        a[r] = lo; a[r + 4] = hi;
    }
#pragma unroll
    for (int q = 0; q < 4; q++) {   // swap 2x2 blocks (bytes between rows r and r+2)
        const int r = (q & 1) + 4 * (q >> 1);
        const uint32_t lo = __byte_perm(a[r], a[r + 2], 0x6240), hi = __byte_perm(a[r], a[r + 2], 0x7351);
        a[r] = lo; a[r + 2] = hi;
    }
#pragma unroll
    for (int r = 0; r < 8; r += 2) {  // swap single nibbles between rows r and r+1
        const uint32_t lo = (a[r] & 0x0F0F0F0Fu) | ((a[r + 1] & 0x0F0F0F0Fu) << 4);
        const uint32_t hi = ((a[r] >> 4) & 0x0F0F0F0Fu) | (a[r + 1] & 0xF0F0F0F0u);
        a[r] = lo; a[r + 1] = hi;
    }
}

__device__ __forceinline__ void load_segment(const Quant2dParams &p, int64_t i, int64_t j0, uint32_t out[8])
{
    if (i >= p.rows || j0 >= p.cols) {
#pragma unroll
        for (int k = 0; k < 8; k++) out[k] = 0u;
        return;
    }
    const uint16_t *src = p.x + i * p.ld_x + j0;
    if (p.x_vec_ok == 2 && j0 + 16 <= p.cols) {
        asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(out[0]), "=r"(out[1]), "=r"(out[2]), "=r"(out[3]), "=r"(out[4]), "=r"(out[5]), "=r"(out[6]),
                       "=r"(out[7])
                     : "l"(src));
    } else if (p.x_vec_ok && j0 + 16 <= p.cols) {
        const uint4 a = __ldg(reinterpret_cast<const uint4 *>(src));
        const uint4 b = __ldg(reinterpret_cast<const uint4 *>(src) + 1);
        out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
        out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
    } else {
#pragma unroll
        for (int k = 0; k < 8; k++) {
            const uint32_t lo = (j0 + 2 * k < p.cols) ? (uint32_t)__ldg(src + 2 * k) : 0u;
            const uint32_t hi = (j0 + 2 * k + 1 < p.cols) ? (uint32_t)__ldg(src + 2 * k + 1) : 0u;
            out[k] = lo | (hi << 16);
        }
    }
}

// The 16 random bytes of the row segment starting at element (i, j0), one Philox call per element: the slow
// generic path for cols % 16 != 0 or the transposed index.
__device__ __forceinline__ void segment_random_bytes(const Quant2dParams &p, int64_t i, int64_t j0, uint32_t R[4])
{
#pragma unroll
    for (int w = 0; w < 4; w++) {
        uint32_t word = 0;
#pragma unroll 1
        for (int b = 0; b < 4; b++) {
            const int64_t j = j0 + 4 * w + b;
            if (j < p.cols) {
                const uint64_t idx = (p.flags & FP4Q_INDEX_TRANSPOSED)
                                         ? (uint64_t)j * (uint64_t)p.rows + (uint64_t)i
                                         : (uint64_t)i * (uint64_t)p.cols + (uint64_t)j;
                word |= philox_byte(p, idx) << (8 * b);
            }
        }
        R[w] = word;
    }
}

#ifndef FP4Q_QUANT_MIN_BLOCKS
#define FP4Q_QUANT_MIN_BLOCKS 4
#endif

// FAST = the CTA's 128x128 tile lies fully inside the tensor, rows are 32-byte aligned (256-bit loads) and
// one Philox block covers each 16-element segment: no per-row bounds or path checks remain in the hot loop.
// BLK = block size: 32 (the method), or 16 / 64 for the block-size study.  A 16x16 block is two lanes (8 rows x 16
// columns each), a 64x64 block sixteen lanes in each of two neighbouring warps, which exchange their maxima through
// `xchg`.  With BLK = 64 the scale is still written once per 32x32 tile (four equal entries per block), so that the
// tensor feeds the GEMMs as it stands; with BLK = 16 the scale matrix has one entry per 16x16 block.
template <int MODE, bool FAST, int BLK>
__device__ __forceinline__ void quantize_tile(const Quant2dParams &p, uint4 *qt_stage, uint4 *rnd_stage, uint32_t *xchg)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = lane >> 3;          // which of the warp's four 32x32 blocks
    const int rg = (lane >> 1) & 3;   // group of 8 rows inside the block
    const int ch = lane & 1;          // 16-column half of the block
    const int64_t bx = (int64_t)blockIdx.x % p.grid_x, by = (int64_t)blockIdx.x / p.grid_x;
    const int64_t tile_row0 = by * 128 + warp * 32, tile_col0 = bx * 128 + t * 32;
    const int64_t row0 = tile_row0 + rg * 8, col0 = tile_col0 + ch * 16;
    const bool tile_exists = FAST || (tile_row0 < p.rows && tile_col0 < p.cols);

    uint32_t raw[8][8];
    if (FAST) {
        const uint16_t *src = p.x + row0 * p.ld_x + col0;
#pragma unroll
        for (int r = 0; r < 8; r++)
            asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(raw[r][0]), "=r"(raw[r][1]), "=r"(raw[r][2]), "=r"(raw[r][3]), "=r"(raw[r][4]),
                           "=r"(raw[r][5]), "=r"(raw[r][6]), "=r"(raw[r][7])
                         : "l"(src + r * p.ld_x));
    } else {
#pragma unroll
        for (int r = 0; r < 8; r++) load_segment(p, row0 + r, col0, raw[r]);
    }

    // The random bytes do not depend on the data: draw them while the loads are in flight and park them in
    // shared memory (each thread reads back only what it wrote), in a rolled loop that keeps the code small.
    if (MODE == FP4Q_ROUND_STOCHASTIC && (FAST || p.rng_aligned)) {
        uint64_t idx = (uint64_t)row0 * (uint64_t)p.cols + (uint64_t)col0;
#pragma unroll 2
        for (int r = 0; r < 8; r++) {
            uint32_t R[4];
            const uint64_t blk = idx >> 4;
            philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), p.tensor_id, 0u, p.keys, R);
            rnd_stage[r * 128 + threadIdx.x] = make_uint4(R[0], R[1], R[2], R[3]);
            idx += (uint64_t)p.cols;
        }
    }

    // block maximum: packed BF16 |.| max with NaN propagation, so that any non-finite entry shows
    // up in the result and routes the block to the scalar path
    __nv_bfloat162 m2 = __float2bfloat162_rn(0.0f);
#pragma unroll
    for (int r = 0; r < 8; r++)
#pragma unroll
        for (int k = 0; k < 8; k++)
            m2 = __hmax2_nan(m2, __habs2(*reinterpret_cast<const __nv_bfloat162 *>(&raw[r][k])));
    constexpr int kShflLo = BLK == 16 ? 2 : 1, kShflHi = BLK == 16 ? 2 : BLK == 32 ? 4 : 8;   // lanes of one block
#pragma unroll
    for (int s = kShflLo; s <= kShflHi; s <<= 1) {
        uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, *reinterpret_cast<uint32_t *>(&m2), s);
        m2 = __hmax2_nan(m2, *reinterpret_cast<__nv_bfloat162 *>(&other));
    }
    const __nv_bfloat16 m1 = __hmax_nan(m2.x, m2.y);
    uint32_t mbits = (uint32_t)(*reinterpret_cast<const uint16_t *>(&m1)) & 0x7FFFu;
    bool nonfinite64 = false;
    if (BLK == 64) {
        // the other 32 rows of the block belong to the neighbouring warp: both maxima (with NaN propagation, and over
        // finite entries only) cross through shared memory, unconditionally, so that every thread reaches the barrier
        uint32_t fm = 0;
#pragma unroll
        for (int r = 0; r < 8; r++)
#pragma unroll
            for (int k = 0; k < 8; k++) {
                const uint32_t lo = raw[r][k] & 0x7FFFu, hi = (raw[r][k] >> 16) & 0x7FFFu;
                if (lo < 0x7F80u && lo > fm) fm = lo;
                if (hi < 0x7F80u && hi > fm) fm = hi;
            }
#pragma unroll
        for (int s = 1; s <= 8; s <<= 1) {
            const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, fm, s);
            fm = other > fm ? other : fm;
        }
        if ((lane & 15) == 0) {
            xchg[(warp * 2 + (t >> 1)) * 2] = mbits;
            xchg[(warp * 2 + (t >> 1)) * 2 + 1] = fm;
        }
        __syncthreads();
        const uint32_t om = xchg[((warp ^ 1) * 2 + (t >> 1)) * 2], of = xchg[((warp ^ 1) * 2 + (t >> 1)) * 2 + 1];
        fm = of > fm ? of : fm;
        nonfinite64 = mbits >= 0x7F80u || om >= 0x7F80u;
        mbits = nonfinite64 ? fm : (om > mbits ? om : mbits);
    }

    const bool nonfinite = BLK == 64 ? nonfinite64 : mbits >= 0x7F80u;
    if (BLK != 64 && __any_sync(0xFFFFFFFFu, nonfinite)) {
        // maximum over the finite entries only
        uint32_t fm = 0;
#pragma unroll
        for (int r = 0; r < 8; r++)
#pragma unroll
            for (int k = 0; k < 8; k++) {
                const uint32_t lo = raw[r][k] & 0x7FFFu, hi = (raw[r][k] >> 16) & 0x7FFFu;
                if (lo < 0x7F80u && lo > fm) fm = lo;
                if (hi < 0x7F80u && hi > fm) fm = hi;
            }
#pragma unroll
        for (int s = kShflLo; s <= kShflHi; s <<= 1) {
            const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, fm, s);
            fm = other > fm ? other : fm;
        }
        if (nonfinite) mbits = fm;
    }

    const int code = scale_code_from_max(mbits);
    const float inv = inv_scale(code);
    if (BLK == 16) {
        if ((lane & 2) == 0 && row0 < p.rows && col0 < p.cols) p.scale[(row0 >> 4) * p.ld_s + (col0 >> 4)] = (uint8_t)code;
    } else if (tile_exists && (lane & 7) == 0) {
        p.scale[(tile_row0 >> 5) * p.ld_s + (tile_col0 >> 5)] = (uint8_t)code;
    }

    uint32_t W[8][2];
    uint8_t *dst_rm = p.q_rm + row0 * p.ld_rm + (col0 >> 1);
    if (FAST && !nonfinite) {
        // hot loop: no bounds checks, no path selection
#pragma unroll
        for (int r = 0; r < 8; r++) {
            uint32_t R[4] = {0u, 0u, 0u, 0u};
            if (MODE == FP4Q_ROUND_STOCHASTIC) {
                const uint4 v = rnd_stage[r * 128 + threadIdx.x];
                R[0] = v.x; R[1] = v.y; R[2] = v.z; R[3] = v.w;
            }
            round_segment<MODE>(raw[r], inv, R, W[r]);
            *reinterpret_cast<uint2 *>(dst_rm + r * p.ld_rm) = make_uint2(W[r][0], W[r][1]);
        }
    } else {
#pragma unroll
        for (int r = 0; r < 8; r++) {
            const int64_t i = row0 + r;
            if (!tile_exists || i >= p.rows) {
                W[r][0] = W[r][1] = 0u;
                continue;
            }
            uint32_t R[4] = {0u, 0u, 0u, 0u};
            if (MODE == FP4Q_ROUND_STOCHASTIC) {
                if (FAST || p.rng_aligned) {
                    const uint4 v = rnd_stage[r * 128 + threadIdx.x];
                    R[0] = v.x; R[1] = v.y; R[2] = v.z; R[3] = v.w;
                } else {
                    segment_random_bytes(p, i, col0, R);
                }
            }
            if (!nonfinite) {
                round_segment<MODE>(raw[r], inv, R, W[r]);
            } else {
                const uint2 w = round_segment_scalar<MODE>(make_uint4(raw[r][0], raw[r][1], raw[r][2], raw[r][3]),
                                                           make_uint4(raw[r][4], raw[r][5], raw[r][6], raw[r][7]),
                                                           make_uint4(R[0], R[1], R[2], R[3]), inv_scale_f16_aligned(code));
                W[r][0] = w.x;
                W[r][1] = w.y;
            }
            *reinterpret_cast<uint2 *>(dst_rm + r * p.ld_rm) = make_uint2(W[r][0], W[r][1]);
        }
    }

    if (p.q_t == nullptr) return;

    // transposed payload: per lane two 8x8 nibble blocks -> 16 words (one per column, 8 rows each)
    uint32_t *stage = reinterpret_cast<uint32_t *>(qt_stage);
#pragma unroll
    for (int g = 0; g < 2; g++) {
        uint32_t a[8];
#pragma unroll
        for (int r = 0; r < 8; r++) a[r] = W[r][g];
        transpose8x8_nibbles(a);
#pragma unroll
        for (int c = 0; c < 8; c++) {
            const int col_local = 32 * t + 16 * ch + 8 * g + c;
            // word index inside the 64-byte row: 4*(source warp) + rg, with the 16-byte chunk index
            // XORed by the column's block index so that a warp's stores spread over the banks
            stage[col_local * 16 + (((warp ^ t) << 2) | rg)] = a[c];
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; k++) {
        const int row_local = (threadIdx.x >> 2) + 32 * k;   // transposed row = source column; its block index is k
        const int chunk = threadIdx.x & 3;                    // 32 source rows = one source warp
        const int64_t col = bx * 128 + row_local;
        if (FAST || (col < p.cols && by * 128 + chunk * 32 < p.rows)) {
            const uint4 v = qt_stage[row_local * 4 + (chunk ^ k)];
            *reinterpret_cast<uint4 *>(p.q_t + col * p.ld_t + by * 64 + chunk * 16) = v;
        }
    }
}

template <int MODE, int BLK = 32>
__global__ void __launch_bounds__(128, FP4Q_QUANT_MIN_BLOCKS) quantize2d_kernel(const __grid_constant__ Quant2dParams p)
{
    __shared__ uint4 qt_stage[128 * 4];   // 128 transposed rows x 64 B (four 16-byte chunks, XOR-swizzled)
    __shared__ uint4 rnd_stage[MODE == FP4Q_ROUND_STOCHASTIC ? 8 * 128 : 1];   // per thread: 8 rows x 16 random bytes
    __shared__ uint32_t xchg[BLK == 64 ? 16 : 1];   // 64x64 blocks: maxima of the four warps' two half blocks
    // Programmatic dependent launch (used by fp4q_quantize2d_multi to chain the launches of independent tensors in
    // one stream): a launch configured as this one's dependent may start filling SMs as soon as every CTA of this
    // grid is resident, i.e. beside this grid's last wave.  Without such a configuration both instructions do nothing.
    asm volatile("griddepcontrol.launch_dependents;");
    const int64_t bx = (int64_t)blockIdx.x % p.grid_x, by = (int64_t)blockIdx.x / p.grid_x;
    const bool full = p.x_vec_ok == 2 && p.rng_aligned && (by + 1) * 128 <= p.rows && (bx + 1) * 128 <= p.cols;
    if (full) quantize_tile<MODE, true, BLK>(p, qt_stage, rnd_stage, xchg);
    else quantize_tile<MODE, false, BLK>(p, qt_stage, rnd_stage, xchg);
    // A dependent grid does not read what its predecessor wrote (different tensors), so it never waited for it; it
    // waits here, after its own stores, so that the grids of a chain still COMPLETE in launch order and whatever is
    // enqueued after the chain sees every tensor of it.
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace fp4q

using namespace fp4q;

// Argument checks and kernel parameters of one tensor.  *n_cta = 0 for an empty tensor (nothing to launch).
static fp4q_status prepare_quantize2d(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x, const fp4q_tensor *out,
                                      fp4q_round mode, uint64_t seed, uint32_t tensor_id, uint32_t flags, Quant2dParams &p,
                                      int64_t *n_cta)
{
    *n_cta = 0;
    if (rows < 0 || cols < 0) return FP4Q_ERR_SHAPE;
    if (mode != FP4Q_ROUND_NEAREST && mode != FP4Q_ROUND_STOCHASTIC) return FP4Q_ERR_UNSUPPORTED;
    if (flags & ~(FP4Q_INDEX_TRANSPOSED | FP4Q_BLOCK_16 | FP4Q_BLOCK_64)) return FP4Q_ERR_UNSUPPORTED;
    if ((flags & FP4Q_BLOCK_16) && (flags & FP4Q_BLOCK_64)) return FP4Q_ERR_UNSUPPORTED;
    const int sgran = (flags & FP4Q_BLOCK_16) ? 16 : 32;   // granularity of the scale matrix
    if (!out) return FP4Q_ERR_NULL;
    if (out->rows != rows || out->cols != cols) return FP4Q_ERR_SHAPE;
    if (rows == 0 || cols == 0) return FP4Q_OK;
    if (!x_bf16 || !out->q_rm || !out->scale) return FP4Q_ERR_NULL;
    if (ld_x < cols || out->ld_rm < round_up(cols, 32) / 2 || out->ld_s < ceil_div(cols, sgran)) return FP4Q_ERR_SHAPE;
    if (out->q_t && out->ld_t < round_up(rows, 32) / 2) return FP4Q_ERR_SHAPE;
    if (!aligned(x_bf16, 2) || !aligned(out->q_rm, 16) || out->ld_rm % 16 != 0) return FP4Q_ERR_ALIGN;
    if (out->q_t && (!aligned(out->q_t, 16) || out->ld_t % 16 != 0)) return FP4Q_ERR_ALIGN;

    p.x = static_cast<const uint16_t *>(x_bf16);
    p.rows = rows; p.cols = cols; p.ld_x = ld_x;
    p.q_rm = out->q_rm; p.ld_rm = out->ld_rm;
    p.q_t = out->q_t; p.ld_t = out->ld_t;
    p.scale = out->scale; p.ld_s = out->ld_s;
    p.grid_x = ceil_div(cols, 128);
    p.tensor_id = tensor_id;
    p.flags = flags;
    p.x_vec_ok = (aligned(x_bf16, 32) && ld_x % 16 == 0) ? 2 : (aligned(x_bf16, 16) && ld_x % 8 == 0) ? 1 : 0;
    p.rng_aligned = cols % 16 == 0 && !(flags & FP4Q_INDEX_TRANSPOSED);
    philox_round_keys(seed, p.keys);
    *n_cta = p.grid_x * ceil_div(rows, 128);
    if (*n_cta > 0x7FFFFFFF) return FP4Q_ERR_UNSUPPORTED;
    return FP4Q_OK;
}

extern "C" fp4q_status fp4q_quantize2d(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x,
                                       const fp4q_tensor *out, fp4q_round mode, uint64_t seed,
                                       uint32_t tensor_id, uint32_t flags, void *stream)
{
    Quant2dParams p;
    int64_t n_cta;
    if (fp4q_status st = prepare_quantize2d(x_bf16, rows, cols, ld_x, out, mode, seed, tensor_id, flags, p, &n_cta)) return st;
    if (n_cta == 0) return FP4Q_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool sr = mode == FP4Q_ROUND_STOCHASTIC;
    if (flags & FP4Q_BLOCK_16) {
        if (sr) quantize2d_kernel<FP4Q_ROUND_STOCHASTIC, 16><<<(unsigned)n_cta, 128, 0, s>>>(p);
        else quantize2d_kernel<FP4Q_ROUND_NEAREST, 16><<<(unsigned)n_cta, 128, 0, s>>>(p);
    } else if (flags & FP4Q_BLOCK_64) {
        if (sr) quantize2d_kernel<FP4Q_ROUND_STOCHASTIC, 64><<<(unsigned)n_cta, 128, 0, s>>>(p);
        else quantize2d_kernel<FP4Q_ROUND_NEAREST, 64><<<(unsigned)n_cta, 128, 0, s>>>(p);
    } else if (sr) {
        quantize2d_kernel<FP4Q_ROUND_STOCHASTIC><<<(unsigned)n_cta, 128, 0, s>>>(p);
    } else {
        quantize2d_kernel<FP4Q_ROUND_NEAREST><<<(unsigned)n_cta, 128, 0, s>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? FP4Q_OK : FP4Q_ERR_CUDA;
}

extern "C" fp4q_status fp4q_quantize2d_multi(const fp4q_quantize_job *jobs, int32_t n_jobs, fp4q_round mode, uint64_t seed,
                                             void *stream)
{
    if (n_jobs < 0) return FP4Q_ERR_SHAPE;
    if (n_jobs > 0 && !jobs) return FP4Q_ERR_NULL;
    // every job is checked before the first launch: an argument error leaves the stream untouched
    for (int32_t j = 0; j < n_jobs; j++) {
        if (jobs[j].flags & (FP4Q_BLOCK_16 | FP4Q_BLOCK_64)) return FP4Q_ERR_UNSUPPORTED;   // 32 x 32 blocks only
        Quant2dParams p;
        int64_t n_cta;
        if (fp4q_status st = prepare_quantize2d(jobs[j].x_bf16, jobs[j].rows, jobs[j].cols, jobs[j].ld_x, jobs[j].out, mode, seed,
                                                jobs[j].tensor_id, jobs[j].flags, p, &n_cta))
            return st;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // One launch of the one-tensor kernel per tensor, each after the first configured as the programmatic dependent of
    // the one before it: the tensors are independent, so a launch may begin beside its predecessor's last wave instead
    // of after it (what two streams would give, in one stream).
    bool first = true;
    for (int32_t j = 0; j < n_jobs; j++) {
        Quant2dParams p;
        int64_t n_cta;
        prepare_quantize2d(jobs[j].x_bf16, jobs[j].rows, jobs[j].cols, jobs[j].ld_x, jobs[j].out, mode, seed, jobs[j].tensor_id,
                           jobs[j].flags, p, &n_cta);
        if (n_cta == 0) continue;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)n_cta);
        cfg.blockDim = dim3(128);
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = first ? 0 : 1;
        const cudaError_t e = mode == FP4Q_ROUND_STOCHASTIC ? cudaLaunchKernelEx(&cfg, quantize2d_kernel<FP4Q_ROUND_STOCHASTIC, 32>, p)
                                                            : cudaLaunchKernelEx(&cfg, quantize2d_kernel<FP4Q_ROUND_NEAREST, 32>, p);
        if (e != cudaSuccess) return FP4Q_ERR_CUDA;
        first = false;
    }
    return FP4Q_OK;
}
