// fp4q_quantize1d / fp4q_quantize1d_t: 1D-block (1 x 32) FP4 quantization, the layout the paper keeps for
// activations (Section 3.1), in both orientations the layer's products need:
//   fp4q_quantize1d    blocks along the rows of x (the channel axis of an activation [tokens, channels]):
//                      the A operand of the forward product;
//   fp4q_quantize1d_t  the encoding of x^T with blocks along the rows of x (the token axis): the B operand of the
//                      weight-gradient product, which contracts over tokens.
// Same arithmetic as the 2D quantizer (shared device functions): truncation-free power-of-two scale from the block
// maximum, E2M1 codes through the hardware converts, nearest-even or (row-wise form only) stochastic rounding
// keyed on the element's index i*cols + j.  Streaming kernels: one coalesced pass over x.
#include <cuda_bf16.h>

#include "common.cuh"
#include "quant_device.cuh"

namespace fp4q {

struct Quant1dParams {
    const uint16_t *x;
    int64_t rows, cols, ld_x;
    uint8_t *q;
    int64_t ld_q;
    uint8_t *scale;
    int64_t ld_s;
    int64_t segs_per_row;   // 16-element segments per row, even
    int x_vec_ok;
    uint32_t tensor_id;
    PhiloxRoundKeys keys;
};

// Each thread owns one whole block of 32 consecutive elements of a row (four 128-bit loads, one 128-bit store): no
// exchange between lanes, and the index arithmetic, the scale code and the scale store are paid once per block.
template <int MODE>
__global__ void __launch_bounds__(256) quantize1d_kernel(const __grid_constant__ Quant1dParams p)
{
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t blocks_per_row = p.segs_per_row >> 1, total = p.rows * blocks_per_row;
    if (gid >= total) return;
    int64_t i, blk;
    if (total <= 0x7FFFFFFF) {   // 32-bit division is several times cheaper than the 64-bit one
        i = (uint32_t)gid / (uint32_t)blocks_per_row;
        blk = (uint32_t)gid - (uint32_t)i * (uint32_t)blocks_per_row;
    } else {
        i = gid / blocks_per_row;
        blk = gid - i * blocks_per_row;
    }
    const int64_t j0 = blk * 32;

    uint32_t raw[16];
    const uint16_t *src = p.x + i * p.ld_x + j0;
    if (p.x_vec_ok && j0 + 32 <= p.cols) {
#pragma unroll
        for (int q = 0; q < 4; q++) {
            const uint4 a = __ldg(reinterpret_cast<const uint4 *>(src) + q);
            raw[4 * q] = a.x; raw[4 * q + 1] = a.y; raw[4 * q + 2] = a.z; raw[4 * q + 3] = a.w;
        }
    } else {
#pragma unroll
        for (int k = 0; k < 16; k++) {
            const uint32_t lo = (j0 + 2 * k < p.cols) ? (uint32_t)__ldg(src + 2 * k) : 0u;
            const uint32_t hi = (j0 + 2 * k + 1 < p.cols) ? (uint32_t)__ldg(src + 2 * k + 1) : 0u;
            raw[k] = lo | (hi << 16);
        }
    }
    // block maximum: packed BF16 |.| max with NaN propagation, so that any non-finite entry shows up in the
    // result and routes the block to the scalar path
    __nv_bfloat162 m2 = __float2bfloat162_rn(0.0f);
#pragma unroll
    for (int k = 0; k < 16; k++) m2 = __hmax2_nan(m2, __habs2(*reinterpret_cast<const __nv_bfloat162 *>(&raw[k])));
    const __nv_bfloat16 m1 = __hmax_nan(m2.x, m2.y);
    uint32_t fm = (uint32_t)(*reinterpret_cast<const uint16_t *>(&m1)) & 0x7FFFu;
    const bool nonfinite = fm >= 0x7F80u;
    if (nonfinite) {   // maximum over the finite entries only
        fm = 0;
#pragma unroll
        for (int k = 0; k < 16; k++) {
            const uint32_t lo = raw[k] & 0x7FFFu, hi = (raw[k] >> 16) & 0x7FFFu;
            if (lo < 0x7F80u && lo > fm) fm = lo;
            if (hi < 0x7F80u && hi > fm) fm = hi;
        }
    }
    const int code = scale_code_from_max(fm);
    p.scale[i * p.ld_s + blk] = (uint8_t)code;

    uint32_t W[4];
#pragma unroll
    for (int h = 0; h < 2; h++) {   // the block's two 16-element segments (one Philox block each: cols % 16 == 0)
        uint32_t R[4] = {0u, 0u, 0u, 0u};
        if (MODE == FP4Q_ROUND_STOCHASTIC) {
            const uint64_t pb = (uint64_t)(i * p.cols + j0 + 16 * h) >> 4;
            philox4x32_10((uint32_t)pb, (uint32_t)(pb >> 32), p.tensor_id, 0u, p.keys, R);
        }
        if (!nonfinite) {
            round_segment<MODE>(raw + 8 * h, inv_scale(code), R, W + 2 * h);
        } else {
            const uint2 w = round_segment_scalar<MODE>(make_uint4(raw[8 * h], raw[8 * h + 1], raw[8 * h + 2], raw[8 * h + 3]),
                                                       make_uint4(raw[8 * h + 4], raw[8 * h + 5], raw[8 * h + 6], raw[8 * h + 7]),
                                                       make_uint4(R[0], R[1], R[2], R[3]), inv_scale_f16_aligned(code));
            W[2 * h] = w.x;
            W[2 * h + 1] = w.y;
        }
    }
    *reinterpret_cast<uint4 *>(p.q + i * p.ld_q + (j0 >> 1)) = make_uint4(W[0], W[1], W[2], W[3]);
}

// The encoding of x^T, nearest rounding.  A warp owns 32 rows x 64 columns: each row is one coalesced 128-byte load,
// a lane keeps its two columns' 32 values in registers, and writes the 16 payload bytes of each column's block.
__global__ void __launch_bounds__(128) quantize1d_t_kernel(const __grid_constant__ Quant1dParams p)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t rb = (int64_t)blockIdx.y * 4 + warp;   // block of 32 rows
    const int64_t i0 = rb * 32, c0 = (int64_t)blockIdx.x * 64 + 2 * lane;
    if (i0 >= p.rows || c0 >= p.cols) return;
    const bool two = c0 + 1 < p.cols;
    uint32_t raw[32];
    if (p.x_vec_ok && two && i0 + 32 <= p.rows) {   // interior: 32 unconditional word loads, one address step each
        const uint32_t *src = reinterpret_cast<const uint32_t *>(p.x + i0 * p.ld_x + c0);
        const int64_t step = p.ld_x >> 1;
#pragma unroll
        for (int r = 0; r < 32; r++) raw[r] = __ldg(src + r * step);
    } else {
#pragma unroll
        for (int r = 0; r < 32; r++) {
            raw[r] = 0u;
            if (i0 + r < p.rows) {
                const uint16_t *src = p.x + (i0 + r) * p.ld_x + c0;
                raw[r] = (uint32_t)__ldg(src) | (two ? (uint32_t)__ldg(src + 1) << 16 : 0u);
            }
        }
    }
    // both columns' maxima at once: packed |.| max with NaN propagation; a non-finite entry routes the lane to the
    // careful path
    __nv_bfloat162 m2 = __float2bfloat162_rn(0.0f);
#pragma unroll
    for (int r = 0; r < 32; r++) m2 = __hmax2_nan(m2, __habs2(*reinterpret_cast<const __nv_bfloat162 *>(&raw[r])));
    uint32_t m0 = *reinterpret_cast<const uint32_t *>(&m2) & 0x7FFFu, m1 = (*reinterpret_cast<const uint32_t *>(&m2) >> 16) & 0x7FFFu;
    const bool nonfinite = m0 >= 0x7F80u || m1 >= 0x7F80u;
    if (nonfinite) {
        m0 = m1 = 0;
#pragma unroll
        for (int r = 0; r < 32; r++) {
            const uint32_t lo = raw[r] & 0x7FFFu, hi = (raw[r] >> 16) & 0x7FFFu;
            if (lo < 0x7F80u && lo > m0) m0 = lo;
            if (hi < 0x7F80u && hi > m1) m1 = hi;
        }
    }
    const int code0 = scale_code_from_max(m0), code1 = scale_code_from_max(m1);
    const float inv0 = inv_scale(code0), inv1 = inv_scale(code1);
    // One convert takes the same column of two consecutive rows: its result byte (row r in the low nibble, row r + 1
    // in the high one) is a payload byte of that column as it stands.
    uint32_t A[4], B[4];   // the two columns' 32 nibbles
#pragma unroll
    for (int g = 0; g < 4; g++) {
        uint32_t a = 0, b = 0;
#pragma unroll
        for (int e = 0; e < 4; e++) {
            uint32_t w0 = raw[8 * g + 2 * e], w1 = raw[8 * g + 2 * e + 1];
            uint32_t lo0 = w0 << 16, hi0 = w0 & 0xFFFF0000u, lo1 = w1 << 16, hi1 = w1 & 0xFFFF0000u;
            if (nonfinite) {   // NaN -> +0; +-Inf saturates to +-6 in the conversion
                if ((lo0 & 0x7FFFFFFFu) > 0x7F800000u) lo0 = 0u;
                if ((hi0 & 0x7FFFFFFFu) > 0x7F800000u) hi0 = 0u;
                if ((lo1 & 0x7FFFFFFFu) > 0x7F800000u) lo1 = 0u;
                if ((hi1 & 0x7FFFFFFFu) > 0x7F800000u) hi1 = 0u;
            }
            a |= cvt_rn_e2m1x2(__uint_as_float(lo1) * inv0, __uint_as_float(lo0) * inv0) << (8 * e);
            b |= cvt_rn_e2m1x2(__uint_as_float(hi1) * inv1, __uint_as_float(hi0) * inv1) << (8 * e);
        }
        A[g] = a;
        B[g] = b;
    }
    *reinterpret_cast<uint4 *>(p.q + c0 * p.ld_q + (i0 >> 1)) = make_uint4(A[0], A[1], A[2], A[3]);
    p.scale[c0 * p.ld_s + rb] = (uint8_t)code0;
    if (two) {
        *reinterpret_cast<uint4 *>(p.q + (c0 + 1) * p.ld_q + (i0 >> 1)) = make_uint4(B[0], B[1], B[2], B[3]);
        p.scale[(c0 + 1) * p.ld_s + rb] = (uint8_t)code1;
    }
}

// Eight consecutive rows of one column (two BF16 per word, low half = even row) through the scalar path, for blocks
// that hold a non-finite value; inv = 2^(-e-14).  Arguments by value, so that nothing of the caller's has to live in
// local memory.
__device__ __noinline__ uint32_t round_column_scalar(uint4 rows, float inv)
{
    const uint32_t r[4] = {rows.x, rows.y, rows.z, rows.w};
    uint32_t w = 0u;
#pragma unroll
    for (int k = 0; k < 4; k++) {
        const uint32_t lo = quantize_scalar<FP4Q_ROUND_NEAREST>(r[k] & 0xFFFFu, inv, 0u);
        const uint32_t hi = quantize_scalar<FP4Q_ROUND_NEAREST>(r[k] >> 16, inv, 0u);
        w |= (lo | (hi << 4)) << (8 * k);
    }
    return w;
}

// The same encoding for tensors whose shape and alignment allow full 128x128 tiles (rows and cols multiples of 128,
// 32-byte aligned rows): the access pattern of the 2D quantizer.  A CTA of 4 warps owns 128x128 elements, a warp 32
// rows x 128 columns, a lane 8 rows x 16 columns (one 256-bit load per row).  A block is now one column of the warp's
// 32 rows: the four lanes that share 16 columns reduce 16 column maxima with two shuffles of packed BF16 pairs, every
// element is scaled by its own column's factor, one convert takes the same column of two consecutive rows (its result
// byte is a payload byte as it stands), and the payload leaves through swizzled staging rows as 64 contiguous bytes
// per column; the four scale bytes of a column (one per warp) leave as
// one 32-bit store.
__global__ void __launch_bounds__(128, 4) quantize1d_t_tile_kernel(const __grid_constant__ Quant1dParams p)
{
    __shared__ uint4 qt_stage[128 * 4];      // 128 output rows (columns of x) x 64 B, 16-byte chunks XOR-swizzled
    __shared__ uint32_t sc_stage[128];       // per column of x: the scale codes of the CTA's four row blocks
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = lane >> 3, rg = (lane >> 1) & 3, ch = lane & 1;
    const int64_t grid_x = p.cols >> 7;
    const int64_t bx = (int64_t)blockIdx.x % grid_x, by = (int64_t)blockIdx.x / grid_x;
    const int64_t row0 = by * 128 + warp * 32 + rg * 8, col0 = bx * 128 + t * 32 + ch * 16;

    uint32_t raw[8][8];
    {
        const uint16_t *src = p.x + row0 * p.ld_x + col0;
#pragma unroll
        for (int r = 0; r < 8; r++)
            asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(raw[r][0]), "=r"(raw[r][1]), "=r"(raw[r][2]), "=r"(raw[r][3]), "=r"(raw[r][4]),
                           "=r"(raw[r][5]), "=r"(raw[r][6]), "=r"(raw[r][7])
                         : "l"(src + r * p.ld_x));
    }
    // column maxima over the lane's 8 rows, then over the four lanes (rg) that hold the other rows of the block
    uint32_t m2[8];
    bool nonfinite = false;
#pragma unroll
    for (int k = 0; k < 8; k++) {
        __nv_bfloat162 m = __float2bfloat162_rn(0.0f);
#pragma unroll
        for (int r = 0; r < 8; r++) m = __hmax2_nan(m, __habs2(*reinterpret_cast<const __nv_bfloat162 *>(&raw[r][k])));
#pragma unroll
        for (int sft = 2; sft <= 4; sft <<= 1) {
            uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, *reinterpret_cast<uint32_t *>(&m), sft);
            m = __hmax2_nan(m, *reinterpret_cast<__nv_bfloat162 *>(&other));
        }
        m2[k] = *reinterpret_cast<uint32_t *>(&m) & 0x7FFF7FFFu;
        nonfinite |= (m2[k] & 0xFFFFu) >= 0x7F80u || (m2[k] >> 16) >= 0x7F80u;
    }
    const bool careful = __any_sync(0xFFFFFFFFu, nonfinite);   // warp-uniform: the shuffles below need every lane
    if (careful) {   // maxima over the finite entries only
#pragma unroll
        for (int k = 0; k < 8; k++) {
            uint32_t lo = 0, hi = 0;
#pragma unroll
            for (int r = 0; r < 8; r++) {
                const uint32_t a = raw[r][k] & 0x7FFFu, b = (raw[r][k] >> 16) & 0x7FFFu;
                if (a < 0x7F80u && a > lo) lo = a;
                if (b < 0x7F80u && b > hi) hi = b;
            }
#pragma unroll
            for (int sft = 2; sft <= 4; sft <<= 1) {
                const uint32_t ol = __shfl_xor_sync(0xFFFFFFFFu, lo, sft), oh = __shfl_xor_sync(0xFFFFFFFFu, hi, sft);
                lo = ol > lo ? ol : lo;
                hi = oh > hi ? oh : hi;
            }
            m2[k] = lo | (hi << 16);
        }
    }
    uint32_t codes[4] = {0u, 0u, 0u, 0u};   // 16 scale codes, one byte each
    float inv[16];
#pragma unroll
    for (int c = 0; c < 16; c++) {
        const int code = scale_code_from_max((m2[c >> 1] >> (16 * (c & 1))) & 0x7FFFu);
        codes[c >> 2] |= (uint32_t)code << (8 * (c & 3));
        inv[c] = careful ? inv_scale_f16_aligned(code) : inv_scale(code);
    }
    if (rg == 0) {
        uint8_t *sc = reinterpret_cast<uint8_t *>(sc_stage);
#pragma unroll
        for (int c = 0; c < 16; c++) sc[(32 * t + 16 * ch + c) * 4 + warp] = (uint8_t)(codes[c >> 2] >> (8 * (c & 3)));
    }
    // Per column the lane's 8 codes (rows row0 .. row0 + 7) as one word: one convert takes the same column of two
    // consecutive rows, so its result byte is a payload byte of that column as it stands.
    uint32_t *stage = reinterpret_cast<uint32_t *>(qt_stage);
#pragma unroll
    for (int c = 0; c < 16; c++) {
        uint32_t word = 0;
        if (!careful) {
#pragma unroll
            for (int e = 0; e < 4; e++) {
                const uint32_t w0 = raw[2 * e][c >> 1], w1 = raw[2 * e + 1][c >> 1];
                const float v0 = __uint_as_float((c & 1) ? (w0 & 0xFFFF0000u) : (w0 << 16)) * inv[c];
                const float v1 = __uint_as_float((c & 1) ? (w1 & 0xFFFF0000u) : (w1 << 16)) * inv[c];
                word |= cvt_rn_e2m1x2(v1, v0) << (8 * e);
            }
        } else {   // rare: kept small and out of the hot loop's instruction footprint
            uint32_t h[4];
#pragma unroll
            for (int e = 0; e < 4; e++) {
                const uint32_t w0 = raw[2 * e][c >> 1], w1 = raw[2 * e + 1][c >> 1];
                h[e] = (c & 1) ? ((w0 >> 16) | (w1 & 0xFFFF0000u)) : ((w0 & 0xFFFFu) | (w1 << 16));
            }
            word = round_column_scalar(make_uint4(h[0], h[1], h[2], h[3]), inv[c]);
        }
        const int col_local = 32 * t + 16 * ch + c;
        // word index inside the 64-byte row: 4*(source warp) + rg, with the 16-byte chunk index XORed by the
        // column's block index so that a warp's stores spread over the banks
        stage[col_local * 16 + (((warp ^ t) << 2) | rg)] = word;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; k++) {
        const int row_local = (threadIdx.x >> 2) + 32 * k;   // output row = column of x; its 32-column group is k
        const int chunk = threadIdx.x & 3;                    // 32 rows of x = one source warp
        const uint4 v = qt_stage[row_local * 4 + (chunk ^ k)];
        *reinterpret_cast<uint4 *>(p.q + (bx * 128 + row_local) * p.ld_q + by * 64 + chunk * 16) = v;
    }
    *reinterpret_cast<uint32_t *>(p.scale + (bx * 128 + threadIdx.x) * p.ld_s + by * 4) = sc_stage[threadIdx.x];
}

}  // namespace fp4q

using namespace fp4q;

extern "C" fp4q_status fp4q_quantize1d(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x, uint8_t *q, int64_t ld_q,
                                       uint8_t *scale, int64_t ld_s, fp4q_round mode, uint64_t seed, uint32_t tensor_id,
                                       void *stream)
{
    if (rows < 0 || cols < 0) return FP4Q_ERR_SHAPE;
    if (mode != FP4Q_ROUND_NEAREST && mode != FP4Q_ROUND_STOCHASTIC) return FP4Q_ERR_UNSUPPORTED;
    if (mode == FP4Q_ROUND_STOCHASTIC && cols % 16 != 0) return FP4Q_ERR_UNSUPPORTED;
    if (rows == 0 || cols == 0) return FP4Q_OK;
    if (!x_bf16 || !q || !scale) return FP4Q_ERR_NULL;
    if (ld_x < cols || ld_q < round_up(cols, 32) / 2 || ld_s < ceil_div(cols, 32)) return FP4Q_ERR_SHAPE;
    if (!aligned(x_bf16, 2) || !aligned(q, 16) || ld_q % 16 != 0) return FP4Q_ERR_ALIGN;
    Quant1dParams p;
    p.x = static_cast<const uint16_t *>(x_bf16);
    p.rows = rows; p.cols = cols; p.ld_x = ld_x;
    p.q = q; p.ld_q = ld_q; p.scale = scale; p.ld_s = ld_s;
    p.segs_per_row = round_up(cols, 32) / 16;
    p.x_vec_ok = aligned(x_bf16, 16) && ld_x % 8 == 0;
    p.tensor_id = tensor_id;
    philox_round_keys(seed, p.keys);
    const int64_t n_cta = ceil_div(rows * (p.segs_per_row / 2), 256);
    if (n_cta > 0x7FFFFFFF) return FP4Q_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (mode == FP4Q_ROUND_STOCHASTIC) quantize1d_kernel<FP4Q_ROUND_STOCHASTIC><<<(unsigned)n_cta, 256, 0, s>>>(p);
    else quantize1d_kernel<FP4Q_ROUND_NEAREST><<<(unsigned)n_cta, 256, 0, s>>>(p);
    return cudaGetLastError() == cudaSuccess ? FP4Q_OK : FP4Q_ERR_CUDA;
}

extern "C" fp4q_status fp4q_quantize1d_t(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x, uint8_t *q, int64_t ld_q,
                                         uint8_t *scale, int64_t ld_s, void *stream)
{
    if (rows < 0 || cols < 0) return FP4Q_ERR_SHAPE;
    if (rows == 0 || cols == 0) return FP4Q_OK;
    if (!x_bf16 || !q || !scale) return FP4Q_ERR_NULL;
    if (ld_x < cols || ld_q < round_up(rows, 32) / 2 || ld_s < ceil_div(rows, 32)) return FP4Q_ERR_SHAPE;
    if (!aligned(x_bf16, 2) || !aligned(q, 16) || ld_q % 16 != 0) return FP4Q_ERR_ALIGN;
    Quant1dParams p = {};
    p.x = static_cast<const uint16_t *>(x_bf16);
    p.rows = rows; p.cols = cols; p.ld_x = ld_x;
    p.q = q; p.ld_q = ld_q; p.scale = scale; p.ld_s = ld_s;
    p.x_vec_ok = aligned(x_bf16, 4) && ld_x % 2 == 0;
    // full 128x128 tiles and aligned rows: the tile kernel (coalesced 64-byte column stores)
    if (rows % 128 == 0 && cols % 128 == 0 && aligned(x_bf16, 32) && ld_x % 16 == 0 && ld_s % 4 == 0 && aligned(scale, 4) &&
        (rows / 128) * (cols / 128) <= 0x7FFFFFFF) {
        quantize1d_t_tile_kernel<<<(unsigned)((rows / 128) * (cols / 128)), 128, 0, static_cast<cudaStream_t>(stream)>>>(p);
        return cudaGetLastError() == cudaSuccess ? FP4Q_OK : FP4Q_ERR_CUDA;
    }
    const int64_t gx = ceil_div(cols, 64), gy = ceil_div(ceil_div(rows, 32), 4);
    if (gx > 0x7FFFFFFF || gy > 65535) return FP4Q_ERR_UNSUPPORTED;
    quantize1d_t_kernel<<<dim3((unsigned)gx, (unsigned)gy), 128, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? FP4Q_OK : FP4Q_ERR_CUDA;
}
