// fp4q_mxfp8_quantize1d: BF16 -> MXFP8 operand (E4M3 payload, one UE8M0 scale per 32 consecutive
// elements of a row), the operand format of the query/key projections.  Streaming kernel: each
// thread owns one block of 32 consecutive elements (four 128-bit loads, two 128-bit stores).
#include <cuda_bf16.h>

#include "common.cuh"

namespace fp4q {

struct Mxfp8QuantParams {
    const uint16_t *x;
    int64_t rows, cols, ld_x;
    uint8_t *q;
    int64_t ld_q;
    uint8_t *scale;
    int64_t ld_s;
    int64_t segs_per_row;   // 16-element segments per row, even
    int x_vec_ok;
};

// {hi, lo} -> two E4M3 bytes (hi in bits 15..8), round to nearest even, saturating to +-448.
__device__ __forceinline__ uint32_t cvt_rn_e4m3x2(float hi, float lo)
{
    uint16_t d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}

__global__ void __launch_bounds__(256) mxfp8_quantize1d_kernel(const __grid_constant__ Mxfp8QuantParams p)
{
    // one whole block of 32 elements per thread: four 128-bit loads, two 128-bit stores, no exchange between lanes
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

    // block maximum: packed BF16 |.| max with NaN propagation; a non-finite entry sends the thread through the
    // careful pass (maximum over the finite magnitudes, NaN -> +0; +-Inf saturates in the conversion)
    __nv_bfloat162 m2 = __float2bfloat162_rn(0.0f);
#pragma unroll
    for (int k = 0; k < 16; k++) m2 = __hmax2_nan(m2, __habs2(*reinterpret_cast<const __nv_bfloat162 *>(&raw[k])));
    const __nv_bfloat16 m1 = __hmax_nan(m2.x, m2.y);
    uint32_t fm = (uint32_t)(*reinterpret_cast<const uint16_t *>(&m1)) & 0x7FFFu;
    if (fm >= 0x7F80u) {
        fm = 0;
#pragma unroll
        for (int k = 0; k < 16; k++) {
            const uint32_t lo = raw[k] & 0x7FFFu, hi = (raw[k] >> 16) & 0x7FFFu;
            if (lo < 0x7F80u && lo > fm) fm = lo;
            if (hi < 0x7F80u && hi > fm) fm = hi;
            if (lo > 0x7F80u) raw[k] &= 0xFFFF0000u;
            if (hi > 0x7F80u) raw[k] &= 0x0000FFFFu;
        }
    }

    // smallest e with 448*2^e >= M: code = be - 8 + (m7 > 0x60), clamped at 0
    const int be = (int)(fm >> 7), m7 = (int)(fm & 0x7F);
    int code = be == 0 ? 0 : be - 8 + (m7 > 0x60 ? 1 : 0);
    code = code < 0 ? 0 : code;
    const float inv = __uint_as_float((uint32_t)(254 - code) << 23);   // 2^(127-code) = 2^-e
    p.scale[i * p.ld_s + blk] = (uint8_t)code;

    uint32_t out[8];
#pragma unroll
    for (int w = 0; w < 8; w++) {
        const uint32_t w0 = raw[2 * w], w1 = raw[2 * w + 1];
        out[w] = cvt_rn_e4m3x2(__uint_as_float(w0 & 0xFFFF0000u) * inv, __uint_as_float(w0 << 16) * inv) |
                 (cvt_rn_e4m3x2(__uint_as_float(w1 & 0xFFFF0000u) * inv, __uint_as_float(w1 << 16) * inv) << 16);
    }
    uint4 *dst = reinterpret_cast<uint4 *>(p.q + i * p.ld_q + j0);
    dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
    dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
}

// The transpose of the same operand: q_t[j, i] = E4M3 of x[i, j] with one scale per column j and 32 consecutive rows i
// (the contraction axis of the backward products).  A warp owns 32 rows x 64 columns: each row is one coalesced
// 128-byte load, a lane keeps its two columns' 32 values in registers, and writes 32 contiguous payload bytes per
// column (one whole sector each).
__global__ void __launch_bounds__(128) mxfp8_quantize1d_t_kernel(const __grid_constant__ Mxfp8QuantParams p)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t rb = (int64_t)blockIdx.y * 4 + warp;            // block of 32 rows
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
    // careful path (maxima over finite magnitudes, NaN -> +0)
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
    int code[2];
    float inv[2];
#pragma unroll
    for (int k = 0; k < 2; k++) {
        const uint32_t fm = k ? m1 : m0;
        const int be = (int)(fm >> 7), m7 = (int)(fm & 0x7F);
        int c = be == 0 ? 0 : be - 8 + (m7 > 0x60 ? 1 : 0);
        code[k] = c < 0 ? 0 : c;
        inv[k] = __uint_as_float((uint32_t)(254 - code[k]) << 23);
    }
    // One convert takes the same column of two consecutive rows: its two result bytes are consecutive payload bytes
    // of that column.  +-Inf saturates to +-448 in the conversion.
    uint32_t A[8], B[8];   // the two columns' 32 payload bytes
#pragma unroll
    for (int w = 0; w < 8; w++) {
        uint32_t a = 0, b = 0;
#pragma unroll
        for (int e = 0; e < 2; e++) {
            const uint32_t w0 = raw[4 * w + 2 * e], w1 = raw[4 * w + 2 * e + 1];
            uint32_t lo0 = w0 << 16, hi0 = w0 & 0xFFFF0000u, lo1 = w1 << 16, hi1 = w1 & 0xFFFF0000u;
            if (nonfinite) {
                if ((lo0 & 0x7FFFFFFFu) > 0x7F800000u) lo0 = 0u;
                if ((hi0 & 0x7FFFFFFFu) > 0x7F800000u) hi0 = 0u;
                if ((lo1 & 0x7FFFFFFFu) > 0x7F800000u) lo1 = 0u;
                if ((hi1 & 0x7FFFFFFFu) > 0x7F800000u) hi1 = 0u;
            }
            a |= cvt_rn_e4m3x2(__uint_as_float(lo1) * inv[0], __uint_as_float(lo0) * inv[0]) << (16 * e);
            b |= cvt_rn_e4m3x2(__uint_as_float(hi1) * inv[1], __uint_as_float(hi0) * inv[1]) << (16 * e);
        }
        A[w] = a;
        B[w] = b;
    }
    uint8_t *dst = p.q + c0 * p.ld_q + i0;
    reinterpret_cast<uint4 *>(dst)[0] = make_uint4(A[0], A[1], A[2], A[3]);
    reinterpret_cast<uint4 *>(dst)[1] = make_uint4(A[4], A[5], A[6], A[7]);
    p.scale[c0 * p.ld_s + rb] = (uint8_t)code[0];
    if (two) {
        dst += p.ld_q;
        reinterpret_cast<uint4 *>(dst)[0] = make_uint4(B[0], B[1], B[2], B[3]);
        reinterpret_cast<uint4 *>(dst)[1] = make_uint4(B[4], B[5], B[6], B[7]);
        p.scale[(c0 + 1) * p.ld_s + rb] = (uint8_t)code[1];
    }
}

// The same encoding for tensors made of full 128x128 tiles with 32-byte aligned rows: the access pattern of the 2D
// FP4 quantizer.  A CTA of 4 warps owns 128x128 elements, a warp 32 rows x 128 columns, a lane 8 rows x 16 columns (one
// 256-bit load per row).  The four lanes that share 16 columns reduce the 16 column maxima of the warp's 32 rows with
// two shuffles of packed BF16 pairs; one convert takes the same column of two consecutive rows, so a lane holds 8
// payload bytes per column as they are stored; they cross 16 KB of shared memory (16-byte chunks XOR-swizzled by the
// column's group) and leave as 128 contiguous bytes per column; the four scale bytes of a column as one word.
__global__ void __launch_bounds__(128, 4) mxfp8_quantize1d_t_tile_kernel(const __grid_constant__ Mxfp8QuantParams p)
{
    __shared__ uint4 stage[128 * 8];         // 128 output rows (columns of x) x 128 B
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
    if (careful) {   // maxima over the finite entries only; NaN -> +0 (+-Inf saturates in the conversion)
#pragma unroll
        for (int k = 0; k < 8; k++) {
            uint32_t lo = 0, hi = 0;
#pragma unroll
            for (int r = 0; r < 8; r++) {
                const uint32_t a = raw[r][k] & 0x7FFFu, b = (raw[r][k] >> 16) & 0x7FFFu;
                if (a < 0x7F80u && a > lo) lo = a;
                if (b < 0x7F80u && b > hi) hi = b;
                if (a > 0x7F80u) raw[r][k] &= 0xFFFF0000u;
                if (b > 0x7F80u) raw[r][k] &= 0x0000FFFFu;
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
    uint32_t codes[4] = {0u, 0u, 0u, 0u};
    float inv[16];
#pragma unroll
    for (int c = 0; c < 16; c++) {
        const uint32_t fm = (m2[c >> 1] >> (16 * (c & 1))) & 0x7FFFu;
        const int be = (int)(fm >> 7), m7 = (int)(fm & 0x7F);
        int code = be == 0 ? 0 : be - 8 + (m7 > 0x60 ? 1 : 0);   // smallest e with 448*2^e >= M
        code = code < 0 ? 0 : code;
        codes[c >> 2] |= (uint32_t)code << (8 * (c & 3));
        inv[c] = __uint_as_float((uint32_t)(254 - code) << 23);
    }
    if (rg == 0) {
        uint8_t *sc = reinterpret_cast<uint8_t *>(sc_stage);
#pragma unroll
        for (int c = 0; c < 16; c++) sc[(32 * t + 16 * ch + c) * 4 + warp] = (uint8_t)(codes[c >> 2] >> (8 * (c & 3)));
    }
    // per column the lane's 8 payload bytes (rows row0 .. row0 + 7), into the column's staging row
#pragma unroll
    for (int c = 0; c < 16; c++) {
        uint32_t w[2];
#pragma unroll
        for (int h = 0; h < 2; h++) {
            uint32_t acc = 0;
#pragma unroll
            for (int e = 0; e < 2; e++) {
                const int r = 4 * h + 2 * e;
                const uint32_t w0 = raw[r][c >> 1], w1 = raw[r + 1][c >> 1];
                const float v0 = __uint_as_float((c & 1) ? (w0 & 0xFFFF0000u) : (w0 << 16)) * inv[c];
                const float v1 = __uint_as_float((c & 1) ? (w1 & 0xFFFF0000u) : (w1 << 16)) * inv[c];
                acc |= cvt_rn_e4m3x2(v1, v0) << (16 * e);
            }
            w[h] = acc;
        }
        const int col_local = 32 * t + 16 * ch + c;
        const int chunk = (warp * 2 + (rg >> 1)) ^ ((col_local >> 4) & 7);
        reinterpret_cast<uint2 *>(stage)[(col_local * 8 + chunk) * 2 + (rg & 1)] = make_uint2(w[0], w[1]);
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 8; k++) {
        const int row_local = (threadIdx.x >> 3) + 16 * k;   // output row = column of x
        const int chunk = threadIdx.x & 7;                    // 16 source rows
        const uint4 v = stage[row_local * 8 + (chunk ^ ((row_local >> 4) & 7))];
        *reinterpret_cast<uint4 *>(p.q + (bx * 128 + row_local) * p.ld_q + by * 128 + chunk * 16) = v;
    }
    *reinterpret_cast<uint32_t *>(p.scale + (bx * 128 + threadIdx.x) * p.ld_s + by * 4) = sc_stage[threadIdx.x];
}

}  // namespace fp4q

using namespace fp4q;

extern "C" fp4q_status fp4q_mxfp8_quantize1d(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x,
                                             uint8_t *q, int64_t ld_q, uint8_t *scale, int64_t ld_s,
                                             void *stream)
{
    if (rows < 0 || cols < 0) return FP4Q_ERR_SHAPE;
    if (rows == 0 || cols == 0) return FP4Q_OK;
    if (!x_bf16 || !q || !scale) return FP4Q_ERR_NULL;
    if (ld_x < cols || ld_q < round_up(cols, 32) || ld_s < ceil_div(cols, 32)) return FP4Q_ERR_SHAPE;
    if (!aligned(x_bf16, 2) || !aligned(q, 16) || ld_q % 16 != 0) return FP4Q_ERR_ALIGN;

    Mxfp8QuantParams p;
    p.x = static_cast<const uint16_t *>(x_bf16);
    p.rows = rows; p.cols = cols; p.ld_x = ld_x;
    p.q = q; p.ld_q = ld_q; p.scale = scale; p.ld_s = ld_s;
    p.segs_per_row = round_up(cols, 32) / 16;
    p.x_vec_ok = aligned(x_bf16, 16) && ld_x % 8 == 0;
    const int64_t total = rows * (p.segs_per_row / 2);
    const int64_t n_cta = ceil_div(total, 256);
    if (n_cta > 0x7FFFFFFF) return FP4Q_ERR_UNSUPPORTED;
    mxfp8_quantize1d_kernel<<<(unsigned)n_cta, 256, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? FP4Q_OK : FP4Q_ERR_CUDA;
}

extern "C" fp4q_status fp4q_mxfp8_quantize1d_t(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x,
                                               uint8_t *q, int64_t ld_q, uint8_t *scale, int64_t ld_s,
                                               void *stream)
{
    if (rows < 0 || cols < 0) return FP4Q_ERR_SHAPE;
    if (rows == 0 || cols == 0) return FP4Q_OK;
    if (!x_bf16 || !q || !scale) return FP4Q_ERR_NULL;
    if (ld_x < cols || ld_q < round_up(rows, 32) || ld_s < ceil_div(rows, 32)) return FP4Q_ERR_SHAPE;
    if (!aligned(x_bf16, 2) || !aligned(q, 16) || ld_q % 16 != 0) return FP4Q_ERR_ALIGN;

    Mxfp8QuantParams p;
    p.x = static_cast<const uint16_t *>(x_bf16);
    p.rows = rows; p.cols = cols; p.ld_x = ld_x;
    p.q = q; p.ld_q = ld_q; p.scale = scale; p.ld_s = ld_s;
    p.segs_per_row = 0;
    p.x_vec_ok = aligned(x_bf16, 4) && ld_x % 2 == 0;
    // full 128x128 tiles and aligned rows: the tile kernel (coalesced 128-byte column stores)
    if (rows % 128 == 0 && cols % 128 == 0 && aligned(x_bf16, 32) && ld_x % 16 == 0 && ld_s % 4 == 0 && aligned(scale, 4) &&
        (rows / 128) * (cols / 128) <= 0x7FFFFFFF) {
        mxfp8_quantize1d_t_tile_kernel<<<(unsigned)((rows / 128) * (cols / 128)), 128, 0, static_cast<cudaStream_t>(stream)>>>(p);
        return cudaGetLastError() == cudaSuccess ? FP4Q_OK : FP4Q_ERR_CUDA;
    }
    const int64_t gx = ceil_div(cols, 64), gy = ceil_div(ceil_div(rows, 32), 4);
    if (gx > 0x7FFFFFFF || gy > 65535) return FP4Q_ERR_UNSUPPORTED;
    mxfp8_quantize1d_t_kernel<<<dim3((unsigned)gx, (unsigned)gy), 128, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? FP4Q_OK : FP4Q_ERR_CUDA;
}
