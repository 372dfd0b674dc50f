// Host-side wrappers around LIBRARY routines that the oracle tests use as independent pins:
// NVIDIA's FP4/FP8/E8M0 conversion helpers (cuda_fp4.h, cuda_fp8.h), cuRAND's Philox4x32-10 round
// function and ATen's philox_engine.  Nothing here is part of the oracle or of the CUDA library;
// everything runs on the host (the file is compiled by nvcc only because the headers want it).
#include <cstdint>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_fp4.h>
#include <nv/target>
#define QUALIFIERS static inline __host__ __device__   // the header's block function has a host branch
#include <curand_philox4x32_x.h>
#ifndef AT_ASSERT
#define AT_ASSERT(...)   // only used by a device-side guard of a function this file never calls
#endif
#include <ATen/core/PhiloxRNGEngine.h>

extern "C" {

// E2M1 code (low 4 bits) -> value, through the half-precision decode of cuda_fp4.h.
float pin_fp4_decode(int code)
{
    __half_raw h = __nv_cvt_fp4_to_halfraw((__nv_fp4_storage_t)(code & 0xF), __NV_E2M1);
    return __half2float(__half(h));
}

// float -> E2M1 code, round to nearest even, saturating (cuda_fp4.h).
int pin_fp4_encode_rn(float x)
{
    return (int)__nv_cvt_float_to_fp4(x, __NV_E2M1, cudaRoundNearest) & 0xF;
}

// float -> E4M3 code, round to nearest even, saturating to finite (cuda_fp8.h).
int pin_e4m3_encode_rn(float x)
{
    return (int)__nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3) & 0xFF;
}

float pin_e4m3_decode(int code)
{
    __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)(code & 0xFF), __NV_E4M3);
    return __half2float(__half(h));
}

// float -> UE8M0 code with the exponent rounded toward +infinity (cuda_fp8.h).
int pin_e8m0_encode_ceil(float x)
{
    return (int)__nv_cvt_float_to_e8m0(x, __NV_SATFINITE, cudaRoundPosInf) & 0xFF;
}

// cuRAND's Philox4x32-10 block function.
void pin_philox_curand(const uint32_t *ctr, const uint32_t *key, uint32_t *out)
{
    uint4 c = make_uint4(ctr[0], ctr[1], ctr[2], ctr[3]);
    uint2 k = make_uint2(key[0], key[1]);
    uint4 r = curand_Philox4x32_10(c, k);
    out[0] = r.x; out[1] = r.y; out[2] = r.z; out[3] = r.w;
}

// ATen's engine: counter = (offset lo, offset hi, subsequence lo, subsequence hi), key = seed.
void pin_philox_aten(uint64_t seed, uint64_t subsequence, uint64_t offset, uint32_t *out)
{
    at::philox_engine eng(seed, subsequence, offset);
    for (int i = 0; i < 4; i++) out[i] = eng();
}

}  // extern "C"
