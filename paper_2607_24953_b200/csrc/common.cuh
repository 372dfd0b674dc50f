// Shared host/device helpers of libfp4q (internal; the public interface is include/fp4q.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fp4q.h"

namespace fp4q {

constexpr int kBlock = 32;  // 2D block size b (Section 3: 32x32 blocks)

static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }
static inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Layout of the GEMM workspace (device memory, caller-owned).
struct Workspace {
    uint32_t status;         // 0 = ok, otherwise an fp4q_status written by a kernel
    uint32_t detail;         // where the kernel gave up (role/stage), for diagnostics
    uint32_t wait_limit;     // polls after which a bounded wait gives up; 0 = the kernels' default
    uint32_t withhold_load;  // development hook, 0 in production: n > 0 = CTA 0 leaves out its n-th stage load
    uint32_t pad[60];
};

}  // namespace fp4q
