// Shared host-side helpers of the CUDA translation units (error plumbing, fast division).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "plan.h"

#define BASP_CUDA_TRY(expr)                                                   \
    do {                                                                      \
        cudaError_t e_ = (expr);                                              \
        if (e_ != cudaSuccess) {                                              \
            basp_set_cuda_error(#expr, (int)e_, cudaGetErrorString(e_));      \
            return BASP_ERR_CUDA;                                             \
        }                                                                     \
    } while (0)

// Division of a 31-bit dividend by a runtime constant: q = umulhi(n, mul) >> shr
// (round-up multiplier of Granlund & Montgomery, exact for n < 2^31).
struct FastDiv {
    uint32_t d, mul, shr;
};

inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f;
    f.d = d;
    if (d == 1) { f.mul = 0; f.shr = 0; return f; }
    uint32_t lg = 0;
    while ((1u << lg) < d) ++lg;                       // ceil(log2 d)
    const unsigned p = 31 + lg;
    f.mul = (uint32_t)(((1ull << p) + d - 1) / d);     // ceil(2^p / d) < 2^32
    f.shr = p - 32;
    return f;
}

__device__ __forceinline__ uint32_t fdiv(uint32_t n, const FastDiv &f) {
    return f.d == 1 ? n : (__umulhi(n, f.mul) >> f.shr);
}

static inline bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }
// A softmax scale the kernels accept: 0 (= 1/sqrt(D)) or a positive finite number (not NaN, not negative, not infinite).
static inline bool scale_ok(float s) { return s >= 0.f && s <= 3.0e38f; }
