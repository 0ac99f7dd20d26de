// Shared declarations of the vitint CUDA library (sm_100a only).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "vitint.h"

namespace vitint {

// Device status word: 0, or VITINT_ERR_TIMEOUT once any bounded wait gave up.  The library
// is built as ONE translation unit (vitint_lib.cu), so this is the only instance.
__device__ int g_device_status = 0;

inline int container_bits(int bits) { return bits == 3 ? 4 : bits; }
inline bool valid_bits(int bits) { return bits == 2 || bits == 3 || bits == 4 || bits == 8; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t row_bytes(int64_t cols, int bits) { return (cols * container_bits(bits) + 7) / 8; }
inline int max_abs_code(int bits, int is_signed) { return is_signed ? (1 << (bits - 1)) : (1 << bits) - 1; }
inline void code_range(int bits, int is_signed, int* qn, int* qp) {
    if (is_signed) { *qn = -(1 << (bits - 1)); *qp = (1 << (bits - 1)) - 1; }
    else           { *qn = 0;                  *qp = (1 << bits) - 1; }
}

// Checks a code descriptor: pointer, sizes, bits, pitch and alignment.
int check_codes(const vitint_codes* c);

int cuda_status(cudaError_t e);

// ---------------------------------------------------------------------------
// device helpers shared by the element-wise kernels
// ---------------------------------------------------------------------------

// clamp(rint(r)) with ties-to-even; NaN maps to the low end like the host reference
// rule "not >= qn".
__device__ __forceinline__ int round_clamp(float r, float qn, float qp) {
    float n = rintf(r);
    n = (n >= qn) ? n : qn;
    n = (n > qp) ? qp : n;
    return (int)n;
}

// GELU(y) = y * Phi(y).  Positive side: 0.5*y*(1 + erf(y/sqrt2)); negative side through
// erfc so the small tail keeps its relative accuracy.
__device__ __forceinline__ float gelu_f32(float y) {
    const float z = y * 0.70710678118654752440f;
    if (y >= 0.0f) return 0.5f * y * (1.0f + erff(z));
    return 0.5f * y * erfcf(-z);
}

}  // namespace vitint
