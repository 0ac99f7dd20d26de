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
// Container actually used by a code matrix (a descriptor may ask for one code per byte).
inline int codes_container(const vitint_codes* c) { return c->container_bits ? c->container_bits : container_bits(c->bits); }
inline int64_t codes_row_bytes(const vitint_codes* c, int64_t cols) { return (cols * codes_container(c) + 7) / 8; }
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

// ---- quantizer arithmetic without the conversion / special-function unit ----------------
// The streaming kernels run several conversions per element; fp32<->int, fp32<->fp64, rint
// and the reciprocal of an IEEE division all issue on the quarter-rate XU pipe, which then
// bounds the kernel long before HBM does.  The helpers below produce the same bits with
// FMA-pipe and integer instructions only.

// Correctly rounded a / b from r = RN(1/b) by one Newton correction on the quotient
// (Markstein): q0 = RN(a*r); rem = a - q0*b (exact in an FMA); q = RN(q0 + rem*r) = RN(a/b)
// whenever b's significand is not all ones and nothing underflows.  A quotient that
// underflows is below 2^-100 in magnitude and quantizes to code 0 either way.
struct Divisor {
    float b, r;
    int exact;   // 0: significand of b is all ones, use the IEEE division instead
};
__device__ __forceinline__ Divisor make_divisor(float b) {
    Divisor d;
    d.b = b;
    d.r = __frcp_rn(b);
    d.exact = ((__float_as_uint(b) & 0x007FFFFFu) != 0x007FFFFFu) ? 1 : 0;
    return d;
}
// Straight-line form for inner loops; valid only when d.exact (callers test that once, outside
// the loop, because a branch per element would serialise the otherwise independent elements).
__device__ __forceinline__ float div_rn_exact(float a, const Divisor& d) {
    const float q0 = a * d.r;
    const float rem = fmaf(-q0, d.b, a);
    return fmaf(rem, d.r, q0);
}
__device__ __forceinline__ float div_rn(float a, const Divisor& d) {
    return d.exact ? div_rn_exact(a, d) : __fdiv_rn(a, d.b);
}

// clamp(rint(r)) as an integer code, ties to even, NaN -> qn.  The clamp to the integer
// bounds commutes with rounding; adding 1.5*2^23 rounds to an integer in the FMA pipe and
// leaves the two's-complement code in the low mantissa bits.
__device__ __forceinline__ uint32_t round_clamp_bits(float r, float qn, float qp) {
    const float c = fminf(fmaxf(r, qn), qp);
    return __float_as_uint(c + 12582912.0f);   // low bits = code (mod 2^22)
}

// (float)v for |v| < 2^22 without a conversion instruction.
__device__ __forceinline__ float small_int_to_float(int v) {
    return __int_as_float(0x4B400000 + v) - 12582912.0f;
}

// GELU(y) = y * Phi(y) = 0.5*y*(1 + erf(y/sqrt 2)), with erf from
//   erf(z) = sign(z) * (1 - 2^(-q(|z|))),   q(z) = -log2(erfc(z)) ~ z*(c0 + c1 z + ... + c6 z^6)
// on |z| <= 4 (beyond that erf is 1 to 2e-8).  The coefficients are a weighted minimax fit
// (max |erf error| 7.8e-8 in exact arithmetic); with ex2.approx (2 ulp) and the fp32 Horner
// steps the absolute error of Phi stays below 2.5e-7, i.e. |GELU error| < 2^-21 * |y|.
// gelu_scaled(y, h) = 2*h*GELU(y); h = 0.5 gives GELU itself, h = 0.5/s_out folds the output step.
__device__ __forceinline__ float gelu_scaled(float y, float h) {
    const float z = fminf(fabsf(y) * 0.70710678118654752440f, 4.0f);
    float q = -1.00217749e-04f;
    q = fmaf(q, z, 4.61550077e-04f);
    q = fmaf(q, z, 2.30229650e-03f);
    q = fmaf(q, z, -2.94525847e-02f);
    q = fmaf(q, z, 1.48963709e-01f);
    q = fmaf(q, z, 9.18328634e-01f);
    q = fmaf(q, z, 1.62791373e+00f);
    q = q * z;
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-q));
    const float erf_abs = 1.0f - e;
    const float t = copysignf(erf_abs, y);
    const float hy = h * y;
    return fmaf(hy, t, hy);
}
__device__ __forceinline__ float gelu_f32(float y) { return gelu_scaled(y, 0.5f); }

}  // namespace vitint
