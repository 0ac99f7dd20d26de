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

// ---- programmatic dependent launch ---------------------------------------------------------
// Every kernel of the library is launched with programmatic stream serialization: its CTAs may
// be scheduled while the previous kernel of the stream is still draining, run their set-up
// (barriers, tensor memory, descriptor prefetch) and then block in grid_dependency_wait() until
// the previous kernel has completed and its writes are visible.  Nothing that another kernel
// may have produced is read, and nothing is written, before that wait.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

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
// whenever b's significand is not all ones and nothing overflows or underflows on the way.
// The quantizers only need the quotient where it can still decide a level, so they first clamp the
// dividend to [lo, hi] = [(Qn - 1) b, (Qp + 1) b] (clamp_dividend): a quotient beyond Qn - 1 / Qp + 1
// clamps to the same end level as the true one, +-inf lands on the end levels like the IEEE quotient
// does, NaN becomes lo (level Qn, as the host rule "not >= Qn" gives), and q0 stays finite.  Steps
// outside [2^-100, 2^100] (where b*(Qp+1), 1/b or the remainder could leave the normal range) take
// the IEEE division instead.
struct Divisor {
    float b, r;
    float lo, hi;   // dividend clamp
    int exact;      // 0: use the IEEE division instead
};
__device__ __forceinline__ Divisor make_divisor(float b, float qn = -128.0f, float qp = 255.0f) {
    Divisor d;
    d.b = b;
    d.r = __frcp_rn(b);
    d.lo = (qn - 1.0f) * b;
    d.hi = (qp + 1.0f) * b;
    const bool in_range = b >= 7.8886090522101181e-31f && b <= 1.2676506002282294e30f;    // 2^-100 .. 2^100
    d.exact = (in_range && (__float_as_uint(b) & 0x007FFFFFu) != 0x007FFFFFu) ? 1 : 0;
    return d;
}
__device__ __forceinline__ float clamp_dividend(float a, const Divisor& d) {
    return fminf(fmaxf(a, d.lo), d.hi);          // NaN -> lo
}
// Straight-line form for inner loops; valid only when d.exact (callers test that once, outside
// the loop, because a branch per element would serialise the otherwise independent elements)
// and for dividends inside [d.lo, d.hi].
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

// ---- packed fp32 pairs ---------------------------------------------------------------------
// sm_100 issues add / mul / fma on two fp32 values held in a 64-bit register pair as ONE
// instruction (f32x2); each half is the IEEE round-to-nearest result of the scalar operation, so
// pairing elements changes no bit of the outcome and halves the issue slots of an
// instruction-bound element-wise stage.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 f2_pack(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2 f2_dup(float v) { return f2_pack(v, v); }
__device__ __forceinline__ void f2_unpack(f32x2 r, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r));
}
__device__ __forceinline__ f32x2 f2_fma(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 f2_mul(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 f2_add(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// GELU(y) = y * Phi(y) = 0.5*y*(1 + erf(y/sqrt 2)), with erf from
//   erf(z) = sign(z) * (1 - 2^(-q(|z|))),   q(z) = -log2(erfc(z)) ~ z*(c0 + c1 z + ... + c6 z^6)
// on |z| <= 4 (beyond that erf is 1 to 2e-8).  The coefficients are a weighted minimax fit
// (max |erf error| 7.8e-8 in exact arithmetic); with ex2.approx (2 ulp) and the fp32 Horner
// steps the absolute error of Phi stays below 2.5e-7, i.e. |GELU error| < 2^-21 * |y|.
// The polynomial runs in t = z/4 (coefficients scaled by exact powers of four), so the clamp
// of z to [0, 4] is the saturate modifier of the multiply that forms t.
__device__ __forceinline__ float gelu_erfc_term(float y) {               // 2^(-q(|y|/sqrt 2)) = erfc(|y|/sqrt 2)
    const float t = __saturatef(fabsf(y) * 0.17677669529663688110f);     // min(|y|/sqrt 2, 4) / 4
    float q = -1.00217749e-04f * 16384.0f;
    q = fmaf(q, t, 4.61550077e-04f * 4096.0f);
    q = fmaf(q, t, 2.30229650e-03f * 1024.0f);
    q = fmaf(q, t, -2.94525847e-02f * 256.0f);
    q = fmaf(q, t, 1.48963709e-01f * 64.0f);
    q = fmaf(q, t, 9.18328634e-01f * 16.0f);
    q = fmaf(q, t, 1.62791373e+00f * 4.0f);
    q = q * t;
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-q));
    return e;
}
// The same term for two elements: the Horner steps run as packed pairs.
__device__ __forceinline__ void gelu_erfc_term2(float y0, float y1, float& e0, float& e1) {
    const f32x2 t = f2_pack(__saturatef(fabsf(y0) * 0.17677669529663688110f),
                            __saturatef(fabsf(y1) * 0.17677669529663688110f));
    f32x2 q = f2_dup(-1.00217749e-04f * 16384.0f);
    q = f2_fma(q, t, f2_dup(4.61550077e-04f * 4096.0f));
    q = f2_fma(q, t, f2_dup(2.30229650e-03f * 1024.0f));
    q = f2_fma(q, t, f2_dup(-2.94525847e-02f * 256.0f));
    q = f2_fma(q, t, f2_dup(1.48963709e-01f * 64.0f));
    q = f2_fma(q, t, f2_dup(9.18328634e-01f * 16.0f));
    q = f2_fma(q, t, f2_dup(1.62791373e+00f * 4.0f));
    q = f2_mul(q, t);
    float q0, q1;
    f2_unpack(q, q0, q1);
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(-q0));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(-q1));
}
// gelu_scaled(y, h) = 2*h*GELU(y); h = 0.5 gives GELU itself, h = 0.5/s_out folds the output step.
// With w = h*y:  w*(1 + erf) = (w + |w|) - |w|*erfc, one rounding after an exact first term.
__device__ __forceinline__ float gelu_scaled(float y, float h) {
    const float e = gelu_erfc_term(y);
    const float w = h * y;
    return fmaf(-fabsf(w), e, w + fabsf(w));
}
// The same value clamped to [0, 1] by the saturate modifier of the last FMA (NaN -> 0).
__device__ __forceinline__ float gelu_scaled_unit(float y, float h) {
    const float e = gelu_erfc_term(y);
    const float w = h * y;
    return __saturatef(fmaf(-fabsf(w), e, w + fabsf(w)));
}
__device__ __forceinline__ float gelu_f32(float y) { return gelu_scaled(y, 0.5f); }

}  // namespace vitint
