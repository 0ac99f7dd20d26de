// a5: scale + row softmax + quantize (Eq. 3), one warp per row.
//
// HBM-bound: 4 bytes read and c/8 bytes written per element.  The row lives in
// registers (lane l owns columns 256*k + 8*l .. +7 of chunk k); the maximum and
// the normaliser are reduced with warp shuffles.
//
// Accuracy target: probabilities within 2 ulp of the exactly rounded softmax.
//   * t_j - max is formed exactly in fp64 (a rounded fp32 difference would already
//     cost |t_j - max| * 2^-24 of relative error after the exponential);
//   * exp(d) = 2^k * exp(r), k = rint(d*log2 e), r = d - k*ln2 reduced in fp64, then a
//     degree-7 Taylor polynomial in fp32 on |r| <= ln2/2 (truncation < 0.1 ulp);
//   * the normaliser is accumulated in fp64 and applied as one fp64 multiply.
#include <climits>

#include "common.cuh"

namespace vitint {

// exp(t - mx) for mx >= t, all in fp32 and integer instructions (no conversion instruction: those run at an eighth of
// the issue rate and used to bound this kernel).
//   * t - mx as an exact two-float sum (TwoSum), so nothing is lost when the two differ by more than a factor of two;
//   * k = rint((t - mx) * log2 e) by the 1.5*2^23 addition, which also leaves k as an integer in the mantissa;
//   * r = (t - mx) - k*ln2 with ln2 split so that k*ln2_hi is exact, the low parts folded in with one FMA;
//   * degree-7 Taylor polynomial on |r| <= ln2/2 (truncation < 0.1 ulp), then 2^k added to the exponent field.
// Results below 2^-125 (relative to the row's largest term, which is 1) are returned as 0: they lie in the range
// where the tolerance is the absolute 2^-126.
__device__ __forceinline__ float exp_reduced(float t, float mx) {
    const float sh = __fadd_rn(t, -mx);
    const float bv = __fadd_rn(sh, -t);
    const float sl = __fadd_rn(__fadd_rn(t, -__fadd_rn(sh, -bv)), __fadd_rn(-mx, -bv));     // sh + sl = t - mx exactly
    const float d = fmaxf(sh, -200.0f);
    const float m = __fmaf_rn(d, 1.44269504088896340736f, 12582912.0f);
    const float kf = __fadd_rn(m, -12582912.0f);
    const int k = __float_as_int(m) - 0x4B400000;
    const float rh = __fmaf_rn(-kf, 0.693145751953125f, d);                  // exact: ln2_hi has 15 significant bits
    const float rl = __fmaf_rn(-kf, 1.42860682030941723212e-6f, sl);         // ln2 - ln2_hi, and the low part of t - mx
    const float rf = __fadd_rn(rh, rl);
    float p = 1.0f / 5040.0f;
    p = fmaf(p, rf, 1.0f / 720.0f);
    p = fmaf(p, rf, 1.0f / 120.0f);
    p = fmaf(p, rf, 1.0f / 24.0f);
    p = fmaf(p, rf, 1.0f / 6.0f);
    p = fmaf(p, rf, 0.5f);
    p = fmaf(p, rf, 1.0f);
    p = fmaf(p, rf, 1.0f);
    // p lies in [0.70, 1.42]: for k >= -125 the product p * 2^k is normal and exact as an exponent addition
    return k >= -125 ? __int_as_float(k * 8388608 + __float_as_int(p)) : 0.0f;
}

template <int C, int NCH>
__global__ void __launch_bounds__(256)
softmax_quantize_kernel(const int32_t* __restrict__ s, int64_t rows, int cols, int64_t ld_s, float c, float p_step,
                        uint8_t* __restrict__ out, int64_t pitch, float* __restrict__ p_out, int64_t ld_p, float qp,
                        int vec_in, int vec_p) {
    grid_dependency_wait();        // inputs may come from the previous kernel of the stream
    grid_dependency_launch();
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int32_t* sr = s + row * ld_s;

    // Columns past the row's end take t = -inf.  Their exponential is exactly 0, so they add nothing to the row
    // sum and quantize to code 0 (the padding value) without any per-element masking further down.
    float t[NCH][8];
    float mx = -INFINITY;
#pragma unroll
    for (int k = 0; k < NCH; ++k) {
        const int col = k * 256 + lane * 8;
        if (vec_in && col + 8 <= ld_s) {
            // whole 32 bytes inside the row's storage (the leading dimension may exceed the column count)
            const int4 a = __ldg(reinterpret_cast<const int4*>(sr + col));
            const int4 b = __ldg(reinterpret_cast<const int4*>(sr + col) + 1);
            t[k][0] = (float)a.x * c; t[k][1] = (float)a.y * c; t[k][2] = (float)a.z * c; t[k][3] = (float)a.w * c;
            t[k][4] = (float)b.x * c; t[k][5] = (float)b.y * c; t[k][6] = (float)b.z * c; t[k][7] = (float)b.w * c;
            if (col + 8 > cols) {
#pragma unroll
                for (int i = 0; i < 8; ++i) if (col + i >= cols) t[k][i] = -INFINITY;
            }
        } else if (col < cols) {
#pragma unroll
            for (int i = 0; i < 8; ++i) t[k][i] = (col + i < cols) ? (float)__ldg(sr + col + i) * c : -INFINITY;
        } else {
            // lanes wholly past the row: nothing to load (kept apart so that a warp whose other lanes all took the
            // vector path does not walk the scalar one as well)
#pragma unroll
            for (int i = 0; i < 8; ++i) t[k][i] = -INFINITY;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) mx = fmaxf(mx, t[k][i]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));

    // two interleaved fp64 partial sums; a float enters as a double built from its bits with integer
    // multiply-adds (every term is zero or a positive normal float; a zero adds 2^-127, nothing beside the
    // row's largest term, which is 1)
    double z0 = 0.0, z1 = 0.0;
#pragma unroll
    for (int k = 0; k < NCH; ++k) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float e = exp_reduced(t[k][i], mx);
            t[k][i] = e;
            const uint32_t eb = __float_as_uint(e);
            uint32_t hi, lo;
            asm("mad.hi.u32 %0, %1, 536870912, 939524096;" : "=r"(hi) : "r"(eb));    // (eb >> 3) + 0x38000000
            asm("mul.lo.u32 %0, %1, 536870912;" : "=r"(lo) : "r"(eb));                // eb << 29
            const double ed = __hiloint2double((int)hi, (int)lo);
            if (i & 1) z1 += ed; else z0 += ed;
        }
    }
    double z = z0 + z1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    const double rz = 1.0 / z;
    const float rzh = (float)rz, rzl = (float)(rz - (double)(float)rz);   // 1/Z as two floats
    const Divisor dv = make_divisor(p_step);

    const int chunk_bytes = 32 * C;                                   // 256 codes
    const int n_out_chunks = (int)((pitch + chunk_bytes - 1) / chunk_bytes);
    for (int k = 0; k < n_out_chunks; ++k) {
        uint32_t w0 = 0, w1 = 0;
        if (k < NCH) {
            float p[8];
#pragma unroll
            for (int u = 0; u < NCH; ++u)
                if (u == k) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) p[i] = fmaf(t[u][i], rzh, t[u][i] * rzl);
                }
            const int col = k * 256 + lane * 8;
            if (p_out && col < cols) {
                float* pr = p_out + row * ld_p + col;
                if (vec_p && col + 8 <= cols) {
                    reinterpret_cast<float4*>(pr)[0] = make_float4(p[0], p[1], p[2], p[3]);
                    reinterpret_cast<float4*>(pr)[1] = make_float4(p[4], p[5], p[6], p[7]);
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) if (col + i < cols) pr[i] = p[i];
                }
            }
            // p >= 0, so only the upper clamp is needed; adding 1.5*2^23 rounds to nearest even and leaves the
            // (unsigned) code in the low mantissa bits, and the codes combine by shift-add without masking
            uint32_t cb[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) cb[i] = __float_as_uint(fminf(div_rn(p[i], dv), qp) + 12582912.0f);
            if (C == 8) {
                w0 = cb[0] + (cb[1] << 8) + (cb[2] << 16) + (cb[3] << 24) - 0x4B400000u * 0x01010101u;
                w1 = cb[4] + (cb[5] << 8) + (cb[6] << 16) + (cb[7] << 24) - 0x4B400000u * 0x01010101u;
            } else {
                uint32_t acc = cb[0];
#pragma unroll
                for (int i = 1; i < 8; ++i) acc += cb[i] << (C * i);
                uint32_t ones = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) ones += 1u << (C * i);
                w0 = acc - 0x4B400000u * ones;
                if (C == 2) w0 &= 0xFFFFu;
            }
        }
        uint8_t* orow = out + row * pitch;
        const int64_t off = (int64_t)k * chunk_bytes + lane * C;       // this lane's C bytes
        if (C == 8) {
            if (off + 8 <= pitch) *reinterpret_cast<uint2*>(orow + off) = make_uint2(w0, w1);
        } else if (C == 4) {
            if (off + 4 <= pitch) *reinterpret_cast<uint32_t*>(orow + off) = w0;
        } else {
            w0 |= __shfl_xor_sync(0xffffffffu, w0, 1) << 16;
            if ((lane & 1) == 0 && off + 4 <= pitch) *reinterpret_cast<uint32_t*>(orow + off) = w0;
        }
    }
}

template <int C>
static int launch_softmax(int nch, const int32_t* s, int64_t rows, int cols, int64_t ld_s, float c, float p_step,
                          uint8_t* out, int64_t pitch, float* p, int64_t ld_p, float qp, int vec_in, int vec_p,
                          cudaStream_t st) {
    const int warps = 8;
    dim3 grid((unsigned)((rows + warps - 1) / warps)), block(32 * warps);
    switch (nch) {
        case 1: launch_kernel(softmax_quantize_kernel<C, 1>, dim3(grid), dim3(block), 0, st, s, rows, cols, ld_s, c, p_step, out, pitch, p, ld_p, qp, vec_in, vec_p); break;
        case 2: launch_kernel(softmax_quantize_kernel<C, 2>, dim3(grid), dim3(block), 0, st, s, rows, cols, ld_s, c, p_step, out, pitch, p, ld_p, qp, vec_in, vec_p); break;
        case 3: launch_kernel(softmax_quantize_kernel<C, 3>, dim3(grid), dim3(block), 0, st, s, rows, cols, ld_s, c, p_step, out, pitch, p, ld_p, qp, vec_in, vec_p); break;
        case 4: launch_kernel(softmax_quantize_kernel<C, 4>, dim3(grid), dim3(block), 0, st, s, rows, cols, ld_s, c, p_step, out, pitch, p, ld_p, qp, vec_in, vec_p); break;
        default: return VITINT_ERR_UNSUPPORTED;
    }
    return cuda_status(cudaGetLastError());
}

// Shift-based softmax with the division-free quantizer (Eq. 4 and the comparator of Section IV-B),
// one warp per row.  Integer and single-rounding fp32 operations only, so the codes are unique:
//   z = fl32(float(S) * c2);  f = floor(z);  r = z - f;  M = (1 + r) * 2^23 as an integer  (2^r ~ 1 + r)
//   E = M << (30 + f - max_j f)   (right shift, dropping bits, when the count is negative)
//   Sigma = sum_j E (exact, 64-bit);  code = #{ k in 1..Qp : float(E) > fl32(fl32((k - 1/2) * step) * float(Sigma)) }
// The thresholds grow with k, so the count is found by a bit-by-bit search (one comparison per code bit).
// Explicit _rn intrinsics keep the compiler from contracting a multiply and a subtract into one FMA.
template <int C, int NCH>
__global__ void __launch_bounds__(256)
softmax_shift_quantize_kernel(const int32_t* __restrict__ s, int64_t rows, int cols, int64_t ld_s, float c2,
                              float p_step, uint8_t* __restrict__ out, int64_t pitch, int code_bits, int vec_in) {
    grid_dependency_wait();        // inputs may come from the previous kernel of the stream
    grid_dependency_launch();
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int32_t* sr = s + row * ld_s;
    int fi[NCH][8];
    uint32_t mant[NCH][8];
    int m = INT_MIN;
#pragma unroll
    for (int k = 0; k < NCH; ++k) {
        const int col = k * 256 + lane * 8;
        int sv[8];
        if (vec_in && col + 8 <= ld_s) {
            // whole 32 bytes inside the row's storage; values past the last column are masked below
            const int4 a = __ldg(reinterpret_cast<const int4*>(sr + col));
            const int4 b = __ldg(reinterpret_cast<const int4*>(sr + col) + 1);
            sv[0] = a.x; sv[1] = a.y; sv[2] = a.z; sv[3] = a.w; sv[4] = b.x; sv[5] = b.y; sv[6] = b.z; sv[7] = b.w;
        } else if (col < cols) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sv[i] = (col + i < cols) ? __ldg(sr + col + i) : 0;
        } else {
            // lanes wholly past the row: nothing to load (kept apart so that a warp whose other lanes all took the
            // vector path does not walk the scalar one as well)
#pragma unroll
            for (int i = 0; i < 8; ++i) sv[i] = 0;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float z = __fmul_rn((float)sv[i], c2);
            const float fl = floorf(z);
            const float res = __fsub_rn(z, fl);
            mant[k][i] = (uint32_t)__fmul_rn(__fadd_rn(1.0f, res), 8388608.0f);
            fi[k][i] = (int)fl;
            if (col + i < cols) m = max(m, fi[k][i]);
            else mant[k][i] = 0u;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));

    unsigned long long sigma = 0ull;
#pragma unroll
    for (int k = 0; k < NCH; ++k) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            // shift count 30 + f - m <= 30; far negative counts shift everything out
            int sh = 30 + fi[k][i] - m;
            sh = mant[k][i] ? max(sh, -63) : 0;
            const unsigned long long mj = (unsigned long long)mant[k][i];
            const unsigned long long e = sh >= 0 ? (mj << sh) : (mj >> (-sh));
            sigma += e;
            // keep E as (high, low) in the two register arrays that are free now
            fi[k][i] = (int)(uint32_t)(e >> 32);
            mant[k][i] = (uint32_t)e;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sigma += __shfl_xor_sync(0xffffffffu, sigma, o);
    const float sig_f = __ull2float_rn(sigma);
    // The comparator references fl32(fl32((t - 1/2) * step) * Sigma), t = 1 .. 2^bits - 1, depend on the row only:
    // formed once per row and kept in registers (entries past the code range stay +inf and are never exceeded).
    float thr[16];
#pragma unroll
    for (int tcode = 1; tcode < 16; ++tcode)
        thr[tcode] = tcode < (1 << code_bits) ? __fmul_rn(__fmul_rn(__fsub_rn((float)tcode, 0.5f), p_step), sig_f) : INFINITY;

    constexpr uint32_t MASK = (1u << C) - 1u;
    const int chunk_bytes = 32 * C;
    const int n_out_chunks = (int)((pitch + chunk_bytes - 1) / chunk_bytes);
    for (int k = 0; k < n_out_chunks; ++k) {
        uint32_t w0 = 0, w1 = 0;
        if (k < NCH) {
#pragma unroll
            for (int u = 0; u < NCH; ++u)
                if (u == k) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const unsigned long long e = ((unsigned long long)(uint32_t)fi[u][i] << 32) | mant[u][i];
                        const float e_f = __ull2float_rn(e);
                        // the references ascend, so the number exceeded is found bit by bit; with the candidates in
                        // registers each step is one comparison and a halving of the candidate list by selects
                        uint32_t code = 0;
                        if (code_bits > 4) {
                            // wide codes: the references are formed on the fly, one comparison per code bit
                            for (int b = code_bits - 1; b >= 0; --b) {
                                const uint32_t tc = code | (1u << b);
                                const float th = __fmul_rn(__fmul_rn(__fsub_rn((float)tc, 0.5f), p_step), sig_f);
                                code = (e_f > th) ? tc : code;
                            }
                        } else {
                        float cand[7];
                        const bool p3 = e_f > thr[8];
#pragma unroll
                        for (int j = 0; j < 7; ++j) cand[j] = p3 ? thr[9 + j] : thr[1 + j];
                        const bool p2 = e_f > cand[3];
#pragma unroll
                        for (int j = 0; j < 3; ++j) cand[j] = p2 ? cand[4 + j] : cand[j];
                        const bool p1 = e_f > cand[1];
                        cand[0] = p1 ? cand[2] : cand[0];
                        const bool p0 = e_f > cand[0];
                        code = (p3 ? 8u : 0u) + (p2 ? 4u : 0u) + (p1 ? 2u : 0u) + (p0 ? 1u : 0u);
                        }
                        const int col = k * 256 + lane * 8 + i;
                        if (col >= cols) code = 0;
                        if (C == 8) { if (i < 4) w0 |= code << (8 * i); else w1 |= code << (8 * (i - 4)); }
                        else w0 |= (code & MASK) << (C * i);
                    }
                }
        }
        uint8_t* orow = out + row * pitch;
        const int64_t off = (int64_t)k * chunk_bytes + lane * C;
        if (C == 8) {
            if (off + 8 <= pitch) *reinterpret_cast<uint2*>(orow + off) = make_uint2(w0, w1);
        } else if (C == 4) {
            if (off + 4 <= pitch) *reinterpret_cast<uint32_t*>(orow + off) = w0;
        } else {
            w0 |= __shfl_xor_sync(0xffffffffu, w0, 1) << 16;
            if ((lane & 1) == 0 && off + 4 <= pitch) *reinterpret_cast<uint32_t*>(orow + off) = w0;
        }
    }
}

template <int C>
static int launch_softmax_shift(int nch, const int32_t* s, int64_t rows, int cols, int64_t ld_s, float c2, float p_step,
                                uint8_t* out, int64_t pitch, int code_bits, int vec_in, cudaStream_t st) {
    const int warps = 8;
    dim3 grid((unsigned)((rows + warps - 1) / warps)), block(32 * warps);
    switch (nch) {
        case 1: launch_kernel(softmax_shift_quantize_kernel<C, 1>, dim3(grid), dim3(block), 0, st, s, rows, cols, ld_s, c2, p_step, out, pitch, code_bits, vec_in); break;
        case 2: launch_kernel(softmax_shift_quantize_kernel<C, 2>, dim3(grid), dim3(block), 0, st, s, rows, cols, ld_s, c2, p_step, out, pitch, code_bits, vec_in); break;
        case 3: launch_kernel(softmax_shift_quantize_kernel<C, 3>, dim3(grid), dim3(block), 0, st, s, rows, cols, ld_s, c2, p_step, out, pitch, code_bits, vec_in); break;
        case 4: launch_kernel(softmax_shift_quantize_kernel<C, 4>, dim3(grid), dim3(block), 0, st, s, rows, cols, ld_s, c2, p_step, out, pitch, code_bits, vec_in); break;
        default: return VITINT_ERR_UNSUPPORTED;
    }
    return cuda_status(cudaGetLastError());
}

}  // namespace vitint

using namespace vitint;

extern "C" int vitint_softmax_quantize(const int32_t* s, int64_t rows, int32_t cols, int64_t ld_s, float c,
                                       float p_step, const vitint_codes* p_out, float* p_f32, int64_t ld_p,
                                       void* stream) {
    if (!s || !p_out) return VITINT_ERR_INVALID_ARG;
    if (int rc = check_codes(p_out)) return rc;
    if (rows <= 0 || cols <= 0 || ld_s < cols || p_out->rows != rows || p_out->cols != cols || p_out->is_signed)
        return VITINT_ERR_INVALID_ARG;
    if (!(p_step > 0.0f && p_step < INFINITY) || !(c == c) || fabsf(c) == INFINITY) return VITINT_ERR_INVALID_ARG;
    if (p_f32 && ld_p < cols) return VITINT_ERR_INVALID_ARG;
    if (cols > 1024) return VITINT_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(s) & 3u) != 0) return VITINT_ERR_ALIGNMENT;
    const int cb = codes_container(p_out);
    int qn, qp;
    code_range(p_out->bits, 0, &qn, &qp);
    const int nch = (cols + 255) / 256;
    const int vec_in = (aligned16(s) && ld_s % 4 == 0) ? 1 : 0;
    const int vec_p = (p_f32 && aligned16(p_f32) && ld_p % 4 == 0) ? 1 : 0;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* o = (uint8_t*)p_out->data;
    if (cb == 2) return launch_softmax<2>(nch, s, rows, cols, ld_s, c, p_step, o, p_out->pitch_bytes, p_f32, ld_p, (float)qp, vec_in, vec_p, st);
    if (cb == 4) return launch_softmax<4>(nch, s, rows, cols, ld_s, c, p_step, o, p_out->pitch_bytes, p_f32, ld_p, (float)qp, vec_in, vec_p, st);
    return launch_softmax<8>(nch, s, rows, cols, ld_s, c, p_step, o, p_out->pitch_bytes, p_f32, ld_p, (float)qp, vec_in, vec_p, st);
}

extern "C" int vitint_softmax_shift_quantize(const int32_t* s, int64_t rows, int32_t cols, int64_t ld_s, float c2,
                                             float p_step, const vitint_codes* p_out, void* stream) {
    if (!s || !p_out) return VITINT_ERR_INVALID_ARG;
    if (int rc = check_codes(p_out)) return rc;
    if (rows <= 0 || cols <= 0 || ld_s < cols || p_out->rows != rows || p_out->cols != cols || p_out->is_signed)
        return VITINT_ERR_INVALID_ARG;
    if (!(p_step > 0.0f && p_step < INFINITY) || !(c2 == c2) || fabsf(c2) == INFINITY) return VITINT_ERR_INVALID_ARG;
    if (cols > 1024) return VITINT_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(s) & 3u) != 0) return VITINT_ERR_ALIGNMENT;
    const int cb = codes_container(p_out);
    const int nch = (cols + 255) / 256;
    const int vec_in = (aligned16(s) && ld_s % 4 == 0) ? 1 : 0;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* o = (uint8_t*)p_out->data;
    if (cb == 2) return launch_softmax_shift<2>(nch, s, rows, cols, ld_s, c2, p_step, o, p_out->pitch_bytes, p_out->bits, vec_in, st);
    if (cb == 4) return launch_softmax_shift<4>(nch, s, rows, cols, ld_s, c2, p_step, o, p_out->pitch_bytes, p_out->bits, vec_in, st);
    return launch_softmax_shift<8>(nch, s, rows, cols, ld_s, c2, p_step, o, p_out->pitch_bytes, p_out->bits, vec_in, st);
}
