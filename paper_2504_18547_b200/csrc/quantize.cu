// a1: quantize + pack, and the LayerNorm + quantize glue.  Both are streaming,
// HBM-bound kernels: 4 + c/8 bytes per element (c = container bits).
#include "common.cuh"

namespace vitint {

// One thread produces one 32-bit word of packed output = 32/C consecutive codes.
// Threads of a warp cover consecutive words of one row, so a warp reads
// 32 * (32/C) * 4 contiguous bytes and writes 128 contiguous bytes.
template <int C>
__global__ void __launch_bounds__(256)
quantize_pack_kernel(const float* __restrict__ x, int64_t rows, int64_t cols, int64_t ldx, float step,
                     const float* __restrict__ row_steps, uint8_t* __restrict__ out, int64_t pitch,
                     int words_per_row, float qn, float qp, int vec_ok) {
    grid_dependency_wait();        // inputs may come from the previous kernel of the stream
    grid_dependency_launch();
    constexpr int E = 32 / C;  // codes per word
    const int w = blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= words_per_row) return;
    const int64_t col0 = (int64_t)w * E;
    for (int64_t row = (int64_t)blockIdx.y * blockDim.y + threadIdx.y; row < rows;
         row += (int64_t)gridDim.y * blockDim.y) {
        const Divisor dv = make_divisor(row_steps ? row_steps[row] : step, qn, qp);
        const float* xr = x + row * ldx + col0;
        float v[E];
        if (vec_ok && col0 + E <= cols) {
#pragma unroll
            for (int i = 0; i < E / 4; ++i) {
                const float4 f = __ldg(reinterpret_cast<const float4*>(xr) + i);
                v[4 * i + 0] = f.x; v[4 * i + 1] = f.y; v[4 * i + 2] = f.z; v[4 * i + 3] = f.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < E; ++i) v[i] = (col0 + i < cols) ? __ldg(xr + i) : 0.0f;
        }
        uint32_t word = 0;
        if (dv.exact) {
#pragma unroll
            for (int i = 0; i < E; ++i)
                word |= (round_clamp_bits(div_rn_exact(clamp_dividend(v[i], dv), dv), qn, qp) & ((1u << C) - 1u)) << (C * i);
        } else {
#pragma unroll
            for (int i = 0; i < E; ++i)
                word |= (round_clamp_bits(__fdiv_rn(v[i], dv.b), qn, qp) & ((1u << C) - 1u)) << (C * i);
        }
        *reinterpret_cast<uint32_t*>(out + row * pitch + (int64_t)w * 4) = word;
    }
}

// One warp per row; the row stays in registers between the statistics and the
// normalisation.  Lane l owns float4 number v*32 + l of the row, v < NV.
// All per-element arithmetic is fp32 on the FMA pipe (no conversions); the corrected
// two-pass mean keeps the result inside a few ulp of the exact normalisation.
// FULL: the row is exactly NV*128 columns and no fp32 copy is written, so no access needs a guard (the guards
// otherwise become branches around every vector: a third of the instructions at 768 columns).
template <int C, int NV, bool FULL>
__global__ void __launch_bounds__(128)
layernorm_quantize_kernel(const float* __restrict__ x, int64_t rows, int cols, int64_t ldx,
                          const float* __restrict__ gamma, const float* __restrict__ beta, float eps, float step,
                          uint8_t* __restrict__ out, int64_t pitch, float* __restrict__ y_out, int64_t ld_y,
                          float qn, float qp) {
    grid_dependency_wait();        // inputs may come from the previous kernel of the stream
    grid_dependency_launch();
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const float* xr = x + row * ldx;
    // The row is held as packed pairs: adds, multiplies and fused multiply-adds below run two elements per
    // instruction (each half is the scalar IEEE result), which is what this issue-bound kernel needs.
    f32x2 f[NV][2];
    f32x2 sum2 = f2_dup(0.0f);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int col = (v * 32 + lane) * 4;
        const float4 t = (FULL || col < cols) ? __ldg(reinterpret_cast<const float4*>(xr + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
        f[v][0] = f2_pack(t.x, t.y);
        f[v][1] = f2_pack(t.z, t.w);
        sum2 = f2_add(sum2, f2_add(f[v][0], f[v][1]));
    }
    float s_lo, s_hi;
    f2_unpack(sum2, s_lo, s_hi);
    float sum = s_lo + s_hi;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float inv_n = 1.0f / (float)cols;
    // Centre on the fp32 estimate of the mean; one more pass gives both the mean of the residuals (which carries
    // the estimate's rounding error even when |mean| >> sigma) and their sum of squares.  The variance is
    // sum(d^2)/n - corr^2 with corr the residual mean: exact algebra, and corr is a rounding-level quantity.
    const float mean0 = sum * inv_n;
    const f32x2 nmean2 = f2_dup(-mean0);
    f32x2 rs2 = f2_dup(0.0f), m22 = f2_dup(0.0f);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int col = (v * 32 + lane) * 4;
        if (FULL || col < cols) {
            f[v][0] = f2_add(f[v][0], nmean2);
            f[v][1] = f2_add(f[v][1], nmean2);
            rs2 = f2_add(rs2, f2_add(f[v][0], f[v][1]));
            m22 = f2_fma(f[v][0], f[v][0], m22);
            m22 = f2_fma(f[v][1], f[v][1], m22);
        }
    }
    float r_lo, r_hi, q_lo, q_hi;
    f2_unpack(rs2, r_lo, r_hi);
    f2_unpack(m22, q_lo, q_hi);
    float rsum = r_lo + r_hi, m2 = q_lo + q_hi;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        rsum += __shfl_xor_sync(0xffffffffu, rsum, o);
        m2 += __shfl_xor_sync(0xffffffffu, m2, o);
    }
    const float corr = rsum * inv_n;
    const f32x2 ncorr2 = f2_dup(-corr);
    // 1/sqrt(var + eps): hardware estimate plus one Newton step (about 1 ulp), all in fp32
    const float var = fmaf(m2, inv_n, eps) - corr * corr;
    float rstd = rsqrtf(var);
    rstd = rstd * fmaf(-0.5f * var, rstd * rstd, 1.5f);
    // y / step as y * RN(1/step): at most 1.5 ulp from the exact quotient, far inside the tolerance
    // that the fp32 normalisation itself is granted, and one instruction instead of three
    const float rstep = __frcp_rn(step);
    const bool sgn = qn < 0.0f;
    const float magic = 12582912.0f + (sgn ? (float)(1 << (C - 1)) : 0.0f);
    const uint32_t top = 1u << (C - 1);
    const uint32_t flip = sgn ? (top | (top << C) | (top << (2 * C)) | (top << (3 * C))) : 0u;   // offset binary -> two's complement

    constexpr int LANES_PER_WORD = 8 / C;          // 4 codes per lane per v -> 4*C bits
    const int words_per_row = (int)(pitch >> 2);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        uint32_t bits = 0;
        const int col = (v * 32 + lane) * 4;
        if (FULL || col < cols) {
            const float4 g = __ldg(reinterpret_cast<const float4*>(gamma + col));
            const float4 b = __ldg(reinterpret_cast<const float4*>(beta + col));
            const f32x2 rstd2 = f2_dup(rstd), rstep2 = f2_dup(rstep), magic2 = f2_dup(magic);
            const f32x2 y01 = f2_fma(f2_mul(f2_add(f[v][0], ncorr2), rstd2), f2_pack(g.x, g.y), f2_pack(b.x, b.y));
            const f32x2 y23 = f2_fma(f2_mul(f2_add(f[v][1], ncorr2), rstd2), f2_pack(g.z, g.w), f2_pack(b.z, b.w));
            float4 y;
            f2_unpack(y01, y.x, y.y);
            f2_unpack(y23, y.z, y.w);
            if (!FULL && y_out) *reinterpret_cast<float4*>(y_out + row * ld_y + col) = y;
            // clamp, then add 1.5*2^23 (+ 2^(C-1) for signed codes): the low mantissa bits hold the code in
            // offset binary, so the four codes combine by shift-add without masking
            float u0, u1, u2, u3;
            f2_unpack(f2_mul(y01, rstep2), u0, u1);
            f2_unpack(f2_mul(y23, rstep2), u2, u3);
            float cx, cy, cz, cw;
            f2_unpack(f2_add(f2_pack(fminf(fmaxf(u0, qn), qp), fminf(fmaxf(u1, qn), qp)), magic2), cx, cy);
            f2_unpack(f2_add(f2_pack(fminf(fmaxf(u2, qn), qp), fminf(fmaxf(u3, qn), qp)), magic2), cz, cw);
            bits = (__float_as_uint(cx) + (__float_as_uint(cy) << C) + (__float_as_uint(cz) << (2 * C)) +
                    (__float_as_uint(cw) << (3 * C)) - 0x4B400000u * (1u + (1u << C) + (1u << (2 * C)) + (1u << (3 * C))));
            bits = (bits ^ flip) & (C == 8 ? 0xFFFFFFFFu : ((1u << ((4 * C) & 31)) - 1u));
        }
        // gather 8/C neighbouring lanes into one 32-bit word
        if (C == 4) {
            bits |= __shfl_xor_sync(0xffffffffu, bits, 1) << 16;
        } else if (C == 2) {
            bits |= __shfl_xor_sync(0xffffffffu, bits, 1) << 8;
            bits |= __shfl_xor_sync(0xffffffffu, bits, 2) << 16;
        }
        const int word = (v * 32 + lane) / LANES_PER_WORD;
        if ((lane % LANES_PER_WORD) == 0 && (FULL || word < words_per_row))
            *reinterpret_cast<uint32_t*>(out + row * pitch + (int64_t)word * 4) = bits;
    }
    // row padding beyond the columns the loop above covers
    for (int word = NV * 32 / LANES_PER_WORD + lane; word < words_per_row; word += 32)
        *reinterpret_cast<uint32_t*>(out + row * pitch + (int64_t)word * 4) = 0u;
}

// One thread expands one 32-bit word of packed codes (32/C codes) into as many bytes.
template <int C>
__global__ void __launch_bounds__(256)
widen_kernel(const uint8_t* __restrict__ in, int64_t in_pitch, uint8_t* __restrict__ out, int64_t out_pitch,
             int64_t rows, int words_in, int is_signed) {
    grid_dependency_wait();        // inputs may come from the previous kernel of the stream
    grid_dependency_launch();
    constexpr int E = 32 / C;
    const int w = blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t row = blockIdx.y; row < rows; row += gridDim.y) {
        if ((int64_t)w * E >= out_pitch) continue;
        const uint32_t word = (w < words_in) ? *reinterpret_cast<const uint32_t*>(in + row * in_pitch + (int64_t)w * 4) : 0u;
        uint32_t o[E / 4];
#pragma unroll
        for (int i = 0; i < E / 4; ++i) o[i] = 0;
#pragma unroll
        for (int i = 0; i < E; ++i) {
            int v = (int)((word >> (C * i)) & ((1u << C) - 1u));
            if (is_signed && (v & (1 << (C - 1)))) v -= (1 << C);
            o[i >> 2] |= ((uint32_t)v & 0xFFu) << (8 * (i & 3));
        }
        uint8_t* dst = out + row * out_pitch + (int64_t)w * E;
#pragma unroll
        for (int i = 0; i < E / 4; ++i)
            if ((int64_t)w * E + 4 * i + 4 <= out_pitch) reinterpret_cast<uint32_t*>(dst)[i] = o[i];
    }
}

template <int C>
static int launch_ln(int nv, const float* x, int64_t rows, int cols, int64_t ldx, const float* gamma,
                     const float* beta, float eps, float step, uint8_t* out, int64_t pitch, float* y, int64_t ld_y,
                     float qn, float qp, cudaStream_t st) {
    const int warps = 4;       // four rows per block: measured best (8: +1 us per call at 25,216 x 768; 16: +3 us)
    dim3 grid((unsigned)((rows + warps - 1) / warps)), block(32 * warps);
    const bool full = cols == nv * 128 && y == nullptr;
#define VITINT_LN_CASE(NVV)                                                                                     \
    case NVV:                                                                                                   \
        if (full)                                                                                               \
            launch_kernel(layernorm_quantize_kernel<C, NVV, true>, dim3(grid), dim3(block), 0, st, x, rows, cols, ldx, gamma, beta,    \
                          eps, step, out, pitch, y, ld_y, qn, qp);                                              \
        else                                                                                                    \
            launch_kernel(layernorm_quantize_kernel<C, NVV, false>, dim3(grid), dim3(block), 0, st, x, rows, cols, ldx, gamma, beta,   \
                          eps, step, out, pitch, y, ld_y, qn, qp);                                              \
        break;
    switch (nv) {
        VITINT_LN_CASE(1) VITINT_LN_CASE(2) VITINT_LN_CASE(3) VITINT_LN_CASE(4) VITINT_LN_CASE(6)
        VITINT_LN_CASE(8) VITINT_LN_CASE(12) VITINT_LN_CASE(16)
        default: return VITINT_ERR_UNSUPPORTED;
    }
#undef VITINT_LN_CASE
    return cuda_status(cudaGetLastError());
}

}  // namespace vitint

using namespace vitint;

extern "C" int vitint_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx, float step,
                               const float* row_steps, const vitint_codes* out, void* stream) {
    if (!x || !out) return VITINT_ERR_INVALID_ARG;
    if (int rc = check_codes(out)) return rc;
    if (rows <= 0 || cols <= 0 || ldx < cols || out->rows != rows || out->cols != cols) return VITINT_ERR_INVALID_ARG;
    if (!row_steps && !(step > 0.0f && step < INFINITY)) return VITINT_ERR_INVALID_ARG;
    const int c = codes_container(out);
    int qn, qp;
    code_range(out->bits, out->is_signed, &qn, &qp);
    const int words = (int)(out->pitch_bytes / 4);
    const int vec_ok = ((reinterpret_cast<uintptr_t>(x) & 15u) == 0 && (ldx % 4) == 0) ? 1 : 0;
    int bx = 32;
    while (bx < 128 && bx < words) bx *= 2;
    const int by = 256 / bx;
    dim3 block(bx, by);
    int64_t gy = (rows + by - 1) / by;
    if (gy > 16384) gy = 16384;
    dim3 grid((words + bx - 1) / bx, (unsigned)gy);
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* o = (uint8_t*)out->data;
    if (c == 2)
        launch_kernel(quantize_pack_kernel<2>, dim3(grid), dim3(block), 0, st, x, rows, cols, ldx, step, row_steps, o, out->pitch_bytes,
                                                        words, (float)qn, (float)qp, vec_ok);
    else if (c == 4)
        launch_kernel(quantize_pack_kernel<4>, dim3(grid), dim3(block), 0, st, x, rows, cols, ldx, step, row_steps, o, out->pitch_bytes,
                                                        words, (float)qn, (float)qp, vec_ok);
    else
        launch_kernel(quantize_pack_kernel<8>, dim3(grid), dim3(block), 0, st, x, rows, cols, ldx, step, row_steps, o, out->pitch_bytes,
                                                        words, (float)qn, (float)qp, vec_ok);
    return cuda_status(cudaGetLastError());
}

extern "C" int vitint_widen(const vitint_codes* in, const vitint_codes* out, void* stream) {
    if (int rc = check_codes(in)) return rc;
    if (int rc = check_codes(out)) return rc;
    if (codes_container(out) != 8 || codes_container(in) == 8 || out->bits != in->bits || in->rows != out->rows ||
        in->cols != out->cols || in->is_signed != out->is_signed)
        return VITINT_ERR_INVALID_ARG;
    const int c = codes_container(in);
    const int e = 32 / c;
    const int words_in = (int)(in->pitch_bytes / 4);
    const int words_out = (int)((out->pitch_bytes + e - 1) / e);    // threads needed to cover the output pitch
    const int threads = words_out > words_in ? words_out : words_in;
    dim3 block(128), grid((threads + 127) / 128, (unsigned)(in->rows < 32768 ? in->rows : 32768));
    cudaStream_t st = (cudaStream_t)stream;
    if (c == 2)
        launch_kernel(widen_kernel<2>, dim3(grid), dim3(block), 0, st, (const uint8_t*)in->data, in->pitch_bytes, (uint8_t*)out->data,
                                                out->pitch_bytes, in->rows, words_in, in->is_signed);
    else
        launch_kernel(widen_kernel<4>, dim3(grid), dim3(block), 0, st, (const uint8_t*)in->data, in->pitch_bytes, (uint8_t*)out->data,
                                                out->pitch_bytes, in->rows, words_in, in->is_signed);
    return cuda_status(cudaGetLastError());
}

extern "C" int vitint_layernorm_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx, const float* gamma,
                                         const float* beta, float eps, float step, const vitint_codes* out,
                                         float* y_f32, int64_t ld_y, void* stream) {
    if (!x || !gamma || !beta || !out) return VITINT_ERR_INVALID_ARG;
    if (int rc = check_codes(out)) return rc;
    if (rows <= 0 || cols <= 0 || ldx < cols || out->rows != rows || out->cols != cols) return VITINT_ERR_INVALID_ARG;
    if (!(step > 0.0f && step < INFINITY) || !(eps >= 0.0f)) return VITINT_ERR_INVALID_ARG;
    if (cols % 4 != 0 || cols > 2048) return VITINT_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(gamma) || !aligned16(beta) || ldx % 4 != 0) return VITINT_ERR_ALIGNMENT;
    if (y_f32 && (!aligned16(y_f32) || ld_y % 4 != 0 || ld_y < cols)) return VITINT_ERR_ALIGNMENT;
    const int c = codes_container(out);
    int qn, qp;
    code_range(out->bits, out->is_signed, &qn, &qp);
    int nv = (int)((cols + 127) / 128);
    const int sizes[] = {1, 2, 3, 4, 6, 8, 12, 16};
    for (int s : sizes) if (s >= nv) { nv = s; break; }
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* o = (uint8_t*)out->data;
    if (c == 2) return launch_ln<2>(nv, x, rows, (int)cols, ldx, gamma, beta, eps, step, o, out->pitch_bytes, y_f32, ld_y, (float)qn, (float)qp, st);
    if (c == 4) return launch_ln<4>(nv, x, rows, (int)cols, ldx, gamma, beta, eps, step, o, out->pitch_bytes, y_f32, ld_y, (float)qn, (float)qp, st);
    return launch_ln<8>(nv, x, rows, (int)cols, ldx, gamma, beta, eps, step, o, out->pitch_bytes, y_f32, ld_y, (float)qn, (float)qp, st);
}
