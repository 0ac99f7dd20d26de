// a5: scale + row softmax + quantize (Eq. 3), half a warp per row.
//
// HBM-bound by bytes: 4 bytes read and c/8 bytes written per element.  The row lives in
// registers; the maximum and the normaliser are reduced with shuffles inside the half-warp.
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

// exp(t - mx) for mx >= t, two elements at a time, in fp32 and integer instructions (no special-function unit;
// every packed operation gives each half the IEEE result of the scalar one).
//   * t - mx as an exact two-float sum (TwoSum), so nothing is lost when the two differ by more than a factor of two;
//   * k = rint((t - mx) * log2 e) by the 1.5*2^23 addition, which also leaves k as an integer in the mantissa;
//   * r = (t - mx) - k*ln2 with ln2 split so that k*ln2_hi is exact, the low parts folded in with one FMA;
//   * degree-7 Taylor polynomial on |r| <= ln2/2 (truncation < 0.1 ulp), then 2^k added to the exponent field.
// Results below 2^-125 (relative to the row's largest term, which is 1) are returned as 0: they lie in the range
// where the tolerance is the absolute 2^-126.  t = -inf (a column past the row's end) gives exactly 0.
__device__ __forceinline__ f32x2 exp_reduced2(f32x2 t, f32x2 nmx) {
    const f32x2 neg1 = f2_dup(-1.0f);
    const f32x2 sh = f2_add(t, nmx);
    const f32x2 bv = f2_fma(t, neg1, sh);                         // sh - t
    const f32x2 u = f2_fma(bv, neg1, sh);                         // sh - bv
    const f32x2 v = f2_fma(u, neg1, t);                           // t - (sh - bv)
    const f32x2 w = f2_fma(bv, neg1, nmx);                        // -mx - bv
    const f32x2 sl = f2_add(v, w);                                // sh + sl = t - mx exactly
    // m = 1.5*2^23 + k for every difference down to about -2^21; further down (and for -inf or NaN) m falls below the
    // threshold tested at the end and the result is 0 whatever the polynomial made of it
    const f32x2 m = f2_fma(sh, f2_dup(1.44269504088896340736f), f2_dup(12582912.0f));
    const f32x2 kf = f2_add(m, f2_dup(-12582912.0f));
    const f32x2 rh = f2_fma(kf, f2_dup(-0.693145751953125f), sh);              // exact: ln2_hi has 15 significant bits
    const f32x2 rl = f2_fma(kf, f2_dup(-1.42860682030941723212e-6f), sl);      // ln2 - ln2_hi, and the low part of t - mx
    const f32x2 rf = f2_add(rh, rl);
    f32x2 p = f2_dup(1.0f / 5040.0f);
    p = f2_fma(p, rf, f2_dup(1.0f / 720.0f));
    p = f2_fma(p, rf, f2_dup(1.0f / 120.0f));
    p = f2_fma(p, rf, f2_dup(1.0f / 24.0f));
    p = f2_fma(p, rf, f2_dup(1.0f / 6.0f));
    p = f2_fma(p, rf, f2_dup(0.5f));
    p = f2_fma(p, rf, f2_dup(1.0f));
    p = f2_fma(p, rf, f2_dup(1.0f));
    // p lies in [0.70, 1.42]: for k >= -125 the product p * 2^k is normal and exact as an exponent addition.  The
    // float m holds 1.5*2^23 + k exactly, and its low 9 bits shifted up by 23 are k's (0x4B400000 << 23 is 0 mod 2^32).
    float m0, m1, p0, p1;
    f2_unpack(m, m0, m1);
    f2_unpack(p, p0, p1);
    const float e0 = m0 >= 12582912.0f - 125.0f ? __int_as_float(__float_as_int(m0) * 8388608 + __float_as_int(p0)) : 0.0f;
    const float e1 = m1 >= 12582912.0f - 125.0f ? __int_as_float(__float_as_int(m1) * 8388608 + __float_as_int(p1)) : 0.0f;
    return f2_pack(e0, e1);
}

constexpr int SM_ROWS_PER_BLOCK = 16;      // half a warp per row, eight warps
constexpr int SM_TAIL_SLOTS = 4;           // up to 63 columns behind the last whole 64-column chunk, 16 per slot

// One row by half a warp.  Lane h (0..15) of the row owns columns 64 j + 4 h .. + 3 of every whole 64-column chunk j
// (one 16-byte load each) and, of the up to 63 columns behind the last whole chunk, column 64 nv + 16 s + h of slot
// s: a row of 197 columns costs 13 element slots per lane instead of the 16 that whole vectors would take.
// NVT is the compiled number of chunk slots (>= the row's whole chunks nv; a surplus slot carries t = -inf and stores
// nothing); NTT the compiled number of tail slots.  The loops are straight-line code: loads and stores are
// predicated, nothing branches per element.  VEC: 16-byte loads are legal; DIV3: the step admits the three-operation
// exact quotient.
// TABLE: the scores are known to lie in -smax .. smax and `tab` (shared memory) holds exp(fl32(s * c)) for each of
// them, tab[s + smax]: e_j is one lookup, no maximum is needed (exp(t_j) / sum_k exp(t_k) is Eq. 3's softmax
// exactly; the maximum is only subtracted there for range, and the caller has checked smax*|c| <= 80).  A score
// outside the range reads a clamped entry and sets `bad`.
// The raw scores of a row in the column mapping of softmax_row (zeros where the row has no column): issued as a
// unit so that a caller can request the next row before it works on the present one.
template <int NVT, int NTT, bool VEC>
struct RowScores {
    int4 a[NVT > 0 ? NVT : 1];
    int tv[NTT > 0 ? NTT : 1];
    __device__ __forceinline__ void load(const int32_t* __restrict__ sr, int cols, int hl) {
        const int nv = cols >> 6;
        const int tail0 = nv << 6, n_tail = cols - tail0;
#pragma unroll
        for (int j = 0; j < NVT; ++j) {
            const int col = j * 64 + hl * 4;
            a[j] = make_int4(0, 0, 0, 0);
            if (j < nv) {
                if (VEC) a[j] = __ldg(reinterpret_cast<const int4*>(sr + col));
                else a[j] = make_int4(__ldg(sr + col), __ldg(sr + col + 1), __ldg(sr + col + 2), __ldg(sr + col + 3));
            }
        }
#pragma unroll
        for (int q = 0; q < NTT; ++q) {
            const int o = q * 16 + hl;
            tv[q] = 0;
            if (o < n_tail) tv[q] = __ldg(sr + tail0 + o);
        }
    }
};

template <int C, int NVT, int NTT, bool VEC, bool DIV3, bool TABLE = false>
__device__ __forceinline__ void softmax_row(const RowScores<NVT, NTT, VEC>& in, int cols, float c, const Divisor dv, float qp,
                                            uint8_t* crow, float* pr, bool vec_p, int hl, const float* tab = nullptr,
                                            int smax = 0, uint32_t* worst = nullptr) {
    // table mode: index v + smax of the score's entry in unsigned arithmetic (a score below -smax wraps to a huge
    // index, so one comparison covers both ends); one unsigned maximum keeps track of the largest index seen, one
    // unsigned minimum keeps the load inside the table
    uint32_t umax = 0u;
    auto lookup = [&](int v) -> float {
        const uint32_t i = (uint32_t)v + (uint32_t)smax;
        umax = max(umax, i);
        return tab[min(i, (uint32_t)(2 * smax))];
    };
    const int nv = cols >> 6;
    const int tail0 = nv << 6, n_tail = cols - tail0;
    const f32x2 c2 = f2_dup(c);
    constexpr int NP = 2 * NVT + (NTT + 1) / 2;          // register pairs: two per chunk, one per two tail slots
    f32x2 t[NP > 0 ? NP : 1];
    float mx = -INFINITY;
    // Columns past the row's end take t = -inf: their exponential is exactly 0, so they add nothing to the row
    // sum and quantize to code 0 without any masking further down.
#pragma unroll
    for (int j = 0; j < NVT; ++j) {
        const bool have = j < nv;
        const int4 a = in.a[j];
        if (TABLE) {
            // (a surplus chunk looks up score 0 and discards it: no branch)
            const float e0 = lookup(a.x), e1 = lookup(a.y), e2 = lookup(a.z), e3 = lookup(a.w);
            t[2 * j] = have ? f2_pack(e0, e1) : f2_dup(0.0f);
            t[2 * j + 1] = have ? f2_pack(e2, e3) : f2_dup(0.0f);
            continue;
        }
        const f32x2 lo = f2_mul(f2_pack((float)a.x, (float)a.y), c2), hi = f2_mul(f2_pack((float)a.z, (float)a.w), c2);
        t[2 * j] = have ? lo : f2_dup(-INFINITY);
        t[2 * j + 1] = have ? hi : f2_dup(-INFINITY);
        float x0, x1, x2, x3;
        f2_unpack(t[2 * j], x0, x1);
        f2_unpack(t[2 * j + 1], x2, x3);
        mx = fmaxf(fmaxf(mx, fmaxf(x0, x1)), fmaxf(x2, x3));
    }
    {
        float x[NTT > 0 ? NTT + 1 : 2];
        x[NTT > 0 ? NTT : 1] = -INFINITY;
#pragma unroll
        for (int q = 0; q < NTT; ++q) {
            const int o = q * 16 + hl;
            const int v = in.tv[q];
            if (TABLE) {
                const float e = lookup(v);
                x[q] = o < n_tail ? e : 0.0f;
                continue;
            }
            x[q] = o < n_tail ? __fmul_rn((float)v, c) : -INFINITY;
            mx = fmaxf(mx, x[q]);
        }
#pragma unroll
        for (int q = 0; q < NTT; q += 2) t[2 * NVT + q / 2] = f2_pack(x[q], x[q + 1]);
    }
    if (!TABLE) {
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    } else {
        *worst = max(*worst, umax);
    }

    // exponentials (kept in the registers of t) and the fp64 row sum
    const f32x2 nmx = f2_dup(-mx);
    double z0 = 0.0, z1 = 0.0;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        if (!TABLE) t[i] = exp_reduced2(t[i], nmx);
        float e0, e1;
        f2_unpack(t[i], e0, e1);
        z0 += (double)e0;
        z1 += (double)e1;
    }
    double z = z0 + z1;
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    // 1/Z to about 2^-45 from the fp32 reciprocal and one Newton step in fp64, then split into two floats (Z lies in
    // [1, cols]; with the table anywhere in [e^-80, cols e^80] by the caller's bound: 1/Z is still a normal float, and a
    // low half that has become subnormal only loses bits of a correction that is itself 2^-24 of the result)
    const double r0 = (double)__frcp_rn((float)z);
    const double rz = r0 * (2.0 - z * r0);
    const float rzh = (float)rz, rzl = (float)(rz - (double)(float)rz);
    const f32x2 rzh2 = f2_dup(rzh), rzl2 = f2_dup(rzl);
    const f32x2 dr2 = f2_dup(dv.r), ndb2 = f2_dup(-dv.b), magic2 = f2_dup(12582912.0f);

    // p = e / Z, code = min(rint(p / p_step), Qp) (p >= 0: no lower clamp); adding 1.5*2^23 rounds to nearest even and
    // leaves the unsigned code in the low mantissa bits.  b0, b1: the two codes' float bits.
    auto quantize_pair = [&](f32x2 e, f32x2& p, uint32_t& b0, uint32_t& b1) {
        p = f2_fma(e, rzh2, f2_mul(e, rzl2));
        float q0, q1;
        if (DIV3) {
            const f32x2 qa = f2_mul(p, dr2);                            // Markstein: RN(p / step) in three operations
            const f32x2 rem = f2_fma(qa, ndb2, p);
            f2_unpack(f2_fma(rem, dr2, qa), q0, q1);
        } else {
            float p0, p1;
            f2_unpack(p, p0, p1);
            q0 = __fdiv_rn(p0, dv.b);
            q1 = __fdiv_rn(p1, dv.b);
        }
        float c0, c1;
        f2_unpack(f2_add(f2_pack(fminf(q0, qp), fminf(q1, qp)), magic2), c0, c1);
        b0 = __float_as_uint(c0);
        b1 = __float_as_uint(c1);
    };
#pragma unroll
    for (int j = 0; j < NVT; ++j) {
        f32x2 pa, pb;
        uint32_t b0, b1, b2, b3;
        quantize_pair(t[2 * j], pa, b0, b1);
        quantize_pair(t[2 * j + 1], pb, b2, b3);
        const int col = j * 64 + hl * 4;
        const bool have = j < nv;
        if (pr != nullptr && have) {
            float f0, f1, f2, f3;
            f2_unpack(pa, f0, f1);
            f2_unpack(pb, f2, f3);
            if (vec_p) *reinterpret_cast<float4*>(pr + col) = make_float4(f0, f1, f2, f3);
            else { pr[col] = f0; pr[col + 1] = f1; pr[col + 2] = f2; pr[col + 3] = f3; }
        }
        // four codes = C/2 bytes, combined by shift-add (the constant high bits of the four floats are removed at once)
        const uint32_t w = b0 + (b1 << C) + (b2 << (2 * C)) + (b3 << (3 * C)) -
                           0x4B400000u * (1u + (1u << C) + (1u << (2 * C)) + (1u << (3 * C)));
        if (have) {
            if (C == 8) *reinterpret_cast<uint32_t*>(crow + col) = w;
            else if (C == 4) *reinterpret_cast<uint16_t*>(crow + (col >> 1)) = (uint16_t)w;
            else crow[col >> 2] = (uint8_t)w;
        }
    }
#pragma unroll
    for (int q2 = 0; q2 < NTT; q2 += 2) {
        f32x2 pa;
        uint32_t b[2];
        quantize_pair(t[2 * NVT + q2 / 2], pa, b[0], b[1]);
        float f[2];
        f2_unpack(pa, f[0], f[1]);
#pragma unroll
        for (int i = 0; i < 2 && q2 + i < NTT; ++i) {
            const int o = (q2 + i) * 16 + hl;
            // neighbouring lanes hold neighbouring columns: 8/C of them share a byte (every lane takes part in the
            // shuffles; lanes past the tail hold code 0)
            uint32_t code = b[i] - 0x4B400000u;
            if (C == 4) code |= __shfl_xor_sync(0xffffffffu, code, 1) << 4;
            if (C == 2) {
                code |= __shfl_xor_sync(0xffffffffu, code, 1) << 2;
                code |= __shfl_xor_sync(0xffffffffu, code, 2) << 4;
            }
            if (o < n_tail) {
                if (pr != nullptr) pr[tail0 + o] = f[i];
                const int col = tail0 + o;
                if (C == 8) crow[col] = (uint8_t)code;
                else if (C == 4) { if ((hl & 1) == 0) crow[col >> 1] = (uint8_t)code; }
                else { if ((hl & 3) == 0) crow[col >> 2] = (uint8_t)code; }
            }
        }
    }
}

template <int C, int NVT, int NTT, bool VEC>
__global__ void __launch_bounds__(32 * SM_ROWS_PER_BLOCK / 2)
softmax_quantize_kernel(const int32_t* __restrict__ s, int64_t rows, int cols, int64_t ld_s, float c, float p_step,
                        uint8_t* __restrict__ out, int64_t pitch, float* __restrict__ p_out, int64_t ld_p, float qp,
                        int vec_p) {
    extern __shared__ __align__(16) uint8_t sm_codes[];   // one output row (pitch bytes) per half-warp
    grid_dependency_wait();        // inputs may come from the previous kernel of the stream
    grid_dependency_launch();
    const int hl = threadIdx.x & 15;
    const int hw = threadIdx.x >> 4;                                   // half-warp of the block
    const int64_t row_raw = (int64_t)blockIdx.x * SM_ROWS_PER_BLOCK + hw;
    const bool row_ok = row_raw < rows;
    const int64_t row = row_ok ? row_raw : rows - 1;                   // a surplus half-warp repeats the last row, stores nothing
    uint8_t* const crow = sm_codes + (size_t)hw * pitch;
    // padding behind the last code (and the unused part of a shared byte) is zero: clear the row buffer first
    for (int o = hl * 16; o < pitch; o += 256) *reinterpret_cast<uint4*>(crow + o) = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();
    float* const pr = (p_out != nullptr && row_ok) ? p_out + row * ld_p : nullptr;
    const Divisor dv = make_divisor(p_step);
    RowScores<NVT, NTT, VEC> in;
    in.load(s + row * ld_s, cols, hl);
    if (dv.exact) softmax_row<C, NVT, NTT, VEC, true>(in, cols, c, dv, qp, crow, pr, vec_p != 0, hl);
    else softmax_row<C, NVT, NTT, VEC, false>(in, cols, c, dv, qp, crow, pr, vec_p != 0, hl);
    __syncwarp();
    // the finished row leaves in 16-byte pieces
    if (row_ok) {
        uint8_t* const orow = out + row * pitch;
        for (int o = hl * 16; o < pitch; o += 256) *reinterpret_cast<uint4*>(orow + o) = *reinterpret_cast<const uint4*>(crow + o);
    }
}

template <int C, int NVT, int NTT>
static int launch_softmax_nv(const int32_t* s, int64_t rows, int cols, int64_t ld_s, float c, float p_step, uint8_t* out,
                             int64_t pitch, float* p, int64_t ld_p, float qp, int vec_in, int vec_p, cudaStream_t st) {
    dim3 grid((unsigned)((rows + SM_ROWS_PER_BLOCK - 1) / SM_ROWS_PER_BLOCK)), block(16 * SM_ROWS_PER_BLOCK);
    const size_t smem = (size_t)SM_ROWS_PER_BLOCK * (size_t)pitch;
    if (smem > 48 * 1024) return VITINT_ERR_UNSUPPORTED;
    if (vec_in) launch_kernel(softmax_quantize_kernel<C, NVT, NTT, true>, grid, block, smem, st, s, rows, cols, ld_s, c, p_step, out, pitch, p, ld_p, qp, vec_p);
    else launch_kernel(softmax_quantize_kernel<C, NVT, NTT, false>, grid, block, smem, st, s, rows, cols, ld_s, c, p_step, out, pitch, p, ld_p, qp, vec_p);
    return cuda_status(cudaGetLastError());
}

template <int C>
static int launch_softmax(const int32_t* s, int64_t rows, int cols, int64_t ld_s, float c, float p_step,
                          uint8_t* out, int64_t pitch, float* p, int64_t ld_p, float qp, int vec_in, int vec_p,
                          cudaStream_t st) {
    const int nv = cols >> 6, n_tail = cols & 63;
    const bool short_tail = n_tail <= 32;           // two tail slots are enough
#define VITINT_SM_CASE(NVT)                                                                                                       \
    if (nv <= NVT) {                                                                                                              \
        if (n_tail == 0) return launch_softmax_nv<C, NVT, 0>(s, rows, cols, ld_s, c, p_step, out, pitch, p, ld_p, qp, vec_in, vec_p, st); \
        if (short_tail) return launch_softmax_nv<C, NVT, 2>(s, rows, cols, ld_s, c, p_step, out, pitch, p, ld_p, qp, vec_in, vec_p, st); \
        return launch_softmax_nv<C, NVT, 4>(s, rows, cols, ld_s, c, p_step, out, pitch, p, ld_p, qp, vec_in, vec_p, st);           \
    }
    VITINT_SM_CASE(0) VITINT_SM_CASE(1) VITINT_SM_CASE(2) VITINT_SM_CASE(3) VITINT_SM_CASE(4) VITINT_SM_CASE(6) VITINT_SM_CASE(9)
    VITINT_SM_CASE(12) VITINT_SM_CASE(16)
#undef VITINT_SM_CASE
    return VITINT_ERR_UNSUPPORTED;
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
            // trunc((1 + res) * 2^23): 1 + res lies in [1, 2], so this is its mantissa with the hidden bit, read off the
            // float's bits (2^24 when the sum rounds to 2) -- no conversion instruction
            mant[k][i] = __float_as_uint(__fadd_rn(1.0f, res)) - 0x3F000000u;
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
    // The code is the number of comparator references fl32(fl32((t - 1/2) * step) * Sigma), t = 1 .. 2^bits - 1, that
    // float(E) exceeds.  k0 = rint(min(E / (step * Sigma), Qp - 3/4)) is at most one off and never Qp, so the two
    // references around it decide: code = k0 - 1 + [E > ref(k0)] + [E > ref(k0 + 1)], each reference formed with the
    // definition's two fp32 multiplications.
    const float inv = __frcp_rn(__fmul_rn(p_step, sig_f));
    const float u_top = (float)((1 << code_bits) - 1) - 0.75f;

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
                        // float(E): E is a 24-bit mantissa times a power of two, or (shifted right) an integer below
                        // 2^24 -- both convert exactly (putting the float together from its bits in the loop above
                        // instead was measured slower: 162 against 149 us)
                        const unsigned long long e = ((unsigned long long)(uint32_t)fi[u][i] << 32) | mant[u][i];
                        const float e_f = __ull2float_rn(e);
                        const float um = __fadd_rn(fminf(__fmul_rn(e_f, inv), u_top), 12582912.0f);   // 1.5*2^23 + k0
                        const float kf = __fadd_rn(um, -12582912.0f);
                        const float r_lo = __fmul_rn(__fmul_rn(__fadd_rn(kf, -0.5f), p_step), sig_f);
                        const float r_hi = __fmul_rn(__fmul_rn(__fadd_rn(kf, 0.5f), p_step), sig_f);
                        uint32_t code = (__float_as_uint(um) & 0xFFu) - 1u + (e_f > r_lo ? 1u : 0u) + (e_f > r_hi ? 1u : 0u);
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
    const int vec_in = (aligned16(s) && ld_s % 4 == 0) ? 1 : 0;
    const int vec_p = (p_f32 && aligned16(p_f32) && ld_p % 4 == 0) ? 1 : 0;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* o = (uint8_t*)p_out->data;
    if (cb == 2) return launch_softmax<2>(s, rows, cols, ld_s, c, p_step, o, p_out->pitch_bytes, p_f32, ld_p, (float)qp, vec_in, vec_p, st);
    if (cb == 4) return launch_softmax<4>(s, rows, cols, ld_s, c, p_step, o, p_out->pitch_bytes, p_f32, ld_p, (float)qp, vec_in, vec_p, st);
    return launch_softmax<8>(s, rows, cols, ld_s, c, p_step, o, p_out->pitch_bytes, p_f32, ld_p, (float)qp, vec_in, vec_p, st);
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
