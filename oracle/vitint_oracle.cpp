// CPU oracle for the operand-reordered integerized ViT matmul path.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
// path computes, written from the paper's equations; it shares no code with the
// CUDA library and is never called by it.  Only the tests, the smoke check and
// the benchmark's CPU-baseline leg load it.
//
// Conventions
//   * integer codes live UNPACKED in int16_t arrays (row-major, explicit leading
//     dimension); packing is a separate, explicitly tested step;
//   * signed b-bit codes span [-2^(b-1), 2^(b-1)-1], unsigned [0, 2^b-1]
//     (the 3-bit comparator ladder -3.5D ... 2.5D of Section IV-B gives levels -4..3);
//   * rounding is to nearest, ties to even, everywhere (one rule; a comparator
//     ladder "x > (k-1/2)D" differs from it only on exact ties);
//   * every fp32 result is produced by a fixed sequence of IEEE-754 operations,
//     compiled with contraction off, so the bits are unique.
//
// Pins (tests/test_oracle_*.py): Eq. 1 reordering identity against an fp64
// dequantize-then-matmul, brute force on tiny operands, closed-form sums, the
// int32 overflow bound, the 3-bit threshold ladder, pack/unpack round trips,
// exact-rational epilogue cases, softmax closed forms and invariants, the shift softmax
// against big-integer / rational arithmetic and its 2^r ~ 1+r error bound, LayerNorm
// against the Welford recurrence of Eq. 5, the comparator LayerNorm quantizer against exact rational
// arithmetic, the direct formula of Fig. 5(a), hand-worked rows and its invariances.  Parity unpinned: none of the
// functions below; the paper's accuracy and power tables are out of scope.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <thread>
#include <vector>

namespace {

int g_threads = 0;

int thread_count() {
    if (g_threads > 0) return g_threads;
    unsigned hc = std::thread::hardware_concurrency();
    return hc ? (int)hc : 1;
}

// Runs body(i) for i in [0, n) on the host cores, contiguous ranges per thread.
void parallel_for(int64_t n, const std::function<void(int64_t)>& body) {
    int nt = (int)std::min<int64_t>(thread_count(), n);
    if (nt <= 1) {
        for (int64_t i = 0; i < n; ++i) body(i);
        return;
    }
    std::vector<std::thread> pool;
    for (int t = 0; t < nt; ++t) {
        int64_t lo = n * t / nt, hi = n * (t + 1) / nt;
        pool.emplace_back([lo, hi, &body]() {
            for (int64_t i = lo; i < hi; ++i) body(i);
        });
    }
    for (auto& th : pool) th.join();
}

inline void code_range(int bits, int is_signed, int* qn, int* qp) {
    if (is_signed) { *qn = -(1 << (bits - 1)); *qp = (1 << (bits - 1)) - 1; }
    else           { *qn = 0;                  *qp = (1 << bits) - 1; }
}

// Round-to-nearest-even then clamp: the comparator quantizer of Section IV-B
// (code = number of thresholds (k-1/2) exceeded), with our tie rule.
inline int16_t round_clamp(float r, int qn, int qp) {
    float n = nearbyintf(r);
    if (!(n >= (float)qn)) n = (float)qn;   // also maps NaN to qn
    if (n > (float)qp) n = (float)qp;
    return (int16_t)n;
}

inline int container_bits(int bits) { return bits == 3 ? 4 : bits; }

// GELU(y) = y * Phi(y), evaluated in fp64 and rounded once.
inline float gelu_ref(float y) {
    double yd = (double)y;
    return (float)(0.5 * yd * (1.0 + std::erf(yd * 0.70710678118654752440)));
}

}  // namespace

extern "C" {

void vo_set_threads(int n) { g_threads = n; }
int vo_get_threads() { return thread_count(); }

// ---- quantizer (Section IV-B comparator quantizer; a1) ---------------------
// q = clamp(rint(x / s)); one IEEE fp32 division, ties-to-even.  row_steps, when
// given, supplies one step per row (per-output-channel weight steps, Eq. 1's
// Delta_W); otherwise `step` is the single per-tensor step (Eq. 2's bar-Delta_X).
void vo_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx, float step, const float* row_steps,
                 int bits, int is_signed, int16_t* q, int64_t ldq) {
    int qn, qp;
    code_range(bits, is_signed, &qn, &qp);
    parallel_for(rows, [&](int64_t m) {
        float s = row_steps ? row_steps[m] : step;
        for (int64_t k = 0; k < cols; ++k) q[m * ldq + k] = round_clamp(x[m * ldx + k] / s, qn, qp);
    });
}

// ---- packed storage format --------------------------------------------------
// Container of 2,4,4,8 bits for 2,3,4,8-bit codes; element i of a row sits in
// byte i/(8/c) at bit offset c*(i mod 8/c); two's complement within the
// container; bytes from the last code to the pitch are zero.
void vo_pack(const int16_t* q, int64_t rows, int64_t cols, int64_t ldq, int bits, uint8_t* out, int64_t pitch) {
    int c = container_bits(bits), per = 8 / c, mask = (1 << c) - 1;
    for (int64_t m = 0; m < rows; ++m) {
        uint8_t* row = out + m * pitch;
        std::memset(row, 0, (size_t)pitch);
        for (int64_t i = 0; i < cols; ++i)
            row[i / per] |= (uint8_t)(((int)q[m * ldq + i] & mask) << (c * (i % per)));
    }
}

void vo_unpack(const uint8_t* in, int64_t rows, int64_t cols, int64_t pitch, int bits, int is_signed, int16_t* q,
               int64_t ldq) {
    int c = container_bits(bits), per = 8 / c, mask = (1 << c) - 1;
    for (int64_t m = 0; m < rows; ++m)
        for (int64_t i = 0; i < cols; ++i) {
            int v = (in[m * pitch + i / per] >> (c * (i % per))) & mask;
            if (is_signed && (v & (1 << (c - 1)))) v -= (1 << c);
            q[m * ldq + i] = (int16_t)v;
        }
}

// ---- integer contraction (Eq. 1, second line: X_q W_q^T; a2, a4, a6) ----------
// acc[m][n] = sum_k a[m][k] * b[n][k], both operands K-contiguous.
void vo_matmul_i32(const int16_t* a, int64_t lda, const int16_t* b, int64_t ldb, int64_t M, int64_t N, int64_t K,
                   int32_t* acc, int64_t ldacc) {
    parallel_for(M, [&](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            int32_t s = 0;
            for (int64_t k = 0; k < K; ++k) s += (int32_t)a[m * lda + k] * (int32_t)b[n * ldb + k];
            acc[m * ldacc + n] = s;
        }
    });
}

// Same contraction in int64: shows what the int32 accumulator must hold.
void vo_matmul_i64(const int16_t* a, int64_t lda, const int16_t* b, int64_t ldb, int64_t M, int64_t N, int64_t K,
                   int64_t* acc, int64_t ldacc) {
    parallel_for(M, [&](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int64_t k = 0; k < K; ++k) s += (int64_t)a[m * lda + k] * (int64_t)b[n * ldb + k];
            acc[m * ldacc + n] = s;
        }
    });
}

// K * max|q_x| * max|q_w| over the declared formats; the contraction is safe in
// int32 when this is < 2^31.
int64_t vo_overflow_bound(int64_t K, int bits_x, int signed_x, int bits_w, int signed_w) {
    int qn, qp;
    code_range(bits_x, signed_x, &qn, &qp);
    int64_t mx = std::max<int64_t>(-qn, qp);
    code_range(bits_w, signed_w, &qn, &qp);
    int64_t mw = std::max<int64_t>(-qn, qp);
    return K * mx * mw;
}

// ---- post-contraction epilogues (Eq. 2: scale after the contraction; a3) -------
// DEQUANT: sc[n] = fl32(s_x * s_w[n]);  y = fmaf(float(acc), sc[n], b[n]);
// optional GELU (fp64, one rounding), then optional residual as one more fp32 add.
void vo_epilogue_dequant(const int32_t* acc, int64_t M, int64_t N, int64_t ldacc, float s_x, const float* s_w,
                         const float* bias, const float* residual, int64_t ld_res, int act, float* y, int64_t ldy) {
    parallel_for(M, [&](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            float sc = (float)((double)s_x * (double)s_w[n]);
            float v = fmaf((float)acc[m * ldacc + n], sc, bias ? bias[n] : 0.0f);
            if (act == 1) v = gelu_ref(v);
            if (residual) v = v + residual[m * ld_res + n];
            y[m * ldy + n] = v;
        }
    });
}

// REQUANT: q = clamp(rint(fmaf(float(acc), alpha[n], beta[n]))), with the folded
// alpha = s_x s_w/s_out and beta = b/s_out of Eq. 2 supplied by the caller.
void vo_epilogue_requant(const int32_t* acc, int64_t M, int64_t N, int64_t ldacc, const float* alpha,
                         const float* beta, int bits, int is_signed, int16_t* q, int64_t ldq) {
    int qn, qp;
    code_range(bits, is_signed, &qn, &qp);
    parallel_for(M, [&](int64_t m) {
        for (int64_t n = 0; n < N; ++n)
            q[m * ldq + n] = round_clamp(fmaf((float)acc[m * ldacc + n], alpha[n], beta[n]), qn, qp);
    });
}

// REQUANT after GELU: g = GELU(fmaf(float(acc), sc[n], b[n])) (fp64 GELU, rounded
// once), q = clamp(rint(g * inv_s[n])) decided in fp32.  An fp32 GELU may differ
// from g by up to gelu_tol_rel*|y|; q_lo/q_hi give the codes reachable inside
// that tolerance, so a checker can accept either neighbour on near-ties only.
void vo_epilogue_gelu_requant(const int32_t* acc, int64_t M, int64_t N, int64_t ldacc, float s_x, const float* s_w,
                              const float* bias, const float* inv_s, int bits, int is_signed, float gelu_tol_rel,
                              int16_t* q, int16_t* q_lo, int16_t* q_hi, int64_t ldq) {
    int qn, qp;
    code_range(bits, is_signed, &qn, &qp);
    parallel_for(M, [&](int64_t m) {
        for (int64_t n = 0; n < N; ++n) {
            float sc = (float)((double)s_x * (double)s_w[n]);
            float y = fmaf((float)acc[m * ldacc + n], sc, bias ? bias[n] : 0.0f);
            float g = gelu_ref(y);
            float tol = gelu_tol_rel * fabsf(y);
            q[m * ldq + n] = round_clamp(g * inv_s[n], qn, qp);
            if (q_lo) q_lo[m * ldq + n] = round_clamp((g - tol) * inv_s[n], qn, qp);
            if (q_hi) q_hi[m * ldq + n] = round_clamp((g + tol) * inv_s[n], qn, qp);
        }
    });
}

// ---- attention matmuls (Section IV-B; a4, a6) -------------------------------
// S[p][i][j] = sum_c Q_p[i][c] K_p[j][c]; slabs are strided views: row stride ld,
// problem p starts at base + p*problem_stride (elements).
void vo_qk(const int16_t* q, int64_t ldq, int64_t pstride_q, const int16_t* k, int64_t ldk, int64_t pstride_k,
           int64_t n_problems, int64_t T, int64_t d, int32_t* S) {
    parallel_for(n_problems, [&](int64_t p) {
        const int16_t* qp_ = q + p * pstride_q;
        const int16_t* kp_ = k + p * pstride_k;
        int32_t* Sp = S + p * T * T;
        for (int64_t i = 0; i < T; ++i)
            for (int64_t j = 0; j < T; ++j) {
                int32_t s = 0;
                for (int64_t c = 0; c < d; ++c) s += (int32_t)qp_[i * ldq + c] * (int32_t)kp_[j * ldk + c];
                Sp[i * T + j] = s;
            }
    });
}

// O[p][i][c] = sum_j P_p[i][j] V_p[j][c]  (unsigned probabilities x signed values).
void vo_pv(const int16_t* P, int64_t ldp, int64_t pstride_p, const int16_t* v, int64_t ldv, int64_t pstride_v,
           int64_t n_problems, int64_t T, int64_t d, int32_t* O) {
    parallel_for(n_problems, [&](int64_t p) {
        const int16_t* Pp = P + p * pstride_p;
        const int16_t* vp = v + p * pstride_v;
        int32_t* Op = O + p * T * d;
        for (int64_t i = 0; i < T; ++i)
            for (int64_t c = 0; c < d; ++c) {
                int32_t s = 0;
                for (int64_t j = 0; j < T; ++j) s += (int32_t)Pp[i * ldp + j] * (int32_t)vp[j * ldv + c];
                Op[i * d + c] = s;
            }
    });
}

// ---- scale + softmax + quantize (Eq. 3; a5) -----------------------------------
// t_j = fl32(float(S_j) * c);  m = max_j t_j;  e_j = exp(t_j - m), Z = sum_j e_j
// (ascending j) and e_j/Z in fp64;  p_j = fl32(e_j / Z).
// Codes are decided in fp32: q_j = clamp(rint(p_j / s_P), 0, 2^b-1) (one IEEE
// division).  q_lo/q_hi are the codes of p_j moved by -/+ ulp_band units in the
// last place: the set of codes an fp32 softmax within that tolerance may produce.
void vo_softmax_quantize(const int32_t* S, int64_t rows, int64_t cols, int64_t lds, float c, float p_step, int bits,
                         int ulp_band, float* p, int64_t ldp, int16_t* q, int16_t* q_lo, int16_t* q_hi,
                         int64_t ldq) {
    int qn, qp;
    code_range(bits, 0, &qn, &qp);
    parallel_for(rows, [&](int64_t r) {
        std::vector<float> t((size_t)cols);
        std::vector<double> e((size_t)cols);
        float mx = -INFINITY;
        for (int64_t j = 0; j < cols; ++j) {
            t[j] = (float)S[r * lds + j] * c;
            mx = std::max(mx, t[j]);
        }
        double Z = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            e[j] = std::exp((double)t[j] - (double)mx);
            Z += e[j];
        }
        for (int64_t j = 0; j < cols; ++j) {
            float pj = (float)(e[j] / Z);
            if (p) p[r * ldp + j] = pj;
            if (q) q[r * ldq + j] = round_clamp(pj / p_step, qn, qp);
            if (q_lo || q_hi) {
                float lo = pj, hi = pj;
                for (int u = 0; u < ulp_band; ++u) {
                    lo = nextafterf(lo, -INFINITY);
                    hi = nextafterf(hi, INFINITY);
                }
                if (lo < 0.0f) lo = 0.0f;
                if (q_lo) q_lo[r * ldq + j] = round_clamp(lo / p_step, qn, qp);
                if (q_hi) q_hi[r * ldq + j] = round_clamp(hi / p_step, qn, qp);
            }
        }
    });
}

// ---- shift-based softmax with the division-free quantizer (Eq. 4, Section IV-B) ---------------
// Follows the paper's steps with integers wherever it says "shift":
//   z_j = fl32(float(S_j) * c2),  c2 = s*log2(e) supplied by the caller      (exponent of 2, Eq. 4 line 1)
//   f_j = floor(z_j),  r_j = z_j - f_j (exact)                                (integer part and residual)
//   M_j = (1 + r_j) * 2^23   as an integer: 2^r ~ 1 + r                       (Eq. 4 last line)
//   E_j = M_j << (30 + f_j - m),  m = max_j f_j; negative counts shift right  ("<< floor(...)")
//         (a common factor 2^(30-m) changes neither side of the comparison below; it only keeps the
//          integers inside 64 bits; bits shifted out on the right are dropped, as a shifter drops them)
//   Sigma = sum_j E_j   (exact integer sum: the systolic row adder)
//   code_j = number of k in 1..Qp with  float(E_j) > fl32(b_k * float(Sigma)),  b_k = fl32((k - 1/2) * step)
//         (comparator references scaled by the row sum instead of dividing by it; strict '>' as drawn)
// Every operation is an integer one or a single IEEE fp32 operation, so the codes are unique.
// p_approx (optional) = float(E_j) / float(Sigma) in fp64, for error studies only.
void vo_softmax_shift_quantize(const int32_t* S, int64_t rows, int64_t cols, int64_t lds, float c2, float p_step,
                               int bits, int16_t* q, int64_t ldq, double* p_approx, int64_t ldp) {
    int qn, qp;
    code_range(bits, 0, &qn, &qp);
    parallel_for(rows, [&](int64_t r) {
        std::vector<int64_t> f((size_t)cols);
        std::vector<uint64_t> M((size_t)cols), E((size_t)cols);
        int64_t m = INT64_MIN;
        for (int64_t j = 0; j < cols; ++j) {
            const float z = (float)S[r * lds + j] * c2;
            const float fl = floorf(z);
            const float res = z - fl;
            f[j] = (int64_t)fl;
            M[j] = (uint64_t)((1.0f + res) * 8388608.0f);
            m = std::max(m, f[j]);
        }
        uint64_t sigma = 0;
        for (int64_t j = 0; j < cols; ++j) {
            const int64_t sh = 30 + f[j] - m;
            E[j] = sh >= 0 ? (M[j] << sh) : (sh > -64 ? (M[j] >> (-sh)) : 0);
            sigma += E[j];
        }
        const float sig_f = (float)sigma;
        for (int64_t j = 0; j < cols; ++j) {
            const float e_f = (float)E[j];
            int code = 0;
            for (int k = 1; k <= qp; ++k) {
                const float b_k = ((float)k - 0.5f) * p_step;
                if (e_f > b_k * sig_f) ++code;
            }
            q[r * ldq + j] = (int16_t)code;
            if (p_approx) p_approx[r * ldp + j] = (double)E[j] / (double)sigma;
        }
    });
}

// ---- LayerNorm glue between integerized linears (fp32 island of Fig. 1(b)) ----
// Two-pass mean / variance in fp64 (biased variance), y = (x-mu)/sqrt(var+eps)*g+b
// in fp64, rounded once.  tol[m][n] = 8*2^-24*(|g_n|*max_row|x-mu|/sigma + |b_n|) is
// the absolute tolerance granted to an fp32 implementation (cancellation near the
// mean makes a per-element ulp bound meaningless).
void vo_layernorm(const float* x, int64_t rows, int64_t cols, int64_t ldx, const float* gamma, const float* beta,
                  float eps, float* y, int64_t ldy, float* tol, int64_t ldt) {
    parallel_for(rows, [&](int64_t m) {
        const float* xr = x + m * ldx;
        double mu = 0.0;
        for (int64_t k = 0; k < cols; ++k) mu += (double)xr[k];
        mu /= (double)cols;
        double var = 0.0, maxdev = 0.0;
        for (int64_t k = 0; k < cols; ++k) {
            double dlt = (double)xr[k] - mu;
            var += dlt * dlt;
            maxdev = std::max(maxdev, std::fabs(dlt));
        }
        var /= (double)cols;
        double sigma = std::sqrt(var + (double)eps);
        for (int64_t k = 0; k < cols; ++k) {
            double v = ((double)xr[k] - mu) / sigma * (double)gamma[k] + (double)beta[k];
            y[m * ldy + k] = (float)v;
            if (tol)
                tol[m * ldt + k] = (float)(8.0 * 5.9604644775390625e-08 *
                                           (std::fabs((double)gamma[k]) * maxdev / sigma + std::fabs((double)beta[k])));
        }
    });
}

// Running statistics of Eq. 5: mu_i = mu_{i-1} + (x_i - mu_{i-1})/i,
// M2_i = M2_{i-1} + (x_i - mu_{i-1})(x_i - mu_i), mu_0 = M2_0 = 0.  The second
// quantity is the unnormalised sum of squared deviations (variance = M2_n / n).
void vo_running_stats(const float* x, int64_t n, double* mu_out, double* m2_out) {
    double mu = 0.0, m2 = 0.0;
    for (int64_t i = 1; i <= n; ++i) {
        double xi = (double)x[i - 1];
        double mu_prev = mu;
        mu = mu_prev + (xi - mu_prev) / (double)i;
        m2 = m2 + (xi - mu_prev) * (xi - mu);
    }
    *mu_out = mu;
    *m2_out = m2;
}

// ---- quantizing LayerNorm (Section IV-C: Eq. 5 running statistics + the division- and
//      square-root-free comparator of Fig. 5(b)) ---------------------------------------------
// Row statistics by the recurrence of Eq. 5 in the order the paper gives, every operation a
// single fp32 one (the paper fixes no precision; fp32 is the reading taken):
//   delta = x_i - mu_{i-1};  mu_i = mu_{i-1} + delta / i;  S_i = S_{i-1} + delta * (x_i - mu_i)
// with mu_0 = S_0 = 0.  S_n is the unnormalised sum of squared deviations (n * variance); the 1/n
// and LayerNorm's epsilon are absorbed as the paper absorbs scales: V = S_n + n*eps multiplies
// references that already carry 1/n.
// Quantizer: code = Qn + number of thresholds s_k = (k - 1/2) * step, k = Qn+1 .. Qp, with
//   (x - mu)/sigma * gamma + beta > s_k.
// For gamma > 0 this is  d > sigma * c_k  with d = x - mu, c_k = (s_k - beta)/gamma, decided without
// sigma and without a division from squares plus sign logic (Fig. 5(b)):
//   c_k <  0 :  true when d >= 0, otherwise  d*d < V * (c_k^2 / n)
//   c_k >= 0 :  false when d <= 0, otherwise  d*d > V * (c_k^2 / n)
// For gamma < 0 the direction flips (d < sigma * c_k): the same logic applied to -d and -c_k.
// The caller supplies ref[j][t] = c^2 / n >= 0 and neg[j][t] = 1 when the (gamma-sign-adjusted) c is
// negative, for column j and threshold t = 0 .. 2^bits-2 (ascending k), and flip[j] = 1 for gamma_j < 0.
void vo_layernorm_compare_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx, const float* ref,
                                   const uint8_t* neg, const uint8_t* flip, float n_eps, int bits, int is_signed,
                                   int16_t* q, int64_t ldq, float* mu_out, float* v_out) {
    int qn, qp;
    code_range(bits, is_signed, &qn, &qp);
    const int n_thr = qp - qn;
    parallel_for(rows, [&](int64_t m) {
        const float* xr = x + m * ldx;
        float mu = 0.0f, S = 0.0f;
        for (int64_t i = 1; i <= cols; ++i) {
            const float xi = xr[i - 1];
            const float delta = xi - mu;
            const float step_mu = delta / (float)i;
            mu = mu + step_mu;
            const float prod = delta * (xi - mu);
            S = S + prod;
        }
        const float V = S + n_eps;
        if (mu_out) mu_out[m] = mu;
        if (v_out) v_out[m] = V;
        for (int64_t j = 0; j < cols; ++j) {
            float d = xr[j] - mu;
            if (flip && flip[j]) d = -d;
            const float d2 = d * d;
            int code = qn;
            for (int t = 0; t < n_thr; ++t) {
                const float rhs = V * ref[j * n_thr + t];
                bool above;
                if (neg[j * n_thr + t]) above = (d >= 0.0f) ? true : (d2 < rhs);
                else                    above = (d <= 0.0f) ? false : (d2 > rhs);
                if (above) ++code;
            }
            q[m * ldq + j] = (int16_t)code;
        }
    });
}

// Quantize y with absolute tolerance tol: the code of y and the codes reachable
// within y -/+ tol under the a1 rule (division by the step, ties-to-even, clamp).
void vo_quantize_band(const float* y, const float* tol, int64_t rows, int64_t cols, int64_t ld, float step, int bits,
                      int is_signed, int16_t* q, int16_t* q_lo, int16_t* q_hi, int64_t ldq) {
    int qn, qp;
    code_range(bits, is_signed, &qn, &qp);
    parallel_for(rows, [&](int64_t m) {
        for (int64_t k = 0; k < cols; ++k) {
            float v = y[m * ld + k], t = tol[m * ld + k];
            q[m * ldq + k] = round_clamp(v / step, qn, qp);
            q_lo[m * ldq + k] = round_clamp((v - t) / step, qn, qp);
            q_hi[m * ldq + k] = round_clamp((v + t) / step, qn, qp);
        }
    });
}

}  // extern "C"
