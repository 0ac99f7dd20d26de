// Host-side preparation of epilogue / quantizer parameters (no device work): the constants that
// the paper absorbs into the stage after a contraction, computed once per layer in fp64 and
// rounded once to fp32.
#include <cmath>

#include "common.cuh"

using namespace vitint;

// Eq. 2: [X_q W_q^T + b / (s_x s_w)] s_x s_w, followed by a quantizer of step s_out, is
// q = clamp(rint(acc * alpha + beta)) with alpha = s_x s_w / s_out and beta = b / s_out.
extern "C" int vitint_fold_requant(float x_step, const float* w_step, const float* bias, const float* out_step,
                                   int64_t n, float* alpha, float* beta) {
    if (!w_step || !out_step || !alpha || !beta || n <= 0) return VITINT_ERR_INVALID_ARG;
    if (!(x_step > 0.0f && x_step < INFINITY)) return VITINT_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i) {
        const double so = (double)out_step[i], sw = (double)w_step[i];
        if (!(so > 0.0 && so < INFINITY) || !(sw > 0.0 && sw < INFINITY)) return VITINT_ERR_INVALID_ARG;
        alpha[i] = (float)(((double)x_step * sw) / so);
        beta[i] = bias ? (float)((double)bias[i] / so) : 0.0f;
    }
    return VITINT_OK;
}

// Fig. 5(b): the comparator decides (x - mu)/sigma * gamma + beta > (k - 1/2) step without sigma or a
// division by comparing signed squares; what it needs per column j and threshold k = Qn+1 .. Qp is the
// signed reference sgn(c) c^2 / cols, c = ((k - 1/2) step - beta_j) / gamma_j, with c negated (and the
// column flagged) where gamma_j < 0 so that the comparison keeps one direction.
extern "C" int vitint_fold_layernorm_references(const float* gamma, const float* beta, float step, int32_t bits,
                                                int32_t is_signed, int64_t cols, float* refs, uint8_t* flip) {
    if (!gamma || !beta || !refs || !flip || cols <= 0) return VITINT_ERR_INVALID_ARG;
    if (!valid_bits(bits) || bits == 8 || !(step > 0.0f && step < INFINITY)) return VITINT_ERR_INVALID_ARG;
    int qn, qp;
    code_range(bits, is_signed, &qn, &qp);
    const int n_thr = qp - qn;
    for (int64_t j = 0; j < cols; ++j) {
        const double g = (double)gamma[j], b = (double)beta[j];
        if (g == 0.0 || !(std::fabs(g) < INFINITY)) return VITINT_ERR_INVALID_ARG;
        const bool neg_gain = g < 0.0;
        flip[j] = neg_gain ? 1 : 0;
        for (int t = 0; t < n_thr; ++t) {
            const double k = (double)(qn + 1 + t);
            double c = ((k - 0.5) * (double)step - b) / g;
            if (neg_gain) c = -c;
            const double sgn = c > 0.0 ? 1.0 : (c < 0.0 ? -1.0 : 0.0);
            refs[j * n_thr + t] = (float)((sgn * c) * c / (double)cols);
        }
    }
    return VITINT_OK;
}
