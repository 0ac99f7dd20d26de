// a5 for scores of known range: softmax + quantize with exp taken from a table.
//
// The scores Q K^T of b-bit codes are bounded (|S| <= 64 * max|q| * max|k|: 4096 for 4-bit codes), so
// exp(fl32(s * c)) has at most a few thousand distinct values.  They are tabulated once (fp64 exp, one rounding)
// and every e_j becomes one shared-memory load instead of the ~20 fp32 operations of an accurate exponential:
// the kernel drops from issue-bound to memory-bound.  exp(t_j) / sum_k exp(t_k) is Eq. 3's softmax exactly (the
// maximum is only subtracted there for range); the row sum is fp64 and 1/Z is carried as two floats, as in the
// general kernel, so the probabilities stay within 2 ulp and the codes are those of the general kernel.
//
// Persistent CTAs: each copies the table (at most 33 KB) into shared memory once and then walks groups of 16 rows,
// half a warp per row, with the column mapping, quantizer and staging of softmax_row.
#include "common.cuh"

namespace vitint {
namespace {

template <int C, int NVT, int NTT>
__global__ void __launch_bounds__(32 * SM_ROWS_PER_BLOCK / 2, 4)      // four CTAs fit the shared memory: no use for fewer than 64 registers
softmax_table_quantize_kernel(const int32_t* __restrict__ s, int64_t rows, int cols, int64_t ld_s,
                              const float* __restrict__ table, int smax, float p_step, uint8_t* __restrict__ out,
                              int64_t pitch, float* __restrict__ p_out, int64_t ld_p, float qp, int vec_p) {
    extern __shared__ __align__(16) uint8_t smt_raw[];
    grid_dependency_wait();        // the table and the scores come from earlier kernels of the stream
    grid_dependency_launch();
    float* const tab = reinterpret_cast<float*>(smt_raw);
    const int n_tab = 2 * smax + 1;
    uint8_t* const codes = smt_raw + (((size_t)n_tab * 4 + 15) & ~(size_t)15);
    for (int i = threadIdx.x; i < n_tab; i += blockDim.x) tab[i] = __ldg(table + i);
    const int hl = threadIdx.x & 15;
    const int hw = threadIdx.x >> 4;
    uint8_t* const crow = codes + (size_t)hw * pitch;
    // padding behind the last code is zero; every row rewrites the same code bytes, so one clearing serves all rows
    for (int o = hl * 16; o < pitch; o += 256) *reinterpret_cast<uint4*>(crow + o) = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    const Divisor dv = make_divisor(p_step);
    uint32_t worst = 0u;                                               // largest table index any score asked for
    const int64_t groups = (rows + SM_ROWS_PER_BLOCK - 1) / SM_ROWS_PER_BLOCK;
    auto row_of = [&](int64_t g) -> int64_t {
        const int64_t r = g * SM_ROWS_PER_BLOCK + hw;
        return r < rows ? r : rows - 1;                                // a surplus half-warp repeats the last row, stores nothing
    };
    // (requesting the next row's scores before working on the present one was measured slower: the second register
    // set halves the resident CTAs or, capped, spills -- 98 to 108 us against 85)
    for (int64_t g = blockIdx.x; g < groups; g += gridDim.x) {
        const bool row_ok = g * SM_ROWS_PER_BLOCK + hw < rows;
        const int64_t row = row_of(g);
        float* const pr = (p_out != nullptr && row_ok) ? p_out + row * ld_p : nullptr;
        RowScores<NVT, NTT, true> in;
        in.load(s + row * ld_s, cols, hl);
        if (dv.exact) softmax_row<C, NVT, NTT, true, true, true>(in, cols, 0.0f, dv, qp, crow, pr, vec_p != 0, hl, tab, smax, &worst);
        else softmax_row<C, NVT, NTT, true, false, true>(in, cols, 0.0f, dv, qp, crow, pr, vec_p != 0, hl, tab, smax, &worst);
        __syncwarp();
        if (row_ok) {
            uint8_t* const orow = out + row * pitch;
            for (int o = hl * 16; o < pitch; o += 256) *reinterpret_cast<uint4*>(orow + o) = *reinterpret_cast<const uint4*>(crow + o);
        }
        __syncwarp();
    }
    // a score outside the declared range: that row's codes are not to be trusted, say so
    if (worst > (uint32_t)(2 * smax)) atomicExch(&g_device_status, (int)VITINT_ERR_INVALID_ARG);
}

template <int C, int NVT, int NTT>
int launch_softmax_table_nv(const int32_t* s, int64_t rows, int cols, int64_t ld_s, const float* table, int smax, float p_step,
                            uint8_t* out, int64_t pitch, float* p, int64_t ld_p, float qp, int vec_p, cudaStream_t st) {
    const size_t smem = (((size_t)(2 * smax + 1) * 4 + 15) & ~(size_t)15) + (size_t)SM_ROWS_PER_BLOCK * (size_t)pitch;
    if (smem > 100 * 1024) return VITINT_ERR_UNSUPPORTED;
    const int64_t groups = (rows + SM_ROWS_PER_BLOCK - 1) / SM_ROWS_PER_BLOCK;
    const int per_sm = (int)(200 * 1024 / smem) < 4 ? (int)(200 * 1024 / smem) : 4;
    int64_t grid = (int64_t)sm_count() * per_sm;
    if (grid > groups) grid = groups;
    auto launch = [&](auto kernel) -> int {
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024) != cudaSuccess)
            return VITINT_ERR_CUDA;
        launch_kernel(kernel, dim3((unsigned)grid), dim3(16 * SM_ROWS_PER_BLOCK), smem, st, s, rows, cols, ld_s, table, smax, p_step, out,
                      pitch, p, ld_p, qp, vec_p);
        return cuda_status(cudaGetLastError());
    };
    return launch(softmax_table_quantize_kernel<C, NVT, NTT>);
}

template <int C>
int launch_softmax_table(const int32_t* s, int64_t rows, int cols, int64_t ld_s, const float* table, int smax, float p_step,
                         uint8_t* out, int64_t pitch, float* p, int64_t ld_p, float qp, int vec_p, cudaStream_t st) {
    const int nv = cols >> 6, n_tail = cols & 63;
    const bool short_tail = n_tail <= 32;
#define VITINT_SMT_CASE(NVT)                                                                                                          \
    if (nv <= NVT) {                                                                                                                  \
        if (n_tail == 0) return launch_softmax_table_nv<C, NVT, 0>(s, rows, cols, ld_s, table, smax, p_step, out, pitch, p, ld_p, qp, vec_p, st); \
        if (short_tail) return launch_softmax_table_nv<C, NVT, 2>(s, rows, cols, ld_s, table, smax, p_step, out, pitch, p, ld_p, qp, vec_p, st); \
        return launch_softmax_table_nv<C, NVT, 4>(s, rows, cols, ld_s, table, smax, p_step, out, pitch, p, ld_p, qp, vec_p, st); \
    }
    VITINT_SMT_CASE(3) VITINT_SMT_CASE(9) VITINT_SMT_CASE(13)
#undef VITINT_SMT_CASE
    return VITINT_ERR_UNSUPPORTED;
}

}  // namespace
}  // namespace vitint

using namespace vitint;

extern "C" size_t vitint_softmax_table_workspace_bytes(int32_t score_bound) {
    if (score_bound <= 0 || score_bound > 8192) return 0;
    return ((size_t)(2 * score_bound + 1) * sizeof(float) + 255) & ~(size_t)255;
}

extern "C" int vitint_softmax_quantize_bounded(const int32_t* s, int64_t rows, int32_t cols, int64_t ld_s, float c,
                                               float p_step, int32_t score_bound, const vitint_codes* p_out, float* p_f32,
                                               int64_t ld_p, void* workspace, size_t workspace_bytes, int32_t table_ready,
                                               void* stream) {
    if (!s || !p_out) return VITINT_ERR_INVALID_ARG;
    if (int rc = check_codes(p_out)) return rc;
    if (rows <= 0 || cols <= 0 || ld_s < cols || p_out->rows != rows || p_out->cols != cols || p_out->is_signed)
        return VITINT_ERR_INVALID_ARG;
    if (!(p_step > 0.0f && p_step < INFINITY) || !(c == c) || fabsf(c) == INFINITY || score_bound <= 0)
        return VITINT_ERR_INVALID_ARG;
    if (p_f32 && ld_p < cols) return VITINT_ERR_INVALID_ARG;
    if (cols > 1024 || score_bound > 8192) return VITINT_ERR_UNSUPPORTED;
    if ((double)score_bound * fabs((double)c) > 80.0) return VITINT_ERR_UNSUPPORTED;   // exp without max subtraction
    if (!aligned16(s) || ld_s % 4 != 0) return VITINT_ERR_ALIGNMENT;           // 16-byte loads only
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < vitint_softmax_table_workspace_bytes(score_bound))
        return VITINT_ERR_WORKSPACE;
    const int cb = codes_container(p_out);
    int qn, qp;
    code_range(p_out->bits, 0, &qn, &qp);
    const int vec_p = (p_f32 && aligned16(p_f32) && ld_p % 4 == 0) ? 1 : 0;
    cudaStream_t st = (cudaStream_t)stream;
    float* table = (float*)workspace;
    if (!table_ready) {
        launch_kernel(exp_table_kernel, dim3((2 * score_bound + 1 + 255) / 256), dim3(256), 0, st, table, (int)score_bound, c);
        if (int rc = cuda_status(cudaGetLastError())) return rc;
    }
    uint8_t* o = (uint8_t*)p_out->data;
    if (cb == 2) return launch_softmax_table<2>(s, rows, cols, ld_s, table, score_bound, p_step, o, p_out->pitch_bytes, p_f32, ld_p, (float)qp, vec_p, st);
    if (cb == 4) return launch_softmax_table<4>(s, rows, cols, ld_s, table, score_bound, p_step, o, p_out->pitch_bytes, p_f32, ld_p, (float)qp, vec_p, st);
    return launch_softmax_table<8>(s, rows, cols, ld_s, table, score_bound, p_step, o, p_out->pitch_bytes, p_f32, ld_p, (float)qp, vec_p, st);
}
