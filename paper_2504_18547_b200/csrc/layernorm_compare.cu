// Quantizing LayerNorm of Section IV-C: the running statistics of Eq. 5 and the division- and
// square-root-free comparator of Fig. 5(b), as two kernels.
//
//   ln_running_stats_kernel    one thread per row walks the row in order:
//                                delta = x_i - mu;  mu += delta / i;  S += delta * (x_i - mu)
//                              every operation a single round-to-nearest fp32 one (no contraction), the
//                              division by i exact-rounded through a reciprocal and one correction step.
//                              Writes (mu, V = S + n*eps) per row.
//   ln_compare_quantize_kernel level = Qn + number of references exceeded.  With d = x - mu (negated where
//                              gamma < 0) the sign logic of the figure collapses into one comparison of
//                              signed squares,  copysign(d*d, d) > V * r,  r = sgn(c) c^2 / n the caller's
//                              signed reference.  The references of a column ascend, fp32 multiplication
//                              by V > 0 keeps their order, so the comparisons are true up to some index
//                              and false after it: the count is found by bisection (b comparisons for
//                              2^b - 1 references) with the candidate references kept in registers.
#include "common.cuh"
#include "ptx.cuh"

namespace vitint {
namespace {

constexpr int LNC_ROWS_PER_THREAD = 16;
constexpr int LNC_BATCH = 4;            // rows whose loads are issued together

constexpr int LNS_MAX_COLS = 4096;    // (float(i), RN(1/i)) pairs tabulated in shared memory

// One step of Eq. 5 for element xi, i = fi: every operation a single rounded fp32 one.  The update of S
// belonging to the PREVIOUS element (its delta in pd, its value in px; mu is still that element's mean) is
// written between the operations of this element's dependent chain delta -> quotient -> mu, so the two
// interleave in issue order; operands and operations are exactly those of the recurrence.
__device__ __forceinline__ void running_step(float xi, float fi, float r, float& mu, float& S, float& pd, float& px) {
    const float delta = __fadd_rn(xi, -mu);
    const float tt = __fadd_rn(px, -mu);
    // RN(delta / i): q0 = RN(delta*r), remainder exact in one FMA, one correction
    const float q0 = __fmul_rn(delta, r);
    const float pp = __fmul_rn(pd, tt);
    const float rem = __fmaf_rn(-q0, fi, delta);
    S = __fadd_rn(S, pp);
    const float q = __fmaf_rn(rem, r, q0);
    mu = __fadd_rn(mu, q);
    pd = delta;
    px = xi;
}

// One warp per 32 rows, a thread walks one row -- but the row reaches the thread through shared memory: the warp
// copies a 128-column chunk of its 32 rows with coalesced 16-byte asynchronous copies (lane l takes the l-th float4 of
// every row: 512 contiguous bytes per row) into a [32][132]-float buffer, and each thread then reads its own row from
// there (132 floats per row: the lanes' 16-byte reads fall on different bank groups).  Read straight from global
// memory, every load instruction of the warp touched 32 different lines, and the load path took as long as the
// dependent chain itself.  Two buffers: the next chunk is on its way while this one is walked.
constexpr int LNS_CHUNK = 128;                 // columns per staged chunk
constexpr int LNS_ROW_FLOATS = LNS_CHUNK + 4;  // padded row of the staging buffer
__global__ void __launch_bounds__(32)
ln_running_stats_kernel(const float* __restrict__ x, int64_t rows, int cols, int64_t ldx, float n_eps,
                        float* __restrict__ stats) {
    // (float(i), RN(1/i)) for every column: one broadcast shared-memory read per element instead of a
    // conversion and a reciprocal (both run on the quarter-rate unit) in front of the dependent chain
    extern __shared__ __align__(16) float2 inv_tab[];
    float* const stage = reinterpret_cast<float*>(inv_tab + ((cols + 1) & ~1));          // 16-byte aligned behind the table
    const int lane = threadIdx.x;
    for (int i = lane; i < cols; i += 32) {
        const float fi = (float)(i + 1);
        inv_tab[i] = make_float2(fi, __frcp_rn(fi));
    }
    __syncwarp();
    grid_dependency_wait();        // x may come from the previous kernel of the stream
    grid_dependency_launch();
    const int64_t row0 = (int64_t)blockIdx.x * 32;
    const int n_chunks = (cols + LNS_CHUNK - 1) / LNS_CHUNK;
    auto request = [&](int c, float* buf) {
        const int col = c * LNS_CHUNK + lane * 4;
        if (col < cols) {                                                              // cols is a multiple of 4
#pragma unroll 8
            for (int r = 0; r < 32; ++r) {
                const int64_t row = row0 + r < rows ? row0 + r : rows - 1;             // a surplus row repeats the last one
                ptx::cp_async16(ptx::smem_addr(buf + r * LNS_ROW_FLOATS + lane * 4), x + row * ldx + col);
            }
        }
        ptx::cp_async_commit();
    };
    float mu = 0.0f, S = 0.0f, pd = 0.0f, px = 0.0f;
    request(0, stage);
    for (int c = 0; c < n_chunks; ++c) {
        float* const buf = stage + (c & 1) * 32 * LNS_ROW_FLOATS;
        if (c + 1 < n_chunks) {
            request(c + 1, stage + ((c + 1) & 1) * 32 * LNS_ROW_FLOATS);
            ptx::cp_async_wait<1>();
        } else {
            ptx::cp_async_wait<0>();
        }
        __syncwarp();                                                                  // every lane's copies have landed
        const float4* mine = reinterpret_cast<const float4*>(buf + lane * LNS_ROW_FLOATS);
        const float2* tab = inv_tab + c * LNS_CHUNK;
        const int nv = (cols - c * LNS_CHUNK < LNS_CHUNK ? cols - c * LNS_CHUNK : LNS_CHUNK) >> 2;
        if (nv == LNS_CHUNK / 4) {
#pragma unroll 8
            for (int v = 0; v < LNS_CHUNK / 4; ++v) {
                const float4 e4 = mine[v];
                const float e[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 t = tab[4 * v + j];
                    running_step(e[j], t.x, t.y, mu, S, pd, px);
                }
            }
        } else {
            for (int v = 0; v < nv; ++v) {
                const float4 e4 = mine[v];
                const float e[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 t = tab[4 * v + j];
                    running_step(e[j], t.x, t.y, mu, S, pd, px);
                }
            }
        }
        __syncwarp();                                                                  // the buffer is free for the chunk after next
    }
    S = __fadd_rn(S, __fmul_rn(pd, __fadd_rn(px, -mu)));      // the last element's term
    const int64_t row = row0 + lane;
    if (row < rows) {
        stats[2 * row] = mu;
        stats[2 * row + 1] = __fadd_rn(S, n_eps);
    }
}

// Block (32, 4): lane = four adjacent columns, threadIdx.y = a group of LNC_ROWS_PER_THREAD rows.
template <int BITS, int C>
__global__ void __launch_bounds__(128)
ln_compare_quantize_kernel(const float* __restrict__ x, int64_t rows, int cols, int64_t ldx,
                           const float* __restrict__ refs, const uint8_t* __restrict__ flip,
                           const float* __restrict__ stats, uint8_t* __restrict__ out, int64_t pitch, int qn) {
    grid_dependency_wait();
    grid_dependency_launch();
    constexpr int NT = (1 << BITS) - 1;
    constexpr int LANES_PER_WORD = 8 / C;                       // lanes whose 4 codes share one 32-bit word
    const int lane = threadIdx.x;
    const int col = (blockIdx.x * 32 + lane) * 4;
    const bool col_ok = col < cols;                             // cols is a multiple of 4
    float r[4][NT];
    float sgn[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        sgn[j] = (col_ok && flip && flip[col + j]) ? -1.0f : 1.0f;
#pragma unroll
        for (int t = 0; t < NT; ++t) r[j][t] = col_ok ? __ldg(refs + (int64_t)(col + j) * NT + t) : 0.0f;
    }
    const int words_per_row = (int)(pitch / 4);
    const int word = (blockIdx.x * 32 + lane) / LANES_PER_WORD;
    const int64_t row0 = ((int64_t)blockIdx.y * 4 + threadIdx.y) * LNC_ROWS_PER_THREAD;
    // Rows go in batches of LNC_BATCH: the loads of the next batch are in flight while this batch's levels are
    // found (a single row per thread would leave too few bytes in flight to keep HBM busy).
    float4 xb[LNC_BATCH], xb_next[LNC_BATCH];
    float2 mb[LNC_BATCH], mb_next[LNC_BATCH];
    auto load_batch = [&](int64_t first, float4 (&xv)[LNC_BATCH], float2 (&mv)[LNC_BATCH]) {
#pragma unroll
        for (int k = 0; k < LNC_BATCH; ++k) {
            const int64_t row = first + k;
            const bool ok = row < rows && row < row0 + LNC_ROWS_PER_THREAD;
            mv[k] = ok ? __ldg(reinterpret_cast<const float2*>(stats) + row) : make_float2(0.f, 1.f);
            xv[k] = (ok && col_ok) ? __ldg(reinterpret_cast<const float4*>(x + row * ldx + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    load_batch(row0, xb_next, mb_next);
    for (int rb = 0; rb < LNC_ROWS_PER_THREAD; rb += LNC_BATCH) {
        if (row0 + rb >= rows) break;                            // uniform across the warp
#pragma unroll
        for (int k = 0; k < LNC_BATCH; ++k) { xb[k] = xb_next[k]; mb[k] = mb_next[k]; }
        load_batch(row0 + rb + LNC_BATCH, xb_next, mb_next);
#pragma unroll
      for (int k = 0; k < LNC_BATCH; ++k) {
        const int64_t row = row0 + rb + k;
        if (row >= rows) break;                                  // uniform across the warp
        const float4 xv = xb[k];
        const float mu = mb[k].x, V = mb[k].y;
        const float e[4] = {xv.x, xv.y, xv.z, xv.w};
        uint32_t bits = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float d = __fmul_rn(__fadd_rn(e[j], -mu), sgn[j]);        // exact sign change
            const float ds = copysignf(__fmul_rn(d, d), d);
            float cand[NT > 1 ? NT / 2 : 1];
            int cnt = 0;
            {
                constexpr int half = (NT + 1) / 2;
                const bool p = ds > __fmul_rn(V, r[j][half - 1]);
                cnt = p ? half : 0;
#pragma unroll
                for (int i = 0; i < half - 1; ++i) cand[i] = p ? r[j][i + half] : r[j][i];
            }
#pragma unroll
            for (int half = (NT + 1) / 4; half >= 1; half >>= 1) {
                const bool p = ds > __fmul_rn(V, cand[half - 1]);
                cnt += p ? half : 0;
#pragma unroll
                for (int i = 0; i < half - 1; ++i) cand[i] = p ? cand[i + half] : cand[i];
            }
            bits |= ((uint32_t)(qn + cnt) & ((1u << C) - 1u)) << (C * j);
        }
        if (!col_ok) bits = 0;
        // gather 8/C neighbouring lanes into one 32-bit word
        if (C == 4) {
            bits |= __shfl_xor_sync(0xffffffffu, bits, 1) << 16;
        } else if (C == 2) {
            bits |= __shfl_xor_sync(0xffffffffu, bits, 1) << 8;
            bits |= __shfl_xor_sync(0xffffffffu, bits, 2) << 16;
        }
        if ((lane % LANES_PER_WORD) == 0 && word < words_per_row)
            *reinterpret_cast<uint32_t*>(out + row * pitch + (int64_t)word * 4) = bits;
      }
    }
}

template <int BITS>
int launch_ln_compare(int c, dim3 grid, cudaStream_t st, const float* x, int64_t rows, int cols, int64_t ldx,
                      const float* refs, const uint8_t* flip, const float* stats, uint8_t* out, int64_t pitch, int qn) {
    const dim3 block(32, 4);
    if (c == 2)
        launch_kernel(ln_compare_quantize_kernel<BITS, 2>, grid, block, 0, st, x, rows, cols, ldx, refs, flip, stats, out, pitch, qn);
    else if (c == 4)
        launch_kernel(ln_compare_quantize_kernel<BITS, 4>, grid, block, 0, st, x, rows, cols, ldx, refs, flip, stats, out, pitch, qn);
    else
        launch_kernel(ln_compare_quantize_kernel<BITS, 8>, grid, block, 0, st, x, rows, cols, ldx, refs, flip, stats, out, pitch, qn);
    return cuda_status(cudaGetLastError());
}

}  // namespace
}  // namespace vitint

using namespace vitint;

extern "C" int vitint_layernorm_compare_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx,
                                                 const float* refs, const uint8_t* flip, float n_eps,
                                                 const vitint_codes* out, float* stats, void* stream) {
    if (!x || !refs || !out || !stats) return VITINT_ERR_INVALID_ARG;
    if (int rc = check_codes(out)) return rc;
    if (rows <= 0 || cols <= 0 || ldx < cols || out->rows != rows || out->cols != cols) return VITINT_ERR_INVALID_ARG;
    if (!(n_eps > 0.0f && n_eps < INFINITY)) return VITINT_ERR_INVALID_ARG;
    if (out->bits == 8 || cols % 4 != 0 || cols > LNS_MAX_COLS) return VITINT_ERR_UNSUPPORTED;
    if (!aligned16(x) || ldx % 4 != 0 || (reinterpret_cast<uintptr_t>(stats) & 7u) != 0) return VITINT_ERR_ALIGNMENT;
    const int c = codes_container(out);
    // one lane covers four columns; with sub-byte containers 8/c lanes share an output word, and the words up
    // to the pitch are written (as zero) by the lanes past the last column
    const int64_t lanes_cols = cols / 4, lanes_pitch = (out->pitch_bytes / 4) * (8 / c);
    const int64_t lanes = lanes_cols > lanes_pitch ? lanes_cols : lanes_pitch;
    int qn, qp;
    code_range(out->bits, out->is_signed, &qn, &qp);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t stats_smem = (size_t)((cols + 1) & ~(int64_t)1) * sizeof(float2) + 2 * 32 * LNS_ROW_FLOATS * sizeof(float);
    if (stats_smem > 48 * 1024 &&
        cudaFuncSetAttribute(ln_running_stats_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stats_smem) != cudaSuccess)
        return VITINT_ERR_CUDA;
    launch_kernel(ln_running_stats_kernel, dim3((unsigned)((rows + 31) / 32)), dim3(32), stats_smem, st, x, rows, (int)cols, ldx,
                  n_eps, stats);
    if (int rc = cuda_status(cudaGetLastError())) return rc;
    const int64_t row_groups = (rows + 4 * LNC_ROWS_PER_THREAD - 1) / (4 * LNC_ROWS_PER_THREAD);
    if (row_groups > 65535) return VITINT_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)((lanes + 31) / 32), (unsigned)row_groups);
    uint8_t* o = (uint8_t*)out->data;
    switch (out->bits) {
        case 2: return launch_ln_compare<2>(c, grid, st, x, rows, (int)cols, ldx, refs, flip, stats, o, out->pitch_bytes, qn);
        case 3: return launch_ln_compare<3>(c, grid, st, x, rows, (int)cols, ldx, refs, flip, stats, o, out->pitch_bytes, qn);
        default: return launch_ln_compare<4>(c, grid, st, x, rows, (int)cols, ldx, refs, flip, stats, o, out->pitch_bytes, qn);
    }
}
