// Integer contraction through the FP4 tensor-core kind (tcgen05 kind::mxf4, e2m1 operands, unit block
// scales, fp32 accumulators): the one route on this hardware to a multiply-accumulate rate above the
// int8 one for very low-bit codes (Section V-B: fewer bits, cheaper MAC).
//
// e2m1 represents 0, 1/2, 1, 3/2, 2, 3, 4, 6 and their negatives, so signed codes of up to 3 bits
// (-4 .. 3) and unsigned codes of up to 2 bits (0 .. 3) are exact operands; products are integers of
// magnitude <= 12 and a sum over K terms stays below 2^24 for K <= 2^20, i.e. inside what an fp32
// accumulator holds exactly.  Whether the tensor core's accumulation really is exact for such sums is a
// property of the hardware; tests/test_gpu_e2m1.py checks it by brute force against the integer oracle.
//
// This is a correctness-first kernel (one CTA per 128 x 256 output tile, operands staged by the threads
// themselves, MMAs issued stage by stage): it exists to establish exactness; the rate such a kind
// offers is measured separately by issuing MMAs back to back.
#include "common.cuh"
#include "ptx.cuh"
#include "tile_ops.cuh"

namespace vitint {
namespace {

constexpr int E_BM = 128, E_BN = 256, E_BK = 256;      // K elements per stage = 128 bytes of packed nibbles
constexpr int E_THREADS = 256;

// Instruction descriptor of the block-scaled FP4 kind: A and B e2m1 (format 1 in [7,10) and [10,13)), both K
// contiguous, N >> 3 in [17,23), scale format ue8m0 in bit 23, M >> 4 in [24,29), scale-factor ids 0, K = 64.
__host__ __device__ inline uint32_t idesc_mxf4(int m, int n) {
    return (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ void mma_mxf4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n\t"
        "}" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}

// Integer code (-4 .. 4) -> e2m1 nibble: magnitudes 0, 1, 2, 3, 4 are the codes 0, 2, 4, 5, 6; bit 3 is the sign.
__device__ __forceinline__ uint32_t e2m1_nibble(int v) {
    const int m = v < 0 ? -v : v;
    return ((0x65420u >> (4 * m)) & 0xFu) | (v < 0 ? 8u : 0u);
}

// One stage of one operand: `rows` rows of E_BK codes (one int8 per code in global memory, K contiguous) ->
// rows of 128 bytes of packed nibbles (element 2i in the low half of byte i), 128-byte swizzle.  Rows or
// columns past the matrix are zero.
__device__ __forceinline__ void stage_operand(const int8_t* __restrict__ src, long long pitch, int row0, int n_rows,
                                              int k0, int K, uint8_t* dst, int rows, int tid) {
    for (int q = tid; q < rows * 8; q += E_THREADS) {          // one 16-byte chunk = 32 codes
        const int r = q >> 3, c = q & 7;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        if (row0 + r < n_rows) {
            const int8_t* p = src + (long long)(row0 + r) * pitch + k0 + c * 32;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int v = (k0 + c * 32 + i < K) ? (int)p[i] : 0;
                w[i >> 3] |= e2m1_nibble(v) << (4 * (i & 7));
            }
        }
        *reinterpret_cast<uint4*>(dst + r * 128 + ((c ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

__global__ void __launch_bounds__(E_THREADS, 1)
linear_e2m1_kernel(const int8_t* __restrict__ a, long long pitch_a, const int8_t* __restrict__ b, long long pitch_b,
                   int M, int N, int K, int32_t* __restrict__ out, long long ld_out, int* __restrict__ inexact) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem_gen = smem_raw + (smem_base - ptx::smem_addr(smem_raw));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        abort_flag = 0;
        ptx::mbar_init(ptx::smem_addr(&bar), 1);
        ptx::fence_mbar_init();
    }
    if (warp == 0) { ptx::tmem_alloc(ptx::smem_addr(&tmem_slot), 512); ptx::tmem_relinquish(); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = tmem_slot;
    // Unit block scales: ue8m0 127 = 2^0 in every byte of the 32 columns behind the accumulator; both scale
    // operands point there, so whichever bytes the hardware picks for a row and a K block, the factor is 1.
    const uint32_t sf_tmem = tmem + 256u;
    if (warp < 4) {
        uint32_t ones[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) ones[i] = 0x7F7F7F7Fu;
        ptx::tmem_st32(sf_tmem + ((uint32_t)(warp * 32) << 16), ones);
        ptx::tmem_st_wait();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const int m0 = blockIdx.y * E_BM, n0 = blockIdx.x * E_BN;
    uint8_t* const sa = smem_gen;
    uint8_t* const sb = smem_gen + E_BM * 128;
    const uint32_t idesc = idesc_mxf4(E_BM, E_BN);
    const int k_stages = (K + E_BK - 1) / E_BK;
    bool ok = true;
    for (int ks = 0; ks < k_stages; ++ks) {
        stage_operand(a, pitch_a, m0, M, ks * E_BK, K, sa, E_BM, tid);
        stage_operand(b, pitch_b, n0, N, ks * E_BK, K, sb, E_BN, tid);
        ptx::fence_proxy_async_smem();
        __syncthreads();
        if (tid == 0) {
            ptx::tc_fence_after();
            const uint64_t a_desc = ptx::smem_desc(smem_base, 16, 1024, ptx::SWIZZLE_128B);
            const uint64_t b_desc = ptx::smem_desc(smem_base + E_BM * 128, 16, 1024, ptx::SWIZZLE_128B);
            const int k_left = K - ks * E_BK;
            const int steps = k_left >= E_BK ? 4 : (k_left + 63) / 64;          // 64 codes = 32 bytes per MMA
            for (int k = 0; k < steps; ++k)
                mma_mxf4(tmem, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 2), idesc, sf_tmem, sf_tmem,
                         (ks | k) != 0 ? 1u : 0u);
            ptx::mma_commit(ptx::smem_addr(&bar));
        }
        // the stage's MMAs have read shared memory once the commit arrives: only then may it be refilled
        ok = mbar_wait(ptx::smem_addr(&bar), (uint32_t)ks & 1u, &abort_flag);
        if (!__syncthreads_and(ok ? 1 : 0)) { ok = false; break; }
    }
    if (ok && warp < 4) {
        ptx::tc_fence_after();
        const int row = m0 + warp * 32 + lane;
        for (int c0 = 0; c0 < E_BN; c0 += 32) {
            uint32_t v[32];
            ptx::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
            ptx::tmem_ld_wait();
            if (row < M) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int n = n0 + c0 + i;
                    if (n < N) {
                        const float f = __uint_as_float(v[i]);
                        const float r = rintf(f);
                        if (r != f) atomicExch(inexact, 1);          // an accumulator that is not an integer
                        out[(long long)row * ld_out + n] = (int32_t)r;
                    }
                }
            }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) { ptx::tc_fence_after(); __syncwarp(); ptx::tmem_dealloc(tmem, 512); }
}

}  // namespace
}  // namespace vitint

using namespace vitint;

extern "C" int vitint_linear_e2m1(const vitint_codes* x, const vitint_codes* w, int32_t* out, int64_t ld_out,
                                  int32_t* inexact_flag, void* stream) {
    if (int rc = check_codes(x)) return rc;
    if (int rc = check_codes(w)) return rc;
    if (!out || !inexact_flag || x->cols != w->cols || ld_out < w->rows) return VITINT_ERR_INVALID_ARG;
    // operands: one code per byte, values representable in e2m1
    auto representable = [](const vitint_codes* c) { return c->is_signed ? c->bits <= 3 : c->bits <= 2; };
    if (codes_container(x) != 8 || codes_container(w) != 8 || !representable(x) || !representable(w))
        return VITINT_ERR_UNSUPPORTED;
    if (x->rows > 0x7fffffff || w->rows > 0x7fffffff || x->cols > (1 << 20)) return VITINT_ERR_UNSUPPORTED;
    const int M = (int)x->rows, N = (int)w->rows, K = (int)x->cols;
    const dim3 grid((N + E_BN - 1) / E_BN, (M + E_BM - 1) / E_BM);
    if (grid.y > 65535) return VITINT_ERR_UNSUPPORTED;
    const size_t smem = (size_t)(E_BM + E_BN) * 128 + 1024;
    const int dev = current_device();
    if (dev < 0) return VITINT_ERR_CUDA;
    static bool attr_set[MAX_DEVICES] = {};
    if (!attr_set[dev]) {
        // more than half of the shared memory: two CTAs (two 512-column tensor-memory allocations) never share an SM
        if (cudaFuncSetAttribute(linear_e2m1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024) != cudaSuccess)
            return VITINT_ERR_CUDA;
        attr_set[dev] = true;
    }
    launch_kernel(linear_e2m1_kernel, grid, dim3(E_THREADS), smem < 120 * 1024 ? (size_t)120 * 1024 : smem,
                  (cudaStream_t)stream, (const int8_t*)x->data, (long long)x->pitch_bytes, (const int8_t*)w->data,
                  (long long)w->pitch_bytes, M, N, K, out, (long long)ld_out, inexact_flag);
    return cuda_status(cudaGetLastError());
}
