// a4 + a5 + a6 fused: per (image, head, 128-query tile)  S = Q K^T  ->  softmax + quantize  ->
// O = P V  ->  requantize, with S, the probabilities and P never leaving the SM.
//
// A persistent CTA runs TWO independent pipelines ("groups"), each with four compute warps
// (thread = query row = TMEM lane) and one control warp (TMA + MMA issue); while one group's
// threads are busy with the softmax the other group's loads and MMAs proceed.
//
// Per item and group:
//   control   TMA: packed Q [128 x 64], K [T x 64], V [T x 64] code slabs -> shared memory
//   compute   unpack to int8 operand tiles (rows of 64 bytes, 64-byte swizzle)
//   control   tcgen05.mma  S[128, T] = Q K^T   (K = 64: two MMAs) into TMEM
//   compute   e_j = EXP[S_j] from a table of exp(fl32(s*c)) over every possible integer score
//             (|S| <= 64*max|q|*max|k|: 8193 entries for 4-bit codes); row sum in fp64;
//             p_j = e_j / Z;  code = clamp(rint(p_j / s_P));  codes written as int8 rows (128-byte
//             swizzle) = the A operand of P V.  e_j is parked in TMEM over S between the passes.
//   control   tcgen05.mma  O[128, 64] = P V  (V is the N-contiguous B operand) into TMEM
//   compute   requantize O, pack, store the head's 64 columns of the [M, D] code matrix
//
// Softmax accuracy: exp(t_j)/sum_k exp(t_k) equals Eq. 3's softmax exactly (the maximum is only
// subtracted there for range); every table entry is a correctly rounded fp32, the sum is fp64,
// and p_j = RN(e_j * (1/Z)) with 1/Z carried as two floats, so p_j stays within 2 ulp.
// The host only selects this kernel when smax*|c| <= 80 (no overflow without max subtraction).
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"
#include "tile_ops.cuh"

namespace vitint {
namespace {

constexpr int AT_GROUPS = 2;
constexpr int AT_COMPUTE_WARPS = 8;   // two warps per TMEM lane quarter: a query row is shared by two threads
constexpr int AT_THREADS = (AT_GROUPS * AT_COMPUTE_WARPS + AT_GROUPS) * 32;   // 576

struct AttnParams {
    int batch, heads, tokens, q_tiles, total_items;
    int c;                       // container bits of Q, K, V (2 or 4: packed, unpacked in the kernel; 8: one code per byte,
                                 // the TMA copy is the tensor-core operand)
    int n_k;                     // MMA N of Q K^T: tokens rounded up to 16
    int kv_rows;                 // tokens rounded up to 32: K extent of P V, rows of the V tile
    int smax;                    // table covers scores -smax .. smax
    int part_bytes;              // bytes of one of the Q / K / V column blocks in a QKV row
    uint32_t off_table, off_ftab, off_group, group_bytes;         // shared-memory layout
    uint32_t off_pq, off_pk, off_pv, off_q, off_k, off_v, off_p, off_col, off_z, off_mx;   // within a group
    const float* table;          // global copy of the exp table, 2*smax+1 floats
    uint32_t ftab_word;          // Eq. 4: word offset of the 16-bit table of integer parts behind the 32-bit table
    float p_step, p_qp;
    const float* alpha_o;        // [D]
    const float* beta_o;         // [D] or null
    int out_c;
    float out_qn, out_qp;
    uint8_t* out;
    long long out_pitch;
};

struct AttnBars {
    uint64_t packed_full, v_full, ops_ready, s_full, p_ready, o_full, o_done, grp_sync, z_sync;
};

// Eq. 4's split of every integer score: z = fl32(s * c2), f = floor z (16-bit table behind the 32-bit one),
// M = trunc((1 + (z - f)) * 2^23), the 24-bit mantissa of 2^r ~ 1 + r (2^24 in the one case where 1 + r rounds to 2).
__global__ void shift_table_kernel(uint32_t* mtab, short* ftab, int smax, float c2) {
    grid_dependency_wait();        // an earlier kernel may still read the table
    grid_dependency_launch();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i > 2 * smax) return;
    const float z = __fmul_rn((float)(i - smax), c2);
    const float fl = floorf(z);
    const float res = __fsub_rn(z, fl);
    mtab[i] = (uint32_t)__fmul_rn(__fadd_rn(1.0f, res), 8388608.0f);
    ftab[i] = (short)(int)fl;
}

// exp(fl32(s * c)) for every integer score, correctly rounded to fp32 (fp64 exp, one rounding).
__global__ void exp_table_kernel(float* table, int smax, float c) {
    grid_dependency_wait();        // an earlier kernel may still read the table
    grid_dependency_launch();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i > 2 * smax) return;
    const float t = __fmul_rn((float)(i - smax), c);
    table[i] = (float)exp((double)t);
}

// SHIFT: the softmax of Eq. 4 (2^z with z split into integer part and residual, 2^r ~ 1 + r, integer shifts, the
// division-free comparator quantizer) instead of exp.  With integer scores of bounded range the pair (floor z,
// mantissa of 1 + r) is one table entry per score, so the arithmetic left per score is the shift, the exact 64-bit
// row sum and the comparison against references scaled by that sum -- every step an integer or a single fp32
// operation in the order of the stand-alone kernel, hence the same codes bit for bit.
template <int C, bool SHIFT>
__global__ void __launch_bounds__(AT_THREADS, 1)
attention_fused_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv,
                       const __grid_constant__ AttnParams P) {
    static_assert(!SHIFT || C == 8, "the Eq. 4 variant takes byte-stored codes");
    extern __shared__ uint8_t smem_raw[];
    __shared__ AttnBars bars[AT_GROUPS];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem_gen = smem_raw + (smem_base - ptx::smem_addr(smem_raw));
    volatile int* abort_ptr = &abort_flag;
    const bool is_control = warp >= AT_GROUPS * AT_COMPUTE_WARPS;
    const int g = is_control ? warp - AT_GROUPS * AT_COMPUTE_WARPS : warp / AT_COMPUTE_WARPS;
    AttnBars& B = bars[g];
    const uint32_t gbase = smem_base + P.off_group + (uint32_t)g * P.group_bytes;
    uint8_t* const ggen = smem_gen + P.off_group + (size_t)g * P.group_bytes;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int k = 0; k < AT_GROUPS; ++k) {
            ptx::mbar_init(ptx::smem_addr(&bars[k].packed_full), 1);
            ptx::mbar_init(ptx::smem_addr(&bars[k].v_full), 1);
            ptx::mbar_init(ptx::smem_addr(&bars[k].ops_ready), AT_COMPUTE_WARPS);
            ptx::mbar_init(ptx::smem_addr(&bars[k].s_full), 1);
            ptx::mbar_init(ptx::smem_addr(&bars[k].p_ready), AT_COMPUTE_WARPS);
            ptx::mbar_init(ptx::smem_addr(&bars[k].o_full), 1);
            ptx::mbar_init(ptx::smem_addr(&bars[k].o_done), AT_COMPUTE_WARPS);
            ptx::mbar_init(ptx::smem_addr(&bars[k].grp_sync), AT_COMPUTE_WARPS * 32);
            ptx::mbar_init(ptx::smem_addr(&bars[k].z_sync), AT_COMPUTE_WARPS * 32);
        }
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == AT_GROUPS * AT_COMPUTE_WARPS) {          // first control warp owns the TMEM allocation
        ptx::tmem_alloc(ptx::smem_addr(&tmem_base_slot), 512);
        ptx::tmem_relinquish();
    }
    grid_dependency_wait();        // the table and the codes come from earlier kernels of the stream
    grid_dependency_launch();
    // the exp table: global -> shared, once per CTA
    {
        float* tab = reinterpret_cast<float*>(smem_gen + P.off_table);
        for (int i = threadIdx.x; i <= 2 * P.smax; i += AT_THREADS) tab[i] = __ldg(P.table + i);
        if constexpr (SHIFT) {
            // the 16-bit table of integer parts sits behind the 32-bit one, in the workspace and here
            const uint32_t* src = reinterpret_cast<const uint32_t*>(P.table) + P.ftab_word;
            uint32_t* dst = reinterpret_cast<uint32_t*>(smem_gen + P.off_ftab);
            for (int i = threadIdx.x; i <= P.smax; i += AT_THREADS) dst[i] = __ldg(src + i);
        }
    }
    if (is_control && lane == 0) { ptx::prefetch_tensormap(&map_q); ptx::prefetch_tensormap(&map_kv); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_grp = tmem_base_slot + (uint32_t)g * 256u;

    const int T = P.tokens;
    const int item0 = blockIdx.x * AT_GROUPS + g, item_stride = gridDim.x * AT_GROUPS;
    constexpr bool DIRECT = (C == 8);                  // byte codes: no packed staging, no unpack
    const int head_bytes = 8 * C;                      // 64 codes
    const uint32_t q_bytes = 128u * head_bytes, kv_bytes = (uint32_t)P.kv_rows * head_bytes;   // TMA boxes

    auto item_coords = [&](int item, int& b, int& h, int& qt) {
        qt = item % P.q_tiles;
        const int bh = item / P.q_tiles;
        h = bh % P.heads;
        b = bh / P.heads;
    };

    if (is_control) {
        // --------------------------- control: TMA + MMA issue ----------------------------
        if (lane == 0) {
            // packed codes: one barrier for the three slabs, which the compute warps unpack.
            // byte codes: Q and K land in their operand tiles under packed_full, V under v_full, so that each
            // buffer is refilled as soon as the MMA that read it has completed.
            auto issue_loads = [&](int item) {
                int b, h, qt;
                item_coords(item, b, h, qt);
                const uint32_t bar = ptx::smem_addr(&B.packed_full);
                ptx::mbar_arrive_expect_tx(bar, q_bytes + (DIRECT ? 1u : 2u) * kv_bytes);
                ptx::tma_load_3d(gbase + (DIRECT ? P.off_q : P.off_pq), &map_q, bar, h * head_bytes, qt * 128, b);
                ptx::tma_load_3d(gbase + (DIRECT ? P.off_k : P.off_pk), &map_kv, bar, P.part_bytes + h * head_bytes, 0, b);
                if (!DIRECT) ptx::tma_load_3d(gbase + P.off_pv, &map_kv, bar, 2 * P.part_bytes + h * head_bytes, 0, b);
            };
            auto issue_v = [&](int item) {
                int b, h, qt;
                item_coords(item, b, h, qt);
                const uint32_t bar = ptx::smem_addr(&B.v_full);
                ptx::mbar_arrive_expect_tx(bar, kv_bytes);
                ptx::tma_load_3d(gbase + P.off_v, &map_kv, bar, 2 * P.part_bytes + h * head_bytes, 0, b);
            };
            const uint32_t idesc_qk = ptx::idesc_i8(128, P.n_k, 1, 1, 0);
            const uint32_t idesc_pv = ptx::idesc_i8(128, 64, 0, 1, 1);
            const uint64_t q_desc = ptx::smem_desc(gbase + P.off_q, 16, 512, ptx::SWIZZLE_64B);
            const uint64_t k_desc = ptx::smem_desc(gbase + P.off_k, 16, 512, ptx::SWIZZLE_64B);
            const uint64_t v_desc = ptx::smem_desc(gbase + P.off_v, 16, 512, ptx::SWIZZLE_64B);
            const int pv_steps = P.kv_rows / 32;
            bool ok = true;
            int pending = -1, pending_v = -1;       // local index of the item whose loads are in flight
            if (item0 < P.total_items) {
                issue_loads(item0); pending = 0;
                if (DIRECT) { issue_v(item0); pending_v = 0; }
            }
            int n = 0;
            for (int item = item0; ok && item < P.total_items; item += item_stride, ++n) {
                const uint32_t ph = (uint32_t)n & 1u;
                const bool has_next = item + item_stride < P.total_items;
                if (DIRECT) {
                    if (!mbar_wait(ptx::smem_addr(&B.packed_full), ph, abort_ptr)) { ok = false; break; }
                    pending = -1;
                } else {
                    if (!mbar_wait(ptx::smem_addr(&B.ops_ready), ph, abort_ptr)) { ok = false; break; }
                    pending = -1;
                    if (has_next) { issue_loads(item + item_stride); pending = n + 1; }
                }
                if (n > 0 && !mbar_wait(ptx::smem_addr(&B.o_done), ph ^ 1u, abort_ptr)) { ok = false; break; }
                ptx::tc_fence_after();
                for (int k = 0; k < 2; ++k)                        // K = 64 -> two MMAs of 32
                    ptx::mma_i8(tmem_grp, q_desc + (uint64_t)(k * 2), k_desc + (uint64_t)(k * 2), idesc_qk, k);
                ptx::mma_commit(ptx::smem_addr(&B.s_full));
                if (DIRECT) {
                    // Q K^T has been read out of the Q and K tiles once s_full completes
                    if (!mbar_wait(ptx::smem_addr(&B.s_full), ph, abort_ptr)) { ok = false; break; }
                    if (has_next) { issue_loads(item + item_stride); pending = n + 1; }
                }
                if (!mbar_wait(ptx::smem_addr(&B.p_ready), ph, abort_ptr)) { ok = false; break; }
                if (DIRECT) {
                    if (!mbar_wait(ptx::smem_addr(&B.v_full), ph, abort_ptr)) { ok = false; break; }
                    pending_v = -1;
                }
                ptx::tc_fence_after();
                for (int ks = 0; ks < pv_steps; ++ks) {
                    const uint64_t p_desc = ptx::smem_desc(gbase + P.off_p + (uint32_t)(ks >> 2) * 16384u, 16, 1024,
                                                           ptx::SWIZZLE_128B) + (uint64_t)((ks & 3) * 2);
                    ptx::mma_i8(tmem_grp, p_desc, v_desc + (uint64_t)(ks * 128), idesc_pv, ks);
                }
                ptx::mma_commit(ptx::smem_addr(&B.o_full));
                if (DIRECT && has_next) {
                    // P V has been read out of the V tile once o_full completes
                    if (!mbar_wait(ptx::smem_addr(&B.o_full), ph, abort_ptr)) { ok = false; break; }
                    issue_v(item + item_stride); pending_v = n + 1;
                }
            }
            if (!ok) {
                // give the copies still in flight a bounded chance to land before the CTA exits
                if (pending >= 0) {
                    const uint32_t bar = ptx::smem_addr(&B.packed_full);
                    for (int spin = 0; spin < (1 << 20) && !ptx::mbar_try_wait(bar, (uint32_t)pending & 1u); ++spin) {}
                }
                if (pending_v >= 0) {
                    const uint32_t bar = ptx::smem_addr(&B.v_full);
                    for (int spin = 0; spin < (1 << 20) && !ptx::mbar_try_wait(bar, (uint32_t)pending_v & 1u); ++spin) {}
                }
            }
        }
    } else {
        // ------------------------------ compute warps ------------------------------------
        const int wq = warp & 3;                                    // TMEM lane quarter
        const int hf = (warp % AT_COMPUTE_WARPS) >> 2;              // which of the row's two threads: even / odd 32-column chunks
        const int tid_g = (warp % AT_COMPUTE_WARPS) * 32 + lane;    // 0..255 within the group
        const int row = wq * 32 + lane;                             // query row of the tile
        double* const zx = reinterpret_cast<double*>(ggen + P.off_z);   // partial row sums, [2][128]
        const uint32_t t_row = tmem_grp + ((uint32_t)(wq * 32) << 16);
        const char* const tab_mid = reinterpret_cast<const char*>(smem_gen + P.off_table) + (size_t)P.smax * 4;
        float* const colp2 = reinterpret_cast<float*>(ggen + P.off_col);  // alpha[64], beta[64] of the head, one copy per item parity
        const int sh_idx = DIRECT ? 0 : 2 * (8 - C) - 2;            // scaled score -> byte offset 4*S
        const int chunks = P.kv_rows / 32;
        const int tab_half = 4 * P.smax;
        const char* const tab_lo = tab_mid - tab_half;
        const double inv_p_step = 1.0 / (double)P.p_step;
        bool ok = true;
        int n = 0;
        for (int item = item0; ok && item < P.total_items; item += item_stride, ++n) {
            const uint32_t ph = (uint32_t)n & 1u;
            int b, h, qt;
            item_coords(item, b, h, qt);
            // the head's output parameters; the copy of the other parity may still be read by a warp that is
            // finishing the previous item, and every reader of this one passes z_sync first
            float* const colp = colp2 + (n & 1) * 128;
            if (tid_g < 64) colp[tid_g] = __ldg(P.alpha_o + h * 64 + tid_g);
            else if (tid_g < 128) colp[tid_g] = P.beta_o ? __ldg(P.beta_o + h * 64 + (tid_g - 64)) : 0.0f;
            bool w = true;
            if constexpr (!DIRECT) {
                // ---- operands: packed -> int8 ---------------------------------------------
                w = mbar_wait(ptx::smem_addr(&B.packed_full), ph, abort_ptr);
                if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
                unpack_rows64<C, 1>(ggen + P.off_pq, ggen + P.off_q, 128, tid_g, AT_COMPUTE_WARPS * 32);
                unpack_rows64<C, 1>(ggen + P.off_pk, ggen + P.off_k, P.n_k, tid_g, AT_COMPUTE_WARPS * 32);
                unpack_rows64<C, 1>(ggen + P.off_pv, ggen + P.off_v, P.kv_rows, tid_g, AT_COMPUTE_WARPS * 32);
                ptx::fence_proxy_async_smem();
                ptx::mbar_arrive(ptx::smem_addr(&B.grp_sync));
                w = mbar_wait(ptx::smem_addr(&B.grp_sync), ph, abort_ptr);
                if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
                if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&B.ops_ready));
            }
            // ---- softmax over the row -------------------------------------------------------
            w = mbar_wait(ptx::smem_addr(&B.s_full), ph, abort_ptr);
            if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
            ptx::tc_fence_after();
            if constexpr (SHIFT) {
                // Two tables over the score range: M[s] = trunc((1 + (z - floor z)) * 2^23) (32-bit) and f[s] = floor z
                // (16-bit), z = fl32(s * c2).  floor z increases with s, so the row's largest score carries the row's
                // largest integer part m and pass 0 needs no lookup at all.
                const int full_chunks = T >> 5;
                const bool warp_live = qt * 128 + wq * 32 < T;
                int* const mx = reinterpret_cast<int*>(ggen + P.off_mx);
                unsigned long long* const sx = reinterpret_cast<unsigned long long*>(ggen + P.off_z);
                const uint32_t* const mtab = reinterpret_cast<const uint32_t*>(smem_gen + P.off_table);
                const short* const ftab = reinterpret_cast<const short*>(smem_gen + P.off_ftab);
                const uint32_t top = (uint32_t)(2 * P.smax);
                // pass 0: the row's largest score
                int smx = INT_MIN;
                for (int ch = hf; warp_live && ch < chunks; ch += 2) {
                    uint32_t v[32];
                    ptx::tmem_ld32(t_row + (uint32_t)(ch * 32), v);
                    ptx::tmem_ld_wait();
                    if (ch < full_chunks) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) smx = max(smx, (int)v[i]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) smx = max(smx, ch * 32 + i < T ? (int)v[i] : INT_MIN);
                    }
                }
                mx[hf * 128 + row] = smx;
                ptx::mbar_arrive(ptx::smem_addr(&B.z_sync));
                w = mbar_wait(ptx::smem_addr(&B.z_sync), 0u, abort_ptr);       // two phases per item: parities 0, 1
                if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
                smx = max(mx[row], mx[128 + row]);
                // pass 1: E_j = M_j << (30 + f_j - m) (>> for the few scores more than 30 octaves down), exact 64-bit
                // row sum, float(E_j) put together from its bits and parked in TMEM over the score
                const int c0 = 30 - (int)ftab[min((uint32_t)(max(smx, -P.smax) + P.smax), top)];
                // Straight-line per score (rows with a wide spread of scores take the right-shift form often, so a
                // branch would mostly run both sides): the 64-bit term is (M * 2^32) >> (32 - sh) with sh kept above
                // -32 (further down everything is shifted out anyway); float(E) is float(M) * 2^sh put together from
                // its bits for sh >= 0, and the conversion of the small remainder by the 2^23 trick otherwise.
                uint32_t sg_lo = 0u, sg_hi = 0u;
                auto term = [&](uint32_t score, bool valid) -> uint32_t {
                    const uint32_t idx = min((uint32_t)((int)score + P.smax), top);
                    const uint32_t m24 = valid ? mtab[idx] : 0u;                       // a real entry is at least 2^23
                    const int sh = max((int)ftab[idx] + c0, -31);
                    const unsigned long long big = ((unsigned long long)m24 << 32) >> (32 - sh);
                    const uint32_t lo = (uint32_t)big, hi = (uint32_t)(big >> 32);
                    asm("add.cc.u32 %0, %0, %2;\n\taddc.u32 %1, %1, %3;" : "+r"(sg_lo), "+r"(sg_hi) : "r"(lo), "r"(hi));
                    const uint32_t up = m24 + 0x4A800000u + ((uint32_t)sh << 23);
                    const uint32_t dn = __float_as_uint(__fadd_rn(__uint_as_float(0x4B000000u + lo), -8388608.0f));
                    return valid ? (sh >= 0 ? up : dn) : 0u;
                };
                for (int ch = hf; warp_live && ch < chunks; ch += 2) {
                    uint32_t v[32];
                    ptx::tmem_ld32(t_row + (uint32_t)(ch * 32), v);
                    ptx::tmem_ld_wait();
                    if (ch < full_chunks) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = term(v[i], true);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = term(v[i], ch * 32 + i < T);      // no score past the last token
                    }
                    ptx::tmem_st32(t_row + (uint32_t)(ch * 32), v);
                }
                unsigned long long sigma = ((unsigned long long)sg_hi << 32) | sg_lo;
                ptx::tmem_st_wait();
                sx[hf * 128 + row] = sigma;
                ptx::mbar_arrive(ptx::smem_addr(&B.z_sync));
                w = mbar_wait(ptx::smem_addr(&B.z_sync), 1u, abort_ptr);
                if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
                sigma = sx[row] + sx[128 + row];
                const float sig_f = __ull2float_rn(sigma);
                // pass 2: the code is the number of references fl32(fl32((k - 1/2) s_P) * Sigma) that float(E_j) exceeds.
                // k0 = rint(min(E_j / (s_P Sigma), Qp - 3/4)) is at most one off and never Qp, so the two references
                // around it decide: code = k0 - 1 + [E > ref(k0)] + [E > ref(k0 + 1)], references formed with the two
                // fp32 multiplications of the definition.  The sum is taken in the float that carries k0 in its low
                // mantissa bits (1.5 * 2^23 - 1 + k0 + the two tests): small integers, exact.
                const float inv = warp_live ? __frcp_rn(__fmul_rn(P.p_step, sig_f)) : 0.0f;
                const float u_top = P.p_qp - 0.75f;
                const f32x2 inv2 = f2_dup(inv), magic2 = f2_dup(12582912.0f), nmagic2 = f2_dup(-12582912.0f), neg1 = f2_dup(-1.0f);
                const f32x2 half2 = f2_dup(0.5f), nhalf2 = f2_dup(-0.5f), ps2 = f2_dup(P.p_step), sg2 = f2_dup(sig_f);
                uint8_t* const prow = ggen + P.off_p + row * 128;
                const int sw = row & 7;
                for (int ch = hf; warp_live && ch < chunks; ch += 2) {
                    uint32_t v[32];
                    ptx::tmem_ld32(t_row + (uint32_t)(ch * 32), v);
                    ptx::tmem_ld_wait();
                    uint32_t wd[8];
#pragma unroll
                    for (int i4 = 0; i4 < 8; ++i4) {
                        uint32_t cb[4];
#pragma unroll
                        for (int j = 0; j < 4; j += 2) {
                            const float e0 = __uint_as_float(v[4 * i4 + j]), e1 = __uint_as_float(v[4 * i4 + j + 1]);
                            float u0, u1;
                            f2_unpack(f2_mul(f2_pack(e0, e1), inv2), u0, u1);
                            const f32x2 um = f2_add(f2_pack(fminf(u0, u_top), fminf(u1, u_top)), magic2);   // 1.5*2^23 + k0
                            const f32x2 kf = f2_add(um, nmagic2);
                            float l0, l1, h0, h1;
                            f2_unpack(f2_mul(f2_mul(f2_add(kf, nhalf2), ps2), sg2), l0, l1);
                            f2_unpack(f2_mul(f2_mul(f2_add(kf, half2), ps2), sg2), h0, h1);
                            const f32x2 t_lo = f2_pack(e0 > l0 ? 1.0f : 0.0f, e1 > l1 ? 1.0f : 0.0f);
                            const f32x2 t_hi = f2_pack(e0 > h0 ? 1.0f : 0.0f, e1 > h1 ? 1.0f : 0.0f);
                            float c0f, c1f;
                            f2_unpack(f2_add(f2_add(um, neg1), f2_add(t_lo, t_hi)), c0f, c1f);
                            cb[j] = __float_as_uint(c0f);                                          // code in the low byte
                            cb[j + 1] = __float_as_uint(c1f);
                        }
                        wd[i4] = __byte_perm(__byte_perm(cb[0], cb[1], 0x4040), __byte_perm(cb[2], cb[3], 0x4040), 0x5410);
                    }
                    const int cc = 2 * ch;
                    uint8_t* const blk = prow + (cc >> 3) * 16384;
                    *reinterpret_cast<uint4*>(blk + (((cc & 7) ^ sw) << 4)) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                    *reinterpret_cast<uint4*>(blk + ((((cc + 1) & 7) ^ sw) << 4)) = make_uint4(wd[4], wd[5], wd[6], wd[7]);
                }
            } else {
            // pass 1: e_j = EXP[S_j] (an integer score is bounded by the code ranges, so the byte offset
            // 4*S always lies inside the table), row sum in fp64, e_j parked in TMEM over S_j
            // four interleaved partial sums: a single fp64 accumulator would chain 32 dependent additions per chunk
            double zp[4] = {0.0, 0.0, 0.0, 0.0};
            const int full_chunks = T >> 5;
            // a warp whose 32 query rows all lie past the last token has nothing to compute: its P rows
            // only feed accumulator rows that are never stored (whatever int8 they hold)
            const bool warp_live = qt * 128 + wq * 32 < T;
            for (int ch = hf; warp_live && ch < chunks; ch += 2) {
                uint32_t v[32];
                ptx::tmem_ld32(t_row + (uint32_t)(ch * 32), v);
                ptx::tmem_ld_wait();
                if (ch < full_chunks) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        // every table entry is a positive normal float (exp of a bounded argument), so its
                        // double is formed from the bits with two integer operations instead of a conversion
                        // (the conversion unit runs at a quarter of the fp64 adder's rate)
                        // Integer multiply-adds run beside the compare / shift / permute unit, which is the busier
                        // one in this kernel: the byte offset, its clamp (one unsigned minimum after biasing) and
                        // both words of the double are formed with them.
                        uint32_t eb;
                        if (DIRECT) {
                            // raw bytes: 4*S + 4*smax, kept inside the table for any operand value
                            const uint32_t off = min((uint32_t)((int)v[i] * 4 + tab_half), (uint32_t)(2 * tab_half));
                            eb = *reinterpret_cast<const uint32_t*>(tab_lo + off);
                        } else {
                            eb = *reinterpret_cast<const uint32_t*>(tab_mid + ((int)v[i] >> sh_idx));
                        }
                        uint32_t hi, lo;
                        asm("mad.hi.u32 %0, %1, 536870912, 939524096;" : "=r"(hi) : "r"(eb));    // (eb >> 3) + 0x38000000
                        asm("mul.lo.u32 %0, %1, 536870912;" : "=r"(lo) : "r"(eb));                // eb << 29
                        zp[i & 3] += __hiloint2double((int)hi, (int)lo);
                        v[i] = eb;
                    }
                } else {
                    // last, partial chunk: columns past the last token hold no score -> no lookup, e = 0
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const bool valid = ch * 32 + i < T;
                        const int off = valid ? (DIRECT ? ((int)v[i] << 2) : ((int)v[i] >> sh_idx)) : 0;
                        uint32_t eb = *reinterpret_cast<const uint32_t*>(tab_mid + max(-tab_half, min(tab_half, off)));
                        if (!valid) eb = 0u;
                        zp[i & 3] += __hiloint2double(valid ? (int)((eb >> 3) + 0x38000000u) : 0, (int)(eb << 29));
                        v[i] = eb;
                    }
                }
                ptx::tmem_st32(t_row + (uint32_t)(ch * 32), v);
            }
            ptx::tmem_st_wait();
            // the row's two threads add their partial sums (every thread takes part in the barrier)
            double z = (zp[0] + zp[1]) + (zp[2] + zp[3]);
            zx[hf * 128 + row] = z;
            ptx::mbar_arrive(ptx::smem_addr(&B.z_sync));
            w = mbar_wait(ptx::smem_addr(&B.z_sync), ph, abort_ptr);
            if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
            z = zx[row] + zx[128 + row];
            // r = 1 / (Z * s_P) as a two-float number: e * r then carries the quantizer argument p / s_P to
            // about half an ulp, i.e. it is the exact-division result for a probability that differs from
            // RN(e / Z) by less than one ulp
            const double rz = warp_live ? inv_p_step / z : 0.0;
            const float rzh = (float)rz;
            const float rzl = (float)(rz - (double)rzh);
            const f32x2 rzh2 = f2_dup(rzh), rzl2 = f2_dup(rzl), magic2 = f2_dup(12582912.0f);
            uint8_t* const prow = ggen + P.off_p + row * 128;
            const int sw = row & 7;
            // pass 2: code = min(rint(e_j / (Z s_P)), Qp) (p >= 0: no lower clamp)
            for (int ch = hf; warp_live && ch < chunks; ch += 2) {
                uint32_t v[32];
                ptx::tmem_ld32(t_row + (uint32_t)(ch * 32), v);
                ptx::tmem_ld_wait();
                uint32_t wd[8];
#pragma unroll
                for (int i4 = 0; i4 < 8; ++i4) {
                    uint32_t cb[4];
#pragma unroll
                    for (int j = 0; j < 4; j += 2) {
                        // two scores per instruction (each half is the scalar IEEE result): e*r_hi + RN(e*r_lo)
                        const f32x2 e2 = f2_pack(__uint_as_float(v[4 * i4 + j]), __uint_as_float(v[4 * i4 + j + 1]));
                        float a0, a1, c0, c1;
                        f2_unpack(f2_fma(e2, rzh2, f2_mul(e2, rzl2)), a0, a1);
                        f2_unpack(f2_add(f2_pack(fminf(a0, P.p_qp), fminf(a1, P.p_qp)), magic2), c0, c1);
                        cb[j] = __float_as_uint(c0);                                           // code in the low byte
                        cb[j + 1] = __float_as_uint(c1);
                    }
                    wd[i4] = __byte_perm(__byte_perm(cb[0], cb[1], 0x4040), __byte_perm(cb[2], cb[3], 0x4040), 0x5410);
                }
                // 32 codes = two 16-byte chunks cc = 2*ch, 2*ch+1 of this row's 256-byte K extent
                const int cc = 2 * ch;
                uint8_t* const blk = prow + (cc >> 3) * 16384;
                *reinterpret_cast<uint4*>(blk + (((cc & 7) ^ sw) << 4)) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                *reinterpret_cast<uint4*>(blk + ((((cc + 1) & 7) ^ sw) << 4)) = make_uint4(wd[4], wd[5], wd[6], wd[7]);
            }
            }   // exp / Eq. 4
            ptx::fence_proxy_async_smem();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&B.p_ready));
            // ---- O = P V: requantize and store ------------------------------------------------
            w = mbar_wait(ptx::smem_addr(&B.o_full), ph, abort_ptr);
            if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
            ptx::tc_fence_after();
            const int token = qt * 128 + row;
            // each of the row's two threads requantizes and stores 32 of the head's 64 columns
            uint32_t ow[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) ow[k] = 0;
            {
                uint32_t v[32];
                ptx::tmem_ld32(t_row + (uint32_t)(hf * 32), v);
                ptx::tmem_ld_wait();
                // straight-line per-column arithmetic first, container-dependent packing afterwards
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int col = hf * 32 + i;
                    const float f = small_int_to_float((int)v[i] >> (8 - C));     // V codes sit in the high bits of their bytes
                    v[i] = round_clamp_bits(fmaf(f, colp[col], colp[64 + col]), P.out_qn, P.out_qp);
                }
                if (P.out_c == 4) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) ow[i >> 3] |= (v[i] & 0xFu) << (4 * (i & 7));
                } else if (P.out_c == 2) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) ow[i >> 4] |= (v[i] & 0x3u) << (2 * (i & 15));
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        ow[i] = __byte_perm(__byte_perm(v[4 * i], v[4 * i + 1], 0x4040),
                                            __byte_perm(v[4 * i + 2], v[4 * i + 3], 0x4040), 0x5410);
                }
            }
            if (token < T) {
                // 32 codes = 4*out_c bytes at column block h*64 + hf*32
                uint8_t* o = P.out + ((long long)b * T + token) * P.out_pitch + (long long)h * (8 * P.out_c) + hf * (4 * P.out_c);
                if (P.out_c == 4) {
                    *reinterpret_cast<uint4*>(o) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                } else if (P.out_c == 2) {
                    *reinterpret_cast<uint2*>(o) = make_uint2(ow[0], ow[1]);
                } else if ((reinterpret_cast<uintptr_t>(o) & 31u) == 0) {
                    // one 32-byte store: a warp's store touches 32 different rows whatever its width
                    const uint32_t lo[4] = {ow[0], ow[1], ow[2], ow[3]}, hi[4] = {ow[4], ow[5], ow[6], ow[7]};
                    ptx::st_global_32B(o, lo, hi);
                } else {
                    reinterpret_cast<uint4*>(o)[0] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                    reinterpret_cast<uint4*>(o)[1] = make_uint4(ow[4], ow[5], ow[6], ow[7]);
                }
            }
            // row padding behind the last head's columns (a caller may choose a pitch beyond the row's codes)
            if (token < T && h == P.heads - 1 && hf == 1) {
                uint8_t* const orow = P.out + ((long long)b * T + token) * P.out_pitch;
                for (long long off = (long long)P.heads * (8 * P.out_c); off + 4 <= P.out_pitch; off += 4)
                    *reinterpret_cast<uint32_t*>(orow + off) = 0u;
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&B.o_done));
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == AT_GROUPS * AT_COMPUTE_WARPS) {
        ptx::tc_fence_after();
        __syncwarp();
        ptx::tmem_dealloc(tmem_base_slot, 512);
    }
}

inline uint32_t up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

}  // namespace
}  // namespace vitint

using namespace vitint;

extern "C" size_t vitint_attention_core_shift_workspace_bytes(int32_t bits) {
    if (bits != 2 && bits != 3 && bits != 4) return 0;
    const int m = 1 << (container_bits(bits) - 1);
    return (size_t)(2 * 64 * m * m + 2) * 6 + 256;                   // 32-bit mantissas + 16-bit integer parts
}

extern "C" size_t vitint_attention_core_workspace_bytes(int32_t bits) {
    if (bits != 2 && bits != 3 && bits != 4) return 0;
    const int m = 1 << (container_bits(bits) - 1);   // sized by the container: any bit pattern indexes inside
    return (size_t)(2 * 64 * m * m + 1) * sizeof(float) + 256;
}

namespace vitint {
int attention_long_launch(const vitint_codes* qkv, int batch, int heads, int tokens, int smax, const float* table, float p_step,
                          float p_qp, const float* alpha_o, const float* beta_o, const vitint_codes* o_out, cudaStream_t st);
}

// Shared by the three entry points below.  build_table: fill `workspace` with the exp table first (one more
// small launch); otherwise the caller has filled it for exactly these steps and bits (vitint_attention_exp_table).
static int attention_core_launch(const vitint_codes* qkv, int32_t batch, int32_t heads, int32_t tokens,
                                 float q_step, float k_step, float p_step, int32_t p_bits, const float* alpha_o,
                                 const float* beta_o, const vitint_codes* o_out, void* workspace,
                                 size_t workspace_bytes, bool build_table, void* stream, bool shift = false) {
    if (int rc = check_codes(qkv)) return rc;
    if (int rc = check_codes(o_out)) return rc;
    if (batch <= 0 || heads <= 0 || tokens <= 0 || !alpha_o) return VITINT_ERR_INVALID_ARG;
    const int64_t M = (int64_t)batch * tokens, D = (int64_t)heads * 64;
    if (qkv->rows != M || qkv->cols != 3 * D || !qkv->is_signed || o_out->rows != M || o_out->cols != D)
        return VITINT_ERR_INVALID_ARG;
    const float steps[3] = {q_step, k_step, p_step};
    for (float s : steps) if (!(s > 0.0f && s < INFINITY)) return VITINT_ERR_INVALID_ARG;
    if (!valid_bits(p_bits)) return VITINT_ERR_INVALID_ARG;
    if (qkv->bits == 8 || batch > 65535) return VITINT_ERR_UNSUPPORTED;
    const int c = codes_container(qkv);                  // 2 / 4: packed; 8: one code per byte
    // beyond 256 tokens S no longer fits tensor memory beside O: the chunked two-pass kernel (byte-stored codes, exp table)
    const bool long_seq = tokens > 256;
    if (long_seq && (shift || c != 8 || tokens > 4096)) return VITINT_ERR_UNSUPPORTED;
    const int m = 1 << (container_bits(qkv->bits) - 1);
    const int smax = 64 * m * m;
    const float cs = (float)((double)q_step * (double)k_step / 8.0);
    // exp without max subtraction must not overflow for any score the declared code range can produce
    // (the table itself is sized by the container so that any bit pattern indexes inside it)
    const int mq = 1 << (qkv->bits - 1);
    if (!shift && 64.0 * mq * mq * (double)cs > 80.0) return VITINT_ERR_UNSUPPORTED;
    // Eq. 4: z = S * c2 with c2 = c * log2 e; the row maximum is subtracted (as shifts), so the only range limit is the
    // 16-bit table of floor z.  Byte-stored codes only.
    const float c2 = (float)((double)cs * 1.4426950408889634);
    if (shift && (c != 8 || (double)smax * (double)c2 > 30000.0)) return VITINT_ERR_UNSUPPORTED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < (shift ? vitint_attention_core_shift_workspace_bytes(qkv->bits)
                                 : vitint_attention_core_workspace_bytes(qkv->bits)))
        return VITINT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    if (long_seq) {
        if (build_table) {
            launch_kernel(exp_table_kernel, dim3((2 * smax + 1 + 255) / 256), dim3(256), 0, st, (float*)workspace, smax, cs);
            if (cudaGetLastError() != cudaSuccess) return VITINT_ERR_CUDA;
        }
        int pqn, pqp;
        code_range(p_bits, 0, &pqn, &pqp);
        return attention_long_launch(qkv, batch, heads, tokens, smax, (const float*)workspace, p_step, (float)pqp, alpha_o,
                                     beta_o, o_out, st);
    }

    AttnParams P{};
    P.batch = batch; P.heads = heads; P.tokens = tokens;
    P.q_tiles = (tokens + 127) / 128;
    P.total_items = batch * heads * P.q_tiles;
    P.c = c;
    P.n_k = (tokens + 15) / 16 * 16;
    P.kv_rows = (tokens + 31) / 32 * 32;
    P.smax = smax;
    P.part_bytes = (int)(D * c / 8);
    P.table = (const float*)workspace;
    P.p_step = p_step;
    int qn, qp;
    code_range(p_bits, 0, &qn, &qp);
    P.p_qp = (float)qp;
    P.alpha_o = alpha_o; P.beta_o = beta_o;
    P.out_c = codes_container(o_out);
    code_range(o_out->bits, o_out->is_signed, &qn, &qp);
    P.out_qn = (float)qn; P.out_qp = (float)qp;
    P.out = (uint8_t*)o_out->data; P.out_pitch = o_out->pitch_bytes;
    // shared-memory layout
    const uint32_t hb = 8u * c;
    P.off_table = 0;
    P.off_group = up((uint32_t)(2 * smax + 1) * 4u, 1024);
    if (shift) {
        // 32-bit mantissas, then (from the next whole word on) the 16-bit integer parts
        P.ftab_word = (uint32_t)(2 * smax + 1);
        P.off_ftab = (uint32_t)(2 * smax + 1) * 4u;
        P.off_group = up(P.off_ftab + (uint32_t)(2 * smax + 2) * 2u, 1024);
    }
    uint32_t o = 0;
    P.off_q = o; o += 128 * 64;
    P.off_k = o; o += up((uint32_t)(c == 8 ? P.kv_rows : P.n_k) * 64, 1024);   // byte codes: the K box is kv_rows high
    P.off_v = o; o += up((uint32_t)P.kv_rows * 64, 1024);
    P.off_p = o; o += (uint32_t)((P.kv_rows + 127) / 128) * 16384u;
    if (c != 8) {
        P.off_pq = o; o += up(128 * hb, 128);
        P.off_pk = o; o += up((uint32_t)P.kv_rows * hb, 128);
        P.off_pv = o; o += up((uint32_t)P.kv_rows * hb, 128);
    }
    P.off_col = o; o += 1024;
    P.off_z = o; o += 2 * 128 * 8;
    P.off_mx = o;
    if (shift) o += 2 * 128 * 4;                           // partial row maxima of the Eq. 4 variant
    P.group_bytes = up(o, 1024);
    const size_t smem = (size_t)P.off_group + (size_t)AT_GROUPS * P.group_bytes + 1024;
    if (smem > 225 * 1024) return VITINT_ERR_UNSUPPORTED;

    CUtensorMap map_q, map_kv;
    {
        // 3-D byte view of the QKV code matrix: (row bytes, token, image); rows past an image's
        // last token read as zero.  Q tiles are 128 rows high, K and V tiles kv_rows.
        EncodeTiledFn fn = encode_fn();
        if (!fn) return VITINT_ERR_CUDA;
        cuuint64_t dims[3] = {(cuuint64_t)codes_row_bytes(qkv, 3 * D), (cuuint64_t)tokens, (cuuint64_t)batch};
        // byte codes land directly in the 64-byte-swizzled operand tiles
        const CUtensorMapSwizzle swz = c == 8 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE;
        cuuint64_t strides[2] = {(cuuint64_t)qkv->pitch_bytes, (cuuint64_t)qkv->pitch_bytes * tokens};
        cuuint32_t estr[3] = {1, 1, 1};
        cuuint32_t box_q[3] = {hb, 128, 1}, box_kv[3] = {hb, (cuuint32_t)P.kv_rows, 1};
        if (fn(&map_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, qkv->data, dims, strides, box_q, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            fn(&map_kv, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, qkv->data, dims, strides, box_kv, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return VITINT_ERR_CUDA;
    }
    if (build_table) {
        if (shift) launch_kernel(shift_table_kernel, dim3((2 * smax + 1 + 255) / 256), dim3(256), 0, st, (uint32_t*)workspace,
                                 reinterpret_cast<short*>((uint32_t*)workspace + (2 * smax + 1)), smax, c2);
        else launch_kernel(exp_table_kernel, dim3((2 * smax + 1 + 255) / 256), dim3(256), 0, st, (float*)workspace, smax, cs);
        if (cudaGetLastError() != cudaSuccess) return VITINT_ERR_CUDA;
    }
    int grid = sm_count();
    const int want = (P.total_items + AT_GROUPS - 1) / AT_GROUPS;
    if (grid > want) grid = want;
    const int dev = current_device();
    if (dev < 0) return VITINT_ERR_CUDA;
    static bool attr_set_dev[MAX_DEVICES][4] = {};
    bool* const attr_set = attr_set_dev[dev];
#define VITINT_ATTN_LAUNCH(CC, SH, SLOT)                                                                           \
    {                                                                                                              \
        if (!attr_set[SLOT]) {                                                                                     \
            if (cudaFuncSetAttribute(attention_fused_kernel<CC, SH>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                                     225 * 1024) != cudaSuccess)                                                   \
                return VITINT_ERR_CUDA;                                                                            \
            attr_set[SLOT] = true;                                                                                 \
        }                                                                                                          \
        launch_kernel(attention_fused_kernel<CC, SH>, dim3(grid), dim3(AT_THREADS), smem, st, map_q, map_kv, P);   \
    }
    if (shift) VITINT_ATTN_LAUNCH(8, true, 3)
    else if (c == 8) VITINT_ATTN_LAUNCH(8, false, 2)
    else if (c == 4) VITINT_ATTN_LAUNCH(4, false, 1)
    else VITINT_ATTN_LAUNCH(2, false, 0)
#undef VITINT_ATTN_LAUNCH
    return cuda_status(cudaGetLastError());
}

extern "C" int vitint_attention_core(const vitint_codes* qkv, int32_t batch, int32_t heads, int32_t tokens,
                                     float q_step, float k_step, float p_step, int32_t p_bits, const float* alpha_o,
                                     const float* beta_o, const vitint_codes* o_out, void* workspace,
                                     size_t workspace_bytes, void* stream) {
    return attention_core_launch(qkv, batch, heads, tokens, q_step, k_step, p_step, p_bits, alpha_o, beta_o, o_out,
                                 workspace, workspace_bytes, true, stream);
}

extern "C" int vitint_attention_core_shift(const vitint_codes* qkv, int32_t batch, int32_t heads, int32_t tokens,
                                           float q_step, float k_step, float p_step, int32_t p_bits, const float* alpha_o,
                                           const float* beta_o, const vitint_codes* o_out, void* workspace,
                                           size_t workspace_bytes, int32_t table_ready, void* stream) {
    return attention_core_launch(qkv, batch, heads, tokens, q_step, k_step, p_step, p_bits, alpha_o, beta_o, o_out,
                                 workspace, workspace_bytes, table_ready == 0, stream, true);
}

extern "C" int vitint_attention_exp_table(int32_t bits, float q_step, float k_step, void* table, size_t table_bytes,
                                          void* stream) {
    if (!valid_bits(bits) || bits == 8) return VITINT_ERR_UNSUPPORTED;
    if (!(q_step > 0.0f && q_step < INFINITY) || !(k_step > 0.0f && k_step < INFINITY)) return VITINT_ERR_INVALID_ARG;
    if (!table || (reinterpret_cast<uintptr_t>(table) & 255u) || table_bytes < vitint_attention_core_workspace_bytes(bits))
        return VITINT_ERR_WORKSPACE;
    const int m = 1 << (container_bits(bits) - 1);
    const int smax = 64 * m * m;
    const float cs = (float)((double)q_step * (double)k_step / 8.0);
    launch_kernel(exp_table_kernel, dim3((2 * smax + 1 + 255) / 256), dim3(256), 0, (cudaStream_t)stream, (float*)table,
                  smax, cs);
    return cuda_status(cudaGetLastError());
}

extern "C" int vitint_attention_core_prepared(const vitint_codes* qkv, int32_t batch, int32_t heads, int32_t tokens,
                                              float q_step, float k_step, float p_step, int32_t p_bits,
                                              const float* alpha_o, const float* beta_o, const vitint_codes* o_out,
                                              const void* table, size_t table_bytes, void* stream) {
    return attention_core_launch(qkv, batch, heads, tokens, q_step, k_step, p_step, p_bits, alpha_o, beta_o, o_out,
                                 const_cast<void*>(table), table_bytes, false, stream);
}

// ---------------------------------------------------------------------------------------
// Allocation-free variant: the exp table lives in a fixed device array of this library.
// ---------------------------------------------------------------------------------------
namespace vitint {
namespace {

constexpr int STATIC_TABLE_FLOATS = 8320;   // largest table (8193 entries, 4-bit containers) plus the 256-byte slack of the workspace query

// Resident on every GPU that loads the library, from load until the process exits (about 33 KB).
static __device__ __align__(256) float g_static_exp_table[STATIC_TABLE_FLOATS];

// the widest codes the table-driven kernel takes (4-bit containers: scores in -4096 .. 4096) must fit the array
static_assert((2 * 64 * 8 * 8 + 1) * sizeof(float) + 256 <= sizeof(float) * STATIC_TABLE_FLOATS,
              "the built-in scratch must hold the exp table of 4-bit codes");

void* g_static_table_addr[MAX_DEVICES];   // device address of the array, per device, once looked up
int g_static_table_rc[MAX_DEVICES];
std::once_flag g_static_table_once[MAX_DEVICES];

// The array's name is only a host-side handle; kernels need its device address.  Looked up once
// per device, with that device current (std::call_once: concurrent first calls from several host
// threads are safe).
int static_table_address(void** out) {
    const int dev = current_device();
    if (dev < 0) return VITINT_ERR_CUDA;
    std::call_once(g_static_table_once[dev], [dev]() {
        void* p = nullptr;
        const bool ok = cudaGetSymbolAddress(&p, g_static_exp_table) == cudaSuccess && p != nullptr;
        g_static_table_addr[dev] = ok ? p : nullptr;
        g_static_table_rc[dev] = ok ? VITINT_OK : VITINT_ERR_CUDA;
    });
    if (g_static_table_rc[dev] != VITINT_OK) return g_static_table_rc[dev];
    *out = g_static_table_addr[dev];
    return VITINT_OK;
}

}  // namespace
}  // namespace vitint

extern "C" int vitint_attention_core_noalloc(const vitint_codes* qkv, int32_t batch, int32_t heads, int32_t tokens,
                                             float q_step, float k_step, float p_step, int32_t p_bits,
                                             const float* alpha_o, const float* beta_o, const vitint_codes* o_out,
                                             void* stream) {
    // argument errors first, so that they are reported exactly as vitint_attention_core reports them
    if (int rc = check_codes(qkv)) return rc;
    if (int rc = check_codes(o_out)) return rc;
    const size_t need = vitint_attention_core_workspace_bytes(qkv->bits);
    if (need == 0) return VITINT_ERR_UNSUPPORTED;                     // 8-bit codes: no table-driven kernel
    void* table = nullptr;
    if (int rc = static_table_address(&table)) return rc;
    return vitint_attention_core(qkv, batch, heads, tokens, q_step, k_step, p_step, p_bits, alpha_o, beta_o, o_out,
                                 table, sizeof(float) * STATIC_TABLE_FLOATS, stream);
}
