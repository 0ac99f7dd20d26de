// a4 + a5 + a6 fused for sequences beyond 256 tokens (577, 785: S no longer fits tensor memory beside O).
//
// Per (image, head, 128-query tile) the keys are walked in chunks of at most 192, twice:
//   pass A   S_c = Q K_c^T (tcgen05, K = 64)  ->  Z += sum_j EXP[S_j]            (table of exp(fl32(s c)), fp64 sum)
//   pass B   S_c again                        ->  codes = min(rint(EXP[S_j] / (Z s_P)), Qp)  ->  P_c in shared memory
//            O += P_c V_c (tcgen05, accumulating in tensor memory across the chunks)
// then O is requantized and stored.  S, the probabilities and P never reach HBM: the unfused sequence writes and
// re-reads 4 T^2 bytes per head (946 MB at 785 tokens, batch 32), which is what bounds it.  The table makes the
// two-pass form exact and cheap: exp(t_j) / sum_k exp(t_k) needs no running maximum and no rescaling of O, and Q K^T
// (a K = 64 contraction) costs next to nothing to repeat.  Arithmetic per score is that of attention_fused_kernel,
// so the codes are the same.
//
// One pipeline per CTA, steps in sequence (every thread passes the same barriers; an expired wait makes the whole CTA
// leave together), two CTAs per SM so that one's loads and MMAs run beside the other's softmax.  Byte-stored codes.
#include "common.cuh"
#include "ptx.cuh"
#include "tile_ops.cuh"

namespace vitint {
namespace {

constexpr int AL_COMPUTE_WARPS = 8;     // two threads per query row, alternate 32-column blocks
constexpr int AL_THREADS = (AL_COMPUTE_WARPS + 1) * 32;
constexpr int AL_MAX_CHUNK = 192;       // S chunk (192 columns) + O (64 columns) = the CTA's 256 tensor-memory columns
constexpr uint32_t AL_O_COL = 192;

struct LongParams {
    int batch, heads, tokens, q_tiles, total_items;
    int chunk, n_chunks;          // keys per chunk (multiple of 32), chunks per row
    int smax;
    int part_bytes;               // bytes of one of the Q / K / V segments in a QKV row
    const float* table;
    float p_step, p_qp;
    const float* alpha_o;
    const float* beta_o;
    uint8_t* out;
    int64_t out_pitch;
    int out_c;
    float out_qn, out_qp;
    uint32_t off_table, off_q, off_k, off_v, off_p, off_z, off_col;
};

struct LongBars {
    uint64_t q_full, kv_full, s_full, o_full;
};

__global__ void __launch_bounds__(AL_THREADS, 2)
attention_long_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv,
                      const __grid_constant__ LongParams P) {
    extern __shared__ uint8_t al_smem_raw[];
    __shared__ LongBars B;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_addr(al_smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem_gen = al_smem_raw + (smem_base - ptx::smem_addr(al_smem_raw));
    volatile int* abort_ptr = &abort_flag;
    const bool is_control = warp == AL_COMPUTE_WARPS;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(ptx::smem_addr(&B.q_full), 1);
        ptx::mbar_init(ptx::smem_addr(&B.kv_full), 1);
        ptx::mbar_init(ptx::smem_addr(&B.s_full), 1);
        ptx::mbar_init(ptx::smem_addr(&B.o_full), 1);
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    if (is_control) {
        ptx::tmem_alloc(ptx::smem_addr(&tmem_base_slot), 256);
        ptx::tmem_relinquish();
    }
    grid_dependency_wait();        // the table and the codes come from earlier kernels of the stream
    grid_dependency_launch();
    {
        float* tab = reinterpret_cast<float*>(smem_gen + P.off_table);
        for (int i = threadIdx.x; i <= 2 * P.smax; i += AL_THREADS) tab[i] = __ldg(P.table + i);
    }
    if (is_control && lane == 0) { ptx::prefetch_tensormap(&map_q); ptx::prefetch_tensormap(&map_kv); }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = tmem_base_slot;

    const int T = P.tokens, CH = P.chunk;
    const uint32_t q_bytes = 128u * 64u, kv_bytes = (uint32_t)CH * 64u;
    const uint32_t idesc_qk = ptx::idesc_i8(128, CH, 1, 1, 0);
    const uint32_t idesc_pv = ptx::idesc_i8(128, 64, 0, 1, 1);
    const uint64_t q_desc = ptx::smem_desc(smem_base + P.off_q, 16, 512, ptx::SWIZZLE_64B);
    const uint64_t k_desc = ptx::smem_desc(smem_base + P.off_k, 16, 512, ptx::SWIZZLE_64B);
    const uint64_t v_desc = ptx::smem_desc(smem_base + P.off_v, 16, 512, ptx::SWIZZLE_64B);
    const int pv_steps = CH / 32, blocks = CH / 32;

    // compute-thread coordinates (the control warp carries them along unused)
    const int wq = warp & 3;                                     // tensor-memory lane quarter
    const int hf = (warp >> 2) & 1;                              // which of the row's two threads
    const int tid_c = warp * 32 + lane;                          // 0..255 for compute threads
    const int row = wq * 32 + lane;
    const uint32_t t_row = tmem + ((uint32_t)(wq * 32) << 16);
    const char* const tab_lo = reinterpret_cast<const char*>(smem_gen + P.off_table);
    const int tab_half = 4 * P.smax;
    double* const zx = reinterpret_cast<double*>(smem_gen + P.off_z);
    float* const colp = reinterpret_cast<float*>(smem_gen + P.off_col);
    const double inv_p_step = 1.0 / (double)P.p_step;
    uint8_t* const prow = smem_gen + P.off_p + row * 128;
    const int sw = row & 7;

    uint32_t n_q = 0, n_kv = 0, n_s = 0, n_o = 0;                // completed phases of each barrier (parity = count & 1)
    bool ok = true;
    for (int item = blockIdx.x; ok && item < P.total_items; item += gridDim.x) {
        const int qt = item % P.q_tiles;
        const int bh = item / P.q_tiles;
        const int h = bh % P.heads, b = bh / P.heads;
        if (!is_control) {
            if (tid_c < 64) colp[tid_c] = __ldg(P.alpha_o + h * 64 + tid_c);
            else if (tid_c < 128) colp[tid_c] = P.beta_o ? __ldg(P.beta_o + h * 64 + (tid_c - 64)) : 0.0f;
        }
        if (is_control && lane == 0) {
            ptx::mbar_arrive_expect_tx(ptx::smem_addr(&B.q_full), q_bytes);
            ptx::tma_load_3d(smem_base + P.off_q, &map_q, ptx::smem_addr(&B.q_full), h * 64, qt * 128, b);
        }
        double zp[4] = {0.0, 0.0, 0.0, 0.0};
        f32x2 rzh2 = f2_dup(0.0f), rzl2 = f2_dup(0.0f);
        const f32x2 magic2 = f2_dup(12582912.0f);
        const bool warp_live = qt * 128 + wq * 32 < T;
        for (int pass = 0; ok && pass < 2; ++pass) {
            for (int c = 0; ok && c < P.n_chunks; ++c) {
                const int key0 = c * CH;
                // ---- loads and S_c = Q K_c^T ---------------------------------------------------------------
                bool w = true;
                if (is_control && lane == 0) {
                    const uint32_t bar = ptx::smem_addr(&B.kv_full);
                    ptx::mbar_arrive_expect_tx(bar, pass ? 2u * kv_bytes : kv_bytes);
                    ptx::tma_load_3d(smem_base + P.off_k, &map_kv, bar, P.part_bytes + h * 64, key0, b);
                    if (pass) ptx::tma_load_3d(smem_base + P.off_v, &map_kv, bar, 2 * P.part_bytes + h * 64, key0, b);
                    if (pass == 0 && c == 0) w = mbar_wait(ptx::smem_addr(&B.q_full), n_q & 1u, abort_ptr);
                    w = w && mbar_wait(bar, n_kv & 1u, abort_ptr);
                    if (w) {
                        ptx::tc_fence_after();
                        for (int k = 0; k < 2; ++k)
                            ptx::mma_i8(tmem, q_desc + (uint64_t)(k * 2), k_desc + (uint64_t)(k * 2), idesc_qk, k);
                        ptx::mma_commit(ptx::smem_addr(&B.s_full));
                    }
                }
                if (pass == 0 && c == 0) ++n_q;
                ++n_kv;
                // every thread waits for S (the control lane included, so that K may be overwritten afterwards)
                w = w && mbar_wait(ptx::smem_addr(&B.s_full), n_s & 1u, abort_ptr);
                ++n_s;
                if (!__syncthreads_and(w ? 1 : 0)) { ok = false; break; }
                ptx::tc_fence_after();
                const bool tail = key0 + CH > T;                        // columns past the last token in this chunk
                if (!is_control && warp_live) {
                    if (pass == 0) {
                        // ---- pass A: row sum of the table entries ------------------------------------------
                        for (int blk = hf; blk < blocks; blk += 2) {
                            if (key0 + blk * 32 >= T) break;
                            uint32_t v[32];
                            ptx::tmem_ld32(t_row + (uint32_t)(blk * 32), v);
                            ptx::tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const uint32_t off = min((uint32_t)((int)v[i] * 4 + tab_half), (uint32_t)(2 * tab_half));
                                const uint32_t eb = *reinterpret_cast<const uint32_t*>(tab_lo + off);
                                // a table entry is a positive normal float: its double from the bits, two integer operations
                                uint32_t hi, lo;
                                asm("mad.hi.u32 %0, %1, 536870912, 939524096;" : "=r"(hi) : "r"(eb));
                                asm("mul.lo.u32 %0, %1, 536870912;" : "=r"(lo) : "r"(eb));
                                const bool valid = !tail || key0 + blk * 32 + i < T;
                                zp[i & 3] += valid ? __hiloint2double((int)hi, (int)lo) : 0.0;
                            }
                        }
                    } else {
                        // ---- pass B: codes of this chunk into the P tile -----------------------------------
                        for (int blk = hf; blk < blocks; blk += 2) {
                            uint32_t v[32];
                            ptx::tmem_ld32(t_row + (uint32_t)(blk * 32), v);
                            ptx::tmem_ld_wait();
                            uint32_t wd[8];
#pragma unroll
                            for (int i4 = 0; i4 < 8; ++i4) {
                                uint32_t cb[4];
#pragma unroll
                                for (int j = 0; j < 4; j += 2) {
                                    float e[2];
#pragma unroll
                                    for (int u = 0; u < 2; ++u) {
                                        const int i = 4 * i4 + j + u;
                                        const uint32_t off = min((uint32_t)((int)v[i] * 4 + tab_half), (uint32_t)(2 * tab_half));
                                        const float ev = *reinterpret_cast<const float*>(tab_lo + off);
                                        e[u] = (!tail || key0 + blk * 32 + i < T) ? ev : 0.0f;
                                    }
                                    const f32x2 e2 = f2_pack(e[0], e[1]);
                                    float a0, a1, c0, c1;
                                    f2_unpack(f2_fma(e2, rzh2, f2_mul(e2, rzl2)), a0, a1);
                                    f2_unpack(f2_add(f2_pack(fminf(a0, P.p_qp), fminf(a1, P.p_qp)), magic2), c0, c1);
                                    cb[j] = __float_as_uint(c0);
                                    cb[j + 1] = __float_as_uint(c1);
                                }
                                wd[i4] = __byte_perm(__byte_perm(cb[0], cb[1], 0x4040), __byte_perm(cb[2], cb[3], 0x4040), 0x5410);
                            }
                            const int cc = 2 * blk;
                            uint8_t* const pblk = prow + (cc >> 3) * 16384;
                            *reinterpret_cast<uint4*>(pblk + (((cc & 7) ^ sw) << 4)) = make_uint4(wd[0], wd[1], wd[2], wd[3]);
                            *reinterpret_cast<uint4*>(pblk + ((((cc + 1) & 7) ^ sw) << 4)) = make_uint4(wd[4], wd[5], wd[6], wd[7]);
                        }
                        ptx::fence_proxy_async_smem();
                    }
                }
                ptx::tc_fence_before();
                __syncthreads();                                        // S has been read; the P tile is complete
                if (pass == 1) {
                    // ---- O += P_c V_c ----------------------------------------------------------------------
                    if (is_control && lane == 0) {
                        ptx::tc_fence_after();
                        for (int ks = 0; ks < pv_steps; ++ks) {
                            const uint64_t p_desc = ptx::smem_desc(smem_base + P.off_p + (uint32_t)(ks >> 2) * 16384u, 16, 1024,
                                                                   ptx::SWIZZLE_128B) + (uint64_t)((ks & 3) * 2);
                            ptx::mma_i8(tmem + AL_O_COL, p_desc, v_desc + (uint64_t)(ks * 128), idesc_pv, (c > 0 || ks > 0) ? 1 : 0);
                        }
                        ptx::mma_commit(ptx::smem_addr(&B.o_full));
                    }
                    // K, V and the P tile are reused by the next chunk: everyone waits for the MMAs that read them
                    w = mbar_wait(ptx::smem_addr(&B.o_full), n_o & 1u, abort_ptr);
                    ++n_o;
                    if (!__syncthreads_and(w ? 1 : 0)) { ok = false; break; }
                }
            }
            if (!ok) break;
            if (pass == 0) {
                // the row's two threads add their partial sums; r = 1 / (Z s_P) as a two-float number
                if (!is_control) zx[hf * 128 + row] = (zp[0] + zp[1]) + (zp[2] + zp[3]);
                __syncthreads();
                if (!is_control) {
                    const double z = zx[row] + zx[128 + row];
                    const double rz = warp_live ? inv_p_step / z : 0.0;
                    const float rzh = (float)rz;
                    rzh2 = f2_dup(rzh);
                    rzl2 = f2_dup((float)(rz - (double)rzh));
                }
                __syncthreads();                                        // zx may be rewritten by the next item
            }
        }
        if (!ok) break;
        // ---- requantize O and store -------------------------------------------------------------------------
        ptx::tc_fence_after();
        if (!is_control) {
            const int token = qt * 128 + row;
            uint32_t ow[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) ow[k] = 0;
            uint32_t v[32];
            ptx::tmem_ld32(t_row + AL_O_COL + (uint32_t)(hf * 32), v);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int col = hf * 32 + i;
                v[i] = round_clamp_bits(fmaf(small_int_to_float((int)v[i]), colp[col], colp[64 + col]), P.out_qn, P.out_qp);
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
                    ow[i] = __byte_perm(__byte_perm(v[4 * i], v[4 * i + 1], 0x4040), __byte_perm(v[4 * i + 2], v[4 * i + 3], 0x4040), 0x5410);
            }
            if (token < T) {
                uint8_t* o = P.out + ((long long)b * T + token) * P.out_pitch + (long long)h * (8 * P.out_c) + hf * (4 * P.out_c);
                if (P.out_c == 4) {
                    *reinterpret_cast<uint4*>(o) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                } else if (P.out_c == 2) {
                    *reinterpret_cast<uint2*>(o) = make_uint2(ow[0], ow[1]);
                } else {
                    reinterpret_cast<uint4*>(o)[0] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                    reinterpret_cast<uint4*>(o)[1] = make_uint4(ow[4], ow[5], ow[6], ow[7]);
                }
                if (h == P.heads - 1 && hf == 1) {
                    uint8_t* const orow = P.out + ((long long)b * T + token) * P.out_pitch;
                    for (long long off = (long long)P.heads * (8 * P.out_c); off + 4 <= P.out_pitch; off += 4)
                        *reinterpret_cast<uint32_t*>(orow + off) = 0u;
                }
            }
        }
        ptx::tc_fence_before();
        __syncthreads();                                                // O and the head's parameters are free again
    }
    // a copy still in flight when the CTA gives up is given a bounded chance to land
    if (!ok && is_control && lane == 0) {
        for (int spin = 0; spin < (1 << 20) && !ptx::mbar_try_wait(ptx::smem_addr(&B.kv_full), (n_kv - 1u) & 1u); ++spin) {}
        for (int spin = 0; spin < (1 << 20) && n_q > 0 && !ptx::mbar_try_wait(ptx::smem_addr(&B.q_full), (n_q - 1u) & 1u); ++spin) {}
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (is_control) {
        ptx::tc_fence_after();
        __syncwarp();
        ptx::tmem_dealloc(tmem_base_slot, 256);
    }
}

inline uint32_t al_up(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

}  // namespace

// Launcher shared with attention_core_launch: byte-stored codes, more than 256 tokens, table already in `table`.
int attention_long_launch(const vitint_codes* qkv, int batch, int heads, int tokens, int smax, const float* table, float p_step,
                          float p_qp, const float* alpha_o, const float* beta_o, const vitint_codes* o_out, cudaStream_t st) {
    const int64_t D = (int64_t)heads * 64;
    LongParams P{};
    P.batch = batch; P.heads = heads; P.tokens = tokens;
    P.q_tiles = (tokens + 127) / 128;
    const long long items = (long long)batch * heads * P.q_tiles;
    if (items > 0x7fffffffll) return VITINT_ERR_UNSUPPORTED;
    P.total_items = (int)items;
    P.n_chunks = (tokens + AL_MAX_CHUNK - 1) / AL_MAX_CHUNK;
    P.chunk = ((tokens + P.n_chunks - 1) / P.n_chunks + 31) / 32 * 32;          // <= 192, a multiple of 32
    P.smax = smax;
    P.part_bytes = (int)D;
    P.table = table;
    P.p_step = p_step; P.p_qp = p_qp;
    P.alpha_o = alpha_o; P.beta_o = beta_o;
    P.out_c = codes_container(o_out);
    int qn, qp;
    code_range(o_out->bits, o_out->is_signed, &qn, &qp);
    P.out_qn = (float)qn; P.out_qp = (float)qp;
    P.out = (uint8_t*)o_out->data; P.out_pitch = o_out->pitch_bytes;
    uint32_t o = 0;
    P.off_table = o; o += al_up((uint32_t)(2 * smax + 1) * 4u, 1024);
    P.off_q = o; o += 128 * 64;
    P.off_k = o; o += al_up((uint32_t)P.chunk * 64, 1024);
    P.off_v = o; o += al_up((uint32_t)P.chunk * 64, 1024);
    P.off_p = o; o += (uint32_t)((P.chunk + 127) / 128) * 16384u;
    P.off_z = o; o += 2 * 128 * 8;
    P.off_col = o; o += 512;
    const size_t smem = (size_t)o + 1024;
    if (smem > 113 * 1024) return VITINT_ERR_UNSUPPORTED;                       // two CTAs per SM

    CUtensorMap map_q, map_kv;
    {
        EncodeTiledFn fn = encode_fn();
        if (!fn) return VITINT_ERR_CUDA;
        cuuint64_t dims[3] = {(cuuint64_t)codes_row_bytes(qkv, 3 * D), (cuuint64_t)tokens, (cuuint64_t)batch};
        cuuint64_t strides[2] = {(cuuint64_t)qkv->pitch_bytes, (cuuint64_t)qkv->pitch_bytes * tokens};
        cuuint32_t estr[3] = {1, 1, 1};
        cuuint32_t box_q[3] = {64, 128, 1}, box_kv[3] = {64, (cuuint32_t)P.chunk, 1};
        if (fn(&map_q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, qkv->data, dims, strides, box_q, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            fn(&map_kv, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, qkv->data, dims, strides, box_kv, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return VITINT_ERR_CUDA;
    }
    int grid = 2 * sm_count();
    if (grid > P.total_items) grid = P.total_items;
    const int dev = current_device();
    if (dev < 0) return VITINT_ERR_CUDA;
    static bool attr_set_dev[MAX_DEVICES] = {};
    if (!attr_set_dev[dev]) {
        if (cudaFuncSetAttribute(attention_long_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024) != cudaSuccess)
            return VITINT_ERR_CUDA;
        attr_set_dev[dev] = true;
    }
    launch_kernel(attention_long_kernel, dim3(grid), dim3(AL_THREADS), smem, st, map_q, map_kv, P);
    return cuda_status(cudaGetLastError());
}

}  // namespace vitint
