// a2/a3/a4/a6: integer GEMM  acc[m][n] = sum_k A[m][k] * B[n][k]  on the 5th-generation
// tensor cores (tcgen05, kind::i8, int32 accumulators in TMEM) with the fused
// post-contraction epilogue of Eq. 2.
//
// One persistent CTA per SM walks 128 x BN output tiles.  Warp roles:
//   warps 0-7  epilogue: stage the tile's per-column scale / bias in shared memory,
//              tcgen05.ld of their 32 TMEM lanes, rescale / bias / GELU / requantize /
//              pack, global stores (warp w owns TMEM lanes 32(w%4).. and a share of the columns);
//   warp  8    TMA producer: packed low-bit tiles -> shared-memory ring; operands that are
//              already 8-bit go straight into the swizzled int8 operand ring;
//   warp  9    MMA issuer (one thread) and owner of the TMEM allocation;
//   warps 10-13 unpack: packed codes -> int8 operand tiles in the shared-memory layout
//              the tensor core expects (128-byte swizzle, K contiguous; or 64-byte
//              swizzle, N contiguous, for the V operand of P*V).  When both operands are
//              stored one code per byte there is nothing to unpack and these four warps
//              serve as a third epilogue warp per lane quarter.
// The accumulator is double buffered in TMEM so the epilogue of tile i overlaps the
// MMAs of tile i+1.
//
// Sign handling without sign extension: a signed c-bit code q is placed in the HIGH
// bits of its byte, i.e. the int8 value is q * 2^(8-c).  The contraction then yields
// acc * 2^shift exactly (host checks that the scaled sum still fits in int32); the
// epilogue folds 2^-shift into the per-column multiplier, which is exact in binary
// floating point, or shifts the integer back when raw accumulators are requested.
#include "common.cuh"
#include "ptx.cuh"
#include "tile_ops.cuh"

namespace vitint {

namespace {

constexpr int BM = 128;   // rows per tile (= TMEM lanes)
constexpr int BK = 128;   // int8 elements per K block (= one 128-byte swizzle row)
constexpr int EPI_WARPS = 8;   // two warps per TMEM lane quarter, each taking a share of the tile's columns
constexpr int UNPACK_WARPS = 4;   // with nothing to unpack these become a third epilogue warp per lane quarter
constexpr int MAX_EPI_WARPS = EPI_WARPS + UNPACK_WARPS;
constexpr int WARP_TMA = 8, WARP_MMA = 9, WARP_UNPACK0 = 10;
constexpr int NUM_THREADS = (WARP_UNPACK0 + UNPACK_WARPS) * 32;
constexpr int MAX_STAGES = 8;
constexpr int MAX_BN = 256;

enum EpiKind { EK_ACC = 0, EK_DEQUANT = 1, EK_DEQUANT_GELU = 2, EK_REQUANT = 3, EK_REQUANT_GELU = 4, EK_QKV_NORM = 5 };
constexpr int NUM_KINDS = 6;

struct GemmParams {
    int M, N, K;
    int bn, m_tiles, n_tiles, n_inner, total_tiles, k_blocks;
    int ca, cb, a_signed, b_signed, shift, b_mn_major;
    int a_direct, b_direct;            // operand already int8: TMA writes the operand ring itself
    int small_acc;                     // |acc| < 2^22: int -> float without a conversion instruction
    int unit_out;                      // GELU + unsigned requantization: the GELU multiplier carries 1/Qp and values clamp to [0, 1]
    int epi_warps;                     // EPI_WARPS, or MAX_EPI_WARPS when both operands come straight from TMA
    uint32_t stage_off;                // fp32 epilogue: byte offset of the per-warp transposition buffers (0 = none)
    int ns_i, ns_p;
    uint32_t ia_bytes, ib_bytes, pa_bytes, pb_bytes, tmem_cols;
    int kind, out_c;
    float out_qn, out_qp, x_step;
    void* out;
    long long ld_out, row_off_outer, row_off_inner, col_off_inner;
    const float* col_a;
    const float* col_b;
    const float* inv_s;
    const float* residual;
    long long ld_res;
    // EK_QKV_NORM: the QKV projection whose Q and K heads pass the quantizing LayerNorm of Section IV-C in the epilogue
    const float* norm_refs;            // [2][64][2^bits - 1] comparator references of the Q and the K norm
    const uint8_t* norm_flip;          // [2][64] or null
    float n_eps;
    int norm_bits, norm_qn, norm_dim;  // code width and lowest level of Q/K; D = heads * 64 (columns per segment)
    float* norm_stats;                 // [2][M * heads][2] (mu, V) or null
    const float* v_alpha;              // [D] requantization of the V segment
    const float* v_beta;               // [D] or null
};

struct Bars {
    uint64_t p_full[MAX_STAGES], p_empty[MAX_STAGES], i_full[MAX_STAGES], i_empty[MAX_STAGES];
    uint64_t acc_full[2], acc_empty[2], epi_sync;
};

struct EpiParams {                      // per-column epilogue parameters of the two tiles in flight
    float a[2][MAX_BN], b[2][MAX_BN], q[2][MAX_BN];
};

// ---- optional timeline of the warp roles (diagnostic builds only, -DVITINT_TRACE) ------------------
// The first TRACE_CTAS CTAs record (clock64() << 8 | tag) into a caller-provided buffer, one sequence
// per role: where the TMA producer, the MMA issuer and two epilogue warps wait, tile by tile.  The
// product library is built without the flag and contains none of this.
#ifdef VITINT_TRACE
constexpr int TRACE_CTAS = 4, TRACE_ROLES = 4, TRACE_SLOTS = 4096;
__device__ long long* g_trace_buf = nullptr;
int g_trace_max_ctas = 0;        // host: when > 0 the persistent grid is capped (how does a CTA run with fewer neighbours?)
struct Tracer {
    long long* p;
    int n;
    __device__ Tracer(int role) : p(nullptr), n(0) {
        if (role >= 0 && g_trace_buf && blockIdx.x < TRACE_CTAS) p = g_trace_buf + ((size_t)blockIdx.x * TRACE_ROLES + role) * TRACE_SLOTS;
    }
    __device__ __forceinline__ void stamp(int tag) {
        if (p && n < TRACE_SLOTS - 1) { p[1 + n] = (clock64() << 8) | (long long)(tag & 255); ++n; p[0] = n; }
    }
};
#define VT_TRACER(name, role) Tracer name(role)
#define VT_STAMP(name, tag) name.stamp(tag)
enum TraceTag { TT_WAIT_EMPTY = 1, TT_GOT_EMPTY = 2, TT_WAIT_FULL = 3, TT_GOT_FULL = 4, TT_ISSUED = 5, TT_WAIT_ACC = 6,
                TT_GOT_ACC = 7, TT_TILE_DONE = 8, TT_START = 9, TT_END = 10 };
#else
#define VT_TRACER(name, role)
#define VT_STAMP(name, tag)
#endif

// K-contiguous operand tile: `rows` rows of 16*C packed bytes -> rows of 128 int8, 128-byte swizzle.
template <int C, int SGN>
__device__ __forceinline__ void unpack_k_major(const uint8_t* src, uint8_t* dst, int rows, int tid, int nthreads) {
    constexpr int LC = C == 2 ? 1 : (C == 4 ? 2 : 3);   // log2(packed chunks per row)
    constexpr int E = 8 / C;
    const int chunks = rows << LC;
#pragma unroll 2
    for (int q = tid; q < chunks; q += nthreads) {
        const int r = q >> LC, j = q & ((1 << LC) - 1);
        const uint4 in = *reinterpret_cast<const uint4*>(src + (size_t)q * 16);
        expand_chunk<C, SGN>(in, dst + r * 128, j * E, r & 7);
    }
}
// N-contiguous B tile (the V operand): 128 rows of K, 64 codes each -> rows of 64 int8 grouped
// by 8 rows (512 bytes), 64-byte swizzle.
template <int C, int SGN>
__device__ __forceinline__ void unpack_mn_major(const uint8_t* src, uint8_t* dst, int tid, int nthreads) {
    constexpr int LH = C == 2 ? 0 : (C == 4 ? 1 : 2);   // log2(packed chunks per 64-code row)
    constexpr int E = 8 / C;
    const int chunks = BK << LH;
#pragma unroll 2
    for (int q = tid; q < chunks; q += nthreads) {
        const int r = q >> LH, h = q & ((1 << LH) - 1);
        const uint4 in = *reinterpret_cast<const uint4*>(src + (size_t)q * 16);
        expand_chunk<C, SGN>(in, dst + (r >> 3) * 512 + (r & 7) * 64, h * E, (r >> 1) & 3);
    }
}

template <int SGN>
__device__ __forceinline__ void unpack_k_major_c(int c, const uint8_t* src, uint8_t* dst, int rows, int tid, int nt) {
    if (c == 4) unpack_k_major<4, SGN>(src, dst, rows, tid, nt);
    else if (c == 2) unpack_k_major<2, SGN>(src, dst, rows, tid, nt);
    else unpack_k_major<8, SGN>(src, dst, rows, tid, nt);
}
template <int SGN>
__device__ __forceinline__ void unpack_mn_major_c(int c, const uint8_t* src, uint8_t* dst, int tid, int nt) {
    if (c == 4) unpack_mn_major<4, SGN>(src, dst, tid, nt);
    else if (c == 2) unpack_mn_major<2, SGN>(src, dst, tid, nt);
    else unpack_mn_major<8, SGN>(src, dst, tid, nt);
}

__device__ __forceinline__ void tile_coords(const GemmParams& P, int tile, int& m_tile, int& n_tile, int& inner,
                                            int& outer) {
    const int per_problem = P.m_tiles * P.n_tiles;
    const int prob = tile / per_problem;
    const int rem = tile - prob * per_problem;
    m_tile = rem / P.n_tiles;
    n_tile = rem - m_tile * P.n_tiles;
    outer = prob / P.n_inner;
    inner = prob - outer * P.n_inner;
}

// Barrier among the epilogue threads, bounded like every other wait (an mbarrier with one
// phase per tile instead of bar.sync, which could not give up).
__device__ __forceinline__ bool epi_barrier(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    ptx::mbar_arrive(bar);
    return mbar_wait(bar, parity, abort_flag);
}

// Epilogue of one row x 32 columns.  v[]: accumulators scaled by 2^shift; pa/pb/pq: the 32
// columns' parameters in shared memory (multiplier already carries 2^-shift).
// FULL: all 32 columns exist and 16-byte vector accesses are legal.
template <int KIND, bool FULL, int SMALL, bool HAS_RES>
__device__ __forceinline__ void epilogue_chunk(const GemmParams& P, const uint32_t (&v)[32], const float* pa,
                                               const float* pb, const float* pq, long long orow, long long colbase,
                                               int n0) {
    const int nvalid = FULL ? 32 : (P.N - n0 < 32 ? P.N - n0 : 32);
    if (KIND == EK_ACC) {
        int32_t* o = (int32_t*)P.out + orow * P.ld_out + colbase + n0;
        // 16-byte stores only where the row really starts on a 16-byte boundary (any leading dimension is allowed)
        if (FULL && (reinterpret_cast<uintptr_t>(o) & 15u) == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                reinterpret_cast<int4*>(o)[i] = make_int4((int)v[4 * i] >> P.shift, (int)v[4 * i + 1] >> P.shift,
                                                          (int)v[4 * i + 2] >> P.shift, (int)v[4 * i + 3] >> P.shift);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) if (i < nvalid) o[i] = (int)v[i] >> P.shift;
        }
        return;
    }
    // residual first: independent 16-byte loads in flight while the arithmetic runs
    const bool deq = (KIND == EK_DEQUANT || KIND == EK_DEQUANT_GELU);
    constexpr bool has_res = HAS_RES;
    float4 res[8];
    if (has_res) {
        const float* r = P.residual + orow * P.ld_res + colbase + n0;
        if (FULL && ((reinterpret_cast<uintptr_t>(r) & 15u) == 0)) {
#pragma unroll
            for (int i = 0; i < 8; ++i) res[i] = __ldg(reinterpret_cast<const float4*>(r) + i);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                res[i].x = (4 * i + 0 < nvalid) ? __ldg(r + 4 * i + 0) : 0.0f;
                res[i].y = (4 * i + 1 < nvalid) ? __ldg(r + 4 * i + 1) : 0.0f;
                res[i].z = (4 * i + 2 < nvalid) ? __ldg(r + 4 * i + 2) : 0.0f;
                res[i].w = (4 * i + 3 < nvalid) ? __ldg(r + 4 * i + 3) : 0.0f;
            }
        }
    }
    float* of = (float*)P.out + orow * P.ld_out + colbase + n0;                   // DEQUANT
    const bool vec_out = FULL && ((reinterpret_cast<uintptr_t>(of) & 15u) == 0);
    // The element loop below is straight-line code (no branch on run-time parameters), so the 32
    // independent per-column chains can overlap; the container width is only looked at when packing.
    // REQUANT: clamp, then add 1.5*2^23 + 2^(c-1) for signed codes (c = container bits): the sum's low
    // mantissa bits hold the code in offset binary (q + 2^(c-1) >= 0).  Offset codes pack with one
    // shift-add each and no masking; the constant high bits are subtracted per word and one XOR of
    // every container's top bit turns offset binary into two's complement.
    const bool sgn = P.out_qn < 0.0f;
    const float magic = 12582912.0f + (sgn ? (float)(1 << (P.out_c - 1)) : 0.0f);
    const float c_lo = P.unit_out ? 0.0f : P.out_qn, c_hi = P.unit_out ? 1.0f : P.out_qp, c_mul = P.unit_out ? P.out_qp : 1.0f;
    uint32_t code[32];
#pragma unroll
    for (int i4 = 0; i4 < 8; ++i4) {
        const float4 a4 = *reinterpret_cast<const float4*>(pa + 4 * i4);
        const float4 b4 = *reinterpret_cast<const float4*>(pb + 4 * i4);
        const float aa[4] = {a4.x, a4.y, a4.z, a4.w}, bb[4] = {b4.x, b4.y, b4.z, b4.w};
        float qq[4] = {0.f, 0.f, 0.f, 0.f};
        if (KIND == EK_REQUANT_GELU) {
            const float4 q4 = *reinterpret_cast<const float4*>(pq + 4 * i4);
            qq[0] = q4.x; qq[1] = q4.y; qq[2] = q4.z; qq[3] = q4.w;
        }
        const float rr[4] = {res[i4].x, res[i4].y, res[i4].z, res[i4].w};
        float y[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = 4 * i4 + j;
            // SMALL 2: scaled accumulator below 2^22, no shift (2^-shift rides on the multiplier);
            // SMALL 1: shift back first; SMALL 0: conversion instruction
            const float f = SMALL == 2 ? small_int_to_float((int)v[i])
                          : SMALL == 1 ? small_int_to_float((int)v[i] >> P.shift) : (float)(int)v[i];
            float val = fmaf(f, aa[j], bb[j]);
            if (KIND == EK_DEQUANT_GELU) val = gelu_f32(val);
            if (KIND == EK_REQUANT_GELU) val = gelu_scaled(val, qq[j]);      // qq = 0.5 / s_out (/ Qp when unit_out)
            if (has_res) val = val + rr[j];
            y[j] = val;
            if (!deq) code[i] = __float_as_uint(fmaf(fminf(fmaxf(val, c_lo), c_hi), c_mul, magic));
        }
        if (deq) {
            if (vec_out) {
                reinterpret_cast<float4*>(of)[i4] = make_float4(y[0], y[1], y[2], y[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) if (4 * i4 + j < nvalid) of[4 * i4 + j] = y[j];
            }
        }
    }
    if (deq) return;
    uint32_t wds[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (!FULL) {
        const uint32_t zero_code = __float_as_uint(magic);            // q = 0
#pragma unroll
        for (int i = 0; i < 32; ++i) if (i >= nvalid) code[i] = zero_code;
    }
    if (P.out_c == 4) {
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            uint32_t acc = code[8 * w];
#pragma unroll
            for (int j = 1; j < 8; ++j) acc += code[8 * w + j] << (4 * j);
            wds[w] = (acc - 0x4B400000u * 0x11111111u) ^ (sgn ? 0x88888888u : 0u);
        }
    } else if (P.out_c == 2) {
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            uint32_t acc = code[16 * w];
#pragma unroll
            for (int j = 1; j < 16; ++j) acc += code[16 * w + j] << (2 * j);
            wds[w] = (acc - 0x4B400000u * 0x55555555u) ^ (sgn ? 0xAAAAAAAAu : 0u);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            wds[i] = __byte_perm(__byte_perm(code[4 * i], code[4 * i + 1], 0x4040),
                                 __byte_perm(code[4 * i + 2], code[4 * i + 3], 0x4040), 0x5410) ^ (sgn ? 0x80808080u : 0u);
    }
    const int out_words = P.out_c;   // 32 codes = 4*out_c bytes
    const long long byte0 = ((colbase + n0) * P.out_c) >> 3;
    uint8_t* o = (uint8_t*)P.out + orow * P.ld_out + byte0;
    if (P.out_c == 4 && byte0 + 16 <= P.ld_out) {
        *reinterpret_cast<uint4*>(o) = make_uint4(wds[0], wds[1], wds[2], wds[3]);
    } else if (P.out_c == 8 && byte0 + 32 <= P.ld_out) {
        reinterpret_cast<uint4*>(o)[0] = make_uint4(wds[0], wds[1], wds[2], wds[3]);
        reinterpret_cast<uint4*>(o)[1] = make_uint4(wds[4], wds[5], wds[6], wds[7]);
    } else {
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (k < out_words && byte0 + 4 * k + 4 <= P.ld_out) reinterpret_cast<uint32_t*>(o)[k] = wds[k];
    }
    // row padding behind the last chunk of the last column tile
    if (P.col_off_inner == 0 && (!FULL || n0 + 32 >= P.N)) {
        for (long long off = byte0 + 4 * out_words; off + 4 <= P.ld_out; off += 4)
            *reinterpret_cast<uint32_t*>((uint8_t*)P.out + orow * P.ld_out + off) = 0u;
    }
}

// Requantizing epilogue of whole 16-column blocks as a ROLLED loop.  The fully unrolled 32-column
// form above is ~900 instructions of straight-line code that every warp walks once per chunk, so it
// streams through the instruction cache; this body (16 independent element chains) is a quarter of
// that and is re-used by every block of the warp's share.  Columns [col_begin, col_end) of the tile,
// all of them real columns; col_begin and col_end are multiples of 16.  Whole-warp call: the TMEM
// load is a warp-wide instruction, so lanes whose row lies past M run the arithmetic too and only
// their stores are masked.
// BYTES: the output container is one byte per code, known at compile time, so the packing of each group of four
// codes can be scheduled right behind their arithmetic instead of after all sixteen (fewer live registers, more
// independent work in flight: fc1 94 -> 91 us).
template <int KIND, int SMALL, bool UNIT, bool BYTES>
__device__ __forceinline__ void epilogue_requant_blocks(const GemmParams& P, const EpiParams& ep, int buf,
                                                       uint32_t t_row, bool row_ok, long long orow, long long col0,
                                                       int col_begin, int col_end) {
    const bool sgn = P.out_qn < 0.0f;
    const float magic = 12582912.0f + (sgn ? (float)(1 << ((BYTES ? 8 : P.out_c) - 1)) : 0.0f);
    uint8_t* const o_row = (uint8_t*)P.out + orow * P.ld_out;
    // Byte codes without an activation: the 16 bytes of an even block wait in registers for the odd block and
    // the two leave as ONE 32-byte store.  A warp's store touches 32 different rows whatever its width, so this
    // halves the number of row segments the load/store unit has to walk (qkv, batch 128: 62 -> 57 us).  The
    // GELU kind keeps 16-byte stores: there the extra registers and branch cost more than the stores.
    constexpr bool PAIR_STORES = (KIND == EK_REQUANT);
    uint32_t held[4] = {0u, 0u, 0u, 0u};
#pragma unroll 1
    for (int col = col_begin; col < col_end; col += 16) {
        uint32_t v[16];
        ptx::tmem_ld16(t_row + (uint32_t)col, v);
        ptx::tmem_ld_wait();
        const float* pa = &ep.a[buf][col];
        const float* pb = &ep.b[buf][col];
        const float* pq = &ep.q[buf][col];
        uint32_t code[16];
#pragma unroll
        for (int i2 = 0; i2 < 8; ++i2) {
            // two columns per step: the fp32 arithmetic runs as packed pairs (bit-identical per element)
            const float2 a2 = reinterpret_cast<const float2*>(pa)[i2], b2 = reinterpret_cast<const float2*>(pb)[i2];
            float f0, f1;
            if (SMALL == 0) {
                f0 = (float)(int)v[2 * i2];
                f1 = (float)(int)v[2 * i2 + 1];
            } else {
                // 1.5*2^23 + acc as float bits, then the packed subtraction of 1.5*2^23
                const int s = SMALL == 1 ? P.shift : 0;
                const f32x2 m = f2_pack(__int_as_float(0x4B400000 + ((int)v[2 * i2] >> s)),
                                        __int_as_float(0x4B400000 + ((int)v[2 * i2 + 1] >> s)));
                f2_unpack(f2_add(m, f2_dup(-12582912.0f)), f0, f1);
            }
            const f32x2 y = f2_fma(f2_pack(f0, f1), f2_pack(a2.x, a2.y), f2_pack(b2.x, b2.y));
            float y0, y1;
            f2_unpack(y, y0, y1);
            if (UNIT) {
                // unsigned codes after GELU: the value arrives clamped to [0, 1] in units of Qp
                const float2 q2 = reinterpret_cast<const float2*>(pq)[i2];
                float e0, e1, w0, w1;
                gelu_erfc_term2(y0, y1, e0, e1);
                f2_unpack(f2_mul(y, f2_pack(q2.x, q2.y)), w0, w1);
                const float u0 = __saturatef(fmaf(-fabsf(w0), e0, w0 + fabsf(w0)));
                const float u1 = __saturatef(fmaf(-fabsf(w1), e1, w1 + fabsf(w1)));
                float c0, c1;
                f2_unpack(f2_fma(f2_pack(u0, u1), f2_dup(P.out_qp), f2_dup(magic)), c0, c1);
                code[2 * i2] = __float_as_uint(c0);
                code[2 * i2 + 1] = __float_as_uint(c1);
            } else {
                if (KIND == EK_REQUANT_GELU) {
                    const float2 q2 = reinterpret_cast<const float2*>(pq)[i2];
                    y0 = gelu_scaled(y0, q2.x);
                    y1 = gelu_scaled(y1, q2.y);
                }
                float c0, c1;
                f2_unpack(f2_add(f2_pack(fminf(fmaxf(y0, P.out_qn), P.out_qp), fminf(fmaxf(y1, P.out_qn), P.out_qp)),
                                 f2_dup(magic)), c0, c1);
                code[2 * i2] = __float_as_uint(c0);
                code[2 * i2 + 1] = __float_as_uint(c1);
            }
        }
        // offset-binary packing as in epilogue_chunk: 16 codes = 2 * out_c bytes
        const long long c = col0 + col;
        if (BYTES) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                w[i] = __byte_perm(__byte_perm(code[4 * i], code[4 * i + 1], 0x4040),
                                   __byte_perm(code[4 * i + 2], code[4 * i + 3], 0x4040), 0x5410) ^ (sgn ? 0x80808080u : 0u);
            const bool odd = ((col - col_begin) & 16) != 0;
            if (PAIR_STORES && !odd && col + 16 < col_end) {
                held[0] = w[0]; held[1] = w[1]; held[2] = w[2]; held[3] = w[3];
            } else if (PAIR_STORES && odd && (reinterpret_cast<uintptr_t>(o_row + c - 16) & 31u) == 0) {
                if (row_ok) ptx::st_global_32B(o_row + c - 16, held, w);
            } else {
                if (PAIR_STORES && odd && row_ok)
                    *reinterpret_cast<uint4*>(o_row + c - 16) = make_uint4(held[0], held[1], held[2], held[3]);
                if (row_ok) *reinterpret_cast<uint4*>(o_row + c) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        } else if (P.out_c == 4) {
            uint32_t w[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t acc = code[8 * h];
#pragma unroll
                for (int j = 1; j < 8; ++j) acc += code[8 * h + j] << (4 * j);
                w[h] = (acc - 0x4B400000u * 0x11111111u) ^ (sgn ? 0x88888888u : 0u);
            }
            if (row_ok) *reinterpret_cast<uint2*>(o_row + (c >> 1)) = make_uint2(w[0], w[1]);
        } else {
            uint32_t acc = code[0];
#pragma unroll
            for (int j = 1; j < 16; ++j) acc += code[j] << (2 * j);
            if (row_ok) *reinterpret_cast<uint32_t*>(o_row + (c >> 2)) = (acc - 0x4B400000u * 0x55555555u) ^ (sgn ? 0xAAAAAAAAu : 0u);
        }
    }
}

constexpr int STAGE_LD = 36;                                  // floats per staged row: 144 bytes keeps 16-byte accesses conflict-free
constexpr int STAGE_FLOATS = 32 * STAGE_LD;                   // one 32 x 32 fp32 block
constexpr int STAGE_BYTES = 2 * STAGE_FLOATS * 4;             // two blocks per epilogue warp: the residual of the next
                                                              // chunk lands in one while the other is worked on

// Starts the asynchronous copy of one 32 x 32 block of the residual into a staging block (coalesced:
// each instruction covers four rows of 128 bytes) and closes it as one copy group of the calling thread.
__device__ __forceinline__ void residual_prefetch(const GemmParams& P, float* block, int lane, long long orow0,
                                                  int rows_valid, long long col) {
    const int cr = lane >> 3, cc = (lane & 7) * 4;
    const float* r0 = P.residual + orow0 * P.ld_res + col + cc;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = cr + 4 * i;
        if (r < rows_valid) ptx::cp_async16(ptx::smem_addr(block + r * STAGE_LD + cc), r0 + (long long)r * P.ld_res);
    }
    ptx::cp_async_commit();
}

// fp32 epilogue of a 32 x 32 block through a shared-memory transposition, so that every global
// access of the warp covers whole 128-byte lines: the TMEM layout gives each thread one ROW of the
// block, while coalesced loads / stores want each instruction to cover four rows of 128 bytes.
//   residual: already copied into `stage` by residual_prefetch (the caller has waited for the copy
//             group and synchronised the warp) -> each thread reads its own row;
//   result  : each thread writes its own row -> stage -> coalesced float4 stores.
// Whole-warp call (rows past M take part and are masked at the global accesses).
template <int KIND, int SMALL, bool HAS_RES>
__device__ __forceinline__ void epilogue_chunk_staged(const GemmParams& P, const uint32_t (&v)[32], const float* pa,
                                                     const float* pb, float* stage, int lane, long long orow0,
                                                     int rows_valid, long long colbase, int n0) {
    const int cr = lane >> 3, cc = (lane & 7) * 4;              // cooperative phase: row cr + 4*i, columns cc..cc+3
    float* const my_row = stage + lane * STAGE_LD;
    float4 y[8];
#pragma unroll
    for (int i4 = 0; i4 < 8; ++i4) {
        const float4 a4 = *reinterpret_cast<const float4*>(pa + 4 * i4);
        const float4 b4 = *reinterpret_cast<const float4*>(pb + 4 * i4);
        float4 r4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (HAS_RES) r4 = *reinterpret_cast<const float4*>(my_row + 4 * i4);
        const float aa[4] = {a4.x, a4.y, a4.z, a4.w}, bb[4] = {b4.x, b4.y, b4.z, b4.w}, rr[4] = {r4.x, r4.y, r4.z, r4.w};
        float o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = 4 * i4 + j;
            const float f = SMALL == 2 ? small_int_to_float((int)v[i])
                          : SMALL == 1 ? small_int_to_float((int)v[i] >> P.shift) : (float)(int)v[i];
            float val = fmaf(f, aa[j], bb[j]);
            if (KIND == EK_DEQUANT_GELU) val = gelu_f32(val);
            if (HAS_RES) val = val + rr[j];
            o[j] = val;
        }
        y[i4] = make_float4(o[0], o[1], o[2], o[3]);
    }
    if (HAS_RES) __syncwarp();                                  // every row has been read before it is overwritten
#pragma unroll
    for (int i4 = 0; i4 < 8; ++i4) *reinterpret_cast<float4*>(my_row + 4 * i4) = y[i4];
    __syncwarp();
    float* o0 = (float*)P.out + orow0 * P.ld_out + colbase + n0 + cc;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = cr + 4 * i;
        const float4 t = *reinterpret_cast<const float4*>(stage + r * STAGE_LD + cc);
        if (r < rows_valid) *reinterpret_cast<float4*>(o0 + (long long)r * P.ld_out) = t;
    }
    __syncwarp();                                               // the buffer is free for the next chunk
}

// NG consecutive 64-channel heads of one accumulator row, starting at tile column `col` (their recurrences are
// independent dependency chains, stepped side by side when NG > 1).
template <int SMALL, int NG>
__device__ __forceinline__ void norm_heads(const GemmParams& P, const EpiParams& ep, int buf, uint32_t t_row, bool row_ok,
                                           long long orow, int tile_col0, int col, const float* refs_s, const float* sgn_s) {
    uint8_t* const o_row = (uint8_t*)P.out + orow * P.ld_out;
    const int heads = P.norm_dim >> 6;
    const uint32_t mask = (1u << P.out_c) - 1u;
    auto to_float = [&](uint32_t v) -> float {
        return SMALL == 2 ? small_int_to_float((int)v) : SMALL == 1 ? small_int_to_float((int)v >> P.shift) : (float)(int)v;
    };
    const float* pa = &ep.a[buf][col];
    const float* pb = &ep.b[buf][col];
    // pass 1: running statistics over each head's 64 channels, in order
    float mu[NG], S[NG];
#pragma unroll
    for (int u = 0; u < NG; ++u) { mu[u] = 0.0f; S[u] = 0.0f; }
#pragma unroll
    for (int blk = 0; blk < 4; ++blk) {
        uint32_t v[NG][16];
#pragma unroll
        for (int u = 0; u < NG; ++u) ptx::tmem_ld16(t_row + (uint32_t)(col + 64 * u + 16 * blk), v[u]);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int idx = 16 * blk + i;
            const float fi = (float)(idx + 1), ri = 1.0f / (float)(idx + 1);       // compile-time constants: i and RN(1/i)
#pragma unroll
            for (int u = 0; u < NG; ++u) {
                const float y = fmaf(to_float(v[u][i]), pa[64 * u + idx], pb[64 * u + idx]);
                const float delta = __fadd_rn(y, -mu[u]);
                // RN(delta / i): quotient estimate, exact remainder in one FMA, one correction
                const float q0 = __fmul_rn(delta, ri);
                const float rem = __fmaf_rn(-q0, fi, delta);
                mu[u] = __fadd_rn(mu[u], __fmaf_rn(rem, ri, q0));
                S[u] = __fadd_rn(S[u], __fmul_rn(delta, __fadd_rn(y, -mu[u])));
            }
        }
    }
#pragma unroll
    for (int u = 0; u < NG; ++u) {
        const int gcol = tile_col0 + col + 64 * u;
        const int seg = gcol / P.norm_dim;
        const float V = __fadd_rn(S[u], P.n_eps);
        if (P.norm_stats != nullptr && row_ok) {
            const int head = (gcol - seg * P.norm_dim) >> 6;
            float* st = P.norm_stats + ((long long)seg * P.M * heads + orow * heads + head) * 2;
            st[0] = mu[u];
            st[1] = V;
        }
        // pass 2: levels
        const float* rs = refs_s + (size_t)seg * 64 * 16;
        const float* sg = sgn_s + seg * 64;
#pragma unroll
        for (int blk = 0; blk < 4; ++blk) {
            uint32_t v[16];
            ptx::tmem_ld16(t_row + (uint32_t)(col + 64 * u + 16 * blk), v);
            ptx::tmem_ld_wait();
            uint32_t code[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int idx = 16 * blk + i;
                const float y = fmaf(to_float(v[i]), pa[64 * u + idx], pb[64 * u + idx]);
                const float d = __fmul_rn(__fadd_rn(y, -mu[u]), sg[idx]);             // exact sign change
                const float ds = copysignf(__fmul_rn(d, d), d);
                const float* r = rs + idx * 16;
                // four bisection steps whatever the code width: entries past the last reference are +inf and never
                // counted, and a fixed depth lets the sixteen columns' dependent loads interleave
                int cnt = 0;
#pragma unroll
                for (int step = 8; step > 0; step >>= 1)
                    cnt += ds > __fmul_rn(V, r[cnt + step - 1]) ? step : 0;
                code[i] = (uint32_t)(P.norm_qn + cnt) & mask;
            }
            const long long c = gcol + 16 * blk;
            if (P.out_c == 8) {
                uint32_t w[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) w[k] = code[4 * k] | (code[4 * k + 1] << 8) | (code[4 * k + 2] << 16) | (code[4 * k + 3] << 24);
                if (row_ok) *reinterpret_cast<uint4*>(o_row + c) = make_uint4(w[0], w[1], w[2], w[3]);
            } else if (P.out_c == 4) {
                uint32_t w[2] = {0u, 0u};
#pragma unroll
                for (int k = 0; k < 16; ++k) w[k >> 3] |= code[k] << (4 * (k & 7));
                if (row_ok) *reinterpret_cast<uint2*>(o_row + (c >> 1)) = make_uint2(w[0], w[1]);
            } else {
                uint32_t w = 0u;
#pragma unroll
                for (int k = 0; k < 16; ++k) w |= code[k] << (2 * k);
                if (row_ok) *reinterpret_cast<uint32_t*>(o_row + (c >> 2)) = w;
            }
        }
    }
}

// Epilogue of the QKV projection with the per-head quantizing LayerNorm of Section IV-C (Eq. 5 statistics, comparator of
// Fig. 5(b)) on the Q and K heads; the V heads are requantized as usual.  A thread owns an accumulator ROW, so the 64
// channels of a head are its own: it walks them in order through the recurrence of Eq. 5
//     delta = y_i - mu;  mu += delta / i;  S += delta * (y_i - mu)          (one rounded fp32 operation each)
// with y_i = fma(float(acc_i), s_x s_w[i], b_i), forms V = S + n*eps, reads the accumulators a second time and finds each
// level as Qn + number of references r with copysign(d*d, d) > V*r, d = y - mu (negated where the gain is negative) by
// bisection over the column's ascending references in shared memory.  The fp32 Q and K never exist in memory.
// refs_s: [2][64][16] (Q then K; entries past 2^bits - 1 unused), sgn_s: [2][64] (+1 / -1).
template <int SMALL>
__device__ __forceinline__ void epilogue_qkv_norm(const GemmParams& P, const EpiParams& ep, int buf, uint32_t t_row, bool row_ok,
                                                  long long orow, int n_tile, int slice, const float* refs_s, const float* sgn_s) {
    const int tile_col0 = n_tile * P.bn;
    const int valid = P.N - tile_col0 < P.bn ? P.N - tile_col0 : P.bn;      // a multiple of 64
    const int groups = valid >> 6, n_slices = P.epi_warps >> 2;
    const int g_begin = groups * slice / n_slices, g_end = groups * (slice + 1) / n_slices;
    const int v_col0 = 2 * P.norm_dim;
    for (int g = g_begin; g < g_end;) {
        const int col = g << 6, gcol = tile_col0 + col;
        if (gcol >= v_col0) {
            // V head: plain requantization of its 64 columns
            if (P.out_c == 8) epilogue_requant_blocks<EK_REQUANT, SMALL, false, true>(P, ep, buf, t_row, row_ok, orow, tile_col0, col, col + 64);
            else epilogue_requant_blocks<EK_REQUANT, SMALL, false, false>(P, ep, buf, t_row, row_ok, orow, tile_col0, col, col + 64);
            g += 1;
        } else {
            // (stepping two heads' recurrences side by side was measured slower: 67 against 53 us at DeiT-S width,
            // batch 64 -- the second chain's registers spill)
            norm_heads<SMALL, 1>(P, ep, buf, t_row, row_ok, orow, tile_col0, col, refs_s, sgn_s);
            g += 1;
        }
    }
    // row padding behind the last column of the matrix
    if (row_ok && slice == n_slices - 1 && tile_col0 + valid >= P.N) {
        uint8_t* const o_row = (uint8_t*)P.out + orow * P.ld_out;
        for (long long off = ((long long)P.N * P.out_c) >> 3; off + 4 <= P.ld_out; off += 4)
            *reinterpret_cast<uint32_t*>(o_row + off) = 0u;
    }
    __syncwarp();
}

// The warps of a lane quarter split the tile's 32-column chunks into contiguous shares.
__device__ __forceinline__ void chunk_share(const GemmParams& P, int slice, int& c_begin, int& c_end) {
    const int n_slices = P.epi_warps >> 2;
    const int n_chunks = (P.bn + 31) / 32, base = n_chunks / n_slices, rem = n_chunks % n_slices;
    c_begin = slice * base + (slice < rem ? slice : rem);
    c_end = c_begin + base + (slice < rem ? 1 : 0);
}

// Residual of the warp's first chunk of a tile, requested before the warp waits for the tile's
// accumulators.  Returns whether a copy group was opened (the chunk takes the staged path).
template <int KIND>
__device__ __forceinline__ bool epilogue_prefetch_first(const GemmParams& P, long long colbase, int n_tile, int slice,
                                                        float* stage, int lane, long long orow0, int rows_valid) {
    constexpr bool is_deq = (KIND == EK_DEQUANT || KIND == EK_DEQUANT_GELU);
    if (!is_deq || stage == nullptr || P.residual == nullptr) return false;
    int c_begin, c_end;
    chunk_share(P, slice, c_begin, c_end);
    const int n0 = n_tile * P.bn + c_begin * 32;
    if (c_begin >= c_end || n0 + 32 > P.N) return false;
    residual_prefetch(P, stage, lane, orow0, rows_valid, colbase + n0);
    return true;
}

template <int KIND, int SMALL>
__device__ __forceinline__ void epilogue_tile(const GemmParams& P, const EpiParams& ep, int buf, uint32_t t_row,
                                              bool row_ok, long long orow, long long colbase, int n_tile, int slice,
                                              float* stage, int lane, int rows_valid, bool first_prefetched,
                                              const float* refs_s, const float* sgn_s) {
    if constexpr (KIND == EK_QKV_NORM) {
        epilogue_qkv_norm<SMALL>(P, ep, buf, t_row, row_ok, orow, n_tile, slice, refs_s, sgn_s);
        return;
    }
    int c_begin, c_end;
    chunk_share(P, slice, c_begin, c_end);
    constexpr bool is_req = (KIND == EK_REQUANT || KIND == EK_REQUANT_GELU);
    if (is_req && (n_tile + 1) * P.bn <= P.N && (P.bn & 31) == 0 && (colbase & 15) == 0) {
        // every column of the tile is real: rolled 16-column blocks
        const long long col0 = colbase + (long long)n_tile * P.bn;
        if (c_begin < c_end) {
            if (KIND == EK_REQUANT_GELU && P.unit_out)
                if (P.out_c == 8) epilogue_requant_blocks<EK_REQUANT_GELU, SMALL, true, true>(P, ep, buf, t_row, row_ok, orow, col0, c_begin * 32, c_end * 32);
                else epilogue_requant_blocks<EK_REQUANT_GELU, SMALL, true, false>(P, ep, buf, t_row, row_ok, orow, col0, c_begin * 32, c_end * 32);
            else
                if (P.out_c == 8) epilogue_requant_blocks<is_req ? KIND : EK_REQUANT, SMALL, false, true>(P, ep, buf, t_row, row_ok, orow, col0, c_begin * 32, c_end * 32);
                else epilogue_requant_blocks<is_req ? KIND : EK_REQUANT, SMALL, false, false>(P, ep, buf, t_row, row_ok, orow, col0, c_begin * 32, c_end * 32);
        }
        // row padding behind the last column of the matrix
        if (row_ok && P.col_off_inner == 0 && n_tile * P.bn + c_end * 32 >= P.N && c_end > c_begin) {
            for (long long off = ((long long)P.N * P.out_c) >> 3; off + 4 <= P.ld_out; off += 4)
                *reinterpret_cast<uint32_t*>((uint8_t*)P.out + orow * P.ld_out + off) = 0u;
        }
        __syncwarp();
        return;
    }
    bool have_res = first_prefetched;                           // the current chunk's residual copy is already open
    for (int chunk = c_begin; chunk < c_end; ++chunk) {
        const int n0 = n_tile * P.bn + chunk * 32;
        if (n0 >= P.N) break;
        uint32_t v[32];
        ptx::tmem_ld32(t_row + (uint32_t)(chunk * 32), v);
        constexpr bool is_deq = (KIND == EK_DEQUANT || KIND == EK_DEQUANT_GELU);
        const bool staged_here = is_deq && stage != nullptr && n0 + 32 <= P.N;
        float* const block = stage + ((chunk - c_begin) & 1) * STAGE_FLOATS;
        const long long orow0 = orow - lane;
        if (staged_here && P.residual != nullptr) {
            // this chunk's residual block is on its way (or is requested now); the next chunk's is requested
            // into the other block before this one is awaited, so its latency hides behind the arithmetic
            if (!have_res) residual_prefetch(P, block, lane, orow0, rows_valid, colbase + n0);
            have_res = chunk + 1 < c_end && n0 + 64 <= P.N;
            if (have_res) {
                residual_prefetch(P, stage + ((chunk + 1 - c_begin) & 1) * STAGE_FLOATS, lane, orow0, rows_valid, colbase + n0 + 32);
                ptx::cp_async_wait<1>();
            } else {
                ptx::cp_async_wait<0>();
            }
            __syncwarp();                                       // every lane's copies have landed
        }
        ptx::tmem_ld_wait();
        if (staged_here) {
            // full 32-column chunk of an fp32 output: coalesced path (stage is only set when the host has
            // checked 16-byte alignment of the output, the residual and their leading dimensions)
            const float* pa = &ep.a[buf][chunk * 32];
            const float* pb = &ep.b[buf][chunk * 32];
            if (P.residual != nullptr) epilogue_chunk_staged<is_deq ? KIND : EK_DEQUANT, SMALL, true>(P, v, pa, pb, block, lane, orow0, rows_valid, colbase, n0);
            else epilogue_chunk_staged<is_deq ? KIND : EK_DEQUANT, SMALL, false>(P, v, pa, pb, block, lane, orow0, rows_valid, colbase, n0);
        } else if (row_ok) {
            const float* pa = &ep.a[buf][chunk * 32];
            const float* pb = &ep.b[buf][chunk * 32];
            const float* pq = &ep.q[buf][chunk * 32];
            constexpr bool can_res = (KIND == EK_DEQUANT || KIND == EK_DEQUANT_GELU);
            if (can_res && P.residual != nullptr) {
                if (n0 + 32 <= P.N) epilogue_chunk<KIND, true, SMALL, can_res>(P, v, pa, pb, pq, orow, colbase, n0);
                else epilogue_chunk<KIND, false, SMALL, can_res>(P, v, pa, pb, pq, orow, colbase, n0);
            } else {
                if (n0 + 32 <= P.N) epilogue_chunk<KIND, true, SMALL, false>(P, v, pa, pb, pq, orow, colbase, n0);
                else epilogue_chunk<KIND, false, SMALL, false>(P, v, pa, pb, pq, orow, colbase, n0);
            }
        }
        __syncwarp();
    }
}

template <int KIND>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ GemmParams P) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ Bars bars;
    __shared__ __align__(16) EpiParams epi_params;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ __align__(16) float norm_refs_s[KIND == EK_QKV_NORM ? 2 * 64 * 16 : 4];   // comparator references of the Q and K norms
    __shared__ float norm_sgn_s[KIND == EK_QKV_NORM ? 2 * 64 : 1];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem_gen = smem_raw + (smem_base - ptx::smem_addr(smem_raw));
    const uint32_t stage_i = P.ia_bytes + P.ib_bytes, stage_p = P.pa_bytes + P.pb_bytes;
    const uint32_t packed_off = (uint32_t)P.ns_i * stage_i;
    const bool any_packed = !(P.a_direct && P.b_direct), any_direct = P.a_direct || P.b_direct;
    volatile int* abort_ptr = &abort_flag;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < MAX_STAGES; ++s) {
            ptx::mbar_init(ptx::smem_addr(&bars.p_full[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&bars.p_empty[s]), UNPACK_WARPS);
            ptx::mbar_init(ptx::smem_addr(&bars.i_full[s]), (any_packed ? UNPACK_WARPS : 0) + (any_direct ? 1 : 0));
            ptx::mbar_init(ptx::smem_addr(&bars.i_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_addr(&bars.acc_full[b]), 1);
            ptx::mbar_init(ptx::smem_addr(&bars.acc_empty[b]), P.epi_warps);
        }
        ptx::mbar_init(ptx::smem_addr(&bars.epi_sync), P.epi_warps * 32);
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == WARP_MMA) {
        ptx::tmem_alloc(ptx::smem_addr(&tmem_base_slot), P.tmem_cols);
        ptx::tmem_relinquish();
    }
    if (warp == WARP_TMA && lane == 0) {
        ptx::prefetch_tensormap(&map_a);
        ptx::prefetch_tensormap(&map_b);
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t acc_stride = P.tmem_cols >> 1;
    grid_dependency_wait();        // operands, parameters and the residual may come from the previous kernel
    grid_dependency_launch();

    if (warp == WARP_TMA) {
        // ------------------------------ TMA producer -------------------------------
        if (lane == 0) {
            VT_TRACER(tr, 0);
            VT_STAMP(tr, TT_START);
            int it = 0;
            bool ok = true;
            const uint32_t packed_bytes = (P.a_direct ? 0u : P.pa_bytes) + (P.b_direct ? 0u : P.pb_bytes);
            const uint32_t direct_bytes = (P.a_direct ? P.ia_bytes : 0u) + (P.b_direct ? P.ib_bytes : 0u);
            if (P.a_direct && P.b_direct) {
                // both operands go straight into the operand ring: slot and phase advance by increments
                const uint32_t full0 = ptx::smem_addr(&bars.i_full[0]), empty0 = ptx::smem_addr(&bars.i_empty[0]);
                const int k_blocks = P.k_blocks, ns = P.ns_i;
                int s = 0;
                uint32_t ph = 1u, dst = smem_base;
                for (int tile = blockIdx.x; ok && tile < P.total_tiles; tile += gridDim.x) {
                    int m_tile, n_tile, inner, outer;
                    tile_coords(P, tile, m_tile, n_tile, inner, outer);
                    const int m0 = m_tile * BM, n0 = n_tile * P.bn;
                    for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                        VT_STAMP(tr, TT_WAIT_EMPTY);
                        if (!mbar_wait(empty0 + 8u * (uint32_t)s, ph, abort_ptr)) { ok = false; break; }
                        VT_STAMP(tr, TT_GOT_EMPTY);
                        const uint32_t full = full0 + 8u * (uint32_t)s;
                        ptx::mbar_arrive_expect_tx(full, direct_bytes);
                        ptx::tma_load_4d(dst, &map_a, full, kb * BK, m0, inner, outer);
                        ptx::tma_load_4d(dst + P.ia_bytes, &map_b, full, kb * BK, n0, inner, outer);
                        if (++s == ns) { s = 0; ph ^= 1u; dst = smem_base; } else dst += stage_i;
                    }
                }
            } else
            for (int tile = blockIdx.x; ok && tile < P.total_tiles; tile += gridDim.x) {
                int m_tile, n_tile, inner, outer;
                tile_coords(P, tile, m_tile, n_tile, inner, outer);
                for (int kb = 0; kb < P.k_blocks; ++kb, ++it) {
                    const int sp = it % P.ns_p, si = it % P.ns_i;
                    const uint32_t php = (uint32_t)(it / P.ns_p) & 1u, phi = (uint32_t)(it / P.ns_i) & 1u;
                    const uint32_t p_full = ptx::smem_addr(&bars.p_full[sp]), i_full = ptx::smem_addr(&bars.i_full[si]);
                    const uint32_t p_dst = smem_base + packed_off + (uint32_t)sp * stage_p;
                    const uint32_t i_dst = smem_base + (uint32_t)si * stage_i;
                    if (any_packed) {
                        if (!mbar_wait(ptx::smem_addr(&bars.p_empty[sp]), php ^ 1u, abort_ptr)) { ok = false; break; }
                        ptx::mbar_arrive_expect_tx(p_full, packed_bytes);
                    }
                    if (any_direct) {
                        VT_STAMP(tr, TT_WAIT_EMPTY);
                        if (!mbar_wait(ptx::smem_addr(&bars.i_empty[si]), phi ^ 1u, abort_ptr)) { ok = false; break; }
                        VT_STAMP(tr, TT_GOT_EMPTY);
                        ptx::mbar_arrive_expect_tx(i_full, direct_bytes);
                    }
                    if (P.a_direct) ptx::tma_load_4d(i_dst, &map_a, i_full, kb * BK, m_tile * BM, inner, outer);
                    else ptx::tma_load_4d(p_dst, &map_a, p_full, kb * 16 * P.ca, m_tile * BM, inner, outer);
                    if (P.b_direct)
                        ptx::tma_load_4d(i_dst + P.ia_bytes, &map_b, i_full, kb * BK, n_tile * P.bn, inner, outer);
                    else if (P.b_mn_major)
                        ptx::tma_load_4d(p_dst + P.pa_bytes, &map_b, p_full, 0, kb * BK, inner, outer);
                    else
                        ptx::tma_load_4d(p_dst + P.pa_bytes, &map_b, p_full, kb * 16 * P.cb, n_tile * P.bn, inner, outer);
                }
            }
            if (!ok) {
                // give the copies still in flight a bounded chance to land before the CTA exits
                for (int j = (it > MAX_STAGES ? it - MAX_STAGES : 0); j < it; ++j) {
                    if (any_packed && j + P.ns_p >= it) {
                        const uint32_t bar = ptx::smem_addr(&bars.p_full[j % P.ns_p]);
                        for (int spin = 0; spin < (1 << 20) && !ptx::mbar_try_wait(bar, (uint32_t)(j / P.ns_p) & 1u); ++spin) {}
                    }
                    if (any_direct && j + P.ns_i >= it) {
                        const uint32_t bar = ptx::smem_addr(&bars.i_full[j % P.ns_i]);
                        for (int spin = 0; spin < (1 << 20) && !ptx::mbar_try_wait(bar, (uint32_t)(j / P.ns_i) & 1u); ++spin) {}
                    }
                }
            }
        }
    } else if (warp == WARP_MMA) {
        // ------------------------------- MMA issuer --------------------------------
        if (lane == 0) {
            const uint32_t idesc = ptx::idesc_i8(BM, P.bn, P.a_signed, P.b_signed, P.b_mn_major);
            VT_TRACER(tr, 1);
            VT_STAMP(tr, TT_START);
            // This one thread feeds the tensor core, and a lone thread runs its dependent scalar instructions a few
            // cycles apart: everything the loop needs is therefore kept in registers and advanced by additions (no
            // division for the ring slot, no descriptor rebuilt per K block); the four MMAs of a whole K block are
            // issued back to back.
            const uint64_t a_desc0 = ptx::smem_desc(smem_base, 16, 1024, ptx::SWIZZLE_128B);
            const uint64_t b_desc0 = P.b_mn_major ? ptx::smem_desc(smem_base + P.ia_bytes, 16, 512, ptx::SWIZZLE_64B)
                                                  : ptx::smem_desc(smem_base + P.ia_bytes, 16, 1024, ptx::SWIZZLE_128B);
            const uint64_t stage_step = (uint64_t)(stage_i >> 4);            // descriptor address field counts 16-byte units
            const uint64_t b_kstep = P.b_mn_major ? 128u : 2u;
            const uint32_t full0 = ptx::smem_addr(&bars.i_full[0]), empty0 = ptx::smem_addr(&bars.i_empty[0]);
            const int k_blocks = P.k_blocks, ns = P.ns_i;
            const int last_steps = (P.K - (k_blocks - 1) * BK + 31) / 32;     // MMAs of the last (possibly partial) K block
            int s = 0, tl = 0;
            uint32_t ph = 0;
            uint64_t a_desc = a_desc0, b_desc = b_desc0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < P.total_tiles; tile += gridDim.x, ++tl) {
                const int buf = tl & 1;
                const uint32_t acc_ph = (uint32_t)(tl >> 1) & 1u;
                VT_STAMP(tr, TT_WAIT_EMPTY);
                if (!mbar_wait(ptx::smem_addr(&bars.acc_empty[buf]), acc_ph ^ 1u, abort_ptr)) { ok = false; break; }
                VT_STAMP(tr, TT_GOT_EMPTY);
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * acc_stride;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    VT_STAMP(tr, TT_WAIT_FULL);
                    if (!mbar_wait(full0 + 8u * (uint32_t)s, ph, abort_ptr)) { ok = false; break; }
                    VT_STAMP(tr, TT_GOT_FULL);
                    ptx::tc_fence_after();
                    // 32 int8 of K per MMA: 32 bytes along a swizzled row, or four 8-row
                    // groups (4 * 512 bytes) when K is the slow axis of the B tile
                    if (kb + 1 < k_blocks || last_steps == 4) {
                        ptx::mma_i8(d_tmem, a_desc, b_desc, idesc, kb != 0 ? 1u : 0u);
                        ptx::mma_i8(d_tmem, a_desc + 2u, b_desc + b_kstep, idesc, 1u);
                        ptx::mma_i8(d_tmem, a_desc + 4u, b_desc + 2u * b_kstep, idesc, 1u);
                        ptx::mma_i8(d_tmem, a_desc + 6u, b_desc + 3u * b_kstep, idesc, 1u);
                    } else {
                        for (int k = 0; k < last_steps; ++k)
                            ptx::mma_i8(d_tmem, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)k * b_kstep, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    ptx::mma_commit(empty0 + 8u * (uint32_t)s);
                    if (++s == ns) { s = 0; ph ^= 1u; a_desc = a_desc0; b_desc = b_desc0; }
                    else { a_desc += stage_step; b_desc += stage_step; }
                }
                if (ok) ptx::mma_commit(ptx::smem_addr(&bars.acc_full[buf]));
                VT_STAMP(tr, TT_ISSUED);
            }
        }
    } else if (warp >= WARP_UNPACK0 + (P.epi_warps - EPI_WARPS)) {
        // --------------------------------- unpack ----------------------------------
        if (any_packed) {
            const int tid_u = threadIdx.x - WARP_UNPACK0 * 32;
            constexpr int NU = UNPACK_WARPS * 32;
            int it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < P.total_tiles; tile += gridDim.x) {
                for (int kb = 0; kb < P.k_blocks; ++kb, ++it) {
                    const int sp = it % P.ns_p, si = it % P.ns_i;
                    const uint32_t php = (uint32_t)(it / P.ns_p) & 1u, phi = (uint32_t)(it / P.ns_i) & 1u;
                    bool w = mbar_wait(ptx::smem_addr(&bars.p_full[sp]), php, abort_ptr);
                    w = w && mbar_wait(ptx::smem_addr(&bars.i_empty[si]), phi ^ 1u, abort_ptr);
                    if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint8_t* pa = smem_gen + packed_off + (size_t)sp * stage_p;
                    const uint8_t* pb = pa + P.pa_bytes;
                    uint8_t* ia = smem_gen + (size_t)si * stage_i;
                    uint8_t* ib = ia + P.ia_bytes;
                    if (!P.a_direct) {
                        if (P.a_signed) unpack_k_major_c<1>(P.ca, pa, ia, BM, tid_u, NU);
                        else unpack_k_major_c<0>(P.ca, pa, ia, BM, tid_u, NU);
                    }
                    if (!P.b_direct) {
                        if (!P.b_mn_major) {
                            if (P.b_signed) unpack_k_major_c<1>(P.cb, pb, ib, P.bn, tid_u, NU);
                            else unpack_k_major_c<0>(P.cb, pb, ib, P.bn, tid_u, NU);
                        } else {
                            if (P.b_signed) unpack_mn_major_c<1>(P.cb, pb, ib, tid_u, NU);
                            else unpack_mn_major_c<0>(P.cb, pb, ib, tid_u, NU);
                        }
                    }
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::mbar_arrive(ptx::smem_addr(&bars.i_full[si]));
                        ptx::mbar_arrive(ptx::smem_addr(&bars.p_empty[sp]));
                    }
                }
            }
        }
    } else {
        // -------------------------------- epilogue ---------------------------------
        const int q4 = warp & 3;   // TMEM lane quarter (fixed by the warp's index in the CTA)
        const int slice = warp < EPI_WARPS ? warp >> 2 : 2 + ((warp - WARP_UNPACK0) >> 2);   // which share of the tile's columns
        const int ewarp = warp < EPI_WARPS ? warp : warp - (WARP_UNPACK0 - EPI_WARPS);   // 0 .. epi_warps-1
        const int tid_e = ewarp * 32 + lane;
        // small accumulators are shifted back as integers; otherwise 2^-shift rides on the multiplier
        const float down = P.small_acc == 1 ? 1.0f : __int_as_float((127 - P.shift) << 23);
        // Per-column parameters of a tile (multiplier, bias, GELU output factor), column c of the tile.
        auto fetch_params = [&](int tile, int c, float& a, float& b, float& q) {
            int m_tile, n_tile, inner, outer;
            tile_coords(P, tile, m_tile, n_tile, inner, outer);
            const int n = n_tile * P.bn + c;
            a = 0.0f; b = 0.0f; q = 0.0f;
            if (n < P.N) {
                const long long cidx = (long long)inner * P.col_off_inner + n;
                if (KIND == EK_REQUANT) {
                    a = __ldg(P.col_a + cidx);
                } else if (KIND == EK_QKV_NORM && n >= 2 * P.norm_dim) {
                    a = __ldg(P.v_alpha + (n - 2 * P.norm_dim));                       // V segment: folded requantization
                } else {
                    a = P.col_a ? __fmul_rn(P.x_step, __ldg(P.col_a + cidx)) : P.x_step;
                    if (KIND == EK_REQUANT_GELU) {                                  // folds GELU's 1/2 (and 1/Qp)
                        q = 0.5f * __ldg(P.inv_s + cidx);
                        if (P.unit_out) q = __fdiv_rn(q, P.out_qp);
                    }
                }
                if (KIND == EK_QKV_NORM && n >= 2 * P.norm_dim) b = P.v_beta ? __ldg(P.v_beta + (n - 2 * P.norm_dim)) : 0.0f;
                else b = P.col_b ? __ldg(P.col_b + cidx) : 0.0f;
                a *= down;
            }
        };
        // The parameters of tile i+1 are fetched while the warps wait for tile i's accumulators and are
        // stored to the other half of epi_params before tile i is processed, so no tile waits for them.
        const bool my_col = KIND != EK_ACC && tid_e < P.bn;          // bn <= 256 <= epilogue threads
        if (my_col && (int)blockIdx.x < P.total_tiles) {
            float a, b, q;
            fetch_params(blockIdx.x, tid_e, a, b, q);
            epi_params.a[0][tid_e] = a;
            epi_params.b[0][tid_e] = b;
            epi_params.q[0][tid_e] = q;
        }
        if constexpr (KIND == EK_QKV_NORM) {
            // comparator references and gain signs of the Q and K norms: read by every epilogue warp after the first tile's
            // group barrier
            const int nt = (1 << P.norm_bits) - 1;
            for (int i = tid_e; i < 2 * 64 * 16; i += P.epi_warps * 32) {
                const int set = i >> 10, c = (i >> 4) & 63, t = i & 15;
                norm_refs_s[i] = t < nt ? __ldg(P.norm_refs + ((size_t)set * 64 + c) * nt + t) : INFINITY;
            }
            for (int i = tid_e; i < 2 * 64; i += P.epi_warps * 32)
                norm_sgn_s[i] = (P.norm_flip != nullptr && __ldg(P.norm_flip + i)) ? -1.0f : 1.0f;
        }
        int tl = 0;
        bool ok = true;
        VT_TRACER(tr, (lane == 0 && ewarp == 0) ? 2 : ((lane == 0 && ewarp == P.epi_warps - 1) ? 3 : -1));
        VT_STAMP(tr, TT_START);
        for (int tile = blockIdx.x; ok && tile < P.total_tiles; tile += gridDim.x, ++tl) {
            int m_tile, n_tile, inner, outer;
            tile_coords(P, tile, m_tile, n_tile, inner, outer);
            const int buf = tl & 1;
            const long long colbase = (long long)inner * P.col_off_inner;
            const int next_tile = tile + (int)gridDim.x;
            const bool fetch_next = my_col && next_tile < P.total_tiles;
            float na = 0.0f, nb = 0.0f, nq = 0.0f;
            if (fetch_next) fetch_params(next_tile, tid_e, na, nb, nq);
            const int row0_in_problem = m_tile * BM + q4 * 32;
            int rows_valid = P.M - row0_in_problem;
            rows_valid = rows_valid < 0 ? 0 : (rows_valid > 32 ? 32 : rows_valid);
            const long long orow0 = (long long)outer * P.row_off_outer + (long long)inner * P.row_off_inner + row0_in_problem;
            float* const stage = P.stage_off ? reinterpret_cast<float*>(smem_gen + P.stage_off + (size_t)ewarp * STAGE_BYTES) : nullptr;
            const bool first_prefetched = epilogue_prefetch_first<KIND>(P, colbase, n_tile, slice, stage, lane, orow0, rows_valid);
            const uint32_t acc_ph = (uint32_t)(tl >> 1) & 1u;
            VT_STAMP(tr, TT_WAIT_ACC);
            bool w = KIND == EK_ACC || epi_barrier(ptx::smem_addr(&bars.epi_sync), (uint32_t)tl & 1u, abort_ptr);
            VT_STAMP(tr, TT_WAIT_FULL);
            w = w && mbar_wait(ptx::smem_addr(&bars.acc_full[buf]), acc_ph, abort_ptr);
            VT_STAMP(tr, TT_GOT_ACC);
            if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
            ptx::tc_fence_after();
            if (fetch_next) {
                // every epilogue warp has arrived at this tile's barrier, so none still reads the other half
                epi_params.a[buf ^ 1][tid_e] = na;
                epi_params.b[buf ^ 1][tid_e] = nb;
                epi_params.q[buf ^ 1][tid_e] = nq;
            }
            const bool row_ok = row0_in_problem + lane < P.M;
            const long long orow = orow0 + lane;
            const uint32_t t_row = tmem_base + (uint32_t)buf * acc_stride + ((uint32_t)(q4 * 32) << 16);
            if (P.small_acc == 2) epilogue_tile<KIND, 2>(P, epi_params, buf, t_row, row_ok, orow, colbase, n_tile, slice, stage, lane, rows_valid, first_prefetched, norm_refs_s, norm_sgn_s);
            else if (P.small_acc == 1) epilogue_tile<KIND, 1>(P, epi_params, buf, t_row, row_ok, orow, colbase, n_tile, slice, stage, lane, rows_valid, first_prefetched, norm_refs_s, norm_sgn_s);
            else epilogue_tile<KIND, 0>(P, epi_params, buf, t_row, row_ok, orow, colbase, n_tile, slice, stage, lane, rows_valid, first_prefetched, norm_refs_s, norm_sgn_s);
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&bars.acc_empty[buf]));
            VT_STAMP(tr, TT_TILE_DONE);
        }
        VT_STAMP(tr, TT_END);
        ptx::cp_async_wait<0>();   // a residual copy requested before a wait that gave up has landed before the CTA exits
    }

    // ---------------------------------- teardown -----------------------------------
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == WARP_MMA) {
        ptx::tc_fence_after();
        __syncwarp();
        ptx::tmem_dealloc(tmem_base, P.tmem_cols);
    }
}

// ---------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// 4-D byte tensor (inner bytes, rows, inner problems, outer problems); out-of-range reads give zero.
int make_map(CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t d3, uint64_t s1,
             uint64_t s2, uint64_t s3, uint32_t box0, uint32_t box1, bool swizzle128) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return VITINT_ERR_CUDA;
    cuuint64_t dims[4] = {d0, d1, d2, d3};
    cuuint64_t strides[3] = {s1, s2, s3};
    cuuint32_t box[4] = {box0, box1, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? VITINT_OK : VITINT_ERR_CUDA;
}

struct Operand {
    const void* data;
    int bits, is_signed;   // value range of the codes
    int container;         // bits per stored code
    uint64_t row_bytes;   // valid bytes of one row (inner extent of the tensor map)
    uint64_t rows;        // rows per problem
    uint64_t pitch, inner_stride, outer_stride;
};

// Per-device caches (a process may use several GPUs): SM count, and which kernels already carry their
// shared-memory opt-in on that device.
constexpr int MAX_DEVICES = 64;
int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return -1;
    return dev;
}
int sm_count() {
    static int n[MAX_DEVICES] = {};
    const int dev = current_device();
    if (dev < 0) return 1;
    if (!n[dev]) {
        int v = 0;
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        n[dev] = v > 0 ? v : 1;
    }
    return n[dev];
}

constexpr uint32_t SMEM_TILE_BUDGET = 204u * 1024u;   // dynamic shared memory spent on operand rings

}  // namespace

// Batched NT integer GEMM launcher shared by the linear layer, Q K^T and P V.
int launch_gemm(const Operand& A, const Operand& B, int M, int N, int K, int n_inner, int n_outer, int b_mn_major,
                GemmParams P, cudaStream_t st) {
    const int ca = A.container, cb = B.container;
    P.M = M; P.N = N; P.K = K;
    P.ca = ca; P.cb = cb; P.a_signed = A.is_signed; P.b_signed = B.is_signed; P.b_mn_major = b_mn_major;
    P.a_direct = ca == 8 ? 1 : 0;
    P.b_direct = (cb == 8 && !b_mn_major) ? 1 : 0;
    P.shift = (A.is_signed ? 8 - ca : 0) + (B.is_signed ? 8 - cb : 0);
    // exact int32 contraction, also after the power-of-two operand scaling
    const long long bound = (long long)K * max_abs_code(A.bits, A.is_signed) * max_abs_code(B.bits, B.is_signed);
    if (bound >= (1ll << 31)) return VITINT_ERR_OVERFLOW_BOUND;
    if ((bound << P.shift) >= (1ll << 31)) return VITINT_ERR_UNSUPPORTED;
    P.small_acc = (bound << P.shift) < (1ll << 22) ? 2 : (bound < (1ll << 22) ? 1 : 0);
    int bn = N >= MAX_BN ? MAX_BN : ((N + 15) / 16) * 16;
    // (Twelve epilogue warps are three per lane quarter, so a 256-column tile is shared 96 / 96 / 64 and waits for the
    // 96; 192-column tiles would share evenly but their MMAs stream a sixth more bytes per output and come close to
    // the issuing thread's rate: fc1 89 -> 101 us, measured.)
    if (b_mn_major) { if (N != 64) return VITINT_ERR_UNSUPPORTED; bn = 64; }
    P.bn = bn;
    P.m_tiles = (M + BM - 1) / BM;
    P.n_tiles = (N + bn - 1) / bn;
    P.n_inner = n_inner;
    const long long tiles = (long long)P.m_tiles * P.n_tiles * n_inner * n_outer;
    if (tiles <= 0 || tiles > 0x7fffffffll) return VITINT_ERR_UNSUPPORTED;
    P.total_tiles = (int)tiles;
    P.k_blocks = (K + BK - 1) / BK;
    P.ia_bytes = BM * BK;
    P.ib_bytes = b_mn_major ? BK * 64 : (uint32_t)bn * BK;
    P.pa_bytes = P.a_direct ? 0u : (uint32_t)(BM * 16 * ca);
    P.pb_bytes = P.b_direct ? 0u : (b_mn_major ? (uint32_t)(BK * 8 * cb) : (uint32_t)bn * 16 * cb);
    const uint32_t stage_i = P.ia_bytes + P.ib_bytes, stage_p = P.pa_bytes + P.pb_bytes;
    // fp32 epilogues go through a per-warp transposition buffer when every access can be a 16-byte one
    bool staged = (P.kind == EK_DEQUANT || P.kind == EK_DEQUANT_GELU) && n_inner == 1 && n_outer == 1 &&
                  aligned16(P.out) && P.ld_out % 4 == 0 &&
                  (!P.residual || (aligned16(P.residual) && P.ld_res % 4 == 0));
    // the fp32 kinds keep 8 epilogue warps: their two staging blocks per warp come out of the ring space
    // ... unless the contraction is short (K <= 1024): such a GEMM is bound by its fp32 epilogue, which gains more
    // from twelve warps than the mainloop loses with two ring stages (proj, batch 128: 45 -> 43 us; with the
    // long contraction of fc2 the same choice costs 17 us)
    // (An fp32 epilogue without staging -- every thread moving its row's columns as 32-byte sectors, four ring stages and
    // twelve warps in return -- was measured as well: proj 43 -> 64 us, fc2 67 -> 78 us.  A warp's access to 32 different
    // rows is served one row at a time, whatever its width.)
    // (Sixteen epilogue warps -- four per lane quarter, equal 64-column shares of a tile -- were measured too: the
    // 576-thread CTA is held to 96 registers a thread, and qkv / fc1 stayed at 57 / 90 us while the fp32 kinds spilled
    // and lost 10 - 14 us.)
    P.epi_warps = (P.a_direct && P.b_direct && (!staged || K <= 1024)) ? MAX_EPI_WARPS : EPI_WARPS;
    if (P.kind == EK_QKV_NORM) P.epi_warps = EPI_WARPS;        // two warps per lane quarter, each taking whole 64-channel heads
    const uint32_t stage_total = staged ? (uint32_t)(P.epi_warps * STAGE_BYTES) : 0u;
    // staging comes out of the ring space; the norm kind keeps 9 KB of reference tables in static shared memory
    const uint32_t ring_budget = SMEM_TILE_BUDGET + 12u * 1024u - stage_total - (P.kind == EK_QKV_NORM ? 16u * 1024u : 0u);
    // The packed ring hides the global-memory latency of the TMA loads; the int8 ring only
    // decouples unpack from MMA issue, unless TMA writes it directly.
    int ns_i, ns_p;
    if (stage_p == 0) {
        ns_i = (int)(ring_budget / stage_i);
        ns_p = 1;
    } else {
        ns_i = (P.a_direct || P.b_direct) ? 3 : 2;
        while (ns_i > 2 && (uint32_t)ns_i * stage_i + 2u * stage_p > ring_budget) --ns_i;
        if ((uint32_t)ns_i * stage_i + 2u * stage_p > ring_budget) return VITINT_ERR_UNSUPPORTED;
        ns_p = (int)((ring_budget - (uint32_t)ns_i * stage_i) / stage_p);
    }
    if (ns_i > MAX_STAGES) ns_i = MAX_STAGES;
    if (ns_p > MAX_STAGES) ns_p = MAX_STAGES;
    if (ns_i < 2) return VITINT_ERR_UNSUPPORTED;
    P.ns_i = ns_i; P.ns_p = ns_p;
    uint32_t cols = 32;
    while (cols < 2u * (uint32_t)((bn + 31) / 32 * 32)) cols <<= 1;
    P.tmem_cols = cols;

    CUtensorMap map_a, map_b;
    if (int rc = make_map(&map_a, A.data, A.row_bytes, A.rows, (uint64_t)n_inner, (uint64_t)n_outer, A.pitch,
                          A.inner_stride, A.outer_stride, P.a_direct ? (uint32_t)BK : 16u * ca, BM, P.a_direct != 0))
        return rc;
    if (b_mn_major) {
        if (int rc = make_map(&map_b, B.data, B.row_bytes, B.rows, (uint64_t)n_inner, (uint64_t)n_outer, B.pitch,
                              B.inner_stride, B.outer_stride, 8u * cb, BK, false))
            return rc;
    } else {
        if (int rc = make_map(&map_b, B.data, B.row_bytes, B.rows, (uint64_t)n_inner, (uint64_t)n_outer, B.pitch,
                              B.inner_stride, B.outer_stride, P.b_direct ? (uint32_t)BK : 16u * cb, (uint32_t)bn,
                              P.b_direct != 0))
            return rc;
    }
    // at least ~120 KB so that two CTAs never share an SM (and its tensor memory)
    const size_t rings = (size_t)ns_i * stage_i + (size_t)ns_p * stage_p;
    P.stage_off = staged ? (uint32_t)rings : 0u;
    size_t smem = rings + stage_total + 1024;
    if (smem < 120 * 1024) smem = 120 * 1024;
    int grid = sm_count();
    if (grid > P.total_tiles) grid = P.total_tiles;
#ifdef VITINT_TRACE
    if (g_trace_max_ctas > 0 && grid > g_trace_max_ctas) grid = g_trace_max_ctas;
#endif
    const int dev = current_device();
    if (dev < 0) return VITINT_ERR_CUDA;
    static bool attr_set_dev[MAX_DEVICES][NUM_KINDS] = {};
    bool* const attr_set = attr_set_dev[dev];
#define VITINT_LAUNCH(KIND)                                                                                        \
    case KIND:                                                                                                     \
        if (!attr_set[KIND]) {                                                                                     \
            if (cudaFuncSetAttribute(gemm_i8_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,            \
                                     (int)SMEM_TILE_BUDGET + (KIND == EK_QKV_NORM ? 0 : 14 * 1024)) != cudaSuccess)      \
                return VITINT_ERR_CUDA;                                                                            \
            attr_set[KIND] = true;                                                                                 \
        }                                                                                                          \
        launch_kernel(gemm_i8_kernel<KIND>, dim3(grid), dim3(NUM_THREADS), smem, st, map_a, map_b, P);            \
        break;
    switch (P.kind) {
        VITINT_LAUNCH(EK_ACC)
        VITINT_LAUNCH(EK_DEQUANT)
        VITINT_LAUNCH(EK_DEQUANT_GELU)
        VITINT_LAUNCH(EK_REQUANT)
        VITINT_LAUNCH(EK_REQUANT_GELU)
        VITINT_LAUNCH(EK_QKV_NORM)
        default: return VITINT_ERR_INVALID_ARG;
    }
#undef VITINT_LAUNCH
    return cuda_status(cudaGetLastError());
}

static int fill_epilogue(GemmParams& P, const vitint_epilogue* epi, float x_step, const float* w_step,
                         const float* bias, void* out, int64_t ld_out, int64_t n_cols_total) {
    if (!epi || !out) return VITINT_ERR_INVALID_ARG;
    P.out = out; P.ld_out = ld_out;
    P.x_step = x_step; P.col_a = nullptr; P.col_b = nullptr; P.inv_s = nullptr; P.residual = nullptr; P.ld_res = 0;
    P.out_c = 4; P.out_qn = 0; P.out_qp = 0;
    if (epi->act != 0 && epi->act != 1) return VITINT_ERR_INVALID_ARG;
    switch (epi->mode) {
        case VITINT_EPI_ACC_I32:
            if (epi->act) return VITINT_ERR_INVALID_ARG;
            if (ld_out < n_cols_total || (reinterpret_cast<uintptr_t>(out) & 3u)) return VITINT_ERR_INVALID_ARG;
            P.kind = EK_ACC;
            break;
        case VITINT_EPI_DEQUANT_F32:
            if (ld_out < n_cols_total || (reinterpret_cast<uintptr_t>(out) & 3u)) return VITINT_ERR_INVALID_ARG;
            if (!(x_step > 0.0f && x_step < INFINITY)) return VITINT_ERR_INVALID_ARG;
            P.col_a = w_step; P.col_b = bias; P.residual = epi->residual; P.ld_res = epi->ld_res;
            if (epi->residual && epi->ld_res < n_cols_total) return VITINT_ERR_INVALID_ARG;
            P.kind = epi->act ? EK_DEQUANT_GELU : EK_DEQUANT;
            break;
        case VITINT_EPI_REQUANT: {
            if (!valid_bits(epi->out_bits)) return VITINT_ERR_INVALID_ARG;
            if (!aligned16(out) || ld_out % 16 != 0) return VITINT_ERR_ALIGNMENT;
            if (ld_out < row_bytes(n_cols_total, epi->out_bits)) return VITINT_ERR_INVALID_ARG;
            int qn, qp;
            code_range(epi->out_bits, epi->out_signed, &qn, &qp);
            if (epi->out_container_bits != 0 && epi->out_container_bits != 8 &&
                epi->out_container_bits != container_bits(epi->out_bits))
                return VITINT_ERR_INVALID_ARG;
            P.out_c = epi->out_container_bits ? epi->out_container_bits : container_bits(epi->out_bits);
            if (ld_out < (n_cols_total * P.out_c + 7) / 8) return VITINT_ERR_INVALID_ARG;
            P.out_qn = (float)qn; P.out_qp = (float)qp;
            if (epi->act == 0) {
                if (!epi->alpha) return VITINT_ERR_INVALID_ARG;
                P.col_a = epi->alpha; P.col_b = epi->beta;
                P.kind = EK_REQUANT;
            } else {
                if (!epi->inv_out_step || !(x_step > 0.0f && x_step < INFINITY)) return VITINT_ERR_INVALID_ARG;
                P.col_a = w_step; P.col_b = bias; P.inv_s = epi->inv_out_step;
                P.kind = EK_REQUANT_GELU;
                P.unit_out = qn == 0 ? 1 : 0;
            }
            break;
        }
        default:
            return VITINT_ERR_INVALID_ARG;
    }
    return VITINT_OK;
}

static int check_slabs(const vitint_slabs* s) {
    if (!s || !s->data) return VITINT_ERR_INVALID_ARG;
    if (!valid_bits(s->bits)) return VITINT_ERR_INVALID_ARG;
    if (!aligned16(s->data) || s->pitch_bytes % 16 || s->image_stride_bytes % 16 || s->head_stride_bytes % 16)
        return VITINT_ERR_ALIGNMENT;
    if (s->pitch_bytes < row_bytes(64, s->bits) || s->image_stride_bytes <= 0 || s->head_stride_bytes <= 0)
        return VITINT_ERR_INVALID_ARG;
    return VITINT_OK;
}

}  // namespace vitint

using namespace vitint;

#ifdef VITINT_TRACE
// Diagnostic builds only: buffer of vitint_trace_words() 64-bit words of device memory, or NULL to stop recording.
extern "C" int vitint_trace_set(long long* buf) {
    return cuda_status(cudaMemcpyToSymbol(g_trace_buf, &buf, sizeof(buf)));
}
extern "C" int vitint_trace_words(void) { return TRACE_CTAS * TRACE_ROLES * TRACE_SLOTS; }
// Diagnostic builds only: cap the persistent grid of the GEMM at n CTAs (0 = one per SM).  Every tile is still computed.
extern "C" int vitint_trace_max_ctas(int n) { g_trace_max_ctas = n; return VITINT_OK; }
#endif

extern "C" int vitint_linear(const vitint_codes* x, float x_step, const vitint_codes* w, const float* w_step,
                             const float* bias, const vitint_epilogue* epi, void* out, int64_t ld_out, void* stream) {
    if (int rc = check_codes(x)) return rc;
    if (int rc = check_codes(w)) return rc;
    if (x->cols != w->cols) return VITINT_ERR_INVALID_ARG;
    if (x->rows > 0x7fffffff || w->rows > 0x7fffffff || x->cols > 0x7fffffff) return VITINT_ERR_UNSUPPORTED;
    GemmParams P{};
    if (int rc = fill_epilogue(P, epi, x_step, w_step, bias, out, ld_out, w->rows)) return rc;
    if ((epi->mode == VITINT_EPI_DEQUANT_F32 || (epi->mode == VITINT_EPI_REQUANT && epi->act == 1)) && !w_step)
        return VITINT_ERR_INVALID_ARG;
    P.row_off_outer = 0; P.row_off_inner = 0; P.col_off_inner = 0;
    Operand A{x->data, x->bits, x->is_signed, codes_container(x), (uint64_t)codes_row_bytes(x, x->cols), (uint64_t)x->rows,
              (uint64_t)x->pitch_bytes, (uint64_t)x->pitch_bytes * (uint64_t)x->rows,
              (uint64_t)x->pitch_bytes * (uint64_t)x->rows};
    Operand B{w->data, w->bits, w->is_signed, codes_container(w), (uint64_t)codes_row_bytes(w, w->cols), (uint64_t)w->rows,
              (uint64_t)w->pitch_bytes, (uint64_t)w->pitch_bytes * (uint64_t)w->rows,
              (uint64_t)w->pitch_bytes * (uint64_t)w->rows};
    return launch_gemm(A, B, (int)x->rows, (int)w->rows, (int)x->cols, 1, 1, 0, P, (cudaStream_t)stream);
}

extern "C" int vitint_linear_qkv_norm(const vitint_codes* x, float x_step, const vitint_codes* w_qkv, const float* w_step,
                                      const float* bias, const float* refs, const uint8_t* flip, float n_eps,
                                      const float* alpha_v, const float* beta_v, const vitint_codes* out, float* stats,
                                      void* stream) {
    if (int rc = check_codes(x)) return rc;
    if (int rc = check_codes(w_qkv)) return rc;
    if (int rc = check_codes(out)) return rc;
    if (!w_step || !refs || !alpha_v) return VITINT_ERR_INVALID_ARG;
    if (x->cols != w_qkv->cols || w_qkv->rows % 192 != 0 || w_qkv->rows <= 0) return VITINT_ERR_INVALID_ARG;
    if (out->rows != x->rows || out->cols != w_qkv->rows || !out->is_signed) return VITINT_ERR_INVALID_ARG;
    if (!(x_step > 0.0f && x_step < INFINITY) || !(n_eps >= 0.0f && n_eps < INFINITY)) return VITINT_ERR_INVALID_ARG;
    if (out->bits > 4) return VITINT_ERR_UNSUPPORTED;               // the reference table holds at most 15 thresholds a channel
    if (x->rows > 0x7fffffff || w_qkv->rows > 0x7fffffff || x->cols > 0x7fffffff) return VITINT_ERR_UNSUPPORTED;
    GemmParams P{};
    int qn, qp;
    code_range(out->bits, 1, &qn, &qp);
    P.kind = EK_QKV_NORM;
    P.out = out->data; P.ld_out = out->pitch_bytes; P.out_c = codes_container(out);
    P.out_qn = (float)qn; P.out_qp = (float)qp;
    P.x_step = x_step; P.col_a = w_step; P.col_b = bias; P.inv_s = nullptr; P.residual = nullptr; P.ld_res = 0;
    P.norm_refs = refs; P.norm_flip = flip; P.n_eps = n_eps; P.norm_bits = out->bits; P.norm_qn = qn;
    P.norm_dim = (int)(w_qkv->rows / 3); P.norm_stats = stats; P.v_alpha = alpha_v; P.v_beta = beta_v;
    P.row_off_outer = 0; P.row_off_inner = 0; P.col_off_inner = 0;
    Operand A{x->data, x->bits, x->is_signed, codes_container(x), (uint64_t)codes_row_bytes(x, x->cols), (uint64_t)x->rows,
              (uint64_t)x->pitch_bytes, (uint64_t)x->pitch_bytes * (uint64_t)x->rows,
              (uint64_t)x->pitch_bytes * (uint64_t)x->rows};
    Operand B{w_qkv->data, w_qkv->bits, w_qkv->is_signed, codes_container(w_qkv), (uint64_t)codes_row_bytes(w_qkv, w_qkv->cols),
              (uint64_t)w_qkv->rows, (uint64_t)w_qkv->pitch_bytes, (uint64_t)w_qkv->pitch_bytes * (uint64_t)w_qkv->rows,
              (uint64_t)w_qkv->pitch_bytes * (uint64_t)w_qkv->rows};
    return launch_gemm(A, B, (int)x->rows, (int)w_qkv->rows, (int)x->cols, 1, 1, 0, P, (cudaStream_t)stream);
}

extern "C" int vitint_qk(const vitint_slabs* q, const vitint_slabs* k, int32_t batch, int32_t heads, int32_t tokens,
                         int32_t* s_out, int64_t ld_s, void* stream) {
    if (int rc = check_slabs(q)) return rc;
    if (int rc = check_slabs(k)) return rc;
    if (batch <= 0 || heads <= 0 || tokens <= 0 || !s_out || ld_s < tokens) return VITINT_ERR_INVALID_ARG;
    GemmParams P{};
    vitint_epilogue epi{};
    epi.mode = VITINT_EPI_ACC_I32;
    if (int rc = fill_epilogue(P, &epi, 1.0f, nullptr, nullptr, s_out, ld_s, tokens)) return rc;
    P.row_off_outer = (long long)heads * tokens; P.row_off_inner = tokens; P.col_off_inner = 0;
    Operand A{q->data, q->bits, q->is_signed, container_bits(q->bits), (uint64_t)row_bytes(64, q->bits), (uint64_t)tokens,
              (uint64_t)q->pitch_bytes, (uint64_t)q->head_stride_bytes, (uint64_t)q->image_stride_bytes};
    Operand B{k->data, k->bits, k->is_signed, container_bits(k->bits), (uint64_t)row_bytes(64, k->bits), (uint64_t)tokens,
              (uint64_t)k->pitch_bytes, (uint64_t)k->head_stride_bytes, (uint64_t)k->image_stride_bytes};
    return launch_gemm(A, B, tokens, tokens, 64, heads, batch, 0, P, (cudaStream_t)stream);
}

extern "C" int vitint_pv(const vitint_codes* p, const vitint_slabs* v, int32_t batch, int32_t heads, int32_t tokens,
                         float p_step, float v_step, const vitint_epilogue* epi, void* out, int64_t ld_out,
                         void* stream) {
    if (int rc = check_codes(p)) return rc;
    if (int rc = check_slabs(v)) return rc;
    if (batch <= 0 || heads <= 0 || tokens <= 0) return VITINT_ERR_INVALID_ARG;
    if (p->rows != (int64_t)batch * heads * tokens || p->cols != tokens) return VITINT_ERR_INVALID_ARG;
    if (!(p_step > 0.0f && p_step < INFINITY) || !(v_step > 0.0f && v_step < INFINITY)) return VITINT_ERR_INVALID_ARG;
    GemmParams P{};
    // the scale product s_P * s_V takes the place of s_x * s_w[n]
    if (int rc = fill_epilogue(P, epi, p_step * v_step, nullptr, nullptr, out, ld_out,
                               (int64_t)heads * 64))
        return rc;
    if (epi->mode == VITINT_EPI_REQUANT && epi->act == 1) return VITINT_ERR_UNSUPPORTED;
    P.row_off_outer = tokens; P.row_off_inner = 0; P.col_off_inner = 64;
    Operand A{p->data, p->bits, p->is_signed, codes_container(p), (uint64_t)codes_row_bytes(p, tokens), (uint64_t)tokens,
              (uint64_t)p->pitch_bytes, (uint64_t)p->pitch_bytes * tokens, (uint64_t)p->pitch_bytes * tokens * heads};
    Operand B{v->data, v->bits, v->is_signed, container_bits(v->bits), (uint64_t)row_bytes(64, v->bits), (uint64_t)tokens,
              (uint64_t)v->pitch_bytes, (uint64_t)v->head_stride_bytes, (uint64_t)v->image_stride_bytes};
    return launch_gemm(A, B, tokens, 64, tokens, heads, batch, 1, P, (cudaStream_t)stream);
}
