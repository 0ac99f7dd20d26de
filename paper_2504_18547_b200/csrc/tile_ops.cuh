// Device helpers shared by the tensor-core kernels: the bounded mbarrier wait and the
// expansion of packed low-bit codes into int8 operand chunks.
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace vitint {

constexpr long long WAIT_LIMIT_CYCLES = 2000000000ll;   // about one second

// Bounded wait.  Gives up after WAIT_LIMIT_CYCLES or as soon as another thread of the CTA
// has given up; the first to give up records the timeout in the device status word.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          long long limit_cycles = WAIT_LIMIT_CYCLES) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        // sleeps in hardware until the phase completes or ~50 us pass, so a waiting warp leaves the
        // issue slots to the warps that have work
        if (ptx::mbar_try_wait_hint(bar, parity, 50000u)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit_cycles) {
            *abort_flag = 1;
            atomicExch(&g_device_status, (int)VITINT_ERR_TIMEOUT);
            return false;
        }
    }
}

// 8 four-bit codes of one word -> 8 bytes in natural order.
template <int SGN>
__device__ __forceinline__ void unpack4(uint32_t w, uint32_t& o0, uint32_t& o1) {
    uint32_t lo, hi;
    if (SGN) { lo = (w << 4) & 0xF0F0F0F0u; hi = w & 0xF0F0F0F0u; }
    else     { lo = w & 0x0F0F0F0Fu;        hi = (w >> 4) & 0x0F0F0F0Fu; }
    o0 = __byte_perm(lo, hi, 0x5140);
    o1 = __byte_perm(lo, hi, 0x7362);
}
// 16 two-bit codes of one word -> 16 bytes in natural order.
template <int SGN>
__device__ __forceinline__ uint4 unpack2(uint32_t w) {
    uint32_t p0, p1, p2, p3;
    if (SGN) {
        p0 = (w << 6) & 0xC0C0C0C0u; p1 = (w << 4) & 0xC0C0C0C0u; p2 = (w << 2) & 0xC0C0C0C0u; p3 = w & 0xC0C0C0C0u;
    } else {
        p0 = w & 0x03030303u; p1 = (w >> 2) & 0x03030303u; p2 = (w >> 4) & 0x03030303u; p3 = (w >> 6) & 0x03030303u;
    }
    const uint32_t a = __byte_perm(p0, p1, 0x5140), b = __byte_perm(p2, p3, 0x5140);
    const uint32_t c = __byte_perm(p0, p1, 0x7362), d = __byte_perm(p2, p3, 0x7362);
    return make_uint4(__byte_perm(a, b, 0x5410), __byte_perm(a, b, 0x7632), __byte_perm(c, d, 0x5410),
                      __byte_perm(c, d, 0x7632));
}

// One 16-byte chunk of packed codes -> 8/C chunks of int8 written at dst[oc ^ sw], oc = oc0 .. oc0 + 8/C - 1.
// `row` points at the first chunk slot of the destination row; `sw` is the row's swizzle mask.
template <int C, int SGN>
__device__ __forceinline__ void expand_chunk(uint4 in, uint8_t* row, int oc0, int sw) {
    if (C == 4) {
        uint4 o0, o1;
        unpack4<SGN>(in.x, o0.x, o0.y);
        unpack4<SGN>(in.y, o0.z, o0.w);
        unpack4<SGN>(in.z, o1.x, o1.y);
        unpack4<SGN>(in.w, o1.z, o1.w);
        *reinterpret_cast<uint4*>(row + ((oc0 ^ sw) << 4)) = o0;
        *reinterpret_cast<uint4*>(row + (((oc0 + 1) ^ sw) << 4)) = o1;
    } else if (C == 2) {
        *reinterpret_cast<uint4*>(row + ((oc0 ^ sw) << 4)) = unpack2<SGN>(in.x);
        *reinterpret_cast<uint4*>(row + (((oc0 + 1) ^ sw) << 4)) = unpack2<SGN>(in.y);
        *reinterpret_cast<uint4*>(row + (((oc0 + 2) ^ sw) << 4)) = unpack2<SGN>(in.z);
        *reinterpret_cast<uint4*>(row + (((oc0 + 3) ^ sw) << 4)) = unpack2<SGN>(in.w);
    } else {
        *reinterpret_cast<uint4*>(row + ((oc0 ^ sw) << 4)) = in;
    }
}


// Rows of 64 int8 (64 codes each), 64-byte swizzle: row r lives at r*64 and its 16-byte chunk
// cc at slot cc ^ ((r >> 1) & 3).  This one layout serves a K-contiguous operand with K = 64
// (SBO = 512) and an N-contiguous operand with N = 64 (eight K rows per 512-byte group).
template <int C, int SGN>
__device__ __forceinline__ void unpack_rows64(const uint8_t* src, uint8_t* dst, int rows, int tid, int nthreads) {
    constexpr int LH = C == 2 ? 0 : (C == 4 ? 1 : 2);   // log2(packed chunks per 64-code row)
    constexpr int E = 8 / C;
    const int chunks = rows << LH;
#pragma unroll 2
    for (int q = tid; q < chunks; q += nthreads) {
        const int r = q >> LH, h = q & ((1 << LH) - 1);
        const uint4 in = *reinterpret_cast<const uint4*>(src + (size_t)q * 16);
        expand_chunk<C, SGN>(in, dst + r * 64, h * E, (r >> 1) & 3);
    }
}

}  // namespace vitint
