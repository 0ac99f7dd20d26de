// Stand-alone probe (its own executable, not part of libvitint.so): the rate at which one SM's tensor core retires
// tcgen05.mma instructions whose operands are already resident in shared memory - MMAs issued back to back on fixed
// tiles (contents zero), all SMs at once, no TMA traffic.  Kinds: i8 (128x256x32), f8f6f4 e4m3 (128x256x32), f16 bf16
// (128x256x16), mxf4 e2m1 with unit block scales (128x256x64), and i8 with the A operand in tensor memory (N = 256
// and 128; the A columns hold whatever the allocation held, only the rate matters).  Every wait is bounded.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -I include probe_mma_rate.cu -o probe_mma_rate
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>

#include "ptx.cuh"

using namespace vitint;

__device__ int g_gave_up = 0;

template <int KIND>
__global__ void __launch_bounds__(128, 1) probe(int iters, int n_stage, long long* out) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar;
    __shared__ uint32_t slot;
    const uint32_t base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    uint32_t* const tiles = reinterpret_cast<uint32_t*>(smem_raw + (base - ptx::smem_addr(smem_raw)));
    for (int i = threadIdx.x; i < 48 * 1024 * n_stage / 4; i += blockDim.x) tiles[i] = 0u;
    if (threadIdx.x == 0) { ptx::mbar_init(ptx::smem_addr(&bar), 1); ptx::fence_mbar_init(); }
    if (threadIdx.x < 32) { ptx::tmem_alloc(ptx::smem_addr(&slot), 512); ptx::tmem_relinquish(); }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tm = slot;
    if (KIND == 3) {                                  // unit ue8m0 scales (0x7F) behind the accumulator
        uint32_t ones[32];
        for (int i = 0; i < 32; ++i) ones[i] = 0x7F7F7F7Fu;
        ptx::tmem_st32(tm + 256u + ((uint32_t)((threadIdx.x >> 5) * 32) << 16), ones);
        ptx::tmem_st_wait();
        ptx::tc_fence_before();
        __syncthreads();
        ptx::tc_fence_after();
    }
    if (threadIdx.x == 0) {
        uint32_t idesc;
        if (KIND == 0) idesc = ptx::idesc_i8(128, 256, 1, 1, 0);
        else if (KIND == 1) idesc = (1u << 4) | ((256u >> 3) << 17) | (8u << 24);                           // f32 accumulators, e4m3 x e4m3
        else if (KIND == 2) idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | (8u << 24);  // f32 accumulators, bf16 x bf16
        else if (KIND == 3) idesc = (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | (1u << 23) | (8u << 24);  // e2m1 x e2m1, ue8m0 scales
        else idesc = ptx::idesc_i8(128, KIND == 4 ? 256 : 128, 1, 1, 0);                                    // i8, A from tensor memory
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            const uint32_t st = base + (uint32_t)(it % n_stage) * 49152u;
            const uint64_t a = ptx::smem_desc(st, 16, 1024, ptx::SWIZZLE_128B), b = ptx::smem_desc(st + 16384u, 16, 1024, ptx::SWIZZLE_128B);
            const uint32_t d = (KIND == 3 || KIND == 4) ? tm : tm + (uint32_t)((it >> 5) & 1) * (KIND == 5 ? 128u : 256u);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (KIND == 0) ptx::mma_i8(d, a + k * 2, b + k * 2, idesc, 1u);
                else if (KIND == 1) asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d), "l"(a + k * 2), "l"(b + k * 2), "r"(idesc) : "memory");
                else if (KIND == 2) asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d), "l"(a + k * 2), "l"(b + k * 2), "r"(idesc) : "memory");
                else if (KIND >= 4) asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d), "r"(tm + 256u + (uint32_t)(((it & 7) * 4 + k) * 8)), "l"(b + k * 2), "r"(idesc) : "memory");
                else asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 1, 0;\n\ttcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%4], [%5], p;\n\t}" ::"r"(d), "l"(a + k * 2), "l"(b + k * 2), "r"(idesc), "r"(tm + 256u), "r"(tm + 256u) : "memory");
            }
        }
        ptx::mma_commit(ptx::smem_addr(&bar));
        bool done = false;
        const long long w0 = clock64();
        while (!done && clock64() - w0 < 4000000000ll) done = ptx::mbar_try_wait(ptx::smem_addr(&bar), 0);
        if (!done) atomicExch(&g_gave_up, 1);
        out[blockIdx.x] = clock64() - t0;
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) { ptx::tc_fence_after(); ptx::tmem_dealloc(tm, 512); }
}

template <int KIND>
void run(const char* name, int iters, int sms, double mhz) {
    const int n_stage = 4;
    long long* d;
    cudaMalloc(&d, sms * 8);
    cudaMemset(d, 0, sms * 8);
    const size_t smem = 49152 * n_stage + 1024;
    cudaFuncSetAttribute(probe<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    for (int rep = 0; rep < 3; ++rep) {
        cudaEvent_t e0, e1;
        cudaEventCreate(&e0);
        cudaEventCreate(&e1);
        cudaEventRecord(e0);
        probe<KIND><<<sms, 128, smem>>>(iters, n_stage, d);
        cudaEventRecord(e1);
        if (cudaDeviceSynchronize() != cudaSuccess) { printf("%s: CUDA error\n", name); exit(1); }
        float ms = 0;
        cudaEventElapsedTime(&ms, e0, e1);
        long long* h = (long long*)malloc(sms * 8);
        cudaMemcpy(h, d, sms * 8, cudaMemcpyDeviceToHost);
        long long mx = 0;
        for (int i = 0; i < sms; ++i) if (h[i] > mx) mx = h[i];
        free(h);
        const double macs = 128.0 * (KIND == 5 ? 128.0 : 256.0) * (KIND == 2 ? 16 : (KIND == 3 ? 64 : 32));
        const double per_mma = (double)mx / (4.0 * iters);
        printf("%s: %.1f clk per MMA per SM -> %.0f MAC/clk/SM; %.3f ms -> %.0f T(FL)OPS over %d SMs\n", name, per_mma, macs / per_mma, ms,
               2.0 * macs * 4.0 * iters * sms / (ms * 1e-3) / 1e12, sms);
    }
    int gave_up = 0;
    cudaMemcpyFromSymbol(&gave_up, g_gave_up, 4);
    if (gave_up) { printf("a wait ran into its limit\n"); exit(2); }
    cudaFree(d);
}

int main() {
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    run<0>("kind::i8       128x256x32", 20000, sms, 0);
    run<1>("kind::f8f6f4   128x256x32", 20000, sms, 0);
    run<2>("kind::f16 bf16 128x256x16", 20000, sms, 0);
    run<3>("kind::mxf4     128x256x64", 20000, sms, 0);
    run<4>("kind::i8, A in tensor memory 128x256x32", 20000, sms, 0);
    run<5>("kind::i8, A in tensor memory 128x128x32", 20000, sms, 0);
    return 0;
}
