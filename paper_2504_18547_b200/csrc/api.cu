// Status strings, version, device status word and descriptor checks.
#include "common.cuh"

namespace vitint {

int cuda_status(cudaError_t e) { return e == cudaSuccess ? VITINT_OK : VITINT_ERR_CUDA; }

int check_codes(const vitint_codes* c) {
    if (!c || !c->data) return VITINT_ERR_INVALID_ARG;
    if (!valid_bits(c->bits) || (c->is_signed != 0 && c->is_signed != 1)) return VITINT_ERR_INVALID_ARG;
    if (c->rows <= 0 || c->cols <= 0) return VITINT_ERR_INVALID_ARG;
    if (!aligned16(c->data) || c->pitch_bytes % 16 != 0) return VITINT_ERR_ALIGNMENT;
    if (c->container_bits != 0 && c->container_bits != 8 && c->container_bits != container_bits(c->bits))
        return VITINT_ERR_INVALID_ARG;
    if (c->pitch_bytes < codes_row_bytes(c, c->cols)) return VITINT_ERR_INVALID_ARG;
    return VITINT_OK;
}

}  // namespace vitint

using namespace vitint;

extern "C" const char* vitint_status_string(int status) {
    switch (status) {
        case VITINT_OK: return "ok";
        case VITINT_ERR_INVALID_ARG: return "invalid argument";
        case VITINT_ERR_UNSUPPORTED: return "unsupported shape or format";
        case VITINT_ERR_ALIGNMENT: return "misaligned pointer or pitch";
        case VITINT_ERR_OVERFLOW_BOUND: return "int32 accumulator bound K*max|q_x|*max|q_w| < 2^31 violated";
        case VITINT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case VITINT_ERR_CUDA: return "CUDA call failed";
        case VITINT_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        default: return "unknown status";
    }
}

extern "C" int vitint_version(void) { return 100; }

extern "C" int64_t vitint_packed_pitch(int64_t cols, int32_t bits) {
    if (cols <= 0 || !valid_bits(bits)) return 0;
    return (row_bytes(cols, bits) + 15) / 16 * 16;
}

extern "C" int vitint_device_status(void) {
    if (cudaDeviceSynchronize() != cudaSuccess) return VITINT_ERR_CUDA;
    int h = 0;
    if (cudaMemcpyFromSymbol(&h, g_device_status, sizeof(int)) != cudaSuccess) return VITINT_ERR_CUDA;
    if (h != 0) {
        int zero = 0;
        cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int));
    }
    return h;
}
