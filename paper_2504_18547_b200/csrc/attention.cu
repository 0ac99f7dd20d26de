// a7: integerized self-attention block (Fig. 1(b)) as a sequence of the library's own
// kernels on one stream: QKV linear (requantizing epilogue) -> Q K^T -> scale + softmax +
// quantize -> P V (requantizing epilogue) -> output projection.  Intermediates live in
// caller-provided scratch memory.
#include <math.h>

#include "common.cuh"

namespace vitint {
namespace {

struct AttnLayout {
    int64_t M, D, n_rows_p;
    int64_t pitch_qkv, pitch_qkv_wide, pitch_p, pitch_o, ld_s;
    size_t off_qkv, off_s, off_p, off_o, off_tab, tab_bytes, total;
};

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

int attn_layout(const vitint_attention_desc* d, AttnLayout* L) {
    if (!d || d->batch <= 0 || d->tokens <= 0 || d->heads <= 0) return VITINT_ERR_INVALID_ARG;
    if (!valid_bits(d->bits) || !valid_bits(d->p_bits)) return VITINT_ERR_INVALID_ARG;
    L->M = (int64_t)d->batch * d->tokens;
    L->D = (int64_t)d->heads * 64;
    L->n_rows_p = (int64_t)d->batch * d->heads * d->tokens;
    L->pitch_qkv = vitint_packed_pitch(3 * L->D, d->bits);
    L->pitch_o = vitint_packed_pitch(L->D, d->bits);
    L->pitch_p = vitint_packed_pitch(d->tokens, d->p_bits);
    L->ld_s = ((int64_t)d->tokens + 3) / 4 * 4;
    size_t off = 0;
    // beyond 256 tokens the fused core takes QKV stored one code per byte: room for that form
    L->pitch_qkv_wide = vitint_packed_pitch(3 * L->D, 8);
    const int64_t pq = d->tokens > 256 ? L->pitch_qkv_wide : L->pitch_qkv;
    L->off_qkv = off; off = align256(off + (size_t)(L->M * pq));
    L->off_s = off;   off = align256(off + (size_t)(L->n_rows_p * L->ld_s) * 4);
    L->off_p = off;   off = align256(off + (size_t)(L->n_rows_p * L->pitch_p));
    L->off_o = off;   off = align256(off + (size_t)(L->M * L->pitch_o));
    L->tab_bytes = vitint_attention_core_workspace_bytes(d->bits);
    L->off_tab = off; off = align256(off + L->tab_bytes);
    L->total = off;
    return VITINT_OK;
}

int copy_codes(const vitint_codes* dst, const void* src, int64_t src_pitch, int64_t rows, int64_t row_bytes_valid,
               cudaStream_t st) {
    if (!dst) return VITINT_OK;
    if (int rc = check_codes(dst)) return rc;
    if (dst->rows != rows || dst->pitch_bytes < row_bytes_valid) return VITINT_ERR_INVALID_ARG;
    const int64_t w = dst->pitch_bytes < src_pitch ? dst->pitch_bytes : src_pitch;
    if (int rc = cuda_status(cudaMemcpy2DAsync(dst->data, (size_t)dst->pitch_bytes, src, (size_t)src_pitch, (size_t)w,
                                               (size_t)rows, cudaMemcpyDeviceToDevice, st)))
        return rc;
    // a destination pitch beyond the source's: the rest of every row is padding and is written as zero
    if (dst->pitch_bytes > w)
        return cuda_status(cudaMemset2DAsync((uint8_t*)dst->data + w, (size_t)dst->pitch_bytes, 0,
                                             (size_t)(dst->pitch_bytes - w), (size_t)rows, st));
    return VITINT_OK;
}

}  // namespace
}  // namespace vitint

using namespace vitint;

extern "C" size_t vitint_attention_block_workspace_bytes(const vitint_attention_desc* d) {
    AttnLayout L;
    if (attn_layout(d, &L) != VITINT_OK) return 0;
    return L.total;
}

extern "C" int vitint_attention_block(const vitint_codes* x, const vitint_attention_desc* d, void* out,
                                      int64_t ld_out, const vitint_codes* dbg_qkv, const vitint_codes* dbg_p,
                                      const vitint_codes* dbg_o, void* workspace, size_t workspace_bytes,
                                      void* stream) {
    AttnLayout L;
    if (int rc = attn_layout(d, &L)) return rc;
    if (int rc = check_codes(x)) return rc;
    if (x->rows != L.M || x->cols != L.D) return VITINT_ERR_INVALID_ARG;
    if (d->w_qkv.rows != 3 * L.D || d->w_qkv.cols != L.D || d->w_proj.rows != L.D || d->w_proj.cols != L.D)
        return VITINT_ERR_INVALID_ARG;
    if (!d->alpha_qkv || !d->alpha_o || !out) return VITINT_ERR_INVALID_ARG;
    const float steps[5] = {d->q_step, d->k_step, d->v_step, d->p_step, d->o_step};
    for (float s : steps) if (!(s > 0.0f && s < INFINITY)) return VITINT_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < L.total)
        return VITINT_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* ws = (uint8_t*)workspace;
    const int cbits = container_bits(d->bits);

    // 1. QKV linear, requantized per output channel (three per-tensor steps).  Beyond 256 tokens, when no copy of QKV
    // or P is asked for and the logits' range allows the table-driven core, the codes are stored one per byte: the form
    // the chunked two-pass core takes (S and P then never reach HBM).
    const int mq = 1 << (d->bits - 1);
    const bool wide_qkv = d->tokens > 256 && d->tokens <= 4096 && !dbg_qkv && !dbg_p && L.tab_bytes && d->bits != 8 &&
                          64.0 * mq * mq * (double)(float)((double)d->q_step * (double)d->k_step / 8.0) <= 80.0;
    vitint_codes qkv{ws + L.off_qkv, L.M, 3 * L.D, wide_qkv ? L.pitch_qkv_wide : L.pitch_qkv, d->bits, 1, wide_qkv ? 8 : 0, 0};
    vitint_epilogue e1{};
    e1.mode = VITINT_EPI_REQUANT; e1.alpha = d->alpha_qkv; e1.beta = d->beta_qkv;
    e1.out_bits = d->bits; e1.out_signed = 1; e1.out_container_bits = wide_qkv ? 8 : 0;
    if (int rc = vitint_linear(x, 1.0f, &d->w_qkv, nullptr, nullptr, &e1, qkv.data, qkv.pitch_bytes, stream)) return rc;
    if (int rc = copy_codes(dbg_qkv, qkv.data, L.pitch_qkv, L.M, row_bytes(3 * L.D, d->bits), st)) return rc;

    vitint_codes o{ws + L.off_o, L.M, L.D, L.pitch_o, d->bits, 1, 0, 0};
    // 2-4 fused when the shape allows and no copy of P is wanted
    int fused = VITINT_ERR_UNSUPPORTED;
    if (!dbg_p && L.tab_bytes)
        fused = vitint_attention_core(&qkv, d->batch, d->heads, d->tokens, d->q_step, d->k_step, d->p_step, d->p_bits,
                                      d->alpha_o, d->beta_o, &o, ws + L.off_tab, L.tab_bytes, stream);
    if (fused != VITINT_OK && fused != VITINT_ERR_UNSUPPORTED) return fused;
    if (fused == VITINT_ERR_UNSUPPORTED && wide_qkv) return fused;      // (the unfused kernels read bit-packed slabs)
    if (fused == VITINT_ERR_UNSUPPORTED) {
        // 2. S = Q K^T per (image, head)
        const int64_t head_bytes = 64 * cbits / 8, seg_bytes = L.D * cbits / 8;
        vitint_slabs q{ws + L.off_qkv, L.pitch_qkv, L.pitch_qkv * d->tokens, head_bytes, d->bits, 1};
        vitint_slabs k = q, v = q;
        k.data = ws + L.off_qkv + seg_bytes;
        v.data = ws + L.off_qkv + 2 * seg_bytes;
        int32_t* S = (int32_t*)(ws + L.off_s);
        if (int rc = vitint_qk(&q, &k, d->batch, d->heads, d->tokens, S, L.ld_s, stream)) return rc;

        // 3. P = quantize(softmax(c * S)),  c = s_q s_k / sqrt(64)
        const float c = (float)((double)d->q_step * (double)d->k_step / 8.0);
        vitint_codes p{ws + L.off_p, L.n_rows_p, d->tokens, L.pitch_p, d->p_bits, 0, 0, 0};
        // the scores of b-bit codes are bounded by 64 * 2^(b-1) * 2^(b-1) (container width: any bit pattern stays
        // inside), so the exp table serves whenever one of that size exists and the range allows it
        const int half = 1 << (cbits - 1);
        const int32_t bound = 64 * half * half;
        int sm = VITINT_ERR_UNSUPPORTED;
        if (L.tab_bytes && vitint_softmax_table_workspace_bytes(bound) != 0 &&
            vitint_softmax_table_workspace_bytes(bound) <= L.tab_bytes)
            sm = vitint_softmax_quantize_bounded(S, L.n_rows_p, d->tokens, L.ld_s, c, d->p_step, bound, &p, nullptr, 0,
                                                 ws + L.off_tab, L.tab_bytes, 0, stream);
        if (sm != VITINT_OK && sm != VITINT_ERR_UNSUPPORTED) return sm;
        if (sm == VITINT_ERR_UNSUPPORTED)
            if (int rc = vitint_softmax_quantize(S, L.n_rows_p, d->tokens, L.ld_s, c, d->p_step, &p, nullptr, 0, stream))
                return rc;
        if (int rc = copy_codes(dbg_p, p.data, L.pitch_p, L.n_rows_p, row_bytes(d->tokens, d->p_bits), st)) return rc;

        // 4. O = P V, requantized to the projection's input step
        vitint_epilogue e4{};
        e4.mode = VITINT_EPI_REQUANT; e4.alpha = d->alpha_o; e4.beta = d->beta_o;
        e4.out_bits = d->bits; e4.out_signed = 1;
        if (int rc = vitint_pv(&p, &v, d->batch, d->heads, d->tokens, d->p_step, d->v_step, &e4, o.data, o.pitch_bytes,
                               stream))
            return rc;
    }
    if (int rc = copy_codes(dbg_o, o.data, L.pitch_o, L.M, row_bytes(L.D, d->bits), st)) return rc;

    // 5. output projection
    return vitint_linear(&o, d->o_step, &d->w_proj, d->w_proj_step, d->b_proj, &d->proj_epi, out, ld_out, stream);
}
