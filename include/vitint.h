/* vitint - integerized ViT matmul path for NVIDIA B200 (sm_100a), C ABI.
 *
 * The library implements the operand-reordered ("integerized") linear layer and
 * attention matmuls of Lin & Shah, "Low-Bit Integerization of Vision
 * Transformers using Operand Reordering for Efficient Hardware": low-bit codes
 * are contracted as integers into int32 accumulators and every step size is
 * applied once, after the contraction (Section III, Eq. 1-3).
 *
 * General rules for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller; the library
 *     allocates no device memory and keeps no reference after the call returns.
 *     Descriptor structs (vitint_codes, vitint_epilogue, ...) are HOST structs.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Work
 *     is enqueued asynchronously on it; results are ready when the stream
 *     reaches that point.
 *   - Return value: VITINT_OK or a negative vitint_status.  Argument errors are
 *     detected on the host before anything is launched.  No exceptions cross
 *     the boundary.
 *   - Kernels never spin without bound: a wait that exceeds its limit makes the
 *     kernel record VITINT_ERR_TIMEOUT in a device status word and return; read
 *     it with vitint_device_status().
 *
 * Packed code format (vitint_codes)
 *   Row-major.  b-bit codes (b = 2, 3, 4, 8) live in containers of c = 2, 4, 4, 8
 *   bits.  Element i of a row occupies bits [c*(i mod 8/c), +c) of byte
 *   i / (8/c) (little-endian inside the byte).  Signed codes are two's
 *   complement sign-extended to the container; signed range
 *   [-2^(b-1), 2^(b-1)-1], unsigned [0, 2^b-1] (the 3-bit comparator ladder
 *   -3.5D ... 2.5D of Section IV-B gives levels -4..3).  `data` and
 *   `pitch_bytes` are multiples of 16; bytes between the last code of a row and
 *   the pitch are ZERO (producers in this library write them as zero, and they
 *   may enter contractions).
 */
#ifndef VITINT_H_
#define VITINT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    VITINT_OK = 0,
    VITINT_ERR_INVALID_ARG = -1,    /* null pointer, non-positive size, bad enum, non-finite or non-positive step */
    VITINT_ERR_UNSUPPORTED = -2,    /* a shape or format this build has no kernel for */
    VITINT_ERR_ALIGNMENT = -3,      /* pointer or pitch not aligned as documented */
    VITINT_ERR_OVERFLOW_BOUND = -4, /* K * max|q_x| * max|q_w| >= 2^31 for the declared formats */
    VITINT_ERR_WORKSPACE = -5,      /* workspace missing, misaligned or too small */
    VITINT_ERR_CUDA = -6,           /* a CUDA runtime / driver call failed */
    VITINT_ERR_TIMEOUT = -7         /* a bounded device-side wait gave up (device status word) */
} vitint_status;

typedef struct {
    void* data;          /* device, 16-byte aligned */
    int64_t rows, cols;  /* logical code counts */
    int64_t pitch_bytes; /* multiple of 16, >= ceil(cols*c/8) */
    int32_t bits;        /* 2, 3, 4 or 8: the value range of the codes */
    int32_t is_signed;   /* 0 / 1 */
    int32_t container_bits; /* 0: the default container of `bits` (2, 4, 4, 8); 8: b-bit codes stored one per
                               byte (what vitint_widen produces).  Other values are invalid. */
    int32_t reserved_;   /* set to 0 */
} vitint_codes;

typedef enum {
    VITINT_EPI_ACC_I32 = 0,     /* raw int32 accumulators */
    VITINT_EPI_DEQUANT_F32 = 1, /* y = fma(float(acc), s_x*s_w[n], b[n]) [GELU] [+ residual] */
    VITINT_EPI_REQUANT = 2      /* codes at the next layer's step */
} vitint_epi_mode;

/* Epilogue applied to the int32 accumulators (Eq. 2: the "equivalent bias" and
 * "post-scaling factor" moved behind the contraction; Section IV-B: operand
 * scales "absorbed within the quantizer").
 *   DEQUANT_F32: sc[n] = fl32(x_step * w_step[n]); y = fmaf((float)acc, sc[n], bias[n] or 0);
 *                act == 1 applies GELU(y) = y*Phi(y) in fp32; then, if residual != NULL,
 *                y += residual[m*ld_res + n] as one more rounded add.  fp32 output.
 *   REQUANT, act == 0: q = clamp(rint(fmaf((float)acc, alpha[n], beta[n]))) with the
 *                folded alpha = s_x s_w / s_out, beta = b / s_out supplied by the caller.
 *   REQUANT, act == 1: y as in DEQUANT, g = GELU(y), q = clamp(rint(g * inv_out_step[n])).
 * Rounding is to nearest, ties to even; the clamp range follows out_bits/out_signed.
 * alpha, beta, inv_out_step: device arrays of N floats. */
typedef struct {
    int32_t mode;               /* vitint_epi_mode */
    int32_t act;                /* 0 none, 1 GELU */
    const float* residual;      /* DEQUANT only, or NULL */
    int64_t ld_res;             /* elements */
    const float* alpha;         /* REQUANT, act 0 */
    const float* beta;          /* REQUANT, act 0 */
    const float* inv_out_step;  /* REQUANT, act 1 */
    int32_t out_bits;           /* REQUANT: 2, 3, 4, 8 */
    int32_t out_signed;
    int32_t out_container_bits; /* REQUANT: 0 = default container of out_bits, 8 = one code per byte */
    int32_t reserved_;          /* set to 0 */
} vitint_epilogue;

const char* vitint_status_string(int status);
int vitint_version(void);

/* Reads (and clears) the device status word of the current device; synchronizes
 * the device.  Returns VITINT_OK, VITINT_ERR_TIMEOUT, VITINT_ERR_INVALID_ARG (a kernel met data that contradicts what
 * its caller declared: vitint_softmax_quantize_bounded) or VITINT_ERR_CUDA. */
int vitint_device_status(void);

/* Self-test of the bounded wait: launches one warp that waits on a barrier nothing ever completes, with a limit of
 * `limit_cycles` SM clock cycles (1 .. 2e9; about a millisecond at 2e6).  When the limit passes the kernel records
 * VITINT_ERR_TIMEOUT in the device status word, writes 1 to *gave_up (device int32, may be NULL) and returns; the
 * context stays usable and the next vitint_device_status() reports (and clears) the timeout.  Asynchronous on
 * `stream`.  Nothing faults, traps or spins without bound. */
int vitint_selftest_wait_timeout(int64_t limit_cycles, int32_t* gave_up, void* stream);

/* Bytes a packed row of `cols` b-bit codes needs, rounded up to 16. */
int64_t vitint_packed_pitch(int64_t cols, int32_t bits);

/* a1. Quantize and pack (Section IV-B comparator quantizer, round-to-nearest-even):
 *   q[m][k] = clamp(rint(x[m*ldx + k] / s_m)), s_m = row_steps[m] if row_steps != NULL
 *   (per-output-channel weight steps, Eq. 1's Delta_W) else `step` (the single input
 *   step of Eq. 2).  One IEEE fp32 division per element; non-finite inputs follow that definition (+-inf and any
 *   quotient beyond the range clamp to the end levels, NaN gives Qn).  The steps in row_steps are the caller's
 *   responsibility: a step that is zero, negative or not finite yields whatever the IEEE quotient rounds and clamps to.
 *   x: device fp32 [rows, ldx] (ldx >= cols, elements).  out: descriptor whose data,
 *   rows (== rows), cols (== cols), pitch_bytes, bits, is_signed are set by the caller;
 *   the whole pitch of every row is written (padding as zero).
 *   Errors: INVALID_ARG (sizes, step <= 0 or not finite when row_steps == NULL, bits),
 *   ALIGNMENT (out->data or pitch not multiples of 16). */
int vitint_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx, float step, const float* row_steps,
                    const vitint_codes* out, void* stream);

/* Re-stores b-bit codes in 8-bit containers (same values, same signedness): out->bits equals
 *   in->bits, out->container_bits is 8, rows/cols equal the input's.  Weights widened once this way let vitint_linear feed the
 *   tensor cores straight from the TMA copy, with no in-kernel unpacking of that operand; the
 *   value range of the codes is unchanged, so Eq. 1's integer contraction is the same.
 *   Errors: INVALID_ARG, ALIGNMENT. */
int vitint_widen(const vitint_codes* in, const vitint_codes* out, void* stream);

/* a2 + a3. Integerized linear layer (Eq. 1-2): acc[m][n] = sum_k q_x[m][k] * q_w[n][k]
 *   in int32, then the epilogue above.
 *   x: codes [M, K];  w: codes [N, K] (one row per output channel);  w_step: device [N]
 *   (DEQUANT and GELU epilogues; may be NULL for ACC_I32 / plain REQUANT);  bias: device
 *   [N] or NULL.  out / ld_out: int32* and elements (ACC_I32), float* and elements
 *   (DEQUANT_F32), packed bytes and pitch in bytes (REQUANT; 16-byte aligned, the row
 *   padding up to ld_out is written as zero).
 *   Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED, OVERFLOW_BOUND (K*max|q_x|*max|q_w| >= 2^31
 *   over the declared code ranges), CUDA. */
int vitint_linear(const vitint_codes* x, float x_step, const vitint_codes* w, const float* w_step,
                  const float* bias, const vitint_epilogue* epi, void* out, int64_t ld_out, void* stream);

/* QKV projection with the per-head quantizing LayerNorm in its epilogue (the self-attention module of Section V-B:
 *   a LayerNorm over each head's 64 channels in front of the Q and K quantizers, statistics by Eq. 5, comparator
 *   quantizer of Fig. 5(b); Section IV-C).  One GEMM over the stacked weights w_qkv [3D, K], D = heads*64:
 *     columns [0, D) (Q) and [D, 2D) (K): y = fma(float(acc), fl32(x_step * w_step[n]), bias[n]); over every group of
 *       64 consecutive columns (a head) the running statistics of Eq. 5 in channel order, V = S + n_eps, and the level
 *       Qn + #{t : copysign(d*d, d) > V * refs[s][j][t]}, d = y - mu negated where flip[s][j] != 0 -- exactly the
 *       arithmetic of vitint_layernorm_compare_quantize on the fp32 rows, which here never reach memory;
 *     columns [2D, 3D) (V): clamp(rint(fma(float(acc), alpha_v[n-2D], beta_v[n-2D]))) as in the REQUANT epilogue.
 *   w_step, bias: device [3D] (the first 2D entries are read; bias may be NULL).  refs: device
 *   [2][64][2^bits - 1] ascending per channel, flip: device [2][64] bytes or NULL (s = 0 for Q, 1 for K; the
 *   arrays vitint_fold_layernorm_references produces, Q's then K's).  n_eps = 64 * eps.
 *   out: signed codes [M, 3D] of at most 4 bits (any container), every byte of every row written.
 *   stats: device fp32 [2][M*heads][2] receiving (mu, V) of every Q and K head row, or NULL.
 *   Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED (codes wider than 4 bits), OVERFLOW_BOUND, CUDA. */
int vitint_linear_qkv_norm(const vitint_codes* x, float x_step, const vitint_codes* w_qkv, const float* w_step,
                           const float* bias, const float* refs, const uint8_t* flip, float n_eps,
                           const float* alpha_v, const float* beta_v, const vitint_codes* out, float* stats,
                           void* stream);

/* a2 through the FP4 tensor-core kind (Section V-B: fewer bits, cheaper multiply-accumulate).  e2m1 represents
 *   0, 1/2, 1, 3/2, 2, 3, 4, 6 and their negatives, so signed codes of at most 3 bits (-4 .. 3) and unsigned codes of
 *   at most 2 bits (0 .. 3) are exact operands of tcgen05 kind::mxf4 with unit block scales; their products are
 *   integers and the fp32 accumulators hold the sums exactly (checked by brute force in the tests).
 *   acc[m][n] = sum_k q_x[m][k] * q_w[n][k], written as int32.
 *   x: codes [M, K], w: codes [N, K], both stored one code per byte (container_bits = 8), K <= 2^20;
 *   out: device int32 [M, ld_out], ld_out >= N;  inexact_flag: device int32, set to 1 if any accumulator was not an
 *   integer (the caller clears it beforehand).  This kernel establishes exactness; it is not tuned for speed.
 *   Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED (packed containers, or codes e2m1 cannot represent), CUDA. */
int vitint_linear_e2m1(const vitint_codes* x, const vitint_codes* w, int32_t* out, int64_t ld_out,
                       int32_t* inexact_flag, void* stream);

/* Strided set of [tokens, head_dim] code slabs inside a larger code matrix (the Q, K
 * or V part of a QKV activation).  Slab (image b, head h) starts at
 * data + b*image_stride_bytes + h*head_stride_bytes; rows are pitch_bytes apart.
 * head_dim is 64.  All three byte quantities are multiples of 16. */
typedef struct {
    const void* data;
    int64_t pitch_bytes, image_stride_bytes, head_stride_bytes;
    int32_t bits, is_signed;
} vitint_slabs;

/* a4. S[p][i][j] = sum_c Q_p[i][c] * K_p[j][c] for every problem p = b*heads + h
 *   (Eq. 3 before the scale).  s_out: int32, problem p at s_out + p*tokens*ld_s, row i at
 *   + i*ld_s (ld_s >= tokens, elements). */
int vitint_qk(const vitint_slabs* q, const vitint_slabs* k, int32_t batch, int32_t heads, int32_t tokens,
              int32_t* s_out, int64_t ld_s, void* stream);

/* a5. Scale + row softmax + quantize (Eq. 3): t_j = fl32((float)S_j * c), p = softmax_j(t)
 *   in fp32 with <= 2 ulp error, q_j = clamp(rint(p_j / p_step), 0, 2^bits - 1) decided in
 *   fp32 (one IEEE division).  s: int32 [rows, ld_s];  p_out: unsigned codes [rows, cols]
 *   (padding written as zero);  p_f32: optional fp32 probabilities [rows, ld_p] or NULL.
 *   cols <= 1024. */
int vitint_softmax_quantize(const int32_t* s, int64_t rows, int32_t cols, int64_t ld_s, float c, float p_step,
                            const vitint_codes* p_out, float* p_f32, int64_t ld_p, void* stream);

/* a5 for scores of known range (the scores Q K^T of b-bit codes satisfy |S| <= 64 * max|q| * max|k|): the same
 *   result as vitint_softmax_quantize -- Eq. 3's softmax of t_j = fl32(S_j * c), probabilities within 2 ulp, codes
 *   clamp(rint(p / p_step), 0, 2^bits - 1) -- with exp(t_j) read from a table of exp(fl32(s * c)), s = -score_bound
 *   .. score_bound (fp64 exp, rounded once), so the kernel is bound by memory traffic instead of arithmetic.
 *   exp(t_j) / sum_k exp(t_k) is the softmax exactly; no maximum is subtracted, hence score_bound * |c| <= 80.
 *   workspace: device memory, 256-byte aligned, at least vitint_softmax_table_workspace_bytes(score_bound) bytes;
 *   it receives the table (one more small launch) unless table_ready != 0, in which case it already holds the table
 *   an earlier call with the same c and score_bound wrote.  s must be 16-byte aligned with ld_s % 4 == 0.
 *   A score outside the declared range cannot touch memory outside the table; it makes that row's codes meaningless
 *   and the next vitint_device_status() returns VITINT_ERR_INVALID_ARG.
 *   Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, UNSUPPORTED (cols > 895, score_bound > 8192, score_bound*|c| > 80:
 *   use vitint_softmax_quantize), CUDA. */
size_t vitint_softmax_table_workspace_bytes(int32_t score_bound);
int vitint_softmax_quantize_bounded(const int32_t* s, int64_t rows, int32_t cols, int64_t ld_s, float c, float p_step,
                                    int32_t score_bound, const vitint_codes* p_out, float* p_f32, int64_t ld_p,
                                    void* workspace, size_t workspace_bytes, int32_t table_ready, void* stream);

/* a5, shift form (Eq. 4 with the division-free comparator quantizer of Section IV-B).  Integer and
 *   single-rounding fp32 operations only, so the codes are unique (bit-exact against the definition):
 *     z_j = fl32((float)S_j * c2)   (c2 = s*log2(e): the exponent of 2);  f_j = floor(z_j), r_j = z_j - f_j;
 *     E_j = ((1 + r_j) * 2^23 as an integer) << (30 + f_j - max_k f_k)   (2^r ~ 1 + r; negative counts shift
 *           right and drop bits; the common factor 2^(30 - max f) only keeps the integers inside 64 bits);
 *     Sigma = sum_j E_j (exact);  q_j = #{ k in 1..2^bits-1 : (float)E_j > fl32(fl32((k - 1/2)*p_step) * (float)Sigma) }
 *   i.e. the comparator references are scaled by the row sum instead of dividing by it; the comparison is
 *   strict, as drawn in the paper (it differs from round-to-nearest-even only on exact ties).
 *   s, rows, cols, ld_s, p_out as in vitint_softmax_quantize.  cols <= 1024. */
int vitint_softmax_shift_quantize(const int32_t* s, int64_t rows, int32_t cols, int64_t ld_s, float c2, float p_step,
                                  const vitint_codes* p_out, void* stream);

/* a6. O[p][i][c] = sum_j P_p[i][j] * V_p[j][c] (Section IV-B, W_attn V), then the epilogue
 *   with s_x*s_w[n] replaced by p_step*v_step (bias NULL; alpha/beta/inv_out_step, when
 *   used, are indexed by the output column h*64 + c).
 *   p: codes with rows = batch*heads*tokens (problem p owns rows p*tokens ...), cols = tokens.
 *   out: [batch*tokens, heads*64] matrix (int32 / fp32 elements, or packed with ld_out = pitch
 *   bytes); problem (b, h) writes rows b*tokens + i, columns h*64 + c. */
int vitint_pv(const vitint_codes* p, const vitint_slabs* v, int32_t batch, int32_t heads, int32_t tokens,
              float p_step, float v_step, const vitint_epilogue* epi, void* out, int64_t ld_out, void* stream);

/* a4 + a5 + a6 fused (Eq. 3 and the W_attn V product of Section IV-B in one kernel): for every
 *   (image, head)  S = Q K^T,  P = quantize(softmax(c S), p_step, unsigned p_bits),  O = P V,
 *   o = clamp(rint(fmaf((float)O, alpha_o[h*64+c], beta_o[h*64+c])))  with c = fl32(q_step k_step/8).
 *   S, the probabilities and P stay on the SM.  Results equal the unfused sequence
 *   vitint_qk -> vitint_softmax_quantize -> vitint_pv up to the fp32 tolerance of the softmax
 *   (probabilities within 2 ulp, hence P codes that may differ on near-ties only).
 *   qkv: signed codes [batch*tokens, 3*heads*64] (Q | K | V column blocks);  o_out: codes
 *   [batch*tokens, heads*64] whose bits / signedness select the output format;  alpha_o: device
 *   [heads*64];  beta_o: device [heads*64] or NULL.
 *   workspace: >= vitint_attention_core_workspace_bytes(bits) bytes of device scratch, 256-byte
 *   aligned (holds a table of exp(fl32(s*c)) over all integer scores s); contents undefined after.
 *   Errors: UNSUPPORTED when tokens > 256, the codes are 8-bit, or 64*max|q|*max|k|*c > 80 (use the
 *   unfused calls then); INVALID_ARG, ALIGNMENT, WORKSPACE, CUDA. */
size_t vitint_attention_core_workspace_bytes(int32_t bits);
int vitint_attention_core(const vitint_codes* qkv, int32_t batch, int32_t heads, int32_t tokens, float q_step,
                          float k_step, float p_step, int32_t p_bits, const float* alpha_o, const float* beta_o,
                          const vitint_codes* o_out, void* workspace, size_t workspace_bytes, void* stream);

/* The same core with the exp table prepared once: the table depends only on the code width and on the steps of
 * Q and K (Eq. 3's scale), which are fixed per layer, so a caller that runs the layer many times fills it once
 *   vitint_attention_exp_table(bits, q_step, k_step, table, table_bytes, stream)
 * (table: device memory, 256-byte aligned, >= vitint_attention_core_workspace_bytes(bits) bytes) and then calls
 * vitint_attention_core_prepared with that table and the SAME bits, q_step and k_step: one kernel launch instead
 * of two, results identical to vitint_attention_core.  The table is only read by the prepared call. */
int vitint_attention_exp_table(int32_t bits, float q_step, float k_step, void* table, size_t table_bytes, void* stream);
int vitint_attention_core_prepared(const vitint_codes* qkv, int32_t batch, int32_t heads, int32_t tokens, float q_step,
                                   float k_step, float p_step, int32_t p_bits, const float* alpha_o,
                                   const float* beta_o, const vitint_codes* o_out, const void* table,
                                   size_t table_bytes, void* stream);

/* The fused attention core with the paper's own softmax (Eq. 4: 2^z with z = S c log2 e split into integer part and
 *   residual, 2^r ~ 1 + r, integer shifts; the division-free comparator quantizer of Section IV-B whose references are
 *   scaled by the row sum).  Arguments as vitint_attention_core; the codes of P and O are those of vitint_qk ->
 *   vitint_softmax_shift_quantize -> vitint_pv bit for bit (every step is an integer or a single fp32 operation).
 *   The per-score pair (floor z, mantissa of 1 + r) comes from two tables over the bounded score range, built into
 *   `workspace` (256-byte aligned, at least vitint_attention_core_shift_workspace_bytes(bits) bytes) by one small
 *   launch, unless table_ready != 0: the workspace then still holds the tables an earlier call with the same bits,
 *   q_step and k_step wrote.  The row maximum is subtracted (as shift counts), so unlike vitint_attention_core this
 *   variant has no limit on the size of the logits.
 *   Errors: as vitint_attention_core; UNSUPPORTED also for codes not stored one per byte (container_bits != 8). */
size_t vitint_attention_core_shift_workspace_bytes(int32_t bits);
int vitint_attention_core_shift(const vitint_codes* qkv, int32_t batch, int32_t heads, int32_t tokens, float q_step,
                                float k_step, float p_step, int32_t p_bits, const float* alpha_o, const float* beta_o,
                                const vitint_codes* o_out, void* workspace, size_t workspace_bytes, int32_t table_ready,
                                void* stream);

/* vitint_attention_core without caller-provided scratch.  (No counterpart in the paper: this is
 *   a packaging variant, not a step of the method.)
 *   Who needs it: code that is not allowed to obtain device memory when it runs the attention
 *   core -- for example a plug-in inside a serving process whose whole device-memory budget was
 *   handed out at start-up by another component, or a latency-critical loop that must avoid
 *   cudaMalloc / cudaFree because those calls may synchronize the device.  Such callers still
 *   pass their own input (qkv) and output (o_out) buffers; only the kernel's scratch -- the table
 *   of exp(fl32(s*c)) over all integer scores -- comes from the library: a fixed device array of
 *   33,280 bytes that every GPU loading the library holds until the process exits.
 *   The function allocates nothing: no cudaMalloc / cudaFree and no allocating library routine.
 *   Limit: the array holds the table of the widest codes the table-driven kernel takes (2-, 3- and
 *   4-bit codes, at most 8193 entries); 8-bit codes are rejected with VITINT_ERR_UNSUPPORTED, as
 *   in vitint_attention_core.  All other arguments, results and errors are those of
 *   vitint_attention_core, argument errors being reported first.
 *   The first call on each device looks up the array's device address (with that device
 *   current; concurrent first calls from several host threads are safe); make that first call
 *   outside any stream capture.
 *   Every call on a device uses the same array and rewrites all the entries it needs, so nothing
 *   carries over between calls -- but two calls that overlap on the GPU (different streams) race
 *   on it: serialize calls per device. */
int vitint_attention_core_noalloc(const vitint_codes* qkv, int32_t batch, int32_t heads, int32_t tokens,
                                  float q_step, float k_step, float p_step, int32_t p_bits, const float* alpha_o,
                                  const float* beta_o, const vitint_codes* o_out, void* stream);

/* a7. Integerized self-attention block (Fig. 1(b)):
 *   QKV linear (requantized with per-channel alpha_qkv/beta_qkv, i.e. three per-tensor
 *   steps q_step, k_step, v_step laid out per output channel) -> Q K^T -> scale, softmax,
 *   quantize to unsigned p_bits at p_step -> P V -> requantize with alpha_o/beta_o to
 *   signed o codes -> output projection with proj_epi.
 *   x: codes [batch*tokens, D], D = heads*64.  w_qkv: codes [3D, D]; w_proj: codes [D, D].
 *   alpha_qkv, beta_qkv: device [3D];  alpha_o: device [D], beta_o: device [D] or NULL.
 *   w_proj_step, b_proj: device [D] as in vitint_linear (x_step of the projection = o_step).
 *   out / ld_out as in vitint_linear for proj_epi.mode.
 *   dbg_qkv / dbg_p / dbg_o: optional descriptors (data may point anywhere suitably sized)
 *   that receive copies of the intermediate codes: QKV [M, 3D], P [batch*heads*tokens, tokens],
 *   O [M, D]; NULL to skip.
 *   workspace: device scratch of at least vitint_attention_block_workspace_bytes(...) bytes,
 *   256-byte aligned; contents are undefined afterwards.
 *   The middle of the block runs as vitint_attention_core when that call supports the shape and
 *   dbg_p is NULL, otherwise as vitint_qk -> vitint_softmax_quantize -> vitint_pv. */
typedef struct {
    int32_t batch, tokens, heads;
    int32_t bits;                 /* activation / weight code width of the block */
    vitint_codes w_qkv;
    const float* alpha_qkv;
    const float* beta_qkv;
    float q_step, k_step, v_step, p_step, o_step;
    int32_t p_bits;
    const float* alpha_o;
    const float* beta_o;
    vitint_codes w_proj;
    const float* w_proj_step;
    const float* b_proj;
    vitint_epilogue proj_epi;
} vitint_attention_desc;

size_t vitint_attention_block_workspace_bytes(const vitint_attention_desc* d);

int vitint_attention_block(const vitint_codes* x, const vitint_attention_desc* d, void* out, int64_t ld_out,
                           const vitint_codes* dbg_qkv, const vitint_codes* dbg_p, const vitint_codes* dbg_o,
                           void* workspace, size_t workspace_bytes, void* stream);

/* Glue between integerized linears (the full-precision LayerNorm island of Fig. 1(b)):
 *   y = (x - mean)/sqrt(var + eps) * gamma + beta per row in fp32 (biased variance), then
 *   the a1 quantizer with `step`.  out: codes [rows, cols];  y_f32: optional fp32 copy of y
 *   [rows, ld_y] or NULL.  cols <= 4096 and a multiple of 4. */
int vitint_layernorm_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx, const float* gamma,
                              const float* beta, float eps, float step, const vitint_codes* out, float* y_f32,
                              int64_t ld_y, void* stream);

/* Quantizing LayerNorm of Section IV-C: running statistics of Eq. 5 and the division- and square-root-free
 * comparator of Fig. 5(b).
 *   statistics, per row, in the order of Eq. 5, every operation one round-to-nearest fp32 operation:
 *     delta = x_i - mu;  mu = mu + delta / i;  S = S + delta * (x_i - mu)      (mu_0 = S_0 = 0)
 *     V = S + n_eps   (S is the unnormalised sum of squared deviations; n_eps = cols * eps)
 *   quantizer: level = Qn + number of references t with  copysign(d*d, d) > V * refs[col][t],
 *     d = x - mu (negated where flip[col] != 0).  This decides (x-mu)/sigma*gamma+beta > (k - 1/2)*step
 *     for k = Qn+1 .. Qp when the caller supplies refs[col][t] = sgn(c) c^2 / cols with
 *     c = ((k - 1/2) step - beta_col) / gamma_col (negated where gamma_col < 0, and then flip[col] = 1).
 * x: device fp32 [rows, ldx], 16-byte aligned, ldx a multiple of 4, finite values.  refs: device fp32
 * [cols][2^bits - 1], ascending along t (the bisection in the kernel relies on it).  flip: device bytes
 * [cols] or NULL (no negative gain).  n_eps > 0.  out: codes [rows, cols] of 2, 3 or 4 bits in any
 * container, cols a multiple of 4 and at most 4096; padding bytes up to the pitch are written as zero.  stats: device fp32
 * [rows][2], receives (mu, V) of every row (it also carries them from the first kernel to the second).
 * Returns VITINT_ERR_UNSUPPORTED for 8-bit codes, VITINT_ERR_ALIGNMENT / VITINT_ERR_INVALID_ARG otherwise.
 * Asynchronous on `stream`; nothing is allocated. */
int vitint_layernorm_compare_quantize(const float* x, int64_t rows, int64_t cols, int64_t ldx, const float* refs,
                                      const uint8_t* flip, float n_eps, const vitint_codes* out, float* stats,
                                      void* stream);

/* Host-side helpers (no device work, HOST pointers): the constants that the method absorbs into the stage behind a
 * contraction, computed in fp64 and rounded once to fp32.
 *   vitint_fold_requant (Eq. 2, "equivalent bias" and "post-scaling factor" followed by a quantizer of step
 *     out_step[i]):  alpha[i] = x_step * w_step[i] / out_step[i],  beta[i] = bias[i] / out_step[i] (0 when bias is
 *     NULL), i < n: the arguments of the REQUANT epilogue.  Steps must be positive and finite.
 *   vitint_fold_layernorm_references (Fig. 5(b)):  for column j and threshold k = Qn+1 .. Qp,
 *     c = ((k - 1/2) step - beta[j]) / gamma[j], negated where gamma[j] < 0 (then flip[j] = 1, else 0);
 *     refs[j][k - Qn - 1] = sgn(c) c^2 / cols: the arguments of vitint_layernorm_compare_quantize.  gamma[j] != 0.
 * Return VITINT_OK or VITINT_ERR_INVALID_ARG. */
int vitint_fold_requant(float x_step, const float* w_step, const float* bias, const float* out_step, int64_t n,
                        float* alpha, float* beta);
int vitint_fold_layernorm_references(const float* gamma, const float* beta, float step, int32_t bits,
                                     int32_t is_signed, int64_t cols, float* refs, uint8_t* flip);

#ifdef __cplusplus
}
#endif
#endif /* VITINT_H_ */
