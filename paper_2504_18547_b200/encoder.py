"""Integerized ViT encoder layer as a fixed sequence of C-ABI calls with preallocated buffers.

LayerNorm+quantize -> QKV linear -> Q K^T -> softmax+quantize -> P V -> projection (+residual)
-> LayerNorm+quantize -> fc1 (GELU, requantize) -> fc2 (+residual).  This module only owns
device buffers and marshals arguments; every step runs in the library's kernels.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B

STAGES_UNFUSED = ("ln1_quant", "qkv_linear", "qk", "softmax_quant", "pv", "proj_linear", "ln2_quant", "fc1_linear",
                  "fc2_linear")
STAGES_FUSED = ("ln1_quant", "qkv_linear", "attention_core", "proj_linear", "ln2_quant", "fc1_linear", "fc2_linear")
# stages that run in the integer GEMM kernel
GEMM_STAGES = ("qkv_linear", "qk", "pv", "proj_linear", "fc1_linear", "fc2_linear")


def _dev(a, device):
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


class EncoderLayer:
    def __init__(self, batch: int, tokens: int, heads: int, mlp_dim: int, bits: int, prm: dict, device="cuda",
                 eps: float = 1e-6, widen_weights: bool = True, fused_attention: bool = True,
                 wide_activations: bool = True, softmax: str = "exp", layernorm: str = "fp32"):
        self.batch, self.tokens, self.heads, self.bits, self.eps = batch, tokens, heads, bits, eps
        self.dim = D = heads * 64
        self.mlp_dim = F = mlp_dim
        self.rows = M = batch * tokens
        self.device = device
        if softmax not in ("exp", "shift"):
            raise ValueError("softmax must be 'exp' (Eq. 3) or 'shift' (Eq. 4 with the comparator quantizer)")
        self.softmax = softmax
        if layernorm not in ("fp32", "compare"):
            raise ValueError("layernorm must be 'fp32' (LayerNorm, then round) or 'compare' (Eq. 5 statistics with the "
                             "division- and square-root-free comparator quantizer)")
        self.layernorm = layernorm
        # the shift-based softmax is a separate kernel: it runs in the unfused attention pipeline
        # the fused core takes the exp softmax for any container and the Eq. 4 softmax for byte-stored codes
        # (beyond 256 tokens the exp core runs its chunked two-pass kernel, which takes byte-stored codes)
        self.fused_attention = (fused_attention and bits != 8
                                and ((softmax == "exp" and (tokens <= 256 or (wide_activations and tokens <= 4096)))
                                     or (softmax == "shift" and wide_activations and tokens <= 256)))
        self.stages = STAGES_FUSED if self.fused_attention else STAGES_UNFUSED
        d = lambda a: _dev(a, device)
        f = lambda k: float(prm[k])
        self.s_ln, self.s_q, self.s_k, self.s_v = f("s_ln"), f("s_q"), f("s_k"), f("s_v")
        self.s_p, self.s_o, self.s_g = f("s_p"), f("s_o"), f("s_g")
        self.ln1_g, self.ln1_b, self.ln2_g, self.ln2_b = d(prm["ln1_g"]), d(prm["ln1_b"]), d(prm["ln2_g"]), d(prm["ln2_b"])
        if layernorm == "compare":
            self.ln_refs = []
            for gk, bk in (("ln1_g", "ln1_b"), ("ln2_g", "ln2_b")):
                r, fl = B.fold_layernorm_references(prm[gk], prm[bk], prm["s_ln"], bits, True, D)
                self.ln_refs.append((d(r), d(fl)))
            self.n_eps = float(np.float32(np.float64(D) * np.float64(np.float32(eps))))
            self.ln_stats = torch.empty((M, 2), dtype=torch.float32, device=device)
        # weights: quantized once by the library's own quantizer (per-output-channel steps)
        self.w = {}
        for name in ("qkv", "proj", "fc1", "fc2"):
            self.w[name] = B.vitint_quantize(d(prm[f"w_{name}"]), 0.0, bits, True, row_steps=d(prm[f"s_w_{name}"]))
        # the low-bit weight codes, re-stored once in 8-bit containers: the GEMM then feeds this
        # operand to the tensor cores straight from the TMA copy
        self.w_packed = dict(self.w)
        if widen_weights and bits != 8:
            self.w = {n: B.vitint_widen(c) for n, c in self.w.items()}
        self.s_w = {n: d(prm[f"s_w_{n}"]) for n in ("proj", "fc1", "fc2")}
        self.bias = {n: d(prm[f"b_{n}"]) for n in ("proj", "fc1", "fc2")}
        seg = np.concatenate([np.full(D, prm["s_q"]), np.full(D, prm["s_k"]), np.full(D, prm["s_v"])]).astype(np.float32)
        a, b = B.fold_requant(prm["s_ln"], prm["s_w_qkv"], prm["b_qkv"], seg)
        self.alpha_qkv, self.beta_qkv = d(a), d(b)
        a, _ = B.fold_requant(prm["s_p"], np.full(D, prm["s_v"], np.float32), None, prm["s_o"])
        self.alpha_o = d(a)
        self.inv_s_g = d((1.0 / np.full(F, prm["s_g"], np.float64)).astype(np.float32))
        self.c = float(np.float32(float(prm["s_q"]) * float(prm["s_k"]) / 8.0))
        self.c2 = float(np.float32(np.float64(np.float32(self.c)) * np.log2(np.e)))   # exponent of two for Eq. 4
        # activations, stored one code per byte: the consumer's TMA copy is then already the
        # tensor-core operand (the unfused attention kernels read packed q, k, v slabs instead)
        ca = 8 if wide_activations and bits != 8 else 0
        cq = ca if self.fused_attention else 0
        self.x1 = B.Codes.empty(M, D, bits, True, device, container=ca)
        self.qkv = B.Codes.empty(M, 3 * D, bits, True, device, container=cq)
        self.ld_s = (tokens + 3) // 4 * 4
        if self.fused_attention and softmax == "shift":
            # the table of Eq. 4's (integer part, mantissa) pairs is built by the first call and reused
            self.attn_table = torch.empty(B.vitint_attention_core_shift_workspace_bytes(bits), dtype=torch.uint8, device=device)
            self.attn_table_ready = False
        elif self.fused_attention:
            # the exp table of the fused core depends only on the code width and the steps of Q and K: filled once
            self.attn_table = B.vitint_attention_exp_table(bits, self.s_q, self.s_k, device=device)
        else:
            self.S = torch.empty((batch * heads * tokens, self.ld_s), dtype=torch.int32, device=device)
            self.P = B.Codes.empty(batch * heads * tokens, tokens, bits, False, device)
            # scores of b-bit codes are bounded by 64 * 2^(b-1) * 2^(b-1): where the table-driven softmax takes that
            # range its exp table is built by the first call and reused afterwards
            half = 1 << ((4 if bits == 3 else bits) - 1)
            self.score_bound = 64 * half * half
            self.sm_table = None
            if (softmax == "exp" and B.vitint_softmax_table_workspace_bytes(self.score_bound) > 0
                    and self.score_bound * abs(self.c) <= 80.0 and tokens <= 895):
                self.sm_table = torch.empty(B.vitint_softmax_table_workspace_bytes(self.score_bound), dtype=torch.uint8,
                                            device=device)
                self.sm_table_ready = False
        self.O = B.Codes.empty(M, D, bits, True, device, container=ca)
        self.h = torch.empty((M, D), dtype=torch.float32, device=device)
        self.x2 = B.Codes.empty(M, D, bits, True, device, container=ca)
        self.g = B.Codes.empty(M, F, bits, False, device, container=ca)
        self.slabs = None if self.fused_attention else [B.Slabs.of_qkv(self.qkv, tokens, D, i) for i in range(3)]
        self.epi_qkv = B.Epilogue(mode=B.EPI_REQUANT, alpha=self.alpha_qkv, beta=self.beta_qkv, out_bits=bits,
                                  out_signed=True, out_container=cq)
        self.epi_o = B.Epilogue(mode=B.EPI_REQUANT, alpha=self.alpha_o, out_bits=bits, out_signed=True, out_container=ca)
        self.epi_fc1 = B.Epilogue(mode=B.EPI_REQUANT, act=1, inv_out_step=self.inv_s_g, out_bits=bits, out_signed=False,
                                  out_container=ca)

    def forward(self, x: torch.Tensor, out: torch.Tensor, events: list | None = None) -> torch.Tensor:
        """x, out: fp32 [batch*tokens, dim] on the device.  `events`, when given, receives
        len(self.stages)+1 recorded CUDA events bracketing the stages."""
        def mark():
            if events is not None:
                e = torch.cuda.Event(enable_timing=True)
                e.record()
                events.append(e)
        b, t, h = self.batch, self.tokens, self.heads
        mark()
        if self.layernorm == "compare":
            B.vitint_layernorm_compare_quantize(x, self.ln_refs[0][0], self.ln_refs[0][1], self.n_eps, self.bits, True,
                                                out=self.x1, stats=self.ln_stats)
        else:
            B.vitint_layernorm_quantize(x, self.ln1_g, self.ln1_b, self.eps, self.s_ln, self.bits, True, out=self.x1)
        mark()
        B.vitint_linear(self.x1, self.s_ln, self.w["qkv"], None, None, self.epi_qkv, out=self.qkv)
        mark()
        if self.fused_attention and self.softmax == "shift":
            B.vitint_attention_core_shift(self.qkv, b, h, t, self.s_q, self.s_k, self.s_p, self.bits, self.alpha_o, None,
                                          out=self.O, workspace=self.attn_table, table_ready=self.attn_table_ready)
            self.attn_table_ready = True
        elif self.fused_attention:
            B.vitint_attention_core_prepared(self.qkv, b, h, t, self.s_q, self.s_k, self.s_p, self.bits, self.alpha_o,
                                             None, out=self.O, table=self.attn_table)
        else:
            B.vitint_qk(self.slabs[0], self.slabs[1], b, h, t, out=self.S, ld_s=self.ld_s)
            mark()
            if self.softmax == "shift":
                B.vitint_softmax_shift_quantize(self.S, t, self.c2, self.s_p, self.bits, out=self.P)
            elif self.sm_table is not None:
                B.vitint_softmax_quantize_bounded(self.S, t, self.c, self.s_p, self.bits, self.score_bound, out=self.P,
                                                  workspace=self.sm_table, table_ready=self.sm_table_ready)
                self.sm_table_ready = True
            else:
                B.vitint_softmax_quantize(self.S, t, self.c, self.s_p, self.bits, out=self.P)
            mark()
            B.vitint_pv(self.P, self.slabs[2], b, h, t, self.s_p, self.s_v, self.epi_o, out=self.O)
        mark()
        B.vitint_linear(self.O, self.s_o, self.w["proj"], self.s_w["proj"], self.bias["proj"],
                        B.Epilogue(mode=B.EPI_DEQUANT_F32, residual=x), out=self.h)
        mark()
        if self.layernorm == "compare":
            B.vitint_layernorm_compare_quantize(self.h, self.ln_refs[1][0], self.ln_refs[1][1], self.n_eps, self.bits,
                                                True, out=self.x2, stats=self.ln_stats)
        else:
            B.vitint_layernorm_quantize(self.h, self.ln2_g, self.ln2_b, self.eps, self.s_ln, self.bits, True, out=self.x2)
        mark()
        B.vitint_linear(self.x2, self.s_ln, self.w["fc1"], self.s_w["fc1"], self.bias["fc1"], self.epi_fc1, out=self.g)
        mark()
        B.vitint_linear(self.g, self.s_g, self.w["fc2"], self.s_w["fc2"], self.bias["fc2"],
                        B.Epilogue(mode=B.EPI_DEQUANT_F32, residual=self.h), out=out)
        mark()
        return out

    def stage_ops(self) -> dict:
        """Integer operations (2 per multiply-accumulate, true shapes) of each contraction."""
        M, D, F, T = self.rows, self.dim, self.mlp_dim, self.tokens
        n = self.batch * self.heads
        return {"qkv_linear": 2 * M * D * 3 * D, "qk": 2 * n * T * T * 64, "pv": 2 * n * T * T * 64,
                "attention_core": 4 * n * T * T * 64, "proj_linear": 2 * M * D * D, "fc1_linear": 2 * M * D * F,
                "fc2_linear": 2 * M * F * D}

    def stage_bytes(self) -> dict:
        """Algorithmic HBM bytes of the streaming stages (4 + c/8 per element)."""
        c = 4 if self.bits == 3 else self.bits
        cx = self.x1.stored_bits
        M, D, T = self.rows, self.dim, self.tokens
        n = self.batch * self.heads * T
        return {"ln1_quant": M * D * 4 + M * D * cx // 8, "ln2_quant": M * D * 4 + M * D * cx // 8,
                "softmax_quant": n * T * 4 + n * ((T * c + 7) // 8)}


class EncoderStack:
    """`layers` integerized encoder layers applied in sequence (each with its own weights and steps);
    the fp32 residual stream ping-pongs between two device buffers."""

    def __init__(self, layer_params: list, batch: int, tokens: int, heads: int, mlp_dim: int, bits: int,
                 device="cuda", **kw):
        self.layers = [EncoderLayer(batch, tokens, heads, mlp_dim, bits, prm, device, **kw) for prm in layer_params]
        rows, dim = batch * tokens, heads * 64
        self.buf = [torch.empty((rows, dim), dtype=torch.float32, device=device) for _ in range(2)]

    def forward(self, x: torch.Tensor, out: torch.Tensor) -> torch.Tensor:
        cur = x
        n = len(self.layers)
        for i, layer in enumerate(self.layers):
            dst = out if i == n - 1 else self.buf[i & 1]
            layer.forward(cur, dst)
            cur = dst
        return out

    def ops(self) -> int:
        return sum(sum(v for k, v in l.stage_ops().items() if k in l.stages) for l in self.layers)


class NormedAttention:
    """The self-attention module laid out as in the paper's power table (Section V-B): separate Q, K and V
    linear layers, a LayerNorm over each head's 64 channels in front of the Q and K quantizers (statistics by
    Eq. 5, comparator quantizer of Fig. 5(b)), Q K^T, the Eq. 4 softmax with its division-free quantizer, P V.
    A fixed sequence of C-ABI calls over preallocated buffers; `qkn` holds the per-head LayerNorm parameters
    (qn_g, qn_b, kn_g, kn_b over 64 channels) and the steps s_qn, s_kn of the normalised values.
    fused=True (default): one QKV GEMM whose epilogue normalises and quantizes the Q and K heads and requantizes V,
    then the fused attention core with the Eq. 4 softmax inside (2 launches; `fused_core=False` keeps Q K^T, softmax
    and P V as three kernels with S and P in memory: 4 launches); fused=False: separate Q, K, V linears with fp32 Q
    and K rows and a LayerNorm kernel pass each (10 launches, the fp32 rows and their statistics left in `f32` /
    `stats` for inspection)."""

    def __init__(self, batch: int, tokens: int, heads: int, bits: int, prm: dict, qkn: dict, device="cuda",
                 eps: float = 1e-6, fused: bool = True, fused_core: bool = True):
        self.fused = fused
        self.fused_core = fused and fused_core and tokens <= 256 and bits != 8
        self.batch, self.tokens, self.heads, self.bits = batch, tokens, heads, bits
        self.dim = D = heads * 64
        self.rows = M = batch * tokens
        d = lambda a: _dev(a, device)
        w = B.vitint_widen(B.vitint_quantize(d(prm["w_qkv"]), 0.0, bits, True, row_steps=d(prm["s_w_qkv"])))
        part = lambda i: B.Codes(w.data[i * D:(i + 1) * D], D, D, bits, True, 8)
        self.w_qkv, self.w_q, self.w_k, self.w_v = w, part(0), part(1), part(2)
        self.s_w_all, self.bias_all = d(prm["s_w_qkv"]), d(prm["b_qkv"])
        self.s_w = [self.s_w_all[i * D:(i + 1) * D] for i in range(2)]
        self.bias = [self.bias_all[i * D:(i + 1) * D] for i in range(2)]
        a, b = B.fold_requant(1.0, prm["s_w_qkv"][2 * D:], prm["b_qkv"][2 * D:], prm["s_v"])
        self._alpha_v_unit, self.beta_v = a, d(b)             # alpha scales with the input step given to forward()
        self.refs = []
        for n in ("q", "k"):
            r, fl = B.fold_layernorm_references(qkn[n + "n_g"], qkn[n + "n_b"], qkn["s_" + n + "n"], bits, True, 64)
            self.refs.append((d(r), d(fl)))
        self.refs_all = torch.stack([r for r, _ in self.refs]).contiguous()
        self.flip_all = torch.stack([f for _, f in self.refs]).contiguous()
        self.n_eps = float(np.float32(np.float64(64) * np.float64(np.float32(eps))))
        self.s_v, self.s_p, self.s_o = float(prm["s_v"]), float(prm["s_p"]), float(prm["s_o"])
        c = np.float32(float(qkn["s_qn"]) * float(qkn["s_kn"]) / 8.0)
        self.c2 = float(np.float32(np.float64(c) * np.log2(np.e)))
        a_o, _ = B.fold_requant(prm["s_p"], np.full(D, prm["s_v"], np.float32), None, prm["s_o"])
        self.alpha_o = d(a_o)
        self._prm = prm
        self._alpha_v_for = None
        c_bits = 4 if bits == 3 else bits
        self.stats_all = torch.empty((2, M * heads, 2), dtype=torch.float32, device=device)
        self.stats = [self.stats_all[0], self.stats_all[1]]
        pitch = D * c_bits // 8
        if self.fused_core:
            # byte-stored QKV codes: the operand form of the fused core
            self.qkv = B.Codes.empty(M, 3 * D, bits, True, device, container=8)
            self.core_ws = torch.empty(B.vitint_attention_core_shift_workspace_bytes(bits), dtype=torch.uint8, device=device)
            self.core_ws_ready = False
            self.slabs = self.v_slabs = None
        elif fused:
            self.qkv = B.Codes.empty(M, 3 * D, bits, True, device)
            qp = self.qkv.pitch
            self.slabs = [B.Slabs(self.qkv.data, i * pitch, qp, qp * tokens, 64 * c_bits // 8, bits, True) for i in range(2)]
            self.v_slabs = B.Slabs(self.qkv.data, 2 * pitch, qp, qp * tokens, 64 * c_bits // 8, bits, True)
        else:
            self.f32 = [torch.empty((M, D), dtype=torch.float32, device=device) for _ in range(2)]
            self.qk_codes = [B.Codes.empty(M * heads, 64, bits, True, device) for _ in range(2)]
            self.slabs = [B.Slabs(c.data, 0, pitch, pitch * tokens, 64 * c_bits // 8, bits, True) for c in self.qk_codes]
            self.v = B.Codes.empty(M, D, bits, True, device)
            self.v_slabs = B.Slabs(self.v.data, 0, self.v.pitch, self.v.pitch * tokens, 64 * c_bits // 8, bits, True)
        self.ld_s = (tokens + 3) // 4 * 4
        if not self.fused_core:
            self.S = torch.empty((batch * heads * tokens, self.ld_s), dtype=torch.int32, device=device)
            self.P = B.Codes.empty(batch * heads * tokens, tokens, bits, False, device)
        self.O = B.Codes.empty(M, D, bits, True, device)
        self.epi_o = B.Epilogue(mode=B.EPI_REQUANT, alpha=self.alpha_o, out_bits=bits, out_signed=True)
        self.s_qn, self.s_kn = float(qkn["s_qn"]), float(qkn["s_kn"])

    def forward(self, x: "B.Codes", s_x: float) -> "B.Codes":
        """x: codes [batch*tokens, dim] with step s_x.  Returns the O codes [batch*tokens, dim]."""
        if self._alpha_v_for != float(s_x):
            D = self.dim
            a, _ = B.fold_requant(s_x, self._prm["s_w_qkv"][2 * D:], None, self._prm["s_v"])
            self.alpha_v = _dev(a, self.O.data.device)
            self._alpha_v_for = float(s_x)
        b, t, h = self.batch, self.tokens, self.heads
        if self.fused:
            B.vitint_linear_qkv_norm(x, s_x, self.w_qkv, self.s_w_all, self.bias_all, self.refs_all, self.flip_all,
                                     self.n_eps, self.alpha_v, self.beta_v, self.bits, out=self.qkv, stats=self.stats_all)
        else:
            for i, w in enumerate((self.w_q, self.w_k)):
                B.vitint_linear(x, s_x, w, self.s_w[i], self.bias[i], B.Epilogue(mode=B.EPI_DEQUANT_F32), out=self.f32[i])
                B.vitint_layernorm_compare_quantize(self.f32[i].view(self.rows * h, 64), self.refs[i][0], self.refs[i][1],
                                                    self.n_eps, self.bits, True, out=self.qk_codes[i], stats=self.stats[i])
            B.vitint_linear(x, s_x, self.w_v, None, None,
                            B.Epilogue(mode=B.EPI_REQUANT, alpha=self.alpha_v, beta=self.beta_v, out_bits=self.bits,
                                       out_signed=True), out=self.v)
        if self.fused_core:
            B.vitint_attention_core_shift(self.qkv, b, h, t, self.s_qn, self.s_kn, self.s_p, self.bits, self.alpha_o, None,
                                          out=self.O, workspace=self.core_ws, table_ready=self.core_ws_ready)
            self.core_ws_ready = True
            return self.O
        B.vitint_qk(self.slabs[0], self.slabs[1], b, h, t, out=self.S, ld_s=self.ld_s)
        B.vitint_softmax_shift_quantize(self.S, t, self.c2, self.s_p, self.bits, out=self.P)
        B.vitint_pv(self.P, self.v_slabs, b, h, t, self.s_p, self.s_v, self.epi_o, out=self.O)
        return self.O

    def ops(self) -> int:
        """Integer operations (2 per multiply-accumulate) of the five contractions."""
        M, D, T = self.rows, self.dim, self.tokens
        return 2 * (3 * M * D * D + 2 * self.batch * self.heads * T * T * 64)


class DeitModel:
    """The whole DeiT-S-shaped model as C-ABI calls: quantize the flattened patches, patch embedding as an
    integerized linear whose fp32 epilogue adds the token table (class / distillation tokens and position
    embeddings; the two token rows of every image carry zero patches), the encoder layers, final LayerNorm +
    quantizer on the class and distillation rows, two classifier heads (the second adds onto the first's logits)."""

    def __init__(self, ends: dict, layer_params: list, batch: int, tokens: int, heads: int, mlp_dim: int, bits: int,
                 device="cuda", eps: float = 1e-6, **layer_kw):
        self.batch, self.tokens, self.bits, self.eps = batch, tokens, bits, eps
        self.dim = D = heads * 64
        M = batch * tokens
        d = lambda a: _dev(a, device)
        self.stack = EncoderStack(layer_params, batch, tokens, heads, mlp_dim, bits, device, eps=eps, **layer_kw)
        q = lambda w, s: B.vitint_widen(B.vitint_quantize(d(w), 0.0, bits, True, row_steps=d(s)))
        self.w_pe, self.s_w_pe, self.b_pe = q(ends["w_pe"], ends["s_w_pe"]), d(ends["s_w_pe"]), d(ends["b_pe"])
        self.table = d(np.tile(np.asarray(ends["tokens"], np.float32), (batch, 1)))
        self.s_patch, self.s_lnf = float(ends["s_patch"]), float(ends["s_lnf"])
        self.lnf_g, self.lnf_b = d(ends["lnf_g"]), d(ends["lnf_b"])
        self.heads_w = [(q(ends["w_" + n], ends["s_w_" + n]), d(ends["s_w_" + n]), d(ends["b_" + n]))
                        for n in ("head", "head_dist")]
        n_cls = ends["w_head"].shape[0]
        self.xq = B.Codes.empty(M, ends["w_pe"].shape[1], bits, True, device, container=8)
        self.x0 = torch.empty((M, D), dtype=torch.float32, device=device)
        self.x_final = torch.empty((M, D), dtype=torch.float32, device=device)
        self.head_codes = [B.Codes.empty(batch, D, bits, True, device, container=8) for _ in range(2)]
        self.logits = [torch.empty((batch, n_cls), dtype=torch.float32, device=device) for _ in range(2)]

    def forward(self, patches: torch.Tensor) -> torch.Tensor:
        """patches: fp32 [batch*tokens, patch_dim] on the device.  Returns the summed logits [batch, classes]."""
        B.vitint_quantize(patches, self.s_patch, self.bits, True, out=self.xq)
        B.vitint_linear(self.xq, self.s_patch, self.w_pe, self.s_w_pe, self.b_pe,
                        B.Epilogue(mode=B.EPI_DEQUANT_F32, residual=self.table), out=self.x0)
        self.stack.forward(self.x0, self.x_final)
        for i, (w, s_w, b) in enumerate(self.heads_w):
            rows = self.x_final[i::self.tokens]                 # class rows (i = 0), distillation rows (i = 1)
            B.vitint_layernorm_quantize(rows, self.lnf_g, self.lnf_b, self.eps, self.s_lnf, self.bits, True,
                                        out=self.head_codes[i])
            B.vitint_linear(self.head_codes[i], self.s_lnf, w, s_w, b,
                            B.Epilogue(mode=B.EPI_DEQUANT_F32, residual=self.logits[0] if i else None),
                            out=self.logits[i])
        return self.logits[1]

    def ops(self) -> int:
        M, D = self.batch * self.tokens, self.dim
        ends = 2 * M * D * self.xq.cols + 2 * 2 * self.batch * D * self.logits[0].shape[1]
        return ends + self.stack.ops()
