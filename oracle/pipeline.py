"""Stage-by-stage compositions of the oracle: attention block (Fig. 1(b)) and a
ViT encoder layer with fp32 LayerNorm / GELU islands between integerized linears.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  Every function returns a
dict holding all intermediate stages so a checker can compare stage by stage.
"""
from __future__ import annotations

import math

import numpy as np

import oracle as vo


def softmax_scale(s_q, s_k, head_dim: int) -> np.float32:
    """c = s_q s_k / sqrt(d), fp64 then one rounding (the scale `s` of Eq. 3)."""
    return np.float32(float(s_q) * float(s_k) / math.sqrt(head_dim))


def inv_step(s) -> np.ndarray:
    return (1.0 / np.asarray(s, dtype=np.float64)).astype(np.float32)


def fold(s_x, s_w, bias, s_out):
    """Eq. 2 folding: alpha = s_x s_w/s_out, beta = b/s_out (fp64, one rounding each)."""
    s_w64 = np.asarray(s_w, dtype=np.float64)
    s_out64 = np.broadcast_to(np.asarray(s_out, dtype=np.float64), s_w64.shape)
    alpha = (float(s_x) * s_w64 / s_out64).astype(np.float32)
    beta = np.zeros_like(alpha) if bias is None else (np.asarray(bias, np.float64) / s_out64).astype(np.float32)
    return alpha, beta


def split_heads(codes, batch: int, tokens: int, heads: int, head_dim: int, col0: int):
    """[batch*tokens, *] code matrix -> [batch*heads, tokens, head_dim] slabs starting at column col0."""
    out = np.empty((batch * heads, tokens, head_dim), dtype=np.int16)
    for b in range(batch):
        for h in range(heads):
            out[b * heads + h] = codes[b * tokens:(b + 1) * tokens, col0 + h * head_dim: col0 + (h + 1) * head_dim]
    return out


def merge_heads(slabs, batch: int, tokens: int, heads: int, head_dim: int):
    out = np.empty((batch * tokens, heads * head_dim), dtype=slabs.dtype)
    for b in range(batch):
        for h in range(heads):
            out[b * tokens:(b + 1) * tokens, h * head_dim:(h + 1) * head_dim] = slabs[b * heads + h]
    return out


def attention_block(x_codes, s_x, prm: dict, batch: int, tokens: int, heads: int, bits: int, head_dim: int = 64,
                    proj: str = "dequant", residual=None, wq: dict | None = None, softmax: str = "exp") -> dict:
    """Integerized self-attention: QKV linear -> Q K^T -> softmax -> quantize -> P V -> proj.

    proj: "dequant" (fp32 output, optional residual) or "requant" (codes at step prm["s_out"]).
    wq: optional pre-quantized weight codes {"w_qkv", "w_proj"}.
    softmax: "exp" (Eq. 3, fp32 island: codes come with a band) or "shift" (Eq. 4 with the division-free
    comparator quantizer: integer and single-rounding operations only, so the codes are unique).
    """
    D = heads * head_dim
    st: dict = {}
    wq = wq or {}
    w_qkv = wq.get("w_qkv")
    if w_qkv is None:
        w_qkv = vo.quantize(prm["w_qkv"], 0.0, bits, True, row_steps=prm["s_w_qkv"])
    w_proj = wq.get("w_proj")
    if w_proj is None:
        w_proj = vo.quantize(prm["w_proj"], 0.0, bits, True, row_steps=prm["s_w_proj"])
    st["w_qkv_codes"], st["w_proj_codes"] = w_qkv, w_proj

    # QKV linear, requantized to three per-tensor steps (one per segment of the output channels)
    s_seg = np.concatenate([np.full(D, prm["s_q"]), np.full(D, prm["s_k"]), np.full(D, prm["s_v"])]).astype(np.float32)
    a_qkv, b_qkv = fold(s_x, prm["s_w_qkv"], prm["b_qkv"], s_seg)
    st["alpha_qkv"], st["beta_qkv"] = a_qkv, b_qkv
    st["acc_qkv"] = vo.matmul_i32(x_codes, w_qkv)
    st["qkv_codes"] = vo.epilogue_requant(st["acc_qkv"], a_qkv, b_qkv, bits, True)

    q = split_heads(st["qkv_codes"], batch, tokens, heads, head_dim, 0)
    k = split_heads(st["qkv_codes"], batch, tokens, heads, head_dim, D)
    v = split_heads(st["qkv_codes"], batch, tokens, heads, head_dim, 2 * D)
    st["S"] = vo.qk(q, k)
    c = softmax_scale(prm["s_q"], prm["s_k"], head_dim)
    st["c"] = c
    n = batch * heads
    if softmax == "shift":
        c2 = np.float32(np.float64(c) * np.log2(np.e))               # exponent of two: z = S * c * log2(e)
        st["c2"] = c2
        pc = vo.softmax_shift_quantize(st["S"].reshape(n * tokens, tokens), c2, prm["s_p"], bits)
        st["p_codes"] = pc.reshape(n, tokens, tokens)
        st["p_lo"] = st["p_hi"] = st["p_codes"]
    else:
        p, pc, plo, phi = vo.softmax_quantize(st["S"].reshape(n * tokens, tokens), c, prm["s_p"], bits)
        st["p"], st["p_codes"] = p.reshape(n, tokens, tokens), pc.reshape(n, tokens, tokens)
        st["p_lo"], st["p_hi"] = plo.reshape(n, tokens, tokens), phi.reshape(n, tokens, tokens)

    st["acc_o"] = vo.pv(st["p_codes"], v)
    a_o, b_o = fold(prm["s_p"], np.full(head_dim, prm["s_v"], np.float32), None, prm["s_o"])
    st["alpha_o"] = a_o
    o_slabs = vo.epilogue_requant(st["acc_o"].reshape(n * tokens, head_dim), a_o, b_o, bits, True)
    st["o_codes"] = merge_heads(o_slabs.reshape(n, tokens, head_dim), batch, tokens, heads, head_dim)

    st["acc_proj"] = vo.matmul_i32(st["o_codes"], w_proj)
    if proj == "dequant":
        st["out"] = vo.epilogue_dequant(st["acc_proj"], prm["s_o"], prm["s_w_proj"], prm["b_proj"], residual)
    else:
        a_p, b_p = fold(prm["s_o"], prm["s_w_proj"], prm["b_proj"], prm["s_out"])
        st["alpha_proj"], st["beta_proj"] = a_p, b_p
        st["out_codes"] = vo.epilogue_requant(st["acc_proj"], a_p, b_p, bits, True)
    return st


def normed_attention(x_codes, s_x, prm: dict, qkn: dict, batch: int, tokens: int, heads: int, bits: int,
                     head_dim: int = 64, eps: float = 1e-6) -> dict:
    """The self-attention module as the paper's power table lays it out (Section V-B): separate Q, K and V linear
    layers; Q and K pass a LayerNorm over each head's channels whose quantizer is the comparator of Fig. 5(b)
    (statistics by Eq. 5); V is requantized directly; Q K^T; the Eq. 4 softmax with its division-free
    quantizer; P V, requantized.  No level is decided after a floating-point island, so every stage is unique."""
    D = heads * head_dim
    M = batch * tokens
    st: dict = {}
    w = vo.quantize(prm["w_qkv"], 0.0, bits, True, row_steps=prm["s_w_qkv"])
    st["w_qkv_codes"] = w
    for i, name in enumerate(("q", "k")):
        sl = slice(i * D, (i + 1) * D)
        acc = vo.matmul_i32(x_codes, w[sl])
        y = vo.epilogue_dequant(acc, s_x, prm["s_w_qkv"][sl], prm["b_qkv"][sl])
        st[name + "_f32"] = y
        ref, neg, flip = vo.layernorm_references(qkn[name + "n_g"], qkn[name + "n_b"], qkn["s_" + name + "n"], bits,
                                                 True, head_dim)
        st[name + "_refs"] = (ref, neg, flip)
        codes, mu, v = vo.layernorm_compare_quantize(y.reshape(M * heads, head_dim), ref, neg, flip, eps, bits, True,
                                                     want_stats=True)
        st[name + "_codes"] = codes.reshape(M, D)
        st[name + "_stats"] = np.stack([mu, v], axis=1)
    sl = slice(2 * D, 3 * D)
    a_v, b_v = fold(s_x, prm["s_w_qkv"][sl], prm["b_qkv"][sl], prm["s_v"])
    st["alpha_v"], st["beta_v"] = a_v, b_v
    st["v_codes"] = vo.epilogue_requant(vo.matmul_i32(x_codes, w[sl]), a_v, b_v, bits, True)
    q = split_heads(st["q_codes"], batch, tokens, heads, head_dim, 0)
    k = split_heads(st["k_codes"], batch, tokens, heads, head_dim, 0)
    v = split_heads(st["v_codes"], batch, tokens, heads, head_dim, 0)
    st["S"] = vo.qk(q, k)
    c = softmax_scale(qkn["s_qn"], qkn["s_kn"], head_dim)
    c2 = np.float32(np.float64(c) * np.log2(np.e))
    st["c"], st["c2"] = c, c2
    n = batch * heads
    st["p_codes"] = vo.softmax_shift_quantize(st["S"].reshape(n * tokens, tokens), c2, prm["s_p"], bits).reshape(
        n, tokens, tokens)
    st["acc_o"] = vo.pv(st["p_codes"], v)
    a_o, b_o = fold(prm["s_p"], np.full(head_dim, prm["s_v"], np.float32), None, prm["s_o"])
    st["alpha_o"] = a_o
    o_slabs = vo.epilogue_requant(st["acc_o"].reshape(n * tokens, head_dim), a_o, b_o, bits, True)
    st["o_codes"] = merge_heads(o_slabs.reshape(n, tokens, head_dim), batch, tokens, heads, head_dim)
    return st


def encoder_layer(x, prm: dict, batch: int, tokens: int, heads: int, bits: int, head_dim: int = 64,
                  eps: float = 1e-6, softmax: str = "exp", layernorm: str = "fp32", gelu_tol_rel: float = 0.0) -> dict:
    """LN1 -> quantize -> attention (+residual) -> LN2 -> quantize -> fc1 -> GELU -> quantize -> fc2 (+residual).
    layernorm="compare": both LayerNorm + quantize stages run as Eq. 5 statistics with the comparator quantizer of
    Fig. 5(b); their levels are then unique (the band collapses to the code itself)."""
    st: dict = {}

    def ln_quant(v, g, b, tag):
        if layernorm == "compare":
            ref, neg, flip = vo.layernorm_references(prm[g], prm[b], prm["s_ln"], bits, True, v.shape[1])
            q = vo.layernorm_compare_quantize(v, ref, neg, flip, eps, bits, True)
            return q, q, q
        y, tol = vo.layernorm(v, prm[g], prm[b], eps)
        st[tag], st[tag + "_tol"] = y, tol
        return vo.quantize_band(y, tol, prm["s_ln"], bits, True)

    st["x1_codes"], st["x1_lo"], st["x1_hi"] = ln_quant(x, "ln1_g", "ln1_b", "ln1")
    att = attention_block(st["x1_codes"], prm["s_ln"], prm, batch, tokens, heads, bits, head_dim, "dequant", x,
                          softmax=softmax)
    st["attn"] = att
    h = att["out"]
    st["h"] = h
    st["x2_codes"], st["x2_lo"], st["x2_hi"] = ln_quant(h, "ln2_g", "ln2_b", "ln2")
    w_fc1 = vo.quantize(prm["w_fc1"], 0.0, bits, True, row_steps=prm["s_w_fc1"])
    w_fc2 = vo.quantize(prm["w_fc2"], 0.0, bits, True, row_steps=prm["s_w_fc2"])
    st["w_fc1_codes"], st["w_fc2_codes"] = w_fc1, w_fc2
    st["acc_fc1"] = vo.matmul_i32(st["x2_codes"], w_fc1)
    inv_g = inv_step(np.full(w_fc1.shape[0], prm["s_g"], np.float32))
    st["inv_s_g"] = inv_g
    st["g_codes"], st["g_lo"], st["g_hi"] = vo.epilogue_gelu_requant(st["acc_fc1"], prm["s_ln"], prm["s_w_fc1"],
                                                                     prm["b_fc1"], inv_g, bits, False,
                                                                     tol_rel=gelu_tol_rel)
    st["acc_fc2"] = vo.matmul_i32(st["g_codes"], w_fc2)
    st["out"] = vo.epilogue_dequant(st["acc_fc2"], prm["s_g"], prm["s_w_fc2"], prm["b_fc2"], h)
    return st


def encoder_stack(x, layer_params: list, batch: int, tokens: int, heads: int, bits: int) -> list:
    """Encoder layers in sequence; returns the list of per-layer stage dicts (the last one's "out" is the result)."""
    stages = []
    cur = x
    for prm in layer_params:
        st = encoder_layer(cur, prm, batch, tokens, heads, bits)
        stages.append(st)
        cur = st["out"]
    return stages


def deit_forward(patches, ends: dict, layer_params: list, batch: int, tokens: int, heads: int, bits: int,
                 eps: float = 1e-6, **layer_modes) -> dict:
    """Whole model: patch embedding as an integerized linear over flattened patches (class / distillation rows are
    zero) plus the token table, the encoder layers, final LayerNorm + quantizer on the class and distillation
    rows, two integerized classifier heads whose logits are summed."""
    st: dict = {}
    xq = vo.quantize(patches, ends["s_patch"], bits, True)
    w_pe = vo.quantize(ends["w_pe"], 0.0, bits, True, row_steps=ends["s_w_pe"])
    table = np.tile(np.asarray(ends["tokens"], np.float32), (batch, 1))
    st["x0"] = vo.epilogue_dequant(vo.matmul_i32(xq, w_pe), ends["s_patch"], ends["s_w_pe"], ends["b_pe"], table)
    cur = st["x0"]
    st["layers"] = []
    for prm in layer_params:
        ls = encoder_layer(cur, prm, batch, tokens, heads, bits, eps=eps, **layer_modes)
        st["layers"].append(ls)
        cur = ls["out"]
    st["x_final"] = cur
    logits = None
    for name, row in (("head", 0), ("head_dist", 1)):
        rows = np.ascontiguousarray(cur[row::tokens])
        y, tol = vo.layernorm(rows, ends["lnf_g"], ends["lnf_b"], eps)
        q, lo, hi = vo.quantize_band(y, tol, ends["s_lnf"], bits, True)
        st[name + "_codes"], st[name + "_lo"], st[name + "_hi"] = q, lo, hi
        w = vo.quantize(ends["w_" + name], 0.0, bits, True, row_steps=ends["s_w_" + name])
        logits = vo.epilogue_dequant(vo.matmul_i32(q, w), ends["s_lnf"], ends["s_w_" + name], ends["b_" + name], logits)
    st["logits"] = logits
    return st


def o_band_from_p_band(p_lo, p_hi, v, alpha_o, bits: int):
    """Codes of O = requant(P V) reachable when every P code may lie anywhere in [p_lo, p_hi] (Section IV-B's
    W_attn V followed by its absorbing quantizer).  The requantizer is monotone in the accumulator (alpha_o > 0),
    so the extremes are reached by taking, per term, the end of the P interval that the sign of V favours.
    p_lo, p_hi: [n, T, T]; v: [n, T, d] signed codes; returns (o_lo, o_hi) as [n*T, d] codes."""
    assert np.all(np.asarray(alpha_o) > 0)
    vp_, vn_ = np.maximum(v, 0).astype(np.int16), np.minimum(v, 0).astype(np.int16)
    n, T, d = v.shape
    acc_lo = vo.pv(p_lo, vp_) + vo.pv(p_hi, vn_)
    acc_hi = vo.pv(p_hi, vp_) + vo.pv(p_lo, vn_)
    zero = np.zeros_like(np.asarray(alpha_o, np.float32))
    o_lo = vo.epilogue_requant(acc_lo.reshape(n * T, d), alpha_o, zero, bits, True)
    o_hi = vo.epilogue_requant(acc_hi.reshape(n * T, d), alpha_o, zero, bits, True)
    return o_lo, o_hi


def encoder_layer_stagewise(x, prm: dict, batch: int, tokens: int, heads: int, bits: int, given: dict,
                            head_dim: int = 64, eps: float = 1e-6, softmax: str = "exp",
                            layernorm: str = "fp32") -> dict:
    """The stages of encoder_layer(), each computed from GIVEN upstream values instead of from this function's own
    previous stage: given["x1"], ["qkv"], ["O"], ["x2"], ["g"] are code matrices, given["h"] the fp32 residual
    stream after the attention block, given["P"] (optional, [batch*heads, T, T]) the attention codes.  A checker
    that has verified another implementation's stage k (exactly, or inside this oracle's band) passes that
    implementation's own stage-k values here and obtains what stage k+1 must be for THOSE inputs, so every
    element of every stage can be compared although a legitimate one-code difference upstream would otherwise
    cascade.  Returns, per stage, the oracle's result (and band where the stage decides a level after a
    floating-point island)."""
    D = heads * head_dim
    n = batch * heads
    st: dict = {}

    def ln_quant(v, g, b):
        if layernorm == "compare":
            ref, neg, flip = vo.layernorm_references(prm[g], prm[b], prm["s_ln"], bits, True, v.shape[1])
            q = vo.layernorm_compare_quantize(v, ref, neg, flip, eps, bits, True)
            return q, q, q
        y, tol = vo.layernorm(v, prm[g], prm[b], eps)
        return vo.quantize_band(y, tol, prm["s_ln"], bits, True)

    # LayerNorm 1 + quantizer, from x
    st["x1_codes"], st["x1_lo"], st["x1_hi"] = ln_quant(x, "ln1_g", "ln1_b")
    # QKV linear from the given LayerNorm codes
    w_qkv = vo.quantize(prm["w_qkv"], 0.0, bits, True, row_steps=prm["s_w_qkv"])
    s_seg = np.concatenate([np.full(D, prm["s_q"]), np.full(D, prm["s_k"]), np.full(D, prm["s_v"])]).astype(np.float32)
    a_qkv, b_qkv = fold(prm["s_ln"], prm["s_w_qkv"], prm["b_qkv"], s_seg)
    st["qkv_codes"] = vo.epilogue_requant(vo.matmul_i32(given["x1"], w_qkv), a_qkv, b_qkv, bits, True)
    # scores and attention codes from the given QKV codes
    q = split_heads(given["qkv"], batch, tokens, heads, head_dim, 0)
    k = split_heads(given["qkv"], batch, tokens, heads, head_dim, D)
    v = split_heads(given["qkv"], batch, tokens, heads, head_dim, 2 * D)
    S = vo.qk(q, k)
    c = softmax_scale(prm["s_q"], prm["s_k"], head_dim)
    if softmax == "shift":
        c2 = np.float32(np.float64(c) * np.log2(np.e))
        pc = vo.softmax_shift_quantize(S.reshape(n * tokens, tokens), c2, prm["s_p"], bits).reshape(n, tokens, tokens)
        st["p_codes"] = st["p_lo"] = st["p_hi"] = pc
    else:
        _, pc, plo, phi = vo.softmax_quantize(S.reshape(n * tokens, tokens), c, prm["s_p"], bits)
        st["p_codes"], st["p_lo"], st["p_hi"] = (a.reshape(n, tokens, tokens) for a in (pc, plo, phi))
    # O = requant(P V): exact from the given P codes, else the interval reachable inside the P band
    a_o, b_o = fold(prm["s_p"], np.full(head_dim, prm["s_v"], np.float32), None, prm["s_o"])
    if given.get("P") is not None:
        o = vo.epilogue_requant(vo.pv(given["P"], v).reshape(n * tokens, head_dim), a_o, b_o, bits, True)
        o = merge_heads(o.reshape(n, tokens, head_dim), batch, tokens, heads, head_dim)
        st["o_codes"] = st["o_lo"] = st["o_hi"] = o
    else:
        o = vo.epilogue_requant(vo.pv(st["p_codes"], v).reshape(n * tokens, head_dim), a_o, b_o, bits, True)
        lo, hi = o_band_from_p_band(st["p_lo"], st["p_hi"], v, a_o, bits)
        st["o_codes"], st["o_lo"], st["o_hi"] = (merge_heads(a.reshape(n, tokens, head_dim), batch, tokens, heads, head_dim)
                                                 for a in (o, lo, hi))
    # projection + residual from the given O codes
    w_proj = vo.quantize(prm["w_proj"], 0.0, bits, True, row_steps=prm["s_w_proj"])
    st["h"] = vo.epilogue_dequant(vo.matmul_i32(given["O"], w_proj), prm["s_o"], prm["s_w_proj"], prm["b_proj"], x)
    # LayerNorm 2 + quantizer from the given residual stream
    st["x2_codes"], st["x2_lo"], st["x2_hi"] = ln_quant(given["h"], "ln2_g", "ln2_b")
    # fc1 + GELU + quantizer from the given LayerNorm codes
    w_fc1 = vo.quantize(prm["w_fc1"], 0.0, bits, True, row_steps=prm["s_w_fc1"])
    w_fc2 = vo.quantize(prm["w_fc2"], 0.0, bits, True, row_steps=prm["s_w_fc2"])
    inv_g = inv_step(np.full(w_fc1.shape[0], prm["s_g"], np.float32))
    st["g_codes"], st["g_lo"], st["g_hi"] = vo.epilogue_gelu_requant(
        vo.matmul_i32(given["x2"], w_fc1), prm["s_ln"], prm["s_w_fc1"], prm["b_fc1"], inv_g, bits, False,
        tol_rel=given.get("gelu_tol_rel", 0.0))
    # fc2 + residual from the given GELU codes and residual stream
    st["out"] = vo.epilogue_dequant(vo.matmul_i32(given["g"], w_fc2), prm["s_g"], prm["s_w_fc2"], prm["b_fc2"],
                                    given["h"])
    return st
