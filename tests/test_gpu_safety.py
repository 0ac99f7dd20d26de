"""Memory-safety and failure-path checks on the GPU that need no fault: guard bands around every output buffer
(the stand-in for a memory checker), the bounded device-side wait, and non-finite quantizer inputs."""
import math

import numpy as np
import pytest
import torch

import oracle as vo
import synth_inputs as si
from oracle import pipeline as vp

pytestmark = pytest.mark.gpu
vt = pytest.importorskip("paper_2504_18547_b200")
from gpu_util import (check_guards, dev, from_codes, guarded_codes, guarded_tensor, padding_is_zero, rand_codes,  # noqa: E402
                      to_codes)


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    """A wait that nothing completes runs into its limit (about a millisecond here): the kernel returns, the
    device status word reports the timeout once, and ordinary calls work afterwards."""
    assert vt.vitint_device_status() == 0
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    vt.vitint_selftest_wait_timeout(2_000_000, flag)
    torch.cuda.synchronize()
    assert int(flag.item()) == 1
    assert vt.vitint_device_status() == -7                      # VITINT_ERR_TIMEOUT, reported ...
    assert vt.vitint_device_status() == 0                       # ... and cleared
    x = si.normal(5, (70, 96))
    got = vt.vitint_quantize(dev(x), 0.25, 4, True)
    assert np.array_equal(from_codes(got), vo.quantize(x, np.float32(0.25), 4, True))
    assert vt.vitint_device_status() == 0
    with pytest.raises(vt.VitintError):
        vt.vitint_selftest_wait_timeout(0)


def test_quantizer_non_finite_inputs_and_extreme_steps():
    """+-inf, NaN, +-FLT_MAX and steps at the ends of the fp32 range follow the definition q = clamp(rint(x / s))
    with one IEEE division, as the oracle computes it."""
    big = np.float32(3.4028235e38)
    x = np.array([[np.inf, -np.inf, np.nan, big, -big, 0.0, 1.0, -1.0, 1e-30, -1e-30, 2.5, -2.5, 7.49, 1e20, -1e20, 0.1]],
                 np.float32)
    for step in (0.25, 1e-30, 1e30, 3e38, 1.2e-38, 1e-41, 1.9999999):
        for bits, signed in ((4, True), (4, False), (2, True), (8, True)):
            s = np.float32(step)
            got = vt.vitint_quantize(dev(x), float(s), bits, signed)
            want = vo.quantize(x, s, bits, signed)
            assert np.array_equal(from_codes(got), want), (step, bits, signed)


def test_outputs_stay_inside_their_buffers():
    """Every entry point writes only what it was given: outputs sit between patterned 4 KB margins, shapes are
    ragged in every direction (1 row, 197 tokens, widths that end inside a vector store, odd pitches)."""
    # a1, widen
    for rows, cols in ((1, 1), (197, 197), (130, 333)):
        x = si.normal(3 + rows, (rows, cols))
        for bits, cont in ((4, 0), (2, 0), (3, 0), (8, 0), (4, 8)):
            out = guarded_codes(rows, cols, bits, True, cont)
            vt.vitint_quantize(dev(x), 0.3, bits, True, out=out)
            assert np.array_equal(from_codes(out), vo.quantize(x, np.float32(0.3), bits, True)) and padding_is_zero(out)
        q = rand_codes(9, (rows, cols), 4, True)
        w8 = guarded_codes(rows, cols, 4, True, 8)
        vt.vitint_widen(to_codes(q, 4, True), out=w8)
        assert np.array_equal(from_codes(w8), q)
    # a2 + a3 in its three forms, packed and byte-stored operands
    for M, K, N in ((1, 64, 16), (197, 192, 200), (300, 320, 264), (129, 1000, 257)):
        qx, qw = rand_codes(11, (M, K), 4, True), rand_codes(12, (N, K), 4, True)
        acc_ref = vo.matmul_i32(qx, qw)
        for wide in (False, True):
            x, w = to_codes(qx, 4, True), to_codes(qw, 4, True)
            if wide:
                x, w = vt.vitint_widen(x), vt.vitint_widen(w)
            acc = guarded_tensor((M, N), torch.int32)
            vt.vitint_linear(x, 1.0, w, None, None, vt.Epilogue(mode=vt.EPI_ACC_I32), out=acc)
            assert np.array_equal(acc.cpu().numpy(), acc_ref)
            s_w = np.full(N, 0.01, np.float32)
            y = guarded_tensor((M, N), torch.float32)
            res = si.normal(13, (M, N))
            vt.vitint_linear(x, 0.5, w, dev(s_w), None, vt.Epilogue(mode=vt.EPI_DEQUANT_F32, residual=dev(res)), out=y)
            assert np.array_equal(y.cpu().numpy().view(np.uint32), vo.epilogue_dequant(acc_ref, np.float32(0.5), s_w, None, res).view(np.uint32))
            alpha, beta = np.full(N, 0.02, np.float32), si.normal(14, (N,), 0.0, 0.5)
            for ob, oc in ((4, 0), (4, 8), (2, 0), (8, 0)):
                qo = guarded_codes(M, N, ob, True, oc)
                vt.vitint_linear(x, 1.0, w, None, None, vt.Epilogue(mode=vt.EPI_REQUANT, alpha=dev(alpha), beta=dev(beta), out_bits=ob,
                                                                   out_signed=True, out_container=oc), out=qo)
                assert np.array_equal(from_codes(qo), vo.epilogue_requant(acc_ref, alpha, beta, ob, True)) and padding_is_zero(qo)
            inv_s = np.full(N, 1.0 / 0.05, np.float32)
            qg = guarded_codes(M, N, 4, False, 8 if wide else 0)
            vt.vitint_linear(x, 0.5, w, dev(s_w), None, vt.Epilogue(mode=vt.EPI_REQUANT, act=1, inv_out_step=dev(inv_s), out_bits=4,
                                                                   out_signed=False, out_container=8 if wide else 0), out=qg)
            assert padding_is_zero(qg)
    # a4, a5, a6 and the fused core
    for batch, tokens, heads in ((1, 197, 2), (2, 50, 1), (1, 129, 1)):
        D = heads * 64
        qkv = rand_codes(21 + tokens, (batch * tokens, 3 * D), 4, True)
        c = to_codes(qkv, 4, True)
        ld_s = (tokens + 3) // 4 * 4
        S = guarded_tensor((batch * heads, tokens, ld_s), torch.int32)
        vt.vitint_qk(vt.Slabs.of_qkv(c, tokens, D, 0), vt.Slabs.of_qkv(c, tokens, D, 1), batch, heads, tokens, out=S, ld_s=ld_s)
        n = batch * heads
        for bits in (4, 2):
            P = guarded_codes(n * tokens, tokens, bits, False)
            vt.vitint_softmax_quantize(S.view(n * tokens, ld_s), tokens, 0.004, 2.0 / (tokens * 3.8), bits, out=P)
            assert padding_is_zero(P)
            P2 = guarded_codes(n * tokens, tokens, bits, False)
            vt.vitint_softmax_shift_quantize(S.view(n * tokens, ld_s), tokens, 0.006, 2.0 / (tokens * 3.8), bits, out=P2)
            assert padding_is_zero(P2)
        P4 = guarded_codes(n * tokens, tokens, 4, False)
        vt.vitint_softmax_quantize(S.view(n * tokens, ld_s), tokens, 0.004, 2.0 / (tokens * 3.8), 4, out=P4)
        O = guarded_tensor((batch * tokens, D), torch.int32)
        vt.vitint_pv(P4, vt.Slabs.of_qkv(c, tokens, D, 2), batch, heads, tokens, 1.0, 1.0, vt.Epilogue(mode=vt.EPI_ACC_I32), out=O)
        alpha = dev(np.full(D, 0.01, np.float32))
        for wide in (False, True):
            for ob, oc, pitch in ((4, 0, None), (4, 8, None), (4, 0, D // 2 + 32), (2, 0, None)):
                oo = guarded_codes(batch * tokens, D, ob, True, oc, pitch)
                vt.vitint_attention_core(vt.vitint_widen(c) if wide else c, batch, heads, tokens, 0.2, 0.2, 2.0 / (tokens * 3.8), 4,
                                         alpha, None, out=oo)
                assert padding_is_zero(oo)
                if wide:
                    # the Eq. 4 variant of the core, same buffers
                    o4 = guarded_codes(batch * tokens, D, ob, True, oc, pitch)
                    vt.vitint_attention_core_shift(vt.vitint_widen(c), batch, heads, tokens, 0.2, 0.2, 2.0 / (tokens * 3.8), 4,
                                                   alpha, None, out=o4)
                    assert padding_is_zero(o4)
    # the chunked core beyond 256 tokens (byte-stored codes): ragged last chunk and last query tile
    for batch, tokens, heads in ((1, 300, 2), (2, 257, 1), (1, 577, 1)):
        D = heads * 64
        c8 = vt.vitint_widen(to_codes(rand_codes(51 + tokens, (batch * tokens, 3 * D), 4, True), 4, True))
        alpha = dev(np.full(D, 0.01, np.float32))
        for ob, oc, pitch in ((4, 0, None), (4, 8, None), (4, 0, D // 2 + 32), (2, 0, None)):
            oo = guarded_codes(batch * tokens, D, ob, True, oc, pitch)
            vt.vitint_attention_core(c8, batch, heads, tokens, 0.2, 0.2, 2.0 / (tokens * 3.8), 4, alpha, None, out=oo)
            assert padding_is_zero(oo)
    # glue
    for rows, cols in ((1, 4), (197, 192), (37, 100)):
        x = si.normal(31 + cols, (rows, cols), 0.5, 1.5)
        g, b = si.normal(32, (cols,), 1.0, 0.1), si.normal(33, (cols,), 0.0, 0.1)
        for bits, cont in ((4, 0), (4, 8), (2, 0)):
            out = guarded_codes(rows, cols, bits, True, cont)
            vt.vitint_layernorm_quantize(dev(x), dev(g), dev(b), 1e-6, 0.4, bits, True, out=out)
            assert padding_is_zero(out)
            refs, flip = vt.vitint_fold_layernorm_references(g, b, np.float32(0.4), bits, True, cols)
            out2, stats = guarded_codes(rows, cols, bits, True, cont), guarded_tensor((rows, 2), torch.float32)
            vt.vitint_layernorm_compare_quantize(dev(x), dev(refs), dev(flip), 1e-4, bits, True, out=out2, stats=stats)
            assert padding_is_zero(out2)
    # QKV projection with the per-head LayerNorm in its epilogue: one head (a 192-column tile) and three heads
    # (three 256-column tiles, the last ragged), odd row counts, packed and byte containers, over-wide pitch
    for M, K, heads in ((1, 64, 1), (197, 128, 1), (131, 192, 3)):
        D = 64 * heads
        qx, qw = rand_codes(41 + M, (M, K), 4, True), rand_codes(42, (3 * D, K), 4, True)
        s_w, bias = np.full(3 * D, 0.01, np.float32), si.normal(43, (3 * D,), 0.0, 0.05)
        g, b = si.normal(44, (64,), 1.0, 0.1), si.normal(45, (64,), 0.0, 0.1)
        g[::5] *= -1.0
        alpha_v, beta_v = np.full(D, 0.02, np.float32), si.normal(46, (D,), 0.0, 0.5)
        for bits, cont, pitch in ((4, 0, None), (4, 8, None), (3, 0, 3 * D // 2 + 48), (2, 0, None)):
            ref, neg, flip = vo.layernorm_references(g, b, np.float32(0.4), bits, True, 64)
            refs, fl = vt.vitint_fold_layernorm_references(g, b, np.float32(0.4), bits, True, 64)
            want = []
            for i in range(2):
                y = vo.epilogue_dequant(vo.matmul_i32(qx, qw[i * D:(i + 1) * D]), np.float32(0.5), s_w[i * D:(i + 1) * D], bias[i * D:(i + 1) * D])
                want.append(vo.layernorm_compare_quantize(y.reshape(M * heads, 64), ref, neg, flip, 1e-6, bits, True).reshape(M, D))
            want.append(vo.epilogue_requant(vo.matmul_i32(qx, qw[2 * D:]), alpha_v, beta_v, bits, True))
            out = guarded_codes(M, 3 * D, bits, True, cont, pitch)
            stats = guarded_tensor((2, M * heads, 2), torch.float32)
            n_eps = float(np.float32(np.float64(64) * np.float64(np.float32(1e-6))))
            vt.vitint_linear_qkv_norm(vt.vitint_widen(to_codes(qx, 4, True)), 0.5, vt.vitint_widen(to_codes(qw, 4, True)), dev(s_w),
                                      dev(bias), torch.stack([dev(refs)] * 2).contiguous(), torch.stack([dev(fl)] * 2).contiguous(),
                                      n_eps, dev(alpha_v), dev(beta_v), bits, out=out, stats=stats)
            assert np.array_equal(from_codes(out), np.concatenate(want, axis=1)) and padding_is_zero(out)
    torch.cuda.synchronize()
    assert vt.vitint_device_status() == 0
    assert check_guards() > 100


def test_attention_block_outputs_and_copies_stay_inside_their_buffers():
    """The composed block with every optional copy requested, fused and unfused, the copies' pitches larger than
    the block's own (their padding must come back as zero)."""
    cfg = si.VIT_TINY_BLOCK
    prm = si.layer_parameters(cfg)
    x = si.activations(cfg)
    s_x = si.lsq_step(x, cfg.bits, True)
    xq = vo.quantize(x, s_x, cfg.bits, True)
    st = vp.attention_block(xq, s_x, prm, cfg.batch, cfg.tokens, cfg.heads, cfg.bits, proj="dequant")
    M, D, T, H = cfg.rows, cfg.dim, cfg.tokens, cfg.heads
    aw = vt.AttentionWeights(
        batch=cfg.batch, tokens=T, heads=H, bits=cfg.bits, w_qkv=to_codes(st["w_qkv_codes"], cfg.bits, True),
        alpha_qkv=dev(st["alpha_qkv"]), beta_qkv=dev(st["beta_qkv"]), q_step=float(prm["s_q"]), k_step=float(prm["s_k"]),
        v_step=float(prm["s_v"]), p_step=float(prm["s_p"]), o_step=float(prm["s_o"]), p_bits=cfg.bits,
        alpha_o=dev(np.tile(st["alpha_o"], H)), beta_o=None, w_proj=to_codes(st["w_proj_codes"], cfg.bits, True),
        w_proj_step=dev(prm["s_w_proj"]), b_proj=dev(prm["b_proj"]), proj_epi=vt.Epilogue(mode=vt.EPI_DEQUANT_F32))
    for want_p in (False, True):
        dq = guarded_codes(M, 3 * D, cfg.bits, True, pitch=vt.packed_pitch(3 * D, cfg.bits) + 48)
        do = guarded_codes(M, D, cfg.bits, True, pitch=vt.packed_pitch(D, cfg.bits) + 16)
        dp = guarded_codes(cfg.batch * H * T, T, cfg.bits, False, pitch=vt.packed_pitch(T, cfg.bits) + 32) if want_p else None
        out = guarded_tensor((M, D), torch.float32)
        ws = guarded_tensor((vt.vitint_attention_block_workspace_bytes(aw),), torch.uint8)
        vt.vitint_attention_block(to_codes(xq, cfg.bits, True), aw, out=out, workspace=ws, dbg_qkv=dq, dbg_p=dp, dbg_o=do)
        assert np.array_equal(from_codes(dq), st["qkv_codes"]) and padding_is_zero(dq) and padding_is_zero(do)
        if want_p:
            assert padding_is_zero(dp)
    torch.cuda.synchronize()
    assert vt.vitint_device_status() == 0
    assert check_guards() == 9
