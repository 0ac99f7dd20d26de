"""GPU parity: every C-ABI entry point against the CPU oracle on the same seeded inputs.

Bar: bit-exact for int32 accumulators, a1 codes and requantized codes; bit-exact fp32 for
the dequantizing epilogue (both sides run the same IEEE operation sequence); <= 2 ulp for
softmax probabilities, with codes inside the oracle's band of codes reachable within that
tolerance; GELU within 2^-21*|y|; LayerNorm within the oracle's per-element tolerance.
"""
import math

import numpy as np
import pytest
import torch

import oracle as vo
import synth_inputs as si
from oracle import pipeline as vp

pytestmark = pytest.mark.gpu

vt = pytest.importorskip("paper_2504_18547_b200")
from gpu_util import GELU_TOL_REL, check_guards, dev, from_codes, guarded_codes, padding_is_zero, rand_codes, to_codes, ulp_diff  # noqa: E402


@pytest.fixture(autouse=True)
def _device_status_clean():
    yield
    assert vt.vitint_device_status() == 0, "a device-side wait timed out"


# ---------------------------------------------------------------------------
# a1
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("bits,signed", [(2, True), (3, True), (4, True), (8, True), (2, False), (4, False), (8, False)])
@pytest.mark.parametrize("rows,cols", [(197, 192), (3, 1), (130, 333), (64, 3072)])
def test_quantize_matches_oracle(bits, signed, rows, cols):
    x = si.normal(100 + bits + rows, (rows, cols), 0.1, 1.3)
    step = si.lsq_step(x, bits, signed)
    got = vt.vitint_quantize(dev(x), float(step), bits, signed)
    assert np.array_equal(from_codes(got), vo.quantize(x, step, bits, signed))
    assert np.array_equal(got.data.cpu().numpy(), vo.pack(vo.quantize(x, step, bits, signed), bits))
    assert padding_is_zero(got)


def test_quantize_row_steps_strided_input_and_ties():
    rows, cols = 70, 200
    w = si.normal(7, (rows, cols + 8), 0.0, 0.02)
    steps = si.lsq_step_rows(w[:, :cols], 4)
    xw = dev(w)[:, :cols]                      # ldx = cols + 8, rows not 16-byte aligned views
    got = vt.vitint_quantize(xw, 0.0, 4, True, row_steps=dev(steps))
    assert np.array_equal(from_codes(got), vo.quantize(w[:, :cols], 0.0, 4, True, row_steps=steps))
    # exact ties and clamps
    ks = np.arange(-12, 12, dtype=np.float32)
    t = ((ks + 0.5) * 0.25).astype(np.float32)[None, :]
    got = vt.vitint_quantize(dev(t), 0.25, 4, True)
    assert np.array_equal(from_codes(got), vo.quantize(t, 0.25, 4, True))


@pytest.mark.parametrize("bits,signed", [(2, True), (3, True), (4, True), (2, False), (4, False)])
@pytest.mark.parametrize("rows,cols", [(70, 197), (5, 1), (300, 768)])
def test_widen_keeps_values(bits, signed, rows, cols):
    q = rand_codes(50 + bits, (rows, cols), bits, signed)
    got = vt.vitint_widen(to_codes(q, bits, signed))
    assert got.bits == bits and got.container == 8 and got.pitch >= cols
    assert np.array_equal(from_codes(got), q) and padding_is_zero(got)


# ---------------------------------------------------------------------------
# a2 + a3
# ---------------------------------------------------------------------------

LIN_SHAPES = [(197, 192, 576), (300, 320, 100), (128, 128, 256), (1, 64, 16), (515, 1000, 264), (260, 3072, 80)]


@pytest.mark.parametrize("M,K,N", LIN_SHAPES)
@pytest.mark.parametrize("bits,xs", [(4, True), (2, True), (3, True), (8, True), (4, False), (8, False), (2, False)])
def test_linear_accumulators_bit_exact(M, K, N, bits, xs):
    qx = rand_codes(1, (M, K), bits, xs)
    qw = rand_codes(2, (N, K), bits, True)
    acc = vt.vitint_linear(to_codes(qx, bits, xs), 1.0, to_codes(qw, bits, True), None, None,
                           vt.Epilogue(mode=vt.EPI_ACC_I32))
    assert np.array_equal(acc.cpu().numpy(), vo.matmul_i32(qx, qw))


def test_linear_extreme_codes_closed_form():
    # all-minimum x all-minimum at K = 4096: the largest magnitude the 4-bit path can produce
    M, K, N = 130, 4096, 48
    qx = np.full((M, K), -8, np.int16)
    qw = np.full((N, K), -8, np.int16)
    qw[1] = 7
    acc = vt.vitint_linear(to_codes(qx, 4, True), 1.0, to_codes(qw, 4, True), None, None,
                           vt.Epilogue(mode=vt.EPI_ACC_I32)).cpu().numpy()
    assert np.all(acc[:, 0] == 64 * K) and np.all(acc[:, 1] == -56 * K)


def test_linear_mixed_widths():
    M, K, N = 200, 256, 96
    qx = rand_codes(3, (M, K), 8, False)
    qw = rand_codes(4, (N, K), 4, True)
    acc = vt.vitint_linear(to_codes(qx, 8, False), 1.0, to_codes(qw, 4, True), None, None,
                           vt.Epilogue(mode=vt.EPI_ACC_I32))
    assert np.array_equal(acc.cpu().numpy(), vo.matmul_i32(qx, qw))


@pytest.mark.parametrize("M,K,N", [(197, 192, 576), (515, 1000, 264), (260, 3072, 768), (1000, 768, 2304)])
@pytest.mark.parametrize("bits,xs", [(4, True), (2, True), (3, True), (4, False)])
def test_linear_with_widened_weights(M, K, N, bits, xs):
    """Weights held in 8-bit containers (TMA-direct operand), activations packed low-bit."""
    qx = rand_codes(7, (M, K), bits, xs)
    qw = rand_codes(8, (N, K), bits, True)
    w8 = vt.vitint_widen(to_codes(qw, bits, True))
    acc = vt.vitint_linear(to_codes(qx, bits, xs), 1.0, w8, None, None, vt.Epilogue(mode=vt.EPI_ACC_I32))
    assert np.array_equal(acc.cpu().numpy(), vo.matmul_i32(qx, qw))


def test_byte_containers_for_low_bit_codes():
    """4-bit-range codes stored one per byte: produced by the quantizer and by a requantizing epilogue,
    consumed by the linear layer (both operands then go from the TMA copy straight to the tensor cores)."""
    M, K, N = 300, 320, 200
    x = si.normal(71, (M, K))
    step = si.lsq_step(x, 4, True)
    out = vt.Codes.empty(M, K, 4, True, container=8)
    got = vt.vitint_quantize(dev(x), float(step), 4, True, out=out)
    qx = vo.quantize(x, step, 4, True)
    assert np.array_equal(from_codes(got), qx) and padding_is_zero(got)
    qw = rand_codes(72, (N, K), 4, True)
    w8 = vt.vitint_widen(to_codes(qw, 4, True))
    acc = vo.matmul_i32(qx, qw)
    got_acc = vt.vitint_linear(got, 1.0, w8, None, None, vt.Epilogue(mode=vt.EPI_ACC_I32))
    assert np.array_equal(got_acc.cpu().numpy(), acc)
    alpha = np.full(N, 0.02, np.float32)
    beta = si.normal(73, (N,), 0.0, 0.5)
    epi = vt.Epilogue(mode=vt.EPI_REQUANT, alpha=dev(alpha), beta=dev(beta), out_bits=4, out_signed=True, out_container=8)
    q8 = vt.vitint_linear(got, 1.0, w8, None, None, epi)
    assert q8.container == 8 and q8.pitch >= N
    assert np.array_equal(from_codes(q8), vo.epilogue_requant(acc, alpha, beta, 4, True)) and padding_is_zero(q8)


BYTE_SHAPES = [(129, 64, 256), (256, 192, 512), (300, 768, 768), (1000, 1000, 1000), (515, 3072, 264), (2049, 384, 2304),
               (257, 1024, 128), (1000, 1008, 1000), (400, 16, 200), (5000, 768, 264)]


@pytest.mark.parametrize("M,K,N", BYTE_SHAPES)
@pytest.mark.parametrize("bits,xs", [(4, True), (8, True), (4, False), (2, True)])
def test_linear_byte_codes_both_operands_bit_exact(M, K, N, bits, xs):
    """Both operands stored one code per byte (the encoder's layout: the TMA copies are the tensor-core operands,
    nothing is unpacked).  Raw accumulators, a requantizing epilogue and the fp32 epilogue with residual, each
    against the oracle bit for bit; M, N and K include ragged last tiles in every direction."""
    qx = rand_codes(31 + M, (M, K), bits, xs)
    qw = rand_codes(32 + N, (N, K), bits, True)
    x8 = vt.vitint_widen(to_codes(qx, bits, xs)) if bits != 8 else to_codes(qx, bits, xs)
    w8 = vt.vitint_widen(to_codes(qw, bits, True)) if bits != 8 else to_codes(qw, bits, True)
    acc = vo.matmul_i32(qx, qw)
    got = vt.vitint_linear(x8, 1.0, w8, None, None, vt.Epilogue(mode=vt.EPI_ACC_I32))
    assert np.array_equal(got.cpu().numpy(), acc)
    if bits == 4 and xs:
        s_w = (np.abs(si.normal(33, (N,), 0.0, 0.01)) + 1e-3).astype(np.float32)
        bias = si.normal(34, (N,), 0.0, 0.05)
        alpha, beta = vp.fold(0.5, s_w, bias, 0.5 * 0.011 * 8 * math.sqrt(K) * 4 / 7)
        for cont in (0, 8):
            epi = vt.Epilogue(mode=vt.EPI_REQUANT, alpha=dev(alpha), beta=dev(beta), out_bits=4, out_signed=True,
                              out_container=cont)
            q = vt.vitint_linear(x8, 1.0, w8, None, None, epi)
            assert np.array_equal(from_codes(q), vo.epilogue_requant(acc, alpha, beta, 4, True)) and padding_is_zero(q)
        res = si.normal(35, (M, N))
        y = vt.vitint_linear(x8, 0.37, w8, dev(s_w), dev(bias), vt.Epilogue(mode=vt.EPI_DEQUANT_F32, residual=dev(res)))
        want = vo.epilogue_dequant(acc, np.float32(0.37), s_w, bias, res)
        assert np.array_equal(y.cpu().numpy().view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("M,K,N", [(197, 192, 576), (300, 320, 100)])
def test_linear_dequant_bias_residual_bit_exact(M, K, N):
    qx = rand_codes(5, (M, K), 4, True)
    qw = rand_codes(6, (N, K), 4, True)
    s_w = (np.abs(si.normal(8, (N,), 0.0, 0.01)) + 1e-3).astype(np.float32)
    bias = si.normal(9, (N,), 0.0, 0.01)
    res = si.normal(10, (M, N))
    acc = vo.matmul_i32(qx, qw)
    for b_, r_ in ((None, None), (bias, None), (bias, res)):
        epi = vt.Epilogue(mode=vt.EPI_DEQUANT_F32, residual=dev(r_))
        y = vt.vitint_linear(to_codes(qx, 4, True), 0.37, to_codes(qw, 4, True), dev(s_w), dev(b_), epi)
        want = vo.epilogue_dequant(acc, np.float32(0.37), s_w, b_, r_)
        assert np.array_equal(y.cpu().numpy().view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("out_bits,out_signed", [(4, True), (2, True), (3, True), (8, True), (4, False), (8, False)])
@pytest.mark.parametrize("M,K,N", [(197, 192, 576), (300, 320, 100), (140, 128, 33)])
def test_linear_requant_bit_exact(M, K, N, out_bits, out_signed):
    qx = rand_codes(11, (M, K), 4, True)
    qw = rand_codes(12, (N, K), 4, True)
    s_w = (np.abs(si.normal(13, (N,), 0.0, 0.01)) + 1e-3).astype(np.float32)
    bias = si.normal(14, (N,), 0.0, 0.05)
    qp = si.code_range(out_bits, out_signed)[1]
    s_out = np.float32(0.5 * 0.011 * 8 * math.sqrt(K) * 4 / qp)
    alpha, beta = vp.fold(0.5, s_w, bias, s_out)
    a2, b2 = vt.vitint_fold_requant(0.5, s_w, bias, s_out)
    assert np.array_equal(alpha, a2) and np.array_equal(beta, b2)
    epi = vt.Epilogue(mode=vt.EPI_REQUANT, alpha=dev(alpha), beta=dev(beta), out_bits=out_bits, out_signed=out_signed)
    got = vt.vitint_linear(to_codes(qx, 4, True), 1.0, to_codes(qw, 4, True), None, None, epi)
    want = vo.epilogue_requant(vo.matmul_i32(qx, qw), alpha, beta, out_bits, out_signed)
    assert np.array_equal(from_codes(got), want)
    assert padding_is_zero(got)
    assert len(np.unique(want)) >= min(4, qp)


def test_linear_gelu_dequant_and_requant():
    M, K, N = 197, 192, 320
    qx = rand_codes(15, (M, K), 4, True)
    qw = rand_codes(16, (N, K), 4, True)
    s_w = (np.abs(si.normal(17, (N,), 0.0, 0.004)) + 5e-4).astype(np.float32)
    bias = si.normal(18, (N,), 0.0, 0.05)
    acc = vo.matmul_i32(qx, qw)
    x, w = to_codes(qx, 4, True), to_codes(qw, 4, True)
    y = vt.vitint_linear(x, 0.6, w, dev(s_w), dev(bias), vt.Epilogue(mode=vt.EPI_DEQUANT_F32, act=1)).cpu().numpy()
    pre = vo.epilogue_dequant(acc, np.float32(0.6), s_w, bias)
    want = vo.epilogue_dequant(acc, np.float32(0.6), s_w, bias, None, act=1)
    assert np.all(np.abs(y.astype(np.float64) - want) <= GELU_TOL_REL * np.abs(pre) + 1e-30)
    inv_s = vp.inv_step(np.full(N, 0.04, np.float32))
    epi = vt.Epilogue(mode=vt.EPI_REQUANT, act=1, inv_out_step=dev(inv_s), out_bits=4, out_signed=False)
    got = from_codes(vt.vitint_linear(x, 0.6, w, dev(s_w), dev(bias), epi))
    q, lo, hi = vo.epilogue_gelu_requant(acc, np.float32(0.6), s_w, bias, inv_s, 4, False, tol_rel=GELU_TOL_REL)
    assert np.all(got >= lo) and np.all(got <= hi)
    assert (got != q).mean() < 1e-3 and len(np.unique(q)) == 16


# ---------------------------------------------------------------------------
# a4, a5, a6
# ---------------------------------------------------------------------------

def _qkv_codes(batch, tokens, heads, bits, seed):
    D = heads * 64
    return rand_codes(seed, (batch * tokens, 3 * D), bits, True)


@pytest.mark.parametrize("bits", [4, 2, 8])
@pytest.mark.parametrize("batch,tokens,heads", [(1, 197, 3), (3, 197, 2), (2, 50, 1), (1, 256, 2), (2, 577, 1), (1, 785, 2)])
def test_qk_bit_exact(batch, tokens, heads, bits):
    D = heads * 64
    qkv = _qkv_codes(batch, tokens, heads, bits, 21)
    c = to_codes(qkv, bits, True)
    S = vt.vitint_qk(vt.Slabs.of_qkv(c, tokens, D, 0), vt.Slabs.of_qkv(c, tokens, D, 1), batch, heads, tokens)
    want = vo.qk(vp.split_heads(qkv, batch, tokens, heads, 64, 0), vp.split_heads(qkv, batch, tokens, heads, 64, D))
    assert np.array_equal(S.cpu().numpy()[:, :, :tokens], want)


@pytest.mark.parametrize("bits", [4, 2, 8])
@pytest.mark.parametrize("batch,tokens,heads", [(1, 197, 3), (3, 197, 2), (2, 50, 1), (1, 256, 2), (2, 577, 1), (1, 785, 2)])
def test_pv_bit_exact(batch, tokens, heads, bits):
    D = heads * 64
    qkv = _qkv_codes(batch, tokens, heads, bits, 22)
    P = rand_codes(23, (batch * heads * tokens, tokens), bits, False)
    c = to_codes(qkv, bits, True)
    O = vt.vitint_pv(to_codes(P, bits, False), vt.Slabs.of_qkv(c, tokens, D, 2), batch, heads, tokens, 1.0, 1.0,
                     vt.Epilogue(mode=vt.EPI_ACC_I32))
    v = vp.split_heads(qkv, batch, tokens, heads, 64, 2 * D)
    want = vp.merge_heads(vo.pv(P.reshape(batch * heads, tokens, tokens), v), batch, tokens, heads, 64)
    assert np.array_equal(O.cpu().numpy(), want)


def test_pv_requant_and_dequant_epilogues():
    batch, tokens, heads, bits = 2, 197, 3, 4
    D = heads * 64
    qkv = _qkv_codes(batch, tokens, heads, bits, 24)
    P = rand_codes(25, (batch * heads * tokens, tokens), bits, False)
    c = to_codes(qkv, bits, True)
    v = vp.split_heads(qkv, batch, tokens, heads, 64, 2 * D)
    acc = vp.merge_heads(vo.pv(P.reshape(batch * heads, tokens, tokens), v), batch, tokens, heads, 64)
    s_p, s_v, s_o = np.float32(0.0026), np.float32(0.17), np.float32(0.31)
    alpha, beta = vp.fold(s_p, np.full(D, s_v, np.float32), None, s_o)
    epi = vt.Epilogue(mode=vt.EPI_REQUANT, alpha=dev(alpha), out_bits=4, out_signed=True)
    got = vt.vitint_pv(to_codes(P, bits, False), vt.Slabs.of_qkv(c, tokens, D, 2), batch, heads, tokens, s_p, s_v, epi)
    want = vo.epilogue_requant(acc, alpha, beta, 4, True)
    assert np.array_equal(from_codes(got), want) and len(np.unique(want)) >= 8
    y = vt.vitint_pv(to_codes(P, bits, False), vt.Slabs.of_qkv(c, tokens, D, 2), batch, heads, tokens, s_p, s_v,
                     vt.Epilogue(mode=vt.EPI_DEQUANT_F32))
    sc = np.float32(s_p * s_v)
    wanty = vo.epilogue_dequant(acc, sc, np.ones(D, np.float32), None)
    assert np.array_equal(y.cpu().numpy().view(np.uint32), wanty.view(np.uint32))


@pytest.mark.parametrize("bits", [4, 2, 3, 8])
@pytest.mark.parametrize("rows,cols,ld", [(591, 197, 200), (64, 197, 197), (33, 50, 52), (40, 577, 580), (24, 785, 785), (9, 1, 4)])
def test_softmax_quantize_within_two_ulp_and_band(rows, cols, ld, bits):
    S = np.zeros((rows, ld), np.int32)
    S[:, :cols] = (si.splitmix64(31 + cols, rows * cols) % np.uint64(1401)).astype(np.int64).reshape(rows, cols) - 700
    S[0, :cols] = 5                                     # uniform row
    if cols > 3:
        S[1, :cols] = -700
        S[1, 2] = 700                                   # one dominant entry, the rest underflow
    c = np.float32(0.0211)
    s_p = np.float32(2.0 / (cols * math.sqrt(si.code_range(bits, False)[1])))
    got, p = vt.vitint_softmax_quantize(dev(S), cols, c, s_p, bits, want_p=True)
    p_ref, q, lo, hi = vo.softmax_quantize(S[:, :cols], c, s_p, bits)
    p = p.cpu().numpy()
    normal = p_ref >= 2.0 ** -126
    assert ulp_diff(p[normal], p_ref[normal]).max() <= 2
    assert np.all(np.abs(p[~normal].astype(np.float64) - p_ref[~normal]) <= 2.0 ** -126)
    g = from_codes(got)
    assert np.all(g >= lo) and np.all(g <= hi)
    assert (g != q).mean() < 1e-3
    assert padding_is_zero(got)


@pytest.mark.parametrize("bits", [4, 2, 3, 8])
@pytest.mark.parametrize("rows,cols,ld,bound", [(591, 197, 200, 700), (5000, 197, 200, 4096), (33, 50, 52, 1024), (40, 577, 580, 700),
                                                (24, 785, 788, 701), (9, 1, 4, 8192), (17, 256, 256, 700), (300, 832, 832, 700),
                                                (64, 197, 200, 4095)])
def test_softmax_quantize_bounded_within_two_ulp_and_band(rows, cols, ld, bits, bound):
    """The table-driven kernel for scores of declared range meets the same contract as the general one: probabilities
    within 2 ulp of the fp64 softmax, codes inside the oracle's band.  5000 rows exceed one pass of the persistent
    grid (148 SMs x 4 CTAs x 16 rows would be 9472; with 73 KB of table two CTAs fit: 4736)."""
    S = np.zeros((rows, ld), np.int32)
    S[:, :cols] = (si.splitmix64(31 + cols, rows * cols) % np.uint64(1401)).astype(np.int64).reshape(rows, cols) - 700
    S[0, :cols] = 5
    if cols > 3:
        S[1, :cols] = -700
        S[1, 2] = 700
    c = np.float32(0.0211 if bound < 2000 else 0.0047)
    if bound == 4095:
        # the edge of the no-maximum range: exp arguments reach +-79.9, whole rows near either end (row sums of
        # about e^79 and e^-79), the two-float 1/Z at the ends of the fp32 range
        c = np.float32(0.0195)
        S[:, :cols] = np.clip(S[:, :cols] * 6, -4095, 4095)
        S[2, :cols] = 4095 - (np.arange(cols) % 7)
        S[3, :cols] = -4095 + (np.arange(cols) % 5)
    s_p = np.float32(2.0 / (cols * math.sqrt(si.code_range(bits, False)[1])))
    got, p = vt.vitint_softmax_quantize_bounded(dev(S), cols, c, s_p, bits, bound, want_p=True)
    assert vt.vitint_device_status() == 0
    p_ref, q, lo, hi = vo.softmax_quantize(S[:, :cols], c, s_p, bits)
    p = p.cpu().numpy()
    normal = p_ref >= 2.0 ** -126
    assert ulp_diff(p[normal], p_ref[normal]).max() <= 2
    assert np.all(np.abs(p[~normal].astype(np.float64) - p_ref[~normal]) <= 2.0 ** -126)
    g = from_codes(got)
    assert np.all(g >= lo) and np.all(g <= hi)
    assert (g != q).mean() < 1e-3
    assert padding_is_zero(got)
    # the same table serves a second call
    ws = torch.empty(vt.vitint_softmax_table_workspace_bytes(bound), dtype=torch.uint8, device="cuda")
    a = vt.vitint_softmax_quantize_bounded(dev(S), cols, c, s_p, bits, bound, workspace=ws)
    b = vt.vitint_softmax_quantize_bounded(dev(S), cols, c, s_p, bits, bound, workspace=ws, table_ready=True)
    assert np.array_equal(from_codes(a), g) and np.array_equal(from_codes(b), g)


def test_softmax_quantize_bounded_rejects_and_flags():
    S = dev(np.zeros((8, 200), np.int32))
    with pytest.raises(vt.VitintError) as e:
        vt.vitint_softmax_quantize_bounded(S, 197, 0.02, 0.003, 4, 4097)       # 4096 * 0.02 > 80
    assert "unsupported" in str(e.value).lower()
    with pytest.raises(vt.VitintError):
        vt.vitint_softmax_quantize_bounded(dev(np.zeros((8, 197), np.int32)), 197, 0.002, 0.003, 4, 4096)   # ld % 4 != 0
    with pytest.raises(vt.VitintError):
        vt.vitint_softmax_quantize_bounded(S, 197, 0.002, 0.003, 4, 9000)      # no table that large
    with pytest.raises(vt.VitintError):
        vt.vitint_softmax_quantize_bounded(S, 197, 0.002, 0.003, 4, 4096,
                                           workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    # a score outside the declared range reads a clamped table entry (nothing faults) and is reported
    Sb = np.zeros((8, 200), np.int32)
    Sb[3, 7] = 5000
    Sb[4, 9] = -2 ** 31
    out = guarded_codes(8, 197, 4, False)
    vt.vitint_softmax_quantize_bounded(dev(Sb), 197, 0.002, 0.003, 4, 4096, out=out)
    assert vt.vitint_device_status() != 0
    assert vt.vitint_device_status() == 0
    check_guards()


@pytest.mark.parametrize("bits", [4, 2, 3, 8])
@pytest.mark.parametrize("rows,cols,ld", [(591, 197, 200), (64, 197, 197), (33, 50, 52), (40, 577, 580), (24, 785, 785), (9, 1, 4)])
def test_softmax_shift_quantize_bit_exact(rows, cols, ld, bits):
    """Eq. 4 softmax with the division-free comparator quantizer: integer / single-rounding arithmetic, unique codes."""
    S = np.zeros((rows, ld), np.int32)
    S[:, :cols] = (si.splitmix64(131 + cols, rows * cols) % np.uint64(1401)).astype(np.int64).reshape(rows, cols) - 700
    S[0, :cols] = 5
    if cols > 3:
        S[1, :cols] = -700
        S[1, 2] = 700
    c2 = np.float32(0.0211 * 1.4426950408889634)
    s_p = np.float32(2.0 / (cols * math.sqrt(si.code_range(bits, False)[1])))
    got = vt.vitint_softmax_shift_quantize(dev(S), cols, c2, s_p, bits)
    want = vo.softmax_shift_quantize(S[:, :cols], c2, s_p, bits)
    assert np.array_equal(from_codes(got), want)
    assert padding_is_zero(got)
    if cols > 3:
        assert want.max() == si.code_range(bits, False)[1]


def test_softmax_error_statistics_on_attention_like_rows():
    rows, cols = 4096, 197
    S = (si.splitmix64(77, rows * cols) % np.uint64(257)).astype(np.int64).reshape(rows, cols) - 128
    c = np.float32(0.0035)
    got, p = vt.vitint_softmax_quantize(dev(S.astype(np.int32)), cols, c, 0.00262, 4, want_p=True)
    p_ref, q, lo, hi = vo.softmax_quantize(S, c, np.float32(0.00262), 4)
    d = ulp_diff(p.cpu().numpy(), p_ref)
    assert d.max() <= 2 and d.mean() < 0.6
    g = from_codes(got)
    assert np.all(g >= lo) and np.all(g <= hi)


@pytest.mark.parametrize("byte_codes", [False, True], ids=["packed_qkv", "byte_qkv"])
@pytest.mark.parametrize("bits", [4, 2, 3])
@pytest.mark.parametrize("batch,tokens,heads,scale", [(1, 197, 3, 1.0), (3, 197, 2, 3.0), (2, 50, 1, 3.0), (1, 256, 2, 2.0),
                                                      (5, 128, 1, 0.3), (2, 129, 2, 2.5), (1, 577, 2, 2.0), (2, 785, 1, 2.5),
                                                      (3, 257, 1, 1.0), (1, 1000, 1, 1.5)])
def test_attention_core_fused(batch, tokens, heads, bits, scale, byte_codes):
    """Fused Q K^T -> softmax -> P V against the oracle stages; rows whose P codes are unique must be bit-exact.
    The Q, K, V codes arrive bit-packed (unpacked inside the kernel) or one per byte (the TMA copy is the operand).
    Beyond 256 tokens the chunked two-pass kernel runs (byte-stored codes; packed codes are declined)."""
    D = heads * 64
    if tokens > 256 and not byte_codes:
        with pytest.raises(vt.VitintError):
            vt.vitint_attention_core(to_codes(_qkv_codes(1, tokens, heads, bits, 3), bits, True), 1, heads, tokens, 0.1, 0.1,
                                     0.01, bits, dev(np.ones(D, np.float32)), None)
        return
    qkv = _qkv_codes(batch, tokens, heads, bits, 61 + tokens)
    qmax = si.code_range(bits, True)[1] + 1
    # random codes give scores with spread ~ 8*qmax^2/3; choose the steps so the logits' spread is `scale`
    s_q = s_k = np.float32(math.sqrt(8.0 * scale * 3.0 / (8.0 * qmax * qmax)))
    s_p = np.float32(2.0 / (tokens * math.sqrt(si.code_range(bits, False)[1])))
    q = vp.split_heads(qkv, batch, tokens, heads, 64, 0)
    k = vp.split_heads(qkv, batch, tokens, heads, 64, D)
    v = vp.split_heads(qkv, batch, tokens, heads, 64, 2 * D)
    S = vo.qk(q, k)
    c = vp.softmax_scale(s_q, s_k, 64)
    n = batch * heads
    _, pc, plo, phi = vo.softmax_quantize(S.reshape(n * tokens, tokens), c, s_p, bits)
    acc = vo.pv(pc.reshape(n, tokens, tokens), v)
    alpha, beta = vp.fold(s_p, np.full(D, 0.17, np.float32), None, np.float32(0.17 * 0.6 * qmax / math.sqrt(8 * scale + 1)))
    beta = si.normal(5, (D,), 0.0, 0.3)
    want = vo.epilogue_requant(vp.merge_heads(acc, batch, tokens, heads, 64), alpha, beta, bits, True)
    qkv_dev = to_codes(qkv, bits, True)
    if byte_codes:
        qkv_dev = vt.vitint_widen(qkv_dev)
    got = from_codes(vt.vitint_attention_core(qkv_dev, batch, heads, tokens, s_q, s_k, s_p, bits, dev(alpha), dev(beta)))
    unique_row = (plo == phi).all(axis=1).reshape(n, tokens)             # [B*H, T]
    ok = np.ones((batch * tokens, D), bool)
    for b in range(batch):
        for h in range(heads):
            ok[b * tokens:(b + 1) * tokens, h * 64:(h + 1) * 64] = unique_row[b * heads + h][:, None]
    assert ok.mean() > 0.8
    assert np.array_equal(got[ok], want[ok])
    # every element, unique row or not: inside the interval of O that the oracle's P band can reach
    acc_lo = vo.pv(plo.reshape(n, tokens, tokens), np.maximum(v, 0)) + vo.pv(phi.reshape(n, tokens, tokens), np.minimum(v, 0))
    acc_hi = vo.pv(phi.reshape(n, tokens, tokens), np.maximum(v, 0)) + vo.pv(plo.reshape(n, tokens, tokens), np.minimum(v, 0))
    assert np.all(alpha > 0)
    o_lo = vo.epilogue_requant(vp.merge_heads(acc_lo, batch, tokens, heads, 64), alpha, beta, bits, True)
    o_hi = vo.epilogue_requant(vp.merge_heads(acc_hi, batch, tokens, heads, 64), alpha, beta, bits, True)
    assert np.all(got >= o_lo) and np.all(got <= o_hi)
    assert len(np.unique(want)) >= 3
    if scale >= 1.0:
        assert len(np.unique(pc)) >= 3
    # the same call with the exp table filled once beforehand gives the same codes, bit for bit, also when the
    # table is reused by a second call
    table = vt.vitint_attention_exp_table(bits, s_q, s_k)
    for _ in range(2):
        out2 = vt.Codes.empty(batch * tokens, D, bits, True)
        vt.vitint_attention_core_prepared(qkv_dev, batch, heads, tokens, s_q, s_k, s_p, bits, dev(alpha), dev(beta),
                                          out=out2, table=table)
        assert np.array_equal(from_codes(out2), got)


@pytest.mark.parametrize("bits", [4, 3, 2])
@pytest.mark.parametrize("batch,tokens,heads,scale", [(2, 197, 2, 1.0), (1, 197, 3, 3.0), (2, 129, 1, 2.5), (1, 256, 2, 2.0),
                                                      (3, 64, 1, 0.5), (1, 198, 6, 3.3)])
def test_fused_attention_shift_softmax_bit_exact(batch, tokens, heads, bits, scale):
    """Eq. 4 inside the fused kernel: the attention codes P (read out through one-hot V slabs and an identity output
    quantizer) and the O codes with the real V equal the oracle's Q K^T -> shift softmax with the division-free
    comparator quantizer -> P V -> requantize bit for bit: every step is an integer or a single fp32 operation."""
    D = heads * 64
    qkv = _qkv_codes(batch, tokens, heads, bits, 261 + tokens + bits)
    qmax = si.code_range(bits, True)[1] + 1
    s_q = s_k = np.float32(math.sqrt(8.0 * scale * 3.0 / (8.0 * qmax * qmax)))
    p_qp = si.code_range(bits, False)[1]
    s_p = np.float32(2.0 / (tokens * math.sqrt(p_qp)))
    q = vp.split_heads(qkv, batch, tokens, heads, 64, 0)
    k = vp.split_heads(qkv, batch, tokens, heads, 64, D)
    v = vp.split_heads(qkv, batch, tokens, heads, 64, 2 * D)
    S = vo.qk(q, k)
    c = vp.softmax_scale(s_q, s_k, 64)
    c2 = np.float32(np.float64(c) * np.log2(np.e))
    n = batch * heads
    pc = vo.softmax_shift_quantize(S.reshape(n * tokens, tokens), c2, s_p, bits).reshape(n, tokens, tokens)
    ones = dev(np.ones(D, np.float32))
    got = np.full((n, tokens, tokens), -1, np.int16)
    for r in range((tokens + 63) // 64):
        sel = qkv.copy()
        sel[:, 2 * D:] = 0
        for b in range(batch):
            for j in range(64 * r, min(tokens, 64 * r + 64)):
                sel[b * tokens + j, 2 * D + (j - 64 * r)::64] = 1
        sel_dev = vt.vitint_widen(to_codes(sel, bits, True))
        out = vt.Codes.empty(batch * tokens, D, 8, True)
        o = from_codes(vt.vitint_attention_core_shift(sel_dev, batch, heads, tokens, s_q, s_k, s_p, bits, ones, None, out=out))
        o = vp.split_heads(o, batch, tokens, heads, 64, 0)
        w = min(64, tokens - 64 * r)
        got[:, :, 64 * r:64 * r + w] = o[:, :, :w]
    assert np.array_equal(got, pc)
    if scale >= 1.0:
        assert len(np.unique(pc)) >= 3
    # the real V: O codes
    s_v, s_o = np.float32(0.17), np.float32(0.31)
    alpha, beta = vp.fold(s_p, np.full(D, s_v, np.float32), None, s_o)
    want = vo.epilogue_requant(vo.pv(pc, v).reshape(n * tokens, 64), alpha[:64], beta[:64], bits, True)
    want = vp.merge_heads(want.reshape(n, tokens, 64), batch, tokens, heads, 64)
    o = vt.vitint_attention_core_shift(vt.vitint_widen(to_codes(qkv, bits, True)), batch, heads, tokens, s_q, s_k, s_p, bits,
                                       dev(alpha), None)
    assert np.array_equal(from_codes(o), want)
    assert vt.vitint_device_status() == 0
    # packed codes are not taken by this variant
    with pytest.raises(vt.VitintError):
        vt.vitint_attention_core_shift(to_codes(qkv, bits, True), batch, heads, tokens, s_q, s_k, s_p, bits, dev(alpha), None)


@pytest.mark.parametrize("byte_codes", [False, True], ids=["packed_qkv", "byte_qkv"])
@pytest.mark.parametrize("bits", [4, 3, 2])
@pytest.mark.parametrize("batch,tokens,heads,scale", [(2, 197, 2, 1.0), (1, 197, 3, 3.0), (2, 129, 1, 2.5), (1, 256, 2, 2.0),
                                                      (3, 64, 1, 0.5), (1, 577, 1, 2.0), (1, 300, 2, 1.0)])
def test_fused_attention_p_codes(batch, tokens, heads, bits, scale, byte_codes):
    """The attention codes P that the fused kernel forms on the SM (table-driven softmax, no max subtraction,
    two-float reciprocal), read out exactly and compared element by element with the oracle's band.
    The kernel is not changed for this: its V operand is a one-hot selector (V[j][c] = 1 iff j = c + 64 r), the
    output quantizer is the identity (alpha 1, beta 0, 8-bit signed output), so O[i][c] = P[i][c + 64 r]; one
    call per r covers every column."""
    D = heads * 64
    if tokens > 256 and not byte_codes:
        pytest.skip("the long-sequence kernel takes byte-stored codes")
    qkv = _qkv_codes(batch, tokens, heads, bits, 161 + tokens + bits)
    qmax = si.code_range(bits, True)[1] + 1
    s_q = s_k = np.float32(math.sqrt(8.0 * scale * 3.0 / (8.0 * qmax * qmax)))
    p_qp = si.code_range(bits, False)[1]
    s_p = np.float32(2.0 / (tokens * math.sqrt(p_qp)))
    q = vp.split_heads(qkv, batch, tokens, heads, 64, 0)
    k = vp.split_heads(qkv, batch, tokens, heads, 64, D)
    S = vo.qk(q, k)
    c = vp.softmax_scale(s_q, s_k, 64)
    n = batch * heads
    _, pc, plo, phi = vo.softmax_quantize(S.reshape(n * tokens, tokens), c, s_p, bits)
    pc, plo, phi = (a.reshape(n, tokens, tokens) for a in (pc, plo, phi))
    ones = dev(np.ones(D, np.float32))
    got = np.full((n, tokens, tokens), -1, np.int16)
    for r in range((tokens + 63) // 64):
        sel = qkv.copy()
        sel[:, 2 * D:] = 0
        for b in range(batch):
            for j in range(64 * r, min(tokens, 64 * r + 64)):
                sel[b * tokens + j, 2 * D + (j - 64 * r)::64] = 1          # the same selector for every head
        sel_dev = to_codes(sel, bits, True)
        if byte_codes:
            sel_dev = vt.vitint_widen(sel_dev)
        out = vt.Codes.empty(batch * tokens, D, 8, True)
        o = from_codes(vt.vitint_attention_core(sel_dev, batch, heads, tokens, s_q, s_k, s_p, bits, ones, None, out=out))
        o = vp.split_heads(o, batch, tokens, heads, 64, 0)                   # [n, T, 64]
        w = min(64, tokens - 64 * r)
        got[:, :, 64 * r:64 * r + w] = o[:, :, :w]
        assert not o[:, :, w:].any()                                         # selector columns past the last token
    assert np.all(got >= plo) and np.all(got <= phi)
    off = float((got != pc).mean())
    print(f"fused P codes, {bits}-bit, T={tokens}: {got.size} codes, off-centre share {off:.2e}, "
          f"band wider than one code on {float((phi > plo).mean()):.2e}")
    assert off < 1e-3
    assert np.all(phi - plo <= 1)
    if scale >= 1.0:
        assert len(np.unique(pc)) >= 3


# ---------------------------------------------------------------------------
# glue
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("cols", [192, 384, 768, 1024, 100])
@pytest.mark.parametrize("bits", [4, 2, 8])
def test_layernorm_quantize(cols, bits):
    rows = 197
    x = si.normal(41 + cols, (rows, cols), 3.0, 2.0)
    x[5] += 100.0                                   # |mean| >> sigma
    g = si.normal(42, (cols,), 1.0, 0.02)
    b = si.normal(43, (cols,), 0.0, 0.02)
    step = si.gaussian_lsq_step(1.0, bits)
    got, y = vt.vitint_layernorm_quantize(dev(x), dev(g), dev(b), 1e-6, step, bits, True, want_y=True)
    y_ref, tol = vo.layernorm(x, g, b, 1e-6)
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= tol)
    q, lo, hi = vo.quantize_band(y_ref, tol, step, bits, True)
    gq = from_codes(got)
    assert np.all(gq >= lo) and np.all(gq <= hi) and (gq != q).mean() < 1e-3
    assert padding_is_zero(got)


@pytest.mark.parametrize("rows,cols", [(197, 192), (197, 768), (70, 64), (1, 4), (133, 1024), (37, 100)])
@pytest.mark.parametrize("bits,container", [(4, 0), (4, 8), (3, 0), (2, 0), (2, 8)])
def test_layernorm_compare_quantize_bit_exact(rows, cols, bits, container):
    """Eq. 5 statistics + the comparator of Fig. 5(b): single fp32 operations in a fixed order on both
    sides, so the row statistics and every level are compared bit for bit (no band)."""
    x = si.normal(900 + cols + rows, (rows, cols), 0.7, 1.9)
    if rows > 5:
        x[5] += 50.0                                 # |mean| >> sigma
        x[3] *= 1e-3
    g = si.normal(901 + cols, (cols,), 1.0, 0.3)
    g[cols // 3] = -0.8                               # a negative gain flips the comparison
    b = si.normal(902 + cols, (cols,), 0.0, 0.3)
    step = si.gaussian_lsq_step(1.0, bits)
    eps = 1e-6
    ref, neg, flip = vo.layernorm_references(g, b, step, bits, True, cols)
    q_ref, mu_ref, v_ref = vo.layernorm_compare_quantize(x, ref, neg, flip, eps, bits, True, want_stats=True)
    refs_g, flip_g = vt.fold_layernorm_references(g, b, step, bits, True, cols)
    # the library's own folding gives the oracle's references (magnitude, sign, flip)
    assert np.array_equal(np.abs(refs_g), ref) and np.array_equal(flip_g, flip)
    assert np.array_equal(np.signbit(refs_g) & (refs_g != 0), (neg != 0) & (ref != 0))
    n_eps = float(np.float32(np.float64(cols) * np.float64(np.float32(eps))))
    out = vt.Codes.empty(rows, cols, bits, True, "cuda", container=container)
    got, stats = vt.vitint_layernorm_compare_quantize(dev(x), dev(refs_g), dev(flip_g), n_eps, bits, True, out=out)
    st = stats.cpu().numpy()
    assert np.array_equal(st[:, 0].view(np.uint32), mu_ref.view(np.uint32))
    assert np.array_equal(st[:, 1].view(np.uint32), v_ref.view(np.uint32))
    assert np.array_equal(from_codes(got), q_ref)
    assert padding_is_zero(got)


def test_layernorm_compare_quantize_widest_row_and_single_row():
    """The widest supported row (4096 columns: the reciprocal table fills 32 KB of shared memory) and a single row."""
    rows, cols, bits = 3, 4096, 3
    x = si.normal(77, (rows, cols), -0.2, 1.1)
    g = si.normal(78, (cols,), 1.0, 0.1)
    b = si.normal(79, (cols,), 0.0, 0.1)
    step = si.gaussian_lsq_step(1.0, bits)
    ref, neg, flip = vo.layernorm_references(g, b, step, bits, True, cols)
    q_ref, mu_ref, v_ref = vo.layernorm_compare_quantize(x, ref, neg, flip, 1e-6, bits, True, want_stats=True)
    refs_g, flip_g = vt.fold_layernorm_references(g, b, step, bits, True, cols)
    n_eps = float(np.float32(np.float64(cols) * np.float64(np.float32(1e-6))))
    for r0, r1 in ((0, rows), (1, 2)):
        got, stats = vt.vitint_layernorm_compare_quantize(dev(x[r0:r1]), dev(refs_g), dev(flip_g), n_eps, bits, True)
        st = stats.cpu().numpy()
        assert np.array_equal(st[:, 0].view(np.uint32), mu_ref[r0:r1].view(np.uint32))
        assert np.array_equal(st[:, 1].view(np.uint32), v_ref[r0:r1].view(np.uint32))
        assert np.array_equal(from_codes(got), q_ref[r0:r1])
    with pytest.raises(vt.VitintError):               # one more group of four columns is beyond the table
        wide = torch.zeros((2, 4100), dtype=torch.float32, device="cuda")
        r2, f2 = vt.fold_layernorm_references(np.ones(4100), np.zeros(4100), step, bits, True, 4100)
        vt.vitint_layernorm_compare_quantize(wide, dev(r2), dev(f2), 1e-3, bits, True)


def test_attention_core_prepared_argument_checks():
    qkv = vt.Codes.empty(197, 3 * 64, 4, True)
    qkv.data.zero_()
    out = vt.Codes.empty(197, 64, 4, True)
    alpha = torch.ones(64, dtype=torch.float32, device="cuda")
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(vt.VitintError):               # table too small for 4-bit codes
        vt.vitint_attention_core_prepared(qkv, 1, 1, 197, 0.1, 0.1, 0.01, 4, alpha, None, out=out, table=small)
    with pytest.raises(vt.VitintError):               # no table-driven kernel for 8-bit codes
        vt.vitint_attention_exp_table(8, 0.1, 0.1, table=small)
    with pytest.raises(vt.VitintError):               # steps must be positive and finite
        vt.vitint_attention_exp_table(4, 0.0, 0.1)


def test_layernorm_compare_quantize_argument_checks():
    x = torch.zeros((8, 64), dtype=torch.float32, device="cuda")
    refs, flip = vt.fold_layernorm_references(np.ones(64), np.zeros(64), 0.5, 4, True, 64)
    with pytest.raises(vt.VitintError):               # eps must be positive: V > 0 keeps the reference order
        vt.vitint_layernorm_compare_quantize(x, dev(refs), dev(flip), 0.0, 4, True)
    with pytest.raises(vt.VitintError):               # 255 references per column are not supported
        vt.vitint_layernorm_compare_quantize(x, dev(refs), dev(flip), 1e-4, 8, True)
    with pytest.raises(vt.VitintError):               # columns must come in fours
        vt.vitint_layernorm_compare_quantize(x[:, :62], dev(refs), dev(flip), 1e-4, 4, True)


# ---------------------------------------------------------------------------
# a7: composed block, staged
# ---------------------------------------------------------------------------

def _attention_weights(cfg, prm, st, proj_epi):
    D = cfg.dim
    return vt.AttentionWeights(
        batch=cfg.batch, tokens=cfg.tokens, heads=cfg.heads, bits=cfg.bits,
        w_qkv=to_codes(st["w_qkv_codes"], cfg.bits, True), alpha_qkv=dev(st["alpha_qkv"]), beta_qkv=dev(st["beta_qkv"]),
        q_step=float(prm["s_q"]), k_step=float(prm["s_k"]), v_step=float(prm["s_v"]), p_step=float(prm["s_p"]),
        o_step=float(prm["s_o"]), p_bits=cfg.bits, alpha_o=dev(np.tile(st["alpha_o"], cfg.heads)), beta_o=None,
        w_proj=to_codes(st["w_proj_codes"], cfg.bits, True), w_proj_step=dev(prm["s_w_proj"]),
        b_proj=dev(prm["b_proj"]), proj_epi=proj_epi)


@pytest.mark.parametrize("cfg", [si.VIT_TINY_BLOCK, si.VIT_TINY_BLOCK.with_(w_std=0.12, seed_index=11),
                                 si.VIT_SMALL_BLOCK.with_(batch=3)], ids=["tiny", "tiny_peaked", "small_b3"])
def test_attention_block_staged(cfg):
    prm = si.layer_parameters(cfg)
    x = si.activations(cfg)
    s_x = si.lsq_step(x, cfg.bits, True)
    xq = vo.quantize(x, s_x, cfg.bits, True)
    st = vp.attention_block(xq, s_x, prm, cfg.batch, cfg.tokens, cfg.heads, cfg.bits, proj="dequant")
    aw = _attention_weights(cfg, prm, st, vt.Epilogue(mode=vt.EPI_DEQUANT_F32))
    M, D, T, H = cfg.rows, cfg.dim, cfg.tokens, cfg.heads
    dq = vt.Codes.empty(M, 3 * D, cfg.bits, True)
    dp = vt.Codes.empty(cfg.batch * H * T, T, cfg.bits, False)
    do = vt.Codes.empty(M, D, cfg.bits, True)
    xg = vt.vitint_quantize(dev(x), float(s_x), cfg.bits, True)
    out = vt.vitint_attention_block(xg, aw, dbg_qkv=dq, dbg_p=dp, dbg_o=do).cpu().numpy()
    # stage 1: QKV codes are unique
    assert np.array_equal(from_codes(dq), st["qkv_codes"])
    # stage 2: P codes inside the band; rows (image, head, token) holding an off-centre code are marked
    gp = from_codes(dp).reshape(cfg.batch * H, T, T)
    assert np.all(gp >= st["p_lo"]) and np.all(gp <= st["p_hi"])
    flipped = (gp != st["p_codes"]).any(axis=2)                        # [B*H, T]
    assert flipped.mean() < 0.02
    # stage 3: O codes exact wherever the P row agreed
    go = from_codes(do)
    o_ok = np.ones((M, D), bool)
    for b in range(cfg.batch):
        for h in range(H):
            o_ok[b * T:(b + 1) * T, h * 64:(h + 1) * 64] = ~flipped[b * H + h][:, None]
    assert np.array_equal(go[o_ok], st["o_codes"][o_ok])
    assert np.all(np.abs(go.astype(int) - st["o_codes"]) <= 1)
    # stage 4: projection bit-exact on token rows whose O codes all agreed
    rows_ok = (go == st["o_codes"]).all(axis=1)
    assert rows_ok.mean() > 0.9
    assert np.array_equal(out[rows_ok].view(np.uint32), st["out"][rows_ok].view(np.uint32))


def test_attention_block_requant_output():
    cfg = si.VIT_SMALL_BLOCK.with_(batch=2)
    prm = si.layer_parameters(cfg)
    x = si.activations(cfg)
    s_x = si.lsq_step(x, cfg.bits, True)
    xq = vo.quantize(x, s_x, cfg.bits, True)
    st = vp.attention_block(xq, s_x, prm, cfg.batch, cfg.tokens, cfg.heads, cfg.bits, proj="requant")
    epi = vt.Epilogue(mode=vt.EPI_REQUANT, alpha=dev(st["alpha_proj"]), beta=dev(st["beta_proj"]), out_bits=cfg.bits,
                      out_signed=True)
    aw = _attention_weights(cfg, prm, st, epi)
    do = vt.Codes.empty(cfg.rows, cfg.dim, cfg.bits, True)
    out = vt.vitint_attention_block(to_codes(xq, cfg.bits, True), aw, dbg_o=do)
    rows_ok = (from_codes(do) == st["o_codes"]).all(axis=1)
    assert rows_ok.mean() > 0.9
    assert np.array_equal(from_codes(out)[rows_ok], st["out_codes"][rows_ok])
    assert len(np.unique(st["out_codes"])) >= 8


# ---------------------------------------------------------------------------
# sweep over the linear shapes of the scaling study
# ---------------------------------------------------------------------------

SWEEP_KN = [192, 384, 768, 1024, 3072, 4096]


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("tokens,batch", [(197, 1), (577, 1), (785, 2)])
def test_linear_sweep_shapes(tokens, batch, bits):
    """K, N over {192 ... 4096}, M = batch*tokens, Gaussian inputs with 1 % outlier channels, every bit width;
    quantize -> integer linear (requantizing epilogue) against the oracle, bit for bit."""
    M = tokens * batch
    for idx, K in enumerate(SWEEP_KN):
        N = SWEEP_KN[(idx * 5 + 2 + bits) % len(SWEEP_KN)]
        x = si.normal(300 + K + bits, (M, K))
        ch = si.choice_without_replacement(9 + K, K, max(1, K // 100))
        x[:, ch] *= np.float32(10.0)
        w = si.normal(400 + N + bits, (N, K), 0.0, 0.02)
        s_x = si.lsq_step(x, bits, True)
        s_w = si.lsq_step_rows(w, bits)
        qx = vo.quantize(x, s_x, bits, True)
        qw = vo.quantize(w, 0.0, bits, True, row_steps=s_w)
        bias = si.normal(500 + N, (N,), 0.0, 0.01)
        s_out = si.gaussian_lsq_step(float(s_x) * float(np.mean(s_w)) * math.sqrt(K) * (2 ** (bits - 1)) / 2, bits)
        alpha, beta = vp.fold(s_x, s_w, bias, s_out)
        gx = vt.vitint_quantize(dev(x), float(s_x), bits, True)
        gw = vt.vitint_quantize(dev(w), 0.0, bits, True, row_steps=dev(s_w))
        assert np.array_equal(from_codes(gx), qx) and np.array_equal(from_codes(gw), qw)
        if bits != 8:
            gw = vt.vitint_widen(gw)
        epi = vt.Epilogue(mode=vt.EPI_REQUANT, alpha=dev(alpha), beta=dev(beta), out_bits=bits, out_signed=True)
        got = vt.vitint_linear(gx, float(s_x), gw, None, None, epi)
        want = vo.epilogue_requant(vo.matmul_i32(qx, qw), alpha, beta, bits, True)
        assert np.array_equal(from_codes(got), want), (K, N)
        assert len(np.unique(want)) >= min(4, 2 ** bits - 1)


@pytest.mark.parametrize("tokens", [577, 785])
def test_unfused_attention_long_sequences(tokens):
    """Token counts beyond one 256-column tile: Q K^T -> softmax+quantize -> P V through the unfused calls."""
    batch, heads, bits = 1, 2, 4
    D = heads * 64
    qkv = _qkv_codes(batch, tokens, heads, bits, 81 + tokens)
    c8 = to_codes(qkv, bits, True)
    S = vt.vitint_qk(vt.Slabs.of_qkv(c8, tokens, D, 0), vt.Slabs.of_qkv(c8, tokens, D, 1), batch, heads, tokens)
    q = vp.split_heads(qkv, batch, tokens, heads, 64, 0)
    k = vp.split_heads(qkv, batch, tokens, heads, 64, D)
    v = vp.split_heads(qkv, batch, tokens, heads, 64, 2 * D)
    S_ref = vo.qk(q, k)
    assert np.array_equal(S.cpu().numpy()[:, :, :tokens], S_ref)
    c = np.float32(0.004)
    s_p = np.float32(2.0 / (tokens * math.sqrt(15.0)))
    n = batch * heads
    P = vt.vitint_softmax_quantize(S.reshape(n * tokens, -1), tokens, c, s_p, bits)
    _, pc, plo, phi = vo.softmax_quantize(S_ref.reshape(n * tokens, tokens), c, s_p, bits)
    gp = from_codes(P)
    assert np.all(gp >= plo) and np.all(gp <= phi) and len(np.unique(pc)) >= 8
    # P V from the oracle's own codes, so the comparison is exact
    O = vt.vitint_pv(to_codes(pc, bits, False), vt.Slabs.of_qkv(c8, tokens, D, 2), batch, heads, tokens, 1.0, 1.0,
                     vt.Epilogue(mode=vt.EPI_ACC_I32))
    want = vp.merge_heads(vo.pv(pc.reshape(n, tokens, tokens), v), batch, tokens, heads, 64)
    assert np.array_equal(O.cpu().numpy(), want)
