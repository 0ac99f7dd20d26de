"""Pins of the CPU oracle against what the paper and the mathematics fix (CPU only).

Each test compares an oracle function with something that is not the oracle:
values the paper prints, exact rational arithmetic, brute force in Python
integers, closed forms, or a library routine for a special case.
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle as vo
import synth_inputs as si
from oracle import pipeline as vp


# ---------------------------------------------------------------------------
# helpers that do not use the oracle
# ---------------------------------------------------------------------------

def f32_from_fraction(fr: Fraction) -> np.float32:
    """Exact round-to-nearest-even of a rational to fp32 (normal range only)."""
    if fr == 0:
        return np.float32(0.0)
    sign = -1 if fr < 0 else 1
    fr = abs(fr)
    e = math.floor(math.log2(fr))
    while Fraction(2) ** e > fr:
        e -= 1
    while Fraction(2) ** (e + 1) <= fr:
        e += 1
    scaled = fr / Fraction(2) ** (e - 23)          # in [2^23, 2^24)
    n = scaled.numerator // scaled.denominator
    rem = scaled - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return np.float32(sign * float(n) * 2.0 ** (e - 23))


def comparator_code(x: float, step: float, bits: int, signed: bool) -> int:
    """Code = lowest level + number of thresholds (k-1/2)*step strictly exceeded (Section IV-B)."""
    qn, qp = si.code_range(bits, signed)
    return qn + sum(1 for k in range(qn + 1, qp + 1) if Fraction(x) > (Fraction(k) - Fraction(1, 2)) * Fraction(step))


# ---------------------------------------------------------------------------
# quantizer
# ---------------------------------------------------------------------------

def test_three_bit_ladder_from_paper(golden_dir):
    rows = [l.split() for l in (golden_dir / "ladder_3bit.txt").read_text().splitlines() if l and l[0] != "#"]
    assert len(rows) == 7
    for step in (0.25, 1.0, 0.0078125):
        for b, below, above in rows:
            thr = float(b) * step
            eps = step / 64.0
            x = np.array([[thr - eps, thr + eps]], dtype=np.float32)
            q = vo.quantize(x, step, 3, True)
            assert q.tolist() == [[int(below), int(above)]]
    # outside the ladder: clamp to the end levels
    q = vo.quantize(np.array([[-100.0, 100.0]], np.float32), 0.25, 3, True)
    assert q.tolist() == [[-4, 3]]


@pytest.mark.parametrize("bits,signed", [(2, True), (3, True), (4, True), (8, True), (2, False), (4, False), (8, False)])
def test_quantizer_equals_comparator_count_off_ties(bits, signed):
    step = 0.125
    x = si.normal(11 + bits, (1, 4096), 0.0, step * (1 << bits) / 3.0)
    q = vo.quantize(x, step, bits, signed)[0]
    for xi, qi in zip(x[0, :600], q[:600]):
        assert comparator_code(float(xi), step, bits, signed) == int(qi)


@pytest.mark.parametrize("bits,signed", [(2, True), (3, True), (4, True), (8, True), (4, False), (8, False)])
def test_quantizer_ties_to_even_and_idempotent(bits, signed):
    qn, qp = si.code_range(bits, signed)
    step = 0.5
    ks = np.arange(qn, qp + 1)
    # exact representable points: codes reproduce themselves
    x = (ks * step).astype(np.float32)[None, :]
    assert vo.quantize(x, step, bits, signed)[0].tolist() == ks.tolist()
    # exact ties (k + 1/2)*step go to the even neighbour (then clamp)
    ties = ((ks[:-1] + 0.5) * step).astype(np.float32)[None, :]
    want = [int(k if k % 2 == 0 else k + 1) for k in ks[:-1]]
    assert vo.quantize(ties, step, bits, signed)[0].tolist() == want


def test_quantizer_per_row_steps_and_true_division():
    # 0.3 is not a power of two: x/s and x*(1/s) differ for some x; the oracle must divide.
    s = np.float32(0.3)
    inv = np.float32(1.0) / s
    xs = np.arange(1, 200001, dtype=np.float32) * np.float32(0.05)
    div = np.rint(xs / s)
    mul = np.rint(xs * inv)
    differ = np.nonzero(div != mul)[0]
    assert differ.size > 0
    x = xs[differ[:64]][None, :]
    q = vo.quantize(x, s, 8, False)
    assert q[0].tolist() == np.clip(div[differ[:64]], 0, 255).astype(int).tolist()
    # per-row steps: row m uses steps[m]
    xr = np.array([[1.0, 2.0, 3.0], [1.0, 2.0, 3.0]], np.float32)
    q = vo.quantize(xr, 0.0, 4, True, row_steps=np.array([1.0, 0.5], np.float32))
    assert q.tolist() == [[1, 2, 3], [2, 4, 6]]


# ---------------------------------------------------------------------------
# packed format
# ---------------------------------------------------------------------------

def test_pack_hand_computed_bytes():
    # 4-bit: element 0 in the low nibble; -1 -> 0xF, -8 -> 0x8
    assert vo.pack(np.array([[1, -1, -8, 7]], np.int16), 4)[0, :2].tolist() == [0xF1, 0x78]
    # 3-bit codes live in 4-bit containers, sign-extended
    assert vo.pack(np.array([[-4, 3]], np.int16), 3)[0, :1].tolist() == [0x3C]
    # 2-bit: four per byte, element i at bit 2*i;  [1,-1,-2,0] -> 01 | 11<<2 | 10<<4 | 00<<6 = 0x2D
    assert vo.pack(np.array([[1, -1, -2, 0]], np.int16), 2)[0, :1].tolist() == [0x2D]
    # 8-bit: plain bytes
    assert vo.pack(np.array([[-128, 127, 255 - 256]], np.int16), 8)[0, :3].tolist() == [0x80, 0x7F, 0xFF]
    # pitch is a multiple of 16 and the tail is zero
    pk = vo.pack(np.full((1, 5), -1, np.int16), 4)
    assert pk.shape == (1, 16) and pk[0, 3:].tolist() == [0] * 13 and pk[0, 2] == 0x0F


@pytest.mark.parametrize("bits,signed", [(2, True), (2, False), (3, True), (3, False), (4, True), (4, False), (8, True), (8, False)])
def test_pack_roundtrip_all_values_all_residues(bits, signed):
    qn, qp = si.code_range(bits, signed)
    vals = np.arange(qn, qp + 1)
    for cols in range(1, 34):
        q = np.array([[vals[(i * 7 + r) % len(vals)] for i in range(cols)] for r in range(len(vals))], np.int16)
        pk = vo.pack(q, bits)
        assert pk.shape[1] % 16 == 0
        assert np.array_equal(vo.unpack(pk, cols, bits, signed), q)


# ---------------------------------------------------------------------------
# integer contraction (Eq. 1)
# ---------------------------------------------------------------------------

def test_contraction_brute_force_every_two_bit_code():
    vals = [-2, -1, 0, 1]
    # every pair of 2-element rows over all 2-bit codes: 16 x 16 dot products, checked with Python ints
    rows = np.array(list(itertools.product(vals, repeat=2)), np.int16)
    acc = vo.matmul_i32(rows, rows)
    for i, a in enumerate(rows):
        for j, b in enumerate(rows):
            assert int(acc[i, j]) == int(a[0]) * int(b[0]) + int(a[1]) * int(b[1])


def test_contraction_rectangular_against_python_ints():
    # M, N, K all different: a transposed operand or swapped index cannot pass
    a = (si.splitmix64(5, 3 * 7) % np.uint64(16)).astype(np.int64).reshape(3, 7) - 8
    b = (si.splitmix64(6, 5 * 7) % np.uint64(16)).astype(np.int64).reshape(5, 7) - 8
    acc = vo.matmul_i32(a, b)
    assert acc.shape == (3, 5)
    for m in range(3):
        for n in range(5):
            assert int(acc[m, n]) == sum(int(a[m, k]) * int(b[n, k]) for k in range(7))


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_contraction_closed_forms(bits):
    qn, qp = si.code_range(bits, True)
    K = 193
    a = np.full((2, K), qp, np.int16)
    a[1] = qn
    b = np.full((3, K), qn, np.int16)
    b[1] = qp
    b[2] = 0
    b[2, 17] = 1                      # one-hot picks a[:, 17]
    acc = vo.matmul_i32(a, b)
    assert acc.tolist() == [[K * qp * qn, K * qp * qp, qp], [K * qn * qn, K * qn * qp, qn]]


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_reordering_identity_against_fp64_dequantized_matmul(bits):
    """(s_x q_x)(s_w q_w)^T + b  ==  [q_x q_w^T] s_x diag(s_w) + b  (Eq. 1, Eq. 2)."""
    M, N, K = 13, 11, 96
    x = si.normal(21, (M, K))
    w = si.normal(22, (N, K), 0.0, 0.02)
    bias = si.normal(23, (N,), 0.0, 0.01)
    s_x = si.lsq_step(x, bits, True)
    s_w = si.lsq_step_rows(w, bits)
    qx = vo.quantize(x, s_x, bits, True)
    qw = vo.quantize(w, 0.0, bits, True, row_steps=s_w)
    y = vo.epilogue_dequant(vo.matmul_i32(qx, qw), s_x, s_w, bias)
    xd = qx.astype(np.float64) * float(s_x)
    wd = qw.astype(np.float64) * s_w.astype(np.float64)[:, None]
    ref = xd @ wd.T + bias.astype(np.float64)
    mag = np.abs(xd) @ np.abs(wd).T + np.abs(bias.astype(np.float64))
    assert np.all(np.abs(y.astype(np.float64) - ref) <= 2.0 ** -22 * mag)
    assert np.abs(ref).max() > 0.05      # the comparison is not vacuous


def test_overflow_bound_and_int64_edge():
    # the declared-range bound
    assert vo.overflow_bound(4096, 4, True, 4, True) == 4096 * 8 * 8
    assert vo.overflow_bound(768, 4, False, 4, True) == 768 * 15 * 8
    assert vo.overflow_bound(100, 8, False, 8, True) == 100 * 255 * 128
    # 8-bit at the edge: K*128*128 reaches 2^31 at K = 131072; one less still fits
    K = 131072
    assert vo.overflow_bound(K, 8, True, 8, True) == 2 ** 31
    a = np.full((1, K), -128, np.int16)
    acc64 = vo.matmul_i64(a, a)
    assert int(acc64[0, 0]) == 2 ** 31                  # needs more than int32
    assert vo.overflow_bound(K - 1, 8, True, 8, True) < 2 ** 31
    acc32 = vo.matmul_i32(a[:, :K - 1], a[:, :K - 1])
    assert int(acc32[0, 0]) == (K - 1) * 16384 == int(vo.matmul_i64(a[:, :K - 1], a[:, :K - 1])[0, 0])


# ---------------------------------------------------------------------------
# epilogues (Eq. 2)
# ---------------------------------------------------------------------------

def test_dequant_epilogue_is_one_fused_multiply_add_exact_rational():
    acc = np.array([[3, -7, 12345, 16777215, -491520]], np.int32)
    s_x = np.float32(0.3)
    s_w = np.array([0.01, 0.7, 1.1e-3, 3.3e-5, 0.123], np.float32)
    bias = np.array([-0.009, 4.9, -13.58, 1e-4, 60457.0], np.float32)
    y = vo.epilogue_dequant(acc, s_x, s_w, bias)
    for n in range(5):
        sc = f32_from_fraction(Fraction(float(s_x)) * Fraction(float(s_w[n])))
        want = f32_from_fraction(Fraction(int(acc[0, n])) * Fraction(float(sc)) + Fraction(float(bias[n])))
        assert y[0, n] == want
    # a case where multiply-then-add rounds differently from the fused form must follow the fused form
    found = False
    for a in range(1, 4000):
        sc = np.float32(0.1)
        b = -np.float32(np.float32(a) * sc)
        fused = f32_from_fraction(Fraction(a) * Fraction(float(sc)) + Fraction(float(b)))
        if fused != np.float32(np.float32(a) * sc + b):
            out = vo.epilogue_dequant(np.array([[a]], np.int32), np.float32(1.0), np.array([sc], np.float32),
                                      np.array([b], np.float32))
            assert out[0, 0] == fused
            found = True
            break
    assert found


def test_dequant_residual_is_a_second_rounded_add():
    acc = np.array([[5, -3]], np.int32)
    s_w = np.array([0.1, 0.2], np.float32)
    bias = np.array([0.3, 0.4], np.float32)
    res = np.array([[1e-3, 7.0]], np.float32)
    y = vo.epilogue_dequant(acc, np.float32(0.7), s_w, bias, res)
    for n in range(2):
        sc = f32_from_fraction(Fraction(float(np.float32(0.7))) * Fraction(float(s_w[n])))
        v = f32_from_fraction(Fraction(int(acc[0, n])) * Fraction(float(sc)) + Fraction(float(bias[n])))
        assert y[0, n] == f32_from_fraction(Fraction(float(v)) + Fraction(float(res[0, n])))


def test_requant_epilogue_exact_cases_and_clamp():
    # alpha, beta powers of two: fmaf is exact, result known by hand
    acc = np.array([[8, 9, 10, 11, 12, -100, 100, 0]], np.int32)
    alpha = np.full(8, 0.25, np.float32)
    beta = np.full(8, 0.25, np.float32)
    # values 2.25 2.5 2.75 3.0 3.25 -24.75 25.25 0.25 -> rint (ties even) 2 2 3 3 3 -25 25 0 -> clamp [-8,7]
    assert vo.epilogue_requant(acc, alpha, beta, 4, True)[0].tolist() == [2, 2, 3, 3, 3, -8, 7, 0]
    assert vo.epilogue_requant(acc, alpha, beta, 4, False)[0].tolist() == [2, 2, 3, 3, 3, 0, 15, 0]


def test_folded_requant_equals_quantized_dequant_off_ties():
    """Eq. 2: [acc + b/(s_x s_w)] s_x s_w / s_out  vs quantizing the dequantized output."""
    M, N, K = 64, 48, 192
    qx = vo.quantize(si.normal(31, (M, K)), 0.6, 4, True)
    w = si.normal(32, (N, K), 0.0, 0.02)
    s_w = si.lsq_step_rows(w, 4)
    qw = vo.quantize(w, 0.0, 4, True, row_steps=s_w)
    bias = si.normal(33, (N,), 0.0, 0.01)
    acc = vo.matmul_i32(qx, qw)
    s_out = np.float32(0.1)
    alpha, beta = vp.fold(np.float32(0.6), s_w, bias, s_out)
    folded = vo.epilogue_requant(acc, alpha, beta, 4, True)
    exact = acc.astype(np.float64) * 0.6000000238418579 * s_w.astype(np.float64) + bias.astype(np.float64)
    u = exact / float(s_out)
    want = np.clip(np.rint(u), -8, 7)
    near_tie = np.abs(u - np.floor(u) - 0.5) < 1e-5
    assert np.array_equal(folded[~near_tie], want[~near_tie].astype(np.int16))
    assert np.all(np.abs(folded - want) <= 1)
    assert (~near_tie).mean() > 0.999
    assert len(np.unique(folded)) >= 12


def test_gelu_against_erf_definition_and_identities():
    y = np.linspace(-6, 6, 2401).astype(np.float32)
    acc = np.arange(2401, dtype=np.int32)[None, :]
    # use acc*0 + bias = y so that the activation input is exactly y
    g = vo.epilogue_dequant(acc * 0, np.float32(1.0), np.ones(2401, np.float32), y, None, act=1)[0]
    ref = np.array([0.5 * float(v) * (1.0 + math.erf(float(v) / math.sqrt(2.0))) for v in y])
    assert np.all(np.abs(g.astype(np.float64) - ref) <= np.abs(ref) * 2.0 ** -23 + 1e-45)
    assert g[1200] == 0.0 and y[1200] == 0.0
    assert g[-1] == y[-1]                                   # Phi(6) rounds to 1 in fp32
    sym = g.astype(np.float64) - g[::-1].astype(np.float64)  # GELU(y) - GELU(-y) = y
    assert np.all(np.abs(sym - y.astype(np.float64)) <= 2.0 ** -22 * np.abs(y) + 1e-30)


def test_gelu_requant_band_brackets_code():
    M, N = 8, 512
    acc = (si.splitmix64(41, M * N) % np.uint64(4001)).astype(np.int64).reshape(M, N) - 2000
    s_w = np.full(N, 1e-3, np.float32)
    bias = si.normal(42, (N,), 0.0, 0.01)
    inv_s = np.full(N, np.float32(1.0 / 0.05), np.float32)
    q0, lo0, hi0 = vo.epilogue_gelu_requant(acc.astype(np.int32), np.float32(0.6), s_w, bias, inv_s, 4, False)
    assert np.array_equal(q0, lo0) and np.array_equal(q0, hi0)          # no tolerance given: the band is the code
    q, lo, hi = vo.epilogue_gelu_requant(acc.astype(np.int32), np.float32(0.6), s_w, bias, inv_s, 4, False,
                                         tol_rel=2.0 ** -23)
    assert np.array_equal(q, q0)
    assert np.all(lo <= q) and np.all(q <= hi) and np.all(hi - lo <= 1)
    assert (hi != lo).mean() < 1e-3
    # independent evaluation of the code in fp64 agrees wherever the band is a single code
    yy = acc.astype(np.float64) * float(np.float32(np.float64(np.float32(0.6)) * np.float64(np.float32(1e-3)))) + bias.astype(np.float64)
    gg = 0.5 * yy * (1.0 + np.vectorize(math.erf)(yy / math.sqrt(2.0)))
    want = np.clip(np.rint(gg * float(inv_s[0])), 0, 15)
    u = gg * float(inv_s[0])
    safe = (np.abs(u - np.floor(u) - 0.5) > 1e-4)
    assert np.array_equal(q[safe], want[safe].astype(np.int16))
    assert q.max() == 15 and q.min() == 0


# ---------------------------------------------------------------------------
# softmax (Eq. 3)
# ---------------------------------------------------------------------------

def test_softmax_rows_sum_to_one_and_closed_forms():
    T = 197
    S = (si.splitmix64(51, 8 * T) % np.uint64(1201)).astype(np.int64).reshape(8, T) - 600
    S[1] = 37                                   # all-equal row -> 1/T
    p, q, lo, hi = vo.softmax_quantize(S, np.float32(0.01), np.float32(0.0026), 4)
    assert np.all(np.abs(p.astype(np.float64).sum(1) - 1.0) <= T * 2.0 ** -24)
    assert np.all(p[1] == np.float32(1.0 / T))
    assert np.all(p >= 0)
    # two-element row: logistic closed form
    for d in (0, 1, 5, -40, 300):
        p2, *_ = vo.softmax_quantize(np.array([[d, 0]], np.int32), np.float32(0.125), np.float32(0.07), 4)
        t = float(np.float32(d) * np.float32(0.125))
        want = 1.0 / (1.0 + math.exp(-t))
        assert abs(float(p2[0, 0]) - want) <= 2.0 ** -24 * want
        other = 1.0 / (1.0 + math.exp(t))
        assert abs(float(p2[0, 1]) - other) <= 2.0 ** -24 * other
    # against a straightforward numpy fp64 softmax
    t = (S.astype(np.float32) * np.float32(0.01)).astype(np.float64)
    e = np.exp(t - t.max(1, keepdims=True))
    ref = e / e.sum(1, keepdims=True)
    assert np.all(np.abs(p.astype(np.float64) - ref) <= 2.0 ** -24 * ref + 1e-45)


def test_softmax_shift_invariance_with_power_of_two_scale():
    T = 64
    S = (si.splitmix64(52, 4 * T) % np.uint64(257)).astype(np.int64).reshape(4, T) - 128
    c = np.float32(2.0 ** -5)                     # exact products: adding k to S adds k*c to t exactly
    p0, q0, *_ = vo.softmax_quantize(S, c, np.float32(0.004), 4)
    p1, q1, *_ = vo.softmax_quantize(S + 1000, c, np.float32(0.004), 4)
    assert np.array_equal(p0, p1) and np.array_equal(q0, q1)


def test_softmax_codes_decided_in_fp32_and_band():
    T = 197
    S = (si.splitmix64(53, 32 * T) % np.uint64(801)).astype(np.int64).reshape(32, T) - 400
    s_p = np.float32(2.0 / (T * math.sqrt(15.0)))
    p, q, lo, hi = vo.softmax_quantize(S, np.float32(0.02), s_p, 4)
    want = np.clip(np.rint(p / s_p), 0, 15).astype(np.int16)      # numpy fp32 division, ties-to-even
    assert np.array_equal(q, want)
    assert np.all(lo <= q) and np.all(q <= hi) and np.all(hi - lo <= 1)
    assert (hi != lo).mean() < 1e-3
    assert q.max() == 15 and (q == 0).any()
    # unsigned range (probabilities are never negative): 2-bit gives 0..3
    _, q2, *_ = vo.softmax_quantize(S, np.float32(0.02), s_p, 2)
    assert q2.min() == 0 and q2.max() == 3


def test_qk_and_pv_orientation():
    n, T, d = 2, 5, 3
    Q = (si.splitmix64(61, n * T * d) % np.uint64(16)).astype(np.int64).reshape(n, T, d) - 8
    K = (si.splitmix64(62, n * T * d) % np.uint64(16)).astype(np.int64).reshape(n, T, d) - 8
    V = (si.splitmix64(63, n * T * d) % np.uint64(16)).astype(np.int64).reshape(n, T, d) - 8
    P = (si.splitmix64(64, n * T * T) % np.uint64(16)).astype(np.int64).reshape(n, T, T)
    S = vo.qk(Q, K)
    O = vo.pv(P, V)
    for p_ in range(n):
        assert np.array_equal(S[p_], Q[p_] @ K[p_].T)      # numpy int64 matmul
        assert np.array_equal(O[p_], P[p_] @ V[p_])


# ---------------------------------------------------------------------------
# LayerNorm glue and Eq. 5
# ---------------------------------------------------------------------------

def test_layernorm_against_running_statistics_of_eq5_and_numpy():
    x = si.normal(71, (6, 768), 0.3, 2.0)
    g = si.normal(72, (768,), 1.0, 0.02)
    b = si.normal(73, (768,), 0.0, 0.02)
    y, tol = vo.layernorm(x, g, b, 1e-6)
    for m in range(6):
        mu, m2 = vo.running_stats(x[m])
        xd = x[m].astype(np.float64)
        assert abs(mu - xd.mean()) < 1e-12 and abs(m2 / 768 - xd.var()) < 1e-10
        ref = (xd - mu) / math.sqrt(m2 / 768 + 1e-6) * g + b
        assert np.all(np.abs(y[m] - ref) <= 2.0 ** -23 * np.abs(ref) + 1e-12)
    ones = np.ones(768, np.float32)
    y0, _ = vo.layernorm(x, ones, 0 * ones, 0.0)
    assert np.all(np.abs(y0.mean(1)) < 1e-6) and np.all(np.abs(y0.astype(np.float64).var(1) - 1.0) < 1e-5)
    assert np.all(tol > 0) and tol.max() < 1e-4


def test_running_stats_small_case_by_hand():
    # x = 1, 2, 4: mu = 7/3, M2 = sum (x-mu)^2 = 42/9
    mu, m2 = vo.running_stats(np.array([1.0, 2.0, 4.0], np.float32))
    assert abs(mu - 7.0 / 3.0) < 1e-15 and abs(m2 - 42.0 / 9.0) < 1e-14


# ---------------------------------------------------------------------------
# op counts (Table I) and the composed block
# ---------------------------------------------------------------------------

def test_table1_counts(golden_dir):
    rows = {l.split()[0]: l.split()[1:] for l in (golden_dir / "table1_counts.txt").read_text().splitlines()
            if l and l[0] != "#"}
    c = si.head_mac_counts(198, 384, 64)
    assert c["linear_pe"] == int(rows["linear"][0]) and round(c["linear_mac"] / 1e6, 2) == float(rows["linear"][1])
    assert c["layernorm_pe"] == int(rows["layernorm"][0])
    assert round(c["layernorm_mac"] / 1e6, 2) == float(rows["layernorm"][1])
    assert c["delay"] == int(rows["delay"][0])
    assert c["matmul_qk_pe"] == int(rows["matmul_qk"][0])
    assert round(c["matmul_qk_mac"] / 1e6, 2) == float(rows["matmul_qk"][1])
    assert c["matmul_pv_pe"] == int(rows["matmul_pv"][0])
    assert round(c["matmul_pv_mac"] / 1e6, 2) == float(rows["matmul_pv"][1])
    m = si.mac_counts(197, 768, 12, 64, 3072)
    assert abs(m["total"] / 1e6 - 1453.95) < 0.01


@pytest.mark.parametrize("w_std", [0.02, 0.12])
def test_attention_block_matches_dequantize_first_datapath(w_std):
    """Fig. 1: the integerized datapath (b) equals the dequantize-first datapath (a) given the same codes."""
    cfg = si.VIT_TINY_BLOCK.with_(w_std=w_std)
    prm = si.layer_parameters(cfg)
    x = si.activations(cfg)
    s_x = si.lsq_step(x, cfg.bits, True)
    xq = vo.quantize(x, s_x, cfg.bits, True)
    st = vp.attention_block(xq, s_x, prm, cfg.batch, cfg.tokens, cfg.heads, cfg.bits)
    D, T, H = cfg.dim, cfg.tokens, cfg.heads
    # (a): dequantize codes, float matmuls
    xd = xq.astype(np.float64) * float(s_x)
    wd = st["w_qkv_codes"].astype(np.float64) * prm["s_w_qkv"].astype(np.float64)[:, None]
    qkv = xd @ wd.T + prm["b_qkv"].astype(np.float64)
    seg = np.concatenate([np.full(D, prm["s_q"]), np.full(D, prm["s_k"]), np.full(D, prm["s_v"])]).astype(np.float64)
    u = qkv / seg
    codes = np.clip(np.rint(u), -8, 7)
    safe = np.abs(u - np.floor(u) - 0.5) > 1e-4
    assert np.array_equal(st["qkv_codes"][safe], codes[safe].astype(np.int16))
    assert st["qkv_codes"].shape == (T, 3 * D)
    # attention for head 1 from the oracle's own codes, in floats
    h = 1
    qd = st["qkv_codes"][:, h * 64:(h + 1) * 64].astype(np.float64) * float(prm["s_q"])
    kd = st["qkv_codes"][:, D + h * 64: D + (h + 1) * 64].astype(np.float64) * float(prm["s_k"])
    vd = st["qkv_codes"][:, 2 * D + h * 64: 2 * D + (h + 1) * 64].astype(np.float64) * float(prm["s_v"])
    logits = qd @ kd.T / 8.0
    e = np.exp(logits - logits.max(1, keepdims=True))
    pr = e / e.sum(1, keepdims=True)
    assert np.all(np.abs(st["p"][h] - pr) <= 4e-6 * pr + 1e-12)
    pd = st["p_codes"][h].astype(np.float64) * float(prm["s_p"])
    od = pd @ vd
    uo = od / float(prm["s_o"])
    want_o = np.clip(np.rint(uo), -8, 7)
    safe_o = np.abs(uo - np.floor(uo) - 0.5) > 1e-4
    got_o = st["o_codes"][:, h * 64:(h + 1) * 64]
    assert np.array_equal(got_o[safe_o], want_o[safe_o].astype(np.int16))
    assert len(np.unique(got_o)) >= 6
    if w_std > 0.1:                      # peaked attention rows: the whole unsigned range is used
        assert len(np.unique(st["p_codes"])) == 16
    # projection output: dequantized float path
    o_all = st["o_codes"].astype(np.float64) * float(prm["s_o"])
    wp = st["w_proj_codes"].astype(np.float64) * prm["s_w_proj"].astype(np.float64)[:, None]
    ref = o_all @ wp.T + prm["b_proj"].astype(np.float64)
    mag = np.abs(o_all) @ np.abs(wp).T + np.abs(prm["b_proj"].astype(np.float64))
    assert np.all(np.abs(st["out"] - ref) <= 2.0 ** -22 * mag)


# ---------------------------------------------------------------------------
# shift-based softmax with the division-free quantizer (Eq. 4)
# ---------------------------------------------------------------------------

def _shift_softmax_by_hand(S_row, c2, step, bits):
    """Independent evaluation with Python integers and exact rational rounding."""
    qp = (1 << bits) - 1
    z = (S_row.astype(np.float32) * np.float32(c2)).astype(np.float32)
    f = np.floor(z)
    r = (z - f).astype(np.float32)
    one_plus_r = (np.float32(1.0) + r).astype(np.float32)
    M = [int(Fraction(float(v)) * (1 << 23)) for v in one_plus_r]
    m = int(f.max())
    E = []
    for Mj, fj in zip(M, f):
        sh = 30 + int(fj) - m
        E.append(Mj << sh if sh >= 0 else (Mj >> -sh if sh > -64 else 0))
    sigma = sum(E)
    sig_f = Fraction(float(f32_from_fraction(Fraction(sigma))))
    codes = []
    for Ej in E:
        e_f = Fraction(float(f32_from_fraction(Fraction(Ej))))
        c = 0
        for k in range(1, qp + 1):
            b_k = f32_from_fraction(Fraction(k) * 1 - Fraction(1, 2)) * np.float32(step)   # (k - 1/2) is exact in fp32
            t_k = f32_from_fraction(Fraction(float(np.float32(b_k))) * sig_f)
            if e_f > Fraction(float(t_k)):
                c += 1
        codes.append(c)
    return codes, [Fraction(e, sigma) for e in E]


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_shift_softmax_against_integer_and_rational_arithmetic(bits):
    S = (si.splitmix64(91 + bits, 6 * 23) % np.uint64(801)).astype(np.int64).reshape(6, 23) - 400
    S[1] = 7                                    # all equal
    S[2, :] = -400
    S[2, 5] = 400                               # one dominant score: the others are shifted far to the right
    c2, step = np.float32(0.0211 * 1.4426950408889634), np.float32(2.0 / (23 * math.sqrt(2 ** bits - 1)))
    q, p = vo.softmax_shift_quantize(S, c2, step, bits, want_p=True)
    for r in range(6):
        codes, probs = _shift_softmax_by_hand(S[r], c2, step, bits)
        assert q[r].tolist() == codes
        assert np.allclose(p[r], [float(x) for x in probs], rtol=1e-15, atol=0)
    assert q.max() == 2 ** bits - 1 and q.min() == 0


def test_shift_softmax_error_bound_of_the_linear_residual():
    """2^r ~ 1 + r overestimates by at most 6.15 % (r = 0.5288), so every probability stays within that
    factor of the exact base-2 softmax; integer-valued exponents make it exact."""
    T = 197
    S = (si.splitmix64(95, 16 * T) % np.uint64(1201)).astype(np.int64).reshape(16, T) - 600
    c2 = np.float32(0.01 * 1.4426950408889634)
    _, p = vo.softmax_shift_quantize(S, c2, np.float32(0.0026), 4, want_p=True)
    z = (S.astype(np.float32) * c2).astype(np.float64)
    e = np.exp2(z - z.max(1, keepdims=True))
    ref = e / e.sum(1, keepdims=True)
    ratio = p[ref > 1e-9] / ref[ref > 1e-9]
    assert ratio.max() <= 1.0616 and ratio.min() >= 1.0 / 1.0616 and ratio.std() > 0.005
    assert np.all(np.abs(p.sum(1) - 1.0) < 1e-12)
    # integer exponents: no residual, the shifts are the exact powers of two
    Si = np.array([[0, 1, 2, 5, -3]], np.int32)
    _, pi = vo.softmax_shift_quantize(Si, np.float32(1.0), np.float32(0.05), 4, want_p=True)
    w = np.array([1, 2, 4, 32, 0.125])
    assert np.allclose(pi[0], w / w.sum(), rtol=1e-15)


def test_shift_softmax_comparator_is_strict_and_scaled_by_the_row_sum():
    # two equal scores: p = 1/2 each; thresholds b_k * Sigma with step 0.25: (k - 1/2)/4 < 1/2  <=>  k < 2.5
    q = vo.softmax_shift_quantize(np.array([[3, 3]], np.int32), np.float32(1.0), np.float32(0.25), 4)
    assert q.tolist() == [[2, 2]]
    # exact tie: p = 1/2 against the reference (k - 1/2) * step = 1/2 at k = 1, step = 1: not exceeded (strict '>')
    q = vo.softmax_shift_quantize(np.array([[3, 3]], np.int32), np.float32(1.0), np.float32(1.0), 4)
    assert q.tolist() == [[0, 0]]


# ---------------------------------------------------------------------------
# quantizing LayerNorm: Eq. 5 statistics + the comparator of Fig. 5(b)
# ---------------------------------------------------------------------------

def _direct_layernorm_codes(x_row, gamma, beta, step, bits, signed, eps):
    """Fig. 5(a) in exact rational arithmetic: code = Qn + #{k : (x-mu)/sigma*gamma+beta > (k-1/2) step}, the
    square root avoided by comparing signed squares of exact rationals.  Also returns the smallest relative
    distance of any comparison from a tie."""
    qn, qp = vo.code_range(bits, signed)
    xs = [Fraction(float(v)) for v in x_row]
    n = len(xs)
    mu = sum(xs) / n
    var = sum((v - mu) ** 2 for v in xs) / n + Fraction(float(np.float32(eps)))
    codes, margin = [], 1.0
    for j, v in enumerate(xs):
        g, b = Fraction(float(gamma[j])), Fraction(float(beta[j]))
        code = qn
        for k in range(qn + 1, qp + 1):
            s = (Fraction(k) - Fraction(1, 2)) * Fraction(float(step))
            lhs = (v - mu) * g                 # (x - mu) * gamma  >  (s - beta) * sigma  ?
            rhs_over_sigma = s - b
            sq = lambda t: t * abs(t)          # strictly increasing: compares like t itself
            a, c = sq(lhs), sq(rhs_over_sigma) * var
            if a > c:
                code += 1
            scale = max(abs(a), abs(c), Fraction(1, 10 ** 30))
            margin = min(margin, float(abs(a - c) / scale))
        codes.append(code)
    return codes, margin


def test_layernorm_comparator_hand_worked_row():
    # x = 1, 2, 3, 4: Eq. 5 gives mu = 1, 1.5, 2, 2.5 and S = 0, 0.5, 2, 5, all exact in binary fp.
    # variance 5/4, z = (x - 2.5)/sqrt(1.25) = -1.342, -0.447, 0.447, 1.342; step 1/2, 3 bits:
    # z/step = -2.68, -0.89, 0.89, 2.68 -> levels -3, -1, 1, 3.
    x = np.array([[1, 2, 3, 4]], np.float32)
    ref, neg, flip = vo.layernorm_references(np.ones(4), np.zeros(4), 0.5, 3, True, 4)
    q, mu, v = vo.layernorm_compare_quantize(x, ref, neg, flip, 0.0, 3, True, want_stats=True)
    assert mu[0] == np.float32(2.5) and v[0] == np.float32(5.0)
    assert q.tolist() == [[-3, -1, 1, 3]]
    # the references themselves: c_k = (k - 1/2)/2 for k = -3..3, ref = c^2/4
    want = [((k - 0.5) * 0.5) ** 2 / 4 for k in range(-3, 4)]
    assert np.allclose(ref[0], np.array(want, np.float32), rtol=0, atol=0)
    assert neg[0].tolist() == [1, 1, 1, 1, 0, 0, 0]
    # epsilon enters as n*eps added to S: x = 0, 2 has S = 2 (variance 1); eps = 3 makes the variance 4,
    # z = -1/2, 1/2, and with step 0.3 (boundaries +-0.15, +-0.45, +-0.75, -1.05) the levels are -2, 2;
    # without eps z = -1, 1 gives -3, 3
    x = np.array([[0, 2]], np.float32)
    ref, neg, flip = vo.layernorm_references(np.ones(2), np.zeros(2), 0.3, 3, True, 2)
    q, mu, v = vo.layernorm_compare_quantize(x, ref, neg, flip, 3.0, 3, True, want_stats=True)
    assert v[0] == np.float32(8.0) and q.tolist() == [[-2, 2]]
    assert vo.layernorm_compare_quantize(x, ref, neg, flip, 0.0, 3, True).tolist() == [[-3, 3]]


def test_layernorm_comparator_is_strict_on_exact_ties():
    # x = 0, 2: Eq. 5 gives mu = 0, 1 and S = 0, 2 exactly; variance 1 (eps = 0), so z = -1, 1 exactly.
    # With step 2 the boundaries (k - 1/2)*2 = ..., -3, -1, 1, 3 hit z: the comparator is '>' as drawn, so
    # z = 1 stays at level 0 (not above the boundary 1) and z = -1 at level -1 (not above -1, above -3).
    x = np.array([[0, 2]], np.float32)
    ref, neg, flip = vo.layernorm_references(np.ones(2), np.zeros(2), 2.0, 3, True, 2)
    q = vo.layernorm_compare_quantize(x, ref, neg, flip, 0.0, 3, True)
    assert q.tolist() == [[-1, 0]]
    # a gain a hair above one moves z = 1 over its boundary (z = -1 moves away from -1, downwards: no change);
    # a gain a hair below one moves z = -1 over its boundary instead
    g = np.full(2, np.nextafter(np.float32(1), np.float32(2)), np.float32)
    ref2, neg2, flip2 = vo.layernorm_references(g, np.zeros(2), 2.0, 3, True, 2)
    assert vo.layernorm_compare_quantize(x, ref2, neg2, flip2, 0.0, 3, True).tolist() == [[-1, 1]]
    g = np.full(2, np.nextafter(np.float32(1), np.float32(0)), np.float32)
    ref3, neg3, flip3 = vo.layernorm_references(g, np.zeros(2), 2.0, 3, True, 2)
    assert vo.layernorm_compare_quantize(x, ref3, neg3, flip3, 0.0, 3, True).tolist() == [[0, 0]]


@pytest.mark.parametrize("bits,signed", [(2, True), (3, True), (4, True), (4, False)])
def test_layernorm_comparator_against_exact_rational_direct_formula(bits, signed):
    rng = np.random.default_rng(2504 + bits)
    rows, cols = 6, 24
    x = rng.normal(0.3, 1.7, (rows, cols)).astype(np.float32)
    gamma = rng.normal(1.0, 0.3, cols).astype(np.float32)
    gamma[3] = -gamma[3]                     # a negative gain flips the comparison
    gamma[11] = -0.7
    beta = rng.normal(0.0, 0.4, cols).astype(np.float32)
    step = np.float32(0.37)
    eps = 1e-5
    ref, neg, flip = vo.layernorm_references(gamma, beta, step, bits, signed, cols)
    assert flip[3] == 1 and flip[11] == 1 and flip.sum() == 2
    q = vo.layernorm_compare_quantize(x, ref, neg, flip, eps, bits, signed)
    checked = 0
    for r in range(rows):
        want, margin = _direct_layernorm_codes(x[r], gamma, beta, step, bits, signed, eps)
        if margin > 1e-4:                    # fp32 statistics move a comparison only this close to a tie
            assert q[r].tolist() == want, r
            checked += 1
    assert checked >= rows - 1


def test_layernorm_comparator_equals_layernorm_then_round_off_ties():
    cfg = si.VIT_BASE_LAYER.with_(batch=1)
    prm = si.layer_parameters(cfg)
    x = si.activations(cfg)[:24]
    y, tol = vo.layernorm(x, prm["ln1_g"], prm["ln1_b"], 1e-6)
    s = np.float32(prm["s_ln"])
    ref, neg, flip = vo.layernorm_references(prm["ln1_g"], prm["ln1_b"], s, cfg.bits, True, x.shape[1])
    q = vo.layernorm_compare_quantize(x, ref, neg, flip, 1e-6, cfg.bits, True)
    # the plain path: fp64 LayerNorm, round to nearest, clamp (numpy, not the oracle's quantizer)
    qn, qp = vo.code_range(cfg.bits, True)
    u = y.astype(np.float64) / float(s)
    plain = np.clip(np.rint(u), qn, qp).astype(np.int16)
    frac = np.abs(u - np.floor(u) - 0.5)
    clear = frac > 1e-3                      # away from a rounding boundary both rules give the same level
    assert clear.mean() > 0.99
    assert np.array_equal(q[clear], plain[clear])
    assert np.abs(q.astype(int) - plain.astype(int)).max() <= 1


def test_layernorm_comparator_invariances_on_exact_data():
    # integers: every step of Eq. 5 that matters stays exact enough that a shift of all inputs by a constant
    # or a scaling by a power of two (eps = 0) leaves the statistics' ratios, hence every level, unchanged
    rng = np.random.default_rng(77)
    x = rng.integers(-8, 9, (5, 16)).astype(np.float32)
    gamma = np.ones(16, np.float32)
    beta = np.zeros(16, np.float32)
    ref, neg, flip = vo.layernorm_references(gamma, beta, 0.3, 4, True, 16)
    q0 = vo.layernorm_compare_quantize(x, ref, neg, flip, 0.0, 4, True)
    q1 = vo.layernorm_compare_quantize(x * 4.0, ref, neg, flip, 0.0, 4, True)
    assert np.array_equal(q0, q1)
    for r in range(5):
        want, margin = _direct_layernorm_codes(x[r] + 64.0, gamma, beta, np.float32(0.3), 4, True, 0.0)
        got = vo.layernorm_compare_quantize((x[r:r + 1] + 64.0), ref, neg, flip, 0.0, 4, True)
        if margin > 1e-4:
            assert got[0].tolist() == want


def test_layernorm_comparator_brute_force_tiny_rows():
    # every row of three values from {-2..2}: exact rational decision vs the oracle (2-bit levels)
    vals = [-2.0, -1.0, 0.0, 1.0, 2.0]
    gamma = np.array([1.0, 0.5, -1.5], np.float32)
    beta = np.array([0.25, -0.5, 0.0], np.float32)
    step = np.float32(0.75)
    ref, neg, flip = vo.layernorm_references(gamma, beta, step, 2, True, 3)
    rows = np.array(list(itertools.product(vals, repeat=3)), np.float32)
    q = vo.layernorm_compare_quantize(rows, ref, neg, flip, 1e-3, 2, True)
    n_checked = 0
    for r in range(rows.shape[0]):
        want, margin = _direct_layernorm_codes(rows[r], gamma, beta, step, 2, True, 1e-3)
        if margin > 1e-5:
            assert q[r].tolist() == want, rows[r]
            n_checked += 1
    assert n_checked > 100


# ---------------------------------------------------------------------------
# band helpers: the tolerances the GPU tests grant must be the stated ones, and narrow
# ---------------------------------------------------------------------------

def test_quantize_band_hand_rows_exact_rationals():
    """vo_quantize_band against exact rational arithmetic: codes of y, y - tol and y + tol under the a1 rule
    (one fp32 subtraction / addition, one fp32 division, ties to even, clamp), including a tie that sits exactly
    at y + tol and one exactly at y - tol."""
    step = np.float32(0.25)
    #            y       tol      (y - tol)/s   (y + tol)/s
    rows = [(0.300, 0.000, ),   # 1.2 -> 1, band 1..1
            (0.350, 0.025, ),   # 1.3 .. 1.5: upper end exactly on the tie 1.5 -> even 2
            (0.400, 0.025, ),   # 1.5 (tie -> 2) .. 1.7 -> 2
            (0.650, 0.025, ),   # 2.5 (tie -> 2) .. 2.7 -> 3
            (-0.13, 0.010, ),   # -0.56 -> -1 .. -0.48 -> 0
            (5.000, 0.500, ),   # clamps at +7
            (-9.00, 4.000, )]   # clamps at -8 on both ends
    y = np.array([[r[0] for r in rows]], np.float32)
    tol = np.array([[r[1] for r in rows]], np.float32)
    q, lo, hi = vo.quantize_band(y, tol, step, 4, True)

    def code(fr):
        v = f32_from_fraction(fr / Fraction(float(step)))
        n = int(np.rint(np.float64(v)))                      # rint of an fp32 value: ties to even
        return max(-8, min(7, n))

    for j in range(len(rows)):
        yj, tj = Fraction(float(y[0, j])), Fraction(float(tol[0, j]))
        lo_in = Fraction(float(f32_from_fraction(yj - tj)))
        hi_in = Fraction(float(f32_from_fraction(yj + tj)))
        assert int(q[0, j]) == code(yj), j
        assert int(lo[0, j]) == code(lo_in), j
        assert int(hi[0, j]) == code(hi_in), j
    # with power-of-two friendly numbers the ties are exact: 0.375/0.25 = 1.5 -> 2 and 0.625/0.25 = 2.5 -> 2
    yy = np.array([[0.25, 0.75]], np.float32)
    tt = np.array([[0.125, 0.125]], np.float32)
    q, lo, hi = vo.quantize_band(yy, tt, step, 4, True)
    assert q.tolist() == [[1, 3]] and lo.tolist() == [[0, 2]] and hi.tolist() == [[2, 4]]


def test_layernorm_tolerance_formula_and_band_is_narrow():
    """The tolerance array of vo_layernorm is 8 * 2^-24 * (|gamma| * max_row|x - mu| / sigma + |beta|), evaluated
    here in Python on two rows; on ViT-Base-shaped rows the band of codes it induces is at most one code wide and
    touches fewer than one code in a thousand."""
    cols = 8
    x = np.array([[1.0, 2.0, 3.0, 4.0, -2.0, 0.5, 7.0, 0.5], [10.0, 10.5, 9.5, 10.25, 9.75, 10.0, 11.0, 9.0]], np.float32)
    g = np.array([1.0, -0.5, 2.0, 0.25, 1.5, 1.0, 0.75, 3.0], np.float32)
    b = np.array([0.0, 0.1, -0.2, 0.3, 0.0, -1.0, 0.5, 0.05], np.float32)
    eps = 1e-6
    y, tol = vo.layernorm(x, g, b, eps)
    for r in range(2):
        xs = [Fraction(float(v)) for v in x[r]]
        mu = sum(xs) / cols
        var = sum((v - mu) ** 2 for v in xs) / cols
        sigma = math.sqrt(float(var) + float(np.float32(eps)))
        maxdev = max(abs(float(v - mu)) for v in xs)
        for k in range(cols):
            want = 8.0 * 2.0 ** -24 * (abs(float(g[k])) * maxdev / sigma + abs(float(b[k])))
            assert abs(float(tol[r, k]) - want) <= 2e-7 * want, (r, k)
            yk = float(xs[k] - mu) / sigma * float(g[k]) + float(b[k])
            assert abs(float(y[r, k]) - yk) <= 1e-6 * max(1.0, abs(yk))
    cfg = si.VIT_BASE_LAYER.with_(batch=2)
    prm = si.layer_parameters(cfg)
    xa = si.activations(cfg)
    ya, ta = vo.layernorm(xa, prm["ln1_g"], prm["ln1_b"], 1e-6)
    assert ta.max() < 1e-5 and ta.min() > 0
    for bits in (4, 3, 2):
        q, lo, hi = vo.quantize_band(ya, ta, si.gaussian_lsq_step(1.0, bits), bits, True)
        assert np.all(lo <= q) and np.all(q <= hi) and np.all(hi - lo <= 1)
        assert (hi != lo).mean() < 1e-3


def test_softmax_band_is_the_two_ulp_neighbourhood():
    """q_lo / q_hi of vo_softmax_quantize are the codes of p moved by two units in the last place, nothing wider:
    recomputed here with numpy's nextafter and an fp32 division."""
    rows, cols = 16, 197
    S = ((si.splitmix64(91, rows * cols) % np.uint64(801)).astype(np.int64) - 400).astype(np.int32).reshape(rows, cols)
    c, s_p = np.float32(0.0123), np.float32(2.0 / (cols * math.sqrt(15.0)))
    p, q, lo, hi = vo.softmax_quantize(S, c, s_p, 4)
    dn, up = p.copy(), p.copy()
    for _ in range(2):
        dn = np.nextafter(dn, np.float32(-np.inf))
        up = np.nextafter(up, np.float32(np.inf))
    dn = np.maximum(dn, np.float32(0))
    code = lambda v: np.clip(np.rint((v / s_p).astype(np.float32)), 0, 15).astype(np.int16)
    assert np.array_equal(lo, code(dn)) and np.array_equal(hi, code(up)) and np.array_equal(q, code(p))
    assert np.all(hi - lo <= 1) and (hi != lo).mean() < 2e-3


def test_o_band_from_p_band_is_the_brute_force_extreme():
    """Every choice of P codes inside [p_lo, p_hi] is enumerated on a tiny case (3 keys, 2 channels, intervals up to
    two codes wide): the smallest and largest O codes found are exactly what the helper returns, with V of both
    signs.  A helper that took the wrong end of the interval for negative V, or transposed V, fails here."""
    import itertools
    T, d, n = 3, 2, 2
    rng = np.random.RandomState(5)
    p_lo = rng.randint(0, 12, size=(n, T, T)).astype(np.int16)
    p_hi = (p_lo + rng.randint(0, 3, size=(n, T, T))).astype(np.int16)
    v = rng.randint(-8, 8, size=(n, T, d)).astype(np.int16)
    v[0, 0, 0], v[0, 1, 0], v[1, 2, 1] = -7, 6, -8
    alpha = np.array([0.11, 0.07], np.float32)
    zero = np.zeros(d, np.float32)
    lo, hi = vp.o_band_from_p_band(p_lo, p_hi, v, alpha, 4)
    lo, hi = lo.reshape(n, T, d), hi.reshape(n, T, d)
    widened = 0
    for b in range(n):
        for i in range(T):
            best_lo, best_hi = np.full(d, 99), np.full(d, -99)
            for row in itertools.product(*[range(p_lo[b, i, j], p_hi[b, i, j] + 1) for j in range(T)]):
                acc = np.array([[sum(int(row[j]) * int(v[b, j, c]) for j in range(T)) for c in range(d)]], np.int32)
                o = vo.epilogue_requant(acc, alpha, zero, 4, True)[0]
                best_lo, best_hi = np.minimum(best_lo, o), np.maximum(best_hi, o)
            assert np.array_equal(best_lo, lo[b, i]) and np.array_equal(best_hi, hi[b, i]), (b, i)
            widened += int((best_hi > best_lo).sum())
    assert widened > 0                                   # the case is not degenerate
    # an interval of zero width gives the code itself
    lo0, hi0 = vp.o_band_from_p_band(p_lo, p_lo, v, alpha, 4)
    want = vo.epilogue_requant(vo.pv(p_lo, v).reshape(n * T, d), alpha, zero, 4, True)
    assert np.array_equal(lo0, want) and np.array_equal(hi0, want)


def test_stagewise_layer_equals_the_free_running_layer_on_its_own_values():
    """encoder_layer_stagewise() fed with the free-running oracle's own stage values reproduces every stage of
    encoder_layer() bit for bit (both softmax forms, both LayerNorm forms); fed with a perturbed upstream stage it
    follows the perturbation, i.e. it really computes each stage from what it is given."""
    cfg = si.VIT_TINY_BLOCK.with_(batch=1, tokens=37, mlp_dim=256)
    T, H, bits = cfg.tokens, cfg.heads, cfg.bits
    prm = si.layer_parameters(cfg)
    x = si.activations(cfg)
    for softmax, layernorm in (("exp", "fp32"), ("shift", "compare")):
        st = vp.encoder_layer(x, prm, cfg.batch, T, H, bits, softmax=softmax, layernorm=layernorm)
        att = st["attn"]
        given = {"x1": st["x1_codes"], "qkv": att["qkv_codes"], "P": att["p_codes"], "O": att["o_codes"], "h": st["h"],
                 "x2": st["x2_codes"], "g": st["g_codes"]}
        sw = vp.encoder_layer_stagewise(x, prm, cfg.batch, T, H, bits, given, softmax=softmax, layernorm=layernorm)
        assert np.array_equal(sw["x1_codes"], st["x1_codes"]) and np.array_equal(sw["qkv_codes"], att["qkv_codes"])
        assert np.array_equal(sw["p_codes"], att["p_codes"]) and np.array_equal(sw["o_codes"], att["o_codes"])
        assert np.array_equal(sw["h"].view(np.uint32), st["h"].view(np.uint32))
        assert np.array_equal(sw["x2_codes"], st["x2_codes"]) and np.array_equal(sw["g_codes"], st["g_codes"])
        assert np.array_equal(sw["out"].view(np.uint32), st["out"].view(np.uint32))
        # without given P the O band contains the exact O
        g2 = dict(given, P=None)
        sw2 = vp.encoder_layer_stagewise(x, prm, cfg.batch, T, H, bits, g2, softmax=softmax, layernorm=layernorm)
        assert np.all(sw2["o_lo"] <= att["o_codes"]) and np.all(att["o_codes"] <= sw2["o_hi"])
        # a changed upstream stage changes what the next stage must be
        g3 = dict(given, x1=np.where(st["x1_codes"] < 7, st["x1_codes"] + 1, st["x1_codes"]).astype(st["x1_codes"].dtype))
        sw3 = vp.encoder_layer_stagewise(x, prm, cfg.batch, T, H, bits, g3, softmax=softmax, layernorm=layernorm)
        assert not np.array_equal(sw3["qkv_codes"], att["qkv_codes"])
        assert np.array_equal(sw3["x1_codes"], st["x1_codes"])      # LayerNorm 1 still comes from x
