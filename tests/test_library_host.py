"""CPU-only checks of the CUDA library's host side: it loads, exports every symbol the header
declares, and rejects bad arguments before anything is launched (no compute call is made)."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def L():
    from paper_2504_18547_b200.build import build_library
    build_library()
    import paper_2504_18547_b200.binding as b
    return b


def test_every_declared_symbol_is_exported(L):
    header = (ROOT / "include" / "vitint.h").read_text()
    names = set(re.findall(r"\b(vitint_[a-z_0-9]+)\s*\(", header))
    assert {"vitint_quantize", "vitint_linear", "vitint_qk", "vitint_pv", "vitint_softmax_quantize",
            "vitint_attention_block", "vitint_layernorm_quantize", "vitint_layernorm_compare_quantize"} <= names
    lib = L.lib()
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_status_strings_and_pitch(L):
    assert L.vitint_version() >= 100
    assert L.vitint_status_string(0) == "ok"
    assert "2^31" in L.vitint_status_string(-4)
    assert L.packed_pitch(197, 4) == 112 and L.packed_pitch(768, 4) == 384 and L.packed_pitch(768, 3) == 384
    assert L.packed_pitch(768, 2) == 192 and L.packed_pitch(5, 8) == 16 and L.packed_pitch(0, 4) == 0


def _codes(L, ptr, rows, cols, pitch, bits, signed=1):
    return L._Codes(ptr, rows, cols, pitch, bits, signed)


def test_argument_errors_are_caught_on_the_host(L):
    lib = L.lib()
    fake = 0x7000_0000_0000          # never dereferenced: all calls below fail validation first
    epi = L._Epilogue(0, 0, None, 0, None, None, None, 4, 1)
    ok_x = _codes(L, fake, 128, 256, 128, 4)
    ok_w = _codes(L, fake, 64, 256, 128, 4)
    out = ctypes.c_void_p(fake)
    br = ctypes.byref
    # null / bad descriptors
    assert lib.vitint_linear(None, 1.0, br(ok_w), None, None, br(epi), out, 64, None) == -1
    bad_bits = _codes(L, fake, 128, 256, 128, 5)
    assert lib.vitint_linear(br(bad_bits), 1.0, br(ok_w), None, None, br(epi), out, 64, None) == -1
    misaligned = _codes(L, fake + 4, 128, 256, 128, 4)
    assert lib.vitint_linear(br(misaligned), 1.0, br(ok_w), None, None, br(epi), out, 64, None) == -3
    bad_pitch = _codes(L, fake, 128, 256, 120, 4)
    assert lib.vitint_linear(br(bad_pitch), 1.0, br(ok_w), None, None, br(epi), out, 64, None) == -3
    short_pitch = _codes(L, fake, 128, 256, 112, 4)
    assert lib.vitint_linear(br(short_pitch), 1.0, br(ok_w), None, None, br(epi), out, 64, None) == -1
    # K mismatch
    w2 = _codes(L, fake, 64, 128, 64, 4)
    assert lib.vitint_linear(br(ok_x), 1.0, br(w2), None, None, br(epi), out, 64, None) == -1
    # output leading dimension too small
    assert lib.vitint_linear(br(ok_x), 1.0, br(ok_w), None, None, br(epi), out, 32, None) == -1
    # dequant without weight steps, requant without alpha
    deq = L._Epilogue(1, 0, None, 0, None, None, None, 4, 1)
    assert lib.vitint_linear(br(ok_x), 1.0, br(ok_w), None, None, br(deq), out, 64, None) == -1
    req = L._Epilogue(2, 0, None, 0, None, None, None, 4, 1)
    assert lib.vitint_linear(br(ok_x), 1.0, br(ok_w), None, None, br(req), out, 32, None) == -1
    # the int32 accumulator bound: 8-bit x 8-bit at K = 2^17 reaches 2^31
    K = 131072
    bx = _codes(L, fake, 128, K, K, 8)
    bw = _codes(L, fake, 64, K, K, 8)
    assert lib.vitint_linear(br(bx), 1.0, br(bw), None, None, br(epi), out, 64, None) == -4
    # quantize: non-positive step, wrong shape
    oc = _codes(L, fake, 10, 20, 16, 4)
    assert lib.vitint_quantize(ctypes.c_void_p(fake), 10, 20, 20, 0.0, None, br(oc), None) == -1
    assert lib.vitint_quantize(ctypes.c_void_p(fake), 10, 21, 21, 1.0, None, br(oc), None) == -1
    assert lib.vitint_quantize(ctypes.c_void_p(fake), 10, 20, 19, 1.0, None, br(oc), None) == -1
    # softmax: too many columns, signed output
    pc = _codes(L, fake, 4, 2000, 1008, 4, 0)
    assert lib.vitint_softmax_quantize(ctypes.c_void_p(fake), 4, 2000, 2000, 1.0, 1.0, br(pc), None, 0, None) == -2
    ps = _codes(L, fake, 4, 100, 64, 4, 1)
    assert lib.vitint_softmax_quantize(ctypes.c_void_p(fake), 4, 100, 100, 1.0, 1.0, br(ps), None, 0, None) == -1
    sl = L._Slabs(fake, 384, 384 * 300, 32, 4, 1)
    assert lib.vitint_qk(br(sl), br(sl), 1, 1, 300, out, 299, None) == -1      # ld_s < tokens
    sl_bad = L._Slabs(fake, 380, 384 * 100, 32, 4, 1)
    assert lib.vitint_qk(br(sl_bad), br(sl), 1, 1, 100, out, 100, None) == -3


def test_attention_workspace_query_and_errors(L):
    lib = L.lib()
    fake = 0x7000_0000_0000
    d = L._AttentionDesc()
    d.batch, d.tokens, d.heads, d.bits, d.p_bits = 2, 197, 3, 4, 4
    n = lib.vitint_attention_block_workspace_bytes(ctypes.byref(d))
    M, D = 2 * 197, 192
    expect_min = M * 288 + 2 * 3 * 197 * 200 * 4 + 2 * 3 * 197 * 112 + M * 96 + (2 * 4096 + 1) * 4 + 256
    assert expect_min <= n <= expect_min + 5 * 256
    assert lib.vitint_attention_core_workspace_bytes(4) == (2 * 4096 + 1) * 4 + 256
    assert lib.vitint_attention_core_workspace_bytes(3) == (2 * 4096 + 1) * 4 + 256
    assert lib.vitint_attention_core_workspace_bytes(2) == (2 * 256 + 1) * 4 + 256
    assert lib.vitint_attention_core_workspace_bytes(8) == 0
    d.batch = 0
    assert lib.vitint_attention_block_workspace_bytes(ctypes.byref(d)) == 0
    d.batch = 2
    x = _codes(L, fake, M, D, 96, 4)
    d.w_qkv = _codes(L, fake, 3 * D, D, 96, 4)
    d.w_proj = _codes(L, fake, D, D, 96, 4)
    d.alpha_qkv, d.alpha_o = fake, fake
    d.q_step = d.k_step = d.v_step = d.p_step = d.o_step = 0.1
    d.proj_epi = L._Epilogue(1, 0, None, 0, None, None, None, 4, 1)
    out = ctypes.c_void_p(fake)
    # no workspace / too small
    assert lib.vitint_attention_block(ctypes.byref(x), ctypes.byref(d), out, D, None, None, None, None, 0, None) == -5
    assert lib.vitint_attention_block(ctypes.byref(x), ctypes.byref(d), out, D, None, None, None,
                                      ctypes.c_void_p(fake), n - 1, None) == -5
    d.q_step = 0.0
    assert lib.vitint_attention_block(ctypes.byref(x), ctypes.byref(d), out, D, None, None, None,
                                      ctypes.c_void_p(fake), n, None) == -1


def test_product_fold_matches_definition(L):
    import numpy as np
    s_w = np.array([0.01, 0.02, 0.5], np.float32)
    b = np.array([0.1, -0.2, 0.0], np.float32)
    a, be = L.vitint_fold_requant(np.float32(0.3), s_w, b, np.float32(0.25))
    assert a.dtype == np.float32 and np.allclose(a, 0.3 * s_w / 0.25, rtol=1e-6)
    assert np.allclose(be, b / 0.25, rtol=1e-6)
    a2, be2 = L.vitint_fold_requant(np.float32(0.3), s_w, None, np.float32(0.25))
    assert np.array_equal(a, a2) and not be2.any()


def test_layernorm_reference_folding_matches_the_oracle_side(L):
    """The library's host-side folding of the comparator references (Fig. 5(b), a C entry point) and the oracle's are two separate
    pieces of code that must hand their sides the same numbers: magnitude, sign and flip flag, bit for bit."""
    import numpy as np
    import oracle as vo
    rng = np.random.default_rng(5)
    cols = 48
    gamma = rng.normal(1.0, 0.4, cols).astype(np.float32)
    gamma[[3, 17]] *= -1.0
    beta = rng.normal(0.0, 0.5, cols).astype(np.float32)
    for bits, signed in ((2, True), (3, True), (4, True), (4, False)):
        step = np.float32(0.31)
        ref, neg, flip = vo.layernorm_references(gamma, beta, step, bits, signed, cols)
        refs, flip_b = L.vitint_fold_layernorm_references(gamma, beta, step, bits, signed, cols)
        assert refs.shape == (cols, 2 ** bits - 1) and refs.dtype == np.float32
        assert np.array_equal(np.abs(refs).view(np.uint32), ref.view(np.uint32))
        assert np.array_equal(np.signbit(refs) & (refs != 0), (neg != 0) & (ref != 0))
        assert np.array_equal(flip_b, flip) and flip_b.sum() == 2
        assert np.all(np.diff(refs.astype(np.float64), axis=1) >= 0)      # ascending along the thresholds
