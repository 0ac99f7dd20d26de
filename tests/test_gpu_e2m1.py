"""The FP4 (e2m1) tensor-core kind as an exact integer multiplier for very low-bit codes: brute force against the
integer oracle.  e2m1 holds 0, 1/2, 1, 3/2, 2, 3, 4, 6 and their negatives, so signed codes of up to 3 bits and
unsigned codes of up to 2 bits are exact operands; the question the tests answer is whether the fp32 accumulation of
their integer products inside the tensor core is exact too, for every code pair and up to the longest contraction
of the ViT-Base layer."""
import numpy as np
import pytest
import torch

import oracle as vo
import synth_inputs as si

pytestmark = pytest.mark.gpu
vt = pytest.importorskip("paper_2504_18547_b200")
from gpu_util import dev, rand_codes  # noqa: E402


def _bytes(q, bits, signed):
    """Codes stored one per byte, rows padded with zeros to a pitch of 16 bytes."""
    rows, cols = q.shape
    pitch = (cols + 15) // 16 * 16
    buf = np.zeros((rows, pitch), np.int8)
    buf[:, :cols] = q
    return vt.Codes(dev(buf).view(torch.uint8), rows, cols, bits, signed, 8)


def _run(qx, bx, sx, qw, bw, sw):
    acc, flag = vt.vitint_linear_e2m1(_bytes(qx, bx, sx), _bytes(qw, bw, sw))
    torch.cuda.synchronize()
    assert vt.vitint_device_status() == 0
    assert int(flag.item()) == 0, "an fp32 accumulator was not an integer"
    return acc.cpu().numpy()


@pytest.mark.parametrize("K", [64, 128, 192, 256, 320, 768, 1000, 3072])
@pytest.mark.parametrize("fmt", [((2, False), (2, True)), ((2, True), (2, True)), ((3, True), (3, True)), ((2, False), (3, True))],
                         ids=["u2xs2", "s2xs2", "s3xs3", "u2xs3"])
def test_every_code_pair_and_random_rows(fmt, K):
    """Row i of x holds one activation code in every column and row j of w one weight code, for every pair of codes:
    acc[i][j] = K * code_i * code_j, the largest sums the formats can produce included.  Further rows are random."""
    (bx, sx), (bw, sw) = fmt
    xn, xp = si.code_range(bx, sx)
    wn, wp = si.code_range(bw, sw)
    xs, ws = np.arange(xn, xp + 1), np.arange(wn, wp + 1)
    qx = np.concatenate([np.repeat(xs[:, None], K, axis=1), rand_codes(5 + K, (150, K), bx, sx)]).astype(np.int16)
    qw = np.concatenate([np.repeat(ws[:, None], K, axis=1), rand_codes(6 + K, (270, K), bw, sw)]).astype(np.int16)
    got = _run(qx, bx, sx, qw, bw, sw)
    want = vo.matmul_i32(qx, qw)
    assert np.array_equal(got, want)
    assert got[0, 0] == K * xn * wn and got[len(xs) - 1, len(ws) - 1] == K * xp * wp


def test_alternating_signs_and_cancellation():
    """Sums whose partial sums swing between large positive and negative values, and sums that cancel exactly."""
    K = 3072
    qx = np.full((4, K), 3, np.int16)
    qw = np.empty((3, K), np.int16)
    qw[0] = np.where(np.arange(K) % 2 == 0, -4, 3)
    qw[1, :K // 2], qw[1, K // 2:] = -4, 3
    qw[2] = np.where(np.arange(K) % 3 == 0, 1, -1)
    got = _run(qx, 2, False, qw, 3, True)
    assert np.array_equal(got, vo.matmul_i32(qx, qw))


def test_vit_base_two_bit_linears_match_the_int8_path():
    """The 2-bit configuration's own shapes: LayerNorm-output x weight (signed x signed, K = 768) and GELU-output x
    weight (unsigned x signed, K = 3072), against the oracle and against the int8 tensor-core path of vitint_linear."""
    for (M, K, N, bx, sx) in ((394, 768, 2304, 2, True), (394, 3072, 768, 2, False)):
        qx, qw = rand_codes(41 + K, (M, K), bx, sx), rand_codes(42 + K, (N, K), 2, True)
        got = _run(qx, bx, sx, qw, 2, True)
        assert np.array_equal(got, vo.matmul_i32(qx, qw))
        ref = vt.vitint_linear(_bytes(qx, bx, sx), 1.0, _bytes(qw, 2, True), None, None, vt.Epilogue(mode=vt.EPI_ACC_I32))
        assert np.array_equal(got, ref.cpu().numpy())


def test_rejects_codes_that_e2m1_cannot_hold():
    x4 = vt.Codes(torch.zeros((8, 64), dtype=torch.uint8, device="cuda"), 8, 64, 4, True, 8)
    u3 = vt.Codes(torch.zeros((8, 64), dtype=torch.uint8, device="cuda"), 8, 64, 3, False, 8)
    ok = vt.Codes(torch.zeros((8, 64), dtype=torch.uint8, device="cuda"), 8, 64, 2, True, 8)
    for bad in (x4, u3):
        with pytest.raises(vt.VitintError) as e:
            vt.vitint_linear_e2m1(bad, ok)
        assert e.value.code == -2
