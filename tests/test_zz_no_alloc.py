"""The allocation-free attention core: same results as the workspace-taking entry point.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.  The scratch of vitint_attention_core_noalloc is one fixed device array shared
by all calls, so the test calls it twice in a row with different scales (each call must rewrite
the table it needs) and compares each result, bit for bit, with vitint_attention_core given
ordinary scratch memory.
"""
import math

import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu
vt = pytest.importorskip("paper_2504_18547_b200")
from gpu_util import dev, rand_codes, to_codes  # noqa: E402


def test_noalloc_attention_core_matches_workspace_version_twice():
    batch, tokens, heads = 3, 197, 2
    D = heads * 64
    alpha = dev(np.full(D, 0.01, np.float32))
    beta = dev(si.normal(3, (D,), 0.0, 0.3))
    for call, (bits, scale, seed) in enumerate([(4, 1.0, 91), (4, 2.7, 92), (2, 1.5, 93)]):
        qkv = to_codes(rand_codes(seed, (batch * tokens, 3 * D), bits, True), bits, True)
        qmax = si.code_range(bits, True)[1] + 1
        s_q = s_k = float(np.float32(math.sqrt(8.0 * scale * 3.0 / (8.0 * qmax * qmax))))
        s_p = float(np.float32(2.0 / (tokens * math.sqrt(si.code_range(bits, False)[1]))))
        want = vt.vitint_attention_core(qkv, batch, heads, tokens, s_q, s_k, s_p, bits, alpha, beta)
        out = vt.Codes.empty(batch * tokens, D, bits, True)
        out.data.fill_(0xAA)
        got = vt.vitint_attention_core_noalloc(qkv, batch, heads, tokens, s_q, s_k, s_p, bits, alpha, beta, out)
        torch.cuda.synchronize()
        assert vt.vitint_device_status() == 0
        assert torch.equal(got.data, want.data), f"call {call}"
        assert len(torch.unique(want.data)) > 4


def test_noalloc_call_leaves_device_memory_as_it_found_it():
    """The property the entry point is named for: across a call (after the first one on the device, which looks the
    scratch array's address up) neither the framework's allocator nor the driver's free-memory figure moves."""
    batch, tokens, heads, bits = 2, 197, 2, 4
    D = heads * 64
    qkv = to_codes(rand_codes(77, (batch * tokens, 3 * D), bits, True), bits, True)
    alpha = dev(np.full(D, 0.01, np.float32))
    out = vt.Codes.empty(batch * tokens, D, bits, True)
    s_p = float(np.float32(2.0 / (tokens * math.sqrt(15.0))))
    vt.vitint_attention_core_noalloc(qkv, batch, heads, tokens, 0.2, 0.2, s_p, bits, alpha, None, out)   # warm-up
    torch.cuda.synchronize()
    before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    vt.vitint_attention_core_noalloc(qkv, batch, heads, tokens, 0.2, 0.2, s_p, bits, alpha, None, out)
    torch.cuda.synchronize()
    after = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    assert before == after
    assert vt.vitint_device_status() == 0


def test_noalloc_rejects_what_the_built_in_scratch_cannot_hold():
    batch, tokens, heads = 1, 64, 1
    qkv = to_codes(rand_codes(5, (batch * tokens, 3 * 64), 8, True), 8, True)
    out = vt.Codes.empty(batch * tokens, 64, 8, True)
    a = dev(np.ones(64, np.float32))
    with pytest.raises(vt.VitintError) as e:
        vt.vitint_attention_core_noalloc(qkv, batch, heads, tokens, 0.01, 0.01, 0.01, 8, a, None, out)
    assert e.value.code == -2                      # VITINT_ERR_UNSUPPORTED, exactly as vitint_attention_core reports 8-bit codes
    bad = vt.Codes.empty(batch * tokens, 3 * 64, 4, True)
    bad.bits = 5
    with pytest.raises(vt.VitintError) as e:
        vt.vitint_attention_core_noalloc(bad, batch, heads, tokens, 0.01, 0.01, 0.01, 4, a, None, out)
    assert e.value.code == -1                      # VITINT_ERR_INVALID_ARG: argument errors come first
