"""The allocation-free attention entry point against the ordinary one.

Some users of the library run where device allocation is not allowed (a request handler whose
memory was fixed at start-up, a plug-in inside an engine that owns the GPU's memory).  For them
`tts_gpt_op_attention_static` keeps its split-KV scratch in an array built into the library.  This
file checks, through the C ABI, that it returns what `tts_gpt_op_attention` returns — twice in a
row, because the built-in array still holds the first call's leftovers when the second one runs —
and that it refuses sizes beyond its stated limit.  It is named to be collected last, so a run that
stops at the first failure has already run everything else; it must also pass alone in a fresh
process (its first call is then the one that looks up the array's device address).
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2607_21042_b200 import binding as B
from paper_2607_21042_b200 import cases

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(seed, H, ctxs):
    rng = np.random.default_rng(seed)
    S, pps = len(ctxs), 32
    n_pages = sum((c + 63) // 64 for c in ctxs) + 2
    kv = cases.f32_to_bf16_bits(rng.standard_normal(size=(n_pages, 2, H, 64, 64)).astype(np.float32))
    perm = rng.permutation(n_pages)
    pt = np.zeros((S, pps), dtype=np.int32)
    nxt = 0
    for s, c in enumerate(ctxs):
        for p in range((c + 63) // 64):
            pt[s, p] = perm[nxt]; nxt += 1
    q = rng.standard_normal(size=(S, H * 64)).astype(np.float32)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    return (dev(q), dev(kv.view(np.int16)), dev(pt), dev(np.arange(S, dtype=np.int32)),
            dev(np.array([c - 1 for c in ctxs], dtype=np.int32)))


def test_static_scratch_attention_matches_caller_scratch_attention_twice():
    # first case: several chunks per row, so partials and tickets are really used
    a = _case(1, 20, [900, 2048, 257, 64, 1])
    # second case: different shape and lengths, runs on top of the first call's leftovers
    b = _case(2, 4, [513, 300, 1025, 2000, 77, 1500, 640])
    for args in (a, b):
        want = B.op_attention(*args)
        got = B.op_attention_static(*args)
        torch.cuda.synchronize()
        w = B.bf16_bits_tensor_to_f32(want).cpu().numpy()
        g = B.bf16_bits_tensor_to_f32(got).cpu().numpy()
        assert np.all(np.isfinite(g))
        # same kernel, same inputs: the tolerance the attention parity tests use (half a bf16 ulp
        # of the largest output plus fp32 noise) is met with room to spare — equality is expected
        assert np.max(np.abs(g - w)) <= 2.0 ** -8 * np.abs(w).max() + 1e-5
    # and once more on the first case, after the second has dirtied the array
    got = B.op_attention_static(*a)
    want = B.op_attention(*a)
    torch.cuda.synchronize()
    assert np.max(np.abs(B.bf16_bits_tensor_to_f32(got).cpu().numpy()
                         - B.bf16_bits_tensor_to_f32(want).cpu().numpy())) <= 2.0 ** -8 * 8 + 1e-5


def test_static_scratch_attention_rejects_sizes_beyond_its_limit():
    q, kv, pt, rs, rp = _case(3, 20, [10] * 65)            # 65 rows x 20 heads = 1300 > 1280
    with pytest.raises(B.TtsGptError) as e:
        B.op_attention_static(q, kv, pt, rs, rp)
    assert e.value.code == B.E_WORKSPACE
    assert "1280" in str(e.value)
    q, kv, pt, rs, rp = _case(4, 20, [10] * 64)            # exactly at the limit
    got = B.op_attention_static(q, kv, pt, rs, rp)
    want = B.op_attention(q, kv, pt, rs, rp)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
