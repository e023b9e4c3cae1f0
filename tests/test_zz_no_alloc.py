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
import numpy as np
import pytest
import torch

from oracle import gpt_oracle as O
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


def _reference(args, H, rows):
    """softmax(q K^T / 8) V per head in fp64, written out, for the given rows of a case."""
    q, kv, pt, rs, rp = [t.cpu().numpy() for t in args]
    kvf = O.bf16_to_f64(kv.view(np.uint16))
    out = {}
    for r in rows:
        n = int(rp[r]) + 1
        K = np.concatenate([kvf[pt[rs[r], p], 0] for p in range((n + 63) // 64)], axis=1)[:, :n]   # [H, n, 64]
        V = np.concatenate([kvf[pt[rs[r], p], 1] for p in range((n + 63) // 64)], axis=1)[:, :n]
        o = np.empty(H * 64)
        for h in range(H):
            s = K[h] @ q[r, h * 64:(h + 1) * 64].astype(np.float64) / 8.0
            o[h * 64:(h + 1) * 64] = O.softmax(s) @ V[h]
        out[r] = o
    return out


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
    # against the definition itself, not only against the sibling entry point
    got = B.bf16_bits_tensor_to_f32(B.op_attention_static(*a)).cpu().numpy().astype(np.float64)
    torch.cuda.synchronize()
    for r, ref in _reference(a, 20, [0, 1, 4]).items():
        assert np.max(np.abs(got[r] - ref)) <= 2.0 ** -8 * np.abs(ref).max() + 1e-5, r
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
    # exactly at the limit, with several chunks in the first and the last row: the last partial slots and
    # the last ticket of the built-in array are used
    ctxs = [10] * 64
    ctxs[0], ctxs[63], ctxs[31] = 700, 1030, 300
    args = _case(4, 20, ctxs)
    got = B.op_attention_static(*args)
    want = B.op_attention(*args)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    g = B.bf16_bits_tensor_to_f32(got).cpu().numpy().astype(np.float64)
    for r, ref in _reference(args, 20, [0, 63]).items():
        assert np.max(np.abs(g[r] - ref)) <= 2.0 ** -8 * np.abs(ref).max() + 1e-5, r
