"""Pins of the fp64 oracle to things other than itself: closed forms, invariants, textbook
values, an independent scalar-loop decoder, and a composition of torch float64 library routines.
A dropped term, a wrong sign or index, or a transposed operand in the oracle fails one of them."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import gpt_oracle as O
from paper_2607_21042_b200 import cases as C

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            a, b = line.split()
            rows.append((float(a), float(b)))
    return rows


# ---------------------------------------------------------------------------------------------
# elementwise pieces
# ---------------------------------------------------------------------------------------------
def test_gelu_erf_matches_normal_table():
    for x, phi in _read_table("standard_normal_cdf.txt"):
        assert abs(O.gelu_erf(np.array([x]))[0] - x * phi) <= 6e-6 * max(1.0, x)


def test_gelu_tanh_matches_hand_values():
    for x, g in _read_table("gelu_tanh_values.txt"):
        assert abs(O.gelu_tanh(np.array([x]))[0] - g) <= 1e-6


def test_gelu_symmetry_and_zero():
    x = np.linspace(-6, 6, 241)
    for g in (O.gelu_tanh, O.gelu_erf):
        assert g(np.zeros(1))[0] == 0.0
        assert np.allclose(g(-x), g(x) - x, rtol=0, atol=1e-14)
    # the two variants differ, but by less than 5e-4 everywhere, and at 1.0 in the 4th decimal
    assert np.max(np.abs(O.gelu_tanh(x) - O.gelu_erf(x))) < 5e-4
    assert abs(O.gelu_erf(np.array([1.0]))[0] - 0.841345) < 1e-6


def test_layer_norm_moments_and_constant_row():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(5, 64)) * 3 + 2
    eps = 1e-5
    y = O.layer_norm(x, np.ones(64), np.zeros(64), eps)
    var = x.var(axis=1)           # biased
    assert np.allclose(y.mean(axis=1), 0, atol=1e-13)
    assert np.allclose(y.var(axis=1), var / (var + eps), rtol=1e-12)
    g = rng.normal(size=64); b = rng.normal(size=64)
    const = np.full((1, 64), 7.25)
    assert np.allclose(O.layer_norm(const, g, b, eps), b, atol=1e-12)
    # affine part: gamma multiplies, beta adds
    assert np.allclose(O.layer_norm(x, g, b, eps), y * g + b, atol=1e-12)
    # eps is inside the square root: a row with variance v scales by 1/sqrt(v+eps)
    tiny = np.array([[1e-3, -1e-3]])
    want = tiny / math.sqrt(1e-6 + eps)
    assert np.allclose(O.layer_norm(tiny, np.ones(2), np.zeros(2), eps), want, rtol=1e-12)


def test_layer_norm_vs_torch():
    rng = np.random.default_rng(2)
    x = rng.normal(size=(3, 40)); g = rng.normal(size=40); b = rng.normal(size=40)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x), (40,), torch.from_numpy(g),
                                         torch.from_numpy(b), 1e-5).numpy()
    assert np.max(np.abs(O.layer_norm(x, g, b, 1e-5) - ref)) < 1e-12


def test_softmax_invariants():
    rng = np.random.default_rng(3)
    s = rng.normal(size=(7, 33)) * 4
    p = O.softmax(s)
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-12)
    assert np.allclose(O.softmax(s + 123.456), p, atol=1e-13)
    assert O.softmax(np.array([[0.3]]))[0, 0] == 1.0
    # closed form for two scores: logistic of the difference
    assert abs(O.softmax(np.array([1.0, 3.0]))[1] - 1 / (1 + math.exp(-2.0))) < 1e-15


# ---------------------------------------------------------------------------------------------
# packed formats
# ---------------------------------------------------------------------------------------------
def test_bf16_widening_exact():
    bits = np.array([0x3F80, 0xBF80, 0x4000, 0x3DCD, 0x0000, 0x8000, 0x0080], dtype=np.uint16)
    want = [1.0, -1.0, 2.0, 0.10009765625, 0.0, -0.0, 2.0 ** -126]
    got = O.bf16_to_f64(bits)
    assert list(got) == want
    # generator's rounding and oracle's widening agree on exactly representable values
    x = np.array([0.5, -3.0, 1.5, 100.0], dtype=np.float32)
    assert np.array_equal(O.bf16_to_f64(C.f32_to_bf16_bits(x)), x.astype(np.float64))
    # round to nearest even at the halfway point: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert C.f32_to_bf16_bits(np.array([1.0 + 2.0 ** -8], np.float32))[0] == 0x3F80
    assert C.f32_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8], np.float32))[0] == 0x3F82


def test_int4_nibble_positions_scalar():
    # every nibble position, written bit by bit with Python integers
    for j in range(8):
        for val in (0, 15, 5):
            word = np.array([[np.uint32(val << (4 * j)).astype(np.uint32)]], dtype=np.uint32).view(np.int32)
            u = O.unpack_int4(word)
            want = [0] * 8
            want[j] = val
            assert list(u[0]) == want
    # a word with all eight distinct nibbles, high bit set (negative as int32)
    word = sum(((k + 8) & 15) << (4 * k) for k in range(8))
    u = O.unpack_int4(np.array([[word]], dtype=np.uint32).view(np.int32))
    assert list(u[0]) == [((k + 8) & 15) for k in range(8)]


def test_int4_int8_round_trip_exact():
    rng = np.random.default_rng(4)
    u = rng.integers(0, 16, size=(6, 256))
    u[0, :16] = np.arange(16)            # every code
    assert np.array_equal(O.unpack_int4(O.pack_int4(u)), u)
    assert np.array_equal(O.unpack_int4(C.pack_int4_words(u)), u)     # generator's packer too
    assert np.array_equal(O.pack_int4(u), C.pack_int4_words(u))
    q = rng.integers(-127, 128, size=(5, 64)).astype(np.int8)
    q[0, :3] = (-127, 127, 0)
    s = C.f32_to_bf16_bits(np.full(5, 0.5, np.float32))
    assert np.array_equal(O.dequant_int8_pc(q, s), q.astype(np.float64) * 0.5)


def test_quantizers_error_bound_and_extremes():
    rng = np.random.default_rng(5)
    wb = C.f32_to_bf16_bits((rng.normal(size=(16, 256)) * 0.02).astype(np.float32))
    w = O.bf16_to_f64(wb)
    q8, s8 = C.quantize_int8_per_channel(wb)
    assert q8.min() >= -127 and q8.max() <= 127
    d8 = O.dequant_int8_pc(q8, s8)
    s = O.bf16_to_f64(s8)[:, None]
    clamped = np.abs(np.rint(w / s)) > 127
    assert np.all((np.abs(d8 - w) <= s / 2 + 1e-15) | clamped)
    assert np.all(np.abs(q8).max(axis=1) >= 126)          # the row maximum maps to about +-127
    w4, s4 = C.quantize_int4_group128(wb)
    u = O.unpack_int4(w4)
    assert u.min() >= 0 and u.max() <= 15
    d4 = O.dequant_int4_g128(w4, s4)
    sg = np.repeat(O.bf16_to_f64(s4), 128, axis=1)
    r = np.rint(w / sg)
    clamped = (r > 7) | (r < -8)
    assert np.all((np.abs(d4 - w) <= sg / 2 + 1e-15) | clamped)
    # zero rows / groups get scale 1 and code 0
    z = np.zeros((2, 128), np.uint16)
    q, sc = C.quantize_int8_per_channel(z)
    assert np.all(q == 0) and np.all(O.bf16_to_f64(sc) == 1.0)
    q, sc = C.quantize_int4_group128(z)
    assert np.all(O.unpack_int4(q) == 8) and np.all(O.bf16_to_f64(sc) == 1.0)


def test_int4_group_scale_applies_to_its_columns():
    # all codes equal (q = +3); groups differ only in scale
    n, k = 3, 384
    u = np.full((n, k), 11)
    words = O.pack_int4(u)
    scales = np.array([[1.0, 2.0, 4.0], [0.5, 0.25, 8.0], [1.0, 1.0, 1.0]], np.float32)
    sb = C.f32_to_bf16_bits(scales)
    w = O.dequant_int4_g128(words, sb)
    for i in range(n):
        for g in range(3):
            assert np.all(w[i, 128 * g:128 * (g + 1)] == 3.0 * scales[i, g])


def test_dequant_linear_equals_scalar_loops():
    rng = np.random.default_rng(6)
    n, k = 5, 256
    wb = C.f32_to_bf16_bits((rng.normal(size=(n, k)) * 0.02).astype(np.float32))
    a = rng.normal(size=k)
    words, sb = C.quantize_int4_group128(wb)
    y = O.dequant_int4_g128(words, sb) @ a
    wu = words.view(np.uint32)
    for i in range(n):
        acc = 0.0
        for kk in range(k):
            nib = (int(wu[i, kk // 8]) >> (4 * (kk % 8))) & 15
            sc = float(O.bf16_to_f64(sb[i:i + 1, kk // 128:kk // 128 + 1])[0, 0])
            acc += sc * (nib - 8) * a[kk]
        assert abs(acc - y[i]) < 1e-12
    q8, s8 = C.quantize_int8_per_channel(wb)
    y8 = O.dequant_int8_pc(q8, s8) @ a
    for i in range(n):
        acc = sum(float(O.bf16_to_f64(s8[i:i + 1])[0]) * int(q8[i, kk]) * a[kk] for kk in range(k))
        assert abs(acc - y8[i]) < 1e-12


# ---------------------------------------------------------------------------------------------
# whole decoder: independent scalar implementation, torch composition, cache vs recompute
# ---------------------------------------------------------------------------------------------
def _toy_cfg(wfmt=C.W_BF16, **kw):
    base = dict(n_layer=2, d_model=128, n_head=2, head_dim=64, d_ff=256, vocab=37, wfmt=wfmt,
                max_pos=16)
    base.update(kw)
    return C.GPTConfig(**base)


def _scalar_decoder(cfg, w, X):
    """Pure-Python decoder written with scalar loops over explicit indices (lists of floats, no
    numpy arithmetic) — an independent implementation for tiny shapes.  Returns logits of every
    row."""
    def tolist(bits):
        return [float(v) for v in O.bf16_to_f64(np.asarray(bits)).ravel()]

    def weight(lin, l, n, k):
        wt = w[lin + "_w"][l]
        if cfg.wfmt == C.W_BF16:
            return float(O.bf16_to_f64(wt[n:n + 1, k:k + 1])[0, 0])
        if cfg.wfmt == C.W_INT8_PC:
            return float(O.bf16_to_f64(w[lin + "_s"][l][n:n + 1])[0]) * int(wt[n, k])
        word = int(wt.view(np.uint32)[n, k // 8])
        nib = (word >> (4 * (k % 8))) & 15
        return float(O.bf16_to_f64(w[lin + "_s"][l][n:n + 1, k // 128:k // 128 + 1])[0, 0]) * (nib - 8)

    def ln(x, g, b):
        n = len(x); mu = sum(x) / n
        var = sum((v - mu) ** 2 for v in x) / n
        return [(x[i] - mu) / math.sqrt(var + cfg.ln_eps) * g[i] + b[i] for i in range(n)]

    def linear(lin, l, a, n_out):
        bias = tolist(w[lin + "_b"][l])
        return [sum(weight(lin, l, n, k) * a[k] for k in range(len(a))) + bias[n] for n in range(n_out)]

    d, H, hd, F = cfg.d_model, cfg.n_head, cfg.head_dim, cfg.d_ff
    T = len(X)
    xs = [list(map(float, r)) for r in X]
    for l in range(cfg.n_layer):
        g1, b1 = tolist(w["ln1_g"][l]), tolist(w["ln1_b"][l])
        g2, b2 = tolist(w["ln2_g"][l]), tolist(w["ln2_b"][l])
        qkv = [linear("qkv", l, ln(xs[t], g1, b1), 3 * d) for t in range(T)]
        for t in range(T):
            o = [0.0] * d
            for h in range(H):
                sc = []
                for j in range(t + 1):
                    sc.append(sum(qkv[t][h * hd + e] * qkv[j][d + h * hd + e] for e in range(hd)) / 8.0)
                m = max(sc); ex = [math.exp(s - m) for s in sc]; z = sum(ex)
                for e in range(hd):
                    o[h * hd + e] = sum(ex[j] / z * qkv[j][2 * d + h * hd + e] for j in range(t + 1))
            proj = linear("o", l, o, d)
            xs[t] = [xs[t][i] + proj[i] for i in range(d)]
            h1 = linear("fc1", l, ln(xs[t], g2, b2), F)
            h1 = [0.5 * v * (1 + math.tanh(math.sqrt(2 / math.pi) * (v + 0.044715 * v ** 3))) for v in h1]
            mlp = linear("fc2", l, h1, d)
            xs[t] = [xs[t][i] + mlp[i] for i in range(d)]
    gf, bf = tolist(w["lnf_g"]), tolist(w["lnf_b"])
    hw = O.bf16_to_f64(w["head_w"])
    out = []
    for t in range(T):
        hf = ln(xs[t], gf, bf)
        out.append([sum(float(hw[v, k]) * hf[k] for k in range(d)) for v in range(cfg.vocab)])
    return np.array(out)


@pytest.mark.parametrize("wfmt", [C.W_BF16, C.W_INT8_PC, C.W_INT4_G128])
def test_oracle_equals_scalar_loop_decoder(wfmt):
    cfg = _toy_cfg(wfmt)
    w = C.make_weights(cfg, seed=11)
    X = O.bf16_to_f64(C.make_prefixes(cfg, [3], seed=11)[0])
    ref = _scalar_decoder(cfg, w, X)
    m = O.OracleModel(cfg, w)
    got, _ = O.forward_full(m, X)
    assert np.max(np.abs(got - ref)) < 1e-11
    st = O.OracleStream(m)
    for t in range(3):
        lg, _ = st.step(X[t])
        assert np.max(np.abs(lg - ref[t])) < 1e-11


def _torch_forward(cfg, m, X):
    """Composition of torch float64 library routines (layer_norm, linear,
    scaled_dot_product_attention with is_causal, gelu)."""
    F = torch.nn.functional
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    x = t(X)
    T = x.shape[0]
    for lay in m.layers:
        a = F.layer_norm(x, (m.d,), t(lay["ln1_g"]), t(lay["ln1_b"]), m.eps)
        z = F.linear(a, t(lay["qkv_w"]), t(lay["qkv_b"]))
        q, k, v = z.split(m.d, dim=1)
        sh = lambda u: u.reshape(T, m.n_head, m.head_dim).transpose(0, 1)
        o = F.scaled_dot_product_attention(sh(q), sh(k), sh(v), is_causal=True)
        o = o.transpose(0, 1).reshape(T, m.d)
        x = x + F.linear(o, t(lay["o_w"]), t(lay["o_b"]))
        a = F.layer_norm(x, (m.d,), t(lay["ln2_g"]), t(lay["ln2_b"]), m.eps)
        h = F.gelu(F.linear(a, t(lay["fc1_w"]), t(lay["fc1_b"])),
                   approximate="tanh" if m.gelu_is_tanh else "none")
        x = x + F.linear(h, t(lay["fc2_w"]), t(lay["fc2_b"]))
    hf = F.layer_norm(x, (m.d,), t(m.lnf_g), t(m.lnf_b), m.eps)
    return F.linear(hf, t(m.head_w)).numpy(), hf.numpy()


@pytest.mark.parametrize("gelu_tanh", [1, 0])
def test_oracle_equals_torch_composition_tiny_config(gelu_tanh):
    cfg = C.tiny_config(gelu_tanh=gelu_tanh)
    w = C.make_weights(cfg, seed=0)
    m = O.OracleModel(cfg, w)
    X = O.bf16_to_f64(C.make_prefixes(cfg, [70], seed=0)[0])
    ref_logits, ref_hid = _torch_forward(cfg, m, X)
    got_logits, got_hid = O.forward_full(m, X)
    assert np.max(np.abs(got_logits - ref_logits)) < 1e-10
    assert np.max(np.abs(got_hid - ref_hid)) < 1e-10


def test_cached_decode_equals_full_recompute_tiny_config():
    wl = C.workload(1)
    w = C.make_weights(wl.cfg, seed=0)
    m = O.OracleModel(wl.cfg, w)
    P = O.bf16_to_f64(C.make_prefixes(wl.cfg, wl.prefix_lens, seed=0)[0])
    run = O.run_stream(m, P, 32)
    lg, hid = O.replay_full(m, P, run["tokens"][:-1])
    assert lg.shape == run["logits"].shape
    assert np.max(np.abs(lg - run["logits"])) < 1e-10
    assert np.max(np.abs(hid - run["hidden"])) < 1e-10
    # replay with forced tokens reproduces the free run when fed its own tokens
    rep = O.run_stream(m, P, 32, forced_tokens=run["tokens"])
    assert np.array_equal(rep["tokens"], run["tokens"])


def test_cached_decode_equals_full_recompute_one_layer_one_head():
    cfg = C.GPTConfig(n_layer=1, d_model=64, n_head=1, head_dim=64, d_ff=128, vocab=19, max_pos=8)
    w = C.make_weights(cfg, seed=3)
    m = O.OracleModel(cfg, w)
    X = O.bf16_to_f64(C.make_prefixes(cfg, [9], seed=3)[0])
    full, _ = O.forward_full(m, X)
    st = O.OracleStream(m)
    for t in range(9):
        lg, _ = st.step(X[t])
        assert np.max(np.abs(lg - full[t])) < 1e-11


def test_attention_closed_forms():
    cfg = _toy_cfg()
    w = C.make_weights(cfg, seed=5)
    m = O.OracleModel(cfg, w)
    X = O.bf16_to_f64(C.make_prefixes(cfg, [6], seed=5)[0])
    lay = m.layers[0]
    # (a) one key: the attention output is the value row itself
    st = O.OracleStream(m)
    st.step(X[0])
    a = O.layer_norm(X[0], lay["ln1_g"], lay["ln1_b"], m.eps)
    v0 = (lay["qkv_w"] @ a + lay["qkv_b"])[2 * m.d:]
    x1 = X[0] + lay["o_w"] @ v0 + lay["o_b"]
    a2 = O.layer_norm(x1, lay["ln2_g"], lay["ln2_b"], m.eps)
    x1 = x1 + lay["fc2_w"] @ m.gelu(lay["fc1_w"] @ a2 + lay["fc1_b"]) + lay["fc2_b"]
    m1 = O.OracleModel(C.GPTConfig(**{**cfg.as_dict(), "n_layer": 1}),
                       {k: (v[:1] if isinstance(v, list) else v) for k, v in w.items()})
    lg, _ = O.OracleStream(m1).step(X[0])
    want = m1.head_w @ O.layer_norm(x1, m1.lnf_g, m1.lnf_b, m1.eps)
    assert np.max(np.abs(lg - want)) < 1e-12
    # (b) zero query weights and bias: uniform attention, output = mean of the cached values
    lay0 = m1.layers[0]
    lay0["qkv_w"][:m.d] = 0.0
    lay0["qkv_b"][:m.d] = 0.0
    st = O.OracleStream(m1)
    for t in range(6):
        st.step(X[t])
    V = np.stack(st.v[0])
    # recompute the last row by hand with o = mean(V)
    full, _ = O.forward_full(m1, X)
    x = X[5]
    x = x + lay0["o_w"] @ V.mean(axis=0) + lay0["o_b"]
    a2 = O.layer_norm(x, lay0["ln2_g"], lay0["ln2_b"], m.eps)
    x = x + lay0["fc2_w"] @ m1.gelu(lay0["fc1_w"] @ a2 + lay0["fc1_b"]) + lay0["fc2_b"]
    want = m1.head_w @ O.layer_norm(x, m1.lnf_g, m1.lnf_b, m1.eps)
    assert np.max(np.abs(full[5] - want)) < 1e-11


def test_streams_are_independent_and_positions_matter():
    cfg = C.tiny_config()
    w = C.make_weights(cfg, seed=0)
    m = O.OracleModel(cfg, w)
    assert np.array_equal(m.token_row(5, 3), m.tok_emb[5] + m.pos_emb[3])
    P = [O.bf16_to_f64(p) for p in C.make_prefixes(cfg, [5, 9], seed=7)]
    a = O.run_stream(m, P[0], 4)
    b = O.run_stream(m, P[1], 4)
    a2 = O.run_stream(m, P[0], 4)
    assert np.array_equal(a["logits"], a2["logits"])
    assert not np.array_equal(a["logits"][0], b["logits"][0])
    shifted = O.run_stream(m, P[0], 4, pos0=7)
    assert np.array_equal(shifted["logits"][0], a["logits"][0])        # prefix rows take no position
    assert not np.array_equal(shifted["logits"][1], a["logits"][1])


# ---------------------------------------------------------------------------------------------
# sampling
# ---------------------------------------------------------------------------------------------
def test_greedy_ties_take_lowest_index():
    lg = np.array([0.1, 2.0, -1.0, 2.0, 2.0])
    assert O.sample_greedy(lg) == 1
    assert O.sample(lg, 0, 1.0, 0.9) == 1 and O.sample(lg, 1, 1.0, 0.9) == 1
    assert list(O.topk_order(lg, 4)) == [1, 3, 4, 0]
    assert abs(O.top2_gap(np.array([0.0, 1.5, 1.25])) - 0.25) < 1e-15


def test_topk_special_cases():
    rng = np.random.default_rng(8)
    lg = rng.normal(size=200)
    order = np.argsort(-lg, kind="stable")
    assert O.sample_topk(lg, 30, 1.0, 0.0) == order[0]
    assert O.sample_topk(lg, 30, 1.0, np.nextafter(1.0, 0.0)) == order[29]
    # k = V, T = 1: plain softmax inverse CDF over the sorted order
    p = O.softmax(lg)[order]
    c = np.cumsum(p)
    for u in (0.05, 0.3, 0.62, 0.97):
        want = order[int(np.searchsorted(c, u, side="right"))]
        assert O.sample_topk(lg, 200, 1.0, u) == want
    # temperature: T -> small concentrates on the maximum; the CDF uses (l - l0)/T
    I, cdf = O.topk_cdf(lg, 5, 0.5)
    w = np.exp((lg[I] - lg[I[0]]) / 0.5)
    assert np.allclose(cdf, np.cumsum(w) / w.sum(), atol=1e-15)
    assert abs(cdf[-1] - 1.0) < 1e-15


def test_topk_frequencies_chi_square():
    lg = np.array([2.0, 1.0, 0.0, -1.0, 3.0, -5.0, 0.5])
    k = 5
    I, cdf = O.topk_cdf(lg, k, 1.0)
    p = np.diff(np.concatenate([[0.0], cdf]))
    us = C.make_uniforms(100000, 1, seed=9)[:, 0]
    counts = np.zeros(k)
    pos = {int(i): r for r, i in enumerate(I)}
    for u in us:
        counts[pos[O.sample_topk(lg, k, 1.0, float(u))]] += 1
    chi2 = ((counts - p * len(us)) ** 2 / (p * len(us))).sum()
    assert chi2 < 18.47         # 99.9 % quantile of chi-square with 4 degrees of freedom
    assert set(pos) == {4, 0, 1, 6, 2}


def _table_model(d=4, emb_rows=12, max_pos=20):
    # hand-made tables: element e of table row i is 10*i + e, of position row p is 1000*p + 100*e
    m = O.OracleModel.__new__(O.OracleModel)
    m.d = d
    m.tok_emb = 10.0 * np.arange(emb_rows)[:, None] + np.arange(d)[None, :]
    m.pos_emb = 1000.0 * np.arange(max_pos)[:, None] + 100.0 * np.arange(d)[None, :]
    return m


def test_assemble_prefix_worked_example():
    # Section II-C: 2 conditioning rows as given, then text ids (3, 0, 1) in a table whose text region
    # starts at row 7, text positions counted from row 5 of the position table
    m = _table_model()
    cond = np.array([[0.5, -1.0, 2.0, 4.0], [9.0, 8.0, 7.0, 6.0]])
    got = O.assemble_prefix(m, cond, [3, 0, 1], text_shift=7, text_pos0=5)
    want = np.array([
        [0.5, -1.0, 2.0, 4.0],
        [9.0, 8.0, 7.0, 6.0],
        [5100.0, 5201.0, 5302.0, 5403.0],     # table row 10 (100..103) + position row 5 (5000, 5100, 5200, 5300)
        [6070.0, 6171.0, 6272.0, 6373.0],     # table row 7 (70..73)    + position row 6
        [7080.0, 7181.0, 7282.0, 7383.0],     # table row 8 (80..83)    + position row 7
    ])
    assert got.shape == (5, 4) and np.array_equal(got, want)


def test_assemble_prefix_invariants():
    m = _table_model()
    rng = np.random.default_rng(3)
    cond = rng.normal(size=(3, 4))
    # no text: the conditioning rows come back untouched, whatever the position table holds
    assert np.array_equal(O.assemble_prefix(m, cond, [], 7, 5), cond)
    a = O.assemble_prefix(m, cond, [2, 4], 7, 5)
    m2 = _table_model(); m2.pos_emb = m2.pos_emb * 0.0
    b = O.assemble_prefix(m2, cond, [2, 4], 7, 5)
    assert np.array_equal(a[:3], b[:3]) and np.array_equal(a[:3], cond)      # no positional term on conditioning rows
    assert np.array_equal(a[3:] - b[3:], m.pos_emb[5:7])                     # text rows carry rows 5, 6 of the position table
    assert np.array_equal(b[3:], m.tok_emb[[9, 11]])                         # and rows id + shift of the merged table
    # the shift only relabels: ids + 1 with shift - 1 is the same prefix; so is a text range moved with the table
    assert np.array_equal(O.assemble_prefix(m, cond, [3, 5], 6, 5), a)
    m3 = _table_model(); m3.pos_emb = np.roll(m.pos_emb, 2, axis=0)
    assert np.array_equal(O.assemble_prefix(m3, cond, [2, 4], 7, 7), a)


def test_assembled_prefix_feeds_the_decoder_like_given_rows():
    # a stream opened from (conditioning rows, text ids) equals one opened from the assembled rows
    cfg = _toy_cfg(emb_rows=43)
    w = C.make_weights(cfg, seed=4)
    m = O.OracleModel(cfg, w)
    rng = np.random.default_rng(5)
    cond = rng.normal(size=(3, cfg.d_model)) * 0.02
    shift = m.tok_emb.shape[0] - 6
    rows = O.assemble_prefix(m, cond, [1, 5, 0, 2], shift, 9)
    assert rows.shape == (7, cfg.d_model)
    run = O.run_stream(m, rows, 3, pos0=2)
    # position matters: the same ids counted from another text position give other logits
    other = O.run_stream(m, O.assemble_prefix(m, cond, [1, 5, 0, 2], shift, 10), 3, pos0=2)
    assert np.abs(run["logits"] - other["logits"]).max() > 1e-6


# ---------------------------------------------------------------------------------------------
# e4m3 KV cache
# ---------------------------------------------------------------------------------------------
def test_e4m3_decode_matches_hand_worked_codes():
    # sign | exponent (bias 7) | mantissa, worked by hand from the format's definition
    assert O.e4m3_decode(0x00) == 0.0
    assert O.e4m3_decode(0x01) == 2.0 ** -9            # smallest subnormal
    assert O.e4m3_decode(0x07) == 7 * 2.0 ** -9
    assert O.e4m3_decode(0x08) == 2.0 ** -6            # smallest normal
    assert O.e4m3_decode(0x38) == 1.0
    assert O.e4m3_decode(0x3C) == 1.5
    assert O.e4m3_decode(0x40) == 2.0
    assert O.e4m3_decode(0x7E) == 448.0                # largest finite: 1.75 * 2^8
    assert O.e4m3_decode(0xBC) == -1.5
    assert np.isnan(O.e4m3_decode(0x7F)) and np.isnan(O.e4m3_decode(0xFF))


def test_e4m3_round_is_the_identity_on_every_code_and_nearest_elsewhere():
    vals = np.array(sorted({O.e4m3_decode(c) for c in range(256) if not np.isnan(O.e4m3_decode(c))}))
    assert len(vals) == 253                                     # 254 finite codes, +0 and -0 coincide
    assert np.array_equal(O.e4m3_round(vals), vals)
    # nearest value by brute force over the whole grid, on a dense set of points (ties excluded here)
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.uniform(-448, 448, 4000), rng.uniform(-1, 1, 4000), rng.uniform(-0.02, 0.02, 4000)])
    near = vals[np.argmin(np.abs(x[:, None] - vals[None, :]), axis=1)]
    assert np.array_equal(O.e4m3_round(x), near)
    # ties go to the even mantissa: the midpoint of 1.0 (mantissa 0) and 1.125 (mantissa 1) is 1.0625 -> 1.0;
    # the midpoint of 1.125 and 1.25 (mantissa 2) -> 1.25; same in the subnormal range
    assert O.e4m3_round(np.array([1.0625]))[0] == 1.0
    assert O.e4m3_round(np.array([1.1875]))[0] == 1.25
    assert O.e4m3_round(np.array([1.5 * 2.0 ** -9]))[0] == 2.0 ** -8
    # saturation, sign symmetry, monotonicity
    assert O.e4m3_round(np.array([1e6, -1e6, 460.0]))[0] == 448.0 and O.e4m3_round(np.array([-1e6]))[0] == -448.0
    xs = np.sort(x)
    assert np.all(np.diff(O.e4m3_round(xs)) >= 0)
    assert np.array_equal(O.e4m3_round(-x), -O.e4m3_round(x))


def test_e4m3_round_matches_the_library_cast():
    # torch's float8_e4m3fn cast is an independent implementation of the same rounding (in range)
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.uniform(-448, 448, 20000), rng.standard_normal(20000) * 0.05]).astype(np.float32)
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    assert np.array_equal(O.e4m3_round(x.astype(np.float64)), lib)


def test_kv_quant_dequant_scale_per_head_slice_and_error_bound():
    rng = np.random.default_rng(2)
    row = O.bf16_round(rng.standard_normal(4 * 64) * np.repeat([0.01, 1.0, 30.0, 1e-6], 64))   # four heads of very different size
    y = O.kv_quant_dequant(row, 64)
    for h in range(4):
        x, z = row[64 * h:64 * h + 64], y[64 * h:64 * h + 64]
        s = float(np.float32(np.abs(x).max()) / np.float32(448.0))
        i = np.argmax(np.abs(x))
        assert np.isclose(z[i], x[i], rtol=2.0 ** -23)                             # the largest value is kept (up to the fp32 scale)
        # error at most half a grid step of the value's binade (relative 2^-4), or half the subnormal step
        assert np.all(np.abs(z - x) <= np.maximum(np.abs(x) * 2.0 ** -4, s * 2.0 ** -10) * (1 + 1e-6))
        codes = z / s
        assert np.array_equal(O.e4m3_round(codes), codes)                          # values sit on the grid of their head
    # scaling a head's slice by a power of two scales its decoded values exactly; other heads unchanged
    row2 = row.copy(); row2[64:128] *= 8.0
    y2 = O.kv_quant_dequant(row2, 64)
    assert np.array_equal(y2[64:128], 8.0 * y[64:128]) and np.array_equal(y2[:64], y[:64])
    assert np.array_equal(O.kv_quant_dequant(np.zeros(64), 64), np.zeros(64))
    # the row is taken as bf16: a perturbation below half a bf16 ulp changes nothing
    assert np.array_equal(O.kv_quant_dequant(row * (1 + 2.0 ** -12), 64), y)


def test_bf16_round_on_hand_written_cases():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, -3.0, 0.0, 2.0 ** -130])
    # 1 + 2^-8 is the midpoint of 1 and 1 + 2^-7: ties to the even mantissa (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    want = np.array([1.0, 1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, -3.0, 0.0, 2.0 ** -130])
    assert np.array_equal(O.bf16_round(x), want)
    rng = np.random.default_rng(3)
    y = rng.standard_normal(1000)
    r = O.bf16_round(y)
    assert np.all(np.abs(r - y) <= np.abs(y) * 2.0 ** -8) and np.array_equal(O.bf16_round(r), r)


def test_e4m3_cache_decoder_equals_recompute_and_plain_attention_on_decoded_rows():
    """With the 8-bit cache, cached decode still equals the no-cache recompute, and both equal ordinary
    attention run on explicitly encoded-and-decoded K and V rows."""
    cfg = C.tiny_config(kv_fmt=C.KV_FP8_E4M3)
    w = C.make_weights(cfg, seed=4)
    model = O.OracleModel(cfg, w)
    X = O.bf16_to_f64(C.make_prefixes(cfg, [20], seed=4)[0])
    st = O.OracleStream(model)
    rows = np.stack([st.step(X[t])[0] for t in range(X.shape[0])])
    full, _ = O.forward_full(model, X)
    assert np.max(np.abs(rows - full)) <= 1e-10
    # the cache holds decoded rows: every cached K row is a fixed point of the encoding
    for l in range(model.n_layer):
        for kt in st.k[l]:
            assert np.array_equal(O.kv_quant_dequant(kt, model.head_dim), kt)
    # and it differs from the exact cache by what the 2^-4 relative grid allows, not more
    plain = O.OracleModel(C.tiny_config(), w)
    exact, _ = O.forward_full(plain, X)
    diff = np.max(np.abs(full - exact))
    assert 0 < diff < 0.25
