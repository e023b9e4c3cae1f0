"""Plain fp64 CPU oracle of the Text-to-Semantic GPT decode step.  TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline / reference arm of ``bench.py``
may import this module.  It shares no code with the CUDA library and never calls it.

What it follows.  The paper (Section II-A) describes the module as a decoder-only autoregressive
GPT in the GPT-2 family that emits semantic codec tokens; Section II-C fixes how it is fed (a
conditioning prefix of embeddings, then tokens that receive a positional embedding from their own
range of the position table) and what it must return at every step (token id, logits and the
hidden state of the last layer); the caption of Table I and Section III-B state that W8A16 /
W4A16 weight-only quantization is applied to it.  The paper prints no dimensions, equations or
worked numbers for the network, so the block below is the textbook pre-LayerNorm GPT-2 block in
fp64 with these readings (LN eps 1e-5 inside the square root with
biased variance, tanh-GELU, bias on every linear, rows [Q;K;V] head-major, scale 1/sqrt(head_dim),
causal mask, untied LM head, hidden = output of the final LayerNorm).

Pins (tests/test_oracle_pins.py): cached decode == full causal recompute; whole forward == a
composition of torch float64 library routines; closed forms and invariants of LayerNorm, GELU,
softmax/attention; exact int8/int4 round trips; sampling special cases and frequencies; prefix
assembly against a worked example with hand-made tables and its invariants.
Parity with the paper's trained model itself is unpinned: the paper prints no value to pin to.

Every function works on float64 numpy arrays.  bf16 inputs arrive as uint16 bit patterns and are
widened exactly.
"""
from __future__ import annotations

import math
import numpy as np

W_BF16, W_INT8_PC, W_INT4_G128 = 0, 1, 2
KV_BF16, KV_FP8_E4M3 = 0, 1


# ---------------------------------------------------------------------------------------------
# exact widening and dequantization (weight-only formats of Table I's caption)
# ---------------------------------------------------------------------------------------------
def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit pattern -> the real number it denotes, as float64 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def unpack_int4(words: np.ndarray) -> np.ndarray:
    """int32 words [N, K/8] -> nibbles u[N, K] in 0..15; column k = 8w + j sits in bits 4j..4j+3
    of word w."""
    w = np.ascontiguousarray(words).view(np.uint32)
    n, kw = w.shape
    u = np.empty((n, kw, 8), dtype=np.int64)
    for j in range(8):
        u[:, :, j] = (w >> np.uint32(4 * j)) & np.uint32(15)
    return u.reshape(n, kw * 8)


def pack_int4(u: np.ndarray) -> np.ndarray:
    """Inverse of unpack_int4 (used by the round-trip pin)."""
    n, k = u.shape
    uu = np.asarray(u, dtype=np.uint32).reshape(n, k // 8, 8)
    w = np.zeros((n, k // 8), dtype=np.uint32)
    for j in range(8):
        w += uu[:, :, j] * np.uint32(1 << (4 * j))
    return w.view(np.int32)


def dequant_int8_pc(q: np.ndarray, s_bits: np.ndarray) -> np.ndarray:
    """W[n,k] = s[n] * q[n,k]  (per-output-channel scale, exact in fp64)."""
    return bf16_to_f64(s_bits)[:, None] * np.asarray(q, dtype=np.int8).astype(np.float64)


def dequant_int4_g128(words: np.ndarray, s_bits: np.ndarray, group: int = 128) -> np.ndarray:
    """W[n,k] = s[n, k // 128] * (u[n,k] - 8)."""
    u = unpack_int4(words).astype(np.float64) - 8.0
    s = bf16_to_f64(s_bits)
    return u * np.repeat(s, group, axis=1)


def dequant(wfmt: int, w, s) -> np.ndarray:
    if wfmt == W_BF16:
        return bf16_to_f64(w)
    if wfmt == W_INT8_PC:
        return dequant_int8_pc(w, s)
    if wfmt == W_INT4_G128:
        return dequant_int4_g128(w, s)
    raise ValueError("unknown weight format")


# ---------------------------------------------------------------------------------------------
# 8-bit KV cache (a precision variant beyond Table I: the cached K and V rows as e4m3 codes)
# ---------------------------------------------------------------------------------------------
E4M3_MAX = 448.0


def e4m3_decode(code: int) -> float:
    """Value of an OCP e4m3 code (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities,
    S.1111.111 is NaN): the format's definition, bit by bit."""
    code = int(code) & 0xFF
    sign = -1.0 if code & 0x80 else 1.0
    e, m = (code >> 3) & 0xF, code & 0x7
    if e == 0xF and m == 0x7:
        return float("nan")
    if e == 0:
        return sign * (m / 8.0) * 2.0 ** -6          # subnormal
    return sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)


def e4m3_round(x: np.ndarray) -> np.ndarray:
    """Nearest e4m3 value (ties to the even mantissa), saturating at +-448: the grid spacing is 2^(e-3)
    for 2^e <= |x| < 2^(e+1), e clamped below at -6 (subnormal spacing 2^-9)."""
    x = np.asarray(x, dtype=np.float64)
    a = np.minimum(np.abs(x), E4M3_MAX)
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.clip(e, -6, 8)
    step = 2.0 ** (e - 3)
    q = np.rint(a / step) * step                     # numpy rounds half to even; a / step is exact
    return np.sign(x) * np.minimum(q, E4M3_MAX)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 value (ties to even) of each entry, returned as float64."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


def kv_quant_dequant(row: np.ndarray, head_dim: int) -> np.ndarray:
    """What an e4m3 KV cache returns for a K or V row [d].  The row is first rounded to bf16 (what the
    16-bit cache would hold); every head's head_dim values then share one scale s = max|x| / 448 (1 if the
    slice is zero), each value is stored as the e4m3 code nearest to x / s and read back as code * s.
    Which code represents a value is a decision taken in one precision on both sides of a comparison:
    scale and quotient are formed in fp32, as a kernel forms them."""
    row = np.asarray(row, dtype=np.float64)
    x = bf16_round(row).astype(np.float32).reshape(-1, head_dim)
    amax = np.abs(x).max(axis=1, keepdims=True)
    s = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    q = (x / s).astype(np.float32)
    return (e4m3_round(q.astype(np.float64)) * s.astype(np.float64)).reshape(row.shape)


# ---------------------------------------------------------------------------------------------
# elementwise pieces
# ---------------------------------------------------------------------------------------------
def layer_norm(x: np.ndarray, g: np.ndarray, b: np.ndarray, eps: float) -> np.ndarray:
    """LayerNorm over the last axis: biased variance, eps inside the square root."""
    mu = x.mean(axis=-1, keepdims=True)
    xc = x - mu
    var = (xc * xc).mean(axis=-1, keepdims=True)
    return xc / np.sqrt(var + eps) * g + b


def gelu_tanh(x: np.ndarray) -> np.ndarray:
    """GPT-2's GELU: 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))."""
    return 0.5 * x * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x * x * x)))


_erf = np.vectorize(math.erf, otypes=[np.float64])


def gelu_erf(x: np.ndarray) -> np.ndarray:
    """Exact GELU: x * Phi(x)."""
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def softmax(s: np.ndarray) -> np.ndarray:
    """Softmax over the last axis, computed after subtracting the row maximum."""
    e = np.exp(s - s.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


# ---------------------------------------------------------------------------------------------
# model
# ---------------------------------------------------------------------------------------------
class OracleModel:
    """All tensors of the decoder as float64 (block linears dequantized exactly from the packed
    form the CUDA library is given)."""

    def __init__(self, cfg, weights: dict):
        c = cfg if isinstance(cfg, dict) else cfg.as_dict()
        self.n_layer = int(c["n_layer"]); self.d = int(c["d_model"]); self.n_head = int(c["n_head"])
        self.head_dim = int(c["head_dim"]); self.d_ff = int(c["d_ff"]); self.vocab = int(c["vocab"])
        self.eps = float(c["ln_eps"]); self.gelu_is_tanh = bool(c["gelu_tanh"])
        self.kv_fmt = int(c.get("kv_fmt", KV_BF16))
        wfmt = int(c["wfmt"])
        assert self.n_head * self.head_dim == self.d
        f = bf16_to_f64
        self.tok_emb = f(weights["tok_emb"]); self.pos_emb = f(weights["pos_emb"])
        self.lnf_g = f(weights["lnf_g"]); self.lnf_b = f(weights["lnf_b"])
        self.head_w = f(weights["head_w"])
        self.head_b = None if weights.get("head_b") is None else f(weights["head_b"])
        self.layers = []
        for l in range(self.n_layer):
            lay = {}
            for k in ("ln1_g", "ln1_b", "ln2_g", "ln2_b"):
                lay[k] = f(weights[k][l])
            for lin in ("qkv", "o", "fc1", "fc2"):
                lay[lin + "_w"] = dequant(wfmt, weights[lin + "_w"][l], weights[lin + "_s"][l])
                lay[lin + "_b"] = f(weights[lin + "_b"][l])
            self.layers.append(lay)

    def gelu(self, x):
        return gelu_tanh(x) if self.gelu_is_tanh else gelu_erf(x)

    def cached(self, row):
        """A K or V row as the cache hands it back: unchanged, or through the e4m3 encoding."""
        return kv_quant_dequant(row, self.head_dim) if self.kv_fmt == KV_FP8_E4M3 else row

    def token_row(self, token: int, pos: int) -> np.ndarray:
        """Input row of a generated token: its embedding plus the positional embedding of its
        index in the semantic-token range (Section II-C)."""
        return self.tok_emb[int(token)] + self.pos_emb[int(pos)]


def assemble_prefix(model: OracleModel, cond_rows: np.ndarray, text_ids, text_shift: int,
                    text_pos0: int) -> np.ndarray:
    """Prefix rows of one utterance (Section II-C, the three input adaptations): the conditioning
    embeddings come first and are used as given, with no positional embedding; text token j follows
    as row ``text_ids[j] + text_shift`` of the merged embedding table (the text region of the table
    starts after the semantic codes, so the shift is their number) plus row ``text_pos0 + j`` of the
    position table (text tokens count positions in a range of their own).  Returns
    [n_cond + n_text, d] float64."""
    cond_rows = np.asarray(cond_rows, dtype=np.float64).reshape(-1, model.d)
    rows = [cond_rows[i].copy() for i in range(cond_rows.shape[0])]
    for j, t in enumerate(text_ids):
        rows.append(model.tok_emb[int(t) + int(text_shift)] + model.pos_emb[int(text_pos0) + j])
    return np.stack(rows) if rows else np.zeros((0, model.d))


class OracleStream:
    """One utterance: per-layer K/V kept in fp64, one row appended per step."""

    def __init__(self, model: OracleModel):
        self.m = model
        self.k = [[] for _ in range(model.n_layer)]   # lists of [d] rows
        self.v = [[] for _ in range(model.n_layer)]
        self.ctx = 0

    def step(self, x_row: np.ndarray):
        """Push one input row through every block using the cache.  Returns (logits[V], hidden[d])
        where hidden is the final-LayerNorm output the LM head reads."""
        m = self.m
        x = np.asarray(x_row, dtype=np.float64).copy()
        H, hd = m.n_head, m.head_dim
        for l, lay in enumerate(m.layers):
            a = layer_norm(x, lay["ln1_g"], lay["ln1_b"], m.eps)
            z = lay["qkv_w"] @ a + lay["qkv_b"]
            q, kt, vt = z[0:m.d], z[m.d:2 * m.d], z[2 * m.d:3 * m.d]
            self.k[l].append(m.cached(kt)); self.v[l].append(m.cached(vt))
            K = np.stack(self.k[l]); V = np.stack(self.v[l])          # [t+1, d]
            o = np.empty(m.d)
            for h in range(H):
                sl = slice(h * hd, (h + 1) * hd)
                s = (K[:, sl] @ q[sl]) / math.sqrt(hd)
                p = softmax(s)
                o[sl] = p @ V[:, sl]
            x = x + lay["o_w"] @ o + lay["o_b"]
            a = layer_norm(x, lay["ln2_g"], lay["ln2_b"], m.eps)
            h1 = m.gelu(lay["fc1_w"] @ a + lay["fc1_b"])
            x = x + lay["fc2_w"] @ h1 + lay["fc2_b"]
        self.ctx += 1
        hf = layer_norm(x, m.lnf_g, m.lnf_b, m.eps)
        logits = m.head_w @ hf
        if m.head_b is not None:
            logits = logits + m.head_b
        return logits, hf


def forward_full(model: OracleModel, X: np.ndarray):
    """Brute-force companion with no cache: all T input rows of one utterance through every block
    with an explicit T x T causal mask.  Returns (logits[T,V], hidden[T,d]).  Row t of the result
    is what ``OracleStream.step`` returns for the t-th row fed."""
    m = model
    x = np.asarray(X, dtype=np.float64).copy()
    T = x.shape[0]
    H, hd = m.n_head, m.head_dim
    allowed = np.tril(np.ones((T, T), dtype=bool))
    for lay in m.layers:
        a = layer_norm(x, lay["ln1_g"], lay["ln1_b"], m.eps)
        z = a @ lay["qkv_w"].T + lay["qkv_b"]
        q, k, v = z[:, 0:m.d], z[:, m.d:2 * m.d], z[:, 2 * m.d:3 * m.d]
        if m.kv_fmt == KV_FP8_E4M3:
            k = np.stack([m.cached(k[t]) for t in range(T)])
            v = np.stack([m.cached(v[t]) for t in range(T)])
        o = np.empty((T, m.d))
        for h in range(H):
            sl = slice(h * hd, (h + 1) * hd)
            s = (q[:, sl] @ k[:, sl].T) / math.sqrt(hd)
            s = np.where(allowed, s, -np.inf)
            o[:, sl] = softmax(s) @ v[:, sl]
        x = x + o @ lay["o_w"].T + lay["o_b"]
        a = layer_norm(x, lay["ln2_g"], lay["ln2_b"], m.eps)
        h1 = m.gelu(a @ lay["fc1_w"].T + lay["fc1_b"])
        x = x + h1 @ lay["fc2_w"].T + lay["fc2_b"]
    hf = layer_norm(x, m.lnf_g, m.lnf_b, m.eps)
    logits = hf @ m.head_w.T
    if m.head_b is not None:
        logits = logits + m.head_b
    return logits, hf


# ---------------------------------------------------------------------------------------------
# sampling (Section I lists sampling among the decode engine's parts; the rule itself is a reading)
# ---------------------------------------------------------------------------------------------
def sample_greedy(logits: np.ndarray) -> int:
    """Smallest index attaining the maximum logit."""
    return int(np.argmax(logits))


def topk_order(logits: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest logits sorted by (logit descending, index ascending)."""
    idx = np.lexsort((np.arange(logits.shape[0]), -np.asarray(logits, dtype=np.float64)))
    return idx[:k]


def topk_cdf(logits: np.ndarray, k: int, temperature: float):
    """(indices I, cumulative probabilities c) of the top-k distribution:
    w_r = exp((logit[I_r] - logit[I_0]) / T), c_r = (w_0 + .. + w_r) / sum w."""
    I = topk_order(logits, k)
    w = np.exp((np.asarray(logits, dtype=np.float64)[I] - float(logits[I[0]])) / float(temperature))
    c = np.cumsum(w) / w.sum()
    return I, c


def sample_topk(logits: np.ndarray, k: int, temperature: float, u: float) -> int:
    """Inverse-CDF draw: the first rank r with u < c_r (u in [0,1)); the last rank if rounding
    leaves none."""
    I, c = topk_cdf(logits, k, temperature)
    for r in range(len(I)):
        if u < c[r]:
            return int(I[r])
    return int(I[-1])


def sample(logits: np.ndarray, top_k: int, temperature: float, u: float) -> int:
    if top_k <= 1:
        return sample_greedy(logits)
    return sample_topk(logits, top_k, temperature, u)


def top2_gap(logits: np.ndarray) -> float:
    """Gap between the largest and second-largest logit (decides whether a greedy mismatch is
    excused)."""
    part = np.partition(np.asarray(logits, dtype=np.float64), -2)[-2:]
    return float(part[1] - part[0])


# ---------------------------------------------------------------------------------------------
# drivers used by tests and the CPU-baseline timing
# ---------------------------------------------------------------------------------------------
def run_stream(model: OracleModel, prefix_rows: np.ndarray, n_decode: int, top_k: int = 0,
               temperature: float = 1.0, uniforms=None, pos0: int = 0, forced_tokens=None):
    """Prefill the prefix rows one by one, sample y_0 from the last prefix row, then take
    ``n_decode`` decode steps.  Step k (1-based) consumes y_{k-1} at position pos0 + k - 1.

    ``uniforms[0]`` is used for y_0 and ``uniforms[k]`` for y_k.  With ``forced_tokens``
    (length n_decode + 1: y_0..y_n) the inputs follow that sequence instead of the oracle's own
    samples (replay mode); the oracle's own choices are still returned.

    Returns dict(tokens=[y_0..y_n] chosen by the oracle, logits=[n+1, V], hidden=[n+1, d]).
    """
    st = OracleStream(model)
    logits = hid = None
    for p in range(prefix_rows.shape[0]):
        logits, hid = st.step(prefix_rows[p])
    u = (lambda i: 0.0) if uniforms is None else (lambda i: float(uniforms[i]))
    toks = [sample(logits, top_k, temperature, u(0))]
    all_logits = [logits]; all_hidden = [hid]
    for kstep in range(1, n_decode + 1):
        y_prev = toks[-1] if forced_tokens is None else int(forced_tokens[kstep - 1])
        logits, hid = st.step(model.token_row(y_prev, pos0 + kstep - 1))
        toks.append(sample(logits, top_k, temperature, u(kstep)))
        all_logits.append(logits); all_hidden.append(hid)
    return {"tokens": np.array(toks, dtype=np.int64), "logits": np.stack(all_logits),
            "hidden": np.stack(all_hidden)}


def replay_full(model: OracleModel, prefix_rows: np.ndarray, tokens, pos0: int = 0):
    """Replay mode through the no-cache forward: given y_0..y_{n-1} (the inputs of decode steps
    1..n), return the logits and hidden rows of the last prefix position and of every decode
    step: arrays [n+1, V] and [n+1, d]."""
    rows = [np.asarray(prefix_rows, dtype=np.float64)]
    if len(tokens):
        rows.append(np.stack([model.token_row(int(t), pos0 + i) for i, t in enumerate(tokens)]))
    X = np.concatenate(rows, axis=0)
    logits, hid = forward_full(model, X)
    P = prefix_rows.shape[0]
    return logits[P - 1:], hid[P - 1:]
