"""Seeded synthetic inputs for the GPT decode step (weights, prefixes, uniforms, lengths).

This module only *draws and packs data*.  It holds none of the decoder's arithmetic: no
LayerNorm, attention, GELU, matmul, dequantization or sampling lives here, so both the CUDA
library's harness and the CPU oracle's tests can be fed from it without sharing any of the
method.  Everything is numpy; nothing here touches a GPU.

The paper evaluates on the Seed-TTS test sets with the trained IndexTTS-2 weights (Section III-A);
neither exists offline, so the five workloads below stand in for them with the same shapes: a
conditioning prefix of a few hundred embeddings (32 speaker latents + emotion + speed, then text;
Section II-C), a few hundred generated semantic tokens at 50 tokens per second of audio
(Section III-C), batch 1-16 concurrent utterances (Table III) and a batch of 128 beyond it.

bf16 tensors are carried as ``uint16`` bit patterns (numpy has no bf16).
"""
from __future__ import annotations

from dataclasses import dataclass, asdict, replace
import numpy as np

W_BF16, W_INT8_PC, W_INT4_G128 = 0, 1, 2
WFMT_NAMES = {W_BF16: "bf16", W_INT8_PC: "w8a16", W_INT4_G128: "w4a16"}

KV_BF16, KV_FP8_E4M3 = 0, 1
KV_NAMES = {KV_BF16: "bf16", KV_FP8_E4M3: "e4m3"}

TAG_WEIGHTS, TAG_PREFIX, TAG_UNIFORMS, TAG_LENGTHS = 1, 2, 3, 4


@dataclass(frozen=True)
class GPTConfig:
    n_layer: int
    d_model: int
    n_head: int
    head_dim: int
    d_ff: int
    vocab: int
    wfmt: int = W_BF16
    max_streams: int = 1
    max_context: int = 2048
    page_tokens: int = 64
    n_pages: int = 32
    max_pos: int = 1024
    gelu_tanh: int = 1
    stop_token: int = -1
    ln_eps: float = 1e-5
    emb_rows: int = 0       # rows of the merged embedding table (semantic codes, then text ids); 0 = vocab
    kv_fmt: int = 0         # KV cache: 0 = bf16, 1 = e4m3 codes with one scale per cached row and head

    @property
    def n_emb_rows(self) -> int:
        return self.emb_rows if self.emb_rows > 0 else self.vocab

    def as_dict(self):
        return asdict(self)


def tiny_config(**kw) -> GPTConfig:
    """Workload 1: 2 layers, d=256, 4 heads of 64, FFN 1024, vocab 1024."""
    base = GPTConfig(n_layer=2, d_model=256, n_head=4, head_dim=64, d_ff=1024, vocab=1024,
                     max_streams=4, max_context=2048, n_pages=4 * 32, max_pos=128)
    return replace(base, **kw)


def full_config(**kw) -> GPTConfig:
    """Workloads 2-5: 24 layers, d=1280, 20 heads of 64, FFN 5120, vocab 8194."""
    base = GPTConfig(n_layer=24, d_model=1280, n_head=20, head_dim=64, d_ff=5120, vocab=8194,
                     max_streams=1, max_context=2048, n_pages=32, max_pos=1024)
    return replace(base, **kw)


def rng_for(seed: int, tag: int) -> np.random.Generator:
    """Independent named sub-stream: PCG64 seeded by (seed, tag)."""
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), int(tag)])))


# ---------------------------------------------------------------------------------------------
# bf16 bit patterns
# ---------------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to the nearest bf16 (ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def _normal_bf16(rng, shape, std, mean=0.0):
    x = rng.standard_normal(size=shape, dtype=np.float32) * np.float32(std)
    if mean != 0.0:
        x = x + np.float32(mean)
    return f32_to_bf16_bits(x)


# ---------------------------------------------------------------------------------------------
# weight-only quantization of a drawn bf16 matrix (data preparation, not the decode path)
# ---------------------------------------------------------------------------------------------
def quantize_int8_per_channel(w_bits: np.ndarray):
    """Symmetric per-output-channel int8: s_n = bf16(max_k |W[n,k]| / 127) (1 if the row is zero),
    q = clamp(rint(W / s_n), -127, 127).  Returns (int8 [N,K], bf16-bit scales [N])."""
    w = bf16_bits_to_f64(w_bits)
    amax = np.abs(w).max(axis=1)
    s_bits = f32_to_bf16_bits((amax / 127.0).astype(np.float32))
    s = bf16_bits_to_f64(s_bits)
    zero = s == 0.0
    if zero.any():
        s_bits = s_bits.copy()
        s_bits[zero] = f32_to_bf16_bits(np.ones(1, np.float32))[0]
        s = bf16_bits_to_f64(s_bits)
    q = np.clip(np.rint(w / s[:, None]), -127, 127).astype(np.int8)
    return q, s_bits


def pack_int4_words(u: np.ndarray) -> np.ndarray:
    """Pack offset-binary nibbles u in [0,15], shape [N,K] (K % 8 == 0), into int32 words [N,K/8]:
    nibble j (bits 4j..4j+3) of word w holds column k = 8w + j."""
    n, k = u.shape
    assert k % 8 == 0
    u = u.astype(np.uint32).reshape(n, k // 8, 8)
    word = np.zeros((n, k // 8), dtype=np.uint32)
    for j in range(8):
        word |= u[:, :, j] << np.uint32(4 * j)
    return word.view(np.int32)


def quantize_int4_group128(w_bits: np.ndarray, group: int = 128):
    """Symmetric int4 with groups of 128 along K: s_{n,g} = bf16(max |W| / 7) over the group
    (1 if zero), q = clamp(rint(W / s), -8, 7), stored as u = q + 8.  Returns
    (int32 words [N,K/8], bf16-bit scales [N,K/128])."""
    w = bf16_bits_to_f64(w_bits)
    n, k = w.shape
    assert k % group == 0
    wg = w.reshape(n, k // group, group)
    amax = np.abs(wg).max(axis=2)
    s_bits = f32_to_bf16_bits((amax / 7.0).astype(np.float32))
    s = bf16_bits_to_f64(s_bits)
    zero = s == 0.0
    if zero.any():
        s_bits = s_bits.copy()
        s_bits[zero] = f32_to_bf16_bits(np.ones(1, np.float32))[0]
        s = bf16_bits_to_f64(s_bits)
    q = np.clip(np.rint(wg / s[:, :, None]), -8, 7).astype(np.int64)
    u = (q + 8).reshape(n, k)
    return pack_int4_words(u), s_bits


# ---------------------------------------------------------------------------------------------
# model weights
# ---------------------------------------------------------------------------------------------
LINEARS = ("qkv", "o", "fc1", "fc2")


def linear_shapes(cfg: GPTConfig):
    d, f = cfg.d_model, cfg.d_ff
    return {"qkv": (3 * d, d), "o": (d, d), "fc1": (f, d), "fc2": (d, f)}


def quantize_weights(w_bf16: dict, wfmt: int) -> dict:
    """Derive the packed W8A16 / W4A16 weight set from a bf16 draw of ``make_weights``: the four block
    linears of every layer are quantized, everything else is shared.  With W_BF16 the draw itself
    comes back."""
    if wfmt == W_BF16:
        return w_bf16
    if wfmt not in (W_INT8_PC, W_INT4_G128):
        raise ValueError("unknown weight format")
    quant = quantize_int8_per_channel if wfmt == W_INT8_PC else quantize_int4_group128
    out = dict(w_bf16)
    for lin in LINEARS:
        qs = [quant(wb) for wb in w_bf16[lin + "_w"]]
        out[lin + "_w"] = [q for q, _ in qs]
        out[lin + "_s"] = [s for _, s in qs]
    return out


def make_weights(cfg: GPTConfig, seed: int = 0) -> dict:
    """Draw every tensor of the decoder in a fixed order from the (seed, TAG_WEIGHTS) stream.

    Weights, embeddings and biases ~N(0, 0.02); LN gamma = 1 + N(0, 0.01); LN beta ~N(0, 0.01);
    all rounded to bf16.  For the quantized formats the four block linears are then quantized
    from those bf16 values; the LM head, embeddings, LN parameters and biases stay bf16.

    Returns a dict: 'tok_emb','pos_emb','lnf_g','lnf_b','head_w' and per-layer lists
    'ln1_g','ln1_b','ln2_g','ln2_b', '<lin>_w','<lin>_s','<lin>_b' for lin in qkv,o,fc1,fc2.
    '<lin>_s' entries are None for bf16.  The un-quantized bf16 draw of each quantized matrix is
    not kept (both sides consume the packed form only).
    """
    rng = rng_for(seed, TAG_WEIGHTS)
    d, v = cfg.d_model, cfg.vocab
    shapes = linear_shapes(cfg)
    w = {k: [] for k in ("ln1_g", "ln1_b", "ln2_g", "ln2_b")}
    for lin in LINEARS:
        for suf in ("_w", "_s", "_b"):
            w[lin + suf] = []
    w["tok_emb"] = _normal_bf16(rng, (cfg.n_emb_rows, d), 0.02)
    w["pos_emb"] = _normal_bf16(rng, (cfg.max_pos, d), 0.02)

    def put_linear(name):
        n, k = shapes[name]
        w[name + "_w"].append(_normal_bf16(rng, (n, k), 0.02))
        w[name + "_s"].append(None)
        w[name + "_b"].append(_normal_bf16(rng, (n,), 0.02))

    for _ in range(cfg.n_layer):
        w["ln1_g"].append(_normal_bf16(rng, (d,), 0.01, 1.0))
        w["ln1_b"].append(_normal_bf16(rng, (d,), 0.01))
        put_linear("qkv")
        put_linear("o")
        w["ln2_g"].append(_normal_bf16(rng, (d,), 0.01, 1.0))
        w["ln2_b"].append(_normal_bf16(rng, (d,), 0.01))
        put_linear("fc1")
        put_linear("fc2")
    w["lnf_g"] = _normal_bf16(rng, (d,), 0.01, 1.0)
    w["lnf_b"] = _normal_bf16(rng, (d,), 0.01)
    w["head_w"] = _normal_bf16(rng, (v, d), 0.02)
    w["head_b"] = None
    return quantize_weights(w, cfg.wfmt)


# ---------------------------------------------------------------------------------------------
# per-workload inputs
# ---------------------------------------------------------------------------------------------
def make_prefixes(cfg: GPTConfig, prefix_lens, seed: int = 0):
    """One bf16 [P_i, d] prefix of N(0,1) embeddings per stream (stands in for the 34
    conditioning embeddings + text embeddings + start token of Section II-C)."""
    rng = rng_for(seed, TAG_PREFIX)
    return [_normal_bf16(rng, (int(p), cfg.d_model), 1.0) for p in prefix_lens]


def make_uniforms(n_steps: int, n_streams: int, seed: int = 0) -> np.ndarray:
    """fp32 uniforms in [0,1), shape [n_steps, n_streams], for top-k sampling."""
    rng = rng_for(seed, TAG_UNIFORMS)
    return rng.random(size=(int(n_steps), int(n_streams)), dtype=np.float32)


@dataclass(frozen=True)
class Workload:
    name: str
    cfg: GPTConfig
    prefix_lens: tuple
    decode_lens: tuple        # decode_step calls per stream
    top_k: int                # 0 = greedy
    temperature: float = 1.0
    seed: int = 0

    @property
    def n_streams(self):
        return len(self.prefix_lens)


def draw_lengths(n_streams, p_lo, p_hi, n_lo=None, n_hi=None, max_context=2048, seed=0):
    """Prefix lengths: uniform integers in [p_lo, p_hi].  Decode lengths (if asked): uniform
    integers in [n_lo, min(n_hi, max_context - P_i)]."""
    rng = rng_for(seed, TAG_LENGTHS)
    p = rng.integers(p_lo, p_hi + 1, size=n_streams)
    if n_lo is None:
        return tuple(int(x) for x in p), None
    n = []
    for pi in p:
        hi = min(n_hi, max_context - int(pi))
        n.append(int(rng.integers(n_lo, hi + 1)))
    return tuple(int(x) for x in p), tuple(n)


def workload(idx: int, wfmt=None, seed: int = 0, kv_fmt: int = KV_BF16) -> Workload:
    """The five workloads (1-based, in the order the baseline lists them).  kv_fmt = KV_FP8_E4M3 gives the
    same workload on an 8-bit KV cache."""
    if kv_fmt != KV_BF16:
        wl = workload(idx, wfmt=wfmt, seed=seed)
        return replace(wl, name=wl.name + "_kv" + KV_NAMES[kv_fmt], cfg=replace(wl.cfg, kv_fmt=kv_fmt))
    if idx == 1:
        cfg = tiny_config(max_streams=1, n_pages=32)
        return Workload("cfg1_tiny_bf16_b1", cfg, (64,), (32,), 0, seed=seed)
    if idx == 2:
        cfg = full_config(wfmt=W_BF16, max_streams=1, n_pages=32)
        return Workload("cfg2_bf16_b1_p400_n500", cfg, (400,), (500,), 0, seed=seed)
    if idx == 3:
        cfg = full_config(wfmt=W_INT8_PC, max_streams=1, n_pages=32)
        return Workload("cfg3_w8a16_b1_p400_n500_topk30", cfg, (400,), (500,), 30, seed=seed)
    if idx == 4:
        p, _ = draw_lengths(16, 200, 800, seed=seed)
        cfg = full_config(wfmt=W_INT4_G128, max_streams=16, n_pages=16 * 32)
        return Workload("cfg4_w4a16_b16_p200-800_n500", cfg, p, (500,) * 16, 0, seed=seed)
    if idx == 5:
        p, n = draw_lengths(128, 200, 1200, 64, 1024, 2048, seed=seed)
        fmt = W_BF16 if wfmt is None else wfmt
        cfg = full_config(wfmt=fmt, max_streams=128, n_pages=128 * 32)
        return Workload("cfg5_%s_b128_ragged_drain" % WFMT_NAMES[fmt], cfg, p, n, 0, seed=seed)
    raise ValueError("workload index must be 1..5")
