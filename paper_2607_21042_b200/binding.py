"""Thin ctypes binding of libtts_gpt.so: same names as the C ABI, argument marshalling only.

PyTorch is used for device memory and streams; every step of the decode path runs inside the
library's CUDA kernels.  If the shared library is missing or fails to load, ``load()`` raises:
there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from .cases import GPTConfig, LINEARS, W_BF16

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtts_gpt.so")

OK, E_ARG, E_NO_PAGES, E_STREAM, E_CTX_OVERFLOW, E_CUDA, E_TIMEOUT, E_WORKSPACE, E_UNSUPPORTED = \
    0, -1, -2, -3, -4, -5, -6, -7, -8

EXPORTS = [
    "tts_gpt_query_workspace", "tts_gpt_create", "tts_gpt_prefill", "tts_gpt_prefill_tokens", "tts_gpt_decode_step", "tts_gpt_decode_step_host", "tts_gpt_decode_steps",
    "tts_gpt_release_stream", "tts_gpt_sync", "tts_gpt_destroy", "tts_gpt_last_error",
    "tts_gpt_stats", "tts_gpt_stream_context", "tts_gpt_debug_shuffle_free_pages",
    "tts_gpt_debug_kernel_launches", "tts_gpt_debug_set_trace", "tts_gpt_debug_expire_wait", "tts_gpt_debug_set_option", "tts_gpt_debug_check_canaries",
    "tts_gpt_op_linear_packed_bytes", "tts_gpt_op_linear_pack", "tts_gpt_op_linear",
    "tts_gpt_op_linear_tc_scratch_bytes", "tts_gpt_op_linear_tc", "tts_gpt_op_attention_scratch_bytes", "tts_gpt_op_attention", "tts_gpt_op_attention_static", "tts_gpt_op_attention_cluster",
    "tts_gpt_op_layernorm",
    "tts_gpt_op_sample",
]


class TtsGptError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("tts_gpt error %d: %s" % (code, msg))
        self.code = code


class ConfigStruct(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layer", "d_model", "n_head", "head_dim", "d_ff", "vocab", "wfmt", "max_streams",
                 "max_context", "page_tokens", "n_pages", "max_pos", "gelu_tanh", "stop_token")] + \
               [("ln_eps", C.c_float), ("emb_rows", C.c_int32), ("kv_fmt", C.c_int32)]


_PP = C.POINTER(C.c_void_p)


class WeightsStruct(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("tok_emb", "pos_emb", "lnf_g", "lnf_b", "head_w", "head_b")] + \
               [(n, _PP) for n in ("ln1_g", "ln1_b", "ln2_g", "ln2_b",
                                   "qkv_w", "qkv_s", "qkv_b", "o_w", "o_s", "o_b",
                                   "fc1_w", "fc1_s", "fc1_b", "fc2_w", "fc2_s", "fc2_b")]


_lib = None


def load() -> C.CDLL:
    """Open the shared library (once).  Raises OSError if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError("%s not found: build it with `python -m paper_2607_21042_b200.build` "
                          "(no CPU fallback exists)" % LIB_PATH)
        lib = C.CDLL(LIB_PATH)
        lib.tts_gpt_last_error.restype = C.c_char_p
        lib.tts_gpt_last_error.argtypes = [C.c_void_p]
        for name in EXPORTS:
            if name != "tts_gpt_last_error":
                getattr(lib, name).restype = C.c_int32
        _lib = lib
    return _lib


def _check(rc, handle=None):
    if rc != OK:
        msg = load().tts_gpt_last_error(handle)
        raise TtsGptError(rc, msg.decode() if msg else "")
    return rc


def _ptr(t):
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, torch.Tensor):
        return C.c_void_p(t.data_ptr())
    return C.c_void_p(int(t))


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _i32_array(vals):
    return (C.c_int32 * len(vals))(*[int(v) for v in vals])


def to_device_bits(arr, device):
    """numpy array of bf16 bit patterns (uint16), int8 codes or int32 words -> device tensor."""
    if arr is None:
        return None
    if isinstance(arr, torch.Tensor):
        return arr.to(device)
    a = np.ascontiguousarray(arr)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(a).to(device)


def config_struct(cfg: GPTConfig) -> ConfigStruct:
    return ConfigStruct(**cfg.as_dict())


def query_workspace(cfg: GPTConfig) -> int:
    n = C.c_size_t(0)
    cs = config_struct(cfg)
    _check(load().tts_gpt_query_workspace(C.byref(cs), C.byref(n)))
    return n.value


class TtsGpt:
    """One engine on one GPU.  Methods mirror the C entry points."""

    def __init__(self, cfg: GPTConfig, weights: dict, device="cuda:0", stream=None):
        self.lib = load()
        self.cfg = cfg
        self.device = torch.device(device)
        self.handle = None
        torch.cuda.set_device(self.device)
        # The engine enqueues on a stream of its own (a non-default stream, so that the step can be
        # captured into a CUDA graph).  Work the caller queued on torch's current stream is ordered
        # before the engine's by `wait_for_caller()`, which prefill calls; decode_step does not (its
        # inputs are normally produced long before), so synchronise or call it yourself when a
        # buffer handed to decode_step was written on another stream just before.
        self.stream = stream if stream is not None else torch.cuda.Stream(self.device)
        dev_w = {}
        for k, v in weights.items():
            if isinstance(v, list):
                dev_w[k] = [to_device_bits(x, self.device) for x in v]
            else:
                dev_w[k] = to_device_bits(v, self.device)
        ws = WeightsStruct()
        keep = []
        for name in ("tok_emb", "pos_emb", "lnf_g", "lnf_b", "head_w", "head_b"):
            setattr(ws, name, _ptr(dev_w.get(name)).value)
        per_layer = ["ln1_g", "ln1_b", "ln2_g", "ln2_b"] + [l + s for l in LINEARS for s in ("_w", "_s", "_b")]
        for name in per_layer:
            ptrs = [(_ptr(t).value or 0) for t in dev_w[name]]
            arr = (C.c_void_p * len(ptrs))(*ptrs)
            keep.append(arr)
            setattr(ws, name, C.cast(arr, _PP))
        nbytes = query_workspace(cfg)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        cs = config_struct(cfg)
        h = C.c_void_p(0)
        torch.cuda.synchronize(self.device)
        _check(self.lib.tts_gpt_create(C.byref(cs), C.byref(ws), C.c_void_p(base), C.c_size_t(nbytes),
                                       C.c_void_p(self.stream.cuda_stream), C.byref(h)))
        self.handle = h
        self.workspace_bytes = nbytes
        del dev_w, keep

    def wait_for_caller(self):
        """Order everything queued so far on torch's current stream before the engine's next work."""
        self.stream.wait_stream(torch.cuda.current_stream(self.device))

    # -- the five calls -----------------------------------------------------------------------
    def prefill(self, prefixes, top_k=0, temperature=1.0, uniforms=None, pos0=None,
                out_tokens=None, out_logits=None, out_hidden=None):
        """prefixes: list of device tensors (int16 view of bf16 bits or torch.bfloat16) [P_i, d].
        Returns (stream_ids list, out_tokens tensor)."""
        n = len(prefixes)
        self.wait_for_caller()
        self._live_prefixes = [p.contiguous() for p in prefixes]
        ptrs = (C.c_void_p * n)(*[p.data_ptr() for p in self._live_prefixes])
        lens = _i32_array([p.shape[0] for p in self._live_prefixes])
        ids = (C.c_int32 * n)()
        if out_tokens is None:
            out_tokens = torch.empty(n, dtype=torch.int32, device=self.device)
        p0 = _i32_array(pos0) if pos0 is not None else None
        _check(self.lib.tts_gpt_prefill(self.handle, C.c_int32(n), ptrs, lens, p0, C.c_int32(top_k),
                                        C.c_float(temperature), _ptr(uniforms), ids, _ptr(out_tokens),
                                        _ptr(out_logits), _ptr(out_hidden)), self.handle)
        return list(ids), out_tokens

    def prefill_tokens(self, cond, text_ids, text_shift, text_pos0, top_k=0, temperature=1.0, uniforms=None,
                       pos0=None, out_tokens=None, out_logits=None, out_hidden=None):
        """Prefixes assembled on the device: cond[i] a device tensor of bf16 bits [n_cond_i, d] (or None),
        text_ids[i] a device int32 tensor [n_text_i] (or None).  Returns (stream_ids list, out_tokens tensor)."""
        n = len(cond)
        self.wait_for_caller()
        self._live_prefixes = [None if p is None else p.contiguous() for p in cond]
        self._live_text = [None if t is None else t.contiguous() for t in text_ids]
        cptrs = (C.c_void_p * n)(*[None if p is None else p.data_ptr() for p in self._live_prefixes])
        tptrs = (C.c_void_p * n)(*[None if t is None else t.data_ptr() for t in self._live_text])
        ncond = _i32_array([0 if p is None else p.shape[0] for p in self._live_prefixes])
        ntext = _i32_array([0 if t is None else t.shape[0] for t in self._live_text])
        ids = (C.c_int32 * n)()
        if out_tokens is None:
            out_tokens = torch.empty(n, dtype=torch.int32, device=self.device)
        p0 = _i32_array(pos0) if pos0 is not None else None
        _check(self.lib.tts_gpt_prefill_tokens(self.handle, C.c_int32(n), cptrs, ncond, tptrs, ntext,
                                               C.c_int32(text_shift), C.c_int32(text_pos0), p0, C.c_int32(top_k),
                                               C.c_float(temperature), _ptr(uniforms), ids, _ptr(out_tokens),
                                               _ptr(out_logits), _ptr(out_hidden)), self.handle)
        return list(ids), out_tokens

    def decode_step(self, stream_ids, out_tokens, in_tokens=None, top_k=0, temperature=1.0,
                    uniforms=None, out_logits=None, out_hidden=None):
        n = len(stream_ids)
        ids = stream_ids if isinstance(stream_ids, C.Array) else _i32_array(stream_ids)
        return _check(self.lib.tts_gpt_decode_step(self.handle, C.c_int32(n), ids, _ptr(in_tokens),
                                                   C.c_int32(top_k), C.c_float(temperature),
                                                   _ptr(uniforms), _ptr(out_tokens), _ptr(out_logits),
                                                   _ptr(out_hidden)), self.handle)

    def decode_step_host(self, stream_ids, out_tokens, in_tokens=None, top_k=0, temperature=1.0,
                         uniforms=None, out_logits=None, out_hidden=None):
        """One step with HOST tensors (ideally pinned): inputs are copied in, results are valid on return."""
        n = len(stream_ids)
        ids = stream_ids if isinstance(stream_ids, C.Array) else _i32_array(stream_ids)
        return _check(self.lib.tts_gpt_decode_step_host(self.handle, C.c_int32(n), ids, _ptr(in_tokens),
                                                        C.c_int32(top_k), C.c_float(temperature),
                                                        _ptr(uniforms), _ptr(out_tokens), _ptr(out_logits),
                                                        _ptr(out_hidden)), self.handle)

    def decode_steps(self, stream_ids, n_steps, out_tokens, in_tokens=None, top_k=0, temperature=1.0,
                     uniforms=None, out_logits=None, out_hidden=None):
        """n_steps steps in one call; the output tensors hold n_steps * len(stream_ids) rows."""
        n = len(stream_ids)
        ids = stream_ids if isinstance(stream_ids, C.Array) else _i32_array(stream_ids)
        return _check(self.lib.tts_gpt_decode_steps(self.handle, C.c_int32(n), ids, _ptr(in_tokens),
                                                    C.c_int32(n_steps), C.c_int32(top_k), C.c_float(temperature),
                                                    _ptr(uniforms), _ptr(out_tokens), _ptr(out_logits),
                                                    _ptr(out_hidden)), self.handle)

    def release_stream(self, stream_id):
        return _check(self.lib.tts_gpt_release_stream(self.handle, C.c_int32(stream_id)), self.handle)

    def sync(self):
        rc = _check(self.lib.tts_gpt_sync(self.handle), self.handle)
        self._live_prefixes = None
        return rc

    def destroy(self):
        if self.handle is not None:
            self.lib.tts_gpt_destroy(self.handle)
            self.handle = None
            self.workspace = None

    # -- introspection ------------------------------------------------------------------------
    def stats(self):
        a, b = C.c_int32(0), C.c_int32(0)
        _check(self.lib.tts_gpt_stats(self.handle, C.byref(a), C.byref(b)), self.handle)
        return {"open_streams": a.value, "free_pages": b.value}

    def stream_context(self, stream_id):
        return int(self.lib.tts_gpt_stream_context(self.handle, C.c_int32(stream_id)))

    def kernel_launches(self):
        n = C.c_uint64(0)
        _check(self.lib.tts_gpt_debug_kernel_launches(self.handle, C.byref(n)), self.handle)
        return n.value

    def set_trace(self, trace_tensor):
        """trace_tensor: int64 device tensor with 8 * slots entries (or None to switch off).
        Returns the number of traced kernels per step."""
        n = C.c_int32(0)
        _check(self.lib.tts_gpt_debug_set_trace(self.handle, _ptr(trace_tensor), C.byref(n)), self.handle)
        return n.value

    def debug_shuffle_free_pages(self, seed):
        return _check(self.lib.tts_gpt_debug_shuffle_free_pages(self.handle, C.c_uint32(seed)), self.handle)

    def set_option(self, name, value):
        """Switch a kernel schedule on or off, or set a threshold (see tts_gpt_debug_set_option)."""
        return _check(self.lib.tts_gpt_debug_set_option(self.handle, C.c_char_p(name.encode()), C.c_int32(int(value))),
                      self.handle)

    def check_canaries(self):
        """Number of guard bytes around the KV pool that were overwritten (0 = intact)."""
        n = C.c_int32(0)
        _check(self.lib.tts_gpt_debug_check_canaries(self.handle, C.byref(n)), self.handle)
        return n.value

    def debug_expire_wait(self, limit_us):
        return _check(self.lib.tts_gpt_debug_expire_wait(self.handle, C.c_uint32(limit_us)), self.handle)

    def raw_call(self, name, *args):
        """Return the raw status of a C entry point (tests of error behaviour)."""
        return getattr(self.lib, name)(self.handle, *args)

    def last_error(self):
        m = self.lib.tts_gpt_last_error(self.handle)
        return m.decode() if m else ""

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


# ---------------------------------------------------------------------------------------------
# single-kernel entry points
# ---------------------------------------------------------------------------------------------
def op_linear_pack(wfmt, w, s, stream=None):
    """w: device tensor in the canonical format [N,K] (bf16 bits int16 / int8 / int32 words
    [N,K/8]); s: scales or None.  Returns the packed device buffer."""
    lib = load()
    N = w.shape[0]
    K = w.shape[1] * (8 if wfmt == 2 else 1)
    nbytes = C.c_size_t(0)
    _check(lib.tts_gpt_op_linear_packed_bytes(C.c_int32(wfmt), C.c_int32(N), C.c_int32(K), C.byref(nbytes)))
    packed = torch.empty(nbytes.value, dtype=torch.uint8, device=w.device)
    assert packed.data_ptr() % 256 == 0
    _check(lib.tts_gpt_op_linear_pack(C.c_int32(wfmt), C.c_int32(N), C.c_int32(K), _ptr(w), _ptr(s),
                                      _ptr(packed), _stream_ptr(stream)))
    return packed, N, K


def op_linear(wfmt, packed, N, K, act, bias=None, stream=None):
    B = act.shape[0]
    out = torch.empty((B, N), dtype=torch.float32, device=act.device)
    _check(load().tts_gpt_op_linear(C.c_int32(wfmt), C.c_int32(N), C.c_int32(K), _ptr(packed), _ptr(bias),
                                    C.c_int32(B), _ptr(act), _ptr(out), _stream_ptr(stream)))
    return out


def op_linear_tc(wfmt, w, s, act, bias=None, ksplit=1, stream=None):
    """Tensor-core linear: w/s in the canonical formats, act int16 (bf16 bits) [B,K] -> fp32 [B,N]."""
    N = w.shape[0]
    K = w.shape[1] * (8 if wfmt == 2 else 1)
    B = act.shape[0]
    n = C.c_size_t(0)
    _check(load().tts_gpt_op_linear_tc_scratch_bytes(C.c_int32(N), C.c_int32(K), C.byref(n)))
    scratch = torch.zeros(n.value + 1024, dtype=torch.uint8, device=w.device)
    base = (scratch.data_ptr() + 1023) // 1024 * 1024
    out = torch.empty((B, N), dtype=torch.float32, device=w.device)
    _check(load().tts_gpt_op_linear_tc(C.c_int32(wfmt), C.c_int32(N), C.c_int32(K), _ptr(w), _ptr(s), _ptr(bias),
                                       C.c_int32(B), _ptr(act), _ptr(out), C.c_int32(ksplit), C.c_void_p(base),
                                       _stream_ptr(stream)))
    (torch.cuda.current_stream() if stream is None else stream).synchronize()
    del scratch
    return out


def op_attention_scratch(R, n_head, device):
    n = C.c_size_t(0)
    _check(load().tts_gpt_op_attention_scratch_bytes(C.c_int32(R), C.c_int32(n_head), C.byref(n)))
    return torch.zeros(n.value, dtype=torch.uint8, device=device)


def op_attention(q, kv_layer, page_table, row_stream, row_pos, scratch=None, stream=None):
    R, dm = q.shape
    H = dm // 64
    out = torch.empty((R, dm), dtype=torch.int16, device=q.device)
    if scratch is None:
        scratch = op_attention_scratch(R, H, q.device)
    _check(load().tts_gpt_op_attention(C.c_int32(R), C.c_int32(H), _ptr(q), _ptr(kv_layer), _ptr(page_table),
                                       C.c_int32(page_table.shape[1]), _ptr(row_stream), _ptr(row_pos),
                                       _ptr(out), _ptr(scratch), _stream_ptr(stream)))
    return out


def op_attention_cluster(q, kv_layer, page_table, row_stream, row_pos, cluster_size, stream=None):
    """cluster_size 1, 2, 4, 8: cluster variant; 0: streaming variant; -1: prefill variant on the CUDA cores,
    -2: prefill variant on the tensor cores (both: rows grouped by stream with ascending positions)."""
    R, dm = q.shape
    H = dm // 64
    out = torch.empty((R, dm), dtype=torch.int16, device=q.device)
    _check(load().tts_gpt_op_attention_cluster(C.c_int32(R), C.c_int32(H), _ptr(q), _ptr(kv_layer),
                                               _ptr(page_table), C.c_int32(page_table.shape[1]),
                                               _ptr(row_stream), _ptr(row_pos), _ptr(out),
                                               C.c_int32(cluster_size), _stream_ptr(stream)))
    return out


STATIC_ATTN_MAX_ROW_HEADS = 1280


def op_attention_static(q, kv_layer, page_table, row_stream, row_pos, stream=None):
    """Attention for callers that may not allocate: scratch is an array inside the library (at most
    STATIC_ATTN_MAX_ROW_HEADS rows x heads).  Only the output tensor is created here, by torch; pass
    your own through the C entry point to avoid even that.  Calls on one device must not overlap."""
    R, dm = q.shape
    H = dm // 64
    out = torch.empty((R, dm), dtype=torch.int16, device=q.device)
    _check(load().tts_gpt_op_attention_static(C.c_int32(R), C.c_int32(H), _ptr(q), _ptr(kv_layer),
                                              _ptr(page_table), C.c_int32(page_table.shape[1]),
                                              _ptr(row_stream), _ptr(row_pos), _ptr(out), _stream_ptr(stream)))
    return out


def op_layernorm(x, g, b, eps, stream=None):
    R, d = x.shape
    out = torch.empty((R, d), dtype=torch.int16, device=x.device)
    _check(load().tts_gpt_op_layernorm(C.c_int32(R), C.c_int32(d), _ptr(x), _ptr(g), _ptr(b), C.c_float(eps),
                                       _ptr(out), _stream_ptr(stream)))
    return out


def op_sample(logits, top_k=0, temperature=1.0, uniforms=None, stream=None):
    R, V = logits.shape
    out = torch.empty(R, dtype=torch.int32, device=logits.device)
    _check(load().tts_gpt_op_sample(C.c_int32(R), C.c_int32(V), _ptr(logits), C.c_int32(top_k),
                                    C.c_float(temperature), _ptr(uniforms), _ptr(out), _stream_ptr(stream)))
    return out


def bf16_bits_tensor_to_f32(t: torch.Tensor) -> torch.Tensor:
    """int16 tensor of bf16 bit patterns -> float32 tensor (host or device)."""
    return t.view(torch.bfloat16).to(torch.float32)
