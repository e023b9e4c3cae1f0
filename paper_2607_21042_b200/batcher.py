"""Chunked decoding with continuous batching on one engine (Sections II-C, II-D: the GPT yields tokens
and per-step hidden states, the later stages consume them a chunk at a time, and several utterances are
synthesised concurrently).

Host-side scheduling only: every step of the model runs in the library's kernels.  ``ContinuousBatcher``
keeps a queue of requests and a set of open streams.  ``run_chunk(n)``

1. admits queued requests, oldest first, while a stream slot is free and the page pool can hold the
   request's whole life (prefix + max_new_tokens), with ONE prefill call for all of them;
2. takes up to ``n`` decode steps for all open streams in ONE ``decode_steps`` call (fewer if a stream
   needs fewer tokens to finish: no stream decodes past its budget);
3. copies the chunk's tokens (and hidden rows, if asked for) to the host, cuts a stream at the stop
   token if the engine has one, releases finished streams so that their slots and pages serve the next
   requests, and returns what each request produced in this chunk.

The engine object needs ``prefill``, ``decode_steps``, ``release_stream``, ``sync`` and a ``cfg`` with
``max_streams``, ``n_pages``, ``max_context``, ``d_model``, ``stop_token``; tests drive the scheduler
with a fake one on the CPU.
"""
from __future__ import annotations

from collections import deque
from dataclasses import dataclass, field
from typing import Any, Deque, Dict, List, Optional

import numpy as np
import torch

PAGE_TOKENS = 64


def pages_for(tokens: int) -> int:
    return (tokens + PAGE_TOKENS - 1) // PAGE_TOKENS


@dataclass
class Request:
    rid: int
    prefix: Any                 # device tensor [P, d] of bf16 bits
    max_new_tokens: int         # tokens to produce, the one sampled by prefill included
    pos0: int = 0
    stream: int = -1            # engine stream id while open
    produced: int = 0
    pages: int = 0              # pages reserved for the request's whole life

    @property
    def prefix_len(self) -> int:
        return int(self.prefix.shape[0])


@dataclass
class ChunkResult:
    rid: int
    tokens: np.ndarray                  # int32 [m]: the tokens this chunk added for the request
    hidden: Optional[np.ndarray]        # uint16 [m, d] bf16 bits, if hidden states are kept
    finished: bool


@dataclass
class ContinuousBatcher:
    engine: Any
    top_k: int = 0
    temperature: float = 1.0
    keep_hidden: bool = False
    device: Any = None
    queue: Deque[Request] = field(default_factory=deque)
    active: List[Request] = field(default_factory=list)
    reserved_pages: int = 0
    next_rid: int = 0
    uniform_source: Any = None          # callable(n) -> device fp32 [n] in [0,1); needed when top_k > 1

    def __post_init__(self):
        cfg = self.engine.cfg
        self.max_streams = int(cfg.max_streams)
        self.n_pages = int(cfg.n_pages)
        self.max_context = int(cfg.max_context)
        self.d = int(cfg.d_model)
        self.stop_token = int(getattr(cfg, "stop_token", -1))
        if self.device is None:
            self.device = getattr(self.engine, "device", "cpu")
        if self.top_k > 1 and self.uniform_source is None:
            raise ValueError("top-k sampling needs a uniform_source")

    # -- requests -------------------------------------------------------------------------------
    def submit(self, prefix, max_new_tokens: int, pos0: int = 0) -> int:
        if max_new_tokens < 1:
            raise ValueError("max_new_tokens must be positive")
        total = int(prefix.shape[0]) + max_new_tokens - 1     # the last token produced is never fed back
        if int(prefix.shape[0]) < 1 or total > self.max_context:
            raise ValueError("request does not fit max_context")
        if pages_for(total) > self.n_pages:
            raise ValueError("request does not fit the page pool")
        rid = self.next_rid
        self.next_rid += 1
        self.queue.append(Request(rid, prefix, max_new_tokens, pos0, pages=pages_for(total)))
        return rid

    def idle(self) -> bool:
        return not self.queue and not self.active

    def _uniforms(self, n):
        return None if self.top_k <= 1 else self.uniform_source(n)

    # -- one chunk ------------------------------------------------------------------------------
    def _admit(self) -> List[Request]:
        new: List[Request] = []
        while self.queue and len(self.active) + len(new) < self.max_streams and \
                self.reserved_pages + self.queue[0].pages <= self.n_pages:
            r = self.queue.popleft()
            self.reserved_pages += r.pages
            new.append(r)
        return new

    def run_chunk(self, n_steps: int) -> List[ChunkResult]:
        """Admit what fits, decode up to n_steps tokens per open stream, retire what finished."""
        if n_steps < 1:
            raise ValueError("n_steps must be positive")
        eng = self.engine
        got_tok: Dict[int, List[np.ndarray]] = {}
        got_hid: Dict[int, List[np.ndarray]] = {}
        new = self._admit()
        if new:
            n = len(new)
            tok = torch.zeros(n, dtype=torch.int32, device=self.device)
            hid = torch.zeros((n, self.d), dtype=torch.int16, device=self.device) if self.keep_hidden else None
            ids, _ = eng.prefill([r.prefix for r in new], top_k=self.top_k, temperature=self.temperature,
                                 uniforms=self._uniforms(n), pos0=[r.pos0 for r in new], out_tokens=tok,
                                 out_hidden=hid)
            eng.sync()
            tok_h = tok.cpu().numpy()
            hid_h = None if hid is None else hid.cpu().numpy().view(np.uint16)
            for i, r in enumerate(new):
                r.stream = int(ids[i])
                r.produced = 1
                got_tok[r.rid] = [tok_h[i:i + 1].copy()]
                if hid_h is not None:
                    got_hid[r.rid] = [hid_h[i:i + 1].copy()]
                self.active.append(r)
        stopped = {r.rid for r in self.active
                   if self.stop_token >= 0 and r.rid in got_tok and int(got_tok[r.rid][0][0]) == self.stop_token}
        run = [r for r in self.active if r.produced < r.max_new_tokens and r.rid not in stopped]
        if run:
            k = min(n_steps, min(r.max_new_tokens - r.produced for r in run))
            n = len(run)
            tok = torch.zeros(k * n, dtype=torch.int32, device=self.device)
            hid = torch.zeros((k * n, self.d), dtype=torch.int16, device=self.device) if self.keep_hidden else None
            eng.decode_steps([r.stream for r in run], k, tok, top_k=self.top_k, temperature=self.temperature,
                             uniforms=self._uniforms(k * n), out_hidden=hid)
            eng.sync()
            tok_h = tok.cpu().numpy().reshape(k, n)
            hid_h = None if hid is None else hid.cpu().numpy().view(np.uint16).reshape(k, n, self.d)
            for i, r in enumerate(run):
                t = tok_h[:, i]
                m = k
                if self.stop_token >= 0:
                    hit = np.nonzero(t == self.stop_token)[0]
                    if len(hit):
                        m = int(hit[0]) + 1          # the stop token itself is delivered, nothing after it
                        stopped.add(r.rid)
                r.produced += k
                got_tok.setdefault(r.rid, []).append(t[:m].copy())
                if hid_h is not None:
                    got_hid.setdefault(r.rid, []).append(hid_h[:m, i].copy())
        out: List[ChunkResult] = []
        still: List[Request] = []
        for r in self.active:
            done = r.produced >= r.max_new_tokens or r.rid in stopped
            if done:
                eng.release_stream(r.stream)
                self.reserved_pages -= r.pages
            else:
                still.append(r)
            if r.rid in got_tok:
                h = np.concatenate(got_hid[r.rid]) if r.rid in got_hid else None
                out.append(ChunkResult(r.rid, np.concatenate(got_tok[r.rid]), h, done))
        self.active = still
        return out

    def run_all(self, chunk: int) -> Dict[int, np.ndarray]:
        """Drain the queue; returns every request's tokens."""
        res: Dict[int, List[np.ndarray]] = {}
        while not self.idle():
            for c in self.run_chunk(chunk):
                res.setdefault(c.rid, []).append(c.tokens)
        return {rid: np.concatenate(v) for rid, v in res.items()}
