"""Host logic of the continuous batcher, driven by a fake engine on the CPU, and (gpu) against solo runs."""
import types

import numpy as np
import pytest
import torch

from paper_2607_21042_b200.batcher import ContinuousBatcher, pages_for


class FakeEngine:
    """Same calls as the binding's engine; tokens follow a rule of the stream's own history only, so a
    request's tokens must not depend on who shares the batch."""
    V = 97

    def __init__(self, max_streams, n_pages, max_context=2048, stop_token=-1):
        self.cfg = types.SimpleNamespace(max_streams=max_streams, n_pages=n_pages, max_context=max_context,
                                         d_model=4, stop_token=stop_token)
        self.device = "cpu"
        self.ctx = {}
        self.last = {}
        self.calls = []
        self.max_open = 0
        self.max_pages = 0

    def _pages(self):
        return sum(pages_for(c) for c in self.ctx.values())

    def _check(self):
        assert len(self.ctx) <= self.cfg.max_streams, "more streams than slots"
        assert self._pages() <= self.cfg.n_pages, "page pool exceeded"
        self.max_open = max(self.max_open, len(self.ctx))
        self.max_pages = max(self.max_pages, self._pages())

    @staticmethod
    def first_token(prefix):
        return int(prefix[:, 0].sum().item()) % FakeEngine.V

    @staticmethod
    def next_token(prev, ctx):
        return (31 * prev + 7 + ctx) % FakeEngine.V

    def prefill(self, prefixes, top_k=0, temperature=1.0, uniforms=None, pos0=None, out_tokens=None, out_hidden=None):
        ids = []
        for i, p in enumerate(prefixes):
            s = min(set(range(self.cfg.max_streams)) - set(self.ctx))
            self.ctx[s] = int(p.shape[0])
            self.last[s] = self.first_token(p)
            out_tokens[i] = self.last[s]
            if out_hidden is not None:
                out_hidden[i] = self.last[s]
            ids.append(s)
        self.calls.append(("prefill", len(prefixes)))
        self._check()
        return ids, out_tokens

    def decode_steps(self, stream_ids, n_steps, out_tokens, top_k=0, temperature=1.0, uniforms=None, out_hidden=None):
        n = len(stream_ids)
        assert len(set(stream_ids)) == n and all(s in self.ctx for s in stream_ids)
        for k in range(n_steps):
            for i, s in enumerate(stream_ids):
                self.ctx[s] += 1
                self.last[s] = self.next_token(self.last[s], self.ctx[s])
                out_tokens[k * n + i] = self.last[s]
                if out_hidden is not None:
                    out_hidden[k * n + i] = self.last[s]
        self.calls.append(("decode", n, n_steps))
        self._check()

    def release_stream(self, s):
        del self.ctx[s], self.last[s]

    def sync(self):
        pass


def _solo(prefix, n_new, stop=-1):
    t = [FakeEngine.first_token(prefix)]
    ctx = int(prefix.shape[0])
    while len(t) < n_new and t[-1] != stop:
        ctx += 1
        t.append(FakeEngine.next_token(t[-1], ctx))
    return np.array(t, dtype=np.int32)


def _requests(rng, n, max_prefix=300, max_new=200):
    out = []
    for _ in range(n):
        p = int(rng.integers(1, max_prefix))
        out.append((torch.from_numpy(rng.integers(0, 50, size=(p, 4)).astype(np.int16)), int(rng.integers(1, max_new))))
    return out


@pytest.mark.parametrize("max_streams,n_pages,chunk", [(4, 40, 25), (1, 8, 7), (16, 30, 50), (8, 200, 1000)])
def test_every_request_gets_its_solo_tokens_within_the_engine_limits(max_streams, n_pages, chunk):
    rng = np.random.default_rng(max_streams * 1000 + n_pages)
    eng = FakeEngine(max_streams, n_pages)
    b = ContinuousBatcher(eng, keep_hidden=True)
    reqs = _requests(rng, 23)
    rids = [b.submit(p, n) for p, n in reqs]
    got = {r: [] for r in rids}
    hid = {r: [] for r in rids}
    finished = []
    guard = 0
    while not b.idle():
        res = b.run_chunk(chunk)
        assert res, "a chunk must make progress"
        for c in res:
            assert len(c.tokens) >= 1 and c.hidden.shape == (len(c.tokens), 4)
            got[c.rid].append(c.tokens); hid[c.rid].append(c.hidden[:, 0])
            if c.finished:
                finished.append(c.rid)
        guard += 1
        assert guard < 10000
    assert sorted(finished) == rids and len(finished) == len(set(finished))
    for rid, (p, n) in zip(rids, reqs):
        t = np.concatenate(got[rid])
        assert np.array_equal(t, _solo(p, n)), rid
        assert np.array_equal(np.concatenate(hid[rid]).astype(np.int32), t)     # hidden rows travel with their tokens
    assert not eng.ctx and b.reserved_pages == 0                                # everything released
    assert eng.max_open <= max_streams and eng.max_pages <= n_pages
    # admission is first come first served: requests open in the order they were submitted
    assert finished[0] in rids


def test_slots_are_refilled_as_streams_finish_and_chunks_never_overshoot():
    eng = FakeEngine(max_streams=2, n_pages=100)
    b = ContinuousBatcher(eng)
    mk = lambda p: torch.ones((p, 4), dtype=torch.int16)
    a = b.submit(mk(10), 5); c = b.submit(mk(20), 30); d = b.submit(mk(5), 3)
    r1 = {x.rid: x for x in b.run_chunk(10)}
    # a and c are admitted together (one prefill), the chunk stops after a's 4 remaining steps
    assert eng.calls[:2] == [("prefill", 2), ("decode", 2, 4)]
    assert len(r1[a].tokens) == 5 and r1[a].finished and len(r1[c].tokens) == 5 and not r1[c].finished and d not in r1
    r2 = {x.rid: x for x in b.run_chunk(10)}
    # d takes a's slot; the chunk is cut to d's 2 remaining steps
    assert eng.calls[2:4] == [("prefill", 1), ("decode", 2, 2)]
    assert len(r2[d].tokens) == 3 and r2[d].finished and len(r2[c].tokens) == 2
    r3 = b.run_chunk(10)
    assert eng.calls[4] == ("decode", 1, 10) and len(r3) == 1 and len(r3[0].tokens) == 10
    assert len(b.run_all(10)[c]) == 13 and b.idle()


def test_page_budget_holds_requests_back_and_stop_token_ends_a_stream():
    eng = FakeEngine(max_streams=8, n_pages=6)
    b = ContinuousBatcher(eng)
    mk = lambda p: torch.ones((p, 4), dtype=torch.int16)
    x = b.submit(mk(200), 57)      # 256 tokens -> 4 pages
    y = b.submit(mk(100), 29)      # 128 tokens -> 2 pages
    z = b.submit(mk(10), 10)       # 1 page: has to wait although slots are free
    b.run_chunk(5)
    assert eng.calls[0] == ("prefill", 2) and len(b.queue) == 1 and b.reserved_pages == 6
    out = b.run_all(64)
    assert len(out[z]) == 10 and b.idle()
    with pytest.raises(ValueError):
        b.submit(mk(2000), 100)            # past max_context
    with pytest.raises(ValueError):
        b.submit(mk(300), 200)             # more pages than the pool has
    # stop token: the solo sequence of a 12-row prefix of ones hits some token; make that the stop token
    seq = _solo(mk(12), 40)
    stop = int(seq[6])
    first = int(np.nonzero(seq == stop)[0][0])
    eng2 = FakeEngine(max_streams=2, n_pages=10, stop_token=stop)
    b2 = ContinuousBatcher(eng2)
    r = b2.submit(mk(12), 40)
    toks = b2.run_all(16)[r]
    assert np.array_equal(toks, seq[:first + 1]) and not eng2.ctx


@pytest.mark.gpu
def test_batcher_on_the_engine_matches_solo_runs():
    """Seven requests through an engine with 3 stream slots, chunks of 5 steps: each request's tokens equal
    those of the same request run alone (up to near-ties of the logits, which the solo run excuses)."""
    from helpers import bits_dev, gpu_run_stream, check_tokens
    from oracle import gpt_oracle as O
    from paper_2607_21042_b200 import binding as B, cases as C
    dev = "cuda:0"
    cfg = C.tiny_config(max_streams=3, n_pages=3 * 8)
    w = C.make_weights(cfg, seed=0)
    model = O.OracleModel(cfg, w)
    eng = B.TtsGpt(cfg, w, dev)
    lens = [70, 5, 130, 33, 64, 1, 90]
    news = [12, 30, 7, 1, 25, 18, 40]
    prefixes = C.make_prefixes(cfg, lens, seed=6)
    b = ContinuousBatcher(eng, keep_hidden=True)
    rids = [b.submit(bits_dev(p), n) for p, n in zip(prefixes, news)]
    got = {r: [] for r in rids}
    hid = {r: [] for r in rids}
    while not b.idle():
        assert eng.stats()["open_streams"] <= 3
        for c in b.run_chunk(5):
            got[c.rid].append(c.tokens); hid[c.rid].append(c.hidden)
    assert eng.stats() == {"open_streams": 0, "free_pages": 3 * 8}
    for rid, p, n in zip(rids, prefixes, news):
        toks = np.concatenate(got[rid])
        assert len(toks) == n and np.concatenate(hid[rid]).shape == (n, cfg.d_model)
        # the oracle replays the batcher's own tokens: every one of them is the oracle's choice or a near-tie
        ref_logits, ref_hidden = O.replay_full(model, O.bf16_to_f64(p), toks[:-1])
        check_tokens(toks, ref_logits, 0, 1.0, None, "request %d" % rid)
        h = O.bf16_to_f64(np.concatenate(hid[rid]))
        assert np.max(np.abs(h - ref_hidden)) <= 2e-2 * max(1.0, np.abs(ref_hidden).max())
    eng.destroy()
