"""Shared pieces of the GPU parity tests: tolerances, conversions, the replay comparison."""
import numpy as np
import torch

from oracle import gpt_oracle as O
from paper_2607_21042_b200 import cases as C

# Parity bar of the decode step against the fp64 oracle: logits max-abs error and relative L2 error;
# a token mismatch is excused where the oracle's decision margin is below GAP.
LOGIT_MAX_ABS = 3e-2
LOGIT_REL_L2 = 1e-2
GAP = 3e-2
# top-k: a mismatch is excused when u is within this distance of an oracle CDF boundary
# ((e^{2*0.03} - 1)/2: both neighbouring weights can move by a factor e^{+-0.03})
CDF_MARGIN = 0.031
# 8-bit (e4m3) KV cache.  The encoding is a step function of the K/V values, and the two sides reach those
# values through different rounding histories (relative difference about 1e-3, the same that gives the
# 16-bit cache its 0.5 % logit error): one to two percent of the cached codes land one step apart (6-12 % of
# the value).  Over the 24 layers this adds, in quadrature, about as much logit error again as the bf16
# operands cause (0.09 x sqrt(0.015 / 50 attended tokens) = 0.16 % of an attention output per layer), so the
# bar is the usual one times 1.5; below 32 attended tokens the flips do not average out (1.1 % of the
# attention output with a single token) and the relative bar is 2.5e-2.
E4M3_MAX_ABS = 4.5e-2
E4M3_REL_L2 = 1.5e-2
E4M3_REL_L2_SHORT = 2.5e-2


def bits_dev(arr, device="cuda:0"):
    a = np.ascontiguousarray(arr)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(a).to(device)


def bits_to_f64(t: torch.Tensor) -> np.ndarray:
    return O.bf16_to_f64(t.cpu().numpy().view(np.uint16))


def logits_errors(gpu: np.ndarray, ref: np.ndarray):
    gpu = np.asarray(gpu, dtype=np.float64)
    err = np.abs(gpu - ref)
    max_abs = float(err.max())
    rel = np.sqrt(((gpu - ref) ** 2).sum(axis=-1)) / np.sqrt((ref ** 2).sum(axis=-1))
    return max_abs, float(np.max(rel))


def assert_logits_close(gpu, ref, what="", max_abs_bar=LOGIT_MAX_ABS, rel_bar=LOGIT_REL_L2):
    max_abs, rel = logits_errors(gpu, ref)
    assert max_abs <= max_abs_bar, "%s: logits max-abs error %.4g > %.3g" % (what, max_abs, max_abs_bar)
    assert rel <= rel_bar, "%s: logits relative L2 error %.4g > %.3g" % (what, rel, rel_bar)
    return max_abs, rel


def check_tokens(gpu_tokens, ref_logits, top_k, temperature, uniforms, what=""):
    """Per step, on identical history: the GPU token equals the oracle's choice from the oracle's
    logits, or the step is excused (greedy: top-2 gap < GAP; top-k: u within CDF_MARGIN of a CDF
    boundary, or the gap at the k / k+1 cut < GAP).  Returns the number of excused steps."""
    excused = 0
    for i, tok in enumerate(gpu_tokens):
        lg = ref_logits[i]
        u = 0.0 if uniforms is None else float(uniforms[i])
        want = O.sample(lg, top_k, temperature, u)
        if int(tok) == want:
            continue
        if top_k <= 1:
            ok = O.top2_gap(lg) < GAP and lg[int(tok)] >= lg.max() - GAP
        else:
            I, c = O.topk_cdf(lg, top_k, temperature)
            near = np.min(np.abs(c - u)) < CDF_MARGIN
            srt = np.sort(lg)[::-1]
            cut = srt[top_k - 1] - srt[top_k] < GAP
            ok = near or cut
        assert ok, "%s: step %d: GPU token %d, oracle %d, not excused" % (what, i, int(tok), want)
        excused += 1
    return excused


def gpu_run_stream(eng, prefix_bits_dev, n_decode, top_k=0, temperature=1.0, uniforms_dev=None,
                   forced_tokens=None, want_hidden=False, pos0=None):
    """Prefill one stream and take n_decode steps, all queued on the engine's stream with one sync
    at the end.  uniforms_dev: fp32 [n_decode+1] on the device.  forced_tokens: int32 device tensor
    [n_decode] of inputs y_0..y_{n-1} (teacher forcing); otherwise the engine feeds itself.
    Returns tokens [n+1], logits [n+1,V], hidden [n+1,d] (bits) and the stream id."""
    V, d = eng.cfg.vocab, eng.cfg.d_model
    dev = eng.device
    n = n_decode
    toks = torch.zeros(n + 1, dtype=torch.int32, device=dev)
    logits = torch.zeros((n + 1, V), dtype=torch.float32, device=dev)
    hidden = torch.zeros((n + 1, d), dtype=torch.int16, device=dev) if want_hidden else None
    torch.cuda.synchronize()
    ids, _ = eng.prefill([prefix_bits_dev], top_k=top_k, temperature=temperature,
                         uniforms=None if uniforms_dev is None else uniforms_dev[0:1],
                         out_tokens=toks[0:1], out_logits=logits[0:1],
                         out_hidden=None if hidden is None else hidden[0:1],
                         pos0=None if pos0 is None else [pos0])
    for k in range(1, n + 1):
        eng.decode_step(ids, toks[k:k + 1],
                        in_tokens=None if forced_tokens is None else forced_tokens[k - 1:k],
                        top_k=top_k, temperature=temperature,
                        uniforms=None if uniforms_dev is None else uniforms_dev[k:k + 1],
                        out_logits=logits[k:k + 1],
                        out_hidden=None if hidden is None else hidden[k:k + 1])
    eng.sync()
    return (toks.cpu().numpy(), logits.cpu().numpy(),
            None if hidden is None else hidden.cpu().numpy().view(np.uint16), ids[0])


def assert_same_up_to_ties(tok_a, lg_a, tok_b, lg_b, what="", tol=LOGIT_MAX_ABS):
    """Two GPU runs of the same stream through different batch shapes (e.g. alone on the CUDA-core
    path vs inside a large batch on the tensor pipe): the fp32 sums are rounded in a different
    order, and every flipped bf16 rounding of an activation decorrelates the two runs further, so
    after 24 layers they differ from each other about as much as each differs from the oracle.
    So: logits agree within `tol` (the parity bar) as long as the histories agree, and the first
    token that differs, if any, sits on a near-tie of that size."""
    n = min(len(tok_a), len(tok_b))
    d = np.nonzero(np.asarray(tok_a[:n]) != np.asarray(tok_b[:n]))[0]
    m = n if len(d) == 0 else int(d[0]) + 1
    diff = float(np.max(np.abs(np.asarray(lg_a[:m], dtype=np.float64) - np.asarray(lg_b[:m], dtype=np.float64))))
    assert diff < tol, "%s: logits differ by %.4g between batch shapes" % (what, diff)
    if len(d):
        srt = np.sort(np.asarray(lg_b[d[0]], dtype=np.float64))
        assert srt[-1] - srt[-2] < tol, "%s: tokens differ at step %d away from a tie" % (what, d[0])
    return m
