/*
 * tts_gpt.h — C ABI of the B200 (sm_100a) decode step of IndexTTS-2's Text-to-Semantic GPT.
 *
 * The paper ("Faster IndexTTS-2") accelerates a decoder-only autoregressive GPT that emits
 * semantic codec tokens one per step (Section II-A), fed by a conditioning prefix of embeddings
 * followed by tokens (Section II-C), batched over concurrent utterances (Sections II-B, II-D),
 * optionally with W8A16 / W4A16 weight-only quantization (Table I caption, Section III-B), and
 * returning at every step the token id, the logits and the hidden state of the last layer
 * (Section II-C).  This library is that engine for one GPU: a paged KV cache of 64-token pages,
 * dequantizing linears, split-KV decode attention, fused LayerNorm / GELU / residual and greedy or
 * top-k sampling, all in hand-written CUDA kernels.
 *
 * General rules
 *  - Alignment: prefix embeddings and out_hidden 16 bytes (rows are moved with vector loads and
 *    stores), token / uniform / logit buffers 4 bytes; a misaligned pointer is refused with E_ARG.
 *  - Every function returns an int32 status: TTS_GPT_OK (0) or a negative TTS_GPT_E_* code.
 *    Nothing throws, aborts or traps the device.  tts_gpt_last_error() describes the last failure.
 *  - Memory: the caller owns every buffer, including the workspace given to tts_gpt_create.  The
 *    library never allocates device memory.  "device" below means a pointer valid on the current
 *    CUDA device, "host" a plain host pointer.  bf16 tensors are 16-bit brain floats, row-major.
 *  - Asynchrony: prefill / decode_step / release_stream validate on the host, enqueue work on the
 *    CUDA stream given at create, and return without waiting.  A host-detectable error is
 *    returned immediately and leaves all state untouched.  Output buffers must stay alive until
 *    the next tts_gpt_sync (or the caller's own synchronisation of that stream).
 *  - A handle is not thread-safe; use one handle per thread / per GPU.
 */
#ifndef TTS_GPT_H_
#define TTS_GPT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tts_gpt tts_gpt_t; /* opaque */

/* Storage format of the KV cache (config field kv_fmt). */
enum { TTS_GPT_KV_BF16 = 0, TTS_GPT_KV_FP8_E4M3 = 1 };

/* Storage format of the four block linears (QKV, attention out, FC1, FC2).  Embeddings,
 * LayerNorm parameters, biases and the LM head are bf16 in every format. */
enum {
  TTS_GPT_W_BF16 = 0,      /* bf16 [N,K] */
  TTS_GPT_W_INT8_PC = 1,   /* int8 [N,K], symmetric, one bf16 scale per output row: W = s[n]*q */
  TTS_GPT_W_INT4_G128 = 2  /* int32 words [N,K/8]; nibble j (bits 4j..4j+3) of word w holds column
                              k = 8w+j as u = q+8; bf16 scales [N,K/128]: W = s[n,k/128]*(u-8) */
};

enum {
  TTS_GPT_OK = 0,
  TTS_GPT_E_ARG = -1,          /* invalid argument or configuration */
  TTS_GPT_E_NO_PAGES = -2,     /* KV page pool exhausted */
  TTS_GPT_E_STREAM = -3,       /* unknown, released or duplicate stream id; no free stream slot */
  TTS_GPT_E_CTX_OVERFLOW = -4, /* a stream would exceed max_context */
  TTS_GPT_E_CUDA = -5,         /* a CUDA runtime call failed */
  TTS_GPT_E_TIMEOUT = -6,      /* a bounded device-side wait expired */
  TTS_GPT_E_WORKSPACE = -7,    /* workspace too small or misaligned */
  TTS_GPT_E_UNSUPPORTED = -8
};

typedef struct {
  int32_t n_layer, d_model, n_head, head_dim, d_ff, vocab; /* head_dim must be 64, n_head*64 = d_model */
  int32_t wfmt;          /* TTS_GPT_W_* of the block linears */
  int32_t max_streams;   /* concurrent utterances, 1..128 */
  int32_t max_context;   /* tokens per stream, multiple of page_tokens, <= 2048 */
  int32_t page_tokens;   /* must be 64 */
  int32_t n_pages;       /* pages in the KV pool (each holds 64 tokens of every layer) */
  int32_t max_pos;       /* rows of pos_emb */
  int32_t gelu_tanh;     /* 1: tanh-form GELU (GPT-2), 0: erf form */
  int32_t stop_token;    /* -1: none */
  float ln_eps;          /* LayerNorm epsilon (inside the square root) */
  int32_t emb_rows;      /* rows of tok_emb: the merged embedding table of Section II-C holds the semantic
                            codes first and the text ids after them; 0 = vocab (no text region) */
  int32_t kv_fmt;        /* KV cache: TTS_GPT_KV_BF16, or TTS_GPT_KV_FP8_E4M3 (beyond the precisions of Table I: every
                            cached token and head keeps its 64 K (and V) values as e4m3 codes with one fp32 scale
                            s = max|x| / 448; a page then takes 4352 instead of 8192 bytes per head and K|V) */
} tts_gpt_config_t;

/* All DEVICE pointers, read only during tts_gpt_create (the library keeps its own re-laid-out
 * copy in the workspace; the caller may free these afterwards).  Per-layer entries are HOST arrays
 * of n_layer device pointers.  Shapes: tok_emb [emb_rows (vocab if 0),d]; pos_emb [max_pos,d]; ln*_g/_b [d];
 * head_w [vocab,d]; head_b [vocab] or NULL; qkv_w [3d,d] with rows ordered Q,K,V and head h owning
 * columns 64h..64h+63 of each; o_w [d,d]; fc1_w [d_ff,d]; fc2_w [d,d_ff]; *_b bf16 [N];
 * *_s bf16 scales (NULL array or NULL entries for bf16 weights). */
typedef struct {
  const void *tok_emb, *pos_emb, *lnf_g, *lnf_b, *head_w, *head_b;
  const void *const *ln1_g, *const *ln1_b, *const *ln2_g, *const *ln2_b;
  const void *const *qkv_w, *const *qkv_s, *const *qkv_b;
  const void *const *o_w, *const *o_s, *const *o_b;
  const void *const *fc1_w, *const *fc1_s, *const *fc1_b;
  const void *const *fc2_w, *const *fc2_s, *const *fc2_b;
} tts_gpt_weights_t;

/* Bytes of device workspace tts_gpt_create needs for this configuration (weights in streaming
 * layout + KV pool + page tables + activations + scratch).  No CUDA call is made. */
int32_t tts_gpt_query_workspace(const tts_gpt_config_t *cfg, size_t *bytes);

/* Build an engine inside `workspace` (device, 256-byte aligned, >= query_workspace bytes).
 * `cuda_stream` is a cudaStream_t (NULL = default stream) on which every later call enqueues.
 * Re-lays the weights out for streaming, clears the page allocator and synchronises the stream
 * once before returning.  The handle itself is a small host object freed by tts_gpt_destroy. */
int32_t tts_gpt_create(const tts_gpt_config_t *cfg, const tts_gpt_weights_t *weights,
                       void *workspace, size_t workspace_bytes, void *cuda_stream, tts_gpt_t **out);

/* Context phase (Section II-C: conditioning embeddings, then text, precede the semantic tokens).
 * Opens n new streams.  prefix_emb: HOST array of n DEVICE pointers to bf16 [prefix_len[i], d]
 * embeddings that are used as given (the caller has already added, or for the conditioning rows
 * not added, positional embeddings).  pos0[i] (HOST, may be NULL = 0) is the index into pos_emb of
 * the stream's first generated token.  Fills the KV cache for positions 0..P_i-1, computes the
 * logits of the last prefix row and samples y_0 from them with (top_k, temperature, uniforms).
 * out_stream_ids: HOST [n], written before return.  out_tokens: DEVICE int32 [n].
 * out_logits: DEVICE fp32 [n,vocab] or NULL.  out_hidden: DEVICE bf16 [n,d] or NULL (final
 * LayerNorm output).  uniforms: DEVICE fp32 [n] in [0,1), needed only when top_k > 1.
 * Errors: E_ARG (n < 1, a prefix_len < 1), E_STREAM (fewer than n free slots), E_CTX_OVERFLOW
 * (prefix_len > max_context), E_NO_PAGES.  All-or-nothing. */
int32_t tts_gpt_prefill(tts_gpt_t *h, int32_t n, const void *const *prefix_emb,
                        const int32_t *prefix_len, const int32_t *pos0, int32_t top_k,
                        float temperature, const float *uniforms, int32_t *out_stream_ids,
                        int32_t *out_tokens, float *out_logits, void *out_hidden);

/* Context phase with the prefix assembled on the device (Section II-C: conditioning embeddings
 * retrieved in front of the sequence, one merged embedding table with text ids shifted past the
 * semantic codes, position ids of the library's own making).  Stream i's prefix is
 *   rows 0 .. n_cond[i]-1:  cond_emb[i] (DEVICE bf16 [n_cond[i], d]) used as given, no positional
 *                           embedding;
 *   then text token j:      tok_emb[text_ids[i][j] + text_shift] + pos_emb[text_pos0 + j]
 * (bf16 rows widened and added in fp32).  cond_emb, text_ids: HOST arrays of n DEVICE pointers
 * (cond_emb[i] 16-byte, text_ids[i] 4-byte aligned; either may be NULL when its count is 0);
 * n_cond, n_text: HOST int32 [n], n_cond[i] + n_text[i] >= 1.  text_shift is the number of semantic
 * codes in front of the text region; a shifted id outside 0..emb_rows-1 is clamped into that range
 * (the ids live on the device and are not inspected by the host).  text_pos0 + n_text[i] must not
 * exceed max_pos.  pos0 and everything after it: as for tts_gpt_prefill, whose errors also apply
 * (with prefix_len = n_cond + n_text). */
int32_t tts_gpt_prefill_tokens(tts_gpt_t *h, int32_t n, const void *const *cond_emb, const int32_t *n_cond,
                               const int32_t *const *text_ids, const int32_t *n_text, int32_t text_shift,
                               int32_t text_pos0, const int32_t *pos0, int32_t top_k, float temperature,
                               const float *uniforms, int32_t *out_stream_ids, int32_t *out_tokens,
                               float *out_logits, void *out_hidden);

/* One incremental decode step (Sections I, II-C) for n distinct open streams (stream_ids: HOST).
 * Stream i consumes one input token — in_tokens[i] (DEVICE int32 [n]) or, if in_tokens is NULL,
 * the token it sampled last — embedded as tok_emb[token] + pos_emb[pos0 + k - 1] on its k-th
 * step, appends that token's K/V at position ctx_i, attends over ctx_i + 1 keys, and returns the
 * logits of the next token, the sampled next token and optionally the final-LayerNorm hidden row.
 * top_k 0 or 1 = greedy (lowest index on ties); top_k in 2..64 = softmax over the top_k logits
 * at `temperature`, inverse CDF with uniforms[i].  Afterwards ctx_i += 1.
 * Errors: E_ARG, E_STREAM (unknown / duplicate id), E_CTX_OVERFLOW (ctx_i + 1 > max_context),
 * E_NO_PAGES.  All-or-nothing; nothing is enqueued on error. */
int32_t tts_gpt_decode_step(tts_gpt_t *h, int32_t n, const int32_t *stream_ids,
                            const int32_t *in_tokens, int32_t top_k, float temperature,
                            const float *uniforms, int32_t *out_tokens, float *out_logits,
                            void *out_hidden);

/* n_steps successive decode steps for the same n streams, queued in one call (Section II-C: the
 * later stages consume tokens and hidden states in chunks, so a caller decodes a chunk at a time).
 * Same result as n_steps calls of tts_gpt_decode_step in which step 1 takes in_tokens (or, if NULL,
 * each stream's last sample) and every later step the token the stream sampled in the step before,
 * on the device.  Step k (0-based) writes out_tokens[k*n + i], out_logits[(k*n + i)*vocab ..] and
 * out_hidden[(k*n + i)*d ..] and draws uniforms[k*n + i]: DEVICE arrays of n_steps*n rows
 * (out_logits, out_hidden, uniforms may be NULL as in tts_gpt_decode_step).
 * Errors as tts_gpt_decode_step, checked for the whole chunk before anything is enqueued:
 * E_CTX_OVERFLOW if a stream lacks room for n_steps more tokens, E_NO_PAGES if the pool cannot
 * supply every page the chunk will need, E_ARG if n_steps < 1.  All-or-nothing. */
int32_t tts_gpt_decode_steps(tts_gpt_t *h, int32_t n, const int32_t *stream_ids,
                             const int32_t *in_tokens, int32_t n_steps, int32_t top_k,
                             float temperature, const float *uniforms, int32_t *out_tokens,
                             float *out_logits, void *out_hidden);

/* tts_gpt_decode_step with HOST buffers: copies in_tokens (HOST int32 [n], or NULL as above) and
 * uniforms (HOST fp32 [n], needed when top_k > 1) to staging arrays inside the workspace, enqueues
 * the step, copies out_tokens (HOST int32 [n]), out_logits (HOST fp32 [n,vocab] or NULL) and
 * out_hidden (HOST bf16 [n,d] or NULL) back and waits for the engine's stream before it returns, so
 * the results are valid on return.  Page-locked host buffers make the copies asynchronous to the
 * host; pageable ones work.  Errors: those of tts_gpt_decode_step (nothing is enqueued but the
 * staging copies) and those of tts_gpt_sync. */
int32_t tts_gpt_decode_step_host(tts_gpt_t *h, int32_t n, const int32_t *stream_ids,
                                 const int32_t *in_tokens, int32_t top_k, float temperature,
                                 const float *uniforms, int32_t *out_tokens, float *out_logits,
                                 void *out_hidden);

/* Close a stream and return its pages to the pool.  E_STREAM if the id is not open. */
int32_t tts_gpt_release_stream(tts_gpt_t *h, int32_t stream_id);

/* Wait for the engine's CUDA stream; returns a deferred device-side error if one was recorded. */
int32_t tts_gpt_sync(tts_gpt_t *h);

/* Free the host handle (after synchronising).  The workspace stays the caller's. */
int32_t tts_gpt_destroy(tts_gpt_t *h);

/* Human-readable description of the last error on this handle (NULL handle: of the last failed
 * create / query on this thread).  The string is owned by the library. */
const char *tts_gpt_last_error(const tts_gpt_t *h);

/* Introspection used by tests and the bench (HOST outputs, any may be NULL): open streams, free
 * pages, and the context length of one stream (-1 if not open). */
int32_t tts_gpt_stats(const tts_gpt_t *h, int32_t *open_streams, int32_t *free_pages);
int32_t tts_gpt_stream_context(const tts_gpt_t *h, int32_t stream_id);

/* Number of this library's kernels enqueued on the handle's stream so far (a replayed CUDA graph
 * counts its kernel nodes on every replay).  HOST output. */
int32_t tts_gpt_debug_kernel_launches(const tts_gpt_t *h, uint64_t *n);

/* Timeline tracing (off by default).  `trace` is a DEVICE array of 8 * n_slots uint64, or NULL to
 * switch tracing off; *n_slots (HOST, may be NULL) receives the number of traced kernels per step
 * (an upper bound: 5 per layer — QKV, attention, O-proj, FC1, FC2 — then the LM head on the
 * small-batch path; 7 per layer — LN1, QKV, attention, O-proj, LN2, FC1, FC2 — on the tensor-core path).  While set, CTA 0 of each
 * traced kernel stores the GPU's global nanosecond timer at entry, after its dependency wait and
 * at its end into trace[8*slot + 0..2] (3..5: inner points of the linear kernels).  Synchronises and drops captured graphs. */
int32_t tts_gpt_debug_set_trace(tts_gpt_t *h, void *trace, int32_t *n_slots);

/* Test aid: permute the free-page list with a seeded shuffle (between calls, any time no stream
 * is open).  Results must not depend on which physical pages a stream receives. */
int32_t tts_gpt_debug_shuffle_free_pages(tts_gpt_t *h, uint32_t seed);

/* Test aid: the KV pool sits between two guard regions of the workspace that are filled with a pattern at
 * creation; *bad_bytes (HOST) receives the number of guard bytes that no longer hold it (0 = no kernel
 * wrote outside the pool on either side).  Waits for the stream. */
int32_t tts_gpt_debug_check_canaries(tts_gpt_t *h, int32_t *bad_bytes);

/* Experiments and tests: switches a kernel schedule of this engine on or off (value 0 / 1) or sets
 * a threshold.  Defaults are what the measurements use.  Waits for the stream and drops captured
 * step graphs.  Names: "graph", "pdl", "tc" and "tc_min_rows" (tensor-core
 * linears), "prefill_pass_rows" (rows per prefill pass: a multiple of 128 up to 1024; the default is chosen at creation
 * from the SM count and the model width, 896 for the 24-layer model on 148 SMs; passes of more than 128 rows need
 * the tensor-core path), "w4_tc_exact" (int4 weights only: by default the operand images of the tensor-core path, used for more than 16 rows,
 * hold code x group scale rounded once to bf16; 1 rewrites them as integer codes and the kernels scale fp32 sums per
 * 128-column group, 0 writes the default back), "attn_tc", "attn_mma", "attn_prefill", "attn_stream", "attn_stream_min_pairs", "attn_cluster_fill",
 * "fc2_ksplit"; "poison_free_pages" (test aid standing in for a memory checker: every free page, and
 * from then on every released page, is filled with NaN in all layers, so that a kernel reading a slot no
 * token was written to poisons its result).  Unknown name or value out of range: TTS_GPT_E_ARG. */
int32_t tts_gpt_debug_set_option(tts_gpt_t *h, const char *name, int32_t value);

/* Test aid for the device-side error path: enqueues a one-thread kernel that waits, with the same
 * bounded wait every kernel of the library uses, at most limit_us microseconds (1..100000) on a
 * barrier that nothing completes, and on expiry sets the engine's error word exactly as a kernel
 * whose copy never arrived would.  The next tts_gpt_sync then returns TTS_GPT_E_TIMEOUT once and
 * clears the word; the engine and the CUDA context stay usable.  Nothing hangs or faults. */
int32_t tts_gpt_debug_expire_wait(tts_gpt_t *h, uint32_t limit_us);

/* ---------------------------------------------------------------------------------------------
 * Single-kernel entry points: the building blocks of the step, callable on their own (unit parity
 * tests, micro-benchmarks).  All pointers DEVICE unless marked HOST; `cuda_stream` as above; each
 * call enqueues and returns.  Matrices, activation rows, q, the KV pool and fp32 outputs must be 16-byte
 * aligned (packed weights and scratch as stated per call); misaligned pointers are refused with E_ARG.
 * ------------------------------------------------------------------------------------------- */

/* Bytes of the streaming layout of one [N,K] linear in format wfmt (weights + scales). */
int32_t tts_gpt_op_linear_packed_bytes(int32_t wfmt, int32_t N, int32_t K, size_t *bytes);

/* Re-lay a canonical [N,K] matrix (formats above) into `packed` (device, 256-byte aligned,
 * >= packed_bytes).  K must be a multiple of 128. */
int32_t tts_gpt_op_linear_pack(int32_t wfmt, int32_t N, int32_t K, const void *w, const void *s,
                               void *packed, void *cuda_stream);

/* out[b,n] = sum_k W[n,k] * act[b,k] + bias[n]  (the weight-only dequantizing linear: Table I
 * caption).  act bf16 [B,K], bias bf16 [N] or NULL, out fp32 [B,N], 1 <= B <= 128. */
int32_t tts_gpt_op_linear(int32_t wfmt, int32_t N, int32_t K, const void *packed, const void *bias,
                          int32_t B, const void *act, float *out, void *cuda_stream);

/* The same linear on the 5th-generation tensor cores (the engine's path for more than 16 rows):
 * w, s in the canonical formats above, K a multiple of 128, 1 <= B <= 128.  ksplit 1 or 4: the
 * kernel of decode steps and one-tile passes (chunks of 32 batch rows per CTA), over all of K or
 * over 4 k-ranges; ksplit -1 .. -4: the kernel of prefill passes of several row tiles (128 rows x
 * 128 features per CTA), here on one row tile, over 1 .. 4 k-ranges.  With more than one range the
 * partial sums are folded in range order, as the engine's next LayerNorm does.  Quantized
 * codes enter the tensor cores as exact bf16 integers; scales multiply fp32 sums (per row for int8,
 * per row and 128-column group for int4).  `scratch` (1024-byte aligned, >= scratch_bytes) receives
 * the operand images. */
int32_t tts_gpt_op_linear_tc_scratch_bytes(int32_t N, int32_t K, size_t *bytes);
int32_t tts_gpt_op_linear_tc(int32_t wfmt, int32_t N, int32_t K, const void *w, const void *s, const void *bias,
                             int32_t B, const void *act, float *out, int32_t ksplit, void *scratch,
                             void *cuda_stream);

/* Bytes of scratch tts_gpt_op_attention needs for R rows of n_head heads. */
int32_t tts_gpt_op_attention_scratch_bytes(int32_t R, int32_t n_head, size_t *bytes);

/* Decode attention over a paged KV cache (Section I: attention kernels + KV-cache management of
 * the decode engine).  Row r belongs to stream row_stream[r] and attends over keys 0..row_pos[r]
 * of that stream: o = softmax(q.K^T / 8) V per head.  q fp32 [R, n_head*64]; kv_layer: one
 * layer's slice of the pool, bf16 [n_pages][2 (K,V)][n_head][64 tokens][64]; page_table int32
 * [*, pages_per_stream]; out bf16 [R, n_head*64].  `scratch` (>= scratch_bytes, 256-byte aligned)
 * must be zero on first use; the kernel leaves it zeroed where that matters. */
int32_t tts_gpt_op_attention(int32_t R, int32_t n_head, const float *q, const void *kv_layer,
                             const int32_t *page_table, int32_t pages_per_stream,
                             const int32_t *row_stream, const int32_t *row_pos, void *out,
                             void *scratch, void *cuda_stream);

/* The engine's attention kernels: same result as tts_gpt_op_attention and no scratch.
 * cluster_size 1, 2, 4 or 8: each (row, head) is split over a thread-block cluster of that many
 * CTAs that merge their partial results through distributed shared memory (small batches).
 * cluster_size 0: the streaming variant the engine uses for large batches, one CTA per (row, head)
 * whose warps pull whole K/V pages into shared memory with bulk asynchronous copies.
 * cluster_size -1: the prefill variant (rows must be ordered as in a prefill pass: grouped by stream,
 * positions ascending inside a stream): 8 consecutive rows per CTA share each K/V page.
 * cluster_size -2: the prefill variant the engine uses, same requirement on the rows: 16 consecutive rows
 * per CTA, Q K^T and P V on the tensor cores (bf16 operands: Q and the softmax weights are rounded to
 * bf16, sums and accumulators stay fp32).  It has no waits.
 * cluster_size -3: the prefill variant the engine uses for passes of more than 128 rows, same requirement on
 * the rows: 128 consecutive rows per CTA, Q K^T and P V as tcgen05 instructions with the scores and the
 * output in tensor memory (same roundings as -2); its waits are bounded.
 * The waits on the copies of variants 0 and -1 are bounded; this stand-alone entry does not report an
 * expired wait (the engine does, as TTS_GPT_E_TIMEOUT).  q, out and kv_layer must be 16-byte aligned. */
int32_t tts_gpt_op_attention_cluster(int32_t R, int32_t n_head, const float *q, const void *kv_layer,
                                     const int32_t *page_table, int32_t pages_per_stream,
                                     const int32_t *row_stream, const int32_t *row_pos, void *out,
                                     int32_t cluster_size, void *cuda_stream);

/* Same attention as tts_gpt_op_attention for callers that cannot hand over scratch memory because
 * they cannot allocate any: code that runs where cudaMalloc is off limits — a per-request handler of
 * a serving process whose whole device budget was carved up at start-up, a plug-in inside a host
 * engine that owns all device memory, a latency-critical audio thread that must never hit the
 * device-wide synchronisation an allocation implies.  (The paper has no counterpart of this call; it
 * is a convenience of this library.)  The split-KV partial results and ticket counters go into an
 * array built into the library image: about 2.7 MB that every GPU loading the library carries
 * until the process exits.  Limit: R * n_head <= TTS_GPT_STATIC_ATTN_MAX_ROW_HEADS; larger calls
 * return TTS_GPT_E_WORKSPACE and enqueue nothing.  The call allocates nothing and frees nothing.
 * The first call on each device (with that device current) looks up the array's device address;
 * make that first call before starting any stream capture.  All calls on a device share the one
 * array: it still holds the previous call's partials (harmless, they are overwritten before use)
 * and the call itself zeroes the tickets it needs on `cuda_stream`; two calls that can overlap on
 * the GPU (different streams without ordering) race on it and must be serialised by the caller.
 * Arguments and results otherwise exactly as tts_gpt_op_attention. */
#define TTS_GPT_STATIC_ATTN_MAX_ROW_HEADS 1280
int32_t tts_gpt_op_attention_static(int32_t R, int32_t n_head, const float *q, const void *kv_layer,
                                    const int32_t *page_table, int32_t pages_per_stream,
                                    const int32_t *row_stream, const int32_t *row_pos, void *out,
                                    void *cuda_stream);

/* LayerNorm over rows: x fp32 [R,d], g/b bf16 [d] -> out bf16 [R,d]. */
int32_t tts_gpt_op_layernorm(int32_t R, int32_t d, const float *x, const void *g, const void *b,
                             float eps, void *out, void *cuda_stream);

/* Sampling (Section I: sampling strategies of the decode engine): logits fp32 [R,V]; top_k <= 1
 * greedy, else top-k softmax at `temperature` with inverse CDF on uniforms[r]; tokens int32 [R]. */
int32_t tts_gpt_op_sample(int32_t R, int32_t V, const float *logits, int32_t top_k,
                          float temperature, const float *uniforms, int32_t *tokens,
                          void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* TTS_GPT_H_ */
