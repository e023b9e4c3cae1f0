// C ABI of the decode engine: host-side validation, workspace carving, the step schedule.
// All arithmetic of the step happens in the kernels of the headers included below.
#include "../../include/tts_gpt.h"

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstdarg>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "linear.cuh"
#include "attention.cuh"
#include "attention_prefill.cuh"
#include "gemm_tc.cuh"
#include "attention_prefill_tc.cuh"
#include "elementwise.cuh"
#include "kv_pages.cuh"
#include "kv_fp8.cuh"

using namespace ttsgpt;

namespace {

thread_local std::string g_last_error;

struct PackedLinear {
  void *w_img = nullptr;   // bf16 only: operand image for the tensor-core path (rows padded to 128)
  void *w = nullptr;
  uint16_t *s = nullptr;
  uint16_t *bias = nullptr;
  int N = 0, K = 0;
};

struct LayerW {
  uint16_t *ln1_g, *ln1_b, *ln2_g, *ln2_b;
  PackedLinear qkv, o, fc1, fc2;
};

}  // namespace

struct tts_gpt {
  tts_gpt_config_t cfg;
  cudaStream_t stream;
  int pps;  // pages per stream
  std::string err;
  // weights (workspace)
  uint16_t *tok_emb, *pos_emb, *lnf_g, *lnf_b;
  PackedLinear head;
  std::vector<LayerW> layers;
  // KV pool
  uint16_t *kv;
  size_t kv_layer_elems;      // 16-bit units of one layer's slice of the pool
  size_t kv_page_elems;       // ... of one page in one layer
  bool kv_fp8 = false;        // e4m3 pages with a scale per cached row and head
  uint16_t *kv_scratch = nullptr;   // 8-bit cache: bf16 pages decoded for the tensor-core prefill attention [kScratchPages][2][H][64*64]
  int *scratch_table = nullptr, *scratch_src = nullptr, *scratch_ntok = nullptr;
  int pass_scratch = 0;             // scratch pages of the prefill pass in flight (0: the pass attends over the codes)
  uint16_t *kv_stage = nullptr;   // 8-bit cache: the pass's new K/V rows as bf16 [kMaxRows][2][d], encoded by kv_quantize_kernel
  // state
  PageState ps;
  RowTable rt;
  StepIO *io;
  // activations
  float *x, *q, *logits;
  int *st_in, *st_tok;          // staging of the host-buffer entry: input tokens, sampled tokens
  float *st_uni, *st_log;       // uniforms, logits [kMaxRows][vocab]
  uint16_t *st_hid;             // hidden rows [kMaxRows][d]
  uint16_t *a, *o, *hbuf, *hf;
  // tensor-core path (more than 16 rows, bf16 weights): activation images and k-split partial sums
  void *a_img = nullptr, *o_img = nullptr, *h_img = nullptr, *hf_img = nullptr;
  float *partials = nullptr;
  bool have_tc = false;
  // attention scratch
  float *attn_partials;
  unsigned int *attn_tickets;
  // host mirrors
  std::vector<char> open;
  std::vector<int> ctx, pos_next;
  int n_free;
  // step graphs by row count
  std::map<int, cudaGraphExec_t> graphs;
  std::map<int, int> graph_nodes;
  bool use_graph;
  bool use_pdl;
  bool use_fc2_ksplit = true;   // 5-16 rows: FC2 splits K (option "fc2_ksplit")
  int pending_parts = 0;        // k-range partial sums of the last FC2 still to be folded into x
  size_t partials_floats = 0;
  bool use_tc = true;   // tensor-core path for more than 16 rows (option "tc")
  bool use_attn_tc = true;   // prefill passes of more than 128 rows: attention on tcgen05 (option "attn_tc")
  bool w4_exact = false;   // int4 weights on the tensor-core path: images hold the integer codes and the kernels scale fp32 group sums (option "w4_tc_exact"); default: images hold code x group scale rounded to bf16
  int prefill_pass_rows = 768;   // rows per prefill pass (option "prefill_pass_rows": a multiple of 128 up to 1024); set at creation
                                 // to the most row tiles whose widest linear still runs as one wave of two CTAs per SM
  int tc_tail_parts = 0;  // partial sums the last FC2 of the tensor-core path left for the final LayerNorm
  bool use_attn_mma = true;      // tensor-core attention in prefill passes (option "attn_mma")
  bool use_attn_prefill = true;  // shared-page attention in prefill passes (option "attn_prefill")
  bool use_attn_stream = true;   // streaming attention for large batches (option "attn_stream")
  int attn_cluster_fill = 1;     // clusters grow until the grid covers the GPU this many times
  int attn_stream_min_pairs = 0; // (row, head) pairs from which it is used; 0: attention_use_stream decides
  int tc_min_rows = 17; // rows from which the tensor-core path is taken (option "tc_min_rows")
  bool poison_free = false;     // option "poison_free_pages": released pages are filled with NaN
  unsigned char *canary_lo = nullptr, *canary_hi = nullptr;   // guard regions either side of the KV pool
  int n_sm = 148;
  unsigned long long launches = 0;
  int *dev_err = nullptr;               // error word set by a kernel whose bounded wait expired:
  volatile int *host_err = nullptr;     //   4 bytes of pinned, device-mapped host memory (read after a sync without a copy)
  unsigned long long *trace = nullptr;  // optional device buffer for kernel timelines
  int trace_next = 0;  // kernels enqueued so far (graph nodes counted per replay)
};

namespace {

int fail(tts_gpt *h, int code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (h) h->err = buf;
  g_last_error = buf;
  return code;
}

#define CUDA_TRY(h, expr)                                                                      \
  do {                                                                                         \
    cudaError_t e_ = (expr);                                                                   \
    if (e_ != cudaSuccess) return fail(h, TTS_GPT_E_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

int check_config(const tts_gpt_config_t *c) {
  if (!c) return fail(nullptr, TTS_GPT_E_ARG, "null config");
  if (c->head_dim != 64 || c->page_tokens != 64) return fail(nullptr, TTS_GPT_E_UNSUPPORTED, "head_dim and page_tokens must be 64");
  if (c->n_layer < 1 || c->n_head < 1 || c->d_model != c->n_head * 64) return fail(nullptr, TTS_GPT_E_ARG, "d_model must equal n_head*64");
  if (c->d_model % 128 || c->d_ff % 128 || c->d_ff < 128) return fail(nullptr, TTS_GPT_E_ARG, "d_model and d_ff must be multiples of 128");
  if (c->d_model > kLnThreads * kLnMaxPerThread) return fail(nullptr, TTS_GPT_E_UNSUPPORTED, "d_model too large");
  if (c->vocab < 2 || c->vocab > kSampleThreads * kSampleMaxPer) return fail(nullptr, TTS_GPT_E_UNSUPPORTED, "vocab out of range");
  if (c->wfmt < 0 || c->wfmt > 2) return fail(nullptr, TTS_GPT_E_ARG, "unknown weight format");
  if (c->max_streams < 1 || c->max_streams > kMaxRows) return fail(nullptr, TTS_GPT_E_ARG, "max_streams must be 1..128");
  if (c->max_context < 64 || c->max_context % 64 || c->max_context > kAttnMaxChunks * kAttnWarps * 64)
    return fail(nullptr, TTS_GPT_E_ARG, "max_context must be a multiple of 64 in 64..2048");
  if (c->n_pages < 1 || c->max_pos < 1) return fail(nullptr, TTS_GPT_E_ARG, "n_pages and max_pos must be positive");
  if (!(c->ln_eps > 0.f)) return fail(nullptr, TTS_GPT_E_ARG, "ln_eps must be positive");
  if (c->emb_rows != 0 && c->emb_rows < c->vocab) return fail(nullptr, TTS_GPT_E_ARG, "emb_rows must be 0 or at least vocab");
  if (c->kv_fmt != TTS_GPT_KV_BF16 && c->kv_fmt != TTS_GPT_KV_FP8_E4M3) return fail(nullptr, TTS_GPT_E_ARG, "unknown KV cache format");
  return TTS_GPT_OK;
}

// rows of the embedding table: the semantic codes and specials the head predicts, then the text region if any
inline int emb_rows_of(const tts_gpt_config_t &c) { return c.emb_rows > 0 ? c.emb_rows : c.vocab; }

constexpr int kScratchPages = 256;          // decoded pages a prefill pass over the 8-bit cache may need
constexpr size_t kCanaryBytes = 4096;      // guard region in front of and behind the KV pool
constexpr unsigned char kCanaryByte = 0xA5;

// Walks the workspace; with base == nullptr only measures.
struct Carver {
  char *base;
  size_t off = 0;
  explicit Carver(void *b) : base((char *)b) {}
  template <typename T>
  T *take(size_t count) {
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off += align256(count * sizeof(T));
    return p;
  }
};

void carve_linear(Carver &cv, PackedLinear &pl, int wf, int N, int K) {
  pl.N = N; pl.K = K;
  pl.w_img = (K % 128 == 0) ? cv.take<char>(weight_image_bytes(N, K)) : nullptr;
  pl.w = cv.take<char>(packed_weight_bytes(wf, N, K));
  size_t sb = packed_scale_bytes(wf, N, K);
  pl.s = sb ? cv.take<uint16_t>(sb / 2) : nullptr;
  pl.bias = cv.take<uint16_t>(N);
}

size_t carve(tts_gpt *h, void *base) {
  const tts_gpt_config_t &c = h->cfg;
  const int d = c.d_model, F = c.d_ff, V = c.vocab, S = c.max_streams;
  h->pps = c.max_context / 64;
  Carver cv(base);
  h->tok_emb = cv.take<uint16_t>((size_t)emb_rows_of(c) * d);
  h->pos_emb = cv.take<uint16_t>((size_t)c.max_pos * d);
  h->lnf_g = cv.take<uint16_t>(d);
  h->lnf_b = cv.take<uint16_t>(d);
  carve_linear(cv, h->head, WF_BF16, V, d);
  h->layers.resize(c.n_layer);
  for (auto &L : h->layers) {
    L.ln1_g = cv.take<uint16_t>(d); L.ln1_b = cv.take<uint16_t>(d);
    L.ln2_g = cv.take<uint16_t>(d); L.ln2_b = cv.take<uint16_t>(d);
    carve_linear(cv, L.qkv, c.wfmt, 3 * d, d);
    carve_linear(cv, L.o, c.wfmt, d, d);
    carve_linear(cv, L.fc1, c.wfmt, F, d);
    carve_linear(cv, L.fc2, c.wfmt, d, F);
  }
  h->kv_fp8 = c.kv_fmt == TTS_GPT_KV_FP8_E4M3;
  h->kv_page_elems = (size_t)2 * c.n_head * (h->kv_fp8 ? (size_t)kFp8BlockBytes / 2 : (size_t)kPageElems);   // 16-bit units of a page in one layer
  h->kv_layer_elems = (size_t)c.n_pages * h->kv_page_elems;
  h->canary_lo = cv.take<unsigned char>(kCanaryBytes);
  h->kv = cv.take<uint16_t>(h->kv_layer_elems * c.n_layer);
  h->canary_hi = cv.take<unsigned char>(kCanaryBytes);
  PageState &ps = h->ps;
  ps.pps = h->pps; ps.n_pages = c.n_pages; ps.max_streams = S;
  ps.ctx_len = cv.take<int>(S);
  ps.page_table = cv.take<int>((size_t)S * h->pps);
  ps.free_list = cv.take<int>(c.n_pages);
  ps.free_top = cv.take<int>(1);
  ps.last_token = cv.take<int>(S);
  ps.pos_next = cv.take<int>(S);
  ps.stop_flag = cv.take<int>(S);
  ps.stream_emb = cv.take<const uint16_t *>(S);
  ps.stream_text = cv.take<const int *>(S);
  ps.stream_ncond = cv.take<int>(S);
  RowTable &rt = h->rt;
  rt.row_stream = cv.take<int>(kMaxPassRows);
  rt.row_pos = cv.take<int>(kMaxPassRows);
  rt.row_token = cv.take<int>(kMaxPassRows);
  rt.row_posidx = cv.take<int>(kMaxPassRows);
  rt.row_emb = cv.take<const uint16_t *>(kMaxPassRows);
  rt.out_rows = cv.take<int>(kMaxRows);
  rt.out_slot = cv.take<int>(kMaxRows);
  rt.row_order = cv.take<int>(kMaxRows);
  h->io = cv.take<StepIO>(1);
  h->x = cv.take<float>((size_t)kMaxPassRows * d);
  h->q = cv.take<float>((size_t)kMaxPassRows * d);
  h->logits = cv.take<float>((size_t)kMaxRows * V);
  h->st_in = cv.take<int>(kMaxRows);
  h->st_tok = cv.take<int>(kMaxRows);
  h->st_uni = cv.take<float>(kMaxRows);
  h->st_log = cv.take<float>((size_t)kMaxRows * V);
  h->st_hid = cv.take<uint16_t>((size_t)kMaxRows * d);
  h->a = cv.take<uint16_t>((size_t)kMaxRows * d);
  h->o = cv.take<uint16_t>((size_t)kMaxRows * d);
  h->hbuf = cv.take<uint16_t>((size_t)kMaxRows * F);
  h->hf = cv.take<uint16_t>((size_t)kMaxRows * d);
  h->kv_stage = h->kv_fp8 ? cv.take<uint16_t>((size_t)kMaxPassRows * 2 * d) : nullptr;
  if (h->kv_fp8) {
    h->kv_scratch = cv.take<uint16_t>((size_t)kScratchPages * 2 * c.n_head * kPageElems);
    h->scratch_table = cv.take<int>((size_t)S * h->pps);
    h->scratch_src = cv.take<int>(kScratchPages);
    h->scratch_ntok = cv.take<int>(kScratchPages);
  }
  const size_t attn_rows = h->kv_fp8 ? kMaxPassRows : kMaxRows;   // the 8-bit cache's attention kernel also serves prefill passes
  h->attn_partials = cv.take<float>(attn_rows * c.n_head * kAttnMaxChunks * kAttnPartialFloats);
  h->attn_tickets = cv.take<unsigned int>(attn_rows * c.n_head);
  h->have_tc = true;
  if (h->have_tc) {
    constexpr int kTiles = kMaxPassRows / kMaxRows;   // row tiles of a prefill pass
    h->a_img = cv.take<char>(kTiles * act_image_bytes(d));
    h->o_img = cv.take<char>(kTiles * act_image_bytes(d));
    h->h_img = cv.take<char>(kTiles * act_image_bytes(F));
    h->hf_img = cv.take<char>(act_image_bytes(d));
    h->partials_floats = (size_t)kTiles * std::max(kTcKSplit, kTwMaxPartials) * kMaxRows * d;   // [row tile][k-range][128][d]
    h->partials = cv.take<float>(h->partials_floats);
  }
  return cv.off;
}

int copy_bf16(tts_gpt *h, uint16_t *dst, const void *src, size_t n, const char *what) {
  if (!src) return fail(h, TTS_GPT_E_ARG, "weights: %s is null", what);
  CUDA_TRY(h, cudaMemcpyAsync(dst, src, n * 2, cudaMemcpyDeviceToDevice, h->stream));
  return TTS_GPT_OK;
}

// int4 weights: the operand images of the tensor-core path, written from the packed streaming layout.  Default: code x
// group scale rounded once to bf16, so that the linears of more than 16 rows run as plain bf16 contractions; with
// w4_exact: the integer codes, and the kernels scale the fp32 sums of each 128-column group.
int write_int4_images(tts_gpt *h) {
  for (int l = 0; l < h->cfg.n_layer; ++l) {
    LayerW &L = h->layers[l];
    const PackedLinear *pl[4] = {&L.qkv, &L.o, &L.fc1, &L.fc2};
    Int4ImageArgs da;
    memset(&da, 0, sizeof da);
    da.raw = h->w4_exact ? 1 : 0;
    unsigned long long end = 0;
    for (int i = 0; i < 4; ++i) {
      if (!pl[i]->w_img) return TTS_GPT_OK;   // no tensor-core path for this shape
      da.src[i] = (const uint4 *)pl[i]->w; da.dst[i] = (uint4 *)pl[i]->w_img; da.scales[i] = pl[i]->s;
      da.K[i] = pl[i]->K;
      end += packed_weight_bytes(WF_INT4, pl[i]->N, pl[i]->K) / 16;
      da.unit_end[i] = end;
    }
    int4_weight_images_kernel<<<(unsigned)((end + 255) / 256), 256, 0, h->stream>>>(da);
    CUDA_TRY(h, cudaGetLastError());
  }
  return TTS_GPT_OK;
}

int load_linear(tts_gpt *h, PackedLinear &pl, int wf, const void *w, const void *s, const void *b, const char *what) {
  if (!w || !b || (wf != WF_BF16 && !s)) return fail(h, TTS_GPT_E_ARG, "weights: %s has a null tensor", what);
  CUDA_TRY(h, launch_pack(wf, pl.N, pl.K, w, s, pl.w, pl.s, h->stream));
  if (pl.w_img && wf == WF_INT4) CUDA_TRY(h, cudaMemsetAsync(pl.w_img, 0, weight_image_bytes(pl.N, pl.K), h->stream));   // written by write_int4_images; rows past the last 8-row tile stay zero
  else if (pl.w_img) CUDA_TRY(h, launch_pack_image(wf, pl.N, pl.K, w, pl.w_img, h->stream));
  CUDA_TRY(h, cudaMemcpyAsync(pl.bias, b, (size_t)pl.N * 2, cudaMemcpyDeviceToDevice, h->stream));
  return TTS_GPT_OK;
}

LinearArgs linear_args(const PackedLinear &pl, const uint16_t *act, int B, int mode) {
  LinearArgs a;
  memset(&a, 0, sizeof a);
  a.w = pl.w; a.scales = pl.s; a.bias = pl.bias; a.act = act;
  a.N = pl.N; a.K = pl.K; a.B = B; a.mode = mode;
  return a;
}
LinearArgs linear_args(tts_gpt *h, const PackedLinear &pl, const uint16_t *act, int B, int mode);

LinearArgs linear_args(tts_gpt *h, const PackedLinear &pl, const uint16_t *act, int B, int mode) {
  LinearArgs a = linear_args(pl, act, B, mode);
  a.err = h->dev_err;
  return a;
}

// gives the next traced kernel of a step its slot
template <typename Args>
void trace_attach(tts_gpt *h, Args &a) {
  a.trace = h->trace;
  a.trace_slot = h->trace ? h->trace_next++ : 0;
}

// Attention for R rows: clusters while (row, head) pairs are scarce, one streaming CTA per pair
// once they cover the GPU several times.
cudaError_t run_attention(tts_gpt *h, AttnArgs &aa, int R, cudaStream_t st, bool pdl) {
  if (h->kv_fp8) {
    // 8-bit cache: the QKV linear left the new K/V rows in the staging area; encode them into their page
    // slots, then attend over e4m3 pages (the same kernel for prefill passes and decode steps)
    unsigned char *kvl = reinterpret_cast<unsigned char *>(const_cast<uint16_t *>(aa.kv_layer));
    cudaError_t e = launch_kv_quantize(h->kv_stage, kvl, aa.page_table, aa.row_stream, aa.row_pos, aa.pps, aa.H, R, st, pdl);
    if (e != cudaSuccess) return e;
    h->launches += 1;
    if (!aa.old_pages_final && h->pass_scratch > 0 && h->use_attn_mma && R >= kAttnPrefillRows) {
      // prefill pass: decode the pages its rows attend over into bf16 scratch pages, then the tensor-core kernel
      e = launch_kv_dequant_pages(kvl, h->kv_scratch, h->scratch_src, h->scratch_ntok, h->pass_scratch, aa.H, st, pdl);
      if (e != cudaSuccess) return e;
      h->launches += 1;
      aa.kv_layer = h->kv_scratch; aa.page_table = h->scratch_table; aa.err = h->dev_err; aa.row_order = nullptr;
      if (h->use_attn_tc && R > kMaxRows) return launch_attention_prefill_tc(aa, R, st, pdl);
      return launch_attention_prefill_mma(aa, R, st, pdl);
    }
    Fp8AttnArgs fa;
    memset(&fa, 0, sizeof fa);
    fa.q = aa.q; fa.kv_layer = kvl; fa.page_table = aa.page_table; fa.row_stream = aa.row_stream; fa.row_pos = aa.row_pos;
    fa.out = aa.out; fa.partials = h->attn_partials; fa.tickets = h->attn_tickets; fa.H = aa.H; fa.pps = aa.pps;
    fa.out_image = aa.out_image; fa.trace = aa.trace; fa.trace_slot = aa.trace_slot;
    fa.err = h->dev_err;
    const bool many = h->attn_stream_min_pairs > 0 ? R * aa.H >= h->attn_stream_min_pairs : attention_use_stream(R, aa.H, h->n_sm);
    if (aa.old_pages_final && h->use_attn_stream && many) {   // decode steps with enough (row, head) pairs
      fa.row_order = h->rt.row_order;
      return launch_attention_fp8_stream(fa, R, st, pdl);
    }
    return launch_attention_fp8(fa, R, attention_fp8_splits(R, aa.H, h->n_sm), st, pdl);
  }
  aa.err = h->dev_err;
  aa.row_order = aa.old_pages_final ? h->rt.row_order : nullptr;   // written by the decode step's set-up kernel
  // prefill passes: rows of one stream share their pages (one CTA per 16 rows and head on the tensor cores;
  // the CUDA-core variant with 8 rows per CTA stays selectable)
  // (passes of several row tiles: 128 rows per CTA on tcgen05)
  if (!aa.old_pages_final && h->use_attn_mma && h->use_attn_tc && R > kMaxRows) return launch_attention_prefill_tc(aa, R, st, pdl);
  if (!aa.old_pages_final && h->use_attn_mma && R >= kAttnPrefillRows) return launch_attention_prefill_mma(aa, R, st, pdl);
  if (!aa.old_pages_final && h->use_attn_prefill && R >= kAttnPrefillRows) return launch_attention_prefill(aa, R, st, pdl);
  const bool stream = h->attn_stream_min_pairs > 0 ? R * aa.H >= h->attn_stream_min_pairs : attention_use_stream(R, aa.H, h->n_sm);
  if (h->use_attn_stream && stream) return launch_attention_stream(aa, R, st, pdl);
  return launch_attention(aa, R, attention_cluster_size(R, aa.H, h->n_sm, h->attn_cluster_fill), st, pdl);
}

// The transformer blocks for R rows already described by the row table, x holding the input rows.
// Every kernel after the first of a step is launched with programmatic dependent launch, so its
// weight loads overlap the tail of its predecessor.
// ---- tensor-core path: more than 16 rows, bf16 weights ----
GemmTcArgs gemm_args(tts_gpt *h, const PackedLinear &pl, const void *act_img, int B, int mode, int ksplit) {
  GemmTcArgs a;
  memset(&a, 0, sizeof a);
  // the LM head has no scales: bf16 in every format; int4 images hold dequantized weights unless the exact form is on
  const bool plain = !pl.s || (h->cfg.wfmt == WF_INT4 && !h->w4_exact);
  a.wfmt = plain ? WF_BF16 : h->cfg.wfmt;
  a.scales = plain ? nullptr : pl.s;
  a.w_img = pl.w_img; a.act_img = act_img; a.bias = pl.bias; a.N = pl.N; a.K = pl.K; a.B = B; a.mode = mode;
  a.ksplit = ksplit; a.err = h->dev_err;
  return a;
}

int launch_ln_tc(tts_gpt *h, int rows, const uint16_t *g, const uint16_t *b, int n_part, const uint16_t *add_bias,
                 void *out_img, uint16_t *out_plain, const int *gather, const int *out_slot, const StepIO *io,
                 int write_back) {
  LnTcArgs la;
  memset(&la, 0, sizeof la);
  la.x = h->x; la.d = h->cfg.d_model; la.partials = h->partials; la.n_part = n_part; la.part_cols = h->cfg.d_model;
  la.add_bias = add_bias; la.g = g; la.b = b; la.eps = h->cfg.ln_eps; la.out_img = out_img; la.out_plain = out_plain;
  la.gather = gather; la.out_slot = out_slot; la.io = io; la.write_back = write_back;
  trace_attach(h, la);
  const int np = (h->cfg.d_model + kLnThreads - 1) / kLnThreads;
  const dim3 grid(rows), block(kLnThreads);
  if (rows > kMaxRows && h->cfg.d_model % 8 == 0) {
    // the many rows of a large prefill pass: one warp per row
    const dim3 rgrid((rows + kLnRowsWarps - 1) / kLnRowsWarps), rblock(kLnRowsWarps * 32);
    if (np <= 1) CUDA_TRY(h, launch_kernel(layernorm_rows_kernel<2>, rgrid, rblock, 0, h->stream, h->use_pdl, la, rows));
    else if (np <= 5) CUDA_TRY(h, launch_kernel(layernorm_rows_kernel<10>, rgrid, rblock, 0, h->stream, h->use_pdl, la, rows));
    else CUDA_TRY(h, launch_kernel(layernorm_rows_kernel<2 * kLnMaxPerThread>, rgrid, rblock, 0, h->stream, h->use_pdl, la, rows));
  } else if (np <= 1) CUDA_TRY(h, launch_kernel(layernorm_tc_kernel<1>, grid, block, 0, h->stream, h->use_pdl, la));
  else if (np <= 5) CUDA_TRY(h, launch_kernel(layernorm_tc_kernel<5>, grid, block, 0, h->stream, h->use_pdl, la));
  else CUDA_TRY(h, launch_kernel(layernorm_tc_kernel<kLnMaxPerThread>, grid, block, 0, h->stream, h->use_pdl, la));
  h->launches += 1;
  return TTS_GPT_OK;
}

int launch_gemm(tts_gpt *h, const GemmTcArgs &a, bool wide, cudaStream_t st, bool pdl) {
  CUDA_TRY(h, wide ? launch_gemm_tcw(a, h->n_sm, st, pdl) : launch_gemm_tc(a, st, pdl));
  return TTS_GPT_OK;
}

// Up to 128 rows (decode steps, small prefill passes): the kernel with chunks of 32 batch rows, O-proj and FC2
// split over 4 k-ranges.  More rows (prefill passes of several row tiles): the wide kernel, one CTA per 128 rows
// x 128 features; O-proj and FC2 split over up to 4 k-ranges.  Either way the next LayerNorm folds the ranges.
int run_layers_tc(tts_gpt *h, int R, bool decode) {
  const tts_gpt_config_t &c = h->cfg;
  const int d = c.d_model;
  cudaStream_t st = h->stream;
  const bool pdl = h->use_pdl;
  const bool wide = R > kMaxRows;
  const int o_ks = wide ? tcw_ksplit_resid(d) : kTcKSplit;
  const int f2_ks = wide ? tcw_ksplit_resid(c.d_ff) : kTcKSplit;
  const int o_parts = o_ks > 1 ? o_ks : 0, f2_parts = f2_ks > 1 ? f2_ks : 0;   // 0: the linear added into x itself
  for (int l = 0; l < c.n_layer; ++l) {
    LayerW &L = h->layers[l];
    uint16_t *kvl = h->kv + h->kv_layer_elems * l;
    int rc;
    // fold the previous layer's FC2 partial sums into x, then LN1 -> image
    rc = launch_ln_tc(h, R, L.ln1_g, L.ln1_b, l == 0 ? 0 : f2_parts, l == 0 ? nullptr : h->layers[l - 1].fc2.bias,
                      h->a_img, nullptr, nullptr, nullptr, nullptr, 1);
    if (rc) return rc;
    GemmTcArgs qa = gemm_args(h, L.qkv, h->a_img, R, EPI_QKV, 1);
    qa.out_f32 = h->q; qa.out_stride = d; qa.kv_layer = kvl; qa.page_table = h->ps.page_table;
    qa.row_stream = h->rt.row_stream; qa.row_pos = h->rt.row_pos; qa.pps = h->pps; qa.d = d; qa.H = c.n_head;
    qa.kv_stage = h->kv_stage;
    trace_attach(h, qa);
    if ((rc = launch_gemm(h, qa, wide, st, pdl))) return rc;
    AttnArgs aa;
    memset(&aa, 0, sizeof aa);
    aa.q = h->q; aa.kv_layer = kvl; aa.page_table = h->ps.page_table; aa.row_stream = h->rt.row_stream;
    aa.row_pos = h->rt.row_pos; aa.out = (uint16_t *)h->o_img; aa.out_image = 1;
    aa.H = c.n_head; aa.pps = h->pps; aa.old_pages_final = decode ? 1 : 0;
    trace_attach(h, aa);
    CUDA_TRY(h, run_attention(h, aa, R, st, pdl));
    GemmTcArgs oa = gemm_args(h, L.o, h->o_img, R, EPI_RESID, o_ks);
    oa.out_f32 = o_parts ? h->partials : h->x; oa.out_stride = d;
    trace_attach(h, oa);
    if ((rc = launch_gemm(h, oa, wide, st, pdl))) return rc;
    rc = launch_ln_tc(h, R, L.ln2_g, L.ln2_b, o_parts, L.o.bias, h->a_img, nullptr, nullptr, nullptr, nullptr, 1);
    if (rc) return rc;
    GemmTcArgs f1 = gemm_args(h, L.fc1, h->a_img, R, EPI_GELU, 1);
    f1.out_img = h->h_img; f1.gelu_tanh = c.gelu_tanh;
    trace_attach(h, f1);
    if ((rc = launch_gemm(h, f1, wide, st, pdl))) return rc;
    GemmTcArgs f2 = gemm_args(h, L.fc2, h->h_img, R, EPI_RESID, f2_ks);
    f2.out_f32 = f2_parts ? h->partials : h->x; f2.out_stride = d;
    trace_attach(h, f2);
    if ((rc = launch_gemm(h, f2, wide, st, pdl))) return rc;
    h->launches += 5;
  }
  h->tc_tail_parts = f2_parts;
  return TTS_GPT_OK;
}

// Final LayerNorm (folding the last FC2's partial sums), LM head, sampling after run_layers_tc.
int run_head_tc(tts_gpt *h, int n_out) {
  const tts_gpt_config_t &c = h->cfg;
  cudaStream_t st = h->stream;
  const bool pdl = h->use_pdl;
  const bool big = n_out > 16;
  int rc = launch_ln_tc(h, n_out, h->lnf_g, h->lnf_b, h->tc_tail_parts, h->layers[c.n_layer - 1].fc2.bias,
                        big ? h->hf_img : nullptr, big ? nullptr : h->hf, h->rt.out_rows, h->rt.out_slot, h->io, 0);
  if (rc) return rc;
  if (big) {
    GemmTcArgs ha = gemm_args(h, h->head, h->hf_img, n_out, EPI_F32, 1);
    ha.out_f32 = h->logits; ha.out_stride = c.vocab;
    CUDA_TRY(h, launch_gemm_tc(ha, st, pdl));
  } else {
    LinearArgs ha = linear_args(h, h->head, h->hf, n_out, EPI_F32);
    ha.out_f32 = h->logits; ha.out_stride = c.vocab;
    CUDA_TRY(h, launch_linear(WF_BF16, ha, st, pdl, 2 * h->n_sm));
  }
  SampleArgs sa;
  memset(&sa, 0, sizeof sa);
  sa.logits = h->logits; sa.V = c.vocab; sa.io = h->io; sa.out_slot = h->rt.out_slot; sa.out_rows = h->rt.out_rows;
  sa.row_stream = h->rt.row_stream; sa.last_token = h->ps.last_token; sa.stop_flag = h->ps.stop_flag;
  sa.stop_token = c.stop_token;
  CUDA_TRY(h, launch_kernel(sample_kernel, dim3(n_out), dim3(kSampleThreads), (size_t)c.vocab * sizeof(float), st, pdl, sa));
  h->launches += 2;
  return TTS_GPT_OK;
}

bool use_tc_path(const tts_gpt *h, int R) {
  return h->have_tc && h->use_tc && R >= h->tc_min_rows;
}

int run_layers(tts_gpt *h, int R, bool decode) {
  h->trace_next = 0;
  if (use_tc_path(h, R)) return run_layers_tc(h, R, decode);
  const tts_gpt_config_t &c = h->cfg;
  const int d = c.d_model;
  cudaStream_t st = h->stream;
  const bool pdl = h->use_pdl;
  const bool fuse_ln = can_fuse_ln(c.wfmt, R, d);
  // 5 to 16 rows: FC2 (K = d_ff) splits K over kSmallKSplit CTAs per row tile, so that a CTA stages a
  // quarter of the wide activation rows; its partial sums are folded into x by the next LayerNorm
  const int fc2_ks = (!fuse_ln && h->use_fc2_ksplit && (c.d_ff / k_per_tile(c.wfmt)) % kSmallKSplit == 0 &&
                      (size_t)kSmallKSplit * kMaxRows * d <= h->partials_floats) ? kSmallKSplit : 1;
  h->pending_parts = 0;
  for (int l = 0; l < c.n_layer; ++l) {
    LayerW &L = h->layers[l];
    uint16_t *kvl = h->kv + h->kv_layer_elems * l;
    {
      LinearArgs qa = linear_args(h, L.qkv, h->a, R, EPI_QKV);
      if (fuse_ln) {
        qa.ln_x = h->x; qa.ln_g = L.ln1_g; qa.ln_b = L.ln1_b; qa.ln_eps = c.ln_eps;
      } else if (fc2_ks > 1) {
        int rc = launch_ln_tc(h, R, L.ln1_g, L.ln1_b, l == 0 ? 0 : fc2_ks, l == 0 ? nullptr : h->layers[l - 1].fc2.bias,
                              nullptr, h->a, nullptr, nullptr, nullptr, 1);
        if (rc) return rc;
      } else {
        CUDA_TRY(h, launch_kernel(layernorm_kernel, dim3(R), dim3(kLnThreads), 0, st, pdl, (const float *)h->x, d,
                                  (const uint16_t *)L.ln1_g, (const uint16_t *)L.ln1_b, c.ln_eps, h->a,
                                  (const int *)nullptr, (const int *)nullptr, (const StepIO *)nullptr));
        h->launches += 1;
      }
      qa.out_f32 = h->q; qa.out_stride = d; qa.kv_layer = kvl; qa.page_table = h->ps.page_table;
      qa.row_stream = h->rt.row_stream; qa.row_pos = h->rt.row_pos; qa.pps = h->pps; qa.d = d; qa.H = c.n_head;
      qa.kv_stage = h->kv_stage;
      trace_attach(h, qa);
      CUDA_TRY(h, launch_linear(c.wfmt, qa, st, pdl, 2 * h->n_sm));
      AttnArgs aa;
      memset(&aa, 0, sizeof aa);
      aa.q = h->q; aa.kv_layer = kvl; aa.page_table = h->ps.page_table; aa.row_stream = h->rt.row_stream;
      aa.row_pos = h->rt.row_pos; aa.out = h->o; aa.partials = h->attn_partials; aa.tickets = h->attn_tickets;
      aa.H = c.n_head; aa.pps = h->pps; aa.old_pages_final = decode ? 1 : 0;
      trace_attach(h, aa);
      CUDA_TRY(h, run_attention(h, aa, R, st, pdl));
    }
    LinearArgs oa = linear_args(h, L.o, h->o, R, EPI_RESID);
    oa.out_f32 = h->x; oa.out_stride = d;
    trace_attach(h, oa);
    CUDA_TRY(h, launch_linear(c.wfmt, oa, st, pdl, 2 * h->n_sm));
    LinearArgs f1 = linear_args(h, L.fc1, h->a, R, EPI_GELU);
    if (fuse_ln) {
      f1.ln_x = h->x; f1.ln_g = L.ln2_g; f1.ln_b = L.ln2_b; f1.ln_eps = c.ln_eps;
    } else {
      CUDA_TRY(h, launch_kernel(layernorm_kernel, dim3(R), dim3(kLnThreads), 0, st, pdl, (const float *)h->x, d,
                                (const uint16_t *)L.ln2_g, (const uint16_t *)L.ln2_b, c.ln_eps, h->a,
                                (const int *)nullptr, (const int *)nullptr, (const StepIO *)nullptr));
      h->launches += 1;
    }
    f1.out_bf16 = h->hbuf; f1.gelu_tanh = c.gelu_tanh;
    trace_attach(h, f1);
    CUDA_TRY(h, launch_linear(c.wfmt, f1, st, pdl, 2 * h->n_sm));
    LinearArgs f2 = linear_args(h, L.fc2, h->hbuf, R, EPI_RESID);
    f2.out_f32 = h->x; f2.out_stride = d;
    if (fc2_ks > 1) { f2.ksplit = fc2_ks; f2.out_f32 = h->partials; }
    trace_attach(h, f2);
    CUDA_TRY(h, launch_linear(c.wfmt, f2, st, pdl, 2 * h->n_sm));
    h->launches += 5;
  }
  h->pending_parts = fc2_ks > 1 ? fc2_ks : 0;   // the last FC2's partial sums: folded by the head's LayerNorm
  return TTS_GPT_OK;
}

// Final LayerNorm (gathered to the wanted rows), LM head, sampling.
int run_head(tts_gpt *h, int n_out, int R) {
  if (use_tc_path(h, R)) return run_head_tc(h, n_out);
  const tts_gpt_config_t &c = h->cfg;
  cudaStream_t st = h->stream;
  const bool pdl = h->use_pdl;
  LinearArgs ha = linear_args(h, h->head, h->hf, n_out, EPI_F32);
  const uint16_t *last_bias = h->layers[c.n_layer - 1].fc2.bias;
  if (h->pending_parts > 0) {
    // the last FC2 left k-range partial sums: this LayerNorm folds them for the wanted rows and
    // writes the normalised rows; the head then runs on those (never on x)
    int rc = launch_ln_tc(h, n_out, h->lnf_g, h->lnf_b, h->pending_parts, last_bias, nullptr, h->hf, h->rt.out_rows,
                          h->rt.out_slot, h->io, 0);
    if (rc) return rc;
    h->pending_parts = 0;
  } else if (can_fuse_ln(WF_BF16, n_out, c.d_model)) {
    ha.ln_x = h->x; ha.ln_g = h->lnf_g; ha.ln_b = h->lnf_b; ha.ln_eps = c.ln_eps;
    ha.ln_gather = h->rt.out_rows; ha.ln_out_slot = h->rt.out_slot; ha.ln_io = h->io;
  } else {
    CUDA_TRY(h, launch_kernel(layernorm_kernel, dim3(n_out), dim3(kLnThreads), 0, st, pdl, (const float *)h->x,
                              c.d_model, (const uint16_t *)h->lnf_g, (const uint16_t *)h->lnf_b, c.ln_eps, h->hf,
                              (const int *)h->rt.out_rows, (const int *)h->rt.out_slot, (const StepIO *)h->io));
    h->launches += 1;
  }
  ha.out_f32 = h->logits; ha.out_stride = c.vocab;
  trace_attach(h, ha);
  CUDA_TRY(h, launch_linear(WF_BF16, ha, st, pdl, 2 * h->n_sm));
  SampleArgs sa;
  memset(&sa, 0, sizeof sa);
  sa.logits = h->logits; sa.V = c.vocab; sa.io = h->io; sa.out_slot = h->rt.out_slot; sa.out_rows = h->rt.out_rows;
  sa.row_stream = h->rt.row_stream; sa.last_token = h->ps.last_token; sa.stop_flag = h->ps.stop_flag;
  sa.stop_token = c.stop_token;
  CUDA_TRY(h, launch_kernel(sample_kernel, dim3(n_out), dim3(kSampleThreads), (size_t)c.vocab * sizeof(float), st, pdl, sa));
  h->launches += 2;
  return TTS_GPT_OK;
}

int run_embed(tts_gpt *h, int R) {
  const tts_gpt_config_t &c = h->cfg;
  embed_kernel<<<R, 256, 0, h->stream>>>(h->rt, h->tok_emb, h->pos_emb, c.d_model, emb_rows_of(c), c.max_pos, h->x);
  CUDA_TRY(h, cudaGetLastError());
  h->launches += 1;
  return TTS_GPT_OK;
}

// Output rows are written with vector stores: the hidden rows need 16-byte alignment, the rest their
// element's.  A misaligned pointer is refused here instead of faulting on the device.
int check_io_alignment(tts_gpt *h, const void *in_tokens, const void *uniforms, const void *out_tokens,
                       const void *out_logits, const void *out_hidden) {
  if ((uintptr_t)in_tokens % 4 || (uintptr_t)uniforms % 4 || (uintptr_t)out_tokens % 4 || (uintptr_t)out_logits % 4)
    return fail(h, TTS_GPT_E_ARG, "token, uniform and logit buffers must be 4-byte aligned");
  if ((uintptr_t)out_hidden % 16) return fail(h, TTS_GPT_E_ARG, "out_hidden must be 16-byte aligned");
  return TTS_GPT_OK;
}

int check_top_k(tts_gpt *h, int top_k, float temperature, const float *uniforms) {
  if (top_k < 0 || top_k > kMaxTopK) return fail(h, TTS_GPT_E_ARG, "top_k must be in 0..%d", kMaxTopK);
  if (top_k > 1 && !(temperature > 0.f)) return fail(h, TTS_GPT_E_ARG, "temperature must be positive");
  if (top_k > 1 && !uniforms) return fail(h, TTS_GPT_E_ARG, "top-k sampling needs uniforms");
  return TTS_GPT_OK;
}

}  // namespace

extern "C" {

int32_t tts_gpt_query_workspace(const tts_gpt_config_t *cfg, size_t *bytes) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!bytes) return fail(nullptr, TTS_GPT_E_ARG, "null bytes");
  tts_gpt tmp;
  tmp.cfg = *cfg;
  *bytes = carve(&tmp, nullptr);
  return TTS_GPT_OK;
}

int32_t tts_gpt_create(const tts_gpt_config_t *cfg, const tts_gpt_weights_t *w, void *workspace,
                       size_t workspace_bytes, void *cuda_stream, tts_gpt_t **out) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!w || !workspace || !out) return fail(nullptr, TTS_GPT_E_ARG, "null argument");
  if ((uintptr_t)workspace % 256) return fail(nullptr, TTS_GPT_E_WORKSPACE, "workspace must be 256-byte aligned");
  tts_gpt *h = new (std::nothrow) tts_gpt();
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "out of host memory");
  h->cfg = *cfg;
  h->stream = (cudaStream_t)cuda_stream;
  const size_t need = carve(h, workspace);
  if (need > workspace_bytes) {
    delete h;
    return fail(nullptr, TTS_GPT_E_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
  }
  const tts_gpt_config_t &c = h->cfg;
  const int d = c.d_model;
#define TRY_(expr) do { rc = (expr); if (rc) { g_last_error = h->err; delete h; return rc; } } while (0)
  TRY_(copy_bf16(h, h->tok_emb, w->tok_emb, (size_t)emb_rows_of(c) * d, "tok_emb"));
  TRY_(copy_bf16(h, h->pos_emb, w->pos_emb, (size_t)c.max_pos * d, "pos_emb"));
  TRY_(copy_bf16(h, h->lnf_g, w->lnf_g, d, "lnf_g"));
  TRY_(copy_bf16(h, h->lnf_b, w->lnf_b, d, "lnf_b"));
  if (!w->head_w) { delete h; return fail(nullptr, TTS_GPT_E_ARG, "weights: head_w is null"); }
  {
    cudaError_t e = launch_pack(WF_BF16, h->head.N, h->head.K, w->head_w, nullptr, h->head.w, nullptr, h->stream);
    if (e == cudaSuccess && h->head.w_img) e = launch_pack_image(WF_BF16, h->head.N, h->head.K, w->head_w, h->head.w_img, h->stream);
    if (e != cudaSuccess) { delete h; return fail(nullptr, TTS_GPT_E_CUDA, "pack head: %s", cudaGetErrorString(e)); }
    if (w->head_b) {
      TRY_(copy_bf16(h, h->head.bias, w->head_b, c.vocab, "head_b"));
    } else {
      h->head.bias = nullptr;
    }
  }
  const void *const *per_layer[] = {w->ln1_g, w->ln1_b, w->ln2_g, w->ln2_b, w->qkv_w, w->qkv_b, w->o_w, w->o_b,
                                    w->fc1_w, w->fc1_b, w->fc2_w, w->fc2_b};
  for (auto p : per_layer)
    if (!p) { delete h; return fail(nullptr, TTS_GPT_E_ARG, "weights: a per-layer pointer array is null"); }
  if (c.wfmt != WF_BF16 && (!w->qkv_s || !w->o_s || !w->fc1_s || !w->fc2_s)) {
    delete h;
    return fail(nullptr, TTS_GPT_E_ARG, "weights: scale arrays are required for quantized formats");
  }
  for (int l = 0; l < c.n_layer; ++l) {
    LayerW &L = h->layers[l];
    TRY_(copy_bf16(h, L.ln1_g, w->ln1_g[l], d, "ln1_g"));
    TRY_(copy_bf16(h, L.ln1_b, w->ln1_b[l], d, "ln1_b"));
    TRY_(copy_bf16(h, L.ln2_g, w->ln2_g[l], d, "ln2_g"));
    TRY_(copy_bf16(h, L.ln2_b, w->ln2_b[l], d, "ln2_b"));
    const bool qz = c.wfmt != WF_BF16;
    TRY_(load_linear(h, L.qkv, c.wfmt, w->qkv_w[l], qz ? w->qkv_s[l] : nullptr, w->qkv_b[l], "qkv"));
    TRY_(load_linear(h, L.o, c.wfmt, w->o_w[l], qz ? w->o_s[l] : nullptr, w->o_b[l], "o"));
    TRY_(load_linear(h, L.fc1, c.wfmt, w->fc1_w[l], qz ? w->fc1_s[l] : nullptr, w->fc1_b[l], "fc1"));
    TRY_(load_linear(h, L.fc2, c.wfmt, w->fc2_w[l], qz ? w->fc2_s[l] : nullptr, w->fc2_b[l], "fc2"));
  }
  if (c.wfmt == WF_INT4) TRY_(write_int4_images(h));
#undef TRY_
  const int init_n = std::max(std::max(c.n_pages, c.max_streams * h->pps), c.max_streams);
  init_pages_kernel<<<(init_n + 255) / 256, 256, 0, h->stream>>>(h->ps);
  cudaError_t e = cudaMemsetAsync(h->attn_tickets, 0, (size_t)(h->kv_fp8 ? kMaxPassRows : kMaxRows) * c.n_head * sizeof(unsigned int), h->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->canary_lo, kCanaryByte, kCanaryBytes, h->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->canary_hi, kCanaryByte, kCanaryBytes, h->stream);
  if (e == cudaSuccess) {
    void *hp = nullptr, *dp = nullptr;
    e = cudaHostAlloc(&hp, sizeof(int), cudaHostAllocMapped);
    if (e == cudaSuccess) {
      *(int *)hp = 0;
      e = cudaHostGetDevicePointer(&dp, hp, 0);
      h->host_err = (volatile int *)hp;
      h->dev_err = (int *)dp;
    }
  }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
  if (e != cudaSuccess) {
    if (h->host_err) cudaFreeHost((void *)h->host_err);
    delete h;
    return fail(nullptr, TTS_GPT_E_CUDA, "create: %s", cudaGetErrorString(e));
  }
  h->open.assign(c.max_streams, 0);
  h->ctx.assign(c.max_streams, 0);
  h->pos_next.assign(c.max_streams, 0);
  h->n_free = c.n_pages;
  // the legacy default stream cannot be captured
  h->use_graph = h->stream != nullptr && h->stream != cudaStreamLegacy;
  h->use_pdl = true;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
    h->n_sm = sms;
  {
    // rows per prefill pass: the wide linears run two CTAs per SM; a pass of t row tiles gives the widest linear
    // t x (features / 128) x k-ranges CTAs, and one CTA too many doubles its time.  Measured on 148 SMs with this
    // model (FC1: 40 feature tiles): 88946 prefix rows in 301 / 279 / 308 ms at 6 / 7 / 8 row tiles.
    const tts_gpt_config_t &c = h->cfg;
    const int widest = std::max(std::max((c.d_ff + 127) / 128, (3 * c.d_model + 127) / 128), tcw_ksplit_resid(c.d_ff) * ((c.d_model + 127) / 128));
    const int t = std::max(1, std::min(kMaxPassRows / kMaxRows, 2 * h->n_sm / std::max(1, widest)));
    h->prefill_pass_rows = t * kMaxRows;
  }
  *out = h;
  return TTS_GPT_OK;
}

// Both prefill entries.  text == nullptr: every prefix row is a given embedding (n_cond is then the
// prefix length); otherwise stream i has n_cond[i] given rows followed by n_text[i] text tokens.
static int prefill_impl(tts_gpt_t *h, int32_t n, const void *const *emb, const int32_t *n_cond,
                        const int32_t *const *text, const int32_t *n_text, int32_t text_shift, int32_t text_pos0,
                        const int32_t *pos0, int32_t top_k, float temperature, const float *uniforms,
                        int32_t *out_stream_ids, int32_t *out_tokens, float *out_logits, void *out_hidden) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  const tts_gpt_config_t &c = h->cfg;
  if (n < 1 || n > c.max_streams || !emb || !n_cond || !out_stream_ids || !out_tokens || (text && !n_text))
    return fail(h, TTS_GPT_E_ARG, "prefill: bad n or null argument");
  int rc = check_top_k(h, top_k, temperature, uniforms);
  if (rc) return rc;
  rc = check_io_alignment(h, nullptr, uniforms, out_tokens, out_logits, out_hidden);
  if (rc) return rc;
  if (text && (text_pos0 < 0 || text_pos0 >= c.max_pos)) return fail(h, TTS_GPT_E_ARG, "prefill: text_pos0 out of range");
  int pages = 0;
  int plen[kMaxRows];
  for (int i = 0; i < n; ++i) {
    const int nc = n_cond[i], nt = text ? n_text[i] : 0;
    if (nc < 0 || nt < 0 || nc + nt < 1) return fail(h, TTS_GPT_E_ARG, "prefill: stream %d has an empty prefix", i);
    if (nc > 0 && !emb[i]) return fail(h, TTS_GPT_E_ARG, "prefill: stream %d has no embedding rows", i);
    if (nt > 0 && !text[i]) return fail(h, TTS_GPT_E_ARG, "prefill: stream %d has no text ids", i);
    if (nc > 0 && (uintptr_t)emb[i] % 16) return fail(h, TTS_GPT_E_ARG, "prefill: prefix %d is not 16-byte aligned", i);
    if (nt > 0 && (uintptr_t)text[i] % 4) return fail(h, TTS_GPT_E_ARG, "prefill: text ids %d are not 4-byte aligned", i);
    if (nt > 0 && text_pos0 + nt > c.max_pos) return fail(h, TTS_GPT_E_ARG, "prefill: text of stream %d runs past max_pos %d", i, c.max_pos);
    plen[i] = nc + nt;
    if (plen[i] > c.max_context) return fail(h, TTS_GPT_E_CTX_OVERFLOW, "prefill: prefix %d exceeds max_context %d", plen[i], c.max_context);
    if (pos0 && (pos0[i] < 0 || pos0[i] >= c.max_pos)) return fail(h, TTS_GPT_E_ARG, "prefill: pos0 out of range");
    pages += (plen[i] + 63) / 64;
  }
  PrefillParams pp;
  memset(&pp, 0, sizeof pp);
  pp.n = n;
  int found = 0;
  for (int s = 0; s < c.max_streams && found < n; ++s)
    if (!h->open[s]) pp.stream_ids[found++] = s;
  if (found < n) return fail(h, TTS_GPT_E_STREAM, "prefill: %d free stream slots, %d needed", found, n);
  if (pages > h->n_free) return fail(h, TTS_GPT_E_NO_PAGES, "prefill: %d pages needed, %d free", pages, h->n_free);
  for (int i = 0; i < n; ++i) {
    pp.prefix_len[i] = plen[i];
    pp.pos0[i] = pos0 ? pos0[i] : 0;
    pp.emb[i] = (const uint16_t *)emb[i];
  }
  prefill_open_kernel<<<1, kMaxRows, 0, h->stream>>>(pp, h->ps);
  CUDA_TRY(h, cudaGetLastError());
  h->launches += 1;
  if (text) {
    TextParams tp;
    memset(&tp, 0, sizeof tp);
    tp.n = n;
    for (int i = 0; i < n; ++i) { tp.stream_ids[i] = pp.stream_ids[i]; tp.n_cond[i] = n_cond[i]; tp.text[i] = text[i]; }
    prefill_text_kernel<<<1, kMaxRows, 0, h->stream>>>(tp, h->ps);
    CUDA_TRY(h, cudaGetLastError());
    h->launches += 1;
  }
  for (int i = 0; i < n; ++i) {
    const int s = pp.stream_ids[i];
    h->open[s] = 1; h->ctx[s] = plen[i]; h->pos_next[s] = pp.pos0[i];
    out_stream_ids[i] = s;
  }
  h->n_free -= pages;

  StepIO io;
  io.in_tokens = nullptr; io.uniforms = uniforms; io.out_tokens = out_tokens; io.out_logits = out_logits;
  io.out_hidden = (uint16_t *)out_hidden; io.top_k = top_k; io.temperature = temperature; io.n_out = 0;
  // rows in stream-major order; a pass takes up to `pass_rows` of them (several row tiles of 128 when the
  // tensor-core path is available, else one)
  const int pass_rows = (h->have_tc && h->use_tc) ? h->prefill_pass_rows : kMaxRows;
  PassParams ps;
  memset(&ps, 0, sizeof ps);
  ps.io = io;
  ps.text_shift = text_shift; ps.text_pos0 = text_pos0; ps.emb_rows = emb_rows_of(c);
  int scratch_pages = 0;   // 8-bit cache: pages the rows of the pass attend over
  auto flush = [&]() -> int {
    if (ps.n_rows == 0) return TTS_GPT_OK;
    ps.io.n_out = ps.n_out;
    ps.run_row0[ps.n_runs] = (short)ps.n_rows;
    if (scratch_pages > kScratchPages || !h->kv_fp8) scratch_pages = 0;   // too many pages: the pass attends over the codes
    ps.n_scratch = scratch_pages;
    ps.run_scratch0[ps.n_runs] = (short)scratch_pages;
    ps.scratch_table = h->scratch_table; ps.scratch_src = h->scratch_src; ps.scratch_ntok = h->scratch_ntok;
    h->pass_scratch = scratch_pages;
    prefill_pass_kernel<<<1, kMaxPassRows, 0, h->stream>>>(ps, h->ps, h->rt, h->io, c.d_model);
    CUDA_TRY(h, cudaGetLastError());
    h->launches += 1;
    int r = run_embed(h, ps.n_rows);
    if (r) return r;
    r = run_layers(h, ps.n_rows, false);
    if (r) return r;
    if (ps.n_out > 0) r = run_head(h, ps.n_out, ps.n_rows);
    ps.n_rows = 0; ps.n_out = 0; ps.n_runs = 0;
    scratch_pages = 0; h->pass_scratch = 0;
    return r;
  };
  for (int i = 0; i < n; ++i) {
    int t = 0;
    while (t < plen[i]) {
      const int take = std::min(plen[i] - t, pass_rows - ps.n_rows);
      ps.run_stream[ps.n_runs] = (short)pp.stream_ids[i];
      ps.run_pos0[ps.n_runs] = (short)t;
      ps.run_row0[ps.n_runs] = (short)ps.n_rows;
      ps.run_scratch0[ps.n_runs] = (short)std::min(scratch_pages, 32767);
      scratch_pages += (t + take - 1) / kPageTokens + 1;
      ++ps.n_runs;
      ps.n_rows += take;
      t += take;
      if (t == plen[i]) {
        ps.out_rows[ps.n_out] = (short)(ps.n_rows - 1);
        ps.out_slot[ps.n_out] = (short)i;
        ++ps.n_out;
      }
      if (ps.n_rows == pass_rows) { rc = flush(); if (rc) return rc; }
    }
  }
  return flush();
}

int32_t tts_gpt_prefill(tts_gpt_t *h, int32_t n, const void *const *prefix_emb, const int32_t *prefix_len,
                        const int32_t *pos0, int32_t top_k, float temperature, const float *uniforms,
                        int32_t *out_stream_ids, int32_t *out_tokens, float *out_logits, void *out_hidden) {
  return prefill_impl(h, n, prefix_emb, prefix_len, nullptr, nullptr, 0, 0, pos0, top_k, temperature, uniforms,
                      out_stream_ids, out_tokens, out_logits, out_hidden);
}

int32_t tts_gpt_prefill_tokens(tts_gpt_t *h, int32_t n, const void *const *cond_emb, const int32_t *n_cond,
                               const int32_t *const *text_ids, const int32_t *n_text, int32_t text_shift,
                               int32_t text_pos0, const int32_t *pos0, int32_t top_k, float temperature,
                               const float *uniforms, int32_t *out_stream_ids, int32_t *out_tokens,
                               float *out_logits, void *out_hidden) {
  if (!text_ids || !n_text) return fail(h, TTS_GPT_E_ARG, "prefill_tokens: null text argument");
  return prefill_impl(h, n, cond_emb, n_cond, text_ids, n_text, text_shift, text_pos0, pos0, top_k, temperature,
                      uniforms, out_stream_ids, out_tokens, out_logits, out_hidden);
}

int32_t tts_gpt_decode_step(tts_gpt_t *h, int32_t n, const int32_t *stream_ids, const int32_t *in_tokens,
                            int32_t top_k, float temperature, const float *uniforms, int32_t *out_tokens,
                            float *out_logits, void *out_hidden) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  const tts_gpt_config_t &c = h->cfg;
  if (n < 1 || n > c.max_streams || !stream_ids || !out_tokens) return fail(h, TTS_GPT_E_ARG, "decode_step: bad n or null argument");
  int rc = check_top_k(h, top_k, temperature, uniforms);
  if (rc) return rc;
  rc = check_io_alignment(h, in_tokens, uniforms, out_tokens, out_logits, out_hidden);
  if (rc) return rc;
  int pages = 0;
  char seen[kMaxRows];
  memset(seen, 0, sizeof seen);
  for (int i = 0; i < n; ++i) {
    const int s = stream_ids[i];
    if (s < 0 || s >= c.max_streams || !h->open[s]) return fail(h, TTS_GPT_E_STREAM, "decode_step: stream %d is not open", s);
    if (seen[s]) return fail(h, TTS_GPT_E_STREAM, "decode_step: stream %d listed twice", s);
    seen[s] = 1;
    if (h->ctx[s] + 1 > c.max_context) return fail(h, TTS_GPT_E_CTX_OVERFLOW, "decode_step: stream %d is at max_context %d", s, c.max_context);
    if (h->pos_next[s] >= c.max_pos) return fail(h, TTS_GPT_E_CTX_OVERFLOW, "decode_step: stream %d ran past max_pos %d", s, c.max_pos);
    if (h->ctx[s] % 64 == 0) ++pages;
  }
  if (pages > h->n_free) return fail(h, TTS_GPT_E_NO_PAGES, "decode_step: %d pages needed, %d free", pages, h->n_free);

  // The step's graph is captured (nothing runs during capture) before anything of the call is committed: a
  // failure to capture or instantiate leaves the engine exactly as it was.
  cudaGraphExec_t exec = nullptr;
  if (h->use_graph) {
    auto it = h->graphs.find(n);
    if (it == h->graphs.end()) {
      cudaGraph_t g = nullptr;
      const unsigned long long before = h->launches;
      CUDA_TRY(h, cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal));
      rc = run_embed(h, n);
      if (!rc) rc = run_layers(h, n, true);
      if (!rc) rc = run_head(h, n, n);
      cudaError_t e = cudaStreamEndCapture(h->stream, &g);
      const int nodes = (int)(h->launches - before);
      h->launches = before;  // captured, not run
      if (rc) { if (g) cudaGraphDestroy(g); return rc; }
      if (e != cudaSuccess) return fail(h, TTS_GPT_E_CUDA, "graph capture: %s", cudaGetErrorString(e));
      cudaGraphExec_t ge = nullptr;
      e = cudaGraphInstantiate(&ge, g, 0);
      cudaGraphDestroy(g);
      if (e != cudaSuccess) return fail(h, TTS_GPT_E_CUDA, "graph instantiate: %s", cudaGetErrorString(e));
      it = h->graphs.emplace(n, ge).first;
      h->graph_nodes[n] = nodes;
    }
    exec = it->second;
  }

  StepParams sp;
  sp.n = n;
  memcpy(sp.stream_ids, stream_ids, (size_t)n * sizeof(int));
  sp.io.in_tokens = in_tokens; sp.io.uniforms = uniforms; sp.io.out_tokens = out_tokens; sp.io.out_logits = out_logits;
  sp.io.out_hidden = (uint16_t *)out_hidden; sp.io.top_k = top_k; sp.io.temperature = temperature; sp.io.n_out = n;
  step_setup_kernel<<<1, kMaxRows, 0, h->stream>>>(sp, h->ps, h->rt, h->io);
  CUDA_TRY(h, cudaGetLastError());
  h->launches += 1;
  for (int i = 0; i < n; ++i) { h->ctx[stream_ids[i]] += 1; h->pos_next[stream_ids[i]] += 1; }
  h->n_free -= pages;

  if (exec) {
    CUDA_TRY(h, cudaGraphLaunch(exec, h->stream));
    h->launches += h->graph_nodes[n];
    return TTS_GPT_OK;
  }
  rc = run_embed(h, n);
  if (!rc) rc = run_layers(h, n, true);
  if (!rc) rc = run_head(h, n, n);
  return rc;
}

int32_t tts_gpt_decode_steps(tts_gpt_t *h, int32_t n, const int32_t *stream_ids, const int32_t *in_tokens,
                             int32_t n_steps, int32_t top_k, float temperature, const float *uniforms,
                             int32_t *out_tokens, float *out_logits, void *out_hidden) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  const tts_gpt_config_t &c = h->cfg;
  if (n_steps < 1) return fail(h, TTS_GPT_E_ARG, "decode_steps: n_steps must be positive");
  if (n < 1 || n > c.max_streams || !stream_ids || !out_tokens) return fail(h, TTS_GPT_E_ARG, "decode_steps: bad n or null argument");
  int rc = check_top_k(h, top_k, temperature, uniforms);
  if (rc) return rc;
  // the whole chunk is validated first, so that no step of it can be refused once the first is queued
  long long pages = 0;
  char seen[kMaxRows];
  memset(seen, 0, sizeof seen);
  for (int i = 0; i < n; ++i) {
    const int s = stream_ids[i];
    if (s < 0 || s >= c.max_streams || !h->open[s]) return fail(h, TTS_GPT_E_STREAM, "decode_steps: stream %d is not open", s);
    if (seen[s]) return fail(h, TTS_GPT_E_STREAM, "decode_steps: stream %d listed twice", s);
    seen[s] = 1;
    if ((long long)h->ctx[s] + n_steps > c.max_context)
      return fail(h, TTS_GPT_E_CTX_OVERFLOW, "decode_steps: stream %d has room for %d more tokens, %d asked", s, c.max_context - h->ctx[s], n_steps);
    if ((long long)h->pos_next[s] + n_steps > c.max_pos)
      return fail(h, TTS_GPT_E_CTX_OVERFLOW, "decode_steps: stream %d would run past max_pos %d", s, c.max_pos);
    pages += (h->ctx[s] + n_steps + 63) / 64 - (h->ctx[s] + 63) / 64;
  }
  if (pages > h->n_free) return fail(h, TTS_GPT_E_NO_PAGES, "decode_steps: %lld pages needed, %d free", pages, h->n_free);
  for (int k = 0; k < n_steps; ++k) {
    const size_t row0 = (size_t)k * n;
    rc = tts_gpt_decode_step(h, n, stream_ids, k == 0 ? in_tokens : nullptr, top_k, temperature,
                             uniforms ? uniforms + row0 : nullptr, out_tokens + row0,
                             out_logits ? out_logits + row0 * c.vocab : nullptr,
                             out_hidden ? (uint16_t *)out_hidden + row0 * c.d_model : nullptr);
    if (rc) return rc;   // only a CUDA failure can get here
  }
  return TTS_GPT_OK;
}

int32_t tts_gpt_release_stream(tts_gpt_t *h, int32_t s) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  if (s < 0 || s >= h->cfg.max_streams || !h->open[s]) return fail(h, TTS_GPT_E_STREAM, "release_stream: stream %d is not open", s);
  if (h->poison_free) {   // before the pages go back: the page table row still names them
    const int np = (h->ctx[s] + 63) / 64;
    if (np > 0)
      poison_pages_kernel<<<256, 256, 0, h->stream>>>(h->kv, h->kv_layer_elems, h->cfg.n_layer, h->kv_page_elems,
                                                      h->ps.page_table + (size_t)s * h->pps, nullptr, np);
  }
  release_kernel<<<1, 32, 0, h->stream>>>(h->ps, s);
  CUDA_TRY(h, cudaGetLastError());
  h->launches += 1;
  h->n_free += (h->ctx[s] + 63) / 64;
  h->open[s] = 0; h->ctx[s] = 0;
  return TTS_GPT_OK;
}

int32_t tts_gpt_decode_step_host(tts_gpt_t *h, int32_t n, const int32_t *stream_ids, const int32_t *in_tokens,
                                 int32_t top_k, float temperature, const float *uniforms, int32_t *out_tokens,
                                 float *out_logits, void *out_hidden) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  const tts_gpt_config_t &c = h->cfg;
  if (n < 1 || n > c.max_streams || !stream_ids || !out_tokens) return fail(h, TTS_GPT_E_ARG, "decode_step_host: bad n or null argument");
  if (top_k > 1 && !uniforms) return fail(h, TTS_GPT_E_ARG, "decode_step_host: top-k sampling needs uniforms");
  if (in_tokens) CUDA_TRY(h, cudaMemcpyAsync(h->st_in, in_tokens, (size_t)n * sizeof(int), cudaMemcpyHostToDevice, h->stream));
  if (top_k > 1) CUDA_TRY(h, cudaMemcpyAsync(h->st_uni, uniforms, (size_t)n * sizeof(float), cudaMemcpyHostToDevice, h->stream));
  const int rc = tts_gpt_decode_step(h, n, stream_ids, in_tokens ? h->st_in : nullptr, top_k, temperature,
                                     top_k > 1 ? h->st_uni : nullptr, h->st_tok, out_logits ? h->st_log : nullptr,
                                     out_hidden ? h->st_hid : nullptr);
  if (rc) return rc;
  CUDA_TRY(h, cudaMemcpyAsync(out_tokens, h->st_tok, (size_t)n * sizeof(int), cudaMemcpyDeviceToHost, h->stream));
  if (out_logits)
    CUDA_TRY(h, cudaMemcpyAsync(out_logits, h->st_log, (size_t)n * c.vocab * sizeof(float), cudaMemcpyDeviceToHost, h->stream));
  if (out_hidden)
    CUDA_TRY(h, cudaMemcpyAsync(out_hidden, h->st_hid, (size_t)n * c.d_model * sizeof(uint16_t), cudaMemcpyDeviceToHost, h->stream));
  return tts_gpt_sync(h);
}

int32_t tts_gpt_sync(tts_gpt_t *h) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  if (h->host_err && *h->host_err) {
    *h->host_err = 0;
    return fail(h, TTS_GPT_E_TIMEOUT, "a kernel's bounded wait for its weight copy expired; results of the last steps are invalid");
  }
  return TTS_GPT_OK;
}

int32_t tts_gpt_destroy(tts_gpt_t *h) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  cudaStreamSynchronize(h->stream);
  for (auto &kv : h->graphs) cudaGraphExecDestroy(kv.second);
  if (h->host_err) cudaFreeHost((void *)h->host_err);
  delete h;
  return TTS_GPT_OK;
}

const char *tts_gpt_last_error(const tts_gpt_t *h) { return h ? h->err.c_str() : g_last_error.c_str(); }

int32_t tts_gpt_stats(const tts_gpt_t *h, int32_t *open_streams, int32_t *free_pages) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  if (open_streams) { int n = 0; for (char o : h->open) n += o; *open_streams = n; }
  if (free_pages) *free_pages = h->n_free;
  return TTS_GPT_OK;
}

int32_t tts_gpt_debug_kernel_launches(const tts_gpt_t *h, uint64_t *n) {
  if (!h || !n) return fail(nullptr, TTS_GPT_E_ARG, "null argument");
  *n = h->launches;
  return TTS_GPT_OK;
}

int32_t tts_gpt_debug_set_trace(tts_gpt_t *h, void *trace, int32_t *n_slots) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  for (auto &kv : h->graphs) cudaGraphExecDestroy(kv.second);  // slots are baked into captured graphs
  h->graphs.clear();
  h->graph_nodes.clear();
  h->trace = (unsigned long long *)trace;
  if (n_slots) *n_slots = 7 * h->cfg.n_layer + 2;   // upper bound: the tensor-core path traces 7 kernels per layer
  return TTS_GPT_OK;
}

int32_t tts_gpt_stream_context(const tts_gpt_t *h, int32_t s) {
  if (!h || s < 0 || s >= h->cfg.max_streams || !h->open[s]) return -1;
  return h->ctx[s];
}

// waits on a barrier nothing completes, for at most limit_ns, then reports like any expired wait
__global__ void expire_wait_kernel(int *err, unsigned long long limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  mbar_init(&bar, 1);
  if (!mbar_wait_bounded(&bar, 0, limit_ns) && err) atomicExch(err, 1);
}

int32_t tts_gpt_debug_expire_wait(tts_gpt_t *h, uint32_t limit_us) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  if (limit_us < 1 || limit_us > 100000) return fail(h, TTS_GPT_E_ARG, "expire_wait: limit_us must be in 1..100000");
  expire_wait_kernel<<<1, 1, 0, h->stream>>>(h->dev_err, (unsigned long long)limit_us * 1000ull);
  CUDA_TRY(h, cudaGetLastError());
  return TTS_GPT_OK;
}

int32_t tts_gpt_debug_set_option(tts_gpt_t *h, const char *name, int32_t value) {
  if (!h || !name) return fail(nullptr, TTS_GPT_E_ARG, "null argument");
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  for (auto &kv : h->graphs) cudaGraphExecDestroy(kv.second);   // the choice is baked into captured step graphs
  h->graphs.clear();
  h->graph_nodes.clear();
  const std::string k(name);
  const bool on = value != 0;
  if (k == "graph") h->use_graph = on && h->stream != nullptr && h->stream != cudaStreamLegacy;
  else if (k == "pdl") h->use_pdl = on;
  else if (k == "tc") h->use_tc = on;
  else if (k == "prefill_pass_rows") { if (value < kMaxRows || value > kMaxPassRows || value % kMaxRows) return fail(h, TTS_GPT_E_ARG, "prefill_pass_rows must be a multiple of 128 from 128 to 1024"); h->prefill_pass_rows = value; }
  else if (k == "tc_min_rows") { if (value < 1 || value > kMaxRows) return fail(h, TTS_GPT_E_ARG, "tc_min_rows must be in 1..%d", kMaxRows); h->tc_min_rows = value; }
  else if (k == "attn_tc") h->use_attn_tc = on;
  else if (k == "w4_tc_exact") {
    if (h->cfg.wfmt != WF_INT4) return fail(h, TTS_GPT_E_ARG, "w4_tc_exact needs int4 weights");
    h->w4_exact = on;
    int rc = write_int4_images(h);   // the images change their meaning with the option
    if (rc) return rc;
    CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  }
  else if (k == "attn_mma") h->use_attn_mma = on;
  else if (k == "attn_prefill") h->use_attn_prefill = on;
  else if (k == "attn_stream") h->use_attn_stream = on;
  else if (k == "attn_stream_min_pairs") h->attn_stream_min_pairs = value > 0 ? value : 0;
  else if (k == "attn_cluster_fill") h->attn_cluster_fill = value > 0 ? value : 1;
  else if (k == "fc2_ksplit") h->use_fc2_ksplit = on;
  else if (k == "poison_free_pages") {
    h->poison_free = on;
    if (on && h->n_free > 0) {   // every page that is free right now
      poison_pages_kernel<<<1024, 256, 0, h->stream>>>(h->kv, h->kv_layer_elems, h->cfg.n_layer, h->kv_page_elems,
                                                       nullptr, h->ps.free_list, h->n_free);
      CUDA_TRY(h, cudaGetLastError());
    }
  }
  else return fail(h, TTS_GPT_E_ARG, "unknown option %s", name);
  return TTS_GPT_OK;
}

int32_t tts_gpt_debug_check_canaries(tts_gpt_t *h, int32_t *bad_bytes) {
  if (!h || !bad_bytes) return fail(nullptr, TTS_GPT_E_ARG, "null argument");
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  std::vector<unsigned char> buf(2 * kCanaryBytes);
  CUDA_TRY(h, cudaMemcpy(buf.data(), h->canary_lo, kCanaryBytes, cudaMemcpyDeviceToHost));
  CUDA_TRY(h, cudaMemcpy(buf.data() + kCanaryBytes, h->canary_hi, kCanaryBytes, cudaMemcpyDeviceToHost));
  int bad = 0;
  for (unsigned char b : buf) bad += b != kCanaryByte;
  *bad_bytes = bad;
  return TTS_GPT_OK;
}

int32_t tts_gpt_debug_shuffle_free_pages(tts_gpt_t *h, uint32_t seed) {
  if (!h) return fail(nullptr, TTS_GPT_E_ARG, "null handle");
  for (char o : h->open) if (o) return fail(h, TTS_GPT_E_STREAM, "shuffle: streams are open");
  std::vector<int> perm(h->cfg.n_pages);
  for (int i = 0; i < h->cfg.n_pages; ++i) perm[i] = i;
  uint64_t x = 0x9E3779B97F4A7C15ull ^ seed;
  for (int i = h->cfg.n_pages - 1; i > 0; --i) {
    x = x * 6364136223846793005ull + 1442695040888963407ull;
    const int j = (int)((x >> 33) % (uint64_t)(i + 1));
    std::swap(perm[i], perm[j]);
  }
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  CUDA_TRY(h, cudaMemcpy(h->ps.free_list, perm.data(), perm.size() * sizeof(int), cudaMemcpyHostToDevice));
  return TTS_GPT_OK;
}

// ---------------------------------------------------------------------------------------------
// single-kernel entry points
// ---------------------------------------------------------------------------------------------
int32_t tts_gpt_op_linear_packed_bytes(int32_t wfmt, int32_t N, int32_t K, size_t *bytes) {
  if (wfmt < 0 || wfmt > 2 || N < 1 || K < 128 || K % 128 || !bytes) return fail(nullptr, TTS_GPT_E_ARG, "op_linear: bad shape");
  *bytes = align256(packed_weight_bytes(wfmt, N, K)) + align256(packed_scale_bytes(wfmt, N, K));
  return TTS_GPT_OK;
}

int32_t tts_gpt_op_linear_pack(int32_t wfmt, int32_t N, int32_t K, const void *w, const void *s, void *packed,
                               void *cuda_stream) {
  size_t bytes;
  int rc = tts_gpt_op_linear_packed_bytes(wfmt, N, K, &bytes);
  if (rc) return rc;
  if (!w || !packed || (wfmt != WF_BF16 && !s) || (uintptr_t)packed % 256) return fail(nullptr, TTS_GPT_E_ARG, "op_linear_pack: null or misaligned");
  char *ps = (char *)packed + align256(packed_weight_bytes(wfmt, N, K));
  CUDA_TRY(nullptr, launch_pack(wfmt, N, K, w, s, packed, ps, (cudaStream_t)cuda_stream));
  return TTS_GPT_OK;
}

int32_t tts_gpt_op_linear(int32_t wfmt, int32_t N, int32_t K, const void *packed, const void *bias, int32_t B,
                          const void *act, float *out, void *cuda_stream) {
  size_t bytes;
  int rc = tts_gpt_op_linear_packed_bytes(wfmt, N, K, &bytes);
  if (rc) return rc;
  if (!packed || !act || !out || B < 1 || B > kMaxRows) return fail(nullptr, TTS_GPT_E_ARG, "op_linear: bad argument");
  if ((uintptr_t)packed % 256 || (uintptr_t)act % 16 || (uintptr_t)out % 16 || (uintptr_t)bias % 16)
    return fail(nullptr, TTS_GPT_E_ARG, "op_linear: packed must be 256-byte, act / out / bias 16-byte aligned");
  PackedLinear pl;
  pl.N = N; pl.K = K; pl.w = (void *)packed;
  pl.s = (uint16_t *)((char *)packed + align256(packed_weight_bytes(wfmt, N, K)));
  pl.bias = (uint16_t *)bias;
  LinearArgs a = linear_args(pl, (const uint16_t *)act, B, EPI_F32);
  a.out_f32 = out; a.out_stride = N;
  CUDA_TRY(nullptr, launch_linear(wfmt, a, (cudaStream_t)cuda_stream, false));
  return TTS_GPT_OK;
}

int32_t tts_gpt_op_linear_tc_scratch_bytes(int32_t N, int32_t K, size_t *bytes) {
  if (N < 1 || K < 64 || K % 64 || !bytes) return fail(nullptr, TTS_GPT_E_ARG, "op_linear_tc: bad shape");
  *bytes = align256(weight_image_bytes(N, K)) + align256(act_image_bytes(K)) +
           align256((size_t)kTcKSplit * kMaxRows * N * sizeof(float)) + align256(packed_scale_bytes(WF_INT4, N, K) + 256);
  return TTS_GPT_OK;
}

int32_t tts_gpt_op_linear_tc(int32_t wfmt, int32_t N, int32_t K, const void *w, const void *s, const void *bias,
                             int32_t B, const void *act, float *out, int32_t ksplit, void *scratch, void *cuda_stream) {
  size_t bytes;
  int rc = tts_gpt_op_linear_tc_scratch_bytes(N, K, &bytes);
  if (rc) return rc;
  const bool wide = ksplit < 0;   // the kernel of the multi-tile prefill passes, here on one row tile
  if (wide) ksplit = -ksplit;
  if (wfmt < 0 || wfmt > 2 || !w || !act || !out || !scratch || B < 1 || B > kMaxRows || (uintptr_t)scratch % 1024 ||
      (!wide && ksplit != 1 && ksplit != kTcKSplit) || ksplit < 1 || ksplit > kTwMaxPartials || K / 64 < ksplit || K % 128 ||
      (wfmt != WF_BF16 && !s) ||
      (uintptr_t)w % 16 || (uintptr_t)s % 16 || (uintptr_t)act % 16 || (uintptr_t)out % 16 || (uintptr_t)bias % 16)
    return fail(nullptr, TTS_GPT_E_ARG, "op_linear_tc: bad or misaligned argument");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char *wimg = (char *)scratch;
  char *aimg = wimg + align256(weight_image_bytes(N, K));
  float *part = (float *)(aimg + align256(act_image_bytes(K)));
  uint16_t *tiled_s = (uint16_t *)(part + (size_t)kTcKSplit * kMaxRows * N);
  CUDA_TRY(nullptr, launch_pack_image(wfmt, N, K, w, wimg, st));
  if (wfmt != WF_BF16) {
    const int G = wfmt == WF_INT8 ? 1 : K / 128;
    const size_t n = (size_t)row_tiles(N) * G * 8;
    pack_scales_kernel<<<(int)((n + 255) / 256), 256, 0, st>>>((const uint16_t *)s, N, G, tiled_s);
  }
  const size_t au = (size_t)B * (K / 8);
  pack_act_image_kernel<<<(unsigned)((au + 255) / 256), 256, 0, st>>>((const uint16_t *)act, B, K, (unsigned char *)aimg);
  CUDA_TRY(nullptr, cudaGetLastError());
  GemmTcArgs a;
  memset(&a, 0, sizeof a);
  a.w_img = wimg; a.act_img = aimg; a.N = N; a.K = K; a.B = B; a.ksplit = ksplit; a.wfmt = wfmt; a.scales = tiled_s;
  if (ksplit == 1) {
    a.mode = EPI_F32; a.bias = (const uint16_t *)bias; a.out_f32 = out; a.out_stride = N;
    CUDA_TRY(nullptr, wide ? launch_gemm_tcw(a, 148, st, false) : launch_gemm_tc(a, st, false));
  } else {   // partial sums per k-range, then folded in range order (what the following LayerNorm does in the engine)
    a.mode = EPI_RESID; a.out_f32 = part; a.out_stride = N;
    CUDA_TRY(nullptr, wide ? launch_gemm_tcw(a, 148, st, false) : launch_gemm_tc(a, st, false));
    fold_partials_kernel<<<(unsigned)(((size_t)B * N + 255) / 256), 256, 0, st>>>(part, ksplit, B, N, (const uint16_t *)bias, out);
    CUDA_TRY(nullptr, cudaGetLastError());
  }
  return TTS_GPT_OK;
}

int32_t tts_gpt_op_attention_scratch_bytes(int32_t R, int32_t n_head, size_t *bytes) {
  if (R < 1 || n_head < 1 || !bytes) return fail(nullptr, TTS_GPT_E_ARG, "op_attention: bad shape");
  *bytes = attention_scratch_bytes(R, n_head);
  return TTS_GPT_OK;
}

int32_t tts_gpt_op_attention(int32_t R, int32_t n_head, const float *q, const void *kv_layer,
                             const int32_t *page_table, int32_t pages_per_stream, const int32_t *row_stream,
                             const int32_t *row_pos, void *out, void *scratch, void *cuda_stream) {
  if ((uintptr_t)q % 16 || (uintptr_t)kv_layer % 16 || (uintptr_t)out % 2 || (uintptr_t)page_table % 4 || (uintptr_t)row_stream % 4 ||
      (uintptr_t)row_pos % 4)
    return fail(nullptr, TTS_GPT_E_ARG, "attention: q and the KV pool must be 16-byte aligned, index arrays 4-byte");
  if (R < 1 || R > 65535 || n_head < 1 || !q || !kv_layer || !page_table || !row_stream || !row_pos || !out || !scratch ||
      pages_per_stream < 1 || pages_per_stream > kAttnMaxChunks * kAttnWarps || (uintptr_t)scratch % 256)
    return fail(nullptr, TTS_GPT_E_ARG, "op_attention: bad argument");
  AttnArgs a;
  a.q = q; a.kv_layer = (const uint16_t *)kv_layer; a.page_table = page_table; a.row_stream = row_stream;
  a.row_pos = row_pos; a.out = (uint16_t *)out; a.H = n_head; a.pps = pages_per_stream; a.old_pages_final = 0;
  a.trace = nullptr; a.trace_slot = 0;
  a.partials = (float *)scratch;
  a.tickets = (unsigned int *)((char *)scratch + align256((size_t)R * n_head * kAttnMaxChunks * kAttnPartialFloats * sizeof(float)));
  CUDA_TRY(nullptr, launch_attention_ticket(a, R, pages_per_stream * kPageTokens, (cudaStream_t)cuda_stream));
  return TTS_GPT_OK;
}

// ---------------------------------------------------------------------------------------------
// Attention without caller-provided scratch: the split-KV partials and tickets live in a fixed
// array inside the library image.
// ---------------------------------------------------------------------------------------------
}  // extern "C"

namespace {
constexpr int kStaticAttnMaxRowHeads = TTS_GPT_STATIC_ATTN_MAX_ROW_HEADS;
constexpr size_t kStaticAttnPartialBytes =
    (size_t)kStaticAttnMaxRowHeads * kAttnMaxChunks * kAttnPartialFloats * sizeof(float);
constexpr size_t kStaticAttnBytes = kStaticAttnPartialBytes + (size_t)kStaticAttnMaxRowHeads * sizeof(unsigned int);
static_assert(kStaticAttnPartialBytes % 256 == 0, "tickets must start 256-byte aligned");
// Lives in every GPU that loads the library, from load until process exit (about 2.7 MB).
static __device__ __align__(256) unsigned char g_static_attn_scratch[kStaticAttnBytes];
// The symbol above is only a host-side stand-in when named in host code: its device address has to
// be asked for, once per device, with that device current.
constexpr int kMaxDevices = 64;
std::atomic<void *> g_static_attn_ptr[kMaxDevices];   // zero-initialised; first calls from several host threads may race
                                                       // harmlessly (they store the same address)
}  // namespace

extern "C" {

int32_t tts_gpt_op_attention_static(int32_t R, int32_t n_head, const float *q, const void *kv_layer,
                                    const int32_t *page_table, int32_t pages_per_stream,
                                    const int32_t *row_stream, const int32_t *row_pos, void *out,
                                    void *cuda_stream) {
  if ((uintptr_t)q % 16 || (uintptr_t)kv_layer % 16 || (uintptr_t)out % 2 || (uintptr_t)page_table % 4 || (uintptr_t)row_stream % 4 ||
      (uintptr_t)row_pos % 4)
    return fail(nullptr, TTS_GPT_E_ARG, "attention: q and the KV pool must be 16-byte aligned, index arrays 4-byte");
  if (R < 1 || R > 65535 || n_head < 1 || !q || !kv_layer || !page_table || !row_stream || !row_pos || !out ||
      pages_per_stream < 1 || pages_per_stream > kAttnMaxChunks * kAttnWarps)
    return fail(nullptr, TTS_GPT_E_ARG, "op_attention_static: bad argument");
  if ((long long)R * n_head > kStaticAttnMaxRowHeads)
    return fail(nullptr, TTS_GPT_E_WORKSPACE,
                "op_attention_static: R*n_head = %lld exceeds the built-in scratch limit of %d row-heads; "
                "use tts_gpt_op_attention with caller scratch",
                (long long)R * n_head, kStaticAttnMaxRowHeads);
  int dev = -1;
  CUDA_TRY(nullptr, cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(nullptr, TTS_GPT_E_UNSUPPORTED, "op_attention_static: device index %d", dev);
  void *resolved = g_static_attn_ptr[dev].load(std::memory_order_relaxed);
  if (!resolved) {  // first call on this device: resolve the array's device address
    CUDA_TRY(nullptr, cudaGetSymbolAddress(&resolved, g_static_attn_scratch));
    if (!resolved) return fail(nullptr, TTS_GPT_E_CUDA, "op_attention_static: no device address for the scratch array");
    g_static_attn_ptr[dev].store(resolved, std::memory_order_relaxed);
  }
  unsigned char *base = (unsigned char *)resolved;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  AttnArgs a;
  a.q = q; a.kv_layer = (const uint16_t *)kv_layer; a.page_table = page_table; a.row_stream = row_stream;
  a.row_pos = row_pos; a.out = (uint16_t *)out; a.H = n_head; a.pps = pages_per_stream; a.old_pages_final = 0;
  a.trace = nullptr; a.trace_slot = 0;
  a.partials = (float *)base;
  a.tickets = (unsigned int *)(base + kStaticAttnPartialBytes);
  // The array keeps whatever the previous call left; the tickets have to start at zero.
  CUDA_TRY(nullptr, cudaMemsetAsync(a.tickets, 0, (size_t)R * n_head * sizeof(unsigned int), st));
  CUDA_TRY(nullptr, launch_attention_ticket(a, R, pages_per_stream * kPageTokens, st));
  return TTS_GPT_OK;
}

int32_t tts_gpt_op_attention_cluster(int32_t R, int32_t n_head, const float *q, const void *kv_layer,
                                     const int32_t *page_table, int32_t pages_per_stream,
                                     const int32_t *row_stream, const int32_t *row_pos, void *out,
                                     int32_t cluster_size, void *cuda_stream) {
  if ((uintptr_t)q % 16 || (uintptr_t)kv_layer % 16 || (uintptr_t)out % 16 || (uintptr_t)page_table % 4 || (uintptr_t)row_stream % 4 ||
      (uintptr_t)row_pos % 4)
    return fail(nullptr, TTS_GPT_E_ARG, "attention: q, out and the KV pool must be 16-byte aligned, index arrays 4-byte");
  if (R < 1 || R > 65535 || n_head < 1 || !q || !kv_layer || !page_table || !row_stream || !row_pos || !out ||
      pages_per_stream < 1)
    return fail(nullptr, TTS_GPT_E_ARG, "op_attention_cluster: bad argument");
  if (cluster_size != -3 && cluster_size != -2 && cluster_size != -1 && cluster_size != 0 && cluster_size != 1 && cluster_size != 2 &&
      cluster_size != 4 && cluster_size != 8)
    return fail(nullptr, TTS_GPT_E_ARG, "op_attention_cluster: cluster_size must be -3, -2, -1, 0, 1, 2, 4 or 8");
  AttnArgs a;
  memset(&a, 0, sizeof a);
  a.q = q; a.kv_layer = (const uint16_t *)kv_layer; a.page_table = page_table; a.row_stream = row_stream;
  a.row_pos = row_pos; a.out = (uint16_t *)out; a.H = n_head; a.pps = pages_per_stream;
  if (cluster_size == 0) {
    CUDA_TRY(nullptr, launch_attention_stream(a, R, (cudaStream_t)cuda_stream, false));
    return TTS_GPT_OK;
  }
  if (cluster_size == -3) {   // rows must be stream-major with ascending positions, as in a prefill pass
    CUDA_TRY(nullptr, launch_attention_prefill_tc(a, R, (cudaStream_t)cuda_stream, false));
    return TTS_GPT_OK;
  }
  if (cluster_size == -2) {   // same requirement on the rows
    CUDA_TRY(nullptr, launch_attention_prefill_mma(a, R, (cudaStream_t)cuda_stream, false));
    return TTS_GPT_OK;
  }
  if (cluster_size == -1) {   // same requirement on the rows
    CUDA_TRY(nullptr, launch_attention_prefill(a, R, (cudaStream_t)cuda_stream, false));
    return TTS_GPT_OK;
  }
  CUDA_TRY(nullptr, launch_attention(a, R, cluster_size, (cudaStream_t)cuda_stream, false));
  return TTS_GPT_OK;
}

int32_t tts_gpt_op_layernorm(int32_t R, int32_t d, const float *x, const void *g, const void *b, float eps,
                             void *out, void *cuda_stream) {
  if (R < 1 || d < 1 || d > kLnThreads * kLnMaxPerThread || !x || !g || !b || !out || (uintptr_t)x % 4 || (uintptr_t)g % 2 ||
      (uintptr_t)b % 2 || (uintptr_t)out % 2)
    return fail(nullptr, TTS_GPT_E_ARG, "op_layernorm: bad or misaligned argument");
  layernorm_kernel<<<R, kLnThreads, 0, (cudaStream_t)cuda_stream>>>(x, d, (const uint16_t *)g, (const uint16_t *)b, eps,
                                                                    (uint16_t *)out, nullptr, nullptr, nullptr);
  CUDA_TRY(nullptr, cudaGetLastError());
  return TTS_GPT_OK;
}

int32_t tts_gpt_op_sample(int32_t R, int32_t V, const float *logits, int32_t top_k, float temperature,
                          const float *uniforms, int32_t *tokens, void *cuda_stream) {
  if (R < 1 || V < 2 || V > kSampleThreads * kSampleMaxPer || !logits || !tokens || top_k < 0 || top_k > kMaxTopK ||
      (top_k > 1 && (!uniforms || !(temperature > 0.f))))
    return fail(nullptr, TTS_GPT_E_ARG, "op_sample: bad argument");
  SampleArgs sa;
  memset(&sa, 0, sizeof sa);
  sa.logits = logits; sa.V = V; sa.top_k = top_k; sa.temperature = temperature; sa.uniforms = uniforms; sa.out_tokens = tokens;
  sample_kernel<<<R, kSampleThreads, (size_t)V * sizeof(float), (cudaStream_t)cuda_stream>>>(sa);
  CUDA_TRY(nullptr, cudaGetLastError());
  return TTS_GPT_OK;
}

}  // extern "C"
