// KV page allocator and per-call set-up kernels (Section I: KV-cache management of the decode
// engine).  The allocator state lives in device memory: a stack of free page ids, one page table
// row and one context length per stream.  Set-up kernels receive the call's small host arrays BY
// VALUE as kernel parameters, so no host staging buffer has to outlive the call and no step waits
// for the host.  The host keeps only counters (free pages, context lengths), which evolve
// deterministically, to reject calls that cannot succeed before anything is enqueued.
#pragma once
#include "common.cuh"
#include "elementwise.cuh"

namespace ttsgpt {

struct PageState {
  int *ctx_len;     // [max_streams]
  int *page_table;  // [max_streams][pps]
  int *free_list;   // [n_pages] stack; free_top entries valid
  int *free_top;    // [1]
  int *last_token;  // [max_streams]
  int *pos_next;    // [max_streams] pos_emb index of the next generated token
  int *stop_flag;   // [max_streams]
  const uint16_t **stream_emb;  // [max_streams] prefix base pointer during prefill
  const int **stream_text;      // [max_streams] text ids behind the given rows (null: none)
  int *stream_ncond;            // [max_streams] rows of the prefix that are given embeddings
  int pps, n_pages, max_streams;
};

__global__ void init_pages_kernel(PageState ps) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < ps.n_pages) ps.free_list[i] = ps.n_pages - 1 - i;  // page 0 is popped first
  if (i < ps.max_streams) { ps.ctx_len[i] = 0; ps.last_token[i] = 0; ps.pos_next[i] = 0; ps.stop_flag[i] = 0; }
  if (i < ps.max_streams * ps.pps) ps.page_table[i] = 0;
  if (i == 0) *ps.free_top = ps.n_pages;
}

// exclusive prefix sum of one int per thread over a block of kMaxRows threads
__device__ __forceinline__ int block_exclusive_scan_128(int v, int *total) {
  __shared__ int warp_tot[kMaxRows / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int base = 0, tot = 0;
  for (int w = 0; w < kMaxRows / 32; ++w) { if (w < warp) base += warp_tot[w]; tot += warp_tot[w]; }
  *total = tot;
  return base + incl - v;
}

struct StepParams {
  int n;
  int stream_ids[kMaxRows];
  StepIO io;
};

// One decode step: each stream whose context length sits on a page boundary pops a page (streams
// in call order take pages in stack order), then the row table is written and ctx_len advances.
__global__ void __launch_bounds__(kMaxRows) step_setup_kernel(const StepParams p, PageState ps, RowTable rt, StepIO *io) {
  const int i = threadIdx.x;
  int s = 0, t = 0, need = 0;
  if (i < p.n) { s = p.stream_ids[i]; t = ps.ctx_len[s]; need = (t % kPageTokens) == 0; }
  int total;
  const int rank = block_exclusive_scan_128(need, &total);
  const int top = *ps.free_top;
  if (i < p.n) {
    if (need) ps.page_table[(size_t)s * ps.pps + t / kPageTokens] = ps.free_list[top - 1 - rank];
    rt.row_stream[i] = s;
    rt.row_pos[i] = t;
    rt.row_token[i] = p.io.in_tokens ? max(p.io.in_tokens[i], 0) : ps.last_token[s];
    rt.row_posidx[i] = ps.pos_next[s];
    rt.out_rows[i] = i;
    rt.out_slot[i] = i;
    ps.ctx_len[s] = t + 1;
    ps.pos_next[s] += 1;
  }
  // attention works through the rows longest first, so that the short ones fill the tail of its grid
  __shared__ int len_s[kMaxRows];
  len_s[i] = i < p.n ? t : -1;
  __syncthreads();
  if (i < p.n) {
    int before = 0;
    for (int j = 0; j < p.n; ++j) before += (len_s[j] > t || (len_s[j] == t && j < i)) ? 1 : 0;
    rt.row_order[before] = i;
  }
  if (i == 0) { *ps.free_top = top - total; *io = p.io; }
}

struct PrefillParams {
  int n;
  int stream_ids[kMaxRows];
  int prefix_len[kMaxRows];
  int pos0[kMaxRows];
  const uint16_t *emb[kMaxRows];
};

// Opens the streams of a prefill call: reserves ceil(P/64) pages each, sets ctx_len = P.
__global__ void __launch_bounds__(kMaxRows) prefill_open_kernel(const PrefillParams p, PageState ps) {
  const int i = threadIdx.x;
  int need = 0;
  if (i < p.n) need = (p.prefix_len[i] + kPageTokens - 1) / kPageTokens;
  int total;
  const int base = block_exclusive_scan_128(need, &total);
  const int top = *ps.free_top;
  if (i < p.n) {
    const int s = p.stream_ids[i];
    for (int j = 0; j < need; ++j) ps.page_table[(size_t)s * ps.pps + j] = ps.free_list[top - 1 - (base + j)];
    ps.ctx_len[s] = p.prefix_len[i];
    ps.pos_next[s] = p.pos0[i];
    ps.stop_flag[s] = 0;
    ps.stream_emb[s] = p.emb[i];
    ps.stream_text[s] = nullptr;            // the whole prefix is given as embeddings unless
    ps.stream_ncond[s] = p.prefix_len[i];   // prefill_text_kernel says otherwise
  }
  __syncthreads();
  if (i == 0) *ps.free_top = top - total;
}

// Prefixes assembled on the device (Section II-C): the first n_cond rows of a stream's prefix are the
// given conditioning embeddings, the rest are text tokens looked up in the merged embedding table.
struct TextParams {
  int n;
  int stream_ids[kMaxRows];
  int n_cond[kMaxRows];
  const int *text[kMaxRows];
};

__global__ void __launch_bounds__(kMaxRows) prefill_text_kernel(const TextParams p, PageState ps) {
  const int i = threadIdx.x;
  if (i < p.n) {
    const int s = p.stream_ids[i];
    ps.stream_text[s] = p.text[i];
    ps.stream_ncond[s] = p.n_cond[i];
  }
}

// A prefill pass: rows in stream-major order, given as runs of consecutive positions of one stream.
struct PassParams {
  int n_rows, n_out, n_runs;
  short run_stream[kMaxRows], run_pos0[kMaxRows], run_row0[kMaxRows + 1];   // run j covers rows run_row0[j] .. run_row0[j+1]-1
  short out_rows[kMaxRows], out_slot[kMaxRows];
  StepIO io;
  int text_shift, text_pos0, emb_rows;   // text rows: table row = id + text_shift (clamped), position row = text_pos0 + j
  // 8-bit cache: the pages the pass's rows attend over, decoded into scratch pages; run j owns the scratch pages
  // run_scratch0[j] .. run_scratch0[j+1]-1 = pages 0.. of its stream (n_scratch = 0: not used)
  int n_scratch;
  short run_scratch0[kMaxRows + 1];
  int *scratch_table, *scratch_src, *scratch_ntok;   // [max_streams][pps], [n_scratch], [n_scratch]
};

// Row table of one prefill pass: up to kMaxPassRows (stream, position) rows taken from the prefixes.
__global__ void __launch_bounds__(kMaxPassRows) prefill_pass_kernel(const PassParams p, PageState ps, RowTable rt, StepIO *io, int d) {
  const int i = threadIdx.x;
  if (i < p.n_rows) {
    int j = 0;
    while (j + 1 < p.n_runs && p.run_row0[j + 1] <= i) ++j;
    const int s = p.run_stream[j], t = p.run_pos0[j] + (i - p.run_row0[j]);
    rt.row_stream[i] = s;
    rt.row_pos[i] = t;
    const int nc = ps.stream_ncond[s];
    if (t < nc) {     // a given embedding row, used as it is
      rt.row_token[i] = -1;
      rt.row_posidx[i] = 0;
      rt.row_emb[i] = ps.stream_emb[s] + (size_t)t * d;
    } else {          // text token j of the stream
      const int jt = t - nc;
      rt.row_token[i] = min(max(ps.stream_text[s][jt] + p.text_shift, 0), p.emb_rows - 1);
      rt.row_posidx[i] = p.text_pos0 + jt;
      rt.row_emb[i] = nullptr;
    }
  }
  if (i < p.n_out) { rt.out_rows[i] = p.out_rows[i]; rt.out_slot[i] = p.out_slot[i]; }
  if (i == 0) *io = p.io;
  if (i < p.n_scratch) {
    int j = 0;
    while (j + 1 < p.n_runs && p.run_scratch0[j + 1] <= i) ++j;
    const int s = p.run_stream[j], pg = i - p.run_scratch0[j];
    const int last_pos = p.run_pos0[j] + (p.run_row0[j + 1] - p.run_row0[j]) - 1;   // last position the run's rows reach
    p.scratch_table[(size_t)s * ps.pps + pg] = i;
    p.scratch_src[i] = ps.page_table[(size_t)s * ps.pps + pg];
    p.scratch_ntok[i] = min(kPageTokens, last_pos + 1 - pg * kPageTokens);
  }
}

// Debug aid: fills the K and V blocks of the given pages, in every layer, with bf16 NaN.  A kernel that reads
// a slot no token was written to (a stale page, a slot beyond the context) then poisons its result.
// pages == nullptr: the n pages on top of the free stack (all free pages when n = *free_top).
__global__ void poison_pages_kernel(uint16_t *kv, size_t kv_layer_elems, int n_layer, size_t page_elems,
                                    const int *pages, const int *free_list, int n) {
  const size_t per_page = page_elems / 8;   // 16-byte units of one page in one layer
  const size_t total = (size_t)n * n_layer * per_page;
  const uint4 nan4 = make_uint4(0x7FC07FC0u, 0x7FC07FC0u, 0x7FC07FC0u, 0x7FC07FC0u);
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t u = i % per_page;
    const size_t t = i / per_page;
    const int l = (int)(t % n_layer), j = (int)(t / n_layer);
    const int page = pages ? pages[j] : free_list[j];
    reinterpret_cast<uint4 *>(kv + kv_layer_elems * l + (size_t)page * page_elems)[u] = nan4;
  }
}

// Returns a stream's pages to the stack (last page first, so that the next stream to open pops
// them in the order this one received them).
__global__ void release_kernel(PageState ps, int s) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const int n = (ps.ctx_len[s] + kPageTokens - 1) / kPageTokens;
  int top = *ps.free_top;
  for (int j = n - 1; j >= 0; --j) ps.free_list[top++] = ps.page_table[(size_t)s * ps.pps + j];
  *ps.free_top = top;
  ps.ctx_len[s] = 0;
}

}  // namespace ttsgpt
