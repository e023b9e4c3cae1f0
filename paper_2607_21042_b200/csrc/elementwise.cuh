// Embedding lookup, LayerNorm and sampling kernels, plus the per-step I/O block they read.
#pragma once
#include "common.cuh"

namespace ttsgpt {

// Per-call I/O pointers and sampling settings, kept in device memory so that a captured CUDA graph
// of the step can be replayed while the caller changes buffers from step to step.
struct StepIO {
  const int *in_tokens;
  const float *uniforms;
  int *out_tokens;
  float *out_logits;
  uint16_t *out_hidden;
  int top_k;
  float temperature;
  int n_out;
};

// Per-pass row table (device arrays of kMaxRows entries).  A row is one (stream, position) pair.
struct RowTable {
  int *row_stream;            // stream slot of the row
  int *row_pos;               // position in the stream's context the row occupies (its K/V slot)
  int *row_token;             // >= 0: token id to embed; -1: take row_emb
  int *row_posidx;            // index into pos_emb for token rows
  const uint16_t **row_emb;   // bf16 [d] embedding of a prefix row
  int *out_rows;              // rows whose logits are wanted, compacted
  int *out_slot;              // position of that row's results in the caller's output arrays
  int *row_order;             // decode steps: rows by descending context length (longest first)
};

// x[r,:] = tok_emb[token] + pos_emb[posidx]   (generated tokens take a positional embedding from
// their own range of the position table; prefix embeddings are used as given: Section II-C)
__global__ void embed_kernel(RowTable rt, const uint16_t *__restrict__ tok_emb, const uint16_t *__restrict__ pos_emb,
                             int d, int vocab, int max_pos, float *__restrict__ x) {
  const int r = blockIdx.x;
  int tok = rt.row_token[r];
  float *xr = x + (size_t)r * d;
  if (tok >= 0) {
    tok = min(tok, vocab - 1);
    const int p = min(max(rt.row_posidx[r], 0), max_pos - 1);
    const uint16_t *te = tok_emb + (size_t)tok * d, *pe = pos_emb + (size_t)p * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) xr[i] = bf16_bits_to_float(te[i]) + bf16_bits_to_float(pe[i]);
  } else {
    const uint16_t *e = rt.row_emb[r];
    for (int i = threadIdx.x; i < d; i += blockDim.x) xr[i] = bf16_bits_to_float(e[i]);
  }
}

__device__ __forceinline__ float block_sum(float v, float *sm) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sm[warp] = v;
  __syncthreads();
  float t = 0.f;
  for (int w = 0; w < nw; ++w) t += sm[w];
  return t;
}

// LayerNorm of fp32 rows (biased variance, eps inside the square root), bf16 out.  With `gather`
// row j of the output is row gather[j] of x; `io` (optional) also receives the rows at out_slot.
constexpr int kLnThreads = 256;
constexpr int kLnMaxPerThread = 8;  // d <= 2048
__global__ void __launch_bounds__(kLnThreads) layernorm_kernel(const float *__restrict__ x, int d,
                                                               const uint16_t *__restrict__ g,
                                                               const uint16_t *__restrict__ b, float eps,
                                                               uint16_t *__restrict__ out, const int *gather,
                                                               const int *out_slot, const StepIO *io) {
  __shared__ float sm[kLnThreads / 32];
  // gamma and beta do not depend on the kernel in front: fetched ahead of the dependency wait
  float gg[kLnMaxPerThread], bb[kLnMaxPerThread];
#pragma unroll
  for (int i = 0; i < kLnMaxPerThread; ++i) {
    const int c = threadIdx.x + i * kLnThreads;
    gg[i] = c < d ? bf16_bits_to_float(g[c]) : 0.f;
    bb[i] = c < d ? bf16_bits_to_float(b[c]) : 0.f;
  }
  pdl_launch_dependents();
  pdl_wait();
  const int j = blockIdx.x;
  const int r = gather ? gather[j] : j;
  const float *xr = x + (size_t)r * d;
  float v[kLnMaxPerThread];
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < kLnMaxPerThread; ++i) {
    const int c = threadIdx.x + i * kLnThreads;
    v[i] = c < d ? xr[c] : 0.f;
    s += v[i];
  }
  const float mu = block_sum(s, sm) / d;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < kLnMaxPerThread; ++i) {
    const int c = threadIdx.x + i * kLnThreads;
    const float t = c < d ? v[i] - mu : 0.f;
    q += t * t;
  }
  const float rstd = rsqrtf(block_sum(q, sm) / d + eps);
  uint16_t *hid = (io && io->out_hidden) ? io->out_hidden + (size_t)(out_slot ? out_slot[j] : j) * d : nullptr;
#pragma unroll
  for (int i = 0; i < kLnMaxPerThread; ++i) {
    const int c = threadIdx.x + i * kLnThreads;
    if (c < d) {
      const uint16_t y = float_to_bf16_bits((v[i] - mu) * rstd * gg[i] + bb[i]);
      out[(size_t)j * d + c] = y;
      if (hid) hid[c] = y;
    }
  }
}

// byte offset of element (row, k) inside an activation image: blocks of 128 rows x 64 columns
// (16 KB each, one per k-chunk), row r at byte r*128, its 16-byte unit u stored at unit u ^ (r % 8)
__host__ __device__ inline size_t act_image_offset(int row, int k) {
  const int kc = k >> 6, u = (k & 63) >> 3;
  return (size_t)kc * (kMaxRows * 128) + (size_t)row * 128 + (size_t)((u ^ (row & 7)) << 4) + (size_t)(k & 7) * 2;
}

// the same for passes of more than 128 rows: row tiles of 128 rows, each a complete image of a K-column matrix
__host__ __device__ inline size_t act_image_offset_tiled(int row, int k, int K) {
  return (size_t)(row >> 7) * (size_t)(K >> 6) * (kMaxRows * 128) + act_image_offset(row & (kMaxRows - 1), k);
}

// LayerNorm in front of a tensor-core linear.  First folds what the previous k-split linear left
// behind into the residual stream, in a fixed order: x[r] += bias + partial[0][r] + partial[1][r] + ...
// (written back unless `write_back` is 0), then normalises and writes the row into the activation
// image (`out_img`) and/or a plain bf16 row (`out_plain`, row j).  With `gather`, row j is x row gather[j].
struct LnTcArgs {
  float *x; int d;
  const float *partials; int n_part, part_cols;   // [row tile][n_part][kMaxRows][part_cols]
  const uint16_t *add_bias;
  const uint16_t *g, *b; float eps;
  void *out_img; uint16_t *out_plain;
  const int *gather, *out_slot; const StepIO *io;
  int write_back;
  unsigned long long *trace;  // optional timeline trace
  int trace_slot;
};
// NP: elements per thread (d <= 256 * NP); the engine instantiates what its d needs.
template <int NP>
__global__ void __launch_bounds__(kLnThreads) layernorm_tc_kernel(const LnTcArgs a) {
  __shared__ float sm[kLnThreads / 32];
  trace_mark(a.trace, a.trace_slot, 0);
  // gamma, beta and the folded bias do not depend on the kernel in front: fetched ahead of the dependency wait
  float gg[NP], bb[NP], bs[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int c = threadIdx.x + i * kLnThreads;
    gg[i] = c < a.d ? bf16_bits_to_float(a.g[c]) : 0.f;
    bb[i] = c < a.d ? bf16_bits_to_float(a.b[c]) : 0.f;
    bs[i] = (c < a.d && a.n_part > 0 && a.add_bias) ? bf16_bits_to_float(a.add_bias[c]) : 0.f;
  }
  pdl_launch_dependents();
  pdl_wait();
  trace_mark(a.trace, a.trace_slot, 1);
  const int j = blockIdx.x;
  const int r = a.gather ? a.gather[j] : j;
  float *xr = a.x + (size_t)r * a.d;
  // all loads of the row (x, bias and up to 4 partial sums per element) are issued before any is
  // used; the sum itself is taken in a fixed order
  constexpr int kMaxPart = 4;
  float v[NP], pp[NP][kMaxPart];
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int c = threadIdx.x + i * kLnThreads;
    v[i] = 0.f;
#pragma unroll
    for (int p = 0; p < kMaxPart; ++p) pp[i][p] = 0.f;
    if (c < a.d) {
      v[i] = xr[c];
      if (a.n_part > 0) {
#pragma unroll
        for (int p = 0; p < kMaxPart; ++p)
          if (p < a.n_part) pp[i][p] = __ldcg(a.partials + (((size_t)(r >> 7) * a.n_part + p) * kMaxRows + (r & (kMaxRows - 1))) * a.part_cols + c);
      }
    }
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int c = threadIdx.x + i * kLnThreads;
    if (c < a.d && a.n_part > 0) {
      float t = v[i] + bs[i];
#pragma unroll
      for (int p = 0; p < kMaxPart; ++p) t += pp[i][p];
      if (a.write_back) xr[c] = t;
      v[i] = t;
    }
    s += v[i];
  }
  const float mu = block_sum(s, sm) / a.d;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int c = threadIdx.x + i * kLnThreads;
    const float t = c < a.d ? v[i] - mu : 0.f;
    q += t * t;
  }
  const float rstd = rsqrtf(block_sum(q, sm) / a.d + a.eps);
  uint16_t *hid = (a.io && a.io->out_hidden) ? a.io->out_hidden + (size_t)(a.out_slot ? a.out_slot[j] : j) * a.d : nullptr;
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int c = threadIdx.x + i * kLnThreads;
    if (c < a.d) {
      const uint16_t y = float_to_bf16_bits((v[i] - mu) * rstd * gg[i] + bb[i]);
      if (a.out_img) *reinterpret_cast<uint16_t *>(reinterpret_cast<unsigned char *>(a.out_img) + act_image_offset_tiled(j, c, a.d)) = y;
      if (a.out_plain) a.out_plain[(size_t)j * a.d + c] = y;
      if (hid) hid[c] = y;
    }
  }
  trace_mark(a.trace, a.trace_slot, 2);
}

// The same operation for the many rows of a large prefill pass: one warp per row, lane l owning the
// groups of 4 consecutive columns f = l + 32 * m, so that every load instruction of the warp covers 512
// contiguous bytes, every store of bf16 values 256, and the two reductions are warp shuffles with no block
// barrier.  The fold into the residual stream keeps the order of layernorm_tc_kernel (x + bias + partial 0
// + partial 1 + ...), so x comes out bit-identical.  Needs d % 8 == 0 and d <= 128 * NF.
constexpr int kLnRowsWarps = 2;
__device__ __forceinline__ void unpack_bf16x4(const uint2 p, float (&f)[4]) {
  f[0] = __uint_as_float(p.x << 16); f[1] = __uint_as_float(p.x & 0xffff0000u);
  f[2] = __uint_as_float(p.y << 16); f[3] = __uint_as_float(p.y & 0xffff0000u);
}
__device__ __forceinline__ void add4(float (&v)[4], const float4 q) { v[0] += q.x; v[1] += q.y; v[2] += q.z; v[3] += q.w; }
template <int NF>
__global__ void __launch_bounds__(kLnRowsWarps * 32) layernorm_rows_kernel(const LnTcArgs a, int rows) {
  trace_mark(a.trace, a.trace_slot, 0);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int nf = a.d >> 2;
  const bool fold = a.n_part > 0;
  // gamma, beta and the folded bias do not depend on the kernel in front: fetched (packed) ahead of the wait
  uint2 gp[NF], bp[NF], sp[NF];
#pragma unroll
  for (int m = 0; m < NF; ++m) {
    const int f = lane + 32 * m;
    gp[m] = bp[m] = sp[m] = make_uint2(0, 0);
    if (f < nf) {
      gp[m] = __ldg(reinterpret_cast<const uint2 *>(a.g) + f);
      bp[m] = __ldg(reinterpret_cast<const uint2 *>(a.b) + f);
      if (fold && a.add_bias) sp[m] = __ldg(reinterpret_cast<const uint2 *>(a.add_bias) + f);
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  trace_mark(a.trace, a.trace_slot, 1);
  const int j = blockIdx.x * kLnRowsWarps + w;
  if (j >= rows) return;
  const int r = a.gather ? a.gather[j] : j;
  float *xr = a.x + (size_t)r * a.d;
  const float4 *pr = reinterpret_cast<const float4 *>(
      a.partials + (((size_t)(r >> 7) * a.n_part) * kMaxRows + (r & (kMaxRows - 1))) * a.part_cols);
  const size_t pstride = (size_t)kMaxRows * a.part_cols / 4;
  // the row is latency-bound: the loads of x and of two partial sums at a time are all issued before
  // the first of them is used, and nothing is stored until every load has come back
  float v[NF][4];
#pragma unroll
  for (int m = 0; m < NF; ++m) {
    const int f = lane + 32 * m;
    const float4 x = f < nf ? __ldcg(reinterpret_cast<const float4 *>(xr) + f) : make_float4(0.f, 0.f, 0.f, 0.f);
    v[m][0] = x.x; v[m][1] = x.y; v[m][2] = x.z; v[m][3] = x.w;
  }
  if (fold) {
    float4 q[NF][2];
#pragma unroll
    for (int pp = 0; pp < 4; pp += 2) {
      if (pp < a.n_part) {
        const bool two = pp + 1 < a.n_part;
#pragma unroll
        for (int m = 0; m < NF; ++m) {
          const int f = lane + 32 * m;
          q[m][0] = q[m][1] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (f < nf) {
            q[m][0] = __ldcg(pr + pp * pstride + f);
            if (two) q[m][1] = __ldcg(pr + (pp + 1) * pstride + f);
          }
        }
        if (pp == 0) {
#pragma unroll
          for (int m = 0; m < NF; ++m) {
            float bs[4];
            unpack_bf16x4(sp[m], bs);
#pragma unroll
            for (int k = 0; k < 4; ++k) v[m][k] += bs[k];
          }
        }
#pragma unroll
        for (int m = 0; m < NF; ++m) { add4(v[m], q[m][0]); add4(v[m], q[m][1]); }
      }
    }
    if (a.write_back) {
#pragma unroll
      for (int m = 0; m < NF; ++m) {
        const int f = lane + 32 * m;
        if (f < nf) reinterpret_cast<float4 *>(xr)[f] = make_float4(v[m][0], v[m][1], v[m][2], v[m][3]);
      }
    }
  }
  float s = 0.f;
#pragma unroll
  for (int m = 0; m < NF; ++m) s += (v[m][0] + v[m][1]) + (v[m][2] + v[m][3]);
  const float mu = warp_sum(s) / a.d;
  float qq = 0.f;
#pragma unroll
  for (int m = 0; m < NF; ++m) {
    if (lane + 32 * m < nf) {
#pragma unroll
      for (int k = 0; k < 4; ++k) { const float t = v[m][k] - mu; qq += t * t; }
    }
  }
  const float rstd = rsqrtf(warp_sum(qq) / a.d + a.eps);
  uint16_t *hid = (a.io && a.io->out_hidden) ? a.io->out_hidden + (size_t)(a.out_slot ? a.out_slot[j] : j) * a.d : nullptr;
#pragma unroll
  for (int m = 0; m < NF; ++m) {
    const int f = lane + 32 * m;
    if (f < nf) {
      float gg[4], bb[4];
      unpack_bf16x4(gp[m], gg);
      unpack_bf16x4(bp[m], bb);
      uint32_t y[2];
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const uint32_t lo = float_to_bf16_bits((v[m][2 * k] - mu) * rstd * gg[2 * k] + bb[2 * k]);
        const uint32_t hi = float_to_bf16_bits((v[m][2 * k + 1] - mu) * rstd * gg[2 * k + 1] + bb[2 * k + 1]);
        y[k] = lo | (hi << 16);
      }
      const uint2 yy = make_uint2(y[0], y[1]);
      if (a.out_img) *reinterpret_cast<uint2 *>(reinterpret_cast<unsigned char *>(a.out_img) + act_image_offset_tiled(j, f * 4, a.d)) = yy;
      if (a.out_plain) *reinterpret_cast<uint2 *>(a.out_plain + (size_t)j * a.d + f * 4) = yy;
      if (hid) *reinterpret_cast<uint2 *>(hid + f * 4) = yy;
    }
  }
  trace_mark(a.trace, a.trace_slot, 2);
}

// ------------------------------------------------------------------------------------------
// sampling
// ------------------------------------------------------------------------------------------
constexpr int kSampleThreads = 1024;
constexpr int kSampleMaxPer = 9;   // vocab <= 9216
constexpr int kMaxTopK = 64;

__device__ __forceinline__ uint32_t float_to_ordered(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SampleArgs {
  const float *logits;   // [n][V], compact
  int V;
  const StepIO *io;      // if non-null: settings and pointers come from here
  int top_k; float temperature; const float *uniforms; int *out_tokens;  // used when io == null
  const int *out_slot, *out_rows, *row_stream;  // optional
  int *last_token;       // optional, indexed by stream
  int *stop_flag; int stop_token;
};

// One CTA per row.  Greedy: arg max, lowest index on ties.  Top-k: the k largest by (logit
// descending, index ascending) found by a 4-pass radix select on the order-preserving integer
// image of the float, then w_r = exp((l_r - l_0)/T), inverse CDF on the caller's uniform.
__global__ void __launch_bounds__(kSampleThreads) sample_kernel(const SampleArgs a) {
  extern __shared__ float lg[];  // V floats
  __shared__ unsigned int hist[256];
  __shared__ unsigned int sh_prefix, sh_remaining, sh_count;
  __shared__ float wv[32]; __shared__ int wi[32];
  __shared__ unsigned int tie_warp[32];
  __shared__ float sel_v[kMaxTopK]; __shared__ int sel_i[kMaxTopK];
  __shared__ float srt_v[kMaxTopK]; __shared__ int srt_i[kMaxTopK];

  pdl_launch_dependents();
  pdl_wait();
  const int j = blockIdx.x;
  const int slot = a.out_slot ? a.out_slot[j] : j;
  const int V = a.V;
  const float *src = a.logits + (size_t)j * V;
  int top_k = a.top_k; float temperature = a.temperature;
  const float *uniforms = a.uniforms; int *out_tokens = a.out_tokens; float *out_logits = nullptr;
  if (a.io) {
    top_k = a.io->top_k; temperature = a.io->temperature; uniforms = a.io->uniforms;
    out_tokens = a.io->out_tokens; out_logits = a.io->out_logits;
  }
  for (int i = threadIdx.x; i < V; i += blockDim.x) {
    const float v = src[i];
    lg[i] = v;
    if (out_logits) out_logits[(size_t)slot * V + i] = v;
  }
  __syncthreads();
  // blocked ownership: thread t owns indices [t*per, t*per+per)
  const int per = (V + blockDim.x - 1) / blockDim.x;
  const int i0 = threadIdx.x * per;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int token;

  if (top_k <= 1) {
    float bv = -INFINITY; int bi = 0x7FFFFFFF;
    for (int q = 0; q < per; ++q) {
      const int i = i0 + q;
      if (i < V) { const float v = lg[i]; if (v > bv) { bv = v; bi = i; } }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) { wv[warp] = bv; wi[warp] = bi; }
    __syncthreads();
    if (threadIdx.x != 0) return;
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
      if (wv[w] > bv || (wv[w] == bv && wi[w] < bi)) { bv = wv[w]; bi = wi[w]; }
    token = bi;
  } else {
    if (top_k > kMaxTopK) top_k = kMaxTopK;
    if (top_k > V) top_k = V;
    uint32_t ok[kSampleMaxPer];
#pragma unroll
    for (int q = 0; q < kSampleMaxPer; ++q) {
      const int i = i0 + q;
      ok[q] = (q < per && i < V) ? float_to_ordered(lg[i]) : 0u;
    }
    if (threadIdx.x == 0) { sh_prefix = 0u; sh_remaining = (unsigned)top_k; sh_count = 0u; }
    uint32_t mask = 0u;
    for (int pass = 3; pass >= 0; --pass) {
      const int shift = 8 * pass;
      if (threadIdx.x < 256) hist[threadIdx.x] = 0u;
      __syncthreads();
      const uint32_t prefix = sh_prefix;
#pragma unroll
      for (int q = 0; q < kSampleMaxPer; ++q) {
        const int i = i0 + q;
        if (q < per && i < V && (ok[q] & mask) == prefix) atomicAdd(&hist[(ok[q] >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (warp == 0) {
        // find the bin (from the top) in which the running count reaches `rem`: lane L owns bins
        // 8L..8L+7; counts above the lane come from a suffix scan over the lanes' totals
        const unsigned int rem = sh_remaining;
        unsigned int hb[8], tot = 0u;
#pragma unroll
        for (int b = 0; b < 8; ++b) { hb[b] = hist[8 * lane + b]; tot += hb[b]; }
        unsigned int suf = tot;   // inclusive suffix sum over lanes >= this one
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned int n = __shfl_down_sync(0xFFFFFFFFu, suf, o);
          if (lane + o < 32) suf += n;
        }
        unsigned int cum = suf - tot;   // entries in bins above this lane's
        if (cum < rem && cum + tot >= rem) {   // the crossing happens inside this lane's bins
          int bin = 7;
          for (; bin > 0; --bin) {
            if (cum + hb[bin] >= rem) break;
            cum += hb[bin];
          }
          sh_remaining = rem - cum;
          sh_prefix = prefix | ((uint32_t)(8 * lane + bin) << shift);
        }
      }
      mask |= 255u << shift;
      __syncthreads();
    }
    const uint32_t thr = sh_prefix;           // ordered image of the k-th largest logit
    const unsigned int need_ties = sh_remaining;  // how many entries equal to it belong to the top k
    // rank ties by index: blocked ownership makes (thread, local order) the index order
    unsigned int my_ties = 0u;
#pragma unroll
    for (int q = 0; q < kSampleMaxPer; ++q) {
      const int i = i0 + q;
      if (q < per && i < V && ok[q] == thr) ++my_ties;
    }
    unsigned int incl = my_ties;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned int n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) tie_warp[warp] = incl;
    __syncthreads();
    unsigned int base = incl - my_ties;
    for (int w = 0; w < warp; ++w) base += tie_warp[w];
#pragma unroll
    for (int q = 0; q < kSampleMaxPer; ++q) {
      const int i = i0 + q;
      if (q < per && i < V) {
        bool take = ok[q] > thr;
        if (ok[q] == thr) { take = base < need_ties; ++base; }
        if (take) {
          const unsigned int p = atomicAdd(&sh_count, 1u);
          if (p < (unsigned)kMaxTopK) { sel_v[p] = lg[i]; sel_i[p] = i; }
        }
      }
    }
    __syncthreads();
    const int k = min((int)sh_count, top_k);
    if ((int)threadIdx.x < k) {
      const float v = sel_v[threadIdx.x]; const int id = sel_i[threadIdx.x];
      int rank = 0;
      for (int q = 0; q < k; ++q) rank += (sel_v[q] > v) || (sel_v[q] == v && sel_i[q] < id);
      srt_v[rank] = v; srt_i[rank] = id;
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    const float inv_t = 1.0f / temperature;
    float w[kMaxTopK];
    float total = 0.f;
    for (int r = 0; r < k; ++r) { w[r] = expf((srt_v[r] - srt_v[0]) * inv_t); total += w[r]; }
    const float u = uniforms ? uniforms[slot] : 0.f;
    float cum = 0.f;
    token = srt_i[k - 1];
    for (int r = 0; r < k; ++r) {
      cum += w[r];
      if (u < cum / total) { token = srt_i[r]; break; }
    }
  }
  // thread 0 only
  out_tokens[slot] = token;
  if (a.last_token) {
    const int s = a.row_stream[a.out_rows ? a.out_rows[j] : j];
    a.last_token[s] = token;
    if (a.stop_flag && token == a.stop_token) a.stop_flag[s] = 1;
  }
}

}  // namespace ttsgpt
