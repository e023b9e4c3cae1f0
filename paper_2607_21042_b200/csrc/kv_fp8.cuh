// 8-bit KV cache: the cached K and V rows as e4m3 codes (a precision variant beyond Table I's FP32 /
// FP16 / W8A16 / W4A16: from 16 streams up the K/V stream is 85-99 % of a decode step's bytes, so the
// bytes of the cache, not of the weights, decide the step time).
//
// Format.  For every cached token and head, the 64 values of K (and of V) share one fp32 scale
// s = max|x| / 448 (1 if all are zero); a value is stored as the e4m3 code nearest to x / s (ties to even,
// finite) and read back as code * s.  A scale per page would need all 64 tokens of the page before the
// first could be encoded, so the scale belongs to the token's row inside the page block.  Pool, per layer:
// [n_pages][2 (K|V)][n_head] blocks of 4352 bytes: 64 tokens x 64 codes, then the 64 scales of the block.
//
// Path.  The QKV linear writes the step's new K/V rows as bf16 into a small staging area;
// `kv_quantize_kernel` encodes them into their page slots (one warp per token, head and K|V);
// `attention_fp8_kernel` is the split-KV decode attention over such pages: a CTA per (row, head, split),
// a warp per page, a lane on 16 codes of one of 8 tokens per load; scores, online softmax and outputs in
// fp32, the scale applied to the 64-term dot product (K) and to the softmax weight (V) rather than to
// every element; partial results of the splits meet through global scratch and the CTA that takes the
// last ticket merges them in split order (no spinning).
#pragma once
#include <cuda_fp8.h>
#include "common.cuh"
#include "elementwise.cuh"
#include "attention.cuh"

namespace ttsgpt {

constexpr int kFp8BlockBytes = kPageTokens * kHeadDim + kPageTokens * 4;   // 4352
constexpr float kE4m3Max = 448.0f;

// 16 e4m3 codes (one 128-bit word) -> 16 floats
__device__ __forceinline__ void e4m3x16_to_float(const uint4 &w, float (&f)[16]) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __half2_raw lo = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(ww[i] & 0xFFFFu), __NV_E4M3);
    const __half2_raw hi = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(ww[i] >> 16), __NV_E4M3);
    const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&lo));
    const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&hi));
    f[4 * i] = a.x; f[4 * i + 1] = a.y; f[4 * i + 2] = b.x; f[4 * i + 3] = b.y;
  }
}

// Encodes the staged K/V rows of a pass into their page slots.  stage: bf16 [R][2][H*64].  grid (H, R),
// 64 threads: warp 0 takes K, warp 1 takes V; a lane takes two neighbouring values.
__global__ void __launch_bounds__(64) kv_quantize_kernel(const uint16_t *__restrict__ stage, unsigned char *__restrict__ kv_layer,
                                                         const int *__restrict__ page_table, const int *__restrict__ row_stream,
                                                         const int *__restrict__ row_pos, int pps, int H) {
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.x, r = blockIdx.y, which = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int d = H * kHeadDim;
  const uint32_t pair = *reinterpret_cast<const uint32_t *>(stage + ((size_t)r * 2 + which) * d + h * kHeadDim + 2 * lane);
  const float x0 = bf16_lo(pair), x1 = bf16_hi(pair);
  const float amax = warp_max(fmaxf(fabsf(x0), fabsf(x1)));
  const float s = amax > 0.f ? amax / kE4m3Max : 1.0f;
  const __nv_fp8x2_storage_t codes = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(x0, s), __fdiv_rn(x1, s)), __NV_SATFINITE, __NV_E4M3);
  const int pos = row_pos[r];
  const int page = page_table[(size_t)row_stream[r] * pps + (pos >> 6)];
  unsigned char *blk = kv_layer + (((size_t)page * 2 + which) * H + h) * kFp8BlockBytes;
  *reinterpret_cast<uint16_t *>(blk + (size_t)(pos & 63) * kHeadDim + 2 * lane) = (uint16_t)codes;
  if (lane == 0) *reinterpret_cast<float *>(blk + kPageTokens * kHeadDim + 4 * (pos & 63)) = s;
}

// The same encoding for the many rows of a large prefill pass: one CTA of 8 warps per row; a warp takes the
// (K|V, head) slices w, w + 8, ... of the row, five at a time with their loads in flight together (a grid of
// one 64-thread CTA per row and head is 18 000 CTAs for a 896-row pass and takes 22 us).  Bit-identical codes.
constexpr int kQrWarps = 8, kQrBatch = 5;
__global__ void __launch_bounds__(kQrWarps * 32) kv_quantize_rows_kernel(const uint16_t *__restrict__ stage, unsigned char *__restrict__ kv_layer,
                                                                         const int *__restrict__ page_table, const int *__restrict__ row_stream,
                                                                         const int *__restrict__ row_pos, int pps, int H) {
  const int r = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pos = row_pos[r];   // the row table is final before the pass's first kernel starts
  const int page = page_table[(size_t)row_stream[r] * pps + (pos >> 6)];
  pdl_launch_dependents();
  pdl_wait();
  const int d = H * kHeadDim, n_items = 2 * H;
  for (int it0 = warp; it0 < n_items; it0 += kQrWarps * kQrBatch) {
    uint32_t pair[kQrBatch];
#pragma unroll
    for (int b = 0; b < kQrBatch; ++b) {
      const int it = it0 + b * kQrWarps;   // item = which * H + head: the staged row is [K of all heads | V of all heads]
      pair[b] = it < n_items ? *reinterpret_cast<const uint32_t *>(stage + (size_t)r * 2 * d + (size_t)it * kHeadDim + 2 * lane) : 0u;
    }
#pragma unroll
    for (int b = 0; b < kQrBatch; ++b) {
      const int it = it0 + b * kQrWarps;
      if (it < n_items) {   // uniform in the warp
        const int which = it / H, h = it - which * H;
        const float x0 = bf16_lo(pair[b]), x1 = bf16_hi(pair[b]);
        const float amax = warp_max(fmaxf(fabsf(x0), fabsf(x1)));
        const float sc = amax > 0.f ? amax / kE4m3Max : 1.0f;
        const __nv_fp8x2_storage_t codes = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(x0, sc), __fdiv_rn(x1, sc)), __NV_SATFINITE, __NV_E4M3);
        unsigned char *blk = kv_layer + (((size_t)page * 2 + which) * H + h) * kFp8BlockBytes;
        *reinterpret_cast<uint16_t *>(blk + (size_t)(pos & 63) * kHeadDim + 2 * lane) = (uint16_t)codes;
        if (lane == 0) *reinterpret_cast<float *>(blk + kPageTokens * kHeadDim + 4 * (pos & 63)) = sc;
      }
    }
  }
}

struct Fp8AttnArgs {
  const float *q;                 // [R][H*64]
  const unsigned char *kv_layer;  // this layer's slice of the e4m3 pool
  const int *page_table, *row_stream, *row_pos;
  uint16_t *out;                  // bf16 [R][H*64], or an activation image of the tensor-core linear
  float *partials;                // [R][H][kAttnMaxChunks][66]
  unsigned int *tickets;          // [R][H], zero between launches
  int H, pps, out_image;
  const int *row_order;           // streaming variant: rows by descending context length, or null
  int *err;                       // streaming variant: set when a bounded wait ran out
  unsigned long long *trace;
  int trace_slot;
};

// Folds 4 tokens of a page (one per slot; lane (tg, sub) holds 16 codes of token 8*slot + tg) into the
// warp's running (m, l, o).  At least one slot of the warp must be valid.
__device__ __forceinline__ void fp8_fold4(const uint4 (&kk)[4], const uint4 (&vv)[4], const float (&ks)[4], const float (&vs)[4],
                                          uint32_t vmask, const float (&qv)[16], float &m, float &l, float (&o)[16]) {
  float s[4];
  float pm = -INFINITY;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float kf[16];
    e4m3x16_to_float(kk[i], kf);
    float d0 = 0.f, d1 = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) { d0 = fmaf(qv[e], kf[e], d0); d1 = fmaf(qv[8 + e], kf[8 + e], d1); }
    float dsum = d0 + d1;
    dsum += __shfl_xor_sync(0xFFFFFFFFu, dsum, 1);
    dsum += __shfl_xor_sync(0xFFFFFFFFu, dsum, 2);
    s[i] = ((vmask >> i) & 1u) ? dsum * ks[i] : -INFINITY;
    pm = fmaxf(pm, s[i]);
  }
  pm = fmaxf(pm, __shfl_xor_sync(0xFFFFFFFFu, pm, 4));
  pm = fmaxf(pm, __shfl_xor_sync(0xFFFFFFFFu, pm, 8));
  pm = fmaxf(pm, __shfl_xor_sync(0xFFFFFFFFu, pm, 16));
  const float m_new = fmaxf(m, pm);
  const float rescale = exp2f(m - m_new);
#pragma unroll
  for (int e = 0; e < 16; ++e) o[e] *= rescale;
  float lp = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const bool ok = (vmask >> i) & 1u;
    const float p = exp2f(s[i] - m_new);      // a slot without a token: exp2(-inf) = 0
    lp += p;
    float vf[16];
    e4m3x16_to_float(ok ? vv[i] : make_uint4(0, 0, 0, 0), vf);   // a stale slot may decode to NaN: 0 * NaN must not reach o
    const float w = ok ? p * vs[i] : 0.f;
#pragma unroll
    for (int e = 0; e < 16; ++e) o[e] = fmaf(w, vf[e], o[e]);
  }
  l = l * rescale + lp;       // lp is per token group; the groups are summed at the end
  m = m_new;
}

__global__ void __launch_bounds__(kAttnWarps * 32) attention_fp8_kernel(const Fp8AttnArgs a) {
  const int c = blockIdx.x, S = gridDim.x, h = blockIdx.y, r = blockIdx.z;
  trace_mark(a.trace, a.trace_slot, 0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tg = lane >> 2, sub = lane & 3;
  __shared__ float sm_m[kAttnWarps], sm_l[kAttnWarps], sm_o[kAttnWarps][kHeadDim];
  __shared__ unsigned int sm_ticket;
  pdl_launch_dependents();
  pdl_wait();
  trace_mark(a.trace, a.trace_slot, 1);
  const int n_tok = min(a.row_pos[r] + 1, a.pps * kPageTokens);
  const int n_pages = (n_tok + kPageTokens - 1) / kPageTokens;
  const int per = (n_pages + S - 1) / S;                   // pages per split
  const int n_chunks = (n_pages + per - 1) / per;          // splits that have pages
  if (c >= n_chunks) return;
  const int p0 = c * per, p1 = min(n_pages, p0 + per);
  const int *pt = a.page_table + (size_t)a.row_stream[r] * a.pps;

  float qv[16];
  {
    const float qs = 0.125f * 1.4426950408889634f;   // scores in log2 units
    const float *qp = a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim + 16 * sub;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float4 t = *reinterpret_cast<const float4 *>(qp + 4 * e);
      qv[4 * e] = t.x * qs; qv[4 * e + 1] = t.y * qs; qv[4 * e + 2] = t.z * qs; qv[4 * e + 3] = t.w * qs;
    }
  }
  float m = -INFINITY, l = 0.f, o[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) o[e] = 0.f;
  for (int page = p0 + warp; page < p1; page += kAttnWarps) {
    const int phys = pt[page];
    const unsigned char *K = a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kFp8BlockBytes;
    const unsigned char *V = a.kv_layer + (((size_t)phys * 2 + 1) * a.H + h) * kFp8BlockBytes;
    const int n_here = min(kPageTokens, n_tok - page * kPageTokens);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      if (32 * half >= n_here) break;                  // warp-uniform
      uint4 kk[4], vv[4];
      float ks[4], vs[4];
      uint32_t vmask = 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = 32 * half + 8 * i + tg;
        kk[i] = ld_stream_u4(K + (size_t)t * kHeadDim + 16 * sub);
        vv[i] = ld_stream_u4(V + (size_t)t * kHeadDim + 16 * sub);
        ks[i] = *reinterpret_cast<const float *>(K + kPageTokens * kHeadDim + 4 * t);
        vs[i] = *reinterpret_cast<const float *>(V + kPageTokens * kHeadDim + 4 * t);
        if (t < n_here) vmask |= 1u << i;
      }
      fp8_fold4(kk, vv, ks, vs, vmask, qv, m, l, o);
    }
  }
  // warp result: sum over the 8 token groups
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 4);
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 8);
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 16);
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 4);
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 8);
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 16);
  }
  if (tg == 0) {
    if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
#pragma unroll
    for (int e = 0; e < 16; ++e) sm_o[warp][16 * sub + e] = o[e];
  }
  __syncthreads();
  trace_mark(a.trace, a.trace_slot, 3);
  const int e = threadIdx.x;
  float M = -INFINITY, L = 0.f, O = 0.f;
  if (e < kHeadDim) {
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, sm_m[w]);
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float f = (sm_m[w] == -INFINITY) ? 0.f : exp2f(sm_m[w] - M);   // a warp without pages contributes nothing
      L = fmaf(sm_l[w], f, L);
      O = fmaf(sm_o[w][e], f, O);
    }
  }
  uint16_t *out = nullptr;
  if (e < kHeadDim)
    out = a.out_image ? reinterpret_cast<uint16_t *>(reinterpret_cast<unsigned char *>(a.out) + act_image_offset_tiled(r, h * kHeadDim + e, a.H * kHeadDim))
                      : a.out + (size_t)r * a.H * kHeadDim + h * kHeadDim + e;
  if (n_chunks == 1) {
    if (e < kHeadDim) *out = float_to_bf16_bits(O / L);
    trace_mark(a.trace, a.trace_slot, 2);
    return;
  }
  float *part = a.partials + (((size_t)r * a.H + h) * kAttnMaxChunks) * kAttnPartialFloats;
  if (e < kHeadDim) {
    float *mine = part + (size_t)c * kAttnPartialFloats;
    if (e == 0) { mine[0] = M; mine[1] = L; }
    mine[2 + e] = O;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) sm_ticket = atomicAdd(&a.tickets[(size_t)r * a.H + h], 1u);
  __syncthreads();
  if (sm_ticket != (unsigned int)(n_chunks - 1)) return;
  __threadfence();
  if (e < kHeadDim) {
    float MM = -INFINITY;
    for (int cc = 0; cc < n_chunks; ++cc) MM = fmaxf(MM, __ldcg(part + (size_t)cc * kAttnPartialFloats));
    float LL = 0.f, OO = 0.f;
    for (int cc = 0; cc < n_chunks; ++cc) {
      const float *p = part + (size_t)cc * kAttnPartialFloats;
      const float f = exp2f(__ldcg(p) - MM);
      LL = fmaf(__ldcg(p + 1), f, LL);
      OO = fmaf(__ldcg(p + 2 + e), f, OO);
    }
    *out = float_to_bf16_bits(OO / LL);
  }
  if (threadIdx.x == 0) a.tickets[(size_t)r * a.H + h] = 0u;  // ready for the next launch
  trace_mark(a.trace, a.trace_slot, 2);
}

// ------------------------------------------------------------------------------------------
// Prefill passes over the 8-bit cache.  The tensor-core prefill attention reads bf16 pages, and the rows
// of a pass share the pages of a few streams, so those pages (a few dozen per pass) are decoded once per
// layer into a scratch pool of bf16 pages with a page table of its own, and the bf16 kernel runs on that.
// A decoded value is code x scale rounded to bf16: the rounding the bf16 cache applies to every value.
// scratch page i = page `scratch_src[i]` of the pool, of which the first scratch_ntok[i] tokens exist (the
// rest is written as zero: a stale slot may decode to NaN).  grid (scratch pages, 2 * H), 128 threads:
// thread = (token, half of its 64 codes).
__global__ void __launch_bounds__(128) kv_dequant_pages_kernel(const unsigned char *__restrict__ kv_layer, uint16_t *__restrict__ scratch,
                                                               const int *__restrict__ scratch_src, const int *__restrict__ scratch_ntok, int H) {
  pdl_launch_dependents();
  pdl_wait();   // the pass's own rows were encoded by the kernel in front
  const int i = blockIdx.x, which = blockIdx.y / H, head = blockIdx.y % H;
  const int t = threadIdx.x >> 1, half = threadIdx.x & 1;
  const unsigned char *blk = kv_layer + (((size_t)scratch_src[i] * 2 + which) * H + head) * kFp8BlockBytes;
  uint16_t *dst = scratch + (((size_t)i * 2 + which) * H + head) * kPageElems + (size_t)t * kHeadDim + 32 * half;
  uint4 out[4] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)};
  if (t < scratch_ntok[i]) {
    const float sc = *reinterpret_cast<const float *>(blk + kPageTokens * kHeadDim + 4 * t);
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      float f[16];
      e4m3x16_to_float(*reinterpret_cast<const uint4 *>(blk + (size_t)t * kHeadDim + 32 * half + 16 * q), f);
      out[2 * q] = make_uint4(pack_bf16x2(f[0] * sc, f[1] * sc), pack_bf16x2(f[2] * sc, f[3] * sc),
                              pack_bf16x2(f[4] * sc, f[5] * sc), pack_bf16x2(f[6] * sc, f[7] * sc));
      out[2 * q + 1] = make_uint4(pack_bf16x2(f[8] * sc, f[9] * sc), pack_bf16x2(f[10] * sc, f[11] * sc),
                                  pack_bf16x2(f[12] * sc, f[13] * sc), pack_bf16x2(f[14] * sc, f[15] * sc));
    }
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) reinterpret_cast<uint4 *>(dst)[q] = out[q];
}

inline cudaError_t launch_kv_dequant_pages(const unsigned char *kv_layer, uint16_t *scratch, const int *src, const int *ntok,
                                           int n_scratch, int H, cudaStream_t st, bool pdl) {
  return launch_kernel(kv_dequant_pages_kernel, dim3(n_scratch, 2 * H), dim3(128), 0, st, pdl, kv_layer, scratch, src, ntok, H);
}

// ------------------------------------------------------------------------------------------
// Streaming variant for decode steps with enough (row, head) pairs to cover the GPU several times
// (the same switch as the bf16 cache's streaming kernel): one CTA per pair, rows longest first,
// warp w owns pages w, w+4, ...  A page's K and V blocks (4352 bytes each: codes, then scales) come
// in by two bulk asynchronous copies into one of the warp's two stages; while the warp folds one
// stage, the copy of its page after next runs into the other, so every resident warp keeps 8.7 KB
// in flight without holding registers for outstanding loads.  The pages of a decode step are final
// before the step starts, except the slot of the new token in the row's last page, which the
// encoding kernel in front writes: every page but the last is requested ahead of the dependency
// wait.
constexpr uint32_t kFp8StageBytes = 2 * kFp8BlockBytes;   // K block | V block
constexpr int kFp8Stages = 2;

__device__ __forceinline__ void fp8_stream_issue(const Fp8AttnArgs &a, const int *pt, int h, int page, unsigned char *stage, uint64_t *bar) {
  const int phys = pt[page];
  const unsigned char *K = a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kFp8BlockBytes;
  mbar_expect_tx(bar, kFp8StageBytes);
  bulk_copy_g2s(stage, K, kFp8BlockBytes, bar);
  bulk_copy_g2s(stage + kFp8BlockBytes, K + (size_t)a.H * kFp8BlockBytes, kFp8BlockBytes, bar);   // the V block of the same page and head
}

__global__ void __launch_bounds__(kAttnWarps * 32, 3) attention_fp8_stream_kernel(const Fp8AttnArgs a) {
  extern __shared__ __align__(128) unsigned char fp8_stages[];   // [warp][stage][K block | V block]
  __shared__ __align__(8) uint64_t bars[kAttnWarps][kFp8Stages];
  __shared__ float sm_m[kAttnWarps], sm_l[kAttnWarps], sm_o[kAttnWarps][kHeadDim];
  const int h = blockIdx.y, r = a.row_order ? a.row_order[blockIdx.z] : blockIdx.z;
  trace_mark(a.trace, a.trace_slot, 0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tg = lane >> 2, sub = lane & 3;
  const int n_tok = min(a.row_pos[r] + 1, a.pps * kPageTokens);   // row and page tables are final before the step's first kernel starts
  const int n_pages = (n_tok + kPageTokens - 1) / kPageTokens;
  const int *pt = a.page_table + (size_t)a.row_stream[r] * a.pps;
  unsigned char *stages = fp8_stages + (size_t)warp * (kFp8Stages * kFp8StageBytes);
  // pages of this warp: warp, warp + 4, ...; iteration it uses stage it % 2
  bool issued[kFp8Stages] = {false, false};
  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kFp8Stages; ++s) mbar_init(&bars[warp][s], 1);
#pragma unroll
    for (int s = 0; s < kFp8Stages; ++s) {
      const int page = warp + kAttnWarps * s;
      if (page < n_pages - 1) { fp8_stream_issue(a, pt, h, page, stages + s * kFp8StageBytes, &bars[warp][s]); issued[s] = true; }
    }
  }
  __syncwarp();
  pdl_launch_dependents();
  pdl_wait();
  trace_mark(a.trace, a.trace_slot, 1);
  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kFp8Stages; ++s) {
      const int page = warp + kAttnWarps * s;
      if (!issued[s] && page < n_pages) fp8_stream_issue(a, pt, h, page, stages + s * kFp8StageBytes, &bars[warp][s]);
    }
  }
  float qv[16];
  {
    const float qs = 0.125f * 1.4426950408889634f;   // scores in log2 units
    const float *qp = a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim + 16 * sub;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float4 t = *reinterpret_cast<const float4 *>(qp + 4 * e);
      qv[4 * e] = t.x * qs; qv[4 * e + 1] = t.y * qs; qv[4 * e + 2] = t.z * qs; qv[4 * e + 3] = t.w * qs;
    }
  }
  float m = -INFINITY, l = 0.f, o[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) o[e] = 0.f;
  int it = 0;
  for (int page = warp; page < n_pages; page += kAttnWarps, ++it) {
    const int s = it & 1;
    uint64_t *bar = &bars[warp][s];
    if (!mbar_wait_bounded(bar, (uint32_t)(it >> 1) & 1u, kAttnWaitNs)) {
      if (a.err) atomicExch(a.err, 1);
      mbar_wait_bounded(bar, (uint32_t)(it >> 1) & 1u, kAttnWaitNs);   // a last chance for the copy in flight towards this CTA
      break;
    }
    const unsigned char *K = stages + s * kFp8StageBytes, *V = K + kFp8BlockBytes;
    const int n_here = min(kPageTokens, n_tok - page * kPageTokens);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      if (32 * half >= n_here) break;                  // warp-uniform
      uint4 kk[4], vv[4];
      float ks[4], vs[4];
      uint32_t vmask = 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = 32 * half + 8 * i + tg;
        kk[i] = *reinterpret_cast<const uint4 *>(K + (size_t)t * kHeadDim + 16 * sub);
        vv[i] = *reinterpret_cast<const uint4 *>(V + (size_t)t * kHeadDim + 16 * sub);
        ks[i] = *reinterpret_cast<const float *>(K + kPageTokens * kHeadDim + 4 * t);
        vs[i] = *reinterpret_cast<const float *>(V + kPageTokens * kHeadDim + 4 * t);
        if (t < n_here) vmask |= 1u << i;
      }
      fp8_fold4(kk, vv, ks, vs, vmask, qv, m, l, o);
    }
    // The stage may be refilled only after every lane's reads of it have returned: the ballot needs a value
    // that every lane computed from what it read, and the fence takes the ballot as an operand.
    const unsigned int done = __ballot_sync(0xFFFFFFFFu, o[0] == o[0] || l >= 0.f);
    if (page + kFp8Stages * kAttnWarps < n_pages && lane == 0) {
      asm volatile("fence.proxy.async.shared::cta; // after %0" ::"r"(done) : "memory");
      fp8_stream_issue(a, pt, h, page + kFp8Stages * kAttnWarps, stages + s * kFp8StageBytes, bar);
    }
  }
  trace_mark(a.trace, a.trace_slot, 3);
  // warp result: sum over the 8 token groups
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 4);
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 8);
  l += __shfl_xor_sync(0xFFFFFFFFu, l, 16);
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 4);
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 8);
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 16);
  }
  if (tg == 0) {
    if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
#pragma unroll
    for (int e = 0; e < 16; ++e) sm_o[warp][16 * sub + e] = o[e];
  }
  __syncthreads();
  const int e = threadIdx.x;
  if (e < kHeadDim) {
    float M = -INFINITY, L = 0.f, O = 0.f;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, sm_m[w]);
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float f = (sm_m[w] == -INFINITY) ? 0.f : exp2f(sm_m[w] - M);   // a warp without pages contributes nothing
      L = fmaf(sm_l[w], f, L);
      O = fmaf(sm_o[w][e], f, O);
    }
    uint16_t *out = a.out_image ? reinterpret_cast<uint16_t *>(reinterpret_cast<unsigned char *>(a.out) + act_image_offset_tiled(r, h * kHeadDim + e, a.H * kHeadDim))
                                : a.out + (size_t)r * a.H * kHeadDim + h * kHeadDim + e;
    *out = float_to_bf16_bits(O / L);
  }
  trace_mark(a.trace, a.trace_slot, 2);
}

inline cudaError_t launch_attention_fp8_stream(const Fp8AttnArgs &a, int R, cudaStream_t st, bool pdl) {
  static PerDeviceOnce attr_once;   // per device: opt-in to more than 48 KB of dynamic shared memory
  const size_t smem = (size_t)kAttnWarps * kFp8Stages * kFp8StageBytes;
  if (attr_once.first()) cudaFuncSetAttribute(attention_fp8_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  return launch_kernel(attention_fp8_stream_kernel, dim3(1, a.H, R), dim3(kAttnWarps * 32), smem, st, pdl, a);
}

// Splits per (row, head): enough CTAs of 4 warps to cover the GPU about four times, at most kAttnMaxChunks.
inline int attention_fp8_splits(int R, int H, int n_sm) {
  int s = (4 * n_sm + R * H - 1) / (R * H);
  if (s > kAttnMaxChunks) s = kAttnMaxChunks;
  return s < 1 ? 1 : s;
}

inline cudaError_t launch_kv_quantize(const uint16_t *stage, unsigned char *kv_layer, const int *page_table, const int *row_stream,
                                      const int *row_pos, int pps, int H, int R, cudaStream_t st, bool pdl) {
  if (R > kMaxRows)   // a prefill pass of several row tiles
    return launch_kernel(kv_quantize_rows_kernel, dim3(R), dim3(kQrWarps * 32), 0, st, pdl, stage, kv_layer, page_table, row_stream, row_pos, pps, H);
  return launch_kernel(kv_quantize_kernel, dim3(H, R), dim3(64), 0, st, pdl, stage, kv_layer, page_table, row_stream, row_pos, pps, H);
}

inline cudaError_t launch_attention_fp8(const Fp8AttnArgs &a, int R, int splits, cudaStream_t st, bool pdl) {
  return launch_kernel(attention_fp8_kernel, dim3(splits, a.H, R), dim3(kAttnWarps * 32), 0, st, pdl, a);
}

}  // namespace ttsgpt
