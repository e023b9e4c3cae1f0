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

struct Fp8AttnArgs {
  const float *q;                 // [R][H*64]
  const unsigned char *kv_layer;  // this layer's slice of the e4m3 pool
  const int *page_table, *row_stream, *row_pos;
  uint16_t *out;                  // bf16 [R][H*64], or an activation image of the tensor-core linear
  float *partials;                // [R][H][kAttnMaxChunks][66]
  unsigned int *tickets;          // [R][H], zero between launches
  int H, pps, out_image;
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

// Splits per (row, head): enough CTAs of 4 warps to cover the GPU about four times, at most kAttnMaxChunks.
inline int attention_fp8_splits(int R, int H, int n_sm) {
  int s = (4 * n_sm + R * H - 1) / (R * H);
  if (s > kAttnMaxChunks) s = kAttnMaxChunks;
  return s < 1 ? 1 : s;
}

inline cudaError_t launch_kv_quantize(const uint16_t *stage, unsigned char *kv_layer, const int *page_table, const int *row_stream,
                                      const int *row_pos, int pps, int H, int R, cudaStream_t st, bool pdl) {
  return launch_kernel(kv_quantize_kernel, dim3(H, R), dim3(64), 0, st, pdl, stage, kv_layer, page_table, row_stream, row_pos, pps, H);
}

inline cudaError_t launch_attention_fp8(const Fp8AttnArgs &a, int R, int splits, cudaStream_t st, bool pdl) {
  return launch_kernel(attention_fp8_kernel, dim3(splits, a.H, R), dim3(kAttnWarps * 32), 0, st, pdl, a);
}

}  // namespace ttsgpt
