// Split-KV decode attention over 64-token pages (Section I: the decode engine's attention kernels
// and KV-cache management).  One warp owns one page of one (row, head): it streams the 8 KB K block
// and the 8 KB V block with 128-bit loads, keeps scores, softmax statistics and the output in fp32
// registers, and uses warp shuffles for the reductions.  Four warps (a 256-token chunk) meet in
// shared memory; when a row needs several chunks the per-chunk (max, sum, output) triples go to
// scratch and the CTA that arrives last at the row's ticket counter merges them in chunk order by
// log-sum-exp (no spinning, no dependence on arrival order).
//
// KV pool, per layer: bf16 [n_pages][2 (K|V)][n_head][64 tokens][64]; each (page, K|V, head) block
// is 8 KB contiguous.
#pragma once
#include "common.cuh"

namespace ttsgpt {

constexpr int kAttnWarps = 4;             // pages per chunk
constexpr int kAttnMaxChunks = 8;         // 2048 tokens / 256
constexpr int kAttnPartialFloats = 66;    // m, l, o[64]

inline size_t attention_scratch_bytes(int R, int H) {
  return align256((size_t)R * H * kAttnMaxChunks * kAttnPartialFloats * sizeof(float)) +
         align256((size_t)R * H * sizeof(unsigned int));
}

struct AttnArgs {
  const float *q;            // [R][H*64]
  const uint16_t *kv_layer;  // this layer's pool slice
  const int *page_table;     // [*, pps]
  const int *row_stream, *row_pos;
  uint16_t *out;             // bf16 [R][H*64]
  float *partials;           // [R][H][kAttnMaxChunks][66]
  unsigned int *tickets;     // [R][H], zero between launches
  int H, pps;
};

__global__ void __launch_bounds__(kAttnWarps * 32) attention_kernel(const AttnArgs a) {
  const int c = blockIdx.x, h = blockIdx.y, r = blockIdx.z;
  const int n_tok = a.row_pos[r] + 1;
  const int n_pages = (n_tok + kPageTokens - 1) / kPageTokens;
  const int n_chunks = (n_pages + kAttnWarps - 1) / kAttnWarps;
  if (c >= n_chunks) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tg = lane >> 3, sub = lane & 7;  // token group (4 tokens per load), 8-element slice of the head
  const int page = c * kAttnWarps + warp;

  __shared__ float sm_m[kAttnWarps], sm_l[kAttnWarps], sm_o[kAttnWarps][kHeadDim];
  __shared__ unsigned int sm_ticket;

  float m = -INFINITY, l = 0.f;
  float o[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) o[e] = 0.f;

  if (page < n_pages) {
    const int phys = a.page_table[(size_t)a.row_stream[r] * a.pps + page];
    const uint16_t *K = a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kPageElems;
    const uint16_t *V = a.kv_layer + (((size_t)phys * 2 + 1) * a.H + h) * kPageElems;
    const int n_here = min(kPageTokens, n_tok - page * kPageTokens);
    // scores come out in log2 units: 1/sqrt(64) * log2(e)
    const float qs = 0.125f * 1.4426950408889634f;
    float qv[8];
    {
      const float4 q0 = *reinterpret_cast<const float4 *>(a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim + 8 * sub);
      const float4 q1 = *reinterpret_cast<const float4 *>(a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim + 8 * sub + 4);
      qv[0] = q0.x * qs; qv[1] = q0.y * qs; qv[2] = q0.z * qs; qv[3] = q0.w * qs;
      qv[4] = q1.x * qs; qv[5] = q1.y * qs; qv[6] = q1.z * qs; qv[7] = q1.w * qs;
    }
    uint4 kk[16], vv[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) kk[i] = ld_stream_u4(K + (size_t)(tg + 4 * i) * kHeadDim + 8 * sub);
#pragma unroll
    for (int i = 0; i < 16; ++i) vv[i] = ld_stream_u4(V + (size_t)(tg + 4 * i) * kHeadDim + 8 * sub);
    float s[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      float d = qv[0] * bf16_lo(kk[i].x);
      d = fmaf(qv[1], bf16_hi(kk[i].x), d);
      d = fmaf(qv[2], bf16_lo(kk[i].y), d);
      d = fmaf(qv[3], bf16_hi(kk[i].y), d);
      d = fmaf(qv[4], bf16_lo(kk[i].z), d);
      d = fmaf(qv[5], bf16_hi(kk[i].z), d);
      d = fmaf(qv[6], bf16_lo(kk[i].w), d);
      d = fmaf(qv[7], bf16_hi(kk[i].w), d);
      d += __shfl_xor_sync(0xFFFFFFFFu, d, 1);
      d += __shfl_xor_sync(0xFFFFFFFFu, d, 2);
      d += __shfl_xor_sync(0xFFFFFFFFu, d, 4);
      const bool valid = tg + 4 * i < n_here;
      s[i] = valid ? d : -INFINITY;
      if (!valid) vv[i] = make_uint4(0, 0, 0, 0);  // stale page contents may hold NaN: 0 * NaN must not reach o
      m = fmaxf(m, s[i]);
    }
    m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 8));
    m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 16));
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float p = exp2f(s[i] - m);  // masked tokens: exp2(-inf) = 0
      l += p;
      o[0] = fmaf(p, bf16_lo(vv[i].x), o[0]);
      o[1] = fmaf(p, bf16_hi(vv[i].x), o[1]);
      o[2] = fmaf(p, bf16_lo(vv[i].y), o[2]);
      o[3] = fmaf(p, bf16_hi(vv[i].y), o[3]);
      o[4] = fmaf(p, bf16_lo(vv[i].z), o[4]);
      o[5] = fmaf(p, bf16_hi(vv[i].z), o[5]);
      o[6] = fmaf(p, bf16_lo(vv[i].w), o[6]);
      o[7] = fmaf(p, bf16_hi(vv[i].w), o[7]);
    }
    l += __shfl_xor_sync(0xFFFFFFFFu, l, 8);
    l += __shfl_xor_sync(0xFFFFFFFFu, l, 16);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 8);
      o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 16);
    }
  }
  if (tg == 0) {
    if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
#pragma unroll
    for (int e = 0; e < 8; ++e) sm_o[warp][8 * sub + e] = o[e];
  }
  __syncthreads();

  // merge the chunk's warps (in warp order)
  float M = -INFINITY, L = 0.f, O = 0.f;
  const int e = threadIdx.x;
  if (e < kHeadDim) {
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, sm_m[w]);
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float f = exp2f(sm_m[w] - M);  // empty warp: m = -inf -> 0
      L = fmaf(sm_l[w], f, L);
      O = fmaf(sm_o[w][e], f, O);
    }
  }
  uint16_t *out = a.out + (size_t)r * a.H * kHeadDim + h * kHeadDim;
  if (n_chunks == 1) {
    if (e < kHeadDim) out[e] = float_to_bf16_bits(O / L);
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
    out[e] = float_to_bf16_bits(OO / LL);
  }
  if (threadIdx.x == 0) a.tickets[(size_t)r * a.H + h] = 0u;  // ready for the next launch
}

inline cudaError_t launch_attention(const AttnArgs &a, int R, int max_tokens, cudaStream_t st) {
  int chunks = (max_tokens + kAttnWarps * kPageTokens - 1) / (kAttnWarps * kPageTokens);
  if (chunks < 1) chunks = 1;
  if (chunks > kAttnMaxChunks) chunks = kAttnMaxChunks;
  dim3 grid(chunks, a.H, R);
  attention_kernel<<<grid, kAttnWarps * 32, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace ttsgpt
