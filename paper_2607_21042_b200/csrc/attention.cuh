// Split-KV decode attention over 64-token pages (Section I: the decode engine's attention kernels
// and KV-cache management).
//
// KV pool, per layer: bf16 [n_pages][2 (K|V)][n_head][64 tokens][64]; each (page, K|V, head) block
// is 8 KB contiguous.
//
// Work split.  A (row, head) pair is handled by a thread-block cluster of S CTAs (S = 1, 2, 4 or 8,
// picked per launch so that the grid fills the GPU: S = 8 at batch 1, S = 1 at batch 128).  The
// row's pages are cut into quarter-page units of 16 tokens dealt round-robin over all 4*S warps of
// the cluster (with S = 1: whole pages over the CTA's 4 warps).  One warp streams 64 tokens of K and
// V at a time (a whole page, or four quarters) with 16+16 independent 128-bit loads per lane, keeps scores, the running softmax statistics
// (max, sum) and the running output in fp32 registers (online softmax across its pages), and uses
// shuffles for the reductions.  The warps of a CTA meet in shared memory; in a cluster every CTA
// stores its (max, sum, output) triple into rank 0's shared memory (distributed shared memory) and,
// after one cluster barrier, rank 0 merges them by log-sum-exp in rank order.  No global scratch, no atomics, no spinning; the
// result does not depend on timing.
//
// A second variant (`attention_ticket_kernel`) exchanges the partial results through global
// scratch and lets the CTA that arrives last at a ticket counter do the merge.  It needs no
// cluster launch and backs the stand-alone entry points.
#pragma once
#include <cooperative_groups.h>
#include "common.cuh"
#include "elementwise.cuh"

namespace ttsgpt {

namespace cg = cooperative_groups;

constexpr int kAttnWarps = 4;             // warps per CTA (pages in flight per CTA)
constexpr int kAttnMaxChunks = 8;         // ticket variant: 2048 tokens / 256
constexpr int kAttnPartialFloats = 66;    // m, l, o[64]
constexpr int kAttnMaxCluster = 8;

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
  float *partials;           // ticket variant: [R][H][kAttnMaxChunks][66]
  unsigned int *tickets;     // ticket variant: [R][H], zero between launches
  int H, pps;
  unsigned long long *trace;  // optional timeline trace
  int trace_slot;
  int out_image;             // 1: `out` is an activation image for the tensor-core linear (see act_image_offset)
  int old_pages_final;       // 1: one row per stream (decode step), pages before a row's last are not written by this step
  const int *row_order;      // streaming variant: grid slot z handles row row_order[z] (null: row z)
  int *err;                  // set to 1 if a bounded wait of the streaming variant expires (may be null)
};

// ------------------------------------------------------------------------------------------
// one page for one warp: scores, page-local softmax statistics, weighted values
// ------------------------------------------------------------------------------------------
struct PageLoad { uint4 kk[16], vv[16]; };

__device__ __forceinline__ void load_page(PageLoad &pl, const uint16_t *K, const uint16_t *V, int tg, int sub) {
#pragma unroll
  for (int i = 0; i < 16; ++i) pl.kk[i] = ld_stream_u4(K + (size_t)(tg + 4 * i) * kHeadDim + 8 * sub);
#pragma unroll
  for (int i = 0; i < 16; ++i) pl.vv[i] = ld_stream_u4(V + (size_t)(tg + 4 * i) * kHeadDim + 8 * sub);
}

// Folds the 16 token slots a lane holds into the warp's running (m, l, o).  Lane (tg, sub) =
// (lane/8, lane%8) holds elements 8*sub..8*sub+7 of 16 tokens (bit i of vmask: slot i is a real
// token); m and l are warp-uniform, o[e] is the lane's partial over its tokens (summed over tg at
// the very end).  At least one slot of the warp must be valid.
// first half: scores of NS slots (log2 units, -inf for slots without a token) and their maximum over the warp
template <int NS>
__device__ __forceinline__ float score_slots(const uint4 (&kk)[16], const float (&qv)[8], uint32_t vmask, float (&s)[16]) {
  float pm = -INFINITY;
#pragma unroll
  for (int i = 0; i < NS; ++i) {
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
    s[i] = ((vmask >> i) & 1u) ? d : -INFINITY;
    pm = fmaxf(pm, s[i]);
  }
  pm = fmaxf(pm, __shfl_xor_sync(0xFFFFFFFFu, pm, 8));
  pm = fmaxf(pm, __shfl_xor_sync(0xFFFFFFFFu, pm, 16));
  return pm;
}

// second half: rescale the running (m, l, o) to the new maximum and add the NS slots' weighted values
template <int NS>
__device__ __forceinline__ void accum_slots(uint4 (&vv)[16], const float (&s)[16], float pm, uint32_t vmask, float &m,
                                            float &l, float (&o)[8]) {
  const float m_new = fmaxf(m, pm);           // finite: the caller only folds batches with a valid token
  const float rescale = exp2f(m - m_new);     // first batch: exp2(-inf) = 0
  float lp = 0.f;
#pragma unroll
  for (int e = 0; e < 8; ++e) o[e] *= rescale;
#pragma unroll
  for (int i = 0; i < NS; ++i) {
    if (!((vmask >> i) & 1u)) vv[i] = make_uint4(0, 0, 0, 0);  // stale page contents may hold NaN: 0 * NaN must not reach o
    const float p = exp2f(s[i] - m_new);  // masked tokens: exp2(-inf) = 0
    lp += p;
    o[0] = fmaf(p, bf16_lo(vv[i].x), o[0]);
    o[1] = fmaf(p, bf16_hi(vv[i].x), o[1]);
    o[2] = fmaf(p, bf16_lo(vv[i].y), o[2]);
    o[3] = fmaf(p, bf16_hi(vv[i].y), o[3]);
    o[4] = fmaf(p, bf16_lo(vv[i].z), o[4]);
    o[5] = fmaf(p, bf16_hi(vv[i].z), o[5]);
    o[6] = fmaf(p, bf16_lo(vv[i].w), o[6]);
    o[7] = fmaf(p, bf16_hi(vv[i].w), o[7]);
  }
  lp += __shfl_xor_sync(0xFFFFFFFFu, lp, 8);
  lp += __shfl_xor_sync(0xFFFFFFFFu, lp, 16);
  l = l * rescale + lp;
  m = m_new;
}

template <int NS>
__device__ __forceinline__ void fold_first(PageLoad &pl, const float (&qv)[8], uint32_t vmask, float &m, float &l,
                                           float (&o)[8]) {
  float s[16];
  const float pm = score_slots<NS>(pl.kk, qv, vmask, s);
  accum_slots<NS>(pl.vv, s, pm, vmask, m, l, o);
}

// ng (warp-uniform): how many groups of 4 slots hold tokens at all; they are always the first ones,
// and the absent ones are not even looked at, which is what makes short batches cheap
__device__ __forceinline__ void fold_slots(PageLoad &pl, const float (&qv)[8], uint32_t vmask, int ng, float &m,
                                           float &l, float (&o)[8]) {
  if (ng >= 4) fold_first<16>(pl, qv, vmask, m, l, o);
  else if (ng == 3) fold_first<12>(pl, qv, vmask, m, l, o);
  else if (ng == 2) fold_first<8>(pl, qv, vmask, m, l, o);
  else fold_first<4>(pl, qv, vmask, m, l, o);
}

__device__ __forceinline__ void fold_page(PageLoad &pl, const float (&qv)[8], int n_here, int tg, float &m, float &l,
                                          float (&o)[8]) {
  uint32_t vmask = 0u;
#pragma unroll
  for (int i = 0; i < 16; ++i) vmask |= (tg + 4 * i < n_here) ? (1u << i) : 0u;
  fold_first<16>(pl, qv, vmask, m, l, o);
}

// Quarter-page batches for clusters: the row's pages are cut into units of 16 tokens, unit u =
// 4*page + quarter; a warp's batch holds 4 units u0, u0+stride, ... (slots 4j..4j+3 = unit j, tokens
// tg, tg+4, tg+8, tg+12 of the quarter), so that even a short context keeps every warp of every
// CTA of the cluster busy with 32 loads in flight.
__device__ __forceinline__ uint32_t load_quarters(PageLoad &pl, const uint16_t *kv_layer, const int *pt, int H, int h,
                                                  int u0, int stride, int n_units, int n_tok, int tg, int sub,
                                                  int &ng) {
  uint32_t vmask = 0u;
  ng = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int u = u0 + stride * j;
    if (u < n_units) {
      ng = j + 1;
      const int page = u >> 2, qt = u & 3;
      const int phys = pt[page];
      const uint16_t *K = kv_layer + (((size_t)phys * 2 + 0) * H + h) * kPageElems + (size_t)(16 * qt) * kHeadDim;
      const uint16_t *V = kv_layer + (((size_t)phys * 2 + 1) * H + h) * kPageElems + (size_t)(16 * qt) * kHeadDim;
      const int left = n_tok - page * kPageTokens - 16 * qt;   // tokens of the row from this quarter on
#pragma unroll
      for (int ii = 0; ii < 4; ++ii) {
        pl.kk[4 * j + ii] = ld_stream_u4(K + (size_t)(tg + 4 * ii) * kHeadDim + 8 * sub);
        pl.vv[4 * j + ii] = ld_stream_u4(V + (size_t)(tg + 4 * ii) * kHeadDim + 8 * sub);
        if (tg + 4 * ii < left) vmask |= 1u << (4 * j + ii);
      }
    } else {
#pragma unroll
      for (int ii = 0; ii < 4; ++ii) { pl.kk[4 * j + ii] = make_uint4(0, 0, 0, 0); pl.vv[4 * j + ii] = make_uint4(0, 0, 0, 0); }
    }
  }
  return vmask;
}

__device__ __forceinline__ void load_q(float (&qv)[8], const float *q) {
  // scores come out in log2 units: 1/sqrt(64) * log2(e)
  const float qs = 0.125f * 1.4426950408889634f;
  const float4 q0 = *reinterpret_cast<const float4 *>(q);
  const float4 q1 = *reinterpret_cast<const float4 *>(q + 4);
  qv[0] = q0.x * qs; qv[1] = q0.y * qs; qv[2] = q0.z * qs; qv[3] = q0.w * qs;
  qv[4] = q1.x * qs; qv[5] = q1.y * qs; qv[6] = q1.z * qs; qv[7] = q1.w * qs;
}

// warp result -> shared memory; then threads 0..63 merge the CTA's warps in warp order
__device__ __forceinline__ void cta_merge(float m, float l, float (&o)[8], int warp, int tg, int sub,
                                          float (&sm_m)[kAttnWarps], float (&sm_l)[kAttnWarps],
                                          float (&sm_o)[kAttnWarps][kHeadDim], float &M, float &L, float &O) {
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 8);
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 16);
  }
  if (tg == 0) {
    if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
#pragma unroll
    for (int e = 0; e < 8; ++e) sm_o[warp][8 * sub + e] = o[e];
  }
  __syncthreads();
  M = -INFINITY; L = 0.f; O = 0.f;
  const int e = threadIdx.x;
  if (e < kHeadDim) {
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, sm_m[w]);
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float f = (sm_m[w] == -INFINITY) ? 0.f : exp2f(sm_m[w] - M);  // idle warp contributes nothing
      L = fmaf(sm_l[w], f, L);
      O = fmaf(sm_o[w][e], f, O);
    }
  }
}

// ------------------------------------------------------------------------------------------
// cluster variant (the engine's path)
// ------------------------------------------------------------------------------------------
// CLUSTER = false: gridDim.x == 1, one CTA per (row, head); the two variants are separate kernels so
// that each carries only its own code (these kernels run for a few microseconds and mostly execute
// every instruction once: instruction fetch shows up in their stall reasons)
template <bool CLUSTER>
__global__ void __launch_bounds__(kAttnWarps * 32) attention_kernel(const AttnArgs a) {
  const int S = CLUSTER ? gridDim.x : 1, c = blockIdx.x, h = blockIdx.y, r = blockIdx.z;
  trace_mark(a.trace, a.trace_slot, 0);
  // The row table and page table were written before the first kernel of the step started, so
  // they may be read ahead of the dependency wait.
  const int n_tok = a.row_pos[r] + 1;
  const int n_pages = (n_tok + kPageTokens - 1) / kPageTokens;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tg = lane >> 3, sub = lane & 7;
  const int *pt = a.page_table + (size_t)a.row_stream[r] * a.pps;

  __shared__ float sm_m[kAttnWarps], sm_l[kAttnWarps], sm_o[kAttnWarps][kHeadDim];
  __shared__ float cl_all[kAttnMaxCluster][kAttnPartialFloats];  // rank 0: every rank's (M, L, O[64])

  float m = -INFINITY, l = 0.f;
  float o[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) o[e] = 0.f;
  float qv[8];
  PageLoad pl;
  // In a decode step the only K/V entry of the row that this step writes is the new token's own
  // (position n_tok-1, by the QKV kernel in front).  The warp's first batch of loads is therefore
  // requested before waiting for that kernel; if it covers the new token, that token's 128-byte K
  // and V rows are fetched again after the wait.
  const int tn = (n_tok - 1) & (kPageTokens - 1);   // the new token's slot in the last page
  if (CLUSTER) {
    // ---- cluster: quarter-page units dealt round-robin over all warps of the cluster ----
    const int GW = S * kAttnWarps, gw = c * kAttnWarps + warp;
    const int n_units = (n_tok + 15) >> 4;   // units that hold at least one token
    const bool early = a.old_pages_final && gw < n_units;
    uint32_t vmask = 0u;
    int ng = 0;
    if (early) vmask = load_quarters(pl, a.kv_layer, pt, a.H, h, gw, GW, n_units, n_tok, tg, sub, ng);
    pdl_launch_dependents();
    pdl_wait();
    trace_mark(a.trace, a.trace_slot, 1);
    load_q(qv, a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim + 8 * sub);
    if (early) {
      const int us = 4 * (n_pages - 1) + (tn >> 4);   // unit of the new token
      if (us % GW == gw && us / GW < 4 && (tn & 3) == tg) {
        const int phys = pt[n_pages - 1];
        const uint4 kn = ld_cg_u4(a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kPageElems + (size_t)tn * kHeadDim + 8 * sub);
        const uint4 vn = ld_cg_u4(a.kv_layer + (((size_t)phys * 2 + 1) * a.H + h) * kPageElems + (size_t)tn * kHeadDim + 8 * sub);
        const int sel = 4 * (us / GW) + ((tn & 15) >> 2);
#pragma unroll
        for (int i = 0; i < 16; ++i) {  // register selects (no dynamic indexing of the page registers)
          const bool hit = i == sel;
          pl.kk[i].x = hit ? kn.x : pl.kk[i].x; pl.kk[i].y = hit ? kn.y : pl.kk[i].y;
          pl.kk[i].z = hit ? kn.z : pl.kk[i].z; pl.kk[i].w = hit ? kn.w : pl.kk[i].w;
          pl.vv[i].x = hit ? vn.x : pl.vv[i].x; pl.vv[i].y = hit ? vn.y : pl.vv[i].y;
          pl.vv[i].z = hit ? vn.z : pl.vv[i].z; pl.vv[i].w = hit ? vn.w : pl.vv[i].w;
        }
      }
    }
    bool loaded = early;
    for (int u0 = gw; u0 < n_units; u0 += 4 * GW) {
      if (!loaded) vmask = load_quarters(pl, a.kv_layer, pt, a.H, h, u0, GW, n_units, n_tok, tg, sub, ng);
      loaded = false;
      fold_slots(pl, qv, vmask, ng, m, l, o);
    }
  } else {
    // ---- one CTA per (row, head): whole pages, warp w takes pages w, w+4, ... ----
    int page = warp;
    const bool early = a.old_pages_final && page < n_pages;
    const uint16_t *K0 = nullptr, *V0 = nullptr;
    if (early) {
      const int phys = pt[page];
      K0 = a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kPageElems;
      V0 = a.kv_layer + (((size_t)phys * 2 + 1) * a.H + h) * kPageElems;
      load_page(pl, K0, V0, tg, sub);
    }
    pdl_launch_dependents();
    pdl_wait();
    trace_mark(a.trace, a.trace_slot, 1);
    load_q(qv, a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim + 8 * sub);
    if (early && page == n_pages - 1 && (tn & 3) == tg) {
      const uint4 kn = ld_cg_u4(K0 + (size_t)tn * kHeadDim + 8 * sub);
      const uint4 vn = ld_cg_u4(V0 + (size_t)tn * kHeadDim + 8 * sub);
      const int sel = tn >> 2;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const bool hit = i == sel;
        pl.kk[i].x = hit ? kn.x : pl.kk[i].x; pl.kk[i].y = hit ? kn.y : pl.kk[i].y;
        pl.kk[i].z = hit ? kn.z : pl.kk[i].z; pl.kk[i].w = hit ? kn.w : pl.kk[i].w;
        pl.vv[i].x = hit ? vn.x : pl.vv[i].x; pl.vv[i].y = hit ? vn.y : pl.vv[i].y;
        pl.vv[i].z = hit ? vn.z : pl.vv[i].z; pl.vv[i].w = hit ? vn.w : pl.vv[i].w;
      }
    }
    bool loaded = early;
    for (; page < n_pages; page += kAttnWarps) {
      if (!loaded) {
        const int phys = pt[page];
        load_page(pl, a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kPageElems,
                  a.kv_layer + (((size_t)phys * 2 + 1) * a.H + h) * kPageElems, tg, sub);
      }
      loaded = false;
      fold_page(pl, qv, min(kPageTokens, n_tok - page * kPageTokens), tg, m, l, o);
    }
  }
  trace_mark(a.trace, a.trace_slot, 3);
  const int e = threadIdx.x;
  // plain row-major bf16, or the image layout of the tensor-core linear that consumes it
  uint16_t *out = nullptr;
  if (e < kHeadDim)
    out = a.out_image ? reinterpret_cast<uint16_t *>(reinterpret_cast<unsigned char *>(a.out) + act_image_offset_tiled(r, h * kHeadDim + e, a.H * kHeadDim))
                      : a.out + (size_t)r * a.H * kHeadDim + h * kHeadDim + e;
  if (!CLUSTER) {
    float M, L, O;
    cta_merge(m, l, o, warp, tg, sub, sm_m, sm_l, sm_o, M, L, O);
    if (e < kHeadDim) *out = float_to_bf16_bits(O / L);
    trace_mark(a.trace, a.trace_slot, 2);
    return;
  }
  // ---- cluster merge: the CTA merges its warps locally, stores its (M, L, O[64]) straight into
  //      rank 0's shared memory (distributed shared memory), one cluster barrier, then rank 0 merges
  //      the S partial results in rank order; the other ranks are done once the barrier is passed ----
  cg::cluster_group cluster = cg::this_cluster();
  float M, L, O;
  cta_merge(m, l, o, warp, tg, sub, sm_m, sm_l, sm_o, M, L, O);
  if (e < kHeadDim) {
    float *dst = cluster.map_shared_rank(&cl_all[0][0], 0) + (size_t)c * kAttnPartialFloats;
    if (e == 0) { dst[0] = M; dst[1] = L; }
    dst[2 + e] = O;
  }
  trace_mark(a.trace, a.trace_slot, 4);
  cluster.sync();
  trace_mark(a.trace, a.trace_slot, 5);
  if (c == 0 && e < kHeadDim) {
    float pm[kAttnMaxCluster], pl_[kAttnMaxCluster], po[kAttnMaxCluster];
#pragma unroll
    for (int rr = 0; rr < kAttnMaxCluster; ++rr) {   // all reads issued before any is used
      pm[rr] = -INFINITY; pl_[rr] = 0.f; po[rr] = 0.f;
      if (rr < S) { pm[rr] = cl_all[rr][0]; pl_[rr] = cl_all[rr][1]; po[rr] = cl_all[rr][2 + e]; }
    }
    float MM = -INFINITY;
#pragma unroll
    for (int rr = 0; rr < kAttnMaxCluster; ++rr) MM = fmaxf(MM, pm[rr]);
    float LL = 0.f, OO = 0.f;
#pragma unroll
    for (int rr = 0; rr < kAttnMaxCluster; ++rr) {
      const float f = (pm[rr] == -INFINITY) ? 0.f : exp2f(pm[rr] - MM);  // a rank without tokens contributes nothing
      LL = fmaf(pl_[rr], f, LL);
      OO = fmaf(po[rr], f, OO);
    }
    *out = float_to_bf16_bits(OO / LL);
  }
  trace_mark(a.trace, a.trace_slot, 2);
}

// Cluster size for R rows of H heads on n_sm SMs: enough CTAs to cover the GPU about once.
inline int attention_cluster_size(int R, int H, int n_sm, int fill = 1) {
  int s = 1;
  while (s < kAttnMaxCluster && R * H * s < fill * n_sm) s *= 2;
  return s;
}

inline cudaError_t launch_attention(const AttnArgs &a, int R, int cluster, cudaStream_t st, bool pdl) {
  cudaLaunchConfig_t cfg;
  cfg.gridDim = dim3(cluster, a.H, R);
  cfg.blockDim = dim3(kAttnWarps * 32);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  int n = 0;
  if (cluster > 1) {
    at[n].id = cudaLaunchAttributeClusterDimension;
    at[n].val.clusterDim.x = cluster; at[n].val.clusterDim.y = 1; at[n].val.clusterDim.z = 1;
    ++n;
  }
  if (pdl) {
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = at;
  cfg.numAttrs = n;
  if (cluster > 1) return cudaLaunchKernelEx(&cfg, attention_kernel<true>, a);
  return cudaLaunchKernelEx(&cfg, attention_kernel<false>, a);
}

// ------------------------------------------------------------------------------------------
// streaming variant (the engine's path once there are enough (row, head) pairs to fill the GPU
// several times): one CTA per (row, head), warp w takes pages w, w+4, ...  A page's K and V blocks
// (8 KB each, contiguous in the pool) come in by two bulk asynchronous copies into the warp's own
// 16 KB stage of shared memory; as soon as the warp has pulled the stage into registers, lane 0
// requests the warp's next page into the same stage, so that the copy runs under the arithmetic
// of the current page and every resident warp keeps 16 KB in flight with no registers tied up by
// outstanding loads.  Only the tokens that exist are copied from a partial last page.
// ------------------------------------------------------------------------------------------
constexpr uint32_t kAttnHalfStage = kPageElems * 2;          // one K or V block: 8 KB
constexpr uint32_t kAttnStageBytes = 2 * kAttnHalfStage;
constexpr unsigned long long kAttnWaitNs = 2000000000ull;

__device__ __forceinline__ void stream_issue(const AttnArgs &a, const int *pt, int h, int page, int n_tok,
                                             unsigned char *stage, uint64_t *bar) {
  const int n_here = min(kPageTokens, n_tok - page * kPageTokens);
  const uint32_t bytes = (uint32_t)n_here * kHeadDim * 2;
  const int phys = pt[page];
  const uint16_t *K = a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kPageElems;
  const uint16_t *V = a.kv_layer + (((size_t)phys * 2 + 1) * a.H + h) * kPageElems;
  mbar_expect_tx(bar, 2 * bytes);
  bulk_copy_g2s(stage, K, bytes, bar);
  bulk_copy_g2s(stage + kAttnHalfStage, V, bytes, bar);
}

__global__ void __launch_bounds__(kAttnWarps * 32, 3) attention_stream_kernel(const AttnArgs a) {
  extern __shared__ __align__(128) unsigned char attn_stages[];   // [warp][K 8 KB | V 8 KB]
  __shared__ __align__(8) uint64_t bars[kAttnWarps];
  __shared__ float sm_m[kAttnWarps], sm_l[kAttnWarps], sm_o[kAttnWarps][kHeadDim];
  const int h = blockIdx.y, r = a.row_order ? a.row_order[blockIdx.z] : blockIdx.z;
  trace_mark(a.trace, a.trace_slot, 0);
  const int n_tok = a.row_pos[r] + 1;   // row and page tables are final before the step's first kernel starts
  const int n_pages = (n_tok + kPageTokens - 1) / kPageTokens;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tg = lane >> 3, sub = lane & 7;
  const int *pt = a.page_table + (size_t)a.row_stream[r] * a.pps;
  unsigned char *stage = attn_stages + (size_t)warp * kAttnStageBytes;
  uint64_t *bar = bars + warp;

  float m = -INFINITY, l = 0.f;
  float o[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) o[e] = 0.f;
  float qv[8];
  const int tn = (n_tok - 1) & (kPageTokens - 1);   // the new token's slot in the last page
  int page = warp;
  // In a decode step only the new token's own K/V rows are written by the kernel in front, so the
  // warp's first page is requested ahead of the dependency wait and those two rows are read again
  // afterwards if the page holds them.
  const bool early = a.old_pages_final && page < n_pages;
  if (lane == 0) {
    mbar_init(bar, 1);
    if (early) stream_issue(a, pt, h, page, n_tok, stage, bar);
  }
  __syncwarp();
  pdl_launch_dependents();
  pdl_wait();
  trace_mark(a.trace, a.trace_slot, 1);
  load_q(qv, a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim + 8 * sub);
  if (!early && page < n_pages && lane == 0) stream_issue(a, pt, h, page, n_tok, stage, bar);
  uint32_t phase = 0;
  bool first = true;
  for (; page < n_pages; page += kAttnWarps) {
    if (!mbar_wait_bounded(bar, phase, kAttnWaitNs)) {
      if (a.err) atomicExch(a.err, 1);
      mbar_wait_bounded(bar, phase, kAttnWaitNs);   // a last chance for the copy in flight towards this CTA
      break;
    }
    phase ^= 1u;
    const int n_here = min(kPageTokens, n_tok - page * kPageTokens);
    uint32_t vmask = 0u;
#pragma unroll
    for (int i = 0; i < 16; ++i) vmask |= (tg + 4 * i < n_here) ? (1u << i) : 0u;
    // the new token's rows, if this page was copied before the kernel in front had written them
    const bool patch = first && early && page == n_pages - 1 && (tn & 3) == tg;
    const int sel = tn >> 2;
    uint4 kn = make_uint4(0, 0, 0, 0), vn = kn;
    if (patch) {
      const int phys = pt[page];
      kn = ld_cg_u4(a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kPageElems + (size_t)tn * kHeadDim + 8 * sub);
      vn = ld_cg_u4(a.kv_layer + (((size_t)phys * 2 + 1) * a.H + h) * kPageElems + (size_t)tn * kHeadDim + 8 * sub);
    }
    first = false;
    uint4 kk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      kk[i] = *reinterpret_cast<const uint4 *>(stage + (size_t)(tg + 4 * i) * (kHeadDim * 2) + 16 * sub);
      if (patch && i == sel) kk[i] = kn;
    }
    float s[16];
    const float pm = score_slots<16>(kk, qv, vmask, s);
    uint4 vv[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      vv[i] = *reinterpret_cast<const uint4 *>(stage + kAttnHalfStage + (size_t)(tg + 4 * i) * (kHeadDim * 2) + 16 * sub);
      if (patch && i == sel) vv[i] = vn;
    }
    // The stage may be overwritten only after every read of it has returned: the K reads have (the
    // scores consumed them); one word of every V read is folded into a value that the fence below
    // takes as an operand, so the copy cannot be issued ahead of those reads either.
    uint32_t seen = 0u;
#pragma unroll
    for (int i = 0; i < 16; ++i) seen ^= vv[i].x;
    __syncwarp();   // every lane has read the stage
    if (page + kAttnWarps < n_pages && lane == 0) {
      asm volatile("fence.proxy.async.shared::cta; // after %0" ::"r"(seen) : "memory");
      stream_issue(a, pt, h, page + kAttnWarps, n_tok, stage, bar);
    }
    accum_slots<16>(vv, s, pm, vmask, m, l, o);
  }
  trace_mark(a.trace, a.trace_slot, 3);
  const int e = threadIdx.x;
  float M, L, O;
  cta_merge(m, l, o, warp, tg, sub, sm_m, sm_l, sm_o, M, L, O);
  if (e < kHeadDim) {
    uint16_t *out = a.out_image ? reinterpret_cast<uint16_t *>(reinterpret_cast<unsigned char *>(a.out) + act_image_offset_tiled(r, h * kHeadDim + e, a.H * kHeadDim))
                                : a.out + (size_t)r * a.H * kHeadDim + h * kHeadDim + e;
    *out = float_to_bf16_bits(O / L);
  }
  trace_mark(a.trace, a.trace_slot, 2);
}

// (row, head) pairs from which the streaming variant is used: the GPU is then covered four times
// over with one CTA per pair (at 16 rows of 20 heads the cluster variant still measured faster)
inline bool attention_use_stream(int R, int H, int n_sm) { return R * H >= 4 * n_sm; }

inline cudaError_t launch_attention_stream(const AttnArgs &a, int R, cudaStream_t st, bool pdl) {
  static PerDeviceOnce attr_once;   // per device: opt-in to more than 48 KB of dynamic shared memory
  const size_t smem = (size_t)kAttnWarps * kAttnStageBytes;
  if (attr_once.first()) {
    cudaFuncSetAttribute(attention_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  }
  return launch_kernel(attention_stream_kernel, dim3(1, a.H, R), dim3(kAttnWarps * 32), smem, st, pdl, a);
}

// ------------------------------------------------------------------------------------------
// prefill variant: the rows of a prefill pass are consecutive positions of a few streams, so rows
// of one stream read the same K/V pages.  A CTA takes 8 consecutive rows of the pass for one head,
// one row per warp; it walks the pages of each stream its rows belong to (rows of a pass are
// stream-major, so a CTA's rows split into at most 8 runs of one stream each), brings a page's K and
// V blocks into shared memory once by bulk asynchronous copies, and every warp whose row belongs
// to that stream and reaches into that page folds it into its own running softmax.  The page
// traffic from L2 drops eightfold against one CTA per row; no merge between warps is needed.
// ------------------------------------------------------------------------------------------
constexpr int kAttnPrefillRows = 8;     // rows (= warps) per CTA
constexpr int kAttnPrefillStages = 4;   // pages in flight or in use per CTA (a ring of 16 KB stages)

// one half page (32 tokens: slots 0..7 of every lane) from a stage into the warp's running softmax
__device__ __forceinline__ void prefill_fold_half(const unsigned char *stage, int half, int n_mine, int tg, int sub,
                                                  const float (&qv)[8], float &m, float &l, float (&o)[8]) {
  uint32_t vmask = 0u;
#pragma unroll
  for (int i = 0; i < 8; ++i) vmask |= (32 * half + tg + 4 * i < n_mine) ? (1u << i) : 0u;
  const unsigned char *base = stage + (size_t)(32 * half + tg) * (kHeadDim * 2) + 16 * sub;
  uint4 kk[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) kk[i] = *reinterpret_cast<const uint4 *>(base + (size_t)(4 * i) * (kHeadDim * 2));
  float sc[16];
  const float pm = score_slots<8>(kk, qv, vmask, sc);
  uint4 vv[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) vv[i] = *reinterpret_cast<const uint4 *>(base + kAttnHalfStage + (size_t)(4 * i) * (kHeadDim * 2));
  accum_slots<8>(vv, sc, pm, vmask, m, l, o);
}

__global__ void __launch_bounds__(kAttnPrefillRows * 32, 3) attention_prefill_kernel(const AttnArgs a, int R) {
  extern __shared__ __align__(128) unsigned char prefill_stages[];   // [stage][K 8 KB | V 8 KB]
  __shared__ __align__(8) uint64_t bars[kAttnPrefillStages];
  __shared__ int seg_stream[kAttnPrefillRows], seg_i0[kAttnPrefillRows], seg_i1[kAttnPrefillRows], seg_last[kAttnPrefillRows];
  __shared__ int n_seg_s;
  const int h = blockIdx.y, r0 = blockIdx.z * kAttnPrefillRows;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tg = lane >> 3, sub = lane & 7;
  const int r = r0 + warp;
  const bool have_row = r < R;
  trace_mark(a.trace, a.trace_slot, 0);
  if (threadIdx.x == 0) {
    for (int i = 0; i < kAttnPrefillStages; ++i) mbar_init(bars + i, 1);
    // runs of rows of one stream (the row table is final before the pass's first kernel starts)
    const int r_end = min(R, r0 + kAttnPrefillRows);
    int n = 0, i0 = r0;
    while (i0 < r_end) {
      const int s = a.row_stream[i0];
      int i1 = i0 + 1;
      while (i1 < r_end && a.row_stream[i1] == s) ++i1;
      seg_stream[n] = s; seg_i0[n] = i0; seg_i1[n] = i1; seg_last[n] = a.row_pos[i1 - 1];
      ++n; i0 = i1;
    }
    n_seg_s = n;
  }
  __syncthreads();
  pdl_launch_dependents();
  pdl_wait();     // the K/V rows of this pass were written by the QKV kernel in front: nothing is read before
  trace_mark(a.trace, a.trace_slot, 1);
  const int n_seg = n_seg_s;
  const int my_pos = have_row ? a.row_pos[r] : -1;
  float m = -INFINITY, l = 0.f;
  float o[8], qv[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) { o[e] = 0.f; qv[e] = 0.f; }
  if (have_row) load_q(qv, a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim + 8 * sub);

  // page jobs in order: for each run, pages 0 .. last_pos/64.  Thread 0 keeps kAttnPrefillStages - 1
  // jobs requested ahead of the one the warps fold.
  int iseg = 0, ip = 0;          // thread 0: the next job to request
  auto issue_next = [&](int slot) {
    if (iseg >= n_seg) return;
    const int last_pos = seg_last[iseg];
    const int n_here = min(kPageTokens, last_pos + 1 - ip * kPageTokens);
    const uint32_t bytes = (uint32_t)n_here * kHeadDim * 2;
    const int phys = a.page_table[(size_t)seg_stream[iseg] * a.pps + ip];
    const uint16_t *K = a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kPageElems;
    unsigned char *stage = prefill_stages + (size_t)slot * kAttnStageBytes;
    mbar_expect_tx(bars + slot, 2 * bytes);
    bulk_copy_g2s(stage, K, bytes, bars + slot);
    bulk_copy_g2s(stage + kAttnHalfStage, K + (size_t)a.H * kPageElems, bytes, bars + slot);
    if (++ip > last_pos / kPageTokens) { ++iseg; ip = 0; }
  };
  if (threadIdx.x == 0)
    for (int i = 0; i < kAttnPrefillStages - 1; ++i) issue_next(i);
  bool dead = false;   // a copy did not arrive in time: stop folding, keep walking the barriers
  int j = 0;
  for (int seg = 0; seg < n_seg; ++seg) {
    const int n_pages = seg_last[seg] / kPageTokens + 1;
    const bool mine = have_row && r >= seg_i0[seg] && r < seg_i1[seg];
    for (int p = 0; p < n_pages; ++p, ++j) {
      const int slot = j % kAttnPrefillStages;
      // the stage job j-1 used is free since the barrier that ended its iteration
      if (threadIdx.x == 0) issue_next((j + kAttnPrefillStages - 1) % kAttnPrefillStages);
      const uint32_t parity = (uint32_t)(j / kAttnPrefillStages) & 1u;
      if (!dead && !mbar_wait_bounded(bars + slot, parity, kAttnWaitNs)) {
        if (a.err) atomicExch(a.err, 1);
        mbar_wait_bounded(bars + slot, parity, kAttnWaitNs);   // a last chance for the copy in flight
        dead = true;
      }
      const unsigned char *stage = prefill_stages + (size_t)slot * kAttnStageBytes;
      const int n_mine = mine ? min(kPageTokens, my_pos + 1 - p * kPageTokens) : 0;   // tokens of this page the row sees
      if (!dead && n_mine > 0) {   // warp-uniform
        prefill_fold_half(stage, 0, n_mine, tg, sub, qv, m, l, o);
        if (n_mine > 32) prefill_fold_half(stage, 1, n_mine, tg, sub, qv, m, l, o);
      }
      __syncthreads();   // every warp is done with this stage (all reads consumed): it may be refilled
      if (threadIdx.x == 0) fence_proxy_async_smem();
    }
  }
  trace_mark(a.trace, a.trace_slot, 3);
  // the warp's result: sum the partial outputs over the 4 token groups, then lanes tg == 0 write 8 values each
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 8);
    o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 16);
  }
  if (have_row && tg == 0 && !dead) {
    const float inv = 1.0f / l;
    const uint4 y = make_uint4(pack_bf16x2(o[0] * inv, o[1] * inv), pack_bf16x2(o[2] * inv, o[3] * inv),
                               pack_bf16x2(o[4] * inv, o[5] * inv), pack_bf16x2(o[6] * inv, o[7] * inv));
    const int col = h * kHeadDim + 8 * sub;
    if (a.out_image) *reinterpret_cast<uint4 *>(reinterpret_cast<unsigned char *>(a.out) + act_image_offset_tiled(r, col, a.H * kHeadDim)) = y;
    else *reinterpret_cast<uint4 *>(a.out + (size_t)r * a.H * kHeadDim + col) = y;
  }
  trace_mark(a.trace, a.trace_slot, 2);
}

inline cudaError_t launch_attention_prefill(const AttnArgs &a, int R, cudaStream_t st, bool pdl) {
  static PerDeviceOnce attr_once;   // per device: opt-in to more than 48 KB of dynamic shared memory
  const size_t smem = (size_t)kAttnPrefillStages * kAttnStageBytes;
  if (attr_once.first()) {
    cudaFuncSetAttribute(attention_prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  }
  const int groups = (R + kAttnPrefillRows - 1) / kAttnPrefillRows;
  return launch_kernel(attention_prefill_kernel, dim3(1, a.H, groups), dim3(kAttnPrefillRows * 32), smem, st, pdl, a, R);
}

// ------------------------------------------------------------------------------------------
// ticket variant: chunks of 4 pages per CTA, partial results through global scratch, merged by
// the CTA that arrives last at the row's ticket counter (no spinning)
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kAttnWarps * 32) attention_ticket_kernel(const AttnArgs a) {
  const int c = blockIdx.x, h = blockIdx.y, r = blockIdx.z;
  // a position beyond the stream's page table (the caller's mistake) is cut to what the table and the grid
  // cover: every chunk then exists, so the ticket completes, the row is written and the ticket returns to zero
  const int n_tok = min(min(a.row_pos[r] + 1, a.pps * kPageTokens), (int)gridDim.x * kAttnWarps * kPageTokens);
  const int n_pages = (n_tok + kPageTokens - 1) / kPageTokens;
  const int n_chunks = (n_pages + kAttnWarps - 1) / kAttnWarps;
  if (c >= n_chunks) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tg = lane >> 3, sub = lane & 7;
  const int page = c * kAttnWarps + warp;

  __shared__ float sm_m[kAttnWarps], sm_l[kAttnWarps], sm_o[kAttnWarps][kHeadDim];
  __shared__ unsigned int sm_ticket;

  float m = -INFINITY, l = 0.f;
  float o[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) o[e] = 0.f;
  if (page < n_pages) {
    const int phys = a.page_table[(size_t)a.row_stream[r] * a.pps + page];
    PageLoad pl;
    load_page(pl, a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kPageElems,
              a.kv_layer + (((size_t)phys * 2 + 1) * a.H + h) * kPageElems, tg, sub);
    float qv[8];
    load_q(qv, a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim + 8 * sub);
    fold_page(pl, qv, min(kPageTokens, n_tok - page * kPageTokens), tg, m, l, o);
  }
  float M, L, O;
  cta_merge(m, l, o, warp, tg, sub, sm_m, sm_l, sm_o, M, L, O);
  const int e = threadIdx.x;
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

inline cudaError_t launch_attention_ticket(const AttnArgs &a, int R, int max_tokens, cudaStream_t st) {
  int chunks = (max_tokens + kAttnWarps * kPageTokens - 1) / (kAttnWarps * kPageTokens);
  if (chunks < 1) chunks = 1;
  if (chunks > kAttnMaxChunks) chunks = kAttnMaxChunks;
  attention_ticket_kernel<<<dim3(chunks, a.H, R), kAttnWarps * 32, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace ttsgpt
