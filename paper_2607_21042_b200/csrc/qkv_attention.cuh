// Batch-1 decode: LayerNorm + QKV projection + split-KV attention in ONE kernel (Sections I, II-C:
// the per-token step of the decode engine is a chain of small kernels, and at one row per step the
// chain, not the memory system, bounds it; this removes one link per layer).
//
// The grid is the attention kernel's: a thread-block cluster of 8 CTAs per head.  The head's 192
// rows of the QKV matrix (64 each of Q, K, V) are 24 row tiles of the streaming layout, 3 per CTA
// (tile c of Q, of K and of V for cluster rank c).  A CTA
//   1. before waiting for the kernel in front: requests its 3 tile rows by bulk asynchronous copies,
//      loads LayerNorm gamma/beta, bias and scales, and requests its share of the row's old K/V
//      units (quarter pages, dealt over the 32 warps of the cluster) into registers;
//   2. after the wait: layer-normalises the fp32 residual row (two block reductions: mean, then the
//      centred sum of squares), rounds it to bf16 into shared memory, multiplies its 24 weight rows
//      with it (fp32 FMAs on the exactly widened weights, K split over the 4 warps, partial sums
//      met in warp order), adds scale and bias;
//   3. stores its 8 values of q (fp32) and of the new token's K and V (rounded to bf16, as the
//      cache holds them) into every rank's shared memory (distributed shared memory), writes K and
//      V to the page in global memory, and passes a cluster barrier;
//   4. runs the attention of the cluster variant on its units, with q and the new token's K/V
//      taken from shared memory, and merges through rank 0 as that kernel does.
// No global scratch, no atomics, no spinning other than the bounded wait for the weight copy.
#pragma once
#include "attention.cuh"
#include "linear.cuh"

namespace ttsgpt {

constexpr int kQaCluster = 8;
constexpr int kQaThreads = kAttnWarps * 32;
constexpr int kQaMaxK = 2048;                 // d_model limit of the fused kernel
constexpr int kQaLnRounds = kQaMaxK / (4 * kQaThreads);   // float4 chunks per thread

struct QkvAttnArgs {
  const void *w;            // tiled QKV weights [3d, d]
  const uint16_t *scales;   // tiled scales or null
  const uint16_t *bias;     // bf16 [3d]
  const float *x;           // fp32 residual rows [R][d]
  const uint16_t *ln_g, *ln_b;
  float ln_eps;
  int d;
  AttnArgs at;              // q, partials, tickets, row_order unused; old_pages_final must be 1
};

inline size_t qkv_attn_smem_bytes(int wf, int d) {
  const int KB = d / k_per_tile(wf);
  return 128 + (size_t)3 * KB * (wf == WF_INT4 ? 528 : 512) + (size_t)d * 2;
}

__device__ __forceinline__ float qa_block_sum(float v, float *sm, int warp, int lane) {
  v = warp_sum(v);
  __syncthreads();            // sm may still be read from the previous reduction
  if (lane == 0) sm[warp] = v;
  __syncthreads();
  return (sm[0] + sm[1]) + (sm[2] + sm[3]);
}

template <int WF>
__global__ void __launch_bounds__(kQaThreads) qkv_attention_kernel(const QkvAttnArgs a) {
  constexpr int KT = WF == WF_BF16 ? 32 : (WF == WF_INT8 ? 64 : 128);
  constexpr int AW = KT / 32;
  const AttnArgs &at = a.at;
  const int c = blockIdx.x, h = blockIdx.y, r = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = a.d, KB = K / KT;
  trace_mark(at.trace, at.trace_slot, 0);

  extern __shared__ __align__(128) unsigned char qa_smem[];
  uint64_t *wbar = reinterpret_cast<uint64_t *>(qa_smem);
  unsigned char *wsm = qa_smem + 128;                                                  // [3][KB] tiles of 512 B
  uint16_t *ssm = reinterpret_cast<uint16_t *>(wsm + (size_t)3 * KB * 512);            // int4: [3][KB][8] scales
  uint16_t *xs = reinterpret_cast<uint16_t *>(wsm + (size_t)3 * KB * (WF == WF_INT4 ? 528 : 512));   // LN row, bf16 [K]
  __shared__ float red[kAttnWarps][24];
  __shared__ float lnred[kAttnWarps];
  __shared__ __align__(16) float q_sh[kHeadDim];
  __shared__ __align__(16) uint16_t kn_sh[kHeadDim], vn_sh[kHeadDim];
  __shared__ float sm_m[kAttnWarps], sm_l[kAttnWarps], sm_o[kAttnWarps][kHeadDim];
  __shared__ float cl_all[kAttnMaxCluster][kAttnPartialFloats];

  // ---- 1. everything that does not depend on the kernel in front ----
  const int rt_per = K / 8;            // row tiles per 1280-row block of Q, K or V (d rows each)
  if (threadIdx.x == 0) {
    const uint32_t tb = (uint32_t)KB * 512u, sb = WF == WF_INT4 ? (uint32_t)KB * 16u : 0u;
    mbar_init(wbar, 1);
    mbar_expect_tx(wbar, 3 * (tb + sb));
    for (int j = 0; j < 3; ++j) {
      const size_t tile = (size_t)j * rt_per + (size_t)h * 8 + c;
      const unsigned char *gw = reinterpret_cast<const unsigned char *>(a.w) + tile * KB * 512;
      for (uint32_t off = 0; off < tb; off += 32768u)
        bulk_copy_g2s(wsm + (size_t)j * tb + off, gw + off, min(32768u, tb - off), wbar);
      if (sb) bulk_copy_g2s(ssm + (size_t)j * KB * 8, a.scales + tile * KB * 8, sb, wbar);
    }
  }
  cg::cluster_group cluster = cg::this_cluster();
  cluster.barrier_arrive();            // completed (barrier_wait below) before the first remote store: every CTA of the cluster runs
  uint2 ln_gg[kQaLnRounds], ln_bb[kQaLnRounds];
#pragma unroll
  for (int i = 0; i < kQaLnRounds; ++i) {
    const int lc = 4 * (threadIdx.x + kQaThreads * i);
    ln_gg[i] = make_uint2(0, 0); ln_bb[i] = make_uint2(0, 0);
    if (lc < K) {
      ln_gg[i] = *reinterpret_cast<const uint2 *>(a.ln_g + lc);
      ln_bb[i] = *reinterpret_cast<const uint2 *>(a.ln_b + lc);
    }
  }
  // epilogue threads 0..23: output j = tid / 8 (0 Q, 1 K, 2 V), element 8c + tid % 8 of the head
  const int ej = threadIdx.x >> 3, eg = threadIdx.x & 7;
  const int n_tok = at.row_pos[r] + 1;          // row and page tables are final before the step's first kernel starts
  const int n_pages = (n_tok + kPageTokens - 1) / kPageTokens;
  const int tn = (n_tok - 1) & (kPageTokens - 1);   // the new token's slot in the last page
  const int *pt = at.page_table + (size_t)at.row_stream[r] * at.pps;
  float e_bias = 0.f, e_scale = 1.f;
  uint16_t *kv_dst = nullptr;
  if (threadIdx.x < 24) {
    const int en = ej * K + h * kHeadDim + 8 * c + eg;     // output feature in [0, 3d)
    e_bias = bf16_bits_to_float(a.bias[en]);
    if (WF == WF_INT8) e_scale = bf16_bits_to_float(a.scales[en]);
    if (ej > 0)
      kv_dst = const_cast<uint16_t *>(at.kv_layer) + (((size_t)pt[n_pages - 1] * 2 + (ej - 1)) * at.H + h) * kPageElems + (size_t)tn * kHeadDim + 8 * c + eg;
  }
  // the warp's old K/V units (every entry but the new token's is final)
  const int tg = lane >> 3, sub = lane & 7;
  const int GW = kQaCluster * kAttnWarps, gw = c * kAttnWarps + warp;
  const int n_units = (n_tok + 15) >> 4;
  const bool have_units = gw < n_units;
  PageLoad pl;
  uint32_t vmask = 0u;
  int ng = 0;
  if (have_units) vmask = load_quarters(pl, at.kv_layer, pt, at.H, h, gw, GW, n_units, n_tok, tg, sub, ng);
  pdl_launch_dependents();
  pdl_wait();
  trace_mark(at.trace, at.trace_slot, 1);

  // ---- 2. LayerNorm of the row into shared memory (bf16, the matmul operand) ----
  {
    const float *xr = a.x + (size_t)r * K;
    float4 xv[kQaLnRounds];
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kQaLnRounds; ++i) {
      const int lc = 4 * (threadIdx.x + kQaThreads * i);
      xv[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (lc < K) xv[i] = *reinterpret_cast<const float4 *>(xr + lc);
      s += (xv[i].x + xv[i].y) + (xv[i].z + xv[i].w);
    }
    const float mu = qa_block_sum(s, lnred, warp, lane) / (float)K;
    float q2 = 0.f;
#pragma unroll
    for (int i = 0; i < kQaLnRounds; ++i) {
      const int lc = 4 * (threadIdx.x + kQaThreads * i);
      if (lc < K) {
        const float d0 = xv[i].x - mu, d1 = xv[i].y - mu, d2 = xv[i].z - mu, d3 = xv[i].w - mu;
        q2 += (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
      }
    }
    const float rstd = rsqrtf(qa_block_sum(q2, lnred, warp, lane) / (float)K + a.ln_eps);
#pragma unroll
    for (int i = 0; i < kQaLnRounds; ++i) {
      const int lc = 4 * (threadIdx.x + kQaThreads * i);
      if (lc < K) {
        uint2 y;
        y.x = pack_bf16x2((xv[i].x - mu) * rstd * bf16_lo(ln_gg[i].x) + bf16_lo(ln_bb[i].x),
                          (xv[i].y - mu) * rstd * bf16_hi(ln_gg[i].x) + bf16_hi(ln_bb[i].x));
        y.y = pack_bf16x2((xv[i].z - mu) * rstd * bf16_lo(ln_gg[i].y) + bf16_lo(ln_bb[i].y),
                          (xv[i].w - mu) * rstd * bf16_hi(ln_gg[i].y) + bf16_hi(ln_bb[i].y));
        *reinterpret_cast<uint2 *>(xs + lc) = y;
      }
    }
    __syncthreads();
  }
  trace_mark(at.trace, at.trace_slot, 7);
  bool dead = false;
  if (!mbar_wait_bounded(wbar, 0, 2000000000ull)) {
    if (at.err) atomicExch(at.err, 1);
    mbar_wait_bounded(wbar, 0, 2000000000ull);   // a last chance for the copies in flight towards this CTA
    dead = true;                                 // keep walking the cluster barriers; the step is reported as failed
  }

  // ---- the 24 dot products: lane (g, t) owns 16 bytes of weight row g of a tile, warp w the k-tiles w, w+4, ..
  {
    const int g = lane >> 2, t = lane & 3;
    const uint4 *wtile = reinterpret_cast<const uint4 *>(wsm);
    float facc[3] = {0.f, 0.f, 0.f};
    if (!dead) {
#pragma unroll 2
      for (int kb = warp; kb < KB; kb += kAttnWarps) {
        const int col = kb * KT + t * (KT / 4);
        uint4 wq[3];
#pragma unroll
        for (int j = 0; j < 3; ++j) wq[j] = wtile[((size_t)j * KB + kb) * 32 + lane];
        float tacc[3] = {0.f, 0.f, 0.f};
#pragma unroll
        for (int q = 0; q < AW; ++q) {
          const uint4 xq = *reinterpret_cast<const uint4 *>(xs + col + 8 * q);
          const float xf[8] = {bf16_lo(xq.x), bf16_hi(xq.x), bf16_lo(xq.y), bf16_hi(xq.y),
                               bf16_lo(xq.z), bf16_hi(xq.z), bf16_lo(xq.w), bf16_hi(xq.w)};
#pragma unroll
          for (int j = 0; j < 3; ++j) {
            const uint32_t ww[4] = {wq[j].x, wq[j].y, wq[j].z, wq[j].w};
            float wv[8];
            if (WF == WF_BF16) {
#pragma unroll
              for (int k = 0; k < 4; ++k) { wv[2 * k] = bf16_lo(ww[k]); wv[2 * k + 1] = bf16_hi(ww[k]); }
            } else if (WF == WF_INT8) {
#pragma unroll
              for (int k = 0; k < 8; ++k) wv[k] = biased_byte_to_float(ww[(2 * q + (k >> 2)) & 3], k & 3);
            } else {
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const uint32_t pr = ((ww[q & 3] >> (4 * e)) & 0x000F000Fu) | 0x43004300u;  // bf16 pair 128+u
                wv[2 * e] = bf16_lo(pr) - 136.f;
                wv[2 * e + 1] = bf16_hi(pr) - 136.f;
              }
            }
            float s0 = (WF == WF_INT4) ? tacc[j] : facc[j];
            float s1 = wv[4] * xf[4];
            s0 = fmaf(wv[0], xf[0], s0); s1 = fmaf(wv[5], xf[5], s1);
            s0 = fmaf(wv[1], xf[1], s0); s1 = fmaf(wv[6], xf[6], s1);
            s0 = fmaf(wv[2], xf[2], s0); s1 = fmaf(wv[7], xf[7], s1);
            s0 = fmaf(wv[3], xf[3], s0);
            s0 += s1;
            if (WF == WF_INT4) tacc[j] = s0; else facc[j] = s0;
          }
        }
        if (WF == WF_INT4) {
#pragma unroll
          for (int j = 0; j < 3; ++j)
            facc[j] = fmaf(bf16_bits_to_float(ssm[((size_t)j * KB + kb) * 8 + g]), tacc[j], facc[j]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 3; ++j) {
      float v = facc[j];
      v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
      v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
      if (t == 0) red[warp][8 * j + g] = v;
    }
  }
  __syncthreads();
  trace_mark(at.trace, at.trace_slot, 6);

  // ---- 3. q and the new token's K, V to every rank of the cluster; K, V to the page ----
  cluster.barrier_wait();              // pairs with barrier_arrive above
  if (threadIdx.x < 24) {
    float v = (red[0][threadIdx.x] + red[1][threadIdx.x]) + (red[2][threadIdx.x] + red[3][threadIdx.x]);
    v = v * e_scale + e_bias;
    const int idx = 8 * c + eg;
    if (ej == 0) {
#pragma unroll
      for (int rr = 0; rr < kQaCluster; ++rr) cluster.map_shared_rank(q_sh, rr)[idx] = v;
    } else {
      const uint16_t b = float_to_bf16_bits(v);
      *kv_dst = b;
      uint16_t *loc = ej == 1 ? kn_sh : vn_sh;
#pragma unroll
      for (int rr = 0; rr < kQaCluster; ++rr) cluster.map_shared_rank(loc, rr)[idx] = b;
    }
  }
  cluster.sync();
  trace_mark(at.trace, at.trace_slot, 4);

  // ---- 4. attention over the warp's units ----
  float m = -INFINITY, l = 0.f;
  float o[8], qv[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) o[e] = 0.f;
  {
    const float qs = 0.125f * 1.4426950408889634f;   // scores in log2 units: 1/sqrt(64) * log2(e)
    const float4 q0 = *reinterpret_cast<const float4 *>(q_sh + 8 * sub), q1 = *reinterpret_cast<const float4 *>(q_sh + 8 * sub + 4);
    qv[0] = q0.x * qs; qv[1] = q0.y * qs; qv[2] = q0.z * qs; qv[3] = q0.w * qs;
    qv[4] = q1.x * qs; qv[5] = q1.y * qs; qv[6] = q1.z * qs; qv[7] = q1.w * qs;
  }
  if (have_units) {
    const int us = 4 * (n_pages - 1) + (tn >> 4);   // unit of the new token
    if (us % GW == gw && us / GW < 4 && (tn & 3) == tg) {
      const uint4 kn = *reinterpret_cast<const uint4 *>(kn_sh + 8 * sub);
      const uint4 vn = *reinterpret_cast<const uint4 *>(vn_sh + 8 * sub);
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
    bool loaded = true;
    for (int u0 = gw; u0 < n_units; u0 += 4 * GW) {
      // a second batch only exists beyond 2048 tokens of context; its loads see the new token in global
      // memory (written above, in front of the cluster barrier)
      if (!loaded) vmask = load_quarters(pl, at.kv_layer, pt, at.H, h, u0, GW, n_units, n_tok, tg, sub, ng);
      loaded = false;
      fold_slots(pl, qv, vmask, ng, m, l, o);
    }
  }
  trace_mark(at.trace, at.trace_slot, 3);
  const int e = threadIdx.x;
  float M, L, O;
  cta_merge(m, l, o, warp, tg, sub, sm_m, sm_l, sm_o, M, L, O);
  if (e < kHeadDim) {
    float *dst = cluster.map_shared_rank(&cl_all[0][0], 0) + (size_t)c * kAttnPartialFloats;
    if (e == 0) { dst[0] = M; dst[1] = L; }
    dst[2 + e] = O;
  }
  cluster.sync();
  trace_mark(at.trace, at.trace_slot, 5);
  if (c == 0 && e < kHeadDim && !dead) {
    float pm[kQaCluster], pl_[kQaCluster], po[kQaCluster];
#pragma unroll
    for (int rr = 0; rr < kQaCluster; ++rr) { pm[rr] = cl_all[rr][0]; pl_[rr] = cl_all[rr][1]; po[rr] = cl_all[rr][2 + e]; }
    float MM = -INFINITY;
#pragma unroll
    for (int rr = 0; rr < kQaCluster; ++rr) MM = fmaxf(MM, pm[rr]);
    float LL = 0.f, OO = 0.f;
#pragma unroll
    for (int rr = 0; rr < kQaCluster; ++rr) {
      const float f = (pm[rr] == -INFINITY) ? 0.f : exp2f(pm[rr] - MM);  // a rank without tokens contributes nothing
      LL = fmaf(pl_[rr], f, LL);
      OO = fmaf(po[rr], f, OO);
    }
    uint16_t *out = at.out_image ? reinterpret_cast<uint16_t *>(reinterpret_cast<unsigned char *>(at.out) + act_image_offset(r, h * kHeadDim + e))
                                 : at.out + (size_t)r * at.H * kHeadDim + h * kHeadDim + e;
    *out = float_to_bf16_bits(OO / LL);
  }
  trace_mark(at.trace, at.trace_slot, 2);
}

// usable when the row's cluster would be 8 CTAs anyway and the tiles of a head divide over them
inline bool can_fuse_qkv_attention(int wf, int R, int d, int H, int n_sm, int cluster_fill) {
  return R == 1 && d <= kQaMaxK && d % 128 == 0 && d % k_per_tile(wf) == 0 && H * kHeadDim == d &&
         attention_cluster_size(R, H, n_sm, cluster_fill) == kQaCluster && qkv_attn_smem_bytes(wf, d) <= 200 * 1024;
}

template <int WF>
inline cudaError_t launch_qkv_attention_wf(const QkvAttnArgs &a, int R, cudaStream_t st, bool pdl) {
  static PerDeviceOnce attr_once;   // per device: opt-in to more than 48 KB of dynamic shared memory
  const size_t smem = qkv_attn_smem_bytes(WF, a.d);
  if (attr_once.first()) cudaFuncSetAttribute(qkv_attention_kernel<WF>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  cudaLaunchConfig_t cfg;
  cfg.gridDim = dim3(kQaCluster, a.at.H, R);
  cfg.blockDim = dim3(kQaThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  int n = 0;
  at[n].id = cudaLaunchAttributeClusterDimension;
  at[n].val.clusterDim.x = kQaCluster; at[n].val.clusterDim.y = 1; at[n].val.clusterDim.z = 1;
  ++n;
  if (pdl) {
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = at;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, qkv_attention_kernel<WF>, a);
}

inline cudaError_t launch_qkv_attention(int wf, const QkvAttnArgs &a, int R, cudaStream_t st, bool pdl) {
  if (wf == WF_BF16) return launch_qkv_attention_wf<WF_BF16>(a, R, st, pdl);
  if (wf == WF_INT8) return launch_qkv_attention_wf<WF_INT8>(a, R, st, pdl);
  return launch_qkv_attention_wf<WF_INT4>(a, R, st, pdl);
}

}  // namespace ttsgpt
