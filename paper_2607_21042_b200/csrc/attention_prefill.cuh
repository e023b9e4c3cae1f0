// Prefill attention on the warp-level tensor-core path (Section I: the decode engine's attention
// kernels; the prefix pass in front of the first decode step).
//
// The rows of a prefill pass are consecutive positions of a few streams, so 16 consecutive rows of
// the pass mostly belong to one stream and attend to the same K/V pages.  A CTA takes one head and
// one tile of 16 rows.  Its 4 warps deal the tile's page jobs (for each run of rows of one stream:
// pages 0 .. last position / 64) round-robin; a warp computes, for one page,
//     S = Q K^T   (16 x 64, bf16 m16n8k16 MMAs, fp32 accumulators),
// masks the tokens a row does not see (its own position is the last one it sees; rows of another
// stream see nothing of this page), updates the running softmax statistics of its 16 rows, and adds
//     O += P V    (P rounded to bf16 as the MMA operand, the row sums kept from the fp32 values).
// The four warps' (max, sum, output) triples meet in shared memory and are merged by log-sum-exp in
// warp order: the result does not depend on timing.
//
// Operand fragments come straight from global memory with 128-bit loads and no shared-memory
// staging.  The contraction index of an MMA may be permuted freely as long as both operands use the
// same permutation, and so may the output column index:
//   * Q K^T: lane (g, c) = (lane / 4, lane % 4) loads the 16-byte chunks c and c + 4 of K row
//     8 * nt + g; the 8 bf16 pairs it holds serve as the (b0, b1) registers of the 4 k-steps, and
//     the Q fragments are built from the same chunks of the Q rows.
//   * P V: the lane loads chunk g of the V rows of tokens 2c, 2c + 1, 8 + 2c, 9 + 2c of a 16-token
//     k-step; halfword j of two such chunks, paired by one byte permute, is the b register of output
//     tile j, whose column g then is dimension 8 * g + j.  A lane therefore ends up with 16
//     consecutive output dimensions (16 * c ..) of rows g and g + 8.
#pragma once
#include "attention.cuh"

namespace ttsgpt {

constexpr int kPrefillMmaRows = 16;    // rows of the pass per CTA
constexpr int kPrefillMmaWarps = 4;

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ __forceinline__ uint32_t prmt(uint32_t x, uint32_t y, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(x), "r"(y), "r"(sel));
  return r;
}

// the 4 bf16 pairs of one 8-float chunk of a Q row
__device__ __forceinline__ void q_chunk_pairs(const float *q, bool have, uint32_t (&p)[4]) {
  uint4 u0 = make_uint4(0, 0, 0, 0), u1 = u0;
  if (have) { u0 = ld_stream_u4(q); u1 = ld_stream_u4(q + 4); }   // issued in program order, ahead of the first K/V requests
  p[0] = pack_bf16x2(__uint_as_float(u0.x), __uint_as_float(u0.y)); p[1] = pack_bf16x2(__uint_as_float(u0.z), __uint_as_float(u0.w));
  p[2] = pack_bf16x2(__uint_as_float(u1.x), __uint_as_float(u1.y)); p[3] = pack_bf16x2(__uint_as_float(u1.z), __uint_as_float(u1.w));
}

__global__ void __launch_bounds__(kPrefillMmaWarps * 32) attention_prefill_mma_kernel(const AttnArgs a, int R) {
  __shared__ int seg_stream[kPrefillMmaRows], seg_i0[kPrefillMmaRows], seg_i1[kPrefillMmaRows], seg_last[kPrefillMmaRows];
  __shared__ int n_seg_s;
  __shared__ float sm_m[kPrefillMmaWarps][kPrefillMmaRows], sm_l[kPrefillMmaWarps][kPrefillMmaRows];
  __shared__ __align__(16) float sm_o[kPrefillMmaWarps][kPrefillMmaRows][kHeadDim + 4];
  const int h = blockIdx.y, r0 = blockIdx.z * kPrefillMmaRows;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  trace_mark(a.trace, a.trace_slot, 0);
  if (threadIdx.x == 0) {
    // runs of rows of one stream (the row table is final before the pass's first kernel starts)
    const int r_end = min(R, r0 + kPrefillMmaRows);
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
  const int n_seg = n_seg_s;
  const int rowA = r0 + g, rowB = rowA + 8;
  const int posA = rowA < R ? a.row_pos[rowA] : -1, posB = rowB < R ? a.row_pos[rowB] : -1;
  // the page ids of the warp's first two jobs, looked up while the kernel in front still runs (the row
  // and page tables are final before the pass starts), so that a job's K/V requests do not queue behind
  // a table read
  int phys_first[2] = {0, 0};
  {
    int job = 0, mine = 0;
    for (int seg = 0; seg < n_seg && mine < 2; ++seg) {
      const int n_pages = seg_last[seg] / kPageTokens + 1;
      for (int p = 0; p < n_pages && mine < 2; ++p, ++job) {
        if ((job & (kPrefillMmaWarps - 1)) != warp) continue;
        const int ph = a.page_table[(size_t)seg_stream[seg] * a.pps + p];
        if (mine == 0) phys_first[0] = ph; else phys_first[1] = ph;
        ++mine;
        // pull the page's K and V blocks (2 x 8 KB, 128 lines) towards L2 meanwhile: earlier passes' pages
        // have been pushed out by the weights since
        const unsigned char *blk = reinterpret_cast<const unsigned char *>(a.kv_layer + (((size_t)ph * 2 + 0) * a.H + h) * kPageElems);
        const size_t v_off = (size_t)a.H * kPageElems * 2;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          prefetch_l2(blk + (size_t)(lane + 32 * i) * 128);
          prefetch_l2(blk + v_off + (size_t)(lane + 32 * i) * 128);
        }
      }
    }
  }
  pdl_wait();     // Q and the K/V rows of this pass were written by the QKV kernel in front
  trace_mark(a.trace, a.trace_slot, 1);

  // Q fragments of the 4 k-steps: k-step ks takes pairs 2ks and 2ks+1 of the lane's 8 pairs
  uint32_t qf[4][4];
  {
    uint32_t pa[2][4], pb[2][4];
    const float *qa = a.q + (size_t)rowA * a.H * kHeadDim + h * kHeadDim;
    const float *qb = a.q + (size_t)rowB * a.H * kHeadDim + h * kHeadDim;
    q_chunk_pairs(qa + 8 * c, rowA < R, pa[0]); q_chunk_pairs(qa + 32 + 8 * c, rowA < R, pa[1]);
    q_chunk_pairs(qb + 8 * c, rowB < R, pb[0]); q_chunk_pairs(qb + 32 + 8 * c, rowB < R, pb[1]);
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      qf[ks][0] = pa[ks >> 1][2 * (ks & 1)];     qf[ks][1] = pb[ks >> 1][2 * (ks & 1)];
      qf[ks][2] = pa[ks >> 1][2 * (ks & 1) + 1]; qf[ks][3] = pb[ks >> 1][2 * (ks & 1) + 1];
    }
  }
  const float qs = 0.125f * 1.4426950408889634f;   // scores in log2 units: 1/sqrt(64) * log2(e)

  float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;   // l: this lane's share of the row sums
  float o[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }

  int job = 0, mine = 0;
  for (int seg = 0; seg < n_seg; ++seg) {
    const int last_pos = seg_last[seg];
    const int n_pages = last_pos / kPageTokens + 1;
    const bool actA = rowA >= seg_i0[seg] && rowA < seg_i1[seg];
    const bool actB = rowB >= seg_i0[seg] && rowB < seg_i1[seg];
    const int *pt = a.page_table + (size_t)seg_stream[seg] * a.pps;
    for (int p = 0; p < n_pages; ++p, ++job) {
      if ((job & (kPrefillMmaWarps - 1)) != warp) continue;   // warp-uniform
      const int n_here = min(kPageTokens, last_pos + 1 - p * kPageTokens);   // tokens of the page any row of the run sees
      const int n_tiles = (n_here + 7) >> 3;
      const int phys = mine == 0 ? phys_first[0] : mine == 1 ? phys_first[1] : pt[p];
      ++mine;
      const uint16_t *K = a.kv_layer + (((size_t)phys * 2 + 0) * a.H + h) * kPageElems;
      const uint16_t *V = K + (size_t)a.H * kPageElems;
      // tokens of this page rows A and B see (0: none)
      const int seeA = actA ? min(kPageTokens, posA + 1 - p * kPageTokens) : 0;
      const int seeB = actB ? min(kPageTokens, posB + 1 - p * kPageTokens) : 0;

      // ---- S = Q K^T: all of the page's K fragments are requested before the first MMA
      uint4 kk[8][2];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        if (nt < n_tiles) {
          const uint16_t *kr = K + (size_t)(8 * nt + g) * kHeadDim;
          kk[nt][0] = ld_stream_u4(kr + 8 * c); kk[nt][1] = ld_stream_u4(kr + 32 + 8 * c);
        }
      }
      float s[8][4];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
        if (nt < n_tiles) {
          mma_bf16_16816(s[nt], qf[0], kk[nt][0].x, kk[nt][0].y);
          mma_bf16_16816(s[nt], qf[1], kk[nt][0].z, kk[nt][0].w);
          mma_bf16_16816(s[nt], qf[2], kk[nt][1].x, kk[nt][1].y);
          mma_bf16_16816(s[nt], qf[3], kk[nt][1].z, kk[nt][1].w);
        }
      }
      // the V fragments travel while the softmax statistics are updated
      uint4 vv[4][4];
#pragma unroll
      for (int kt = 0; kt < 4; ++kt) {
        if (2 * kt < n_tiles) {
          const uint16_t *vr = V + (size_t)(16 * kt + 2 * c) * kHeadDim + 8 * g;
          vv[kt][0] = ld_stream_u4(vr); vv[kt][1] = ld_stream_u4(vr + kHeadDim);
          vv[kt][2] = ld_stream_u4(vr + 8 * kHeadDim); vv[kt][3] = ld_stream_u4(vr + 9 * kHeadDim);
        }
      }
      // ---- mask, row maxima
      float pmA = -INFINITY, pmB = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const int t = 8 * nt + 2 * c;
        s[nt][0] = (t < seeA) ? s[nt][0] * qs : -INFINITY;
        s[nt][1] = (t + 1 < seeA) ? s[nt][1] * qs : -INFINITY;
        s[nt][2] = (t < seeB) ? s[nt][2] * qs : -INFINITY;
        s[nt][3] = (t + 1 < seeB) ? s[nt][3] * qs : -INFINITY;
        pmA = fmaxf(pmA, fmaxf(s[nt][0], s[nt][1]));
        pmB = fmaxf(pmB, fmaxf(s[nt][2], s[nt][3]));
      }
      pmA = fmaxf(pmA, __shfl_xor_sync(0xFFFFFFFFu, pmA, 1)); pmA = fmaxf(pmA, __shfl_xor_sync(0xFFFFFFFFu, pmA, 2));
      pmB = fmaxf(pmB, __shfl_xor_sync(0xFFFFFFFFu, pmB, 1)); pmB = fmaxf(pmB, __shfl_xor_sync(0xFFFFFFFFu, pmB, 2));
      const float mA_new = fmaxf(mA, pmA), mB_new = fmaxf(mB, pmB);
      // a row that has seen nothing yet keeps m = -inf; its exponents are taken against 0
      const float refA = (mA_new == -INFINITY) ? 0.f : mA_new, refB = (mB_new == -INFINITY) ? 0.f : mB_new;
      const float scA = exp2f(mA - refA), scB = exp2f(mB - refB);
      mA = mA_new; mB = mB_new;
      float sumA = 0.f, sumB = 0.f;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        s[nt][0] = exp2f(s[nt][0] - refA); s[nt][1] = exp2f(s[nt][1] - refA);
        s[nt][2] = exp2f(s[nt][2] - refB); s[nt][3] = exp2f(s[nt][3] - refB);
        sumA += s[nt][0] + s[nt][1];
        sumB += s[nt][2] + s[nt][3];
      }
      lA = lA * scA + sumA; lB = lB * scB + sumB;
#pragma unroll
      for (int j = 0; j < 8; ++j) { o[j][0] *= scA; o[j][1] *= scA; o[j][2] *= scB; o[j][3] *= scB; }

      // ---- O += P V
#pragma unroll
      for (int kt = 0; kt < 4; ++kt) {
        if (2 * kt < n_tiles) {
          uint32_t pf[4];
          pf[0] = pack_bf16x2(s[2 * kt][0], s[2 * kt][1]);         pf[1] = pack_bf16x2(s[2 * kt][2], s[2 * kt][3]);
          pf[2] = pack_bf16x2(s[2 * kt + 1][0], s[2 * kt + 1][1]); pf[3] = pack_bf16x2(s[2 * kt + 1][2], s[2 * kt + 1][3]);
          const int t0 = 16 * kt + 2 * c;
          uint4 v0 = vv[kt][0], v1 = vv[kt][1], v2 = vv[kt][2], v3 = vv[kt][3];
          // tokens nobody sees may hold stale bits (NaN): 0 * NaN must not reach o
          const uint4 z = make_uint4(0, 0, 0, 0);
          if (t0 >= n_here) v0 = z;
          if (t0 + 1 >= n_here) v1 = z;
          if (t0 + 8 >= n_here) v2 = z;
          if (t0 + 9 >= n_here) v3 = z;
          mma_bf16_16816(o[0], pf, prmt(v0.x, v1.x, 0x5410), prmt(v2.x, v3.x, 0x5410));
          mma_bf16_16816(o[1], pf, prmt(v0.x, v1.x, 0x7632), prmt(v2.x, v3.x, 0x7632));
          mma_bf16_16816(o[2], pf, prmt(v0.y, v1.y, 0x5410), prmt(v2.y, v3.y, 0x5410));
          mma_bf16_16816(o[3], pf, prmt(v0.y, v1.y, 0x7632), prmt(v2.y, v3.y, 0x7632));
          mma_bf16_16816(o[4], pf, prmt(v0.z, v1.z, 0x5410), prmt(v2.z, v3.z, 0x5410));
          mma_bf16_16816(o[5], pf, prmt(v0.z, v1.z, 0x7632), prmt(v2.z, v3.z, 0x7632));
          mma_bf16_16816(o[6], pf, prmt(v0.w, v1.w, 0x5410), prmt(v2.w, v3.w, 0x5410));
          mma_bf16_16816(o[7], pf, prmt(v0.w, v1.w, 0x7632), prmt(v2.w, v3.w, 0x7632));
        }
      }
    }
  }
  trace_mark(a.trace, a.trace_slot, 3);

  // ---- the warp's result into shared memory: lane (g, c) holds dimensions 16c + j (o[j][0], o[j][2]) and
  // 16c + 8 + j (o[j][1], o[j][3]) of rows g and g + 8
  lA += __shfl_xor_sync(0xFFFFFFFFu, lA, 1); lA += __shfl_xor_sync(0xFFFFFFFFu, lA, 2);
  lB += __shfl_xor_sync(0xFFFFFFFFu, lB, 1); lB += __shfl_xor_sync(0xFFFFFFFFu, lB, 2);
  if (c == 0) { sm_m[warp][g] = mA; sm_m[warp][g + 8] = mB; sm_l[warp][g] = lA; sm_l[warp][g + 8] = lB; }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    sm_o[warp][g][16 * c + j] = o[j][0];     sm_o[warp][g][16 * c + 8 + j] = o[j][1];
    sm_o[warp][g + 8][16 * c + j] = o[j][2]; sm_o[warp][g + 8][16 * c + 8 + j] = o[j][3];
  }
  __syncthreads();
  // ---- merge in warp order: thread t takes row t / 8, dimensions 8 * (t % 8) ..
  const int row = threadIdx.x >> 3, d0 = 8 * (threadIdx.x & 7);
  const int r = r0 + row;
  if (r < R) {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kPrefillMmaWarps; ++w) M = fmaxf(M, sm_m[w][row]);
    float L = 0.f, y[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) y[e] = 0.f;
#pragma unroll
    for (int w = 0; w < kPrefillMmaWarps; ++w) {
      const float f = exp2f(sm_m[w][row] - M);   // a warp that saw nothing of this row: exp2(-inf) = 0
      L = fmaf(sm_l[w][row], f, L);
      const float4 x0 = *reinterpret_cast<const float4 *>(&sm_o[w][row][d0]);
      const float4 x1 = *reinterpret_cast<const float4 *>(&sm_o[w][row][d0 + 4]);
      y[0] = fmaf(x0.x, f, y[0]); y[1] = fmaf(x0.y, f, y[1]); y[2] = fmaf(x0.z, f, y[2]); y[3] = fmaf(x0.w, f, y[3]);
      y[4] = fmaf(x1.x, f, y[4]); y[5] = fmaf(x1.y, f, y[5]); y[6] = fmaf(x1.z, f, y[6]); y[7] = fmaf(x1.w, f, y[7]);
    }
    const float inv = 1.0f / L;
    const uint4 yy = make_uint4(pack_bf16x2(y[0] * inv, y[1] * inv), pack_bf16x2(y[2] * inv, y[3] * inv),
                                pack_bf16x2(y[4] * inv, y[5] * inv), pack_bf16x2(y[6] * inv, y[7] * inv));
    const int col = h * kHeadDim + d0;
    if (a.out_image) *reinterpret_cast<uint4 *>(reinterpret_cast<unsigned char *>(a.out) + act_image_offset_tiled(r, col, a.H * kHeadDim)) = yy;
    else *reinterpret_cast<uint4 *>(a.out + (size_t)r * a.H * kHeadDim + col) = yy;
  }
  trace_mark(a.trace, a.trace_slot, 2);
}

inline cudaError_t launch_attention_prefill_mma(const AttnArgs &a, int R, cudaStream_t st, bool pdl) {
  const int groups = (R + kPrefillMmaRows - 1) / kPrefillMmaRows;
  return launch_kernel(attention_prefill_mma_kernel, dim3(1, a.H, groups), dim3(kPrefillMmaWarps * 32), 0, st, pdl, a, R);
}

}  // namespace ttsgpt
