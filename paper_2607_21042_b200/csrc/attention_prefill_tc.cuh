// Prefill attention on the 5th-generation tensor cores (tcgen05) for passes of several row tiles
// (Section I: the decode engine's attention kernels; the prefix pass in front of the first decode step).
//
// A CTA takes one head and a tile of 128 consecutive rows of the pass (accumulator lane = row) and walks
// the tile's page jobs (for each run of rows of one stream: pages 0 .. last position / 64), one page of
// 64 tokens at a time:
//     S = Q K^T     tcgen05.mma M=128 (rows) x N=64 (tokens) x K=64 (dimensions), 4 instructions, S in tensor memory
//     softmax       thread t owns row t: S out of tensor memory, mask (causal inside the stream; nothing for
//                   rows of another stream), running maximum and sum in fp32, P rounded to bf16 into shared memory
//     O += P V      M=128 x N=64 (dimensions) x K=64 (tokens), 4 instructions; V is read as stored (token-major =
//                   MN-major for this product); O stays in tensor memory and is rescaled there when a row's
//                   maximum moves
// Warps 0-3 are the softmax threads, warp 4 stages pages (16-byte asynchronous copies into three slots, with the
// 128-byte swizzle the tensor core expects) and issues the instructions.  The Q K^T of page j+1 and the P V of
// page j-1 run while page j goes through the softmax.  Every wait is bounded.
#pragma once
#include "attention_prefill.cuh"
#include "gemm_tc.cuh"

namespace ttsgpt {

constexpr int kPtRows = 128;
constexpr int kPtThreads = 160;
constexpr int kPtSlots = 3;
constexpr int kPtMaxJobs = 256;   // two partial long streams + streams of at most 128 rows

__device__ __forceinline__ void pt_cp16(void *smem, const void *gmem, bool real) {
  // a row that does not exist is filled with zeros (stale shared memory may hold NaN, and 0 * NaN must not reach O)
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem)), "l"(gmem), "r"(real ? 16 : 0) : "memory");
}
__device__ __forceinline__ void pt_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void pt_wait_but() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// 2^x by the special-function unit (relative error 2^-22, 2^-inf = 0): this kernel evaluates it once per score, and
// the library exp2f costs several times the instructions
__device__ __forceinline__ float pt_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// one lane polls a barrier (a poll reads the global timer), the warp barrier passes on what it saw
__device__ __forceinline__ void pt_warp_wait(uint64_t *bar, uint32_t parity, volatile int *failed, int *err, int lane) {
  if (lane == 0) tc_wait(bar, parity, failed, err);
  __syncwarp();
}

// 32 lanes x 32 columns of 32-bit into tensor memory: register c of lane l -> TMEM[lane base + l][column base + c]
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
        "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
        "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// one page (64 tokens x 128 bytes, K then V) into a slot, chunk j of token row t at chunk j ^ (t & 7)
__device__ __forceinline__ void pt_stage(unsigned char *slot, const uint16_t *K, const uint16_t *V, int n_here, int lane) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int idx = lane + 32 * i, t = idx >> 3, j = idx & 7;
    const int off = t * 128 + ((j ^ (t & 7)) << 4);
    pt_cp16(slot + off, K + (size_t)t * kHeadDim + 8 * j, t < n_here);
    pt_cp16(slot + kPageElems * 2 + off, V + (size_t)t * kHeadDim + 8 * j, t < n_here);
  }
  pt_commit();
}

__global__ void __launch_bounds__(kPtThreads) attention_prefill_tc_kernel(const AttnArgs a, int R) {
  extern __shared__ __align__(16) unsigned char pt_smem_raw[];
  unsigned char *base = pt_smem_raw + ((1024u - (smem_u32(pt_smem_raw) & 1023u)) & 1023u);
  unsigned char *Qs = base;                   // 128 rows x 64 dimensions bf16, K-major, 128-byte swizzle
  unsigned char *Ps = base + 16384;           // 128 rows x 64 tokens bf16, same layout
  unsigned char *slots = base + 32768;        // [3][K 64 tokens x 128 B | V 64 tokens x 128 B]
  uint64_t *q_full = reinterpret_cast<uint64_t *>(slots + kPtSlots * 16384);
  uint64_t *s_full = q_full + 1, *s_free = q_full + 2, *p_full = q_full + 3, *pv_done = q_full + 4;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(q_full + 5);
  volatile int *failed = reinterpret_cast<volatile int *>(tmem_slot + 1);
  __shared__ int row_s[kPtRows], row_p[kPtRows];
  __shared__ int seg_stream[kPtRows], seg_i0[kPtRows], seg_i1[kPtRows], seg_last[kPtRows];
  __shared__ unsigned short jobs[kPtMaxJobs];   // (run << 8) | page, in run order
  __shared__ int n_job_s;

  const int h = blockIdx.y, r0 = blockIdx.z * kPtRows;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  trace_mark(a.trace, a.trace_slot, 0);
  if (threadIdx.x < kPtRows) {
    const int r = r0 + threadIdx.x;   // the row table is final before the pass's first kernel starts
    row_s[threadIdx.x] = r < R ? a.row_stream[r] : -1;
    row_p[threadIdx.x] = r < R ? a.row_pos[r] : -1;
  }
  if (threadIdx.x == 0) {
    mbar_init(q_full, kPtRows); mbar_init(s_full, 1); mbar_init(s_free, kPtRows); mbar_init(p_full, kPtRows); mbar_init(pv_done, 1);
    *failed = 0;
  }
  if (warp == 4) tmem_alloc(tmem_slot, 128);   // S: columns 0-63, O: columns 64-127
  __syncthreads();
  if (threadIdx.x == 0) {
    const int n_rows = min(R - r0, kPtRows);
    int n = 0, i0 = 0;
    while (i0 < n_rows) {   // runs of rows of one stream
      const int s = row_s[i0];
      int i1 = i0 + 1;
      while (i1 < n_rows && row_s[i1] == s) ++i1;
      seg_stream[n] = s; seg_i0[n] = r0 + i0; seg_i1[n] = r0 + i1; seg_last[n] = row_p[i1 - 1];
      ++n; i0 = i1;
    }
    int nj = 0;
    for (int sg = 0; sg < n; ++sg)
      for (int pg = 0; pg <= seg_last[sg] / kPageTokens && nj < kPtMaxJobs; ++pg) jobs[nj++] = (unsigned short)((sg << 8) | pg);
    n_job_s = nj;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  const int n_job = n_job_s;
  pdl_launch_dependents();
  pdl_wait();     // Q and the K/V rows of this pass were written by the QKV kernel in front
  trace_mark(a.trace, a.trace_slot, 1);

  if (warp == 4) {
    // ---- pages into the slots, instructions to the tensor core ----
    auto stage = [&](int j) {
      if (j < n_job) {
        const int sg = jobs[j] >> 8, pg = jobs[j] & 255;
        const int n_here = min(kPageTokens, seg_last[sg] + 1 - pg * kPageTokens);
        const int ph = a.page_table[(size_t)seg_stream[sg] * a.pps + pg];
        const uint16_t *K = a.kv_layer + (((size_t)ph * 2 + 0) * a.H + h) * kPageElems;
        pt_stage(slots + (size_t)(j % kPtSlots) * 16384, K, K + (size_t)a.H * kPageElems, n_here, lane);
      } else {
        pt_commit();   // an empty group keeps the count of groups per job uniform
      }
    };
    stage(0); stage(1); stage(2);
    if (lane == 0) tc_wait(q_full, 0, failed, a.err);
    const uint32_t idesc_qk = tc_instr_desc(kPtRows, 64);
    const uint32_t idesc_pv = tc_instr_desc(kPtRows, 64) | (1u << 16);   // B (= V) is MN-major: token rows of 64 dimensions
    auto pv = [&](int j) {   // O (+)= P V for job j
      tc_wait(p_full, (uint32_t)j & 1u, failed, a.err);
      tc_fence_after_sync();
      const uint64_t dp = tc_smem_desc(Ps), dv = tc_smem_desc(slots + (size_t)(j % kPtSlots) * 16384 + kPageElems * 2);
#pragma unroll
      for (int k = 0; k < 4; ++k)   // 16 tokens per instruction: 32 bytes along a P row, two 8-row groups (2048 bytes) down V
        tc_mma(tmem + 64u, dp + 2 * k, dv + 128 * k, idesc_pv, (j == 0 && k == 0) ? 0u : 1u);
      tc_commit(pv_done);
    };
    for (int j = 0; j < n_job; ++j) {
      // page j + 1 goes into the slot page j - 2 used, free once P V of job j - 2 has completed
      if (j + 1 >= kPtSlots) {
        if (lane == 0) tc_wait(pv_done, (uint32_t)(j - 2) & 1u, failed, a.err);
        __syncwarp();
        stage(j + 1);
      } else {
        pt_commit();
      }
      pt_wait_but<1>();            // everything but the group just committed: page j has landed
      fence_proxy_async_smem();    // the tensor core reads the slot through the async proxy
      __syncwarp();
      if (lane == 0) {
        if (j > 0) tc_wait(s_free, (uint32_t)(j - 1) & 1u, failed, a.err);   // the softmax threads hold S of job j - 1 in registers
        tc_fence_after_sync();
        const uint64_t dq = tc_smem_desc(Qs), dk = tc_smem_desc(slots + (size_t)(j % kPtSlots) * 16384);
#pragma unroll
        for (int k = 0; k < 4; ++k) tc_mma(tmem, dq + 2 * k, dk + 2 * k, idesc_qk, k == 0 ? 0u : 1u);   // 16 dimensions per instruction
        tc_commit(s_full);
        if (j > 0) pv(j - 1);
      }
      __syncwarp();
    }
    if (lane == 0 && n_job > 0) pv(n_job - 1);
    __syncwarp();
  } else {
    // ---- softmax: thread t owns row t of the tile = accumulator lane t ----
    const int t = threadIdx.x, r = r0 + t;
    const uint32_t t_lane = tmem + ((uint32_t)(32 * warp) << 16);
    {
      // Q row of this head as bf16 into the swizzled tile (a row beyond the pass is zero)
      const float *qp = a.q + (size_t)r * a.H * kHeadDim + h * kHeadDim;
#pragma unroll
      for (int c8 = 0; c8 < 8; ++c8) {
        float4 x0 = make_float4(0.f, 0.f, 0.f, 0.f), x1 = x0;
        if (r < R) { x0 = *reinterpret_cast<const float4 *>(qp + 8 * c8); x1 = *reinterpret_cast<const float4 *>(qp + 8 * c8 + 4); }
        *reinterpret_cast<uint4 *>(Qs + t * 128 + ((c8 ^ (t & 7)) << 4)) =
            make_uint4(pack_bf16x2(x0.x, x0.y), pack_bf16x2(x0.z, x0.w), pack_bf16x2(x1.x, x1.y), pack_bf16x2(x1.z, x1.w));
      }
      fence_proxy_async_smem();
      mbar_arrive(q_full);
    }
    const float qs = 0.125f * 1.4426950408889634f;   // scores in log2 units: 1/sqrt(64) * log2(e)
    const int pos = row_p[t];
    float m = -INFINITY, l = 0.f;
    for (int j = 0; j < n_job; ++j) {
      pt_warp_wait(s_full, (uint32_t)j & 1u, failed, a.err, lane);
      tc_fence_after_sync();
      float s[64];
      {
        float lo[32], hi[32];
        tmem_ld32(t_lane, lo);
        tmem_ld32(t_lane + 32u, hi);
#pragma unroll
        for (int c = 0; c < 32; ++c) { s[c] = lo[c]; s[32 + c] = hi[c]; }
      }
      tc_fence_before_sync();
      mbar_arrive(s_free);
      const int sg = jobs[j] >> 8, pg = jobs[j] & 255;
      const bool act = r >= seg_i0[sg] && r < seg_i1[sg];
      const int see = act ? min(kPageTokens, pos + 1 - pg * kPageTokens) : 0;   // tokens of the page this row sees
      // four independent chains for the maximum and for the sum: one chain of 64 dependent operations per row and
      // page was the longest thing in the loop
      float pm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < 64; ++c) { s[c] = c < see ? s[c] * qs : -INFINITY; pm4[c & 3] = fmaxf(pm4[c & 3], s[c]); }
      const float pm = fmaxf(fmaxf(pm4[0], pm4[1]), fmaxf(pm4[2], pm4[3]));
      const float m_new = fmaxf(m, pm);
      const float ref = (m_new == -INFINITY) ? 0.f : m_new;   // a row that has seen nothing yet keeps m = -inf
      const float sc = pt_exp2(m - ref);
      m = m_new;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < 64; ++c) { s[c] = pt_exp2(s[c] - ref); sum4[c & 3] += s[c]; }
      const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      l = l * sc + sum;
      // P and O belong to the tensor core until P V of the job before has completed
      if (j > 0) { pt_warp_wait(pv_done, (uint32_t)(j - 1) & 1u, failed, a.err, lane); tc_fence_after_sync(); }
#pragma unroll
      for (int c8 = 0; c8 < 8; ++c8)
        *reinterpret_cast<uint4 *>(Ps + t * 128 + ((c8 ^ (t & 7)) << 4)) =
            make_uint4(pack_bf16x2(s[8 * c8], s[8 * c8 + 1]), pack_bf16x2(s[8 * c8 + 2], s[8 * c8 + 3]),
                       pack_bf16x2(s[8 * c8 + 4], s[8 * c8 + 5]), pack_bf16x2(s[8 * c8 + 6], s[8 * c8 + 7]));
      __syncwarp();
      if (j > 0 && !__all_sync(0xFFFFFFFFu, sc == 1.0f)) {   // some row's maximum moved: rescale the warp's rows of O
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          float o[32];
          tmem_ld32(t_lane + 64u + 32u * hh, o);
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] *= sc;
          tmem_st32(t_lane + 64u + 32u * hh, o);
        }
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(p_full);
    }
    trace_mark(a.trace, a.trace_slot, 3);
    if (n_job > 0) {
      pt_warp_wait(pv_done, (uint32_t)(n_job - 1) & 1u, failed, a.err, lane);
      tc_fence_after_sync();
      const float inv = l > 0.f ? 1.0f / l : 0.f;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        float o[32];
        tmem_ld32(t_lane + 64u + 32u * hh, o);
        if (r < R && !*failed) {
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            const uint4 y = make_uint4(pack_bf16x2(o[8 * c8] * inv, o[8 * c8 + 1] * inv), pack_bf16x2(o[8 * c8 + 2] * inv, o[8 * c8 + 3] * inv),
                                       pack_bf16x2(o[8 * c8 + 4] * inv, o[8 * c8 + 5] * inv), pack_bf16x2(o[8 * c8 + 6] * inv, o[8 * c8 + 7] * inv));
            const int col = h * kHeadDim + 32 * hh + 8 * c8;
            if (a.out_image) *reinterpret_cast<uint4 *>(reinterpret_cast<unsigned char *>(a.out) + act_image_offset_tiled(r, col, a.H * kHeadDim)) = y;
            else *reinterpret_cast<uint4 *>(a.out + (size_t)r * a.H * kHeadDim + col) = y;
          }
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  trace_mark(a.trace, a.trace_slot, 2);
  if (warp == 4) tmem_dealloc(tmem, 128);
}

inline size_t attention_prefill_tc_smem_bytes() { return 32768 + (size_t)kPtSlots * 16384 + 1024 + 256; }

inline cudaError_t launch_attention_prefill_tc(const AttnArgs &a, int R, cudaStream_t st, bool pdl) {
  static PerDeviceOnce attr_once;   // per device: opt-in to more than 48 KB of dynamic shared memory
  if (attr_once.first())
    cudaFuncSetAttribute(attention_prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_prefill_tc_smem_bytes());
  const int groups = (R + kPtRows - 1) / kPtRows;
  return launch_kernel(attention_prefill_tc_kernel, dim3(1, a.H, groups), dim3(kPtThreads), attention_prefill_tc_smem_bytes(), st, pdl, a, R);
}

}  // namespace ttsgpt
