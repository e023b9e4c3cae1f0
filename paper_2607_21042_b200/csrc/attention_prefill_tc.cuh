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
// Warps 0-3 and 4-7 are two softmax groups that take alternate pages, each with its own S, P and O (the two
// partial results meet at the end); one thread of warp 8 issues the instructions, with Q K^T a page ahead of the
// groups; warps 9 and 10 stage the K and V halves of the pages (16-byte asynchronous copies into six slots, with
// the 128-byte swizzle the tensor core expects).  Every wait is bounded.
#pragma once
#include "attention_prefill.cuh"
#include "gemm_tc.cuh"

namespace ttsgpt {

constexpr int kPtRows = 128;
constexpr int kPtThreads = 352;
constexpr int kPtSlots = 6;
constexpr int kPtMergePitch = 65;   // floats per row of the merge buffer: lane = row, conflict-free
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

// half a page (K or V of one head: 64 tokens x 128 bytes) into its half of a slot, chunk j of token row t at
// chunk j ^ (t & 7)
__device__ __forceinline__ void pt_stage(unsigned char *dst, const uint16_t *src, int n_here, int lane) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int idx = lane + 32 * i, t = idx >> 3, j = idx & 7;
    pt_cp16(dst + t * 128 + ((j ^ (t & 7)) << 4), src + (size_t)t * kHeadDim + 8 * j, t < n_here);
  }
  pt_commit();
}

__global__ void __launch_bounds__(kPtThreads) attention_prefill_tc_kernel(const AttnArgs a, int R) {
  extern __shared__ __align__(16) unsigned char pt_smem_raw[];
  unsigned char *base = pt_smem_raw + ((1024u - (smem_u32(pt_smem_raw) & 1023u)) & 1023u);
  unsigned char *Qs = base;                   // 128 rows x 64 dimensions bf16, K-major, 128-byte swizzle
  unsigned char *Ps = base + 16384;           // [2 groups] 128 rows x 64 tokens bf16, same layout
  unsigned char *slots = base + 49152;        // [6][K 64 tokens x 128 B | V 64 tokens x 128 B]
  float *Ms = reinterpret_cast<float *>(slots + kPtSlots * 16384);   // [128][65] group 1's O for the merge
  uint64_t *q_full = reinterpret_cast<uint64_t *>(Ms + kPtRows * kPtMergePitch);
  uint64_t *s_full = q_full + 1, *s_free = q_full + 3, *p_full = q_full + 5, *pv_done = q_full + 7;   // [2] each, by group
  uint64_t *page_full = q_full + 9;   // [kPtSlots] K and V of the slot's page have landed
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(q_full + 9 + kPtSlots);
  volatile int *failed = reinterpret_cast<volatile int *>(tmem_slot + 1);
  __shared__ int row_s[kPtRows], row_p[kPtRows];
  __shared__ int seg_stream[kPtRows], seg_i0[kPtRows], seg_i1[kPtRows], seg_last[kPtRows];
  __shared__ unsigned short jobs[kPtMaxJobs];   // (run << 8) | page, in run order
  __shared__ int n_job_s;
  __shared__ unsigned run_open[kPtRows / 32];   // bit l of word w: row 32 w + l opens a run
  __shared__ int job_ph[kPtMaxJobs];            // physical page of each job
  __shared__ float ref1_s[kPtRows], l1_s[kPtRows];   // group 1's reference score and sum per row

  const int h = blockIdx.y, r0 = blockIdx.z * kPtRows;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  trace_mark(a.trace, a.trace_slot, 0);
  if (threadIdx.x < kPtRows) {
    const int r = r0 + threadIdx.x;   // the row table is final before the pass's first kernel starts
    row_s[threadIdx.x] = r < R ? a.row_stream[r] : -1;
    row_p[threadIdx.x] = r < R ? a.row_pos[r] : -1;
  }
  if (threadIdx.x == 0) {
    mbar_init(q_full, kPtRows);
    for (int sl = 0; sl < kPtSlots; ++sl) mbar_init(page_full + sl, 2);
    for (int g = 0; g < 2; ++g) { mbar_init(s_full + g, 1); mbar_init(s_free + g, kPtRows); mbar_init(p_full + g, kPtRows); mbar_init(pv_done + g, 1); }
    *failed = 0;
  }
  if (warp == 8) tmem_alloc(tmem_slot, 256);   // S of group g: columns 64 g .. + 63, O of group g: columns 128 + 64 g .. + 63
  __syncthreads();
  // runs of rows of one stream, found by all rows at once: a row that differs from the one before opens a run, the
  // number of openings up to a row is its run's index (this set-up is not hidden behind the kernel in front)
  const int n_rows = min(R - r0, kPtRows);
  if (threadIdx.x < kPtRows) {
    const int t = threadIdx.x;
    const bool first = t < n_rows && (t == 0 || row_s[t] != row_s[t - 1]);
    const unsigned b = __ballot_sync(0xFFFFFFFFu, first);
    if (lane == 0) run_open[warp] = b;
  }
  __syncthreads();
  if (threadIdx.x < kPtRows) {
    const int t = threadIdx.x;
    int idx = __popc(run_open[warp] & (0xFFFFFFFFu >> (31 - lane))) - 1;
    for (int w = 0; w < warp; ++w) idx += __popc(run_open[w]);
    if (t < n_rows) {
      if (t == 0 || row_s[t] != row_s[t - 1]) { seg_stream[idx] = row_s[t]; seg_i0[idx] = r0 + t; }
      if (t == n_rows - 1 || row_s[t + 1] != row_s[t]) { seg_i1[idx] = r0 + t + 1; seg_last[idx] = row_p[t]; }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int n = __popc(run_open[0]) + __popc(run_open[1]) + __popc(run_open[2]) + __popc(run_open[3]);
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
  // the physical pages of all jobs up front (the page table is final before the pass's first kernel starts): a
  // page-table read in front of every page's copies would put an L2 round trip into each turn of the producer's loop
  for (int j = threadIdx.x; j < n_job; j += kPtThreads)
    job_ph[j] = a.page_table[(size_t)seg_stream[jobs[j] >> 8] * a.pps + (jobs[j] & 255)];
  __syncthreads();
  pdl_launch_dependents();
  pdl_wait();     // Q and the K/V rows of this pass were written by the QKV kernel in front
  trace_mark(a.trace, a.trace_slot, 1);

  if (warp >= 9) {
    // ---- copy warps: warp 9 brings the K half of every page into its slot, warp 10 the V half ----
    const int part = warp - 9;
    auto stage = [&](int j) {
      if (j < n_job) {
        const int sg = jobs[j] >> 8, pg = jobs[j] & 255;
        const int n_here = min(kPageTokens, seg_last[sg] + 1 - pg * kPageTokens);
        const uint16_t *src = a.kv_layer + (((size_t)job_ph[j] * 2 + part) * a.H + h) * kPageElems;
        pt_stage(slots + (size_t)(j % kPtSlots) * 16384 + part * (kPageElems * 2), src, n_here, lane);
      } else {
        pt_commit();   // an empty group keeps the count of groups per job uniform
      }
    };
    stage(0); stage(1); stage(2);
    pt_wait_but<2>();            // page 0 has landed
    fence_proxy_async_smem();    // the tensor core reads the slots through the async proxy
    __syncwarp();
    if (lane == 0 && n_job > 0) mbar_arrive(page_full);
    for (int i = 0; i < n_job; ++i) {
      // page i + 3 goes into the slot page i - 3 used, free once P V of job i - 3 has completed
      if (i >= 3) {
        if (lane == 0) tc_wait(pv_done + ((i - 3) & 1), (uint32_t)((i - 3) >> 1) & 1u, failed, a.err);
        __syncwarp();
      }
      stage(i + 3);
      pt_wait_but<2>();            // everything but the two groups just committed: page i + 1 has landed
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0 && i + 1 < n_job) mbar_arrive(page_full + (i + 1) % kPtSlots);
    }
  } else if (warp == 8) {
    // ---- one thread issues the instructions to the tensor core ----
    if (lane == 0) {
      const uint32_t idesc_qk = tc_instr_desc(kPtRows, 64);
      const uint32_t idesc_pv = tc_instr_desc(kPtRows, 64) | (1u << 16);   // B (= V) is MN-major: token rows of 64 dimensions
      auto qk = [&](int j) {   // S of group j % 2 = Q K^T for job j; that group holds S of its job before in registers
        const int g = j & 1, k = j >> 1;
        tc_wait(page_full + j % kPtSlots, (uint32_t)(j / kPtSlots) & 1u, failed, a.err);
        if (k > 0) tc_wait(s_free + g, (uint32_t)(k - 1) & 1u, failed, a.err);
        tc_fence_after_sync();
        const uint64_t dq = tc_smem_desc(Qs), dk = tc_smem_desc(slots + (size_t)(j % kPtSlots) * 16384);
#pragma unroll
        for (int q = 0; q < 4; ++q) tc_mma(tmem + 64u * g, dq + 2 * q, dk + 2 * q, idesc_qk, q == 0 ? 0u : 1u);   // 16 dimensions per instruction
        tc_commit(s_full + g);
      };
      auto pv = [&](int j) {   // O of group j % 2 (+)= P V for job j
        const int g = j & 1, k = j >> 1;
        tc_wait(p_full + g, (uint32_t)k & 1u, failed, a.err);
        tc_fence_after_sync();
        const uint64_t dp = tc_smem_desc(Ps + g * 16384), dv = tc_smem_desc(slots + (size_t)(j % kPtSlots) * 16384 + kPageElems * 2);
#pragma unroll
        for (int q = 0; q < 4; ++q)   // 16 tokens per instruction: 32 bytes along a P row, two 8-row groups (2048 bytes) down V
          tc_mma(tmem + 128u + 64u * g, dp + 2 * q, dv + 128 * q, idesc_pv, (k == 0 && q == 0) ? 0u : 1u);
        tc_commit(pv_done + g);
      };
      tc_wait(q_full, 0, failed, a.err);
      if (n_job > 0) qk(0);
      for (int i = 0; i < n_job; ++i) {
        // Q K^T runs a job ahead of the softmax groups: S of job i + 1 is under way before this thread blocks on P of
        // job i - 1, so a group finds its next S complete when it has handed over its P
        if (i + 1 < n_job) qk(i + 1);
        if (i > 0) pv(i - 1);
      }
      if (n_job > 0) pv(n_job - 1);
    }
    __syncwarp();
  } else {
    // ---- softmax: group g = warps 4 g .. 4 g + 3 takes jobs g, g + 2, ...; thread t of a group owns row t = accumulator
    //      lane t, with the group's own S, P and O; the two partial results meet at the end ----
    const int g = warp >> 2, t = threadIdx.x & (kPtRows - 1), r = r0 + t;
    const uint32_t t_lane = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
    const uint32_t t_S = t_lane + 64u * g, t_O = t_lane + 128u + 64u * g;
    unsigned char *Pg = Ps + g * 16384;
    if (g == 0) {
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
    int k = 0;
    for (int j = g; j < n_job; j += 2, ++k) {
      pt_warp_wait(s_full + g, (uint32_t)k & 1u, failed, a.err, lane);
      tc_fence_after_sync();
      float s[64];
      {
        float lo[32], hi[32];
        tmem_ld32(t_S, lo);
        tmem_ld32(t_S + 32u, hi);
#pragma unroll
        for (int c = 0; c < 32; ++c) { s[c] = lo[c]; s[32 + c] = hi[c]; }
      }
      tc_fence_before_sync();
      mbar_arrive(s_free + g);
      const int sg = jobs[j] >> 8, pg = jobs[j] & 255;
      const bool act = r >= seg_i0[sg] && r < seg_i1[sg];
      const int see = act ? min(kPageTokens, pos + 1 - pg * kPageTokens) : 0;   // tokens of the page this row sees
      // all but the last page of a row's own stream are seen whole by every row of the warp: no masks there
      if (!__all_sync(0xFFFFFFFFu, see == kPageTokens)) {
#pragma unroll
        for (int c = 0; c < 64; ++c) s[c] = c < see ? s[c] : -INFINITY;
      }
      // four independent chains for the maximum and for the sum: one chain of 64 dependent operations per row and
      // page was the longest thing in the loop.  The scale (positive) is applied to the maximum and inside the
      // exponential's argument: one multiply-add per score.
      float pm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < 64; ++c) pm4[c & 3] = fmaxf(pm4[c & 3], s[c]);
      const float pm = fmaxf(fmaxf(pm4[0], pm4[1]), fmaxf(pm4[2], pm4[3])) * qs;
      const float m_new = fmaxf(m, pm);
      const float ref = (m_new == -INFINITY) ? 0.f : m_new;   // a row that has seen nothing yet keeps m = -inf
      const float sc = pt_exp2(m - ref);
      m = m_new;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < 64; ++c) { s[c] = pt_exp2(fmaf(s[c], qs, -ref)); sum4[c & 3] += s[c]; }
      const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      l = l * sc + sum;
      // the group's P and O belong to the tensor core until P V of the group's job before has completed
      if (k > 0) { pt_warp_wait(pv_done + g, (uint32_t)(k - 1) & 1u, failed, a.err, lane); tc_fence_after_sync(); }
#pragma unroll
      for (int c8 = 0; c8 < 8; ++c8)
        *reinterpret_cast<uint4 *>(Pg + t * 128 + ((c8 ^ (t & 7)) << 4)) =
            make_uint4(pack_bf16x2(s[8 * c8], s[8 * c8 + 1]), pack_bf16x2(s[8 * c8 + 2], s[8 * c8 + 3]),
                       pack_bf16x2(s[8 * c8 + 4], s[8 * c8 + 5]), pack_bf16x2(s[8 * c8 + 6], s[8 * c8 + 7]));
      __syncwarp();
      if (k > 0 && !__all_sync(0xFFFFFFFFu, sc == 1.0f)) {   // some row's maximum moved: rescale the warp's rows of O
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          float o[32];
          tmem_ld32(t_O + 32u * hh, o);
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] *= sc;
          tmem_st32(t_O + 32u * hh, o);
        }
      }
      fence_proxy_async_smem();
      tc_fence_before_sync();
      mbar_arrive(p_full + g);
    }
    trace_mark(a.trace, a.trace_slot, 3);
    // ---- the two groups' partial results: O = (O0 2^(m0 - M) + O1 2^(m1 - M)) / (l0 2^(m0 - M) + l1 2^(m1 - M)) ----
    if (k > 0) { pt_warp_wait(pv_done + g, (uint32_t)(k - 1) & 1u, failed, a.err, lane); tc_fence_after_sync(); }
    if (g == 1) {
      ref1_s[t] = m; l1_s[t] = l;   // without a job of its own: m = -inf, l = 0, and Ms is not read
      if (k > 0) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          float o[32];
          tmem_ld32(t_O + 32u * hh, o);
#pragma unroll
          for (int c = 0; c < 32; ++c) Ms[t * kPtMergePitch + 32 * hh + c] = o[c];
        }
      }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(2 * kPtRows) : "memory");   // every softmax thread, once
    if (g == 0 && n_job > 0) {
      const float m1 = ref1_s[t], l1 = l1_s[t];
      const float M = fmaxf(m, m1);
      const float a0 = (m == -INFINITY) ? 0.f : pt_exp2(m - M), a1 = (m1 == -INFINITY) ? 0.f : pt_exp2(m1 - M);
      const float lt = l * a0 + l1 * a1;
      const float inv = lt > 0.f ? 1.0f / lt : 0.f;
      const float w0 = a0 * inv, w1 = a1 * inv;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        float o[32];
        tmem_ld32(t_O + 32u * hh, o);
        if (a1 != 0.f) {
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = o[c] * w0 + Ms[t * kPtMergePitch + 32 * hh + c] * w1;
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] *= w0;
        }
        if (r < R && !*failed) {
#pragma unroll
          for (int c8 = 0; c8 < 4; ++c8) {
            const uint4 y = make_uint4(pack_bf16x2(o[8 * c8], o[8 * c8 + 1]), pack_bf16x2(o[8 * c8 + 2], o[8 * c8 + 3]),
                                       pack_bf16x2(o[8 * c8 + 4], o[8 * c8 + 5]), pack_bf16x2(o[8 * c8 + 6], o[8 * c8 + 7]));
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
  if (warp == 8) tmem_dealloc(tmem, 256);
}

inline size_t attention_prefill_tc_smem_bytes() { return 49152 + (size_t)kPtSlots * 16384 + (size_t)kPtRows * kPtMergePitch * 4 + 1024 + 256; }

inline cudaError_t launch_attention_prefill_tc(const AttnArgs &a, int R, cudaStream_t st, bool pdl) {
  static PerDeviceOnce attr_once;   // per device: opt-in to more than 48 KB of dynamic shared memory
  if (attr_once.first())
    cudaFuncSetAttribute(attention_prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attention_prefill_tc_smem_bytes());
  const int groups = (R + kPtRows - 1) / kPtRows;
  return launch_kernel(attention_prefill_tc_kernel, dim3(1, a.H, groups), dim3(kPtThreads), attention_prefill_tc_smem_bytes(), st, pdl, a, R);
}

}  // namespace ttsgpt
