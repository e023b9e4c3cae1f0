// Weight-only dequantizing linear (Table I caption: W8A16 / W4A16 applied to the GPT; bf16 is the
// unquantized case): out[b,n] = sum_k W[n,k] act[b,k] (+ bias, + epilogue), bf16 activations,
// fp32 accumulation, optional LayerNorm of the fp32 input fused in front.
//
// Streaming layout.  At engine creation every [N,K] matrix is re-laid into 512-byte tiles of 8
// output rows x KT columns (KT = 32 bf16 / 64 int8 / 128 int4), stored tile after tile as
// [row-tile][k-tile].  Inside a tile lane (g,t) = (lane/4, lane%4) owns the 16 bytes of row g that
// cover columns t*KT/4 .. +KT/4-1: one coalesced 128-bit load per lane fetches a tile in the order
// the warp-level MMA wants its 8-wide operand.  The batch is the 16-wide M operand (rows 0..15 of
// an m-tile), the 8 weight rows the N operand; int8 / int4 codes are widened to bf16 integers in
// registers (exact) and the bf16 scale multiplies the fp32 partial sums (per row for int8, per row
// and 128-column group for int4).
//
// A CTA owns 1, 2 or 4 adjacent 8-row tiles (one contiguous block of the streaming layout) and
// splits K over its 10 warps.  Its very first action is one bulk asynchronous copy (TMA, untiled,
// completion on an mbarrier) of that whole block into shared memory: weights do not depend on the
// previous kernel, so under programmatic dependent launch the copy overlaps the predecessor's
// tail and occupies no registers.  Only then does the CTA wait for its predecessor, stage (or
// layer-normalise) the activation rows, wait for the weights (bounded wait, error word on
// expiry), form the products — fp32 FMAs for up to 4 batch rows, the tensor pipe above — and the
// warps' partial sums meet in shared memory in warp order (results do not depend on timing).
// Batches above 16 loop over m-tiles re-using the weights in shared memory.
#pragma once
#include "common.cuh"
#include "elementwise.cuh"

namespace ttsgpt {

enum { WF_BF16 = 0, WF_INT8 = 1, WF_INT4 = 2 };
enum { EPI_F32 = 0, EPI_QKV = 1, EPI_RESID = 2, EPI_GELU = 3 };

constexpr int kLinearWarps = 10;  // divides the k-tile counts of K=1280 and K=5120 in every format
constexpr int kLinearThreads = kLinearWarps * 32;
constexpr int kSmallKSplit = 4;     // k-ranges of FC2 between 5 and 16 rows (partial sums folded by the next LayerNorm)
constexpr int kLnFuseMaxRows = 4;   // LayerNorm is fused into the linear up to this batch: every CTA repeats
                                    // it, which beats a separate launch only while the rows are few

__host__ __device__ inline int k_per_tile(int wf) { return wf == WF_BF16 ? 32 : (wf == WF_INT8 ? 64 : 128); }
__host__ __device__ inline int row_tiles(int N) { return (N + 7) / 8; }
// bytes of the tiled weights / of the tiled scales
inline size_t packed_weight_bytes(int wf, int N, int K) { return (size_t)row_tiles(N) * (K / k_per_tile(wf)) * 512; }
inline size_t packed_scale_bytes(int wf, int N, int K) {
  if (wf == WF_INT8) return (size_t)row_tiles(N) * 8 * 2;
  if (wf == WF_INT4) return (size_t)row_tiles(N) * (K / 128) * 8 * 2;
  return 0;
}

// ------------------------------------------------------------------------------------------
// canonical -> streaming re-layout (run once at creation).  One thread per 16-byte unit.
// ------------------------------------------------------------------------------------------
__global__ void pack_bf16_kernel(const uint16_t *__restrict__ w, int N, int K, uint4 *__restrict__ dst) {
  const int KB = K / 32;
  size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (unit >= (size_t)row_tiles(N) * KB * 32) return;
  const int lane = unit & 31;
  const size_t tile = unit >> 5;
  const int kb = tile % KB, rt = tile / KB;
  const int row = rt * 8 + (lane >> 2), k = kb * 32 + 8 * (lane & 3);
  uint4 v = make_uint4(0, 0, 0, 0);
  if (row < N) v = *reinterpret_cast<const uint4 *>(w + (size_t)row * K + k);
  dst[unit] = v;
}

// int8 codes are stored biased (u = q + 128) so that one byte-permute drops them into the mantissa
// of a float magic number.
__global__ void pack_int8_kernel(const int8_t *__restrict__ w, int N, int K, uint4 *__restrict__ dst) {
  const int KB = K / 64;
  size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (unit >= (size_t)row_tiles(N) * KB * 32) return;
  const int lane = unit & 31;
  const size_t tile = unit >> 5;
  const int kb = tile % KB, rt = tile / KB;
  const int row = rt * 8 + (lane >> 2), k = kb * 64 + 16 * (lane & 3);
  uint4 v = make_uint4(0x80808080u, 0x80808080u, 0x80808080u, 0x80808080u);
  if (row < N) {
    v = *reinterpret_cast<const uint4 *>(w + (size_t)row * K + k);
    v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u;
  }
  dst[unit] = v;
}

// Canonical word: nibble j holds column 8w+j.  Streaming word: columns (0,1) sit in nibbles (0,4),
// (2,3) in (1,5), (4,5) in (2,6), (6,7) in (3,7), so that (word >> 4e) & 0x000F000F yields the
// pair of adjacent columns (2e, 2e+1) in the low / high half-words.
__device__ __forceinline__ uint32_t permute_nibbles(uint32_t c) {
  uint32_t r = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t nib = (c >> (4 * j)) & 15u;
    const int pos = (j >> 1) + 4 * (j & 1);
    r |= nib << (4 * pos);
  }
  return r;
}
__global__ void pack_int4_kernel(const uint32_t *__restrict__ w, int N, int K, uint4 *__restrict__ dst) {
  const int KB = K / 128;
  size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (unit >= (size_t)row_tiles(N) * KB * 32) return;
  const int lane = unit & 31;
  const size_t tile = unit >> 5;
  const int kb = tile % KB, rt = tile / KB;
  const int row = rt * 8 + (lane >> 2), k = kb * 128 + 32 * (lane & 3);
  uint4 v = make_uint4(0x88888888u, 0x88888888u, 0x88888888u, 0x88888888u);
  if (row < N) {
    const uint4 c = *reinterpret_cast<const uint4 *>(w + (size_t)row * (K / 8) + k / 8);
    v = make_uint4(permute_nibbles(c.x), permute_nibbles(c.y), permute_nibbles(c.z), permute_nibbles(c.w));
  }
  dst[unit] = v;
}
// scales: int8 [N] -> [rt][8]; int4 [N][K/128] -> [rt][kb][8]; padding rows get 0
__global__ void pack_scales_kernel(const uint16_t *__restrict__ s, int N, int G, uint16_t *__restrict__ dst) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)row_tiles(N) * G * 8) return;
  const int r = i & 7;
  const size_t t = i >> 3;
  const int g = t % G, rt = t / G;
  const int row = rt * 8 + r;
  dst[i] = row < N ? s[(size_t)row * G + g] : (uint16_t)0;
}

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------
struct LinearArgs {
  const void *w;          // tiled weights
  const uint16_t *scales; // tiled scales (int8 / int4) or null
  const uint16_t *bias;   // bf16 [N] or null
  const uint16_t *act;    // bf16 [B][K]  (unused when ln_x is set)
  int N, K, B, mode;
  // fused LayerNorm in front (B <= kLnFuseMaxRows, K <= kLnFuseMaxK): act = LN(ln_x[gather[b]])
  const float *ln_x;      // fp32 [*][K] or null
  const uint16_t *ln_g, *ln_b;
  float ln_eps;
  const int *ln_gather;   // optional row indices into ln_x
  const int *ln_out_slot; // with ln_io: row of io->out_hidden that receives LN row b
  const StepIO *ln_io;    // optional: CTA 0 also writes the LN rows to io->out_hidden
  float *out_f32;         // EPI_F32: out[b*out_stride+n] = v ; EPI_RESID: out[b*out_stride+n] += v ; EPI_QKV: q
  int out_stride;
  uint16_t *out_bf16;     // EPI_GELU: h[b*N+n] = bf16(gelu(v))
  int gelu_tanh;
  // EPI_QKV: rows [0,d) -> q (fp32), [d,2d) -> K pages, [2d,3d) -> V pages
  uint16_t *kv_layer;
  uint16_t *kv_stage;         // if set, K/V rows go here as bf16 [B][2][d] instead of into their page slots (8-bit KV cache)
  const int *page_table, *row_stream, *row_pos;
  int pps, d, H;
  unsigned long long *trace;  // optional timeline trace (see trace_mark)
  int trace_slot;
  int *err;                   // optional device error word: set to 1 if the weight copy never arrives
  int ksplit;                 // 0 or 1: whole K per CTA; n > 1 (EPI_RESID only, no fused LN): gridDim.y = n k-ranges,
                              // out_f32 = partial sums [n][kMaxRows][N] without bias, folded by the next LayerNorm
};

// exact int8 (biased byte) -> float via the 2^23 magic number
__device__ __forceinline__ float biased_byte_to_float(uint32_t word, int i) {
  const uint32_t m = __byte_perm(word, 0x4B000000u, 0x7540u | (uint32_t)i);
  return __uint_as_float(m) - 8388736.0f;  // 2^23 + 128
}
// exact int4 pair (two nibbles in the low bits of each half-word) -> bf16x2 of (u - 8)
__device__ __forceinline__ uint32_t nib_pair_to_bf16x2(uint32_t masked) {
  uint32_t m = masked | 0x43004300u;  // bf16 128 + u
  __nv_bfloat162 v = *reinterpret_cast<__nv_bfloat162 *>(&m);
  const uint32_t c136 = 0x43084308u;
  v = __hsub2(v, *reinterpret_cast<const __nv_bfloat162 *>(&c136));
  return *reinterpret_cast<uint32_t *>(&v);
}

// row stride (in bf16 elements) of the LayerNorm staging buffer; the odd multiple of 16 bytes keeps
// the 8 batch rows of a fragment load on different banks
__host__ __device__ inline int ln_stage_stride(int wf, int K) { return K + (wf == WF_BF16 ? 32 : 8); }

// MODE: how the activation fragments are obtained
//   ACT_DIRECT  bf16 activations read from global memory, a few k-tiles at a time (large B*K)
//   ACT_STAGED  bf16 activations copied to shared memory first (one round trip for the whole CTA)
//   ACT_LN      fp32 rows layer-normalised into shared memory first
enum { ACT_DIRECT = 0, ACT_STAGED = 1, ACT_LN = 2 };
constexpr int kStageMaxBytes = 44 * 1024;
constexpr int kLinearSmemBudget = 108 * 1024;  // per CTA, so that two CTAs share an SM

// NB: 0 = tensor-pipe path (any batch, 16 rows per m-tile); 1 or 4 = CUDA-core path for batches of
// at most NB rows.  On this part one warp-level MMA occupies the tensor pipe of its SM partition
// for about 32 cycles whatever the number of real batch rows, so below 5 rows plain fp32 FMAs on
// the widened weights are cheaper.
template <int WF, int RT, int MODE, int NB>
__global__ void __launch_bounds__(kLinearThreads, 2) linear_kernel(const LinearArgs a) {
  constexpr bool LN = MODE == ACT_LN;
  constexpr bool STAGED = MODE != ACT_DIRECT;
  constexpr int KT = WF == WF_BF16 ? 32 : (WF == WF_INT8 ? 64 : 128);
  constexpr int AW = KT / 32;  // uint4 activation loads per lane, k-tile and batch row
  constexpr int C = 8 * RT;    // output columns (weight rows) of this CTA
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int KBG = a.K / KT;                          // k-tiles of the whole matrix
  const int KB = KBG / (int)gridDim.y;               // k-tiles of this CTA's k-range
  const int kb_off = (int)blockIdx.y * KB;           // its first k-tile
  const int tile0 = blockIdx.x * RT, n_rt = row_tiles(a.N);
  trace_mark(a.trace, a.trace_slot, 0);

  // shared memory: [barrier | weights RT*KB*512 | int4 scales RT*KB*16 | partial sums | activation rows]
  extern __shared__ __align__(128) unsigned char smem_raw[];
  uint64_t *wbar = reinterpret_cast<uint64_t *>(smem_raw);
  unsigned char *wsm = smem_raw + 128;
  uint16_t *ssm = reinterpret_cast<uint16_t *>(wsm + (size_t)RT * KB * 512);
  float *red = reinterpret_cast<float *>(wsm + (size_t)RT * KB * (WF == WF_INT4 ? 528 : 512));  // [warps][16][C]
  uint16_t *stage = reinterpret_cast<uint16_t *>(red + kLinearWarps * 16 * C);

  // ---- the CTA's weights (contiguous in the streaming layout) start moving into shared memory
  //      before anything else: they do not depend on the previous kernel ----
  if (threadIdx.x == 0) {
    const int n_valid = min(RT, n_rt - tile0);
    const uint32_t wbytes = (uint32_t)n_valid * KB * 512u;
    const uint32_t sbytes = WF == WF_INT4 ? (uint32_t)n_valid * KB * 16u : 0u;
    mbar_init(wbar, 1);
    mbar_expect_tx(wbar, wbytes + sbytes);
    if (gridDim.y == 1) {   // all of K: the CTA's tiles are one contiguous range
      const unsigned char *gw = reinterpret_cast<const unsigned char *>(a.w) + (size_t)tile0 * KB * 512;
      for (uint32_t off = 0; off < wbytes; off += 32768u)
        bulk_copy_g2s(wsm + off, gw + off, min(32768u, wbytes - off), wbar);
      if (sbytes) bulk_copy_g2s(ssm, a.scales + (size_t)tile0 * KB * 8, sbytes, wbar);
    } else {                // a k-range: one contiguous piece per row tile
      for (int j = 0; j < n_valid; ++j) {
        const unsigned char *gw = reinterpret_cast<const unsigned char *>(a.w) + ((size_t)(tile0 + j) * KBG + kb_off) * 512;
        const uint32_t tb = (uint32_t)KB * 512u;
        for (uint32_t off = 0; off < tb; off += 32768u)
          bulk_copy_g2s(wsm + (size_t)j * tb + off, gw + off, min(32768u, tb - off), wbar);
        if (sbytes) bulk_copy_g2s(ssm + (size_t)j * KB * 8, a.scales + ((size_t)(tile0 + j) * KBG + kb_off) * 8, (uint32_t)KB * 16u, wbar);
      }
    }
  }

  // ---- everything else that no kernel of the step writes: LN gamma/beta, bias, scales, KV slots ----
  const int ecol = threadIdx.x % C;             // this thread's output column in every epilogue round
  const int en = tile0 * 8 + ecol;              // = output feature n
  float e_bias = 0.f, e_scale = 1.f;
  if (en < a.N) {
    if (a.bias) e_bias = bf16_bits_to_float(a.bias[en]);
    if (WF == WF_INT8) e_scale = bf16_bits_to_float(a.scales[en]);
  }
  // EPI_QKV: where this thread's K/V outputs go (row table and page table are final before the
  // first kernel of the step starts); batches above 16 rows look the slot up in the epilogue
  constexpr int ER = (16 * C + kLinearThreads - 1) / kLinearThreads;  // epilogue rounds
  uint16_t *kv_dst[ER];
#pragma unroll
  for (int e = 0; e < ER; ++e) {
    kv_dst[e] = nullptr;
    const int b = (threadIdx.x + e * kLinearThreads) / C;
    if (a.mode == EPI_QKV && en >= a.d && en < a.N && b < a.B && b < 16) {
      const int which = en >= 2 * a.d;  // 0 = K, 1 = V
      const int col = en - (which ? 2 * a.d : a.d);
      if (a.kv_stage) {
        kv_dst[e] = a.kv_stage + ((size_t)b * 2 + which) * a.d + col;
      } else {
        const int pos = a.row_pos[b];
        const int page = a.page_table[(size_t)a.row_stream[b] * a.pps + (pos >> 6)];
        kv_dst[e] = a.kv_layer + (((size_t)page * 2 + which) * a.H + (col >> 6)) * kPageElems +
                    (size_t)(pos & 63) * kHeadDim + (col & 63);
      }
    }
  }
  uint2 ln_gg = make_uint2(0, 0), ln_bb = make_uint2(0, 0);
  const int lc = threadIdx.x * 4;               // fused LN: this thread's 4 columns (K <= 1280)
  if (LN && lc < a.K) {
    ln_gg = *reinterpret_cast<const uint2 *>(a.ln_g + lc);
    ln_bb = *reinterpret_cast<const uint2 *>(a.ln_b + lc);
  }
  pdl_launch_dependents();
  pdl_wait();
  trace_mark(a.trace, a.trace_slot, 1);

  // ---- optional fused LayerNorm: the CTA splits each row over all threads (4 columns each) and
  //      handles up to RPR rows per round.  Each thread forms the mean and the centered sum of
  //      squares of its 4 values; (mean, M2) pairs of equal weight are then merged pairwise
  //      (mean = (ma+mb)/2, M2 = M2a + M2b + (mb-ma)^2 * n/2), first by shuffles, then across the
  //      warps through shared memory: one block barrier, no cancellation.
  const int stride = ln_stage_stride(WF, KB * KT);   // staged columns: this CTA's k-range
  constexpr int RPR = NB == 1 ? 1 : 4;  // rows per LayerNorm round (a one-row launch carries the code of one row only)
  if (LN) {
    float2 *lnred = reinterpret_cast<float2 *>(red);  // [warps][RPR] (mean, M2), reused later for the partial sums
    const int nw_used = (a.K / 4 + 31) / 32;           // warps that hold columns (K is a multiple of 128)
    const float inv_nw = 1.0f / nw_used, inv_k = 1.0f / a.K;
    for (int b0 = 0; b0 < a.B; b0 += RPR) {
      float4 xv[RPR];
      float mean[RPR], m2[RPR];
#pragma unroll
      for (int r = 0; r < RPR; ++r) {
        xv[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        const int b = b0 + r;
        if (b < a.B && lc < a.K) {
          const int src = a.ln_gather ? a.ln_gather[b] : b;
          xv[r] = *reinterpret_cast<const float4 *>(a.ln_x + (size_t)src * a.K + lc);
        }
      }
#pragma unroll
      for (int r = 0; r < RPR; ++r) {
        mean[r] = 0.f; m2[r] = 0.f;
        if (b0 + r >= a.B) break;
        mean[r] = 0.25f * ((xv[r].x + xv[r].y) + (xv[r].z + xv[r].w));
        const float d0 = xv[r].x - mean[r], d1 = xv[r].y - mean[r], d2 = xv[r].z - mean[r], d3 = xv[r].w - mean[r];
        m2[r] = (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
        float cnt = 4.f;  // values behind each side of a merge
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const float mb = __shfl_xor_sync(0xFFFFFFFFu, mean[r], o);
          const float qb = __shfl_xor_sync(0xFFFFFFFFu, m2[r], o);
          const float dl = mb - mean[r];
          m2[r] = m2[r] + qb + dl * dl * (0.5f * cnt);
          mean[r] = 0.5f * (mean[r] + mb);
          cnt *= 2.f;
        }
      }
      {  // lane r publishes row r (every lane holds every row's warp-level result)
        float mm = mean[0], qq = m2[0];
#pragma unroll
        for (int r = 1; r < RPR; ++r) { mm = lane == r ? mean[r] : mm; qq = lane == r ? m2[r] : qq; }
        if (lane < RPR) lnred[warp * RPR + lane] = make_float2(mm, qq);
      }
      __syncthreads();
#pragma unroll
      for (int r = 0; r < RPR; ++r) {
        const int b = b0 + r;
        if (b >= a.B) break;
        // merge of the warps' (mean, M2), each over 128 values: the grand mean is the mean of the
        // warp means, M2 = sum M2_w + 128 * sum (mean_w - mean)^2
        float msum = 0.f;
        for (int w = 0; w < nw_used; ++w) msum += lnred[w * RPR + r].x;
        const float mu = msum * inv_nw;
        float m2t = 0.f;
        for (int w = 0; w < nw_used; ++w) {
          const float2 o2 = lnred[w * RPR + r];
          const float dl = o2.x - mu;
          m2t += o2.y + 128.f * dl * dl;
        }
        const float rstd = rsqrtf(m2t * inv_k + a.ln_eps);
        if (lc < a.K) {
          uint2 y;
          y.x = pack_bf16x2((xv[r].x - mu) * rstd * bf16_lo(ln_gg.x) + bf16_lo(ln_bb.x),
                            (xv[r].y - mu) * rstd * bf16_hi(ln_gg.x) + bf16_hi(ln_bb.x));
          y.y = pack_bf16x2((xv[r].z - mu) * rstd * bf16_lo(ln_gg.y) + bf16_lo(ln_bb.y),
                            (xv[r].w - mu) * rstd * bf16_hi(ln_gg.y) + bf16_hi(ln_bb.y));
          *reinterpret_cast<uint2 *>(stage + (size_t)b * stride + lc) = y;
          if (blockIdx.x == 0 && a.ln_io && a.ln_io->out_hidden)
            *reinterpret_cast<uint2 *>(a.ln_io->out_hidden + (size_t)(a.ln_out_slot ? a.ln_out_slot[b] : b) * a.K + lc) = y;
        }
      }
      __syncthreads();
    }
  } else if (MODE == ACT_STAGED) {
    const int k8 = (KB * KT) >> 3;
    const uint16_t *src = a.act + (size_t)kb_off * KT;
    for (int idx = threadIdx.x; idx < a.B * k8; idx += kLinearThreads) {
      const int b = idx / k8, c8 = idx - b * k8;
      *reinterpret_cast<uint4 *>(stage + (size_t)b * stride + 8 * c8) =
          *reinterpret_cast<const uint4 *>(src + (size_t)b * a.K + 8 * c8);
    }
    __syncthreads();
  } else {
    __syncthreads();  // the barrier's initialisation by thread 0 must be visible before anyone polls it
  }
  trace_mark(a.trace, a.trace_slot, 3);

  // ---- the weights must have landed by now (they were requested before the dependency wait) ----
  if (!mbar_wait_bounded(wbar, 0, 2000000000ull)) {
    if (a.err) atomicExch(a.err, 1);
    // give the copies still in flight towards this CTA's shared memory a last chance to finish
    mbar_wait_bounded(wbar, 0, 2000000000ull);
    return;
  }
  const uint4 *wtile = reinterpret_cast<const uint4 *>(wsm);   // tile (j, kb) at ((j*KB + kb)*32 + lane)
  trace_mark(a.trace, a.trace_slot, 6);

  for (int m0 = 0; m0 < a.B; m0 += 16) {
    // the residual's old value, fetched while the products run
    float e_old[ER];
#pragma unroll
    for (int e = 0; e < ER; ++e) {
      e_old[e] = 0.f;
      const int o = threadIdx.x + e * kLinearThreads;
      const int b = m0 + o / C;
      if (a.mode == EPI_RESID && gridDim.y == 1 && o < 16 * C && b < a.B && en < a.N) e_old[e] = a.out_f32[(size_t)b * a.out_stride + en];
    }
    if (NB > 0) {
      // ---- CUDA-core path: lane (g,t) multiplies its 16 bytes of weight row g with the matching
      //      activation columns of up to NB batch rows; the 4 lanes of a row meet by shuffles ----
      constexpr int NBA = NB > 0 ? NB : 1;  // array extent (the branch is dead for NB == 0)
      float facc[RT][NBA];
#pragma unroll
      for (int j = 0; j < RT; ++j)
#pragma unroll
        for (int b = 0; b < NBA; ++b) facc[j][b] = 0.f;
#pragma unroll 1   // small code matters more than overlap here: a one-row step executes most instructions once, and fetching them costs about what executing them does
      for (int kb = warp; kb < KB; kb += kLinearWarps) {
        const int col = kb * KT + t * (KT / 4);
        uint4 wq[RT];
#pragma unroll
        for (int j = 0; j < RT; ++j) wq[j] = wtile[((size_t)j * KB + kb) * 32 + lane];
        float tacc[RT][NBA];  // int4: sums of one 128-column group, scaled afterwards
        if (WF == WF_INT4) {
#pragma unroll
          for (int j = 0; j < RT; ++j)
#pragma unroll
            for (int b = 0; b < NBA; ++b) tacc[j][b] = 0.f;
        }
#pragma unroll
        for (int q = 0; q < AW; ++q) {
          float xf[NBA][8];
#pragma unroll
          for (int b = 0; b < NBA; ++b) {
            uint4 xv = make_uint4(0, 0, 0, 0);
            if (b < a.B) xv = *reinterpret_cast<const uint4 *>(stage + (size_t)b * stride + col + 8 * q);
            xf[b][0] = bf16_lo(xv.x); xf[b][1] = bf16_hi(xv.x); xf[b][2] = bf16_lo(xv.y); xf[b][3] = bf16_hi(xv.y);
            xf[b][4] = bf16_lo(xv.z); xf[b][5] = bf16_hi(xv.z); xf[b][6] = bf16_lo(xv.w); xf[b][7] = bf16_hi(xv.w);
          }
#pragma unroll
          for (int j = 0; j < RT; ++j) {
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
#pragma unroll
            for (int b = 0; b < NBA; ++b) {
              // two independent chains of four products keep the FMA pipe busy
              float s0 = (WF == WF_INT4) ? tacc[j][b] : facc[j][b];
              float s1 = wv[4] * xf[b][4];
              s0 = fmaf(wv[0], xf[b][0], s0); s1 = fmaf(wv[5], xf[b][5], s1);
              s0 = fmaf(wv[1], xf[b][1], s0); s1 = fmaf(wv[6], xf[b][6], s1);
              s0 = fmaf(wv[2], xf[b][2], s0); s1 = fmaf(wv[7], xf[b][7], s1);
              s0 = fmaf(wv[3], xf[b][3], s0);
              s0 += s1;
              if (WF == WF_INT4) tacc[j][b] = s0; else facc[j][b] = s0;
            }
          }
        }
        if (WF == WF_INT4) {
#pragma unroll
          for (int j = 0; j < RT; ++j) {
            const float sc = bf16_bits_to_float(ssm[((size_t)j * KB + kb) * 8 + g]);  // this lane's row
#pragma unroll
            for (int b = 0; b < NBA; ++b) facc[j][b] = fmaf(sc, tacc[j][b], facc[j][b]);
          }
        }
      }
      trace_mark(a.trace, a.trace_slot, 4);
#pragma unroll
      for (int j = 0; j < RT; ++j)
#pragma unroll
        for (int b = 0; b < NBA; ++b) {
          float v = facc[j][b];
          v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
          v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
          if (t == 0) red[((size_t)warp * 16 + b) * C + 8 * j + g] = v;
        }
    } else {
      // ---- tensor-pipe path: the batch is the 16-row M operand, the 8 weight rows the N operand ----
      float acc[RT][4];
#pragma unroll
      for (int j = 0; j < RT; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
      const int r0 = m0 + g, r1 = m0 + g + 8;
      const uint16_t *row0 = STAGED ? stage + (size_t)r0 * stride : a.act + (size_t)r0 * a.K + (size_t)kb_off * KT;
      const uint16_t *row1 = STAGED ? stage + (size_t)r1 * stride : a.act + (size_t)r1 * a.K + (size_t)kb_off * KT;
      const bool v0 = r0 < a.B, v1 = r1 < a.B;
      // activation fragments: G k-tiles are fetched together so that their latencies overlap
      constexpr int G = STAGED ? 1 : 8 / AW;   // up to 64 registers of activation fragments in flight
      for (int kb0 = warp; kb0 < KB; kb0 += G * kLinearWarps) {
        uint4 xg0[G][AW], xg1[G][AW];
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
          const int kb = kb0 + gi * kLinearWarps;
          const int col = kb * KT + t * (KT / 4);
#pragma unroll
          for (int q = 0; q < AW; ++q) {
            xg0[gi][q] = (v0 && kb < KB) ? *reinterpret_cast<const uint4 *>(row0 + col + 8 * q) : make_uint4(0, 0, 0, 0);
            xg1[gi][q] = (v1 && kb < KB) ? *reinterpret_cast<const uint4 *>(row1 + col + 8 * q) : make_uint4(0, 0, 0, 0);
          }
        }
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
          const int kb = kb0 + gi * kLinearWarps;
          if (kb < KB) {
            const uint4 *x0 = xg0[gi], *x1 = xg1[gi];
#pragma unroll
            for (int j = 0; j < RT; ++j) {
              const uint4 wq = wtile[((size_t)j * KB + kb) * 32 + lane];
              const uint32_t ww[4] = {wq.x, wq.y, wq.z, wq.w};
              if (WF == WF_BF16) {
                mma_bf16_16816(acc[j], x0[0].x, x1[0].x, x0[0].y, x1[0].y, ww[0], ww[1]);
                mma_bf16_16816(acc[j], x0[0].z, x1[0].z, x0[0].w, x1[0].w, ww[2], ww[3]);
              } else if (WF == WF_INT8) {
#pragma unroll
                for (int s = 0; s < 4; ++s) {
                  const uint32_t b0 = pack_bf16x2(biased_byte_to_float(ww[s], 0), biased_byte_to_float(ww[s], 1));
                  const uint32_t b1 = pack_bf16x2(biased_byte_to_float(ww[s], 2), biased_byte_to_float(ww[s], 3));
                  const uint4 xa = x0[(s >> 1) % AW], xb = x1[(s >> 1) % AW];
                  if (s & 1) mma_bf16_16816(acc[j], xa.z, xb.z, xa.w, xb.w, b0, b1);
                  else mma_bf16_16816(acc[j], xa.x, xb.x, xa.y, xb.y, b0, b1);
                }
              } else {
                float tmp[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int wd = 0; wd < 4; ++wd) {
                  const uint4 xa = x0[wd % AW], xb = x1[wd % AW];
                  {
                    const uint32_t b0 = nib_pair_to_bf16x2(ww[wd] & 0x000F000Fu);
                    const uint32_t b1 = nib_pair_to_bf16x2((ww[wd] >> 4) & 0x000F000Fu);
                    mma_bf16_16816(tmp, xa.x, xb.x, xa.y, xb.y, b0, b1);
                  }
                  {
                    const uint32_t b0 = nib_pair_to_bf16x2((ww[wd] >> 8) & 0x000F000Fu);
                    const uint32_t b1 = nib_pair_to_bf16x2((ww[wd] >> 12) & 0x000F000Fu);
                    mma_bf16_16816(tmp, xa.z, xb.z, xa.w, xb.w, b0, b1);
                  }
                }
                // scales of weight rows 2t, 2t+1 for this 128-column group
                const uint32_t s2 = *reinterpret_cast<const uint32_t *>(ssm + ((size_t)j * KB + kb) * 8 + 2 * t);
                const float s_lo = bf16_lo(s2), s_hi = bf16_hi(s2);
                acc[j][0] = fmaf(s_lo, tmp[0], acc[j][0]);
                acc[j][1] = fmaf(s_hi, tmp[1], acc[j][1]);
                acc[j][2] = fmaf(s_lo, tmp[2], acc[j][2]);
                acc[j][3] = fmaf(s_hi, tmp[3], acc[j][3]);
              }
            }
          }
        }
      }
      trace_mark(a.trace, a.trace_slot, 4);
      // partial sums of the warps meet in shared memory and are added in warp order
#pragma unroll
      for (int j = 0; j < RT; ++j) {
        *reinterpret_cast<float2 *>(red + ((size_t)warp * 16 + g) * C + 8 * j + 2 * t) = make_float2(acc[j][0], acc[j][1]);
        *reinterpret_cast<float2 *>(red + ((size_t)warp * 16 + g + 8) * C + 8 * j + 2 * t) = make_float2(acc[j][2], acc[j][3]);
      }
    }
    __syncthreads();
    trace_mark(a.trace, a.trace_slot, 5);
#pragma unroll
    for (int e = 0; e < ER; ++e) {
      const int o = threadIdx.x + e * kLinearThreads;
      const int bl = o / C;
      const int n = en, b = m0 + bl;
      if (o < 16 * C && n < a.N && b < a.B) {
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < kLinearWarps; ++w) v += red[((size_t)w * 16 + bl) * C + ecol];
        if (WF == WF_INT8) v *= e_scale;
        if (gridDim.y > 1) {   // partial sum of this k-range; bias and residual are added by the folding LayerNorm
          a.out_f32[((size_t)blockIdx.y * kMaxRows + b) * a.N + n] = v;
          continue;
        }
        v += e_bias;
        if (a.mode == EPI_F32) {
          a.out_f32[(size_t)b * a.out_stride + n] = v;
        } else if (a.mode == EPI_RESID) {
          a.out_f32[(size_t)b * a.out_stride + n] = e_old[e] + v;
        } else if (a.mode == EPI_GELU) {
          v = a.gelu_tanh ? gelu_tanh_f(v) : gelu_erf_f(v);
          a.out_bf16[(size_t)b * a.N + n] = float_to_bf16_bits(v);
        } else {  // EPI_QKV
          if (n < a.d) {
            a.out_f32[(size_t)b * a.out_stride + n] = v;
          } else if (m0 == 0) {
            *kv_dst[e] = float_to_bf16_bits(v);
          } else {
            const int which = n >= 2 * a.d;  // 0 = K, 1 = V
            const int col = n - (which ? 2 * a.d : a.d);
            const int head = col >> 6, ee = col & 63;
            if (a.kv_stage) {
              a.kv_stage[((size_t)b * 2 + which) * a.d + col] = float_to_bf16_bits(v);
            } else {
              const int pos = a.row_pos[b];
              const int page = a.page_table[(size_t)a.row_stream[b] * a.pps + (pos >> 6)];
              a.kv_layer[(((size_t)page * 2 + which) * a.H + head) * kPageElems + (size_t)(pos & 63) * kHeadDim + ee] =
                  float_to_bf16_bits(v);
            }
          }
        }
      }
    }
    __syncthreads();
  }
  trace_mark(a.trace, a.trace_slot, 2);
}

// Shared memory of one CTA.
inline size_t linear_smem_bytes(int wf, int rt, int mode, int B, int K) {
  const int KB = K / k_per_tile(wf);
  size_t s = 128 + (size_t)rt * KB * (wf == WF_INT4 ? 528 : 512) + (size_t)kLinearWarps * 16 * 8 * rt * sizeof(float);
  if (mode != ACT_DIRECT) s += (size_t)B * ln_stage_stride(wf, K) * sizeof(uint16_t);
  return s;
}

// Launch shape: all CTAs of a launch should be resident at once (2 per SM), so that every weight
// byte of the layer is requested before the kernel waits for its predecessor; a CTA's weights and
// activation rows must fit its share of shared memory.
struct LinearPlan { int rt, grid; };
inline LinearPlan plan_linear(int wf, int N, int K, int B, int mode, int max_ctas) {   // K, max_ctas: per k-range
  const int tiles = row_tiles(N);
  LinearPlan p;
  p.rt = 1;
  while (p.rt < 4 && (tiles + p.rt - 1) / p.rt > max_ctas &&
         linear_smem_bytes(wf, p.rt * 2, mode, B, K) <= (size_t)kLinearSmemBudget)
    p.rt *= 2;
  p.grid = (tiles + p.rt - 1) / p.rt;
  return p;
}

template <int WF, int RT, int MODE, int NB>
inline cudaError_t launch_linear_nb(const LinearArgs &a, int grid, cudaStream_t st, bool pdl) {
  const int ks = a.ksplit > 1 ? a.ksplit : 1;
  const size_t smem = linear_smem_bytes(WF, RT, MODE, a.B, a.K / ks);
  static PerDeviceOnce attr_once;   // per device: opt-in to more than 48 KB of dynamic shared memory
  if (attr_once.first()) {
    cudaFuncSetAttribute(linear_kernel<WF, RT, MODE, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  }
  return launch_kernel(linear_kernel<WF, RT, MODE, NB>, dim3(grid, ks), dim3(kLinearThreads), smem, st, pdl, a);
}

template <int WF, int RT, int MODE>
inline cudaError_t launch_linear_inst(const LinearArgs &a, int grid, cudaStream_t st, bool pdl) {
  if (MODE != ACT_DIRECT) {  // batches of up to 4 rows always fit the staging buffer
    if (a.B == 1) return launch_linear_nb<WF, RT, (MODE == ACT_DIRECT ? ACT_STAGED : MODE), 1>(a, grid, st, pdl);
    if (a.B <= 4) return launch_linear_nb<WF, RT, (MODE == ACT_DIRECT ? ACT_STAGED : MODE), 4>(a, grid, st, pdl);
  }
  return launch_linear_nb<WF, RT, MODE, 0>(a, grid, st, pdl);
}

template <int WF, int MODE>
inline cudaError_t launch_linear_wf(const LinearArgs &a, int max_ctas, cudaStream_t st, bool pdl) {
  const int ks = a.ksplit > 1 ? a.ksplit : 1;
  const LinearPlan p = plan_linear(WF, a.N, a.K / ks, a.B, MODE, max_ctas / ks);
  if (linear_smem_bytes(WF, p.rt, MODE, a.B, a.K / ks) > 200 * 1024) return cudaErrorInvalidValue;
  if (p.rt == 1) return launch_linear_inst<WF, 1, MODE>(a, p.grid, st, pdl);
  if (p.rt == 2) return launch_linear_inst<WF, 2, MODE>(a, p.grid, st, pdl);
  return launch_linear_inst<WF, 4, MODE>(a, p.grid, st, pdl);
}

// Whether LayerNorm can be fused in front of a linear with this shape (one float4 of the row per thread).
inline bool can_fuse_ln(int wf, int B, int K) {
  (void)wf;
  return B <= kLnFuseMaxRows && K <= 4 * kLinearThreads;
}

template <int WF>
inline cudaError_t launch_linear_mode(const LinearArgs &a, int max_ctas, cudaStream_t st, bool pdl) {
  if (a.ln_x) return launch_linear_wf<WF, ACT_LN>(a, max_ctas, st, pdl);
  if ((size_t)a.B * ln_stage_stride(WF, a.K / (a.ksplit > 1 ? a.ksplit : 1)) * sizeof(uint16_t) <= (size_t)kStageMaxBytes)
    return launch_linear_wf<WF, ACT_STAGED>(a, max_ctas, st, pdl);
  return launch_linear_wf<WF, ACT_DIRECT>(a, max_ctas, st, pdl);
}

// K must be a multiple of 128.
inline cudaError_t launch_linear(int wf, const LinearArgs &a, cudaStream_t st, bool pdl = false, int max_ctas = 296) {
  if (a.ln_x && !can_fuse_ln(wf, a.B, a.K)) return cudaErrorInvalidValue;
  if (a.ksplit > 1 && (a.ln_x || a.mode != EPI_RESID || (a.K / k_per_tile(wf)) % a.ksplit != 0)) return cudaErrorInvalidValue;
  if (wf == WF_BF16) return launch_linear_mode<WF_BF16>(a, max_ctas, st, pdl);
  if (wf == WF_INT8) return launch_linear_mode<WF_INT8>(a, max_ctas, st, pdl);
  return launch_linear_mode<WF_INT4>(a, max_ctas, st, pdl);
}

inline cudaError_t launch_pack(int wf, int N, int K, const void *w, const void *s, void *dst_w, void *dst_s,
                               cudaStream_t st) {
  const size_t units = (size_t)row_tiles(N) * (K / k_per_tile(wf)) * 32;
  const int blocks = (int)((units + 255) / 256);
  if (wf == WF_BF16) pack_bf16_kernel<<<blocks, 256, 0, st>>>((const uint16_t *)w, N, K, (uint4 *)dst_w);
  else if (wf == WF_INT8) pack_int8_kernel<<<blocks, 256, 0, st>>>((const int8_t *)w, N, K, (uint4 *)dst_w);
  else pack_int4_kernel<<<blocks, 256, 0, st>>>((const uint32_t *)w, N, K, (uint4 *)dst_w);
  if (wf != WF_BF16) {
    const int G = wf == WF_INT8 ? 1 : K / 128;
    const size_t n = (size_t)row_tiles(N) * G * 8;
    pack_scales_kernel<<<(int)((n + 255) / 256), 256, 0, st>>>((const uint16_t *)s, N, G, (uint16_t *)dst_s);
  }
  return cudaGetLastError();
}

}  // namespace ttsgpt
