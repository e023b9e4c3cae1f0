// One decode step of a few rows (batch 1 to 4) as ONE persistent kernel (Section II-C: the
// incremental decode iteration; Table I caption: weight-only W8A16 / W4A16 linears inside it).
//
// Why.  At batch 1 a step streams about 1 GB of weights (0.15 ms at HBM speed) through some 120
// dependent stages of a few microseconds each.  Run as one kernel per stage, the memory system idles
// while each stage hands over to the next.  Here one CTA per SM stays resident for the whole step:
//
//  * Static ownership.  CTA c owns the same slice of output features of every linear of every layer
//    (rows [N c / G, N (c+1) / G) of an [N, K] matrix; FC2 is cut into d_ff / d column blocks, all of
//    them for the CTA's rows).  Weights are stored once more at creation as "records" (one output
//    feature x d columns, with its scales), so a CTA's share of a linear is a few contiguous ranges.
//  * A producer warp streams the CTA's records and its share of the KV pages, in the order the
//    step consumes them, into a ring in shared memory with bulk asynchronous copies (completion on
//    mbarriers).  Weights and old K/V do not depend on the activations, so the stream runs ahead of
//    the arithmetic, across stage boundaries, as far as the ring (about 200 KB per SM) allows.
//  * Stage hand-over without grid barriers.  Every value a stage produces (q, k, v, attention
//    partials, the residual stream, the FC1 output) is published as one 64-bit word {value, tag}
//    in global memory; the tag names launch, layer and stage.  Consumers read the words they need
//    and retry those whose tag is not yet the expected one, so data and "ready" flag arrive in the
//    same L2 round trip and a consumer waits only for what it reads.  A 64-bit access is single-copy
//    atomic, so a word is either the old or the new pair, never a mixture.
//  * 16 consumer warps.  A lane keeps the activation columns it multiplies (columns 256 j + 8 lane ..
//    + 7) in registers for the whole stage; a warp takes whole records, so a product needs no
//    exchange beyond one shuffle reduction.  Accumulation is fp32; int8 / int4 codes are widened
//    exactly and the bf16 scale multiplies fp32 sums (per row for int8, per 128-column group for int4).
//
// Every wait (tagged word, ring slot, copy barrier) is bounded: on expiry the CTA raises the engine's
// error word and an abort flag that makes all remaining waits of the launch return at once, so the
// kernel always runs to its end; copies in flight are waited for (again bounded) before it returns.
// The launch is cooperative: either all CTAs are co-resident or the launch fails.
#pragma once
#include "common.cuh"
#include "elementwise.cuh"
#include "linear.cuh"

namespace ttsgpt {

constexpr int kPsWarps = 12;                      // consumer warps
constexpr int kPsConsumers = kPsWarps * 32;
constexpr int kPsThreads = kPsConsumers + 32;     // + the producer warp
constexpr int kPsQueue = 32;                      // ring items in flight
constexpr int kPsMaxRows = 4;                     // rows (streams) of a step
constexpr int kPsMaxOwn = 16;                     // output features of a d-wide linear one CTA may own
constexpr int kPsMaxSplit = 8;                    // KV splits per (row, head)
constexpr int kPsChunkTokens = 128;               // tokens per ring item of K/V
constexpr int kPsPartialWords = 128;              // 64 pairs: o[e] and (m | l)
constexpr uint32_t kPsItemBytes = 16 * 1024;      // target size of a ring item of weights
constexpr unsigned long long kPsWaitNs = 1000000000ull;
enum { PS_TAG_Q = 1, PS_TAG_P = 2, PS_TAG_O = 3, PS_TAG_XA = 4, PS_TAG_H = 5, PS_TAG_XB = 6 };

// One record: the d columns of one output feature, then a tail with its scale(s) and its bias as fp32,
// padded to 16 bytes.  Everything a product needs arrives with the one copy that brings the record.
__host__ __device__ inline int ps_codes_bytes(int wf, int d) { return wf == WF_BF16 ? d * 2 : (wf == WF_INT8 ? d : d / 2); }
__host__ __device__ inline int ps_bias_offset(int wf, int d) {   // from the start of the record
  if (wf == WF_BF16) return d * 2;
  if (wf == WF_INT8) return d + 4;            // the row's bf16 scale sits at d
  return d / 2 + d / 128 * 2;                 // the group scales sit at d / 2 (d is a multiple of 256: 4-byte aligned)
}
__host__ __device__ inline int ps_record_bytes(int wf, int d) { return (ps_bias_offset(wf, d) + 4 + 15) & ~15; }
inline size_t ps_weight_bytes(int wf, int N, int K, int d) { return (size_t)(K / d) * N * ps_record_bytes(wf, d); }
__host__ __device__ inline int ps_rows_per_item(int rs, int wg) {
  int ri = (int)(kPsItemBytes / (uint32_t)rs);
  if (ri < 1) ri = 1;
  return ri < wg ? ri : wg;
}
__host__ __device__ inline void ps_range(int N, int c, int G, int &n0, int &n1) {
  n0 = (int)((long long)N * c / G);
  n1 = (int)((long long)N * (c + 1) / G);
}
// KV splits per (row, head): as many as keep every (row, head, split) on a CTA of its own
__host__ __device__ inline int ps_splits(int R, int H, int G) {
  int s = G / (R * H);
  if (s > kPsMaxSplit) s = kPsMaxSplit;
  return s < 1 ? 1 : s;
}
inline bool ps_supported(int d, int d_ff, int H, int n_layer, int V, int G) {
  return d % 256 == 0 && d <= 2048 && d_ff % d == 0 && (d_ff / d == 1 || d_ff / d == 2 || d_ff / d == 4) &&
         n_layer <= 31 && (d + G - 1) / G <= kPsMaxOwn && H <= G && V >= 1;
}

// ------------------------------------------------------------------------------------------
// canonical [N][K] -> records [K/d][N][record]  (once, at creation)
// ------------------------------------------------------------------------------------------
__global__ void ps_pack_kernel(int wf, const void *__restrict__ w, const uint16_t *__restrict__ s,
                               const uint16_t *__restrict__ bias, int N, int K, int d, unsigned char *__restrict__ dst) {
  const int rs = ps_record_bytes(wf, d), upr = rs / 16, ks = K / d, cb = ps_codes_bytes(wf, d);
  const size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (unit >= (size_t)ks * N * upr) return;
  const int u = (int)(unit % upr);
  const size_t rec = unit / upr;
  const int n = (int)(rec % N), q = (int)(rec / N);
  uint4 v = make_uint4(0, 0, 0, 0);
  if (16 * u < cb) {
    if (wf == WF_BF16) {
      v = *reinterpret_cast<const uint4 *>((const uint16_t *)w + (size_t)n * K + (size_t)q * d + 8 * u);
    } else if (wf == WF_INT8) {   // codes, stored biased (q + 128): one byte permute widens them
      v = *reinterpret_cast<const uint4 *>((const int8_t *)w + (size_t)n * K + (size_t)q * d + 16 * u);
      v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u;
    } else {                      // nibbles re-ordered so that (word >> 4e) & 0x000F000F is the column pair (2e, 2e+1)
      const uint4 c = *reinterpret_cast<const uint4 *>((const uint32_t *)w + (size_t)n * (K / 8) + (size_t)q * (d / 8) + 4 * u);
      v = make_uint4(permute_nibbles(c.x), permute_nibbles(c.y), permute_nibbles(c.z), permute_nibbles(c.w));
    }
  } else {
    // tail: scales, then the bias (column block 0 only, so that the blocks of a row add it once)
    const int boff = ps_bias_offset(wf, d) - cb, G = d / 128;
    uint32_t ww[4] = {0, 0, 0, 0};
    for (int i = 0; i < 4; ++i) {
      const int bo = 16 * u - cb + 4 * i;     // byte offset of this word inside the tail
      if (bo == boff) {
        ww[i] = (bias && q == 0) ? ((uint32_t)bias[n] << 16) : 0u;
      } else if (wf == WF_INT8 && bo == 0) {
        ww[i] = s[n];
      } else if (wf == WF_INT4 && bo < 2 * G) {
        const int g = bo / 2;
        ww[i] = (uint32_t)s[(size_t)n * (K / 128) + (size_t)q * G + g];
        if (g + 1 < G) ww[i] |= (uint32_t)s[(size_t)n * (K / 128) + (size_t)q * G + g + 1] << 16;
      }
    }
    v = make_uint4(ww[0], ww[1], ww[2], ww[3]);
  }
  *reinterpret_cast<uint4 *>(dst + rec * rs + 16 * u) = v;
}
inline cudaError_t launch_ps_pack(int wf, int N, int K, int d, const void *w, const void *s, const void *bias, void *dst,
                                  cudaStream_t st) {
  const size_t units = (size_t)(K / d) * N * (ps_record_bytes(wf, d) / 16);
  ps_pack_kernel<<<(unsigned)((units + 255) / 256), 256, 0, st>>>(wf, w, (const uint16_t *)s, (const uint16_t *)bias, N, K, d,
                                                                  (unsigned char *)dst);
  return cudaGetLastError();
}

struct PsLayerDesc {
  const unsigned char *qkv_w, *o_w, *fc1_w, *fc2_w;   // records
  const uint16_t *ln1_g, *ln1_b, *ln2_g, *ln2_b;
};

struct PsArgs {
  const PsLayerDesc *layers; int n_layer;
  const unsigned char *head_w; const uint16_t *lnf_g, *lnf_b;
  uint16_t *kv; size_t kv_layer_elems;                  // the pool and the elements of one layer's slice
  const uint16_t *tok_emb, *pos_emb; int emb_rows, max_pos;
  int d, d_ff, H, V; float ln_eps; int gelu_tanh;
  const int *row_stream, *row_pos, *row_token, *row_posidx, *page_table; int pps, R;
  const StepIO *io; uint32_t seq;
  unsigned long long *xa, *xb, *hb, *qb, *kn, *pb, *ob;   // tagged words: [rows][d] x2, [rows][d_ff], [rows][d], [rows][2][d], [rows][H][8][66], [rows][d]
  float *logits;
  int *abort_g, *err;
  unsigned long long *trace;
  int trace_detail;      // the trace buffer also has two slots per CTA behind the per-layer ones
  uint32_t ring_bytes;
};
inline size_t ps_exchange_words(int d, int d_ff, int H) {
  return (size_t)kPsMaxRows * ((size_t)d * 2 + d_ff + d + 2 * d + (size_t)H * kPsMaxSplit * kPsPartialWords + d);
}

// ------------------------------------------------------------------------------------------
// tagged words
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void ps_st(unsigned long long *p, uint32_t bits, uint32_t tag) {
  const unsigned long long v = ((unsigned long long)tag << 32) | bits;
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void ps_ld2(const unsigned long long *p, unsigned long long &a, unsigned long long &b) {
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0,%1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
}

// ------------------------------------------------------------------------------------------
// shared memory
// ------------------------------------------------------------------------------------------
struct PsShared {
  uint64_t full[kPsQueue];          // copy barriers of the ring items
  uint32_t q_off[kPsQueue];         // ring offset of an item
  int done[kPsQueue];               // consumers that finished with an item
  unsigned long long it_vend[kPsQueue];   // producer only: virtual end of the item
  int it_expect[kPsQueue];          // producer only: consumers to wait for
  int abort_s;                      // set once a wait of this CTA gave up (or another CTA's did)
  unsigned long long dbg_t[kPsWarps][4];  // TEMPDBG
  unsigned long long dbg_wait;      // detail trace: time thread 0 spent waiting for ring items
  PsArgs args;                      // copy of the launch arguments (read by every stage function)
  float *xs;                        // residual rows of the last LayerNorm, fp32 [R][d]
  uint16_t *act;                    // input rows of the next linear, bf16 [R][d_ff]
  unsigned char *ring;
  // the CTA's plan, computed once: row ranges of the linears (QKV, O / FC2, FC1, head), its attention item,
  // and per batch row the position and page of the new token
  int rng[4][2];
  int S, has_item, at_r, at_h, at_s;
  int row_pos[kPsMaxRows], row_page[kPsMaxRows];
  float lnred[kPsWarps][2];
  float comb[kPsMaxRows][4][kPsMaxOwn];
  float at_m[kPsWarps], at_l[kPsWarps], at_o[kPsWarps][kHeadDim];
};
inline size_t ps_fixed_smem(int d, int d_ff, int R) {   // control block, the residual rows (fp32), the activation rows (bf16)
  return ((sizeof(PsShared) + 127) & ~(size_t)127) + (size_t)R * d * 4 + (size_t)R * d_ff * 2;
}

// The slow side of every spin loop, kept out of line (the stage code has to stay small).  Called every 64
// polls with the time of the first call (0 on the first): returns that time, or ~0 to give up — the
// launch-wide abort flag is up, or the wait has lasted longer than its limit, in which case it raises
// the flag and the engine's error word.
__device__ __noinline__ unsigned long long ps_spin_check(PsShared *sh, unsigned long long t0) {
  volatile int *ab = &sh->abort_s;
  if (*ab) return ~0ull;
  if (*reinterpret_cast<volatile int *>(sh->args.abort_g)) { *ab = 1; return ~0ull; }
  const unsigned long long now = global_timer_ns();
  if (t0 == 0ull) return now;
  if (now - t0 > kPsWaitNs) {
    *ab = 1;
    atomicExch(sh->args.abort_g, 1);
    if (sh->args.err) atomicExch(sh->args.err, 1);
    return ~0ull;
  }
  return t0;
}
__device__ __noinline__ void ps_wait_item_slow(PsShared *sh, uint32_t it) {
  volatile int *ab = &sh->abort_s;
  if (*ab) return;
  const unsigned long long w0 = (sh->args.trace_detail && threadIdx.x == 0) ? global_timer_ns() : 0ull;
  const bool ok = mbar_wait_bounded(&sh->full[it % kPsQueue], (it / kPsQueue) & 1u, kPsWaitNs);
  if (w0) sh->dbg_wait += global_timer_ns() - w0;
  if (!ok) {
    *ab = 1;
    atomicExch(sh->args.abort_g, 1);
    if (sh->args.err) atomicExch(sh->args.err, 1);
  }
}
// waits for ring item `it` to have landed; gives up like every other wait
__device__ __forceinline__ void ps_wait_item(PsShared *sh, uint32_t it) {
  if (!mbar_try_wait(&sh->full[it % kPsQueue], (it / kPsQueue) & 1u)) ps_wait_item_slow(sh, it);
}

// Reads the NB pairs of tagged words  first, first + step, ...  (pair p = words 2p, 2p+1; pairs >= n are
// skipped) until all carry `tag`; v0 / v1 receive the two values of each pair.
template <int NB>
__device__ __forceinline__ void ps_poll(PsShared *sh, const unsigned long long *buf, int first, int step, int n, uint32_t tag,
                                        uint32_t (&v0)[NB], uint32_t (&v1)[NB]) {
  unsigned spins = 0;
  unsigned long long t0 = 0ull;
  const unsigned long long filler = (unsigned long long)tag << 32;
  while (true) {
    bool all = true;
#pragma unroll
    for (int i = 0; i < NB; ++i) {
      unsigned long long a = filler, b = filler;
      if (first + i * step < n) ps_ld2(buf + 2 * (size_t)(first + i * step), a, b);
      v0[i] = (uint32_t)a; v1[i] = (uint32_t)b;
      all = all && (uint32_t)(a >> 32) == tag && (uint32_t)(b >> 32) == tag;
    }
    if (all) break;
    if ((++spins & 63u) == 0u) {
      t0 = ps_spin_check(sh, t0);
      if (t0 == ~0ull) break;
    }
  }
}

__device__ __forceinline__ void ps_bar_consumers() { asm volatile("bar.sync 1, %0;" ::"n"(kPsConsumers) : "memory"); }

// ------------------------------------------------------------------------------------------
// products: 256 columns of one record against the lane's 8 activation values of that column chunk
// ------------------------------------------------------------------------------------------
// bf16 / int8: adds into (s0, s1).  int4: adds scale x (sum - 136 x asum) into s0: nibble u stands for
// u - 8; the pair mask leaves bf16(128 + u) in each half-word, every product a (128 + u) is exact, and
// 136 x (sum of the lane's a) is taken off before the group's scale multiplies.
template <int WF>
__device__ __forceinline__ void ps_dot_chunk(const unsigned char *rec, int j, int lane, int d, const float (&a)[8], float asum,
                                             float &s0, float &s1) {
  if (WF == WF_BF16) {
    const uint4 w = *reinterpret_cast<const uint4 *>(rec + 512 * j + 16 * lane);
    s0 = fmaf(bf16_lo(w.x), a[0], s0); s1 = fmaf(bf16_hi(w.x), a[1], s1);
    s0 = fmaf(bf16_lo(w.y), a[2], s0); s1 = fmaf(bf16_hi(w.y), a[3], s1);
    s0 = fmaf(bf16_lo(w.z), a[4], s0); s1 = fmaf(bf16_hi(w.z), a[5], s1);
    s0 = fmaf(bf16_lo(w.w), a[6], s0); s1 = fmaf(bf16_hi(w.w), a[7], s1);
  } else if (WF == WF_INT8) {
    const uint2 w = *reinterpret_cast<const uint2 *>(rec + 256 * j + 8 * lane);
    s0 = fmaf(biased_byte_to_float(w.x, 0), a[0], s0); s1 = fmaf(biased_byte_to_float(w.x, 1), a[1], s1);
    s0 = fmaf(biased_byte_to_float(w.x, 2), a[2], s0); s1 = fmaf(biased_byte_to_float(w.x, 3), a[3], s1);
    s0 = fmaf(biased_byte_to_float(w.y, 0), a[4], s0); s1 = fmaf(biased_byte_to_float(w.y, 1), a[5], s1);
    s0 = fmaf(biased_byte_to_float(w.y, 2), a[6], s0); s1 = fmaf(biased_byte_to_float(w.y, 3), a[7], s1);
  } else {
    const uint32_t w = *reinterpret_cast<const uint32_t *>(rec + 128 * j + 4 * lane);
    float t0 = 0.f, t1 = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t pr = ((w >> (4 * e)) & 0x000F000Fu) | 0x43004300u;
      t0 = fmaf(bf16_lo(pr), a[2 * e], t0);
      t1 = fmaf(bf16_hi(pr), a[2 * e + 1], t1);
    }
    const float g = bf16_bits_to_float(*reinterpret_cast<const uint16_t *>(rec + d / 2 + 2 * (2 * j + (lane >> 4))));
    s0 = fmaf(g, (t0 + t1) - 136.f * asum, s0);
  }
}

// What a stage function needs beyond shared memory; passed by value (registers).
struct PsCtx {
  PsShared *sh;
  uint32_t item;         // index of the next ring item in the CTA's stream (consumers and producer count alike)
  uint32_t tag0;         // launch part of the tags
  int layer;
};

enum { PS_EPI_QKV = 0, PS_EPI_O = 1, PS_EPI_FC1 = 2, PS_EPI_FC2 = 3, PS_EPI_HEAD = 4 };

// One linear for this CTA's rows of an [N, ks*d] matrix against the act rows; `mode` says which linear
// and what becomes of the products (bias is part of the record).  A warp takes up to kPsRowsPerPass of
// its records at a time and walks the column chunks once for all of them: a chunk's 8 activation values
// per lane are loaded once and meet every record (few registers, several independent sums in flight);
// then lane u finishes record u, so the epilogue exists once and runs for all records at the same time.
// Called from one place: one copy of this code serves every stage (the kernel is a loop over stages whose
// code has to stay in the instruction cache).
constexpr int kPsRowsPerPass = 4;
template <int WF>
__device__ __forceinline__ uint32_t ps_linear(PsCtx cx, int mode) {
  PsShared *sh = cx.sh;
  const PsArgs &a = sh->args;
  const int rgi = mode == PS_EPI_QKV ? 0 : (mode == PS_EPI_FC1 ? 2 : (mode == PS_EPI_HEAD ? 3 : 1));
  const int n0 = sh->rng[rgi][0], n1 = sh->rng[rgi][1];
  const int ks = mode == PS_EPI_FC2 ? a.d_ff / a.d : 1;
  const int d = a.d, F = a.d_ff, R = a.R, H = a.H, jw = d >> 8;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned char *ring = sh->ring;
  const int rs = ps_record_bytes(WF, d), boff = ps_bias_offset(WF, d);
  const int wg = kPsWarps / ks, q = warp / wg, i = warp % wg;
  const int ri = ps_rows_per_item(rs, wg), nrows = n1 - n0, ipq = (nrows + ri - 1) / ri;
  const uint32_t tg = cx.tag0 + (uint32_t)cx.layer * 8u;
  const bool dbg = sh->args.trace_detail && mode == PS_EPI_O && cx.layer == sh->args.n_layer / 2 && lane == 0;  // TEMPDBG
  if (dbg) sh->dbg_t[warp][0] = global_timer_ns();  // TEMPDBG
#pragma unroll 1
  for (int r = 0; r < R; ++r) {
    const uint16_t *arow = sh->act + (size_t)r * F + (size_t)q * d + 8 * lane;
#pragma unroll 1
    for (int rel0 = i; rel0 < nrows; rel0 += wg * kPsRowsPerPass) {
      const unsigned char *rec[kPsRowsPerPass];
      float s0[kPsRowsPerPass], s1[kPsRowsPerPass];
#pragma unroll
      for (int u = 0; u < kPsRowsPerPass; ++u) {
        const int rel = rel0 + u * wg;
        s0[u] = 0.f; s1[u] = 0.f;
        rec[u] = ring;
        if (rel < nrows) {
          const int p = rel / ri;
          const uint32_t it = cx.item + (uint32_t)(p * ks + q);
          if (r == 0) ps_wait_item(sh, it);
          rec[u] = ring + sh->q_off[it % kPsQueue] + (size_t)(rel - p * ri) * rs;
        }
      }
      if (dbg) sh->dbg_t[warp][1] = global_timer_ns();  // TEMPDBG
#pragma unroll 1
      for (int j = 0; j < jw; ++j) {
        const uint4 xv = *reinterpret_cast<const uint4 *>(arow + 256 * j);
        const float av[8] = {bf16_lo(xv.x), bf16_hi(xv.x), bf16_lo(xv.y), bf16_hi(xv.y),
                             bf16_lo(xv.z), bf16_hi(xv.z), bf16_lo(xv.w), bf16_hi(xv.w)};
        const float asum = ((av[0] + av[1]) + (av[2] + av[3])) + ((av[4] + av[5]) + (av[6] + av[7]));
#pragma unroll
        for (int u = 0; u < kPsRowsPerPass; ++u)
          if (rel0 + u * wg < nrows) ps_dot_chunk<WF>(rec[u], j, lane, d, av, asum, s0[u], s1[u]);
      }
      if (dbg) sh->dbg_t[warp][2] = global_timer_ns();  // TEMPDBG
      // lane u ends up with record u's sum and finishes it
      float v = 0.f;
      const unsigned char *myrec = ring;
#pragma unroll
      for (int u = 0; u < kPsRowsPerPass; ++u) {
        const float t = warp_sum(s0[u] + s1[u]);
        if (lane == u) { v = t; myrec = rec[u]; }
      }
      const int rel = rel0 + lane * wg;
      if (lane < kPsRowsPerPass && rel < nrows) {
        if (WF == WF_INT8) v *= bf16_bits_to_float(*reinterpret_cast<const uint16_t *>(myrec + d));   // per-row scale
        v += *reinterpret_cast<const float *>(myrec + boff);
        const int n = n0 + rel;
        if (mode == PS_EPI_QKV) {
          // q as fp32; the new token's k and v as bf16, into their page slot and to the attention stage
          if (n < d) {
            ps_st(a.qb + (size_t)r * d + n, __float_as_uint(v), tg + PS_TAG_Q);
          } else {
            const int which = n >= 2 * d, col = n - (which ? 2 * d : d);
            const uint16_t bits = float_to_bf16_bits(v);
            const int pos = sh->row_pos[r], page = sh->row_page[r];
            uint16_t *kvl = a.kv + a.kv_layer_elems * cx.layer;
            kvl[(((size_t)page * 2 + which) * H + (col >> 6)) * kPageElems + (size_t)(pos & 63) * kHeadDim + (col & 63)] = bits;
            ps_st(a.kn + ((size_t)r * 2 + which) * d + col, (uint32_t)bits << 16, tg + PS_TAG_Q);
          }
        } else if (mode == PS_EPI_O) {
          ps_st(a.xa + (size_t)r * d + n, __float_as_uint(v + sh->xs[(size_t)r * d + n]), tg + PS_TAG_XA);
        } else if (mode == PS_EPI_FC1) {
          const float gv = a.gelu_tanh ? gelu_tanh_f(v) : gelu_erf_f(v);
          ps_st(a.hb + (size_t)r * F + n, float_to_bf16_bits(gv), tg + PS_TAG_H);
        } else if (mode == PS_EPI_FC2) {
          sh->comb[r][q][rel] = v;
        } else {
          a.logits[(size_t)r * a.V + n] = v;
        }
      }
      if (r == R - 1) {
        __syncwarp();   // every lane has read its part of the records
        if (lane < kPsRowsPerPass && rel < nrows) atomicAdd(&sh->done[(cx.item + (uint32_t)((rel / ri) * ks + q)) % kPsQueue], 1);
      }
    }
  }
  if (dbg) sh->dbg_t[warp][3] = global_timer_ns();  // TEMPDBG
  return cx.item + (uint32_t)(ks * ipq);
}

// LayerNorm stage.  Input rows: the residual rows published under `tag` in `buf`, or (buf == nullptr)
// the step's input rows: token embedding + positional embedding of the token's index in the semantic
// range.  Thread t owns columns 2t, 2t+1 and, if it exists, 2(t + consumers), + 1.  (mean, M2) pairs are
// merged pairwise inside a warp (equal counts) and across the warps by their counts: no cancellation.
// Leaves the fp32 rows in xs and the normalised bf16 rows in act (and in `hidden` if given).  gamma and
// beta are the next ring item.  Two consumer barriers per row.
__device__ __forceinline__ uint32_t ps_ln_stage(PsCtx cx, const unsigned long long *buf, uint32_t tag, uint16_t *hidden) {
  PsShared *sh = cx.sh;
  const PsArgs &a = sh->args;
  const int d = a.d, F = a.d_ff, R = a.R;
  const int np = d / 2, t = threadIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool h0 = t < np, h1 = t + kPsConsumers < np;
  const uint32_t it = cx.item, slot = it % kPsQueue;
  float gg[4] = {0.f, 0.f, 0.f, 0.f}, bb[4] = {0.f, 0.f, 0.f, 0.f};
  const float cnt0 = (h0 ? 2.f : 0.f) + (h1 ? 2.f : 0.f);   // uniform over a warp (d / 2 is a multiple of 32)
#pragma unroll 1
  for (int r = 0; r < R; ++r) {
    float xv[4] = {0.f, 0.f, 0.f, 0.f};
    if (buf) {
      uint32_t v0[2], v1[2];
      ps_poll<2>(sh, buf + (size_t)r * d, t, kPsConsumers, np, tag, v0, v1);
      xv[0] = __uint_as_float(v0[0]); xv[1] = __uint_as_float(v1[0]);
      xv[2] = __uint_as_float(v0[1]); xv[3] = __uint_as_float(v1[1]);
    } else {
      const int tok = min(max(a.row_token[r], 0), a.emb_rows - 1);
      const int pp = min(max(a.row_posidx[r], 0), a.max_pos - 1);
      const uint16_t *te = a.tok_emb + (size_t)tok * d, *pe = a.pos_emb + (size_t)pp * d;
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int p = t + k * kPsConsumers;
        if (p < np) {
          const uint32_t tw = *reinterpret_cast<const uint32_t *>(te + 2 * p), pw = *reinterpret_cast<const uint32_t *>(pe + 2 * p);
          xv[2 * k] = bf16_lo(tw) + bf16_lo(pw);
          xv[2 * k + 1] = bf16_hi(tw) + bf16_hi(pw);
        }
      }
    }
    if (r == 0) {
      ps_wait_item(sh, it);
      const uint16_t *g = reinterpret_cast<const uint16_t *>(sh->ring + sh->q_off[slot]), *b = g + d;
      if (h0) {
        const uint32_t gw = *reinterpret_cast<const uint32_t *>(g + 2 * t), bw = *reinterpret_cast<const uint32_t *>(b + 2 * t);
        gg[0] = bf16_lo(gw); gg[1] = bf16_hi(gw); bb[0] = bf16_lo(bw); bb[1] = bf16_hi(bw);
      }
      if (h1) {
        const uint32_t gw = *reinterpret_cast<const uint32_t *>(g + 2 * (t + kPsConsumers));
        const uint32_t bw = *reinterpret_cast<const uint32_t *>(b + 2 * (t + kPsConsumers));
        gg[2] = bf16_lo(gw); gg[3] = bf16_hi(gw); bb[2] = bf16_lo(bw); bb[3] = bf16_hi(bw);
      }
      __syncwarp();
      if (lane == 0) atomicAdd(&sh->done[slot], 1);
    }
    float mean = 0.f, m2 = 0.f;
    if (h1) {
      mean = 0.25f * ((xv[0] + xv[1]) + (xv[2] + xv[3]));
      const float d0 = xv[0] - mean, d1 = xv[1] - mean, d2 = xv[2] - mean, d3 = xv[3] - mean;
      m2 = (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
    } else if (h0) {
      mean = 0.5f * (xv[0] + xv[1]);
      const float d0 = xv[0] - mean, d1 = xv[1] - mean;
      m2 = d0 * d0 + d1 * d1;
    }
    float cnt = cnt0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float mb = __shfl_xor_sync(0xFFFFFFFFu, mean, o);
      const float qb = __shfl_xor_sync(0xFFFFFFFFu, m2, o);
      const float dl = mb - mean;
      m2 = m2 + qb + dl * dl * (0.5f * cnt);
      mean = 0.5f * (mean + mb);
      cnt *= 2.f;
    }
    if (lane == 0) { sh->lnred[warp][0] = mean; sh->lnred[warp][1] = m2; }
    ps_bar_consumers();
    float msum = 0.f;
#pragma unroll 1
    for (int w = 0; w < kPsWarps; ++w) {
      const float nw = (32 * w < np ? 64.f : 0.f) + (32 * w + kPsConsumers < np ? 64.f : 0.f);
      msum = fmaf(nw, sh->lnred[w][0], msum);
    }
    const float mu = msum / (float)d;
    float m2t = 0.f;
#pragma unroll 1
    for (int w = 0; w < kPsWarps; ++w) {
      const float nw = (32 * w < np ? 64.f : 0.f) + (32 * w + kPsConsumers < np ? 64.f : 0.f);
      const float dl = sh->lnred[w][0] - mu;
      m2t += sh->lnred[w][1] + nw * dl * dl;
    }
    const float rstd = rsqrtf(m2t / (float)d + a.ln_eps);
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      if (k == 0 ? h0 : h1) {
        const int c = 2 * (t + k * kPsConsumers);
        const uint32_t y = pack_bf16x2((xv[2 * k] - mu) * rstd * gg[2 * k] + bb[2 * k], (xv[2 * k + 1] - mu) * rstd * gg[2 * k + 1] + bb[2 * k + 1]);
        *reinterpret_cast<uint32_t *>(sh->act + (size_t)r * F + c) = y;
        *reinterpret_cast<float2 *>(sh->xs + (size_t)r * d + c) = make_float2(xv[2 * k], xv[2 * k + 1]);
        if (hidden) *reinterpret_cast<uint32_t *>(hidden + (size_t)r * d + c) = y;
      }
    }
    ps_bar_consumers();   // act / xs complete; lnred free for the next row
  }
  return cx.item + 1;
}

// A published bf16 vector (values in the low half-words of the words of `buf`, K per row) -> act rows.
__device__ __forceinline__ void ps_poll_act(PsShared *sh, const unsigned long long *buf, int K, uint32_t tag) {
  const int np = K / 2, F = sh->args.d_ff, R = sh->args.R;
#pragma unroll 1
  for (int r = 0; r < R; ++r) {
    uint16_t *dst = sh->act + (size_t)r * F;
#pragma unroll 1
    for (int base = threadIdx.x; base < np; base += kPsConsumers * 8) {
      uint32_t v0[8], v1[8];
      ps_poll<8>(sh, buf + (size_t)r * K, base, kPsConsumers, np, tag, v0, v1);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (base + i * kPsConsumers < np) *reinterpret_cast<uint32_t *>(dst + 2 * (base + i * kPsConsumers)) = (v0[i] & 0xFFFFu) | (v1[i] << 16);
    }
  }
}

// tokens [t0, t1) of split s of a row with n_tok tokens (the last one being the new token)
__device__ __forceinline__ void ps_split_range(int n_tok, int S, int s, int &t0, int &t1) {
  const int n16 = (n_tok + 15) >> 4, c16 = (n16 + S - 1) / S;
  t0 = min(n_tok, s * c16 * 16);
  t1 = min(n_tok, t0 + c16 * 16);
}

// Attention stage of one layer: this CTA's (row, head, split), if it has one.  Lane (tgp, sub) = (lane / 8,
// lane % 8) works on elements 8 sub .. 8 sub + 7 of one token of a group of 4; the old tokens' K and V come
// from the ring in chunks, the new token's k and v from the QKV stage of this step (the lanes that meet
// it read them from the exchange words).  Split 0 of a (row, head) merges the head's partial results and
// publishes the head's 64 outputs as bf16.  A partial result is 64 pairs of words: pair e holds o[e] and
// (m for even e, l for odd e).  One consumer barrier.
__device__ __forceinline__ uint32_t ps_attention(PsCtx cx) {
  PsShared *sh = cx.sh;
  const PsArgs &a = sh->args;
  const int S = sh->S, at_r = sh->at_r, at_h = sh->at_h, at_s = sh->at_s;
  const bool has_item = sh->has_item != 0;
  const int d = a.d, H = a.H, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t tg = cx.tag0 + (uint32_t)cx.layer * 8u;
  uint32_t item = cx.item;
  if (has_item) {
    int t0, t1;
    const int n_tok = sh->row_pos[at_r] + 1;
    ps_split_range(n_tok, S, at_s, t0, t1);
    const int pos = n_tok - 1, old_end = min(t1, pos);
    const bool has_new = pos >= t0 && pos < t1;
    const int tgp = lane >> 3, sub = lane & 7;
    float m = -INFINITY, lsum = 0.f, o[8], qv[8];
    {
      const float qs = 0.125f * 1.4426950408889634f;   // scores in log2 units
      uint32_t v0[4], v1[4];
      ps_poll<4>(sh, a.qb, (at_r * d + at_h * kHeadDim + 8 * sub) >> 1, 1, 0x7FFFFFFF, tg + PS_TAG_Q, v0, v1);
#pragma unroll
      for (int e = 0; e < 4; ++e) { qv[2 * e] = __uint_as_float(v0[e]) * qs; qv[2 * e + 1] = __uint_as_float(v1[e]) * qs; o[2 * e] = 0.f; o[2 * e + 1] = 0.f; }
    }
    const int n_old = max(old_end - t0, 0);
    const int n_chunks = max((n_old + kPsChunkTokens - 1) / kPsChunkTokens, has_new ? 1 : 0);
#pragma unroll 1
    for (int c = 0; c < n_chunks; ++c) {
      const int nt = min(max(n_old - c * kPsChunkTokens, 0), kPsChunkTokens);    // old tokens of the chunk
      const int extra = (has_new && c == n_chunks - 1) ? 1 : 0;                 // the new token rides with the last chunk
      const uint32_t slot = item % kPsQueue;
      const unsigned char *Kb = sh->ring, *Vb = sh->ring;
      if (nt > 0) {
        ps_wait_item(sh, item);
        Kb = sh->ring + sh->q_off[slot];
        Vb = Kb + (size_t)nt * 128;
      }
#pragma unroll 1
      for (int g = warp; 4 * g < nt + extra; g += kPsWarps) {
        const int tl = 4 * g + tgp;
        float kf[8], vf[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) { kf[e] = 0.f; vf[e] = 0.f; }
        if (tl < nt) {
          const uint4 kk = *reinterpret_cast<const uint4 *>(Kb + (size_t)tl * 128 + 16 * sub);
          const uint4 vv = *reinterpret_cast<const uint4 *>(Vb + (size_t)tl * 128 + 16 * sub);
          kf[0] = bf16_lo(kk.x); kf[1] = bf16_hi(kk.x); kf[2] = bf16_lo(kk.y); kf[3] = bf16_hi(kk.y);
          kf[4] = bf16_lo(kk.z); kf[5] = bf16_hi(kk.z); kf[6] = bf16_lo(kk.w); kf[7] = bf16_hi(kk.w);
          vf[0] = bf16_lo(vv.x); vf[1] = bf16_hi(vv.x); vf[2] = bf16_lo(vv.y); vf[3] = bf16_hi(vv.y);
          vf[4] = bf16_lo(vv.z); vf[5] = bf16_hi(vv.z); vf[6] = bf16_lo(vv.w); vf[7] = bf16_hi(vv.w);
        }
        if (4 * g + 3 >= nt && extra) {      // the group that holds the new token (warp-uniform)
          uint32_t k0[4], k1[4], w0[4], w1[4];
          const int lim = tl == nt ? 0x7FFFFFFF : 0;   // only the lanes of that token read
          ps_poll<4>(sh, a.kn, ((at_r * 2 + 0) * d + at_h * kHeadDim + 8 * sub) >> 1, 1, lim, tg + PS_TAG_Q, k0, k1);
          ps_poll<4>(sh, a.kn, ((at_r * 2 + 1) * d + at_h * kHeadDim + 8 * sub) >> 1, 1, lim, tg + PS_TAG_Q, w0, w1);
          if (tl == nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              kf[2 * e] = __uint_as_float(k0[e]); kf[2 * e + 1] = __uint_as_float(k1[e]);
              vf[2 * e] = __uint_as_float(w0[e]); vf[2 * e + 1] = __uint_as_float(w1[e]);
            }
          }
        }
        const bool valid = tl < nt + extra;
        float sc = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) sc = fmaf(qv[e], kf[e], sc);
        sc += __shfl_xor_sync(0xFFFFFFFFu, sc, 1);
        sc += __shfl_xor_sync(0xFFFFFFFFu, sc, 2);
        sc += __shfl_xor_sync(0xFFFFFFFFu, sc, 4);
        // online softmax update of the warp's (m, l, o) with this group of up to 4 tokens (one per tgp)
        const float s = valid ? sc : -INFINITY;
        float pm = fmaxf(s, __shfl_xor_sync(0xFFFFFFFFu, s, 8));
        pm = fmaxf(pm, __shfl_xor_sync(0xFFFFFFFFu, pm, 16));
        const float m_new = fmaxf(m, pm);             // finite: the group holds at least one token
        const float resc = exp2f(m - m_new);
        const float p = exp2f(s - m_new);
        lsum = lsum * resc + p;
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = fmaf(p, vf[e], o[e] * resc);
        m = m_new;
      }
      if (nt > 0) {
        __syncwarp();
        if (lane == 0) atomicAdd(&sh->done[slot], 1);
        ++item;
      }
    }
    lsum += __shfl_xor_sync(0xFFFFFFFFu, lsum, 8);
    lsum += __shfl_xor_sync(0xFFFFFFFFu, lsum, 16);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 8);
      o[e] += __shfl_xor_sync(0xFFFFFFFFu, o[e], 16);
    }
    if (tgp == 0) {
      if (sub == 0) { sh->at_m[warp] = m; sh->at_l[warp] = lsum; }
#pragma unroll
      for (int e = 0; e < 8; ++e) sh->at_o[warp][8 * sub + e] = o[e];
    }
  }
  ps_bar_consumers();
  if (has_item && tid < kHeadDim) {
    const int e = tid;
    float M = -INFINITY, Ls = 0.f, O = 0.f;
#pragma unroll 1
    for (int w = 0; w < kPsWarps; ++w) M = fmaxf(M, sh->at_m[w]);
#pragma unroll 1
    for (int w = 0; w < kPsWarps; ++w) {
      const float f = (sh->at_m[w] == -INFINITY) ? 0.f : exp2f(sh->at_m[w] - M);
      Ls = fmaf(sh->at_l[w], f, Ls);
      O = fmaf(sh->at_o[w][e], f, O);
    }
    unsigned long long *mine = a.pb + ((size_t)(at_r * H + at_h) * kPsMaxSplit + at_s) * kPsPartialWords;
    if (S > 1 && at_s != 0) {
      ps_st(mine + 2 * e, __float_as_uint(O), tg + PS_TAG_P);
      ps_st(mine + 2 * e + 1, __float_as_uint((e & 1) ? Ls : M), tg + PS_TAG_P);
    } else {
      if (S > 1) {
        // split 0: the other splits' (o[e], m | l), folded in split order
        uint32_t po[kPsMaxSplit], pq[kPsMaxSplit];
        unsigned spins = 0;
        unsigned long long tw0 = 0ull;
        const uint32_t want = tg + PS_TAG_P;
        while (true) {
          bool all = true;
#pragma unroll
          for (int s = 1; s < kPsMaxSplit; ++s) {
            unsigned long long x = (unsigned long long)want << 32, y = x;
            if (s < S) ps_ld2(mine + (size_t)s * kPsPartialWords + 2 * e, x, y);
            po[s] = (uint32_t)x; pq[s] = (uint32_t)y;
            all = all && (uint32_t)(x >> 32) == want && (uint32_t)(y >> 32) == want;
          }
          if (all) break;
          if ((++spins & 63u) == 0u) {
            tw0 = ps_spin_check(sh, tw0);
            if (tw0 == ~0ull) break;
          }
        }
        float MM = M, LL, OO;
        float pmv[kPsMaxSplit], plv[kPsMaxSplit];
#pragma unroll
        for (int s = 1; s < kPsMaxSplit; ++s) {
          const float mine_q = __uint_as_float(pq[s]);
          const float other_q = __shfl_xor_sync(0xFFFFFFFFu, mine_q, 1);   // even lanes hold m, odd lanes l
          pmv[s] = (e & 1) ? other_q : mine_q;
          plv[s] = (e & 1) ? mine_q : other_q;
          if (s < S) MM = fmaxf(MM, pmv[s]);
        }
        const float f0 = (M == -INFINITY) ? 0.f : exp2f(M - MM);
        LL = Ls * f0; OO = O * f0;
#pragma unroll
        for (int s = 1; s < kPsMaxSplit; ++s) {
          if (s < S) {
            const float f = (pmv[s] == -INFINITY) ? 0.f : exp2f(pmv[s] - MM);
            LL = fmaf(plv[s], f, LL);
            OO = fmaf(__uint_as_float(po[s]), f, OO);
          }
        }
        Ls = LL; O = OO;
      }
      ps_st(a.ob + (size_t)at_r * d + at_h * kHeadDim + e, float_to_bf16_bits(O / Ls), tg + PS_TAG_O);
    }
  }
  return item;
}

// ------------------------------------------------------------------------------------------
// the producer: one lane streams the CTA's records and K/V into the ring, in consumption order
// ------------------------------------------------------------------------------------------
struct PsProducer {
  PsShared *sh;
  unsigned char *ring;
  uint32_t size;
  uint32_t item = 0, oldest = 0, roff = 0;
  unsigned long long vpos = 0, vfree = 0;

  __device__ bool free_oldest() {
    const uint32_t slot = oldest % kPsQueue;
    volatile int *dn = &sh->done[slot];
    unsigned spins = 0;
    unsigned long long t0 = 0ull;
    while (*dn < sh->it_expect[slot]) {
      if ((++spins & 63u) == 0u) {
        t0 = ps_spin_check(sh, t0);
        if (t0 == ~0ull) return false;
      }
    }
    *dn = 0;
    vfree = sh->it_vend[slot];
    ++oldest;
    return true;
  }
  // reserves `bytes` (a multiple of 16) of ring space for the next item; returns its shared-memory address or null
  __device__ __forceinline__ unsigned char *begin(uint32_t bytes, int expect) {
    if (*reinterpret_cast<volatile int *>(&sh->abort_s)) return nullptr;
    const uint32_t al = (bytes + 127u) & ~127u;
    if (roff + al > size) { vpos += size - roff; roff = 0; }
    while (vpos + al - vfree > size || item - oldest >= (uint32_t)kPsQueue) {
      if (oldest == item || !free_oldest()) return nullptr;
    }
    const uint32_t slot = item % kPsQueue;
    sh->q_off[slot] = roff;
    sh->it_vend[slot] = vpos + al;
    sh->it_expect[slot] = expect;
    mbar_expect_tx(&sh->full[slot], bytes);
    unsigned char *dst = ring + roff;
    vpos += al; roff += al;
    return dst;
  }
  __device__ void copy(unsigned char *dst, const void *src, uint32_t bytes) {
    const uint32_t slot = item % kPsQueue;
    for (uint32_t off = 0; off < bytes; off += 16384u)
      bulk_copy_g2s(dst + off, (const unsigned char *)src + off, min(16384u, bytes - off), &sh->full[slot]);
  }
  __device__ void end() { ++item; }

};

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------
template <int WF>
__global__ void __launch_bounds__(kPsThreads, 1) step_persistent_kernel(const PsArgs a) {
  extern __shared__ __align__(128) unsigned char ps_smem[];
  PsShared *sh = reinterpret_cast<PsShared *>(ps_smem);
  const int d = a.d, F = a.d_ff, H = a.H, R = a.R, L = a.n_layer;
  float *xs = reinterpret_cast<float *>(ps_smem + ((sizeof(PsShared) + 127) & ~(size_t)127));
  uint16_t *act = reinterpret_cast<uint16_t *>(xs + (size_t)R * d);
  unsigned char *ring = reinterpret_cast<unsigned char *>(act + (size_t)R * F);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, G = gridDim.x;
  const int KS = F / d;                         // column blocks of FC2
  const int S = ps_splits(R, H, G);
  const bool has_item = cta < R * H * S;        // this CTA's (row, head, split) of the attention stage
  const int at_r = cta / (H * S), at_h = (cta / S) % H, at_s = cta % S;

  if (tid == 0) {
    for (int i = 0; i < kPsQueue; ++i) { mbar_init(&sh->full[i], 1); sh->done[i] = 0; }
    sh->abort_s = 0;
    sh->dbg_wait = 0ull;
    sh->args = a;
    sh->xs = xs; sh->act = act; sh->ring = ring;
    ps_range(3 * d, cta, G, sh->rng[0][0], sh->rng[0][1]);
    ps_range(d, cta, G, sh->rng[1][0], sh->rng[1][1]);
    ps_range(F, cta, G, sh->rng[2][0], sh->rng[2][1]);
    ps_range(a.V, cta, G, sh->rng[3][0], sh->rng[3][1]);
    sh->S = S; sh->has_item = has_item ? 1 : 0; sh->at_r = at_r; sh->at_h = at_h; sh->at_s = at_s;
    for (int r = 0; r < R; ++r) {
      const int pos = a.row_pos[r];
      sh->row_pos[r] = pos;
      sh->row_page[r] = a.page_table[(size_t)a.row_stream[r] * a.pps + (pos >> 6)];
    }
  }
  __syncthreads();

  if (warp == kPsWarps) {
    // ================= producer =================
    if (lane != 0) return;
    PsProducer pr;
    pr.sh = sh; pr.ring = ring; pr.size = a.ring_bytes;
    const int rs = ps_record_bytes(WF, d);
    int n_tok = 0, t0 = 0, t1 = 0;
    const int *pt = nullptr;
    if (has_item) {
      n_tok = a.row_pos[at_r] + 1;
      ps_split_range(n_tok, S, at_s, t0, t1);
      pt = a.page_table + (size_t)a.row_stream[at_r] * a.pps;
    }
    const int old_end = min(t1, n_tok - 1);   // the new token's K/V does not come from the pages
    // The CTA's stream as a list of entries: per layer LN1 parameters, QKV records, K/V chunks, O records,
    // LN2 parameters, FC1 records, FC2 records; then the final LayerNorm's parameters and the head's
    // records.  One emission site serves all of them.
    enum { E_LN1 = 0, E_QKV = 1, E_KV = 2, E_O = 3, E_LN2 = 4, E_FC1 = 5, E_FC2 = 6 };
    PsLayerDesc ly = a.layers[0], next = ly;
    const int n_entries = 7 * L + 2;
    for (int en = 0; en < n_entries; ++en) {
      const int l = en / 7, kind = en < 7 * L ? en % 7 : (en == 7 * L ? E_LN1 : E_QKV);
      const bool fin = en >= 7 * L;
      if (!fin && kind == E_LN1) {
        ly = next;
        if (l + 1 < L) next = a.layers[l + 1];    // requested a layer ahead of its use
      }
      const uint16_t *kvl = a.kv + a.kv_layer_elems * l;
      const bool is_ln = kind == E_LN1 || kind == E_LN2;
      // linear entries: matrix, rows, column blocks, record size
      const unsigned char *w = nullptr;
      int N = 0, ks = 1, rsz = rs;
      if (fin && kind == E_QKV) { w = a.head_w; N = a.V; rsz = ps_record_bytes(WF_BF16, d); }
      else if (kind == E_QKV) { w = ly.qkv_w; N = 3 * d; }
      else if (kind == E_O) { w = ly.o_w; N = d; }
      else if (kind == E_FC1) { w = ly.fc1_w; N = F; }
      else if (kind == E_FC2) { w = ly.fc2_w; N = d; ks = KS; }
      int n0 = 0, n1 = 0;
      ps_range(N, cta, G, n0, n1);
      const int nrows = n1 - n0, wg = kPsWarps / ks, ri = ps_rows_per_item(rsz, wg), ipq = (nrows + ri - 1) / ri;
      const int n_items = is_ln ? 1 : (kind == E_KV ? (old_end > t0 ? (old_end - t0 + kPsChunkTokens - 1) / kPsChunkTokens : 0) : ipq * ks);
      for (int ii = 0; ii < n_items; ++ii) {
        uint32_t bytes;
        int expect, p = 0, q = 0, ta = 0, nt = 0;
        if (is_ln) { bytes = (uint32_t)d * 4u; expect = kPsWarps; }
        else if (kind == E_KV) { ta = t0 + ii * kPsChunkTokens; nt = min(old_end, ta + kPsChunkTokens) - ta; bytes = (uint32_t)nt * 256u; expect = kPsWarps; }
        else { p = ii / ks; q = ii % ks; expect = min(ri, nrows - p * ri); bytes = (uint32_t)expect * rsz; }
        unsigned char *dst = pr.begin(bytes, expect);
        if (dst) {
          if (is_ln) {
            const uint16_t *g = fin ? a.lnf_g : (kind == E_LN1 ? ly.ln1_g : ly.ln2_g);
            const uint16_t *b = fin ? a.lnf_b : (kind == E_LN1 ? ly.ln1_b : ly.ln2_b);
            pr.copy(dst, g, (uint32_t)d * 2u);
            pr.copy(dst + (size_t)d * 2, b, (uint32_t)d * 2u);
          } else if (kind == E_KV) {
            for (int which = 0; which < 2; ++which) {
              unsigned char *dw = dst + (size_t)which * nt * 128;
              for (int t = ta; t < ta + nt;) {
                const int page = t >> 6, in_page = t & 63, n = min(ta + nt - t, 64 - in_page);
                const uint16_t *src = kvl + (((size_t)pt[page] * 2 + which) * H + at_h) * kPageElems + (size_t)in_page * kHeadDim;
                pr.copy(dw + (size_t)(t - ta) * 128, src, (uint32_t)n * 128u);
                t += n;
              }
            }
          } else {
            pr.copy(dst, w + ((size_t)q * N + n0 + p * ri) * rsz, bytes);
          }
        }
        pr.end();
      }
    }
    // nothing may be in flight towards this CTA's shared memory when it exits
    if (!*reinterpret_cast<volatile int *>(&sh->abort_s)) {
      while (pr.oldest < pr.item)
        if (!pr.free_oldest()) break;
    }
    for (uint32_t it = pr.oldest; it < pr.item; ++it)   // after a give-up: the copies already issued still land
      mbar_wait_bounded(&sh->full[it % kPsQueue], (it / kPsQueue) & 1u, 20000000ull);
    return;
  }

  // ================= consumers =================
  PsCtx cx;
  cx.sh = sh; cx.item = 0; cx.tag0 = a.seq << 8; cx.layer = 0;
  const bool tr = a.trace != nullptr && cta == 0 && tid == 0;
  // detail trace of one layer: 16 marks per CTA (thread 0), behind the per-layer slots of CTA 0
  unsigned long long *dt = (a.trace != nullptr && a.trace_detail && tid == 0) ? a.trace + 8 * (size_t)(L + 1) + 64 * (size_t)cta : nullptr;
  const int dl = L / 2;
#define PS_MARK(k) do { if (dt && l == dl) dt[k] = global_timer_ns(); } while (0)
  // The step as a loop over stages (5 per layer, then the LM head).  Every stage function is expanded
  // exactly once inside this loop: the code of a layer stays small enough to live in the instruction
  // cache, and nothing is called, so nothing is spilled (with all of shared memory taken by the ring, L1
  // has no room for a stack).
  enum { ST_QKV = 0, ST_ATT = 1, ST_O = 2, ST_FC1 = 3, ST_FC2 = 4 };
  const int n_stage = 5 * L + 1;
  for (int sx = 0; sx < n_stage; ++sx) {
    const bool head = sx == 5 * L;
    const int l = head ? L - 1 : sx / 5, st = head ? ST_QKV : sx % 5;
    cx.layer = l;
    const uint32_t tg = cx.tag0 + (uint32_t)l * 8u;
    if (st == ST_ATT) {
      cx.item = ps_attention(cx);
      PS_MARK(7);
      if (tr) a.trace[8 * l + 2] = global_timer_ns();
      continue;
    }
    // ---- input of the stage's linear ----
    if (sx > 0) ps_bar_consumers();   // every warp is done with the act rows of the stage before
    if (st == ST_QKV || st == ST_FC1) {
      // LayerNorm of the residual rows: LN1 (after FC2 of the layer before, or the step's input rows), LN2, final
      const unsigned long long *src = st == ST_FC1 ? a.xa : (sx == 0 ? nullptr : a.xb);
      const uint32_t want = st == ST_FC1 ? tg + PS_TAG_XA : (head ? tg + PS_TAG_XB : tg - 8u + PS_TAG_XB);
      if (st == ST_QKV) { PS_MARK(0); if (dt && l == dl) sh->dbg_wait = 0ull; }
      cx.item = ps_ln_stage(cx, src, want, (head && cta == 0 && a.io->out_hidden) ? a.io->out_hidden : nullptr);
      if (st == ST_QKV) { PS_MARK(2); if (tr && !head) a.trace[8 * l + 0] = global_timer_ns(); } else PS_MARK(11);
    } else {
      // attention output (bf16) or FC1 output (bf16)
      ps_poll_act(sh, st == ST_O ? a.ob : a.hb, st == ST_O ? d : F, tg + (st == ST_O ? PS_TAG_O : PS_TAG_H));
      if (st == ST_O) PS_MARK(8); else PS_MARK(13);
      ps_bar_consumers();
    }
    // ---- the linear ----
    const int mode = head ? PS_EPI_HEAD : (st == ST_QKV ? PS_EPI_QKV : (st == ST_FC1 ? PS_EPI_FC1 : (st == ST_O ? PS_EPI_O : PS_EPI_FC2)));
    if (WF != WF_BF16 && head) cx.item = ps_linear<WF_BF16>(cx, mode);
    else cx.item = ps_linear<WF>(cx, mode);
    if (head) { if (tr) a.trace[8 * L + 0] = global_timer_ns(); break; }
    if (st == ST_FC2) {
      // the column blocks of a row are summed in block order, then residual -> xb
      PS_MARK(14);
      ps_bar_consumers();
      const int on0 = sh->rng[1][0], own = sh->rng[1][1] - on0;
      if (tid < R * own) {
        const int r = tid / own, rel = tid % own;
        float v = sh->comb[r][0][rel];
        for (int q = 1; q < KS; ++q) v += sh->comb[r][q][rel];
        v += xs[(size_t)r * d + on0 + rel];
        ps_st(a.xb + (size_t)r * d + on0 + rel, __float_as_uint(v), tg + PS_TAG_XB);
      }
      PS_MARK(15);
      if (dt && l == dl) dt[3] = sh->dbg_wait;
    } else if (st == ST_QKV) PS_MARK(4); else if (st == ST_O) { PS_MARK(9); if (a.trace_detail && l == dl) { ps_bar_consumers(); if (dt) { for (int w = 0; w < kPsWarps; ++w) for (int k = 0; k < 4; ++k) dt[16 + 4 * w + k] = sh->dbg_t[w][k]; } } } else PS_MARK(12);  // TEMPDBG
    if (tr) a.trace[8 * l + (st == ST_QKV ? 1 : st == ST_O ? 3 : st == ST_FC1 ? 4 : 5)] = global_timer_ns();
  }
#undef PS_MARK
}

inline size_t ps_smem_bytes(int d, int d_ff, int R, uint32_t ring) { return ps_fixed_smem(d, d_ff, R) + ring; }

template <int WF>
inline cudaError_t launch_ps_inst(const PsArgs &a, int grid, size_t smem, cudaStream_t st) {
  static PerDeviceOnce once;
  if (once.first()) {
    int dev = 0, optin = 0;   // the ring takes what a step's fixed buffers leave: opt in to all a CTA may have
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    cudaError_t e = cudaFuncSetAttribute(step_persistent_kernel<WF>, cudaFuncAttributeMaxDynamicSharedMemorySize, optin);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg;
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kPsThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeCooperative;
  at[0].val.cooperative = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, step_persistent_kernel<WF>, a);
}

inline cudaError_t launch_step_persistent(int wf, const PsArgs &a, int grid, size_t smem, cudaStream_t st) {
  if (wf == WF_BF16) return launch_ps_inst<WF_BF16>(a, grid, smem, st);
  if (wf == WF_INT8) return launch_ps_inst<WF_INT8>(a, grid, smem, st);
  return launch_ps_inst<WF_INT4>(a, grid, smem, st);
}

}  // namespace ttsgpt
