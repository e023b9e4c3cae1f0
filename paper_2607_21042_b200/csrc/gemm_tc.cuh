// Batched linear on the 5th-generation tensor cores (tcgen05) for more than 16 rows: at these
// batch sizes the layer is a dense contraction out[b,n] = sum_k W[n,k] act[b,k], bf16 operands,
// fp32 accumulation in tensor memory (Table I / III regime: many concurrent utterances).
//
// Operand images.  Both operands are kept in global memory in exactly the byte order the tensor
// core wants them in shared memory (K-major, 128-byte swizzle): a k-chunk of 64 columns of 128
// rows is one 16 KB block in which row r sits at byte r*128 and the 16-byte unit u of that row is
// stored at unit (u ^ (r % 8)).  Weights [N,K] become blocks [n/128][k/64]; activations of up to
// 128 rows become blocks [k/64] (rows are batch rows, so the 32 rows of a batch chunk are 4 KB
// contiguous inside a block).  A stage of the pipeline is therefore filled by two plain bulk
// asynchronous copies (16 KB of weights, 4 KB of activations): no tensor maps, no alignment rules
// beyond 16 bytes.  The kernels that produce activations (LayerNorm, attention, the GELU epilogue
// below) write this image directly.
//
// A CTA owns a 128-row weight tile (the M operand), one chunk of 32 batch rows (the N operand) and
// a contiguous range of k-chunks; with 4 batch chunks of 32 and, for the two linears that feed the
// residual stream, 4 k-ranges, every linear of the block runs on 120-160 CTAs.  Warp 0 produces
// (bulk copies into a 4-stage ring guarded by full/empty mbarriers; the weight copies of the first
// stages are issued before the dependency wait), warps 1 and 10 issue the MMAs (4 per k-chunk, M=128,
// N=32, K=16; even and odd k-chunks into two accumulators) and commit each stage back to the producer, and warps 2-9 read the 128x32 fp32
// accumulator out of tensor memory and run the epilogue.  K-split partial sums go to a scratch
// array that the following LayerNorm kernel folds into the residual stream in a fixed order.
// Every wait is bounded; on expiry the CTA sets the error word, stops waiting and still releases
// its tensor memory.
#pragma once
#include "common.cuh"
#include "linear.cuh"

namespace ttsgpt {

// Measured on B200 (FC1 shape, 128 rows): chunks of 32 rows with a 5-stage ring (160 CTAs, two per
// SM) beat chunks of 64 rows with 4 or 8 stages by 6-13 us per linear although the latter re-read
// the weights from L2 only twice: more CTAs keep more copies in flight and overlap their epilogues.
constexpr int kTcStages = 4;            // even: a stage is always consumed by the same MMA issuer (see the issuers); 4 x 20 KB
constexpr int kTcTileM = 128;          // weight rows per CTA
constexpr int kTcChunkN = 32;          // batch rows per CTA (the N operand; weights are re-read once per chunk)
constexpr int kTcKChunk = 64;          // columns per pipeline stage (128 bytes of bf16)
constexpr uint32_t kTcABytes = kTcTileM * 128;   // 16 KB
constexpr uint32_t kTcBBytes = kTcChunkN * 128;  // 4 KB
static_assert(kTcChunkN == 32, "the epilogue reads one 32-column accumulator slice per thread");
constexpr int kTcThreads = 352;          // warp 0: producer, warp 1: MMA issuer, warps 2-9: epilogue
constexpr int kTcEpiThreads = 256;
constexpr int kTcEpiCols = 16;           // accumulator columns (batch rows) per epilogue thread: two warps share a lane quarter
constexpr int kTcKSplit = 4;            // k-ranges of the two linears that feed the residual stream
constexpr unsigned long long kTcWaitNs = 2000000000ull;

// byte offset of element (row, k) inside an operand image whose blocks hold `rows_per_block` rows
__host__ __device__ inline size_t image_offset(int row, int k, int rows_per_block) {
  const int kc = k >> 6, u = (k & 63) >> 3;
  return (size_t)kc * rows_per_block * 128 + (size_t)row * 128 + (size_t)((u ^ (row & 7)) << 4) + (size_t)(k & 7) * 2;
}
inline size_t weight_image_bytes(int N, int K) { return (size_t)((N + 127) / 128) * (K / 64) * kTcABytes; }
inline size_t act_image_bytes(int K) { return (size_t)(K / 64) * kMaxRows * 128; }

// canonical bf16 [N,K] -> weight image, one thread per 16-byte unit of the destination
__global__ void pack_weight_image_kernel(const uint16_t *__restrict__ w, int N, int K, uint4 *__restrict__ dst) {
  const int KC = K / 64;
  const size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t total = (size_t)((N + 127) / 128) * KC * (kTcABytes / 16);
  if (unit >= total) return;
  const int within = unit % (kTcABytes / 16);
  const size_t blk = unit / (kTcABytes / 16);
  const int kc = blk % KC, nt = blk / KC;
  const int r = within >> 3, pu = within & 7;   // row in tile, physical 16-byte unit
  const int u = pu ^ (r & 7);                   // logical unit stored there
  const int n = nt * 128 + r, k = kc * 64 + u * 8;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (n < N) v = *reinterpret_cast<const uint4 *>(w + (size_t)n * K + k);
  dst[unit] = v;
}

// Quantized formats: the image holds the integer codes widened to bf16 (exact: |q| <= 127), the
// scales multiply fp32 sums later (per row in the epilogue for int8, per row and 128-column group
// for int4), so the tensor-core path dequantizes exactly like the register path does.
__device__ __forceinline__ uint32_t two_ints_to_bf16x2(int lo, int hi) {
  return pack_bf16x2((float)lo, (float)hi);
}
__global__ void pack_weight_image_int8_kernel(const int8_t *__restrict__ w, int N, int K, uint4 *__restrict__ dst) {
  const int KC = K / 64;
  const size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (unit >= (size_t)((N + 127) / 128) * KC * (kTcABytes / 16)) return;
  const int within = unit % (kTcABytes / 16);
  const size_t blk = unit / (kTcABytes / 16);
  const int kc = blk % KC, nt = blk / KC;
  const int r = within >> 3, u = (within & 7) ^ (r & 7);
  const int n = nt * 128 + r, k = kc * 64 + u * 8;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (n < N) {
    const int8_t *p = w + (size_t)n * K + k;
    v.x = two_ints_to_bf16x2(p[0], p[1]); v.y = two_ints_to_bf16x2(p[2], p[3]);
    v.z = two_ints_to_bf16x2(p[4], p[5]); v.w = two_ints_to_bf16x2(p[6], p[7]);
  }
  dst[unit] = v;
}
__global__ void pack_weight_image_int4_kernel(const uint32_t *__restrict__ w, int N, int K, uint4 *__restrict__ dst) {
  const int KC = K / 64;
  const size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (unit >= (size_t)((N + 127) / 128) * KC * (kTcABytes / 16)) return;
  const int within = unit % (kTcABytes / 16);
  const size_t blk = unit / (kTcABytes / 16);
  const int kc = blk % KC, nt = blk / KC;
  const int r = within >> 3, u = (within & 7) ^ (r & 7);
  const int n = nt * 128 + r, k = kc * 64 + u * 8;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (n < N) {
    const uint32_t word = w[(size_t)n * (K / 8) + k / 8];   // canonical: nibble j = column k + j, stored as q + 8
    int q[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) q[j] = (int)((word >> (4 * j)) & 15u) - 8;
    v.x = two_ints_to_bf16x2(q[0], q[1]); v.y = two_ints_to_bf16x2(q[2], q[3]);
    v.z = two_ints_to_bf16x2(q[4], q[5]); v.w = two_ints_to_bf16x2(q[6], q[7]);
  }
  dst[unit] = v;
}

// int4 weights: the operand images of a layer's four linears written from the packed streaming layout of
// linear.cuh (half a byte per weight), either dequantized (code x group scale, rounded once to bf16: the
// linears then run as plain bf16 contractions) or as the integer codes (raw: the grouped kernels scale fp32
// group sums).  One thread per 16-byte unit of the source = 32 columns of one row inside one 128-column
// group = four 16-byte units of one k-chunk of the image.  Image rows past the last 8-row tile of the
// source are never written: the caller zeroes the image first.
struct Int4ImageArgs {
  const uint4 *src[4];         // packed int4 tiles [row tile of 8][K/128][32 lanes]
  uint4 *dst[4];               // operand images
  const uint16_t *scales[4];   // tiled scales [N/8][K/128][8]
  int K[4];
  int raw;                     // 1: integer codes, 0: code x scale
  unsigned long long unit_end[4];   // running totals of source units
};
__global__ void __launch_bounds__(256) int4_weight_images_kernel(const Int4ImageArgs a) {
  const unsigned long long unit = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  int s = 0;
  while (s < 3 && unit >= a.unit_end[s]) ++s;
  const bool live = unit < a.unit_end[3];
  uint4 v = make_uint4(0, 0, 0, 0);
  float sc = 0.f;
  uint4 *out = nullptr;
  if (live) {
    const size_t local = (size_t)(unit - (s ? a.unit_end[s - 1] : 0ull));
    const int KB = a.K[s] / 128, KC = a.K[s] / 64;
    const int lane = (int)(local & 31);
    const size_t tile = local >> 5;
    const int kb = (int)(tile % KB), rt = (int)(tile / KB);
    const int row = rt * 8 + (lane >> 2), k = kb * 128 + 32 * (lane & 3);
    v = __ldg(a.src[s] + local);
    sc = a.raw ? 1.0f : bf16_bits_to_float(__ldg(a.scales[s] + ((size_t)rt * KB + kb) * 8 + (row & 7)));
    // units (k % 64) / 8 .. + 3 of image row `row`, k-chunk k / 64; logical unit u sits at u ^ (row % 8)
    out = a.dst[s] + ((size_t)(row >> 7) * KC + (k >> 6)) * (kTcABytes / 16) + (size_t)(row & 127) * 8;
  }
  if (live) {
    const int lane = (int)(unit & 31);   // unit_end values are multiples of 32
    const int row7 = (lane >> 2) & 7, u0 = ((32 * (lane & 3)) & 63) >> 3;
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t y[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t pair = (w[q] >> (4 * e)) & 0x000F000Fu;   // columns 2e, 2e+1 of the word, stored as code + 8
        y[e] = pack_bf16x2((float)((int)(pair & 0xffffu) - 8) * sc, (float)((int)(pair >> 16) - 8) * sc);
      }
      out[(u0 + q) ^ row7] = make_uint4(y[0], y[1], y[2], y[3]);
    }
  }
}

inline cudaError_t launch_pack_image(int wf, int N, int K, const void *w, void *img, cudaStream_t st) {
  const size_t units = weight_image_bytes(N, K) / 16;
  const unsigned blocks = (unsigned)((units + 255) / 256);
  if (wf == WF_BF16) pack_weight_image_kernel<<<blocks, 256, 0, st>>>((const uint16_t *)w, N, K, (uint4 *)img);
  else if (wf == WF_INT8) pack_weight_image_int8_kernel<<<blocks, 256, 0, st>>>((const int8_t *)w, N, K, (uint4 *)img);
  else pack_weight_image_int4_kernel<<<blocks, 256, 0, st>>>((const uint32_t *)w, N, K, (uint4 *)img);
  return cudaGetLastError();
}

// plain bf16 [B,K] -> activation image (used by the stand-alone entry point)
__global__ void pack_act_image_kernel(const uint16_t *__restrict__ act, int B, int K, unsigned char *__restrict__ dst) {
  const int k8 = K >> 3;
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)B * k8) return;
  const int b = idx / k8, k = (int)(idx % k8) * 8;
  *reinterpret_cast<uint4 *>(dst + image_offset(b, k, kMaxRows)) = *reinterpret_cast<const uint4 *>(act + (size_t)b * K + k);
}

// ---- tcgen05 / tensor-memory primitives ----
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// arrives on the mbarrier once every MMA issued so far by this thread has completed
__device__ __forceinline__ void tc_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// K-major, 128-byte swizzle: 8-row groups 1024 bytes apart, version 1, layout type 2
__device__ __forceinline__ uint64_t tc_smem_desc(const void *p) {
  const uint32_t a = smem_u32(p);
  uint64_t d = 0;
  d |= (uint64_t)((a >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;                 // leading-dimension byte offset (unused with swizzle), in 16-byte units
  d |= (uint64_t)(1024 >> 4) << 32;       // stride-dimension byte offset: next 8-row group
  d |= (uint64_t)1 << 46;                 // descriptor version
  d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
  return d;
}
// bf16 x bf16 -> fp32, both operands K-major
__device__ __forceinline__ uint32_t tc_instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// 32 lanes x 32 columns of 32-bit: register c of lane l = TMEM[lane base + l][column base + c]
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// 32 lanes x 16 columns of 32-bit
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

struct GemmTcArgs {
  const void *w_img;        // weight image [N/128][K/64] blocks
  const void *act_img;      // activation image [K/64] blocks of 128 rows
  const uint16_t *bias;     // bf16 [N] or null
  const uint16_t *scales;   // tiled scales of linear.cuh: int8 [N/8][8]; int4 [N/8][K/128][8]
  int wfmt;                 // WF_* : bf16 = no scale, int8 = per row, int4 = per row and 128-column group
  int N, K, B, mode;        // mode: EPI_* of linear.cuh
  int ksplit;               // k-ranges (gridDim.z)
  int stages;               // wide kernel: ring depth, set by its launcher
  float *out_f32;           // EPI_F32: out[b*out_stride+n]; EPI_QKV: q; EPI_RESID: x (ksplit == 1) or partials [ksplit][128][N]
  int out_stride;
  void *out_img;            // EPI_GELU: activation image of the next linear (row length N)
  int gelu_tanh;
  uint16_t *kv_layer;
  uint16_t *kv_stage;       // if set, K/V rows go here as bf16 [B][2][d] instead of into their page slots (8-bit KV cache)
  const int *page_table, *row_stream, *row_pos;
  int pps, d, H;
  int *err;
  unsigned long long *trace;  // optional timeline trace (see trace_mark)
  int trace_slot;
};

// a wait that gives up for good once any wait of the CTA has expired
__device__ __forceinline__ void tc_wait(uint64_t *bar, uint32_t parity, volatile int *failed, int *err) {
  if (*failed) return;
  if (!mbar_wait_bounded(bar, parity, kTcWaitNs)) {
    *failed = 1;
    if (err) atomicExch(err, 1);
  }
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// GROUPED (int4 weights): the MMAs of each 128-column group accumulate into one of two 32-column
// tensor-memory buffers; while the next group runs in the other buffer, the epilogue warps read the
// finished group out, multiply it by the group's scale of their weight row and add it to fp32
// registers.  Otherwise one 32-column accumulator collects the whole k-range.
template <bool GROUPED>
__global__ void __launch_bounds__(kTcThreads) gemm_tc_kernel(const GemmTcArgs a) {
  extern __shared__ __align__(16) unsigned char tc_smem_raw[];
  // [stages x (A 16 KB | B 4 KB)] on a 1024-byte boundary (the swizzle pattern repeats every 1024
  // bytes of shared-memory address), then barriers and small state
  unsigned char *ring = tc_smem_raw + ((1024u - (smem_u32(tc_smem_raw) & 1023u)) & 1023u);
  uint64_t *full = reinterpret_cast<uint64_t *>(ring + kTcStages * (kTcABytes + kTcBBytes));
  uint64_t *empty = full + kTcStages;
  uint64_t *acc_done = empty + kTcStages;
  uint64_t *grp_done = acc_done + 1;   // [2] group buffer filled (MMA warp -> all)
  uint64_t *grp_free = grp_done + 2;   // [2] group buffer read out (all epilogue threads -> MMA warp)
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(grp_free + 2);
  volatile int *failed = reinterpret_cast<volatile int *>(tmem_slot + 1);
  uint16_t **kv_base = reinterpret_cast<uint16_t **>(tmem_slot + 4);   // [32] EPI_QKV: page slot of each batch row

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nt = blockIdx.x, bc = blockIdx.y, ks = blockIdx.z;
  trace_mark(a.trace, a.trace_slot, 0);
  const int KC = a.K / kTcKChunk;
  int per = (KC + a.ksplit - 1) / a.ksplit;
  if (GROUPED) per = (per + 1) & ~1;   // k-ranges hold whole 128-column groups (2 k-chunks each)
  const int kc0 = ks * per, kc1 = min(KC, kc0 + per);
  const int n_it = kc1 - kc0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kTcStages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    mbar_init(acc_done, GROUPED ? 1 : 2);   // both MMA issuers commit to it
    mbar_init(grp_done, 1); mbar_init(grp_done + 1, 1);
    mbar_init(grp_free, kTcEpiThreads); mbar_init(grp_free + 1, kTcEpiThreads);
    *failed = 0;
  }
  if (warp == 0) tmem_alloc(tmem_slot, 2 * kTcChunkN);
  if (a.mode == EPI_QKV && threadIdx.x >= 64 && threadIdx.x < 64 + kTcChunkN) {   // page slots of this chunk's batch rows
    const int bl = threadIdx.x - 64;
    const int b = bc * kTcChunkN + bl;
    uint16_t *p = nullptr;
    if (b < a.B) {
      if (a.kv_stage) {
        p = a.kv_stage + (size_t)b * 2 * a.d;
      } else {
        const int pos = a.row_pos[b];
        const int page = a.page_table[(size_t)a.row_stream[b] * a.pps + (pos >> 6)];
        p = a.kv_layer + ((size_t)page * 2 * a.H) * kPageElems + (size_t)(pos & 63) * kHeadDim;
      }
    }
    kv_base[bl] = p;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_d = *tmem_slot;

  const unsigned char *gA = reinterpret_cast<const unsigned char *>(a.w_img) + ((size_t)nt * KC + kc0) * kTcABytes;
  const unsigned char *gB = reinterpret_cast<const unsigned char *>(a.act_img) + (size_t)kc0 * (kMaxRows * 128) + (size_t)bc * kTcBBytes;

  const int pre = min(n_it, kTcStages);
  if (threadIdx.x == 0) {
    for (int i = 0; i < pre; ++i) {   // weights do not depend on the previous kernel
      mbar_expect_tx(full + i, kTcABytes + kTcBBytes);
      bulk_copy_g2s(ring + (size_t)i * (kTcABytes + kTcBBytes), gA + (size_t)i * kTcABytes, kTcABytes, full + i);
    }
  }
  // per-row epilogue constants do not depend on the kernel in front either
  float e_rsc = 1.f, e_bias = 0.f;
  if (warp >= 2) {
    const int n = nt * kTcTileM + (warp & 3) * 32 + lane;
    if (n < a.N) {
      if (a.wfmt == WF_INT8) e_rsc = bf16_bits_to_float(a.scales[n]);   // per-row scale of the integer codes
      if (a.bias && (a.mode != EPI_RESID || a.ksplit == 1)) e_bias = bf16_bits_to_float(a.bias[n]);
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  trace_mark(a.trace, a.trace_slot, 1);
  if (warp == 0) {
    // ---- producer ----
    if (lane == 0) {
      for (int i = 0; i < pre; ++i)
        bulk_copy_g2s(ring + (size_t)i * (kTcABytes + kTcBBytes) + kTcABytes, gB + (size_t)i * (kMaxRows * 128), kTcBBytes, full + i);
      for (int i = pre; i < n_it; ++i) {
        const int s = i % kTcStages;
        tc_wait(empty + s, ((i / kTcStages) - 1) & 1, failed, a.err);
        mbar_expect_tx(full + s, kTcABytes + kTcBBytes);
        bulk_copy_g2s(ring + (size_t)s * (kTcABytes + kTcBBytes), gA + (size_t)i * kTcABytes, kTcABytes, full + s);
        bulk_copy_g2s(ring + (size_t)s * (kTcABytes + kTcBBytes) + kTcABytes, gB + (size_t)i * (kMaxRows * 128), kTcBBytes, full + s);
      }
      trace_mark(a.trace, a.trace_slot, 3);   // last copy issued
    }
    __syncwarp();   // the warp arrives at the final barrier as a whole
  } else if (warp == 1 || warp == 10) {
    // ---- MMA issuers: two threads of different warps, each with its own accumulator.  Ungrouped:
    //      warp 1 takes the even k-chunks into accumulator 0, warp 10 the odd ones into accumulator 1; the
    //      epilogue adds the two.  Measured: the rate of the chain stays what it is (about 0.33 us per
    //      k-chunk and CTA), but the accumulators are complete 0.8 us after the last stage is handed over
    //      instead of 1.35 us.  The ring has an even number of stages so that a stage is always consumed
    //      by the same issuer: a thread may wait on an mbarrier at most one phase ahead, and with an odd
    //      ring the issuer that runs ahead would ask for a phase whose predecessor is still pending and
    //      be told it is complete ----
    const int par = GROUPED ? 0 : (warp == 10 ? 1 : 0);
    const int stride = GROUPED ? 1 : 2;
    if (lane == 0 && !(GROUPED && warp == 10)) {
      const uint32_t idesc = tc_instr_desc(kTcTileM, kTcChunkN);
      for (int i = par; i < n_it; i += stride) {
        const int s = i % kTcStages;
        tc_wait(full + s, (i / kTcStages) & 1, failed, a.err);
        const int g = i >> 1;   // group of this k-chunk inside the k-range
        if (GROUPED && (i & 1) == 0 && g >= 2) tc_wait(grp_free + (g & 1), ((g >> 1) - 1) & 1, failed, a.err);
        tc_fence_after_sync();
        const unsigned char *sa = ring + (size_t)s * (kTcABytes + kTcBBytes);
        const uint64_t da = tc_smem_desc(sa), db = tc_smem_desc(sa + kTcABytes);
        const uint32_t dst = GROUPED ? tmem_d + (uint32_t)(g & 1) * kTcChunkN : tmem_d + (uint32_t)par * kTcChunkN;
#pragma unroll
        for (int j = 0; j < kTcKChunk / 16; ++j) {  // 32 bytes further along K per step: +2 in 16-byte units
          const bool fresh = GROUPED ? ((i & 1) == 0 && j == 0) : (i == par && j == 0);
          tc_mma(dst, da + 2 * j, db + 2 * j, idesc, fresh ? 0u : 1u);
        }
        tc_commit(empty + s);   // the stage may be refilled once these MMAs have read it
        if (GROUPED && ((i & 1) == 1 || i == n_it - 1)) tc_commit(grp_done + (g & 1));
      }
      if (!GROUPED) tc_commit(acc_done);
    }
    __syncwarp();   // as above
  }

  // ---- epilogue (warps 2-9; warps w and w+4 share a lane quarter and take 16 columns each): a warp may touch the 32 accumulator lanes 32*(warp%4)..+31 = weight
  //      rows n; columns = batch rows ----
  if (warp >= 2 && warp < 10) {
  const int lw = warp & 3;
  const int c0 = ((warp - 2) >> 2) * kTcEpiCols;   // this thread's first accumulator column
  const int n = nt * kTcTileM + lw * 32 + lane;
  float v[kTcEpiCols];
  if (GROUPED) {
#pragma unroll
    for (int c = 0; c < kTcEpiCols; ++c) v[c] = 0.f;
    const int n_groups = (n_it + 1) >> 1;
    const int KG = a.K / 128;
    for (int g = 0; g < n_groups; ++g) {
      // scale of this thread's weight row for the group (tiled scales: [n/8][K/128][8])
      float sc = 0.f;
      if (n < a.N) sc = bf16_bits_to_float(a.scales[((size_t)(n >> 3) * KG + (kc0 >> 1) + g) * 8 + (n & 7)]);
      tc_wait(grp_done + (g & 1), (g >> 1) & 1, failed, a.err);
      tc_fence_after_sync();
      __syncwarp();
      float t[kTcEpiCols];
      tmem_ld16(tmem_d + ((uint32_t)(lw * 32) << 16) + (uint32_t)(g & 1) * 32u + (uint32_t)c0, t);
      tc_fence_before_sync();
      mbar_arrive(grp_free + (g & 1));   // the buffer may take the group after next
#pragma unroll
      for (int c = 0; c < kTcEpiCols; ++c) v[c] = fmaf(sc, t[c], v[c]);
    }
  } else {
    tc_wait(acc_done, 0, failed, a.err);
    trace_mark(a.trace, a.trace_slot, 4, 64);   // accumulator complete
    tc_fence_after_sync();
    __syncwarp();
    tmem_ld16(tmem_d + ((uint32_t)(lw * 32) << 16) + (uint32_t)c0, v);
    if (n_it >= 2) {   // the odd k-chunks' accumulator
      float t2[kTcEpiCols];
      tmem_ld16(tmem_d + ((uint32_t)(lw * 32) << 16) + (uint32_t)kTcChunkN + (uint32_t)c0, t2);
#pragma unroll
      for (int c = 0; c < kTcEpiCols; ++c) v[c] += t2[c];
    }
    trace_mark(a.trace, a.trace_slot, 5, 64);   // accumulator in registers
  }
  if (n_it <= 0) {   // an empty k-range contributes nothing (the accumulator was never written)
#pragma unroll
    for (int c = 0; c < kTcEpiCols; ++c) v[c] = 0.f;
  }
  if (n < a.N && !*failed) {
    // one straight-line store loop per destination kind: a single loop that branches on the epilogue
    // mode for every batch row compiled into code whose speed varied 2-4x with unrelated edits
    const int nb = min(kTcEpiCols, a.B - bc * kTcChunkN - c0);   // real batch rows among this thread's columns
#pragma unroll
    for (int c = 0; c < kTcEpiCols; ++c) v[c] = fmaf(v[c], e_rsc, e_bias);   // int8: per-row scale (1 otherwise), then bias
    if (a.mode == EPI_GELU) {
      if (a.gelu_tanh) {
#pragma unroll
        for (int c = 0; c < kTcEpiCols; ++c) v[c] = gelu_tanh_f(v[c]);
      } else {
#pragma unroll
        for (int c = 0; c < kTcEpiCols; ++c) v[c] = gelu_erf_f(v[c]);
      }
      // element (b, n) of the next linear's activation image: rows are 128 bytes apart, the 16-byte
      // unit of column n moves with b % 8 (swizzle)
      unsigned char *img = reinterpret_cast<unsigned char *>(a.out_img) + (size_t)(n >> 6) * (kMaxRows * 128) + (size_t)(n & 7) * 2;
      const int u = (n & 63) >> 3;
#pragma unroll
      for (int c = 0; c < kTcEpiCols; ++c) {
        const int b = bc * kTcChunkN + c0 + c;
        if (c < nb) *reinterpret_cast<uint16_t *>(img + (size_t)b * 128 + (size_t)((u ^ (b & 7)) << 4)) = float_to_bf16_bits(v[c]);
      }
    } else if (a.mode == EPI_QKV && n >= a.d) {
      const int which = n >= 2 * a.d;
      const int col = n - (which ? 2 * a.d : a.d);
      const size_t off = a.kv_stage ? (size_t)which * a.d + col : ((size_t)which * a.H + (col >> 6)) * kPageElems + (col & 63);
#pragma unroll
      for (int c = 0; c < kTcEpiCols; ++c)
        if (c < nb) kv_base[c0 + c][off] = float_to_bf16_bits(v[c]);
    } else {
      // fp32 rows: logits, q, the residual stream, or this k-range's partial sums
      const bool partial = a.mode == EPI_RESID && a.ksplit > 1;
      float *dst = partial ? a.out_f32 + ((size_t)ks * kMaxRows + bc * kTcChunkN + c0) * a.N + n
                           : a.out_f32 + (size_t)(bc * kTcChunkN + c0) * a.out_stride + n;
      const size_t step = partial ? (size_t)a.N : (size_t)a.out_stride;
      if (a.mode == EPI_RESID && !partial) {
#pragma unroll
        for (int c = 0; c < kTcEpiCols; ++c)
          if (c < nb) dst[c * step] += v[c];
      } else {
#pragma unroll
        for (int c = 0; c < kTcEpiCols; ++c)
          if (c < nb) dst[c * step] = v[c];
      }
    }
  }
  trace_mark(a.trace, a.trace_slot, 6, 64);     // this thread's epilogue done
  }
  tc_fence_before_sync();
  __syncthreads();
  trace_mark(a.trace, a.trace_slot, 2, 64);   // by an epilogue thread: its own stores precede the mark
  if (warp == 0) tmem_dealloc(tmem_d, 2 * kTcChunkN);
}

// ------------------------------------------------------------------------------------------
// Wide variant for passes of more than 128 rows (prefill): all 128 rows of a row tile in one
// instruction.
//
// A tcgen05.mma with M = 128 takes about 72 ns on this part whether its N extent is 32 or 128, so
// the kernel above, whose instructions are 32 batch rows wide, wastes three quarters of each.  It
// still wins while a pass has at most 128 rows, because it spreads a linear over four times as many
// CTAs without any merge.  A prefill pass of several row tiles has enough independent output tiles
// for the wide shape: here the operand roles are swapped, the activation block of a k-chunk (128
// rows x 64 columns, 16 KB) is the M operand, a 128-row weight block the N operand, and one CTA
// computes a whole [128 rows] x [128 output features] tile for its k-range: K/16 instructions where
// four CTAs of the kernel above issue K/16 each, and the weights cross from L2 once per 128 rows
// instead of once per 32.  Grid = feature tiles x k-ranges x row tiles.  Accumulator lane = row,
// column = output feature; the epilogue parks the accumulator rows in the idle ring and writes
// them out with the lanes along the row.  The residual linears split K over up to 4 CTAs whose
// partial sums the next LayerNorm folds (partials [row tile][range][128][N]); the others take all
// of K in one CTA.
constexpr int kTwMaxStages = 6;                 // ring depth: 6 stages with one CTA per SM, 3 when two CTAs share an SM
constexpr uint32_t kTwStageBytes = 2 * 16384;   // activations (M operand) | weights (N operand)
constexpr int kTwThreads = 320;                 // warp 0 producer, warp 1 MMA issuer, warps 2-9 epilogue
constexpr int kTwMaxPartials = 4;               // k-ranges the following LayerNorm folds


// bf16 destinations of the wide kernel's epilogue: four parked rows per instruction, lane = (row in the group
// of four, 16-byte unit = 8 features).  KIND 0: tanh-GELU into the next linear's activation image, 1: erf-GELU
// into it, 2: K/V rows into their page slots (or the staging rows of the 8-bit cache).
template <int KIND>
__device__ __forceinline__ void tw_rows_bf16(const unsigned char *patch, int rows, int r4, int u, int lw, const float (&sc8)[8],
                                             const float (&bi8)[8], unsigned char *blk, uint16_t *const *kv_base, size_t kv_off) {
#pragma unroll 2
  for (int r = r4; r < rows; r += 4) {
    const int bb = lw * 32 + r;
    float x[8];
    *reinterpret_cast<float4 *>(x) = *reinterpret_cast<const float4 *>(patch + r * 272 + u * 32);
    *reinterpret_cast<float4 *>(x + 4) = *reinterpret_cast<const float4 *>(patch + r * 272 + u * 32 + 16);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      x[e] = fmaf(x[e], sc8[e], bi8[e]);
      if (KIND == 0) x[e] = gelu_tanh_f(x[e]);
      if (KIND == 1) x[e] = gelu_erf_f(x[e]);
    }
    const uint4 pk = make_uint4(pack_bf16x2(x[0], x[1]), pack_bf16x2(x[2], x[3]), pack_bf16x2(x[4], x[5]), pack_bf16x2(x[6], x[7]));
    if (KIND == 2) reinterpret_cast<uint4 *>(kv_base[bb] + kv_off)[u] = pk;
    else *reinterpret_cast<uint4 *>(blk + (size_t)bb * 128 + ((u ^ (bb & 7)) << 4)) = pk;   // the unit moves with bb % 8
  }
}

template <bool GROUPED>
__global__ void __launch_bounds__(kTwThreads) gemm_tcw_kernel(const GemmTcArgs a) {
  extern __shared__ __align__(16) unsigned char tc_smem_raw[];
  unsigned char *ring = tc_smem_raw + ((1024u - (smem_u32(tc_smem_raw) & 1023u)) & 1023u);
  const int n_stage = a.stages;
  uint64_t *full = reinterpret_cast<uint64_t *>(ring + n_stage * kTwStageBytes);
  uint64_t *empty = full + kTwMaxStages;
  uint64_t *acc_done = empty + kTwMaxStages;
  uint64_t *grp_done = acc_done + 1;   // [2]
  uint64_t *grp_free = grp_done + 2;   // [2]
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(grp_free + 2);
  volatile int *failed = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float *s_bias = reinterpret_cast<float *>(tmem_slot + 6);         // [128] bias of this tile's features (16-byte aligned)
  float *s_rsc = s_bias + 128;                                      // [128] int8: per-feature scale, else 1
  uint16_t **kv_base = reinterpret_cast<uint16_t **>(s_rsc + 128);  // [128] EPI_QKV: where batch row b's K/V go

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nt = blockIdx.x, ks = blockIdx.y;
  const int row0 = blockIdx.z * kMaxRows;              // first row of this CTA's row tile
  const int Bt = min(kMaxRows, a.B - row0);            // rows of the tile
  trace_mark(a.trace, a.trace_slot, 0);
  const int KC = a.K / kTcKChunk;
  int per = (KC + a.ksplit - 1) / a.ksplit;
  if (GROUPED) per = (per + 1) & ~1;   // k-ranges hold whole 128-column groups (2 k-chunks each)
  const int kc0 = min(KC, ks * per), kc1 = min(KC, kc0 + per);
  const int n_it = kc1 - kc0;
  constexpr uint32_t kCols = GROUPED ? 256u : 128u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stage; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    mbar_init(acc_done, 1);
    mbar_init(grp_done, 1); mbar_init(grp_done + 1, 1);
    mbar_init(grp_free, kTcEpiThreads); mbar_init(grp_free + 1, kTcEpiThreads);
    *failed = 0;
  }
  if (warp == 0) tmem_alloc(tmem_slot, kCols);
  if (threadIdx.x >= 64 && threadIdx.x < 192) {
    const int b = threadIdx.x - 64;
    uint16_t *p = nullptr;
    if (a.mode == EPI_QKV && b < Bt) {
      if (a.kv_stage) {
        p = a.kv_stage + (size_t)(row0 + b) * 2 * a.d;
      } else {
        const int pos = a.row_pos[row0 + b];
        const int page = a.page_table[(size_t)a.row_stream[row0 + b] * a.pps + (pos >> 6)];
        p = a.kv_layer + ((size_t)page * 2 * a.H) * kPageElems + (size_t)(pos & 63) * kHeadDim;
      }
    }
    kv_base[b] = p;
  } else if (threadIdx.x >= 192) {
    const int c = threadIdx.x - 192;
    const int n = nt * 128 + c;
    float rs = 1.f, bi = 0.f;
    if (n < a.N) {
      if (a.wfmt == WF_INT8) rs = bf16_bits_to_float(a.scales[n]);
      if (a.bias && !(a.mode == EPI_RESID && a.ksplit > 1)) bi = bf16_bits_to_float(a.bias[n]);
    }
    s_rsc[c] = rs; s_bias[c] = bi;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_d = *tmem_slot;

  const unsigned char *gW = reinterpret_cast<const unsigned char *>(a.w_img) + ((size_t)nt * KC + kc0) * kTcABytes;
  const unsigned char *gX = reinterpret_cast<const unsigned char *>(a.act_img) + ((size_t)blockIdx.z * KC + kc0) * (kMaxRows * 128);

  const int pre = min(n_it, n_stage);
  if (threadIdx.x == 0) {
    for (int i = 0; i < pre; ++i) {   // weights do not depend on the previous kernel
      mbar_expect_tx(full + i, kTwStageBytes);
      bulk_copy_g2s(ring + (size_t)i * kTwStageBytes + 16384, gW + (size_t)i * kTcABytes, 16384, full + i);
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  trace_mark(a.trace, a.trace_slot, 1);
  if (warp == 0) {
    if (lane == 0) {
      for (int i = 0; i < pre; ++i)
        bulk_copy_g2s(ring + (size_t)i * kTwStageBytes, gX + (size_t)i * (kMaxRows * 128), 16384, full + i);
      for (int i = pre; i < n_it; ++i) {
        const int s = i % n_stage;
        tc_wait(empty + s, ((i / n_stage) - 1) & 1, failed, a.err);
        mbar_expect_tx(full + s, kTwStageBytes);
        bulk_copy_g2s(ring + (size_t)s * kTwStageBytes + 16384, gW + (size_t)i * kTcABytes, 16384, full + s);
        bulk_copy_g2s(ring + (size_t)s * kTwStageBytes, gX + (size_t)i * (kMaxRows * 128), 16384, full + s);
      }
      trace_mark(a.trace, a.trace_slot, 3);   // last copy issued
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = tc_instr_desc(128, 128);
      for (int i = 0; i < n_it; ++i) {
        const int s = i % n_stage;
        tc_wait(full + s, (i / n_stage) & 1, failed, a.err);
        const int g = i >> 1;
        if (GROUPED && (i & 1) == 0 && g >= 2) tc_wait(grp_free + (g & 1), ((g >> 1) - 1) & 1, failed, a.err);
        tc_fence_after_sync();
        const unsigned char *sx = ring + (size_t)s * kTwStageBytes;
        const uint64_t da = tc_smem_desc(sx), db = tc_smem_desc(sx + 16384);
        const uint32_t dst = GROUPED ? tmem_d + (uint32_t)(g & 1) * 128u : tmem_d;
#pragma unroll
        for (int j = 0; j < kTcKChunk / 16; ++j) {
          const bool fresh = GROUPED ? ((i & 1) == 0 && j == 0) : (i == 0 && j == 0);
          tc_mma(dst, da + 2 * j, db + 2 * j, idesc, fresh ? 0u : 1u);
        }
        tc_commit(empty + s);
        if (GROUPED && ((i & 1) == 1 || i == n_it - 1)) tc_commit(grp_done + (g & 1));
      }
      if (!GROUPED) tc_commit(acc_done);
    }
    __syncwarp();
  } else {
    // ---- epilogue: warp w may read accumulator lanes 32*(w%4)..+31 = batch rows; warps w and w+4 share a lane
    //      quarter and take 64 of the 128 columns (output features) each ----
    const int lw = warp & 3;
    const int b = lw * 32 + lane;
    const int cb = ((warp - 2) >> 2) * 64;
    const uint32_t t_row = tmem_d + ((uint32_t)(lw * 32) << 16) + (uint32_t)cb;
    float v[64];
    if (GROUPED) {
#pragma unroll
      for (int c = 0; c < 64; ++c) v[c] = 0.f;
      const int n_groups = (n_it + 1) >> 1;
      const int KG = a.K / 128;
      for (int g = 0; g < n_groups; ++g) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          // scales of this group for 32 features (tiled scales [n/8][K/128][8]: 8 features are 16 bytes); same
          // addresses in every lane, fetched ahead of the wait
          uint4 sc[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int n = nt * 128 + cb + hh * 32 + q * 8;
            sc[q] = n < a.N ? __ldg(reinterpret_cast<const uint4 *>(a.scales + ((size_t)(n >> 3) * KG + (kc0 >> 1) + g) * 8))
                            : make_uint4(0, 0, 0, 0);
          }
          if (hh == 0) {
            tc_wait(grp_done + (g & 1), (g >> 1) & 1, failed, a.err);
            tc_fence_after_sync();
            __syncwarp();
          }
          float t[32];
          tmem_ld32(t_row + (uint32_t)(g & 1) * 128u + (uint32_t)(hh * 32), t);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t wds[4] = {sc[q].x, sc[q].y, sc[q].z, sc[q].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float s0 = __uint_as_float(wds[e] << 16), s1 = __uint_as_float(wds[e] & 0xffff0000u);
              v[hh * 32 + q * 8 + 2 * e] = fmaf(s0, t[q * 8 + 2 * e], v[hh * 32 + q * 8 + 2 * e]);
              v[hh * 32 + q * 8 + 2 * e + 1] = fmaf(s1, t[q * 8 + 2 * e + 1], v[hh * 32 + q * 8 + 2 * e + 1]);
            }
          }
        }
        tc_fence_before_sync();
        mbar_arrive(grp_free + (g & 1));
      }
    } else {
#pragma unroll
      for (int c = 0; c < 64; ++c) v[c] = 0.f;
      tc_wait(acc_done, 0, failed, a.err);
      trace_mark(a.trace, a.trace_slot, 4, 64);   // accumulator complete
      tc_fence_after_sync();
      __syncwarp();
      if (n_it > 0) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          float t[32];
          tmem_ld32(t_row + (uint32_t)(hh * 32), t);
#pragma unroll
          for (int c = 0; c < 32; ++c) v[hh * 32 + c] += t[c];
        }
      }
      trace_mark(a.trace, a.trace_slot, 5, 64);   // accumulator in registers
    }
    {
      // ---- out of the registers: a thread owns a batch row, but rows are kilobytes apart in every destination, so
      //      each warp parks its 32 rows x 64 raw sums in its own patch of the (now idle) ring and a short rolled
      //      loop writes them out with the lanes along the row, applying scale, bias and GELU on the way.  The loop
      //      is kept small on purpose: this code runs once per CTA, from a cold instruction cache. ----
      const int n0 = nt * 128 + cb;                 // this warp's 64 features
      const int nv = min(64, a.N - n0);
      const int rows = min(32, Bt - lw * 32);       // real rows of this warp
      unsigned char *patch = ring + (size_t)(warp - 2) * (32 * 272);
      {
        float4 *mine = reinterpret_cast<float4 *>(patch + lane * 272);   // 256 bytes per row, pitch 272: conflict-free
#pragma unroll
        for (int q = 0; q < 16; ++q) mine[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
      }
      __syncwarp();
      const bool as_bf16 = a.mode == EPI_GELU || (a.mode == EPI_QKV && n0 >= a.d);
      const bool partial = a.mode == EPI_RESID && a.ksplit > 1;
      const bool use_bias = a.bias && !partial;
      if (*failed || nv <= 0) {
        // nothing is stored after an expired wait, or for features beyond N
      } else if (as_bf16) {
        // four rows per instruction: lane = (row in the group of four, 16-byte unit = 8 features of the row)
        const int r4 = lane >> 3, u = lane & 7;
        float sc8[8], bi8[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) { sc8[e] = s_rsc[cb + 8 * u + e]; bi8[e] = use_bias ? s_bias[cb + 8 * u + e] : 0.f; }
        const int which = n0 >= 2 * a.d;
        const int col = n0 - (which ? 2 * a.d : a.d);
        const size_t kv_off = a.kv_stage ? (size_t)which * a.d + col : ((size_t)which * a.H + (col >> 6)) * kPageElems;
        unsigned char *blk = reinterpret_cast<unsigned char *>(a.out_img) + ((size_t)blockIdx.z * (a.N >> 6) + (n0 >> 6)) * (kMaxRows * 128);
        // one loop per destination kind, so that each is straight-line code (this runs once per CTA, from a cold
        // instruction cache: a loop that chose per element between the two GELU forms took four times as long)
        if (a.mode == EPI_GELU && a.gelu_tanh)
          tw_rows_bf16<0>(patch, rows, r4, u, lw, sc8, bi8, blk, kv_base, kv_off);
        else if (a.mode == EPI_GELU)
          tw_rows_bf16<1>(patch, rows, r4, u, lw, sc8, bi8, blk, kv_base, kv_off);
        else
          tw_rows_bf16<2>(patch, rows, r4, u, lw, sc8, bi8, blk, kv_base, kv_off);
      } else {
        // fp32 rows: logits, q, the residual stream, or this k-range's partial sums
        const bool add = a.mode == EPI_RESID && !partial;
        float *dst0 = partial ? a.out_f32 + (((size_t)blockIdx.z * a.ksplit + ks) * kMaxRows + lw * 32) * a.N + n0
                              : a.out_f32 + (size_t)(row0 + lw * 32) * a.out_stride + n0;
        const size_t pitch = partial ? (size_t)a.N : (size_t)a.out_stride;
        if (!add && nv == 64 && (reinterpret_cast<uintptr_t>(dst0) & 15) == 0 && (pitch & 3) == 0) {
          // two rows per instruction, 16 bytes per lane
          const int r2 = lane >> 4, u16 = lane & 15;
          float sc4[4], bi4[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) { sc4[e] = s_rsc[cb + 4 * u16 + e]; bi4[e] = use_bias ? s_bias[cb + 4 * u16 + e] : 0.f; }
#pragma unroll 4
          for (int r = r2; r < rows; r += 2) {
            float4 x = *reinterpret_cast<const float4 *>(patch + r * 272 + u16 * 16);
            x.x = fmaf(x.x, sc4[0], bi4[0]); x.y = fmaf(x.y, sc4[1], bi4[1]); x.z = fmaf(x.z, sc4[2], bi4[2]); x.w = fmaf(x.w, sc4[3], bi4[3]);
            *reinterpret_cast<float4 *>(dst0 + (size_t)r * pitch + 4 * u16) = x;
          }
        } else {
          // any alignment, ragged last tile, or adding into the residual stream: one row per step, two features per lane
          float sc2[2], bi2[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) { sc2[e] = s_rsc[cb + lane + 32 * e]; bi2[e] = use_bias ? s_bias[cb + lane + 32 * e] : 0.f; }
#pragma unroll 2
          for (int r = 0; r < rows; ++r) {
            const float *src = reinterpret_cast<const float *>(patch + r * 272);
            float *dst = dst0 + r * pitch;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int c = lane + 32 * e;
              if (c < nv) {
                const float x = fmaf(src[c], sc2[e], bi2[e]);
                dst[c] = add ? dst[c] + x : x;
              }
            }
          }
        }
      }
    }
    trace_mark(a.trace, a.trace_slot, 6, 64);
  }
  tc_fence_before_sync();
  __syncthreads();
  trace_mark(a.trace, a.trace_slot, 2, 64);
  if (warp == 0) tmem_dealloc(tmem_d, kCols);
}

inline size_t gemm_tcw_smem_bytes(int stages) { return (size_t)stages * kTwStageBytes + 1024 + 2304; }

// k-ranges of a residual linear in the wide kernel: at least 4 k-chunks per CTA, at most what LayerNorm folds
inline int tcw_ksplit_resid(int K) { return std::max(1, std::min(kTwMaxPartials, (K / 64) / 8)); }

// n_sm: SMs of the device; a grid that fits at one CTA per SM gets the deep ring
inline cudaError_t launch_gemm_tcw(const GemmTcArgs &a0, int n_sm, cudaStream_t st, bool pdl) {
  static PerDeviceOnce attr_once;
  if (attr_once.first()) {
    cudaFuncSetAttribute(gemm_tcw_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_tcw_smem_bytes(kTwMaxStages));
    cudaFuncSetAttribute(gemm_tcw_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_tcw_smem_bytes(kTwMaxStages));
  }
  GemmTcArgs a = a0;
  dim3 grid((a.N + 127) / 128, a.ksplit, (a.B + kMaxRows - 1) / kMaxRows);
  a.stages = (int)(grid.x * grid.y * grid.z) <= n_sm ? kTwMaxStages : 3;
  if (a.wfmt == WF_INT4)
    return launch_kernel(gemm_tcw_kernel<true>, grid, dim3(kTwThreads), gemm_tcw_smem_bytes(a.stages), st, pdl, a);
  return launch_kernel(gemm_tcw_kernel<false>, grid, dim3(kTwThreads), gemm_tcw_smem_bytes(a.stages), st, pdl, a);
}

// out[b,n] = bias[n] + partial[0][b,n] + partial[1][b,n] + ...  (stand-alone entry point)
__global__ void fold_partials_kernel(const float *__restrict__ part, int n_part, int B, int N,
                                     const uint16_t *__restrict__ bias, float *__restrict__ out) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)B * N) return;
  const int b = i / N, n = i % N;
  float v = bias ? bf16_bits_to_float(bias[n]) : 0.f;
  for (int p = 0; p < n_part; ++p) v += part[((size_t)p * kMaxRows + b) * N + n];
  out[i] = v;
}

inline size_t gemm_tc_smem_bytes() { return (size_t)kTcStages * (kTcABytes + kTcBBytes) + 1024 + 512; }

inline cudaError_t launch_gemm_tc(const GemmTcArgs &a, cudaStream_t st, bool pdl) {
  static PerDeviceOnce attr_once;   // per device: opt-in to more than 48 KB of dynamic shared memory
  if (attr_once.first()) {
    cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_tc_smem_bytes());
    cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_tc_smem_bytes());
  }
  dim3 grid((a.N + kTcTileM - 1) / kTcTileM, (a.B + kTcChunkN - 1) / kTcChunkN, a.ksplit);
  if (a.wfmt == WF_INT4)
    return launch_kernel(gemm_tc_kernel<true>, grid, dim3(kTcThreads), gemm_tc_smem_bytes(), st, pdl, a);
  return launch_kernel(gemm_tc_kernel<false>, grid, dim3(kTcThreads), gemm_tc_smem_bytes(), st, pdl, a);
}

}  // namespace ttsgpt
