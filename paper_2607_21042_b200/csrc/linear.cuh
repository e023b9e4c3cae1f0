// Weight-only dequantizing linear (Table I caption: W8A16 / W4A16 applied to the GPT; bf16 is the
// unquantized case): out[b,n] = sum_k W[n,k] act[b,k] (+ bias, + epilogue), bf16 activations,
// fp32 accumulation.
//
// Streaming layout.  At engine creation every [N,K] matrix is re-laid into 1 KB tiles of 16 output
// rows x KT columns (KT = 32 bf16 / 64 int8 / 128 int4, i.e. always 1 KB), stored tile after tile
// as [row-tile nt][k-tile kb].  Inside a tile the bytes sit in the order the warp-level MMA wants
// its A operand: first 512 B = for lane 0..31 the 16 bytes of row (lane/4) covering columns
// KT/4*(lane%4) .. +KT/4-1 of the tile, second 512 B = the same for row (lane/4)+8.  A warp then
// fetches a tile with two fully coalesced 128-bit loads per lane and feeds registers straight to
// the tensor pipe; int8 / int4 codes are widened to bf16 integers in registers (exact) and the
// bf16 scale multiplies the fp32 partial sums (per row for int8, per row and 128-column group for
// int4).  A CTA owns one 16-row tile and splits K over its warps; partial sums meet in shared
// memory in a fixed order, so results do not depend on timing.
#pragma once
#include "common.cuh"

namespace ttsgpt {

enum { WF_BF16 = 0, WF_INT8 = 1, WF_INT4 = 2 };
enum { EPI_F32 = 0, EPI_QKV = 1, EPI_RESID = 2, EPI_GELU = 3 };

constexpr int kLinearThreads = 320;  // 10 warps: divides the k-tile counts of K=1280 and K=5120

__host__ __device__ inline int k_per_tile(int wf) { return wf == WF_BF16 ? 32 : (wf == WF_INT8 ? 64 : 128); }
__host__ __device__ inline int row_tiles(int N) { return (N + 15) / 16; }
// bytes of the tiled weights / of the tiled scales
inline size_t packed_weight_bytes(int wf, int N, int K) { return (size_t)row_tiles(N) * (K / k_per_tile(wf)) * 1024; }
inline size_t packed_scale_bytes(int wf, int N, int K) {
  if (wf == WF_INT8) return (size_t)row_tiles(N) * 16 * 2;
  if (wf == WF_INT4) return (size_t)row_tiles(N) * (K / 128) * 16 * 2;
  return 0;
}

// ------------------------------------------------------------------------------------------
// canonical -> streaming re-layout (run once at creation)
// ------------------------------------------------------------------------------------------
// One thread per 16-byte unit of the destination.
__global__ void pack_bf16_kernel(const uint16_t *__restrict__ w, int N, int K, uint4 *__restrict__ dst) {
  const int KB = K / 32;
  size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t total = (size_t)row_tiles(N) * KB * 64;
  if (unit >= total) return;
  int lane = unit & 31, half = (unit >> 5) & 1;
  size_t tile = unit >> 6;
  int kb = tile % KB, nt = tile / KB;
  int row = nt * 16 + (lane >> 2) + 8 * half, k = kb * 32 + 8 * (lane & 3);
  uint4 v = make_uint4(0, 0, 0, 0);
  if (row < N) v = *reinterpret_cast<const uint4 *>(w + (size_t)row * K + k);
  dst[unit] = v;
}

// int8 codes are stored biased (u = q + 128) so that one byte-permute drops them into the mantissa
// of a float magic number.
__global__ void pack_int8_kernel(const int8_t *__restrict__ w, int N, int K, uint4 *__restrict__ dst) {
  const int KB = K / 64;
  size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t total = (size_t)row_tiles(N) * KB * 64;
  if (unit >= total) return;
  int lane = unit & 31, half = (unit >> 5) & 1;
  size_t tile = unit >> 6;
  int kb = tile % KB, nt = tile / KB;
  int row = nt * 16 + (lane >> 2) + 8 * half, k = kb * 64 + 16 * (lane & 3);
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
    uint32_t nib = (c >> (4 * j)) & 15u;
    int pos = (j >> 1) + 4 * (j & 1);
    r |= nib << (4 * pos);
  }
  return r;
}
__global__ void pack_int4_kernel(const uint32_t *__restrict__ w, int N, int K, uint4 *__restrict__ dst) {
  const int KB = K / 128;
  size_t unit = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t total = (size_t)row_tiles(N) * KB * 64;
  if (unit >= total) return;
  int lane = unit & 31, half = (unit >> 5) & 1;
  size_t tile = unit >> 6;
  int kb = tile % KB, nt = tile / KB;
  int row = nt * 16 + (lane >> 2) + 8 * half, k = kb * 128 + 32 * (lane & 3);
  uint4 v = make_uint4(0x88888888u, 0x88888888u, 0x88888888u, 0x88888888u);
  if (row < N) {
    uint4 c = *reinterpret_cast<const uint4 *>(w + (size_t)row * (K / 8) + k / 8);
    v = make_uint4(permute_nibbles(c.x), permute_nibbles(c.y), permute_nibbles(c.z), permute_nibbles(c.w));
  }
  dst[unit] = v;
}
// scales: int8 [N] -> [nt][16]; int4 [N][K/128] -> [nt][kb][16]; padding rows get 0
__global__ void pack_scales_kernel(const uint16_t *__restrict__ s, int N, int G, uint16_t *__restrict__ dst) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t total = (size_t)row_tiles(N) * G * 16;
  if (i >= total) return;
  int r = i & 15;
  size_t t = i >> 4;
  int g = t % G, nt = t / G;
  int row = nt * 16 + r;
  dst[i] = row < N ? s[(size_t)row * G + g] : (uint16_t)0;
}

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------
struct LinearArgs {
  const void *w;          // tiled weights
  const uint16_t *scales; // tiled scales (int8 / int4) or null
  const uint16_t *bias;   // bf16 [N] or null
  const uint16_t *act;    // bf16 [B][K]
  int N, K, B, mode;
  float *out_f32;         // EPI_F32: out[b*out_stride+n] = v ; EPI_RESID: out[b*out_stride+n] += v ; EPI_QKV: q
  int out_stride;
  uint16_t *out_bf16;     // EPI_GELU: h[b*N+n] = bf16(gelu(v))
  int gelu_tanh;
  // EPI_QKV: rows [0,d) -> q (fp32), [d,2d) -> K pages, [2d,3d) -> V pages
  uint16_t *kv_layer;
  const int *page_table, *row_stream, *row_pos;
  int pps, d, H;
};

// exact int8 (biased byte) -> float via the 2^23 magic number
__device__ __forceinline__ float biased_byte_to_float(uint32_t word, int i) {
  uint32_t m = __byte_perm(word, 0x4B000000u, 0x7540u | (uint32_t)i);
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

template <int WF, int NT>
__global__ void __launch_bounds__(kLinearThreads) linear_kernel(const LinearArgs a) {
  constexpr int KT = WF == WF_BF16 ? 32 : (WF == WF_INT8 ? 64 : 128);
  constexpr int AW = KT / 32;  // uint4 activation loads per lane, tile and batch row
  extern __shared__ float red[];  // [nwarps][16][NT*8]
  const int nt = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nwarps = blockDim.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int KB = a.K / KT;
  const uint4 *wt = reinterpret_cast<const uint4 *>(a.w) + (size_t)nt * KB * 64;
  const uint16_t *sc = a.scales;

  for (int b0 = 0; b0 < a.B; b0 += NT * 8) {
    float acc[NT][4];
#pragma unroll
    for (int j = 0; j < NT; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;

#pragma unroll 4
    for (int kb = warp; kb < KB; kb += nwarps) {
      const uint4 wa = ld_stream_u4(wt + (size_t)kb * 64 + lane);
      const uint4 wb = ld_stream_u4(wt + (size_t)kb * 64 + 32 + lane);
      uint4 xa[NT][AW];
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const int b = b0 + 8 * j + g;
#pragma unroll
        for (int q = 0; q < AW; ++q) {
          xa[j][q] = make_uint4(0, 0, 0, 0);
          if (b < a.B)
            xa[j][q] = *reinterpret_cast<const uint4 *>(a.act + (size_t)b * a.K + (size_t)kb * KT + t * (KT / 4) + 8 * q);
        }
      }
      if (WF == WF_BF16) {
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          mma_bf16_16816(acc[j], wa.x, wb.x, wa.y, wb.y, xa[j][0].x, xa[j][0].y);
          mma_bf16_16816(acc[j], wa.z, wb.z, wa.w, wb.w, xa[j][0].z, xa[j][0].w);
        }
      } else if (WF == WF_INT8) {
        const uint32_t wwa[4] = {wa.x, wa.y, wa.z, wa.w}, wwb[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const uint32_t a0 = pack_bf16x2(biased_byte_to_float(wwa[s], 0), biased_byte_to_float(wwa[s], 1));
          const uint32_t a2 = pack_bf16x2(biased_byte_to_float(wwa[s], 2), biased_byte_to_float(wwa[s], 3));
          const uint32_t a1 = pack_bf16x2(biased_byte_to_float(wwb[s], 0), biased_byte_to_float(wwb[s], 1));
          const uint32_t a3 = pack_bf16x2(biased_byte_to_float(wwb[s], 2), biased_byte_to_float(wwb[s], 3));
#pragma unroll
          for (int j = 0; j < NT; ++j) {
            const uint4 x = xa[j][s >> 1];
            const uint32_t b0r = (s & 1) ? x.z : x.x, b1r = (s & 1) ? x.w : x.y;
            mma_bf16_16816(acc[j], a0, a1, a2, a3, b0r, b1r);
          }
        }
      } else {
        float tmp[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) tmp[j][0] = tmp[j][1] = tmp[j][2] = tmp[j][3] = 0.f;
        const uint32_t wwa[4] = {wa.x, wa.y, wa.z, wa.w}, wwb[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
        for (int wd = 0; wd < 4; ++wd) {
#pragma unroll
          for (int hs = 0; hs < 2; ++hs) {  // the word's two MMA steps
            const uint32_t ua = wwa[wd] >> (8 * hs), ub = wwb[wd] >> (8 * hs);
            const uint32_t a0 = nib_pair_to_bf16x2(ua & 0x000F000Fu);
            const uint32_t a2 = nib_pair_to_bf16x2((ua >> 4) & 0x000F000Fu);
            const uint32_t a1 = nib_pair_to_bf16x2(ub & 0x000F000Fu);
            const uint32_t a3 = nib_pair_to_bf16x2((ub >> 4) & 0x000F000Fu);
#pragma unroll
            for (int j = 0; j < NT; ++j) {
              const uint4 x = xa[j][wd];
              const uint32_t b0r = hs ? x.z : x.x, b1r = hs ? x.w : x.y;
              mma_bf16_16816(tmp[j], a0, a1, a2, a3, b0r, b1r);
            }
          }
        }
        const float s_lo = bf16_bits_to_float(sc[((size_t)nt * KB + kb) * 16 + g]);
        const float s_hi = bf16_bits_to_float(sc[((size_t)nt * KB + kb) * 16 + g + 8]);
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          acc[j][0] = fmaf(s_lo, tmp[j][0], acc[j][0]);
          acc[j][1] = fmaf(s_lo, tmp[j][1], acc[j][1]);
          acc[j][2] = fmaf(s_hi, tmp[j][2], acc[j][2]);
          acc[j][3] = fmaf(s_hi, tmp[j][3], acc[j][3]);
        }
      }
    }

    // partial sums of the warps meet in shared memory and are added in warp order
    constexpr int C = NT * 8;
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      float *r0 = red + ((size_t)warp * 16 + g) * C + 8 * j + 2 * t;
      float *r1 = red + ((size_t)warp * 16 + g + 8) * C + 8 * j + 2 * t;
      r0[0] = acc[j][0]; r0[1] = acc[j][1];
      r1[0] = acc[j][2]; r1[1] = acc[j][3];
    }
    __syncthreads();
    if (threadIdx.x < 16 * C) {
      const int r = threadIdx.x / C, c = threadIdx.x % C;
      const int n = nt * 16 + r, b = b0 + c;
      if (n < a.N && b < a.B) {
        float v = 0.f;
        for (int w = 0; w < nwarps; ++w) v += red[((size_t)w * 16 + r) * C + c];
        if (WF == WF_INT8) v *= bf16_bits_to_float(sc[(size_t)nt * 16 + r]);
        if (a.bias) v += bf16_bits_to_float(a.bias[n]);
        if (a.mode == EPI_F32) {
          a.out_f32[(size_t)b * a.out_stride + n] = v;
        } else if (a.mode == EPI_RESID) {
          a.out_f32[(size_t)b * a.out_stride + n] += v;
        } else if (a.mode == EPI_GELU) {
          v = a.gelu_tanh ? gelu_tanh_f(v) : gelu_erf_f(v);
          a.out_bf16[(size_t)b * a.N + n] = float_to_bf16_bits(v);
        } else {  // EPI_QKV
          if (n < a.d) {
            a.out_f32[(size_t)b * a.out_stride + n] = v;
          } else {
            const int which = n >= 2 * a.d;  // 0 = K, 1 = V
            const int col = n - (which ? 2 * a.d : a.d);
            const int head = col >> 6, e = col & 63;
            const int pos = a.row_pos[b];
            const int page = a.page_table[(size_t)a.row_stream[b] * a.pps + (pos >> 6)];
            a.kv_layer[(((size_t)page * 2 + which) * a.H + head) * kPageElems + (size_t)(pos & 63) * kHeadDim + e] =
                float_to_bf16_bits(v);
          }
        }
      }
    }
    __syncthreads();
  }
}

inline cudaError_t launch_linear(int wf, const LinearArgs &a, cudaStream_t st) {
  const int grid = row_tiles(a.N);
  const int nt = a.B > 8 ? 2 : 1;
  const size_t smem = (size_t)(kLinearThreads / 32) * 16 * nt * 8 * sizeof(float);
#define TTS_LAUNCH(WF, NT) linear_kernel<WF, NT><<<grid, kLinearThreads, smem, st>>>(a)
  if (wf == WF_BF16) { if (nt == 1) TTS_LAUNCH(WF_BF16, 1); else TTS_LAUNCH(WF_BF16, 2); }
  else if (wf == WF_INT8) { if (nt == 1) TTS_LAUNCH(WF_INT8, 1); else TTS_LAUNCH(WF_INT8, 2); }
  else { if (nt == 1) TTS_LAUNCH(WF_INT4, 1); else TTS_LAUNCH(WF_INT4, 2); }
#undef TTS_LAUNCH
  return cudaGetLastError();
}

inline cudaError_t launch_pack(int wf, int N, int K, const void *w, const void *s, void *dst_w, void *dst_s,
                               cudaStream_t st) {
  const size_t units = (size_t)row_tiles(N) * (K / k_per_tile(wf)) * 64;
  const int blocks = (int)((units + 255) / 256);
  if (wf == WF_BF16) pack_bf16_kernel<<<blocks, 256, 0, st>>>((const uint16_t *)w, N, K, (uint4 *)dst_w);
  else if (wf == WF_INT8) pack_int8_kernel<<<blocks, 256, 0, st>>>((const int8_t *)w, N, K, (uint4 *)dst_w);
  else pack_int4_kernel<<<blocks, 256, 0, st>>>((const uint32_t *)w, N, K, (uint4 *)dst_w);
  if (wf != WF_BF16) {
    const int G = wf == WF_INT8 ? 1 : K / 128;
    const size_t n = (size_t)row_tiles(N) * G * 16;
    pack_scales_kernel<<<(int)((n + 255) / 256), 256, 0, st>>>((const uint16_t *)s, N, G, (uint16_t *)dst_s);
  }
  return cudaGetLastError();
}

}  // namespace ttsgpt
