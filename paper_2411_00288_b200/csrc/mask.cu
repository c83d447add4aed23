// Mask selection (Eq. 1), mask application + 2:4 packing (Eq. 6, Fig. 1) and its inverse.
// All three are one-off, memory-bound, integer-only kernels: values are compared and moved,
// never computed with.
#include <cuda_runtime.h>

#include "layout.cuh"
#include "ssconv.h"

namespace ssconv {

// ---------------------------------------------------------------------------------------
// select_mask
// ---------------------------------------------------------------------------------------

// Eq. 1 without the one-hot: first maximum of the six scores of each group.
__global__ void select_logits_kernel(const float2* __restrict__ scores, int64_t G, uint8_t* __restrict__ pattern) {
  int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (g >= G) return;
  float2 a = scores[3 * g], b = scores[3 * g + 1], c = scores[3 * g + 2];
  float v[6] = {a.x, a.y, b.x, b.y, c.x, c.y};
  int best = 0;
  float bv = v[0];
#pragma unroll
  for (int i = 1; i < 6; ++i) {
    if (v[i] > bv) {
      bv = v[i];
      best = i;
    }
  }
  pattern[g] = (uint8_t)best;
}

// Magnitude heuristic: keep the two largest |w| of the group.  Magnitudes are compared as
// the 15-bit integers below the sign bit (monotone in |w|, +0 == -0); a position beats
// another when it is larger, or equal and earlier, so exactly two positions are beaten by
// fewer than two others.
__device__ __forceinline__ uint32_t magnitude_pattern4(const uint32_t (&a)[4]) {
  int first = -1, second = -1;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int beaten = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (j == i) continue;
      beaten += (a[j] > a[i]) || (a[j] == a[i] && j < i);
    }
    if (beaten < 2) {
      if (first < 0) first = i; else second = i;
    }
  }
  // lexicographic index of the pair (first < second):
  // {0,1}->0 {0,2}->1 {0,3}->2 {1,2}->3 {1,3}->4 {2,3}->5
  return (uint32_t)(first == 0 ? second - 1 : (first == 1 ? second + 1 : 5));
}
__device__ __forceinline__ uint32_t magnitude_pattern(uint32_t lo, uint32_t hi) {
  const uint32_t a[4] = {lo & 0x7FFFu, (lo >> 16) & 0x7FFFu, hi & 0x7FFFu, (hi >> 16) & 0x7FFFu};
  return magnitude_pattern4(a);
}

__global__ void select_magnitude_kernel(const uint2* __restrict__ w, int64_t G, uint8_t* __restrict__ pattern) {
  int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (g >= G) return;
  uint2 v = w[g];
  pattern[g] = (uint8_t)magnitude_pattern(v.x, v.y);
}

// The same for e4m3 weights: a group is four bytes, a magnitude the 7 bits below the sign bit.
__global__ void select_magnitude_e4m3_kernel(const uint32_t* __restrict__ w, int64_t G, uint8_t* __restrict__ pattern) {
  int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (g >= G) return;
  const uint32_t v = w[g];
  const uint32_t a[4] = {v & 0x7Fu, (v >> 8) & 0x7Fu, (v >> 16) & 0x7Fu, (v >> 24) & 0x7Fu};
  pattern[g] = (uint8_t)magnitude_pattern4(a);
}

// bf16 -> e4m3: y = nearest e4m3 value of x * scale (the product rounded to fp32 first), ties to even,
// magnitudes beyond 448 saturate.  One thread per pair of elements.
__global__ void quantize_e4m3_kernel(const uint32_t* __restrict__ x, uint16_t* __restrict__ y, int64_t pairs, float scale) {
  int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= pairs) return;
  const uint32_t v = x[i];
  const float lo = __uint_as_float(v << 16) * scale, hi = __uint_as_float(v & 0xFFFF0000u) * scale;
  uint16_t out;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(out) : "f"(hi), "f"(lo));
  y[i] = out;
}

// ---------------------------------------------------------------------------------------
// General N:M bookkeeping (Sec. 3.1): blocks of M consecutive weights of which N are kept, one of
// n = C(M, N) patterns per block, numbered lexicographically in the kept positions.  The hardware
// operation exists for 2:4 only; other N:M masks are selected and applied here and the masked weights
// run through the dense kernel (Eq. 6 with a dense product).  M <= 8, so a pattern is a byte and its
// kept positions a bitmask; the table of all patterns (at most C(8,4) = 70) travels as a kernel argument.
// ---------------------------------------------------------------------------------------
struct NmTable {
  int N, M, n;
  uint8_t kept_mask[70];  // bit i set: position i of the block is kept
};

__global__ void nm_select_logits_kernel(const float* __restrict__ scores, int64_t G, int n, uint8_t* __restrict__ pattern) {
  int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (g >= G) return;
  const float* s = scores + g * n;
  int best = 0;
  float bv = s[0];
  for (int i = 1; i < n; ++i) {
    const float v = s[i];
    if (v > bv) {
      bv = v;
      best = i;
    }
  }
  pattern[g] = (uint8_t)best;
}

// Keep the N largest magnitudes of the block (15-bit integers below the bf16 sign bit); a position
// beats another when it is larger, or equal and earlier; the kept ones are beaten by fewer than N.
__global__ void nm_select_magnitude_kernel(const uint16_t* __restrict__ w, int64_t G, NmTable t,
                                           uint8_t* __restrict__ pattern) {
  int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (g >= G) return;
  uint32_t a[8];
  for (int i = 0; i < t.M; ++i) a[i] = w[g * t.M + i] & 0x7FFFu;
  uint32_t mask = 0;
  for (int i = 0; i < t.M; ++i) {
    int beaten = 0;
    for (int j = 0; j < t.M; ++j)
      if (j != i) beaten += (a[j] > a[i]) || (a[j] == a[i] && j < i);
    if (beaten < t.N) mask |= 1u << i;
  }
  int p = 0;
  for (int i = 0; i < t.n; ++i)
    if (t.kept_mask[i] == mask) p = i;
  pattern[g] = (uint8_t)p;
}

// Eq. 6 for an N:M mask: dropped positions become +0, kept values are copied bit for bit.
__global__ void nm_apply_mask_kernel(const uint16_t* __restrict__ w, const uint8_t* __restrict__ pattern, int64_t G,
                                     NmTable t, uint16_t* __restrict__ w_masked) {
  int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (g >= G) return;
  const uint32_t p = pattern[g];
  const uint32_t mask = p < (uint32_t)t.n ? t.kept_mask[p] : t.kept_mask[0];  // (an index out of range: pattern 0)
  for (int i = 0; i < t.M; ++i) w_masked[g * t.M + i] = ((mask >> i) & 1u) ? w[g * t.M + i] : (uint16_t)0;
}

// ---------------------------------------------------------------------------------------
// 8-bit (e4m3) weights: compress / decompress
// ---------------------------------------------------------------------------------------
// Geometry with k-blocks of 128 channels (make_geometry(d, 128)).  Value blob: bytes [Mp][64 * kblocks_pad]:
// byte 64 b + 2 q + s holds kept value s (0 = lower position) of the q-th group of four channels of
// k-block b.  Metadata: per (128-row tile, pair of k-blocks) two images of 2048 bytes, one per k-block,
// each what one tcgen05.cp 128x128b moves into 4 TMEM columns: lane = row, its four words hold the 32
// 4-bit codes of the row's groups in order (nibble n of word w = group 8 w + n); the sparse MMA over the
// first 64 channels of a k-block reads the first two columns, the one over the second 64 the other two.
// (Found by probing the instruction with an identity activation matrix and single flipped codes.)
__global__ void compress_values_e4m3_kernel(ssconv_desc_t d, Geometry geo, const uint32_t* __restrict__ w,
                                            const uint8_t* __restrict__ pattern, uint16_t* __restrict__ w_comp) {
  int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  int64_t total = (int64_t)geo.Mp * geo.kblocks_pad * 32;
  if (t >= total) return;
  int q = (int)(t % 32);
  int b = (int)((t / 32) % geo.kblocks_pad);
  int co = (int)(t / (32 * (int64_t)geo.kblocks_pad));
  uint32_t out = 0;
  if (co < d.C_out && b < geo.kblocks) {
    int tap = b % geo.taps;
    int c = (b / geo.taps) * 128 + 4 * q;
    if (c < d.C_in) {
      int64_t g = ((int64_t)co * geo.taps + tap) * (d.C_in / 4) + c / 4;
      uint32_t v = w[g];
      uint32_t code = pattern_code(pattern[g]);
      out = ((v >> (8 * (code & 3u))) & 0xFFu) | (((v >> (8 * ((code >> 2) & 3u))) & 0xFFu) << 8);
    }
  }
  w_comp[(int64_t)co * (32 * geo.kblocks_pad) + 32 * b + q] = (uint16_t)out;
}

__global__ void compress_meta_e4m3_kernel(ssconv_desc_t d, Geometry geo, const uint8_t* __restrict__ pattern,
                                          uint32_t* __restrict__ meta) {
  // one thread per metadata word: (tile, stage, image i, lane L, word j)
  int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  int64_t total = (int64_t)geo.m_tiles * geo.stages * 2 * 128 * 4;
  if (t >= total) return;
  int j = (int)(t % 4);
  int L = (int)((t / 4) % 128);
  int i = (int)((t / 512) % 2);
  int s = (int)((t / 1024) % geo.stages);
  int mt = (int)(t / (1024 * (int64_t)geo.stages));
  int b = 2 * s + i;
  int tap = b % geo.taps;
  int co = mt * kTileM + L;
  uint32_t word = 0;
#pragma unroll
  for (int n = 0; n < 8; ++n) {
    int c = (b / geo.taps) * 128 + 4 * (8 * j + n);
    uint32_t code = 0x4u;
    if (co < d.C_out && b < geo.kblocks && c < d.C_in) {
      int64_t g = ((int64_t)co * geo.taps + tap) * (d.C_in / 4) + c / 4;
      code = pattern_code(pattern[g]);
    }
    word |= code << (4 * n);
  }
  meta[t] = word;
}

__global__ void decompress_e4m3_kernel(ssconv_desc_t d, Geometry geo, const uint16_t* __restrict__ w_comp,
                                       const uint32_t* __restrict__ meta, uint32_t* __restrict__ w_out,
                                       uint8_t* __restrict__ pattern_out) {
  int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  int groups_per_tap = d.C_in / 4;
  int64_t G = (int64_t)d.C_out * geo.taps * groups_per_tap;
  if (g >= G) return;
  int c = (int)(g % groups_per_tap) * 4;
  int tap = (int)((g / groups_per_tap) % geo.taps);
  int co = (int)(g / ((int64_t)groups_per_tap * geo.taps));
  int b = (c / 128) * geo.taps + tap;
  int q = (c % 128) / 4;
  int mt = co / kTileM, L = co % kTileM;
  uint32_t word = meta[((((int64_t)mt * geo.stages + (b >> 1)) * 2 + (b & 1)) * 128 + L) * 4 + q / 8];
  uint32_t code = (word >> (4 * (q % 8))) & 0xFu;
  uint32_t pair = w_comp[(int64_t)co * (32 * geo.kblocks_pad) + 32 * b + q];
  uint32_t out = ((pair & 0xFFu) << (8 * (code & 3u))) | ((pair >> 8) << (8 * ((code >> 2) & 3u)));
  w_out[g] = out;
  if (pattern_out) pattern_out[g] = (uint8_t)code_pattern(code);
}

// ---------------------------------------------------------------------------------------
// compress: values
// ---------------------------------------------------------------------------------------
// One thread per (row, k-block, group-in-block): writes the two kept values (one 32-bit
// store), +0 for padding.
__global__ void compress_values_kernel(ssconv_desc_t d, Geometry geo, const uint2* __restrict__ w,
                                       const uint8_t* __restrict__ pattern, uint32_t* __restrict__ w_comp) {
  int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  int64_t total = (int64_t)geo.Mp * geo.kblocks_pad * 16;
  if (t >= total) return;
  int q = (int)(t % 16);
  int b = (int)((t / 16) % geo.kblocks_pad);
  int co = (int)(t / (16 * (int64_t)geo.kblocks_pad));
  uint32_t out = 0;
  if (co < d.C_out && b < geo.kblocks) {
    int tap = b % geo.taps;
    int c = (b / geo.taps) * kBlockK + 4 * q;
    if (c < d.C_in) {
      int64_t g = ((int64_t)co * geo.taps + tap) * (d.C_in / 4) + c / 4;
      uint2 v = w[g];
      uint32_t vals[4] = {v.x & 0xFFFFu, v.x >> 16, v.y & 0xFFFFu, v.y >> 16};
      uint32_t code = pattern_code(pattern[g]);
      out = vals[code & 3u] | (vals[(code >> 2) & 3u] << 16);
    }
  }
  // row-major [Mp][KC] bf16; this thread's pair sits at column 32*b + 2*q
  w_comp[((int64_t)co * geo.KC + 32 * b + 2 * q) / 2] = out;
}

// ---------------------------------------------------------------------------------------
// compress: metadata
// ---------------------------------------------------------------------------------------
// One thread per 32-bit metadata word (layout.cuh says what a word holds).
__global__ void compress_meta_kernel(ssconv_desc_t d, Geometry geo, const uint8_t* __restrict__ pattern,
                                     uint32_t* __restrict__ meta) {
  int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  int64_t total = (int64_t)geo.m_tiles * geo.stages * 128 * 4;
  if (t >= total) return;
  int j = (int)(t % 4);
  int L = (int)((t / 4) % 128);
  int s = (int)((t / 512) % geo.stages);
  int mt = (int)(t / (512 * (int64_t)geo.stages));
  int b = 2 * s + (j >> 1);
  int tap = b % geo.taps;
  int cbase = (b / geo.taps) * kBlockK + (j & 1) * 32 + 16 * ((L >> 3) & 1);
  uint32_t word = 0;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    int co = mt * kTileM + (L & 7) + 16 * (L >> 4) + 8 * h;
#pragma unroll
    for (int gi = 0; gi < 4; ++gi) {
      int c = cbase + 4 * gi;
      uint32_t code = 0x4u;
      if (co < d.C_out && b < geo.kblocks && c < d.C_in) {
        int64_t g = ((int64_t)co * geo.taps + tap) * (d.C_in / 4) + c / 4;
        code = pattern_code(pattern[g]);
      }
      word |= code << (16 * h + 4 * gi);
    }
  }
  meta[t] = word;
}

// ---------------------------------------------------------------------------------------
// decompress
// ---------------------------------------------------------------------------------------
// One thread per group: reads its code and its two values back and scatters them.
__global__ void decompress_kernel(ssconv_desc_t d, Geometry geo, const uint32_t* __restrict__ w_comp,
                                  const uint32_t* __restrict__ meta, uint2* __restrict__ w_out,
                                  uint8_t* __restrict__ pattern_out) {
  int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  int groups_per_tap = d.C_in / 4;
  int64_t G = (int64_t)d.C_out * geo.taps * groups_per_tap;
  if (g >= G) return;
  int c = (int)(g % groups_per_tap) * 4;
  int tap = (int)((g / groups_per_tap) % geo.taps);
  int co = (int)(g / ((int64_t)groups_per_tap * geo.taps));
  int b = (c / kBlockK) * geo.taps + tap;
  int cl = c % kBlockK;
  // metadata word and nibble of this group
  int mt = co / kTileM, r = co % kTileM;
  int h = (r >> 3) & 1;
  int L = (r & 7) + 8 * ((cl % 32) / 16) + 16 * (r >> 4);
  int s = b >> 1;
  int j = (b & 1) * 2 + cl / 32;
  int gi = (cl % 16) / 4;
  uint32_t word = meta[(((int64_t)mt * geo.stages + s) * 128 + L) * 4 + j];
  uint32_t code = (word >> (16 * h + 4 * gi)) & 0xFu;
  uint32_t pair = w_comp[((int64_t)co * geo.KC + 32 * b + cl / 2) / 2];
  uint32_t vals[4] = {0, 0, 0, 0};
  vals[code & 3u] = pair & 0xFFFFu;
  vals[(code >> 2) & 3u] = pair >> 16;
  w_out[g] = make_uint2(vals[0] | (vals[1] << 16), vals[2] | (vals[3] << 16));
  if (pattern_out) pattern_out[g] = (uint8_t)code_pattern(code);
}

// ---------------------------------------------------------------------------------------
// host launchers (called from the C ABI)
// ---------------------------------------------------------------------------------------
static inline unsigned blocks_for(int64_t n, int threads) { return (unsigned)((n + threads - 1) / threads); }

cudaError_t launch_select(int mode, const void* scores, int64_t G, uint8_t* pattern, cudaStream_t st) {
  if (G == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
  if (mode == SSCONV_MASK_LOGITS_F32)
    select_logits_kernel<<<blocks_for(G, T), T, 0, st>>>((const float2*)scores, G, pattern);
  else if (mode == SSCONV_MASK_MAGNITUDE_E4M3)
    select_magnitude_e4m3_kernel<<<blocks_for(G, T), T, 0, st>>>((const uint32_t*)scores, G, pattern);
  else
    select_magnitude_kernel<<<blocks_for(G, T), T, 0, st>>>((const uint2*)scores, G, pattern);
  return cudaGetLastError();
}

// All N-subsets of {0..M-1} in lexicographic order of the kept positions, as bitmasks.
static bool make_nm_table(int N, int M, NmTable* t) {
  if (M < 1 || M > 8 || N < 1 || N > M) return false;
  t->N = N;
  t->M = M;
  t->n = 0;
  int idx[8];
  for (int i = 0; i < N; ++i) idx[i] = i;
  while (true) {
    uint32_t mask = 0;
    for (int i = 0; i < N; ++i) mask |= 1u << idx[i];
    t->kept_mask[t->n++] = (uint8_t)mask;
    int i = N - 1;
    while (i >= 0 && idx[i] == M - N + i) --i;
    if (i < 0) break;
    ++idx[i];
    for (int j = i + 1; j < N; ++j) idx[j] = idx[j - 1] + 1;
  }
  return true;
}
int nm_pattern_count(int N, int M) {
  NmTable t;
  return make_nm_table(N, M, &t) ? t.n : 0;
}
cudaError_t launch_nm_select(int mode, const void* scores, int64_t G, int N, int M, uint8_t* pattern, cudaStream_t st) {
  NmTable t;
  if (!make_nm_table(N, M, &t)) return cudaErrorInvalidValue;
  if (G == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
  if (mode == SSCONV_MASK_LOGITS_F32)
    nm_select_logits_kernel<<<blocks_for(G, T), T, 0, st>>>((const float*)scores, G, t.n, pattern);
  else
    nm_select_magnitude_kernel<<<blocks_for(G, T), T, 0, st>>>((const uint16_t*)scores, G, t, pattern);
  return cudaGetLastError();
}
cudaError_t launch_nm_apply(const void* w, const uint8_t* pattern, int64_t G, int N, int M, void* w_masked,
                            cudaStream_t st) {
  NmTable t;
  if (!make_nm_table(N, M, &t)) return cudaErrorInvalidValue;
  if (G == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
  nm_apply_mask_kernel<<<blocks_for(G, T), T, 0, st>>>((const uint16_t*)w, pattern, G, t, (uint16_t*)w_masked);
  return cudaGetLastError();
}

cudaError_t launch_quantize_e4m3(const void* x, void* y, int64_t n, float scale, cudaStream_t st) {
  const int T = 256;
  if (n == 0) return cudaSuccess;
  count_launch();
  quantize_e4m3_kernel<<<blocks_for(n / 2, T), T, 0, st>>>((const uint32_t*)x, (uint16_t*)y, n / 2, scale);
  return cudaGetLastError();
}

cudaError_t launch_compress_e4m3(const ssconv_desc_t& d, const void* w, const uint8_t* pattern, void* w_comp, void* meta,
                                 cudaStream_t st) {
  Geometry geo = make_geometry(d, 128);
  const int T = 256;
  int64_t nv = (int64_t)geo.Mp * geo.kblocks_pad * 32;
  count_launch();
  compress_values_e4m3_kernel<<<blocks_for(nv, T), T, 0, st>>>(d, geo, (const uint32_t*)w, pattern, (uint16_t*)w_comp);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  int64_t nm = (int64_t)geo.m_tiles * geo.stages * 1024;
  count_launch();
  compress_meta_e4m3_kernel<<<blocks_for(nm, T), T, 0, st>>>(d, geo, pattern, (uint32_t*)meta);
  return cudaGetLastError();
}

cudaError_t launch_decompress_e4m3(const ssconv_desc_t& d, const void* w_comp, const void* meta, void* w_out,
                                   uint8_t* pattern_out, cudaStream_t st) {
  Geometry geo = make_geometry(d, 128);
  const int T = 256;
  int64_t G = (int64_t)d.C_out * geo.taps * (d.C_in / 4);
  count_launch();
  decompress_e4m3_kernel<<<blocks_for(G, T), T, 0, st>>>(d, geo, (const uint16_t*)w_comp, (const uint32_t*)meta,
                                                         (uint32_t*)w_out, pattern_out);
  return cudaGetLastError();
}

cudaError_t launch_compress(const ssconv_desc_t& d, const void* w, const uint8_t* pattern, void* w_comp, void* meta,
                            cudaStream_t st) {
  Geometry geo = make_geometry(d);
  const int T = 256;
  int64_t nv = (int64_t)geo.Mp * geo.kblocks_pad * 16;
  count_launch();
  compress_values_kernel<<<blocks_for(nv, T), T, 0, st>>>(d, geo, (const uint2*)w, pattern, (uint32_t*)w_comp);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  int64_t nm = (int64_t)geo.m_tiles * geo.stages * 512;
  count_launch();
  compress_meta_kernel<<<blocks_for(nm, T), T, 0, st>>>(d, geo, pattern, (uint32_t*)meta);
  return cudaGetLastError();
}

cudaError_t launch_decompress(const ssconv_desc_t& d, const void* w_comp, const void* meta, void* w_out,
                              uint8_t* pattern_out, cudaStream_t st) {
  Geometry geo = make_geometry(d);
  const int T = 256;
  int64_t G = (int64_t)d.C_out * geo.taps * (d.C_in / 4);
  count_launch();
  decompress_kernel<<<blocks_for(G, T), T, 0, st>>>(d, geo, (const uint32_t*)w_comp, (const uint32_t*)meta,
                                                    (uint2*)w_out, pattern_out);
  return cudaGetLastError();
}

}  // namespace ssconv
