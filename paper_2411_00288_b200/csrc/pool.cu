// Max-pooling and a partial unfold over NHWC bf16 activations.
//
// Max-pooling: the pooling step between the stem and the first block of
// a ResNet-shaped stack.  Purely HBM-bound: every input element is read once (neighbouring windows
// overlap in L1/L2), every output element written once.  One thread per 8 channels (16 bytes) of
// one output pixel; consecutive threads take consecutive channel groups, so a warp reads and writes
// whole 128-byte lines whenever C >= 64.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "layout.cuh"
#include "ssconv.h"

namespace ssconv {

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
  __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&a);
  __nv_bfloat162 y = *reinterpret_cast<__nv_bfloat162*>(&b);
  __nv_bfloat162 m = __hmax2(x, y);
  return *reinterpret_cast<uint32_t*>(&m);
}

__global__ void __launch_bounds__(256) maxpool_nhwc_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int N,
                                                           int H, int W, int C8, int Ho, int Wo, int k, int stride,
                                                           int pad) {
  const long long total = (long long)N * Ho * Wo * C8;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int c = (int)(i % C8);
  long long pix = i / C8;
  const int wo = (int)(pix % Wo);
  pix /= Wo;
  const int ho = (int)(pix % Ho);
  const int n = (int)(pix / Ho);
  const uint32_t neg_inf2 = 0xFF80FF80u;  // bf16 -inf twice: padding never wins
  uint4 m = make_uint4(neg_inf2, neg_inf2, neg_inf2, neg_inf2);
  for (int kh = 0; kh < k; ++kh) {
    const int h = ho * stride - pad + kh;
    if (h < 0 || h >= H) continue;
    for (int kw = 0; kw < k; ++kw) {
      const int w = wo * stride - pad + kw;
      if (w < 0 || w >= W) continue;
      const uint4 v = __ldg(x + ((long long)(n * H + h) * W + w) * C8 + c);
      m.x = max_bf16x2(m.x, v.x);
      m.y = max_bf16x2(m.y, v.y);
      m.z = max_bf16x2(m.z, v.z);
      m.w = max_bf16x2(m.w, v.w);
    }
  }
  y[i] = m;
}

// The 3 x 3 window of stride 2 and padding 1 (the pooling of the ResNets): a thread walks kPoolRows
// output rows of one (column, 8 channels) and keeps the maximum over the three columns of the odd image
// row that two neighbouring windows share, so every image row is loaded once per thread (six 16-byte
// loads per output instead of nine, all independent).
constexpr int kPoolRows = 8;
__device__ __forceinline__ uint4 max4(uint4 a, uint4 b) {
  return make_uint4(max_bf16x2(a.x, b.x), max_bf16x2(a.y, b.y), max_bf16x2(a.z, b.z), max_bf16x2(a.w, b.w));
}
__global__ void __launch_bounds__(256) maxpool3s2_nhwc_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int N,
                                                              int H, int W, int C8, int Ho, int Wo, int strips) {
  const long long total = (long long)N * strips * Wo * C8;
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int c = (int)(i % C8);
  i /= C8;
  const int wo = (int)(i % Wo);
  i /= Wo;
  const int strip = (int)(i % strips);
  const int n = (int)(i / strips);
  const uint32_t neg_inf2 = 0xFF80FF80u;  // bf16 -inf twice: padding never wins
  const uint4 lowest = make_uint4(neg_inf2, neg_inf2, neg_inf2, neg_inf2);
  const int w0 = 2 * wo - 1;
  const bool left = w0 >= 0, right = w0 + 2 < W;
  const uint4* img = x + (long long)n * H * W * C8 + c;
  // maximum over the window's three columns of image row h
  auto row_max = [&](int h) -> uint4 {
    if (h < 0 || h >= H) return lowest;
    const uint4* centre = img + ((long long)h * W + w0 + 1) * C8;
    uint4 m = __ldg(centre);
    if (left) m = max4(m, __ldg(centre - C8));
    if (right) m = max4(m, __ldg(centre + C8));
    return m;
  };
  const int ho0 = strip * kPoolRows;
  uint4 prev = row_max(2 * ho0 - 1);
  uint4* out = y + (((long long)n * Ho + ho0) * Wo + wo) * C8 + c;
#pragma unroll 2
  for (int r = 0; r < kPoolRows; ++r) {
    const int ho = ho0 + r;
    if (ho >= Ho) break;
    const uint4 m1 = row_max(2 * ho), m2 = row_max(2 * ho + 1);
    out[(long long)r * Wo * C8] = max4(max4(prev, m1), m2);
    prev = m2;
  }
}

// Partial unfold along the width (the unfold U(X) of Eq. 5 restricted to one filter row): the KW
// taps of a filter row become channels,
//   y[n, h, wo, kw C + c] = x[n, h, wo s - p + kw d, c]   (0 outside the image and for channels >= KW C),
// so that a KH x KW convolution over C channels equals a KH x 1 convolution with unit horizontal
// stride over C_pad channels of y.  For layers with very few input channels (an RGB stem padded to 8)
// this turns 16-byte pixels into 128-byte ones, which the convolution's loads handle at full rate.
// One thread per 16 bytes of y; HBM-bound on the write of y.
__global__ void __launch_bounds__(256) unfold_w_kernel(const uint4* __restrict__ x, uint4* __restrict__ y,
                                                       long long total, int W, int C8, int Wo, int Cp8, int KW,
                                                       int stride, int pad, int dil) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int ch = (int)(i % Cp8);       // 16-byte chunk of the output pixel
  const long long pix = i / Cp8;       // (n h) * Wo + wo
  const int wo = (int)(pix % Wo);
  const long long row = pix / Wo;      // n * H + h
  const int kw = ch / C8, c = ch - kw * C8;
  const int w = wo * stride - pad + kw * dil;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (kw < KW && w >= 0 && w < W) v = __ldg(x + (row * W + w) * C8 + c);
  y[i] = v;
}

// Channel padding: y[p, c] = x[p, c] for c < C, 0 for C <= c < C_pad (an RGB image into the 8-channel
// form the dense entry point takes).  One thread per 16 bytes of y; the reads are scalar (a pixel of
// 3 channels is 6 bytes), which is harmless at this size: the step moves about a quarter of the
// bytes of the layer that follows it.
__global__ void __launch_bounds__(256) pad_channels_kernel(const __nv_bfloat16* __restrict__ x, uint4* __restrict__ y,
                                                           long long total, int C, int Cp8) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int ch = (int)(i % Cp8) * 8;
  const long long pix = i / Cp8;
  const unsigned short* src = reinterpret_cast<const unsigned short*>(x) + pix * C;
  unsigned short v[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) v[j] = (ch + j < C) ? __ldg(src + ch + j) : (unsigned short)0;
  uint4 o;
  o.x = v[0] | ((uint32_t)v[1] << 16);
  o.y = v[2] | ((uint32_t)v[3] << 16);
  o.z = v[4] | ((uint32_t)v[5] << 16);
  o.w = v[6] | ((uint32_t)v[7] << 16);
  y[i] = o;
}

// Space to depth: blocks of `s` x `s` pixels of the zero-padded image become the channels of one
// pixel,  y[n, r, q, (bh s + bw) C + c] = x[n, s r - pad + bh, s q - pad + bw, c]  (0 outside the image
// and in the channels beyond s s C), for r < Hb, q < Wb.  A K x K convolution of stride s and padding
// pad over x is then a ceil(K/s) x ceil(K/s) convolution of unit stride and no padding over y (with
// weights rearranged by the same call, as K x K "images" with pad 0), when Hb = H_out + ceil(K/s) - 1
// rows are produced: few-channel images turn into pixels wide enough for the tensor-core path without
// the (K-fold) duplication of an unfold.  One thread per V channels (16 or 8 bytes) of y; scalar reads.
template <int V>
__global__ void __launch_bounds__(256) space_to_depth_kernel(const unsigned short* __restrict__ x, uint32_t* __restrict__ y,
                                                             int H, int W, int C, int s, int pad, int Hb, int Wb,
                                                             int CpV) {
  // one grid row per row of y (n, r); threads along the row's chunks of V channels (q, k)
  const int col = blockIdx.y * blockDim.x + threadIdx.x;
  if (col >= Wb * CpV) return;
  const int row = blockIdx.x;
  const int n = row / Hb, r = row - n * Hb;
  const int q = col / CpV, k = col - q * CpV;
  // channel V k of the pixel = (block pixel blk = bh s + bw, channel c); the next V - 1 follow incrementally
  int blk = (V * k) / C, c = V * k - blk * C;
  int bh = blk / s, bw = blk - bh * s;
  const unsigned short* img = x + (size_t)n * H * W * C;
  unsigned short v[V];
#pragma unroll
  for (int j = 0; j < V; ++j) {
    const int h = s * r - pad + bh, w = s * q - pad + bw;
    v[j] = (bh < s && h >= 0 && h < H && w >= 0 && w < W) ? __ldg(img + ((size_t)h * W + w) * C + c) : (unsigned short)0;
    if (++c == C) {
      c = 0;
      if (++bw == s) {
        bw = 0;
        ++bh;
      }
    }
  }
  uint32_t* dst = y + ((size_t)row * Wb * CpV + col) * (V / 2);
  if (V == 8) {
    *reinterpret_cast<uint4*>(dst) = make_uint4(v[0] | ((uint32_t)v[1] << 16), v[2] | ((uint32_t)v[3] << 16),
                                                v[4 % V] | ((uint32_t)v[5 % V] << 16), v[6 % V] | ((uint32_t)v[7 % V] << 16));
  } else {
    *reinterpret_cast<uint2*>(dst) = make_uint2(v[0] | ((uint32_t)v[1] << 16), v[2] | ((uint32_t)v[3] << 16));
  }
}

// The same for RGB images and blocks of S x S pixels, S = 2 or 4, with unpadded pixels of 3 S S channels
// (24 or 96 bytes): a row of y interleaves pieces of 3 S elements of S image rows, so a block stages the S
// rows in shared memory (16-byte loads; element (w + pad) 3 + c of a staged row is channel c of column w,
// zeros outside the image) and writes the row of y as 8-byte words: pixel q is elements 3 S q .. 3 S q + 3 S - 1
// of the first row, then of the second, and so on.  Every image byte is read once and every byte of y
// written once.
template <int S>
__global__ void __launch_bounds__(128) space_to_depth_rgb_kernel(const uint4* __restrict__ x, uint2* __restrict__ y, int H,
                                                                 int W, int pad, int Hb, int Wb) {
  extern __shared__ uint32_t s2d_rows[];  // S rows of 3 S Wb / 2 words (3 S Wb elements)
  const int row = blockIdx.x;
  const int n = row / Hb, r = row - n * Hb;
  constexpr int kPieceWords = 3 * S / 2;       // words of one image row in one pixel of y
  const int words = kPieceWords * Wb;          // words of a staged row
  unsigned short* el = reinterpret_cast<unsigned short*>(s2d_rows);
  const int lead = pad * 3, body = W * 3, len = 2 * words;
#pragma unroll
  for (int dy = 0; dy < S; ++dy) {
    const int h = S * r - pad + dy;
    unsigned short* dst = el + dy * len;
    if (h < 0 || h >= H) {
      for (int i = threadIdx.x; i < words; i += blockDim.x) s2d_rows[dy * words + i] = 0u;
      continue;
    }
    for (int i = threadIdx.x; i < lead; i += blockDim.x) dst[i] = 0;
    for (int i = lead + body + threadIdx.x; i < len; i += blockDim.x) dst[i] = 0;
    const uint4* src = x + ((size_t)n * H + h) * (size_t)(body / 8);
    for (int i = threadIdx.x; i < body / 8; i += blockDim.x) {
      const uint4 v = __ldg(src + i);
      const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int e = lead + 8 * i + 2 * j;
        if (e < len) dst[e] = (unsigned short)(wv[j] & 0xFFFFu);
        if (e + 1 < len) dst[e + 1] = (unsigned short)(wv[j] >> 16);
      }
    }
  }
  __syncthreads();
  const int out_words = S * words / 2;  // 8-byte words of the row of y
  uint2* out = y + (size_t)row * out_words;
  if (S == 2) {
    const uint32_t* r0 = s2d_rows;
    const uint32_t* r1 = s2d_rows + words;
    for (int u = threadIdx.x; u < out_words; u += blockDim.x) {
      const int q = u / 3, part = u - 3 * q;
      uint2 o;
      if (part == 0) o = make_uint2(r0[3 * q], r0[3 * q + 1]);
      else if (part == 1) o = make_uint2(r0[3 * q + 2], r1[3 * q]);
      else o = make_uint2(r1[3 * q + 1], r1[3 * q + 2]);
      out[u] = o;
    }
  } else {
    // a pixel of y is S pieces of kPieceWords (an even number of) words: 8-byte word p of pixel q comes from
    // row p / (kPieceWords / 2), words kPieceWords q + 2 (p % (kPieceWords / 2)) and the next
    constexpr int kHalf = kPieceWords / 2;
    for (int u = threadIdx.x; u < out_words; u += blockDim.x) {
      const int q = u / (S * kHalf), p = u - q * (S * kHalf);
      const int dy = p / kHalf, part = p - dy * kHalf;
      out[u] = *reinterpret_cast<const uint2*>(s2d_rows + dy * words + kPieceWords * q + 2 * part);
    }
  }
}

cudaError_t launch_space_to_depth(const void* x, void* y, int N, int H, int W, int C, int s, int pad, int Hb, int Wb,
                                  int C_pad, cudaStream_t st) {
  count_launch();
  if ((s == 2 || s == 4) && C == 3 && C_pad == 3 * s * s && W % 8 == 0 && (reinterpret_cast<uintptr_t>(x) & 15u) == 0 &&
      Wb <= 1024 / s) {
    // (an image row ends at a 16-byte boundary when W is a multiple of 8; the staged rows take 6 s s Wb bytes)
    if (s == 2)
      space_to_depth_rgb_kernel<2><<<(unsigned)(N * Hb), 128, (size_t)Wb * 24, st>>>(
          static_cast<const uint4*>(x), static_cast<uint2*>(y), H, W, pad, Hb, Wb);
    else
      space_to_depth_rgb_kernel<4><<<(unsigned)(N * Hb), 128, (size_t)Wb * 96, st>>>(
          static_cast<const uint4*>(x), static_cast<uint2*>(y), H, W, pad, Hb, Wb);
    return cudaGetLastError();
  }
  const int T = 256;
  if (C_pad % 8 == 0) {
    const int per_row = Wb * (C_pad / 8);
    space_to_depth_kernel<8><<<dim3((unsigned)(N * Hb), (unsigned)((per_row + T - 1) / T)), T, 0, st>>>(
        static_cast<const unsigned short*>(x), static_cast<uint32_t*>(y), H, W, C, s, pad, Hb, Wb, C_pad / 8);
  } else {
    const int per_row = Wb * (C_pad / 4);
    space_to_depth_kernel<4><<<dim3((unsigned)(N * Hb), (unsigned)((per_row + T - 1) / T)), T, 0, st>>>(
        static_cast<const unsigned short*>(x), static_cast<uint32_t*>(y), H, W, C, s, pad, Hb, Wb, C_pad / 4);
  }
  return cudaGetLastError();
}

// Folding of f neighbouring output pixels of a row into the output channels (a rearrangement of the
// weights of Eq. 4, no arithmetic): output pixel f i + j of a convolution with KW taps of stride s and
// dilation d along the width is channel block j of pixel i of a convolution with
// KW' = (f - 1) s + (KW - 1) d + 1 undilated taps of stride f s,
//   W'[j C_out + c, kh, kw', :] = W[c, kh, kw, :]  where kw' = j s + kw d,   0 elsewhere.
// A layer of C_out <= 64 fills the 128 accumulator rows of a tile this way instead of half of them.
// Bytes, not elements: `tap` is the size of one (row, tap) vector, so the same kernel moves bf16 or
// 8-bit weights and the 2:4 patterns of their groups (whose groups of four lie inside one tap vector).
__global__ void __launch_bounds__(256) fold_weights_kernel(const uint8_t* __restrict__ w, uint8_t* __restrict__ out,
                                                           long long total, int C_out, int KH, int KW, int KWf, int s, int d,
                                                           int tap) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int b = (int)(i % tap);
  long long t = i / tap;
  const int kwf = (int)(t % KWf);
  t /= KWf;
  const int kh = (int)(t % KH);
  const int row = (int)(t / KH);
  const int j = row / C_out, c = row - j * C_out;
  const int off = kwf - j * s;
  uint8_t v = 0;
  if (off >= 0 && off % d == 0 && off / d < KW) v = w[(((long long)c * KH + kh) * KW + off / d) * tap + b];
  out[i] = v;
}
__global__ void fold_bias_kernel(const float* __restrict__ bias, float* __restrict__ out, int C_out, int total) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < total) out[i] = bias[i % C_out];
}

cudaError_t launch_fold_weights(const void* w, void* out, int C_out, int KH, int KW, int KWf, int s, int d, int f,
                                long long tap_bytes, const float* bias, float* bias_out, cudaStream_t st) {
  const long long total = (long long)f * C_out * KH * KWf * tap_bytes;
  if (w != nullptr && total > 0) {
    count_launch();
    fold_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(static_cast<const uint8_t*>(w),
                                                                       static_cast<uint8_t*>(out), total, C_out, KH, KW,
                                                                       KWf, s, d, (int)tap_bytes);
    if (cudaGetLastError() != cudaSuccess) return cudaErrorUnknown;
  }
  if (bias != nullptr) {
    count_launch();
    fold_bias_kernel<<<(unsigned)((f * C_out + 255) / 256), 256, 0, st>>>(bias, bias_out, C_out, f * C_out);
  }
  return cudaGetLastError();
}

// Depthwise convolution (groups = C_in = C_out), dense, direct: every output element is its own sum over
// the KH x KW window of one channel (Eq. 4 with a single input channel per output channel).  The paper
// leaves such layers untouched by the mask (Sec. 4); they are here so that a ConvNeXt-shaped block
// chains through the library.  One thread per 8 channels of an output pixel: 16-byte loads of pixels
// and of the tap-major weights [KH, KW, C], fp32 accumulation, bias, one rounding to bf16.
__global__ void __launch_bounds__(256) depthwise_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w,
                                                        const float* __restrict__ bias, uint4* __restrict__ y, int N,
                                                        int H, int W, int C8, int Ho, int Wo, int KH, int KW, int stride,
                                                        int pad, int dil, uint32_t flags) {
  const long long total = (long long)N * Ho * Wo * C8;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int c = (int)(i % C8);
  long long pix = i / C8;
  const int wo = (int)(pix % Wo);
  pix /= Wo;
  const int ho = (int)(pix % Ho);
  const int n = (int)(pix / Ho);
  float acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
  for (int kh = 0; kh < KH; ++kh) {
    const int h = ho * stride - pad + kh * dil;
    if (h < 0 || h >= H) continue;
    for (int kw = 0; kw < KW; ++kw) {
      const int ww = wo * stride - pad + kw * dil;
      if (ww < 0 || ww >= W) continue;
      const uint4 xv = __ldg(x + ((long long)(n * H + h) * W + ww) * C8 + c);
      const uint4 wv = __ldg(w + (long long)(kh * KW + kw) * C8 + c);
      const uint32_t xa[4] = {xv.x, xv.y, xv.z, xv.w}, wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        acc[2 * j] = fmaf(__uint_as_float(xa[j] << 16), __uint_as_float(wa[j] << 16), acc[2 * j]);
        acc[2 * j + 1] = fmaf(__uint_as_float(xa[j] & 0xFFFF0000u), __uint_as_float(wa[j] & 0xFFFF0000u), acc[2 * j + 1]);
      }
    }
  }
  uint32_t out[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float lo = acc[2 * j], hi = acc[2 * j + 1];
    if (flags & SSCONV_FLAG_BIAS) {
      lo += bias[8 * c + 2 * j];
      hi += bias[8 * c + 2 * j + 1];
    }
    if (flags & SSCONV_FLAG_RELU) {
      lo = fmaxf(lo, 0.0f);
      hi = fmaxf(hi, 0.0f);
    }
    __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    out[j] = *reinterpret_cast<uint32_t*>(&b);
  }
  y[i] = make_uint4(out[0], out[1], out[2], out[3]);
}

// Unit stride, no dilation, KW = 3, 5 or 7: a thread computes kDwRun consecutive output pixels of a row for
// its 8 channels, so an image pixel is loaded once per filter row for all the outputs of the run it
// touches (10 loads per row for 4 outputs of a 7-wide filter instead of 28) and the row's weights are
// unpacked to fp32 once; what remains is the 8 KH KW multiply-adds per output, in fp32, two per instruction.
constexpr int kDwRun = 8;
// Two fp32 multiply-adds in one instruction (sm_100: fma.rn.f32x2 on register pairs): d = a * b + d per half.
__device__ __forceinline__ void fma2(unsigned long long& d, unsigned long long a, unsigned long long b) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}
// A bf16 pair widened to an fp32 pair (low element in the low half).
__device__ __forceinline__ unsigned long long widen2(uint32_t v) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(v << 16), "r"(v & 0xFFFF0000u));
  return r;
}
template <int KW>
__global__ void __launch_bounds__(128, 4) depthwise_run_kernel(const uint2* __restrict__ x, const uint2* __restrict__ w,
                                                               const float* __restrict__ bias, uint2* __restrict__ y, int N,
                                                               int H, int W, int C4, int Ho, int Wo, int KH, int pad,
                                                               int runs, uint32_t flags) {
  // (4 channels = 8 bytes per thread: half the registers of a 16-byte version, twice the resident warps)
  const long long total = (long long)N * Ho * runs * C4;
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int c = (int)(i % C4);
  i /= C4;
  const int run = (int)(i % runs);
  i /= runs;
  const int ho = (int)(i % Ho);
  const int n = (int)(i / Ho);
  const int wo0 = run * kDwRun;
  unsigned long long acc[kDwRun][2];  // fp32 pairs
#pragma unroll
  for (int t = 0; t < kDwRun; ++t) acc[t][0] = acc[t][1] = 0ull;
  for (int kh = 0; kh < KH; ++kh) {
    const int h = ho - pad + kh;
    if (h < 0 || h >= H) continue;
    unsigned long long wf[KW][2];
#pragma unroll
    for (int kw = 0; kw < KW; ++kw) {
      const uint2 wv = __ldg(w + (long long)(kh * KW + kw) * C4 + c);
      wf[kw][0] = widen2(wv.x);
      wf[kw][1] = widen2(wv.y);
    }
    // all pixels of the row first (independent loads in flight together), then the arithmetic
    const uint2* row = x + ((long long)(n * H + h) * W) * C4 + c;
    uint2 xv[kDwRun + KW - 1];
#pragma unroll
    for (int col = 0; col < kDwRun + KW - 1; ++col) {
      const int ww = wo0 - pad + col;
      const bool in = ww >= 0 && ww < W;
      xv[col] = in ? __ldg(row + (long long)(in ? ww : 0) * C4) : make_uint2(0u, 0u);
    }
#pragma unroll
    for (int col = 0; col < kDwRun + KW - 1; ++col) {
      const unsigned long long x0 = widen2(xv[col].x), x1 = widen2(xv[col].y);
#pragma unroll
      for (int kw = 0; kw < KW; ++kw) {
        const int t = col - kw;  // the output of the run that meets this pixel at tap kw
        if (t >= 0 && t < kDwRun) {
          fma2(acc[t][0], x0, wf[kw][0]);
          fma2(acc[t][1], x1, wf[kw][1]);
        }
      }
    }
  }
  float bv[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) bv[j] = (flags & SSCONV_FLAG_BIAS) ? bias[4 * c + j] : 0.0f;
  uint2* out = y + ((long long)(n * Ho + ho) * Wo + wo0) * C4 + c;
#pragma unroll
  for (int t = 0; t < kDwRun; ++t) {
    if (wo0 + t >= Wo) break;
    uint32_t o[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      float lo = __uint_as_float((uint32_t)acc[t][j]) + bv[2 * j];
      float hi = __uint_as_float((uint32_t)(acc[t][j] >> 32)) + bv[2 * j + 1];
      if (flags & SSCONV_FLAG_RELU) {
        lo = fmaxf(lo, 0.0f);
        hi = fmaxf(hi, 0.0f);
      }
      __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
      o[j] = *reinterpret_cast<uint32_t*>(&b2);
    }
    out[(long long)t * C4] = make_uint2(o[0], o[1]);
  }
}

// Unit stride, no dilation, square K x K filter, C a multiple of 32: a thread computes a tile of
// kDwTileH x kDwTileW output pixels for one pair of channels, so that an image pixel is loaded and widened
// once for all the (up to K per direction) outputs of the tile it meets: (kDwTileH + K - 1)(kDwTileW + K - 1)
// four-byte loads for kDwTileH kDwTileW K^2 paired multiply-adds (140 for 1568 with K = 7), against one load
// per K paired multiply-adds in the row-run kernel above.  Sixteen lanes hold sixteen neighbouring channel
// pairs of one tile (64 contiguous bytes per pixel); a block's eight tiles share the same 32 channels,
// whose filter it keeps in shared memory as fp32 pairs.  The loop over image rows stays rolled (the filter
// row under which image row r meets output row o is r - o, looked up at run time): unrolled, the kernel
// waited on instruction fetch.  Addresses are a per-row pointer plus 32-bit offsets, constants when the
// channel count is one of the instantiated ones (C2T, in channel pairs; 0 = taken from the argument).
// The tile is TW = 8 pixels wide, or 7 where that divides the output width and 8 does not (feature maps
// of 7, 14, 28 and 56 pixels: no multiply-adds spent beyond the row's end); output rows beyond the
// map's last are skipped.
constexpr int kDwTileH = 4;
__device__ __forceinline__ float2 widen_f2(uint32_t v) {
  return make_float2(__uint_as_float(v << 16), __uint_as_float(v & 0xFFFF0000u));
}
template <int K, int C2T, int TW>
__global__ void __launch_bounds__(128, 4) depthwise_tile_kernel(const uint32_t* __restrict__ x, const uint32_t* __restrict__ w,
                                                                const float* __restrict__ bias, uint32_t* __restrict__ y,
                                                                int H, int W, int C2r, int Ho, int Wo, int pad, int tiles_h,
                                                                int tiles_w, long long tiles, uint32_t flags) {
  const int C2 = C2T ? C2T : C2r;
  __shared__ float2 w_s[K * K][16];
  const int sub = threadIdx.x & 15;
  const int c2 = blockIdx.y * 16 + sub;
  for (int i = threadIdx.x; i < K * K * 16; i += 128)
    w_s[i >> 4][i & 15] = widen_f2(__ldg(w + (long long)(i >> 4) * C2 + blockIdx.y * 16 + (i & 15)));
  __syncthreads();
  long long tile = (long long)blockIdx.x * 8 + (threadIdx.x >> 4);
  if (tile >= tiles) return;
  const int tw = (int)(tile % tiles_w);
  tile /= tiles_w;
  const int th = (int)(tile % tiles_h);
  const int n = (int)(tile / tiles_h);
  const int h0 = th * kDwTileH, w0 = tw * TW;
  constexpr int kCols = TW + K - 1, kRows = kDwTileH + K - 1;
  float2 acc[kDwTileH][TW];
  {
    float2 b = make_float2(0.0f, 0.0f);
    if (flags & SSCONV_FLAG_BIAS) b = __ldg(reinterpret_cast<const float2*>(bias) + c2);
#pragma unroll
    for (int o = 0; o < kDwTileH; ++o)
#pragma unroll
      for (int t = 0; t < TW; ++t) acc[o][t] = b;
  }
  const int wi0 = w0 - pad;  // image column under the tile's first output at tap 0
  const bool cols_in = wi0 >= 0 && wi0 + kCols <= W;
  // image column wi0 of image row h0 - pad (possibly outside the image: dereferenced only where it is inside)
  const uint32_t* rowp = x + (((long long)n * H + (h0 - pad)) * W + wi0) * C2 + c2;
  const int row_step = W * C2;
  const float2* wp = &w_s[0][sub];
#pragma unroll 1
  for (int r = 0; r < kRows; ++r, rowp += row_step) {
    const int h = h0 - pad + r;
    if (h < 0 || h >= H) continue;
    float2 xv[kCols];
    if (cols_in) {
#pragma unroll
      for (int col = 0; col < kCols; ++col) xv[col] = widen_f2(__ldg(rowp + col * C2));
    } else {
#pragma unroll
      for (int col = 0; col < kCols; ++col) {
        uint32_t v = 0u;
        if (wi0 + col >= 0 && wi0 + col < W) v = __ldg(rowp + col * C2);
        xv[col] = widen_f2(v);
      }
    }
#pragma unroll
    for (int o = 0; o < kDwTileH; ++o) {
      const int ky = r - o;  // filter row under which image row r meets output row o of the tile
      if (ky < 0 || ky >= K || h0 + o >= Ho) continue;
      const float2* wr = wp + ky * (K * 16);
#pragma unroll
      for (int kx = 0; kx < K; ++kx) {
        const float2 wk = wr[kx * 16];
#pragma unroll
        for (int t = 0; t < TW; ++t) acc[o][t] = __ffma2_rn(xv[t + kx], wk, acc[o][t]);
      }
    }
  }
#pragma unroll
  for (int o = 0; o < kDwTileH; ++o) {
    if (h0 + o >= Ho) break;
    uint32_t* out = y + (((long long)n * Ho + h0 + o) * Wo + w0) * C2 + c2;
#pragma unroll
    for (int t = 0; t < TW; ++t) {
      if (w0 + t >= Wo) break;
      float lo = acc[o][t].x, hi = acc[o][t].y;
      if (flags & SSCONV_FLAG_RELU) {
        lo = fmaxf(lo, 0.0f);
        hi = fmaxf(hi, 0.0f);
      }
      __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
      out[t * C2] = *reinterpret_cast<uint32_t*>(&b2);
    }
  }
}

cudaError_t launch_depthwise(const void* x, const void* w, const float* bias, void* y, int N, int H, int W, int C, int Ho,
                             int Wo, int KH, int KW, int stride, int pad, int dil, uint32_t flags, cudaStream_t st) {
  const long long total = (long long)N * Ho * Wo * (C / 8);
  if (total == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
  if (stride == 1 && dil == 1 && KH == KW && (KW == 3 || KW == 5 || KW == 7) && C % 32 == 0) {
    const int tw = (KW == 7 && Wo % 7 == 0 && Wo % 8 != 0) ? 7 : 8;
    const int tiles_h = (Ho + kDwTileH - 1) / kDwTileH, tiles_w = (Wo + tw - 1) / tw;
    const long long tiles = (long long)N * tiles_h * tiles_w;
    const dim3 grid((unsigned)((tiles + 7) / 8), (unsigned)(C / 32));
    const uint32_t* xp = static_cast<const uint32_t*>(x);
    const uint32_t* wp = static_cast<const uint32_t*>(w);
    uint32_t* yp = static_cast<uint32_t*>(y);
#define SSCONV_DW_TILE(KK, CC, TT) \
  depthwise_tile_kernel<KK, CC, TT><<<grid, 128, 0, st>>>(xp, wp, bias, yp, H, W, C / 2, Ho, Wo, pad, tiles_h, tiles_w, tiles, flags)
#define SSCONV_DW_TILE7(CC)  \
  do {                       \
    if (tw == 7)             \
      SSCONV_DW_TILE(7, CC, 7); \
    else                     \
      SSCONV_DW_TILE(7, CC, 8); \
  } while (0)
    if (KW == 3)
      SSCONV_DW_TILE(3, 0, 8);
    else if (KW == 5)
      SSCONV_DW_TILE(5, 0, 8);
    else if (C == 96)
      SSCONV_DW_TILE7(48);
    else if (C == 192)
      SSCONV_DW_TILE7(96);
    else if (C == 384)
      SSCONV_DW_TILE7(192);
    else if (C == 768)
      SSCONV_DW_TILE7(384);
    else
      SSCONV_DW_TILE7(0);
#undef SSCONV_DW_TILE7
#undef SSCONV_DW_TILE
    return cudaGetLastError();
  }
  if (stride == 1 && dil == 1 && (KW == 3 || KW == 5 || KW == 7)) {
    const int runs = (Wo + kDwRun - 1) / kDwRun;
    const long long threads = (long long)N * Ho * runs * (C / 4);
    const unsigned grid = (unsigned)((threads + 127) / 128);
    const uint2* xp = static_cast<const uint2*>(x);
    const uint2* wp = static_cast<const uint2*>(w);
    uint2* yp = static_cast<uint2*>(y);
    if (KW == 3)
      depthwise_run_kernel<3><<<grid, 128, 0, st>>>(xp, wp, bias, yp, N, H, W, C / 4, Ho, Wo, KH, pad, runs, flags);
    else if (KW == 5)
      depthwise_run_kernel<5><<<grid, 128, 0, st>>>(xp, wp, bias, yp, N, H, W, C / 4, Ho, Wo, KH, pad, runs, flags);
    else
      depthwise_run_kernel<7><<<grid, 128, 0, st>>>(xp, wp, bias, yp, N, H, W, C / 4, Ho, Wo, KH, pad, runs, flags);
    return cudaGetLastError();
  }
  depthwise_kernel<<<(unsigned)((total + T - 1) / T), T, 0, st>>>(static_cast<const uint4*>(x), static_cast<const uint4*>(w),
                                                                  bias, static_cast<uint4*>(y), N, H, W, C / 8, Ho, Wo, KH,
                                                                  KW, stride, pad, dil, flags);
  return cudaGetLastError();
}

// Layer normalisation over the channels of each pixel (the normalisation of a ConvNeXt block; not part
// of the paper's method): y = (x - mean) / sqrt(var + eps) * gamma + beta with the biased variance, in
// fp32, one rounding to bf16.  One warp per pixel; a lane holds C / 32 rounded up channels in registers.
__global__ void __launch_bounds__(256) layernorm_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ gamma,
                                                        const float* __restrict__ beta, __nv_bfloat16* __restrict__ y,
                                                        long long pixels, int C, float eps) {
  const long long pix = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (pix >= pixels) return;
  const __nv_bfloat16* xp = x + pix * C;
  float sum = 0.0f;
  for (int c = lane; c < C; c += 32) sum += __bfloat162float(xp[c]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float mean = sum / (float)C;
  float sq = 0.0f;
  for (int c = lane; c < C; c += 32) {
    const float d = __bfloat162float(xp[c]) - mean;
    sq += d * d;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const float rstd = rsqrtf(sq / (float)C + eps);
  for (int c = lane; c < C; c += 32)
    y[pix * C + c] = __float2bfloat16_rn((__bfloat162float(xp[c]) - mean) * rstd * gamma[c] + beta[c]);
}

// C a multiple of 8 and at most 1024: a group of G lanes (a power of two, G >= C / 8 up to 32) per pixel,
// a lane holding V 16-byte pieces of it in registers: one read and one write of the tensor, 16 bytes at
// a time, statistics by shuffles within the group.
template <int V>
__global__ void __launch_bounds__(256) layernorm_vec_kernel(const uint4* __restrict__ x, const float* __restrict__ gamma,
                                                            const float* __restrict__ beta, uint4* __restrict__ y,
                                                            long long pixels, int C8, int G, float eps) {
  const int lane = threadIdx.x & 31;
  const int sub = lane & (G - 1);
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long pix = warp * (32 / G) + lane / G;
  const bool live = pix < pixels;
  float f[V][8];
  float sum = 0.0f;
#pragma unroll
  for (int k = 0; k < V; ++k) {
    const int idx = sub + k * G;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (live && idx < C8) v = __ldg(x + pix * C8 + idx);
    const uint32_t a[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      f[k][2 * j] = __uint_as_float(a[j] << 16);
      f[k][2 * j + 1] = __uint_as_float(a[j] & 0xFFFF0000u);
      sum += f[k][2 * j] + f[k][2 * j + 1];
    }
  }
  for (int o = G >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float inv_c = 1.0f / (float)(8 * C8);
  const float mean = sum * inv_c;
  float sq = 0.0f;
#pragma unroll
  for (int k = 0; k < V; ++k) {
    if (sub + k * G < C8) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float d = f[k][j] - mean;
        sq += d * d;
      }
    }
  }
  for (int o = G >> 1; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  const float rstd = rsqrtf(sq * inv_c + eps);
#pragma unroll
  for (int k = 0; k < V; ++k) {
    const int idx = sub + k * G;
    if (!live || idx >= C8) continue;
    const float4 g0 = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * idx);
    const float4 g1 = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * idx + 1);
    const float4 b0 = __ldg(reinterpret_cast<const float4*>(beta) + 2 * idx);
    const float4 b1 = __ldg(reinterpret_cast<const float4*>(beta) + 2 * idx + 1);
    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      __nv_bfloat162 p = __floats2bfloat162_rn((f[k][2 * j] - mean) * rstd * gg[2 * j] + bb[2 * j],
                                               (f[k][2 * j + 1] - mean) * rstd * gg[2 * j + 1] + bb[2 * j + 1]);
      o[j] = *reinterpret_cast<uint32_t*>(&p);
    }
    y[pix * C8 + idx] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

cudaError_t launch_layernorm(const void* x, const float* gamma, const float* beta, void* y, long long pixels, int C,
                             float eps, cudaStream_t st) {
  if (pixels == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
  const bool aligned = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(gamma) |
                         reinterpret_cast<uintptr_t>(beta)) & 15u) == 0;
  if (C % 8 == 0 && C <= 1024 && aligned) {
    const int C8 = C / 8;
    // lanes per pixel: the largest power of two dividing C8 if that leaves at most four pieces per lane
    // (every lane busy: 96 channels = 4 lanes x 3 pieces), else the smallest power of two covering C8
    int G = 1;
    while (G < 32 && C8 % (2 * G) == 0) G <<= 1;
    if (C8 / G > 4) {
      G = 1;
      while (G < C8 && G < 32) G <<= 1;
    }
    const int V = (C8 + G - 1) / G;
    const long long warps = (pixels + (32 / G) - 1) / (32 / G);
    const unsigned grid = (unsigned)((warps * 32 + T - 1) / T);
    const uint4* xp = static_cast<const uint4*>(x);
    uint4* yp = static_cast<uint4*>(y);
    if (V == 1)
      layernorm_vec_kernel<1><<<grid, T, 0, st>>>(xp, gamma, beta, yp, pixels, C8, G, eps);
    else if (V == 2)
      layernorm_vec_kernel<2><<<grid, T, 0, st>>>(xp, gamma, beta, yp, pixels, C8, G, eps);
    else if (V == 3)
      layernorm_vec_kernel<3><<<grid, T, 0, st>>>(xp, gamma, beta, yp, pixels, C8, G, eps);
    else
      layernorm_vec_kernel<4><<<grid, T, 0, st>>>(xp, gamma, beta, yp, pixels, C8, G, eps);
    return cudaGetLastError();
  }
  layernorm_kernel<<<(unsigned)((pixels * 32 + T - 1) / T), T, 0, st>>>(static_cast<const __nv_bfloat16*>(x), gamma, beta,
                                                                        static_cast<__nv_bfloat16*>(y), pixels, C, eps);
  return cudaGetLastError();
}

cudaError_t launch_pad_channels(const void* x, void* y, long long pixels, int C, int C_pad, cudaStream_t st) {
  const long long total = pixels * (C_pad / 8);
  if (total == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
  pad_channels_kernel<<<(unsigned)((total + T - 1) / T), T, 0, st>>>(static_cast<const __nv_bfloat16*>(x),
                                                                     static_cast<uint4*>(y), total, C, C_pad / 8);
  return cudaGetLastError();
}

cudaError_t launch_unfold_w(const void* x, void* y, long long rows, int W, int C, int KW, int stride, int pad, int dil,
                            int C_pad, cudaStream_t st) {
  const int span = W + 2 * pad - dil * (KW - 1) - 1;
  const int Wo = span < 0 ? 0 : span / stride + 1;
  const long long total = rows * Wo * (C_pad / 8);
  if (total == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
  unfold_w_kernel<<<(unsigned)((total + T - 1) / T), T, 0, st>>>(static_cast<const uint4*>(x), static_cast<uint4*>(y),
                                                                 total, W, C / 8, Wo, C_pad / 8, KW, stride, pad, dil);
  return cudaGetLastError();
}

cudaError_t launch_maxpool(const void* x, void* y, int N, int H, int W, int C, int k, int stride, int pad,
                           cudaStream_t st) {
  const int Ho = (H + 2 * pad - k) / stride + 1, Wo = (W + 2 * pad - k) / stride + 1;
  const long long total = (long long)N * Ho * Wo * (C / 8);
  if (total == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
  if (k == 3 && stride == 2 && pad == 1 && W >= 2) {
    const int strips = (Ho + kPoolRows - 1) / kPoolRows;
    const long long threads = (long long)N * strips * Wo * (C / 8);
    maxpool3s2_nhwc_kernel<<<(unsigned)((threads + T - 1) / T), T, 0, st>>>(
        static_cast<const uint4*>(x), static_cast<uint4*>(y), N, H, W, C / 8, Ho, Wo, strips);
    return cudaGetLastError();
  }
  maxpool_nhwc_kernel<<<(unsigned)((total + T - 1) / T), T, 0, st>>>(static_cast<const uint4*>(x),
                                                                     static_cast<uint4*>(y), N, H, W, C / 8, Ho, Wo,
                                                                     k, stride, pad);
  return cudaGetLastError();
}

}  // namespace ssconv
