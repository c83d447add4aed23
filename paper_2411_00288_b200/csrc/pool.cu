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
// the (K-fold) duplication of an unfold.  One thread per 16 bytes of y; scalar reads.
__global__ void __launch_bounds__(256) space_to_depth_kernel(const unsigned short* __restrict__ x, uint4* __restrict__ y,
                                                             int H, int W, int C, int s, int pad, int Hb, int Wb,
                                                             int Cp8) {
  // one grid row per row of y (n, r); threads along the row's 16-byte chunks (q, k)
  const int col = blockIdx.y * blockDim.x + threadIdx.x;
  if (col >= Wb * Cp8) return;
  const int row = blockIdx.x;
  const int n = row / Hb, r = row - n * Hb;
  const int q = col / Cp8, k = col - q * Cp8;
  // channel 8 k of the pixel = (block pixel blk = bh s + bw, channel c); the next seven follow incrementally
  int blk = (8 * k) / C, c = 8 * k - blk * C;
  int bh = blk / s, bw = blk - bh * s;
  const unsigned short* img = x + (size_t)n * H * W * C;
  unsigned short v[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
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
  uint4 o;
  o.x = v[0] | ((uint32_t)v[1] << 16);
  o.y = v[2] | ((uint32_t)v[3] << 16);
  o.z = v[4] | ((uint32_t)v[5] << 16);
  o.w = v[6] | ((uint32_t)v[7] << 16);
  y[(size_t)row * Wb * Cp8 + col] = o;
}

cudaError_t launch_space_to_depth(const void* x, void* y, int N, int H, int W, int C, int s, int pad, int Hb, int Wb,
                                  int C_pad, cudaStream_t st) {
  const int T = 256;
  const int per_row = Wb * (C_pad / 8);
  count_launch();
  space_to_depth_kernel<<<dim3((unsigned)(N * Hb), (unsigned)((per_row + T - 1) / T)), T, 0, st>>>(
      static_cast<const unsigned short*>(x), static_cast<uint4*>(y), H, W, C, s, pad, Hb, Wb, C_pad / 8);
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

cudaError_t launch_depthwise(const void* x, const void* w, const float* bias, void* y, int N, int H, int W, int C, int Ho,
                             int Wo, int KH, int KW, int stride, int pad, int dil, uint32_t flags, cudaStream_t st) {
  const long long total = (long long)N * Ho * Wo * (C / 8);
  if (total == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
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

cudaError_t launch_layernorm(const void* x, const float* gamma, const float* beta, void* y, long long pixels, int C,
                             float eps, cudaStream_t st) {
  if (pixels == 0) return cudaSuccess;
  const int T = 256;
  count_launch();
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
  maxpool_nhwc_kernel<<<(unsigned)((total + T - 1) / T), T, 0, st>>>(static_cast<const uint4*>(x),
                                                                     static_cast<uint4*>(y), N, H, W, C / 8, Ho, Wo,
                                                                     k, stride, pad);
  return cudaGetLastError();
}

}  // namespace ssconv
