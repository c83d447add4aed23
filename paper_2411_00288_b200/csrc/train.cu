// The mask-learning step's elementwise parts (Sec. 3.1): the relaxed choice vector of every
// group (Eq. 3), the soft mask block b = D z (Eq. 2 with that z), the effective weights
// M .* W (Eq. 6 with the soft mask) that the dense convolution then uses, and the gradient
// from dL/dW_eff back to the choice weights.  One thread per group of four weights; both
// kernels move 70-90 bytes per group and do a handful of flops: HBM-bound.
#include <cuda_runtime.h>

#include "layout.cuh"
#include "ssconv.h"

namespace ssconv {

// The six patterns keep positions {0,1},{0,2},{0,3},{1,2},{1,3},{2,3}: position 0 is kept by
// patterns 0,1,2, position 1 by 0,3,4, position 2 by 1,3,5, position 3 by 2,4,5.
__device__ __forceinline__ void block_from_choice(const float (&z)[6], float (&b)[4]) {
  b[0] = z[0] + z[1] + z[2];
  b[1] = z[0] + z[3] + z[4];
  b[2] = z[1] + z[3] + z[5];
  b[3] = z[2] + z[4] + z[5];
}

__device__ __forceinline__ void load6(const float* p, int64_t g, float (&v)[6]) {
  const float2* q = reinterpret_cast<const float2*>(p) + 3 * g;
  const float2 a = q[0], b = q[1], c = q[2];
  v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y; v[4] = c.x; v[5] = c.y;
}
__device__ __forceinline__ void store6(float* p, int64_t g, const float (&v)[6]) {
  float2* q = reinterpret_cast<float2*>(p) + 3 * g;
  q[0] = make_float2(v[0], v[1]);
  q[1] = make_float2(v[2], v[3]);
  q[2] = make_float2(v[4], v[5]);
}
__device__ __forceinline__ float bf16_bits_to_f32(uint32_t bits16) { return __uint_as_float(bits16 << 16); }
__device__ __forceinline__ uint32_t f32_pair_to_bf16(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// Eq. 3 in fp32: z = softmax((logits + noise) / tau), evaluated with the maximum subtracted
// (which cancels in the quotient); then b = D z and W_eff = b .* W rounded once to bf16.
__global__ void soft_mask_kernel(const float* __restrict__ logits, const float* __restrict__ noise, float inv_tau,
                                 const uint2* __restrict__ w, int64_t G, float* __restrict__ z_out,
                                 uint2* __restrict__ w_eff) {
  const int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (g >= G) return;
  float s[6];
  load6(logits, g, s);
  if (noise != nullptr) {
    float n[6];
    load6(noise, g, n);
#pragma unroll
    for (int i = 0; i < 6; ++i) s[i] += n[i];
  }
  float m = s[0];
#pragma unroll
  for (int i = 1; i < 6; ++i) m = fmaxf(m, s[i]);
  float z[6], sum = 0.0f;
#pragma unroll
  for (int i = 0; i < 6; ++i) {
    z[i] = expf((s[i] - m) * inv_tau);
    sum += z[i];
  }
  const float inv = 1.0f / sum;
#pragma unroll
  for (int i = 0; i < 6; ++i) z[i] *= inv;
  if (z_out != nullptr) store6(z_out, g, z);
  if (w_eff != nullptr) {
    float b[4];
    block_from_choice(z, b);
    const uint2 v = w[g];
    uint2 o;
    o.x = f32_pair_to_bf16(b[0] * bf16_bits_to_f32(v.x & 0xFFFFu), b[1] * bf16_bits_to_f32(v.x >> 16));
    o.y = f32_pair_to_bf16(b[2] * bf16_bits_to_f32(v.y & 0xFFFFu), b[3] * bf16_bits_to_f32(v.y >> 16));
    w_eff[g] = o;
  }
}

// Chain rule from G = dL/dW_eff to the choice weights: dL/db_j = G_j W_j, dL/dz_i = the sum of
// dL/db over the two positions pattern i keeps, dL/dlogit_i = z_i (dL/dz_i - sum_k z_k dL/dz_k) / tau.
__global__ void mask_grad_kernel(const float* __restrict__ z_in, float inv_tau, const uint2* __restrict__ w,
                                 const float4* __restrict__ g_w_eff, int64_t G, float* __restrict__ g_logits) {
  const int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (g >= G) return;
  float z[6];
  load6(z_in, g, z);
  const uint2 v = w[g];
  const float4 up = g_w_eff[g];
  const float gb0 = up.x * bf16_bits_to_f32(v.x & 0xFFFFu), gb1 = up.y * bf16_bits_to_f32(v.x >> 16);
  const float gb2 = up.z * bf16_bits_to_f32(v.y & 0xFFFFu), gb3 = up.w * bf16_bits_to_f32(v.y >> 16);
  const float gz[6] = {gb0 + gb1, gb0 + gb2, gb0 + gb3, gb1 + gb2, gb1 + gb3, gb2 + gb3};
  float inner = 0.0f;
#pragma unroll
  for (int i = 0; i < 6; ++i) inner += z[i] * gz[i];
  float out[6];
#pragma unroll
  for (int i = 0; i < 6; ++i) out[i] = z[i] * (gz[i] - inner) * inv_tau;
  store6(g_logits, g, out);
}

// AdamW on the choice weights (Appendix, training details): decoupled weight decay, bias-corrected
// moments; c1 = 1 / (1 - beta1^t) and c2 = 1 / (1 - beta2^t) come from the host.  28 bytes per
// element: HBM-bound.
__device__ __forceinline__ void adamw_one(float& t, float g, float& m, float& v, float lr, float beta1, float beta2,
                                          float eps, float wd, float c1, float c2) {
  m = beta1 * m + (1.0f - beta1) * g;
  v = beta2 * v + (1.0f - beta2) * g * g;
  t = t - lr * (m * c1 / (sqrtf(v * c2) + eps) + wd * t);
}
// Four elements per thread (16-byte accesses); the last n % 4 elements are handled one by one.
__global__ void adamw_kernel(float* __restrict__ theta, const float* __restrict__ g, float* __restrict__ m,
                             float* __restrict__ v, int64_t n, float lr, float beta1, float beta2, float eps,
                             float wd, float c1, float c2) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  const int64_t n4 = n >> 2;
  if (i < n4) {
    float4 t = reinterpret_cast<float4*>(theta)[i];
    const float4 gi = reinterpret_cast<const float4*>(g)[i];
    float4 mi = reinterpret_cast<float4*>(m)[i], vi = reinterpret_cast<float4*>(v)[i];
    adamw_one(t.x, gi.x, mi.x, vi.x, lr, beta1, beta2, eps, wd, c1, c2);
    adamw_one(t.y, gi.y, mi.y, vi.y, lr, beta1, beta2, eps, wd, c1, c2);
    adamw_one(t.z, gi.z, mi.z, vi.z, lr, beta1, beta2, eps, wd, c1, c2);
    adamw_one(t.w, gi.w, mi.w, vi.w, lr, beta1, beta2, eps, wd, c1, c2);
    reinterpret_cast<float4*>(m)[i] = mi;
    reinterpret_cast<float4*>(v)[i] = vi;
    reinterpret_cast<float4*>(theta)[i] = t;
  } else if (i < n4 + (n & 3)) {
    const int64_t j = 4 * n4 + (i - n4);
    float t = theta[j], mi = m[j], vi = v[j];
    adamw_one(t, g[j], mi, vi, lr, beta1, beta2, eps, wd, c1, c2);
    m[j] = mi;
    v[j] = vi;
    theta[j] = t;
  }
}

cudaError_t launch_adamw(float* theta, const float* g, float* m, float* v, int64_t n, float lr, float beta1,
                         float beta2, float eps, float wd, float c1, float c2, cudaStream_t st) {
  const int threads = 256;
  const int64_t work = (n >> 2) + (n & 3);
  adamw_kernel<<<(unsigned)((work + threads - 1) / threads), threads, 0, st>>>(theta, g, m, v, n, lr, beta1, beta2,
                                                                                 eps, wd, c1, c2);
  count_launch();
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Stability quantities of Sec. 3.2
// ---------------------------------------------------------------------------------------
// Maximum absolute row sums of W [C_out x K], of the part a 2:4 mask drops, (B - 1) .* W (the additive
// perturbation of Lemma 3.3), and of the part it keeps, B .* W.  One block per row (output channel);
// a thread adds the magnitudes of its groups in fp32, the block sums them in a fixed order, and the
// row's three sums go into the result by an integer maximum (non-negative floats order like their bit
// patterns), so the result does not depend on timing.  out must be zero when the kernel starts.
__device__ __forceinline__ float block_sum_256(float v, float* scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float total = 0.0f;
  if (threadIdx.x == 0)
    for (int i = 0; i < 8; ++i) total += scratch[i];
  return total;  // valid in thread 0
}
__global__ void __launch_bounds__(256) mask_norms_kernel(const uint2* __restrict__ w, const uint8_t* __restrict__ pattern,
                                                         int64_t groups_per_row, float* __restrict__ out) {
  __shared__ float scratch[8];
  const int64_t row0 = (int64_t)blockIdx.x * groups_per_row;
  float all = 0.0f, kept = 0.0f, dropped = 0.0f;
  for (int64_t g = threadIdx.x; g < groups_per_row; g += 256) {
    const uint2 v = w[row0 + g];
    const float a[4] = {fabsf(bf16_bits_to_f32(v.x & 0xFFFFu)), fabsf(bf16_bits_to_f32(v.x >> 16)),
                        fabsf(bf16_bits_to_f32(v.y & 0xFFFFu)), fabsf(bf16_bits_to_f32(v.y >> 16))};
    const uint32_t code = pattern_code(pattern[row0 + g]);  // pos0 | pos1 << 2
    const float grp_all = (a[0] + a[1]) + (a[2] + a[3]);
    const float grp_kept = a[code & 3u] + a[(code >> 2) & 3u];
    all += grp_all;
    kept += grp_kept;
    dropped += grp_all - grp_kept;
  }
  const float s_all = block_sum_256(all, scratch);
  const float s_drop = block_sum_256(dropped, scratch);
  const float s_kept = block_sum_256(kept, scratch);
  if (threadIdx.x == 0) {
    atomicMax(reinterpret_cast<int*>(out), __float_as_int(s_all));
    atomicMax(reinterpret_cast<int*>(out) + 1, __float_as_int(fmaxf(s_drop, 0.0f)));
    atomicMax(reinterpret_cast<int*>(out) + 2, __float_as_int(s_kept));
  }
}

// ||x||_inf of n bf16 values (n a multiple of 8 handled 16 bytes at a time, the rest one by one).
__global__ void __launch_bounds__(256) absmax_kernel(const uint16_t* __restrict__ x, int64_t n, float* __restrict__ out) {
  uint32_t m = 0;  // largest magnitude as the 15 bits below the sign, which order like |x|
  const int64_t n8 = n >> 3;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n8; i += (int64_t)gridDim.x * blockDim.x) {
    const uint4 v = reinterpret_cast<const uint4*>(x)[i];
    const uint32_t words[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      m = max(m, words[k] & 0x7FFFu);
      m = max(m, (words[k] >> 16) & 0x7FFFu);
    }
  }
  if (blockIdx.x == 0)
    for (int64_t i = 8 * n8 + threadIdx.x; i < n; i += blockDim.x) m = max(m, (uint32_t)x[i] & 0x7FFFu);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_down_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0 && m != 0) atomicMax(reinterpret_cast<int*>(out), (int)(m << 16));
}

cudaError_t launch_mask_norms(const void* w, const uint8_t* pattern, int C_out, int64_t K, float* out, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(out, 0, 3 * sizeof(float), st);
  if (e != cudaSuccess) return e;
  mask_norms_kernel<<<(unsigned)C_out, 256, 0, st>>>((const uint2*)w, pattern, K / 4, out);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_absmax(const void* x, int64_t n, float* out, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(out, 0, sizeof(float), st);
  if (e != cudaSuccess) return e;
  int64_t blocks = ((n >> 3) + 255) / 256;
  blocks = blocks < 1 ? 1 : (blocks > 148 * 8 ? 148 * 8 : blocks);
  absmax_kernel<<<(unsigned)blocks, 256, 0, st>>>((const uint16_t*)x, n, out);
  count_launch();
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Gradient with respect to a layer's input
// ---------------------------------------------------------------------------------------
// For unit stride, dL/dx is itself a convolution of dL/dy: with the filter taps reversed and the roles
// of input and output channels exchanged, padded by dil (K - 1) - pad.  This kernel writes those
// weights, w_t[ci][KH-1-kh][KW-1-kw][co] = w[co][kh][kw][ci]; the dense forward kernel then does the
// work.  One thread per element of w_t (writes contiguous; the strided reads hit L2: weights are small).
__global__ void __launch_bounds__(256) dgrad_weights_kernel(const uint16_t* __restrict__ w, uint16_t* __restrict__ w_t,
                                                            int C_out, int KH, int KW, int C_in) {
  const int64_t total = (int64_t)C_in * KH * KW * C_out;
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int co = (int)(i % C_out);
  int64_t r = i / C_out;
  const int kw = (int)(r % KW);
  r /= KW;
  const int kh = (int)(r % KH);
  const int ci = (int)(r / KH);
  w_t[i] = w[(((int64_t)co * KH + (KH - 1 - kh)) * KW + (KW - 1 - kw)) * C_in + ci];
}

cudaError_t launch_dgrad_weights(const void* w, void* w_t, int C_out, int KH, int KW, int C_in, cudaStream_t st) {
  const int64_t total = (int64_t)C_in * KH * KW * C_out;
  dgrad_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>((const uint16_t*)w, (uint16_t*)w_t, C_out, KH,
                                                                        KW, C_in);
  count_launch();
  return cudaGetLastError();
}

// For a stride above 1 the same holds once dL/dy is spread out: dyz[n][ho sh][wo sw][:] = dy[n][ho][wo][:],
// zeros elsewhere, with extents Hz = H + 2 pad - dil (KH - 1) (at least sh (Ho - 1) + 1: input rows past the
// last filter placement get their zero gradient from the zero rows at the end).  One thread per 16 bytes
// of dyz; HBM-bound on the write.
__global__ void __launch_bounds__(256) dgrad_spread_kernel(const uint4* __restrict__ dy, uint4* __restrict__ dyz,
                                                           long long total, int Ho, int Wo, int C8, int Hz, int Wz,
                                                           int sh, int sw) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int c = (int)(i % C8);
  long long r = i / C8;
  const int wz = (int)(r % Wz);
  r /= Wz;
  const int hz = (int)(r % Hz);
  const long long n = r / Hz;
  const int ho = hz / sh, wo = wz / sw;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (ho * sh == hz && wo * sw == wz && ho < Ho && wo < Wo) v = __ldg(dy + ((n * Ho + ho) * Wo + wo) * C8 + c);
  dyz[i] = v;
}

cudaError_t launch_dgrad_spread(const void* dy, void* dyz, int N, int Ho, int Wo, int C, int Hz, int Wz, int sh, int sw,
                                cudaStream_t st) {
  const long long total = (long long)N * Hz * Wz * (C / 8);
  if (total == 0) return cudaSuccess;
  dgrad_spread_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>((const uint4*)dy, (uint4*)dyz, total, Ho, Wo,
                                                                       C / 8, Hz, Wz, sh, sw);
  count_launch();
  return cudaGetLastError();
}

// Strided layers without the zeros: the input pixels fall into stride_h x stride_w residue classes of
// their padded position, (h + pad) mod s = a.  A pixel of class a only ever met the filter taps
// kh = a, a + s, a + 2 s, ... (J_a of them), at the outputs ho = i - j for kh = a + j s, i = (h + pad) / s:
//   dx[h] = sum_j dy[i - j] w[a + j s],
// a unit-stride convolution of dy with J_a x J_b taps per class (all classes together have the layer's
// KH x KW taps, where the zero-spread form multiplies KH x KW taps at every input pixel).  As a
// cross-correlation with padding J - 1 its output row t is i = t.  This kernel writes the weights of one
// class, w_c[ci][u_h][u_w][co] = w[co][a + (J_a - 1 - u_h) s_h][b + (J_b - 1 - u_w) s_w][ci].
__global__ void __launch_bounds__(256) dgrad_class_weights_kernel(const uint16_t* __restrict__ w, uint16_t* __restrict__ w_c,
                                                                  int C_out, int KH, int KW, int C_in, int a, int b,
                                                                  int Ja, int Jb, int sh, int sw) {
  const int64_t total = (int64_t)C_in * Ja * Jb * C_out;
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int co = (int)(i % C_out);
  int64_t r = i / C_out;
  const int uw = (int)(r % Jb);
  r /= Jb;
  const int uh = (int)(r % Ja);
  const int ci = (int)(r / Ja);
  const int kh = a + (Ja - 1 - uh) * sh, kw = b + (Jb - 1 - uw) * sw;
  w_c[i] = w[(((int64_t)co * KH + kh) * KW + kw) * C_in + ci];
}

// All classes in one convolution: the classes' output channels side by side (class k = a s_w + b holds
// channels [k C_in, (k + 1) C_in)), every class on the common window of Jh x Jw = ceil(KH / s_h) x
// ceil(KW / s_w) taps with zeros where its own taps end:
//   w_all[k C_in + ci][u_h][u_w][co] = w[co][a + (Jh - 1 - u_h) s_h][b + (Jw - 1 - u_w) s_w][ci]  (0 past KH, KW).
// One launch instead of s_h s_w small ones; the zero taps cost multiply-adds (16 tap-classes for the 9
// taps of a 3x3 stride-2 layer, against 36 for the zero-spread form).
__global__ void __launch_bounds__(256) dgrad_fused_weights_kernel(const uint16_t* __restrict__ w, uint16_t* __restrict__ w_all,
                                                                  int C_out, int KH, int KW, int C_in, int Jh, int Jw,
                                                                  int sh, int sw) {
  // A block transposes one 32 (ci) x 32 (co) tile of one (class, tap): reads run along ci, writes along co.
  __shared__ uint16_t tile[32][33];
  int z = blockIdx.z;
  const int uw = z % Jw;
  z /= Jw;
  const int uh = z % Jh;
  const int k = z / Jh;
  const int a = k / sw, b = k - a * sw;
  const int kh = a + (Jh - 1 - uh) * sh, kw = b + (Jw - 1 - uw) * sw;
  const bool tap = kh < KH && kw < KW;
  const int ci0 = blockIdx.x * 32, co0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
#pragma unroll
  for (int r = ty; r < 32; r += 8) {
    const int co = co0 + r, ci = ci0 + tx;
    tile[r][tx] = (tap && co < C_out && ci < C_in) ? w[(((int64_t)co * KH + kh) * KW + kw) * C_in + ci] : (uint16_t)0;
  }
  __syncthreads();
#pragma unroll
  for (int r = ty; r < 32; r += 8) {
    const int ci = ci0 + r, co = co0 + tx;
    if (ci < C_in && co < C_out)
      w_all[((((int64_t)k * C_in + ci) * Jh + uh) * Jw + uw) * C_out + co] = tile[tx][r];
  }
}

cudaError_t launch_dgrad_fused_weights(const void* w, void* w_all, int C_out, int KH, int KW, int C_in, int Jh, int Jw,
                                       int sh, int sw, cudaStream_t st) {
  if (C_in == 0 || C_out == 0) return cudaSuccess;
  const dim3 grid((unsigned)((C_in + 31) / 32), (unsigned)((C_out + 31) / 32), (unsigned)(sh * sw * Jh * Jw));
  dgrad_fused_weights_kernel<<<grid, 256, 0, st>>>((const uint16_t*)w, (uint16_t*)w_all, C_out, KH, KW, C_in, Jh, Jw, sh,
                                                   sw);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_dgrad_class_weights(const void* w, void* w_c, int C_out, int KH, int KW, int C_in, int a, int b,
                                       int Ja, int Jb, int sh, int sw, cudaStream_t st) {
  const int64_t total = (int64_t)C_in * Ja * Jb * C_out;
  if (total == 0) return cudaSuccess;
  dgrad_class_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>((const uint16_t*)w, (uint16_t*)w_c, C_out,
                                                                              KH, KW, C_in, a, b, Ja, Jb, sh, sw);
  count_launch();
  return cudaGetLastError();
}

// dx[n, h, w, :] = T_class[n, (h + pad_h) / s_h, (w + pad_w) / s_w, :] with class = the residues of the
// padded position; zero for a class without taps and beyond a class tensor's extent (no filter placement
// reaches those pixels).  `pitch8` = 16-byte units between pixels of a class tensor (C_in / 8, or the
// channels of all classes when they share one tensor).  One thread per 16 bytes of dx.
__global__ void __launch_bounds__(256) dgrad_gather_kernel(DgradClasses cls, uint4* __restrict__ dx, long long total, int H,
                                                           int W, int C8, int pitch8, int sh, int sw, int ph, int pw) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int c = (int)(i % C8);
  long long r = i / C8;
  const int w = (int)(r % W);
  r /= W;
  const int h = (int)(r % H);
  const long long n = r / H;
  const int hp = h + ph, wp = w + pw;
  const int ih = hp / sh, iw = wp / sw;
  const int k = (hp - ih * sh) * sw + (wp - iw * sw);
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  const uint4* t = static_cast<const uint4*>(cls.t[k]);
  if (t != nullptr && ih < cls.rows[k] && iw < cls.cols[k])
    v = __ldg(t + ((n * cls.rows[k] + ih) * cls.cols[k] + iw) * pitch8 + c);
  dx[i] = v;
}

cudaError_t launch_dgrad_gather(const DgradClasses& cls, void* dx, int N, int H, int W, int C, int pitch, int sh, int sw,
                                int ph, int pw, cudaStream_t st) {
  const long long total = (long long)N * H * W * (C / 8);
  if (total == 0) return cudaSuccess;
  dgrad_gather_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(cls, (uint4*)dx, total, H, W, C / 8, pitch / 8, sh,
                                                                       sw, ph, pw);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_soft_mask(const float* logits, const float* noise, float tau, const void* w, int64_t G, float* z,
                             void* w_eff, cudaStream_t st) {
  const int threads = 256;
  const int64_t blocks = (G + threads - 1) / threads;
  soft_mask_kernel<<<(unsigned)blocks, threads, 0, st>>>(logits, noise, 1.0f / tau, (const uint2*)w, G, z,
                                                         (uint2*)w_eff);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_mask_grad(const float* z, float tau, const void* w, const float* g_w_eff, int64_t G,
                             float* g_logits, cudaStream_t st) {
  const int threads = 256;
  const int64_t blocks = (G + threads - 1) / threads;
  mask_grad_kernel<<<(unsigned)blocks, threads, 0, st>>>(z, 1.0f / tau, (const uint2*)w, (const float4*)g_w_eff, G,
                                                         g_logits);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssconv
