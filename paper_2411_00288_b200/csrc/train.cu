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
