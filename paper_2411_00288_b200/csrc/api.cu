// extern "C" boundary: argument validation and dispatch to the launchers.  Nothing here
// touches device memory, synchronises or allocates.
#include <cuda_runtime.h>

#include "layout.cuh"
#include "ssconv.h"

namespace ssconv {
cudaError_t launch_select(int mode, const void* scores, int64_t G, uint8_t* pattern, cudaStream_t st);
cudaError_t launch_compress(const ssconv_desc_t& d, const void* w, const uint8_t* pattern, void* w_comp, void* meta,
                            cudaStream_t st);
cudaError_t launch_decompress(const ssconv_desc_t& d, const void* w_comp, const void* meta, void* w_out,
                              uint8_t* pattern_out, cudaStream_t st);
int32_t launch_forward_sparse(const ssconv_desc_t& d, const void* x, const void* w_comp, const void* meta,
                              const float* bias, const void* residual, void* y, void* ws, size_t ws_bytes,
                              int32_t* dev_status, cudaStream_t stream);
int32_t launch_forward_dense(const ssconv_desc_t& d, const void* x, const void* w, const float* bias,
                             const void* residual, void* y, void* ws, size_t ws_bytes, int32_t* dev_status,
                             cudaStream_t stream, const int64_t* x_strides = nullptr);
cudaError_t launch_space_to_depth(const void* x, void* y, int N, int H, int W, int C, int s, int pad, int Hb, int Wb,
                                  int C_pad, cudaStream_t st);
int32_t plan_query_sms(const ssconv_desc_t& d, bool sparse, int sm_count, int32_t* bn, int32_t* split, int32_t* ctas,
                       int32_t* ring_groups, int32_t* pair);
cudaError_t launch_wait_timeout_selftest(long long limit_cycles, int32_t* dev_status, cudaStream_t st);
int32_t launch_forward_fp8(const ssconv_desc_t& d, bool sparse, const void* x, const void* weights, const void* meta,
                           const float* bias, float out_scale, void* y, int32_t* dev_status, cudaStream_t stream);
cudaError_t launch_quantize_e4m3(const void* x, void* y, int64_t n, float scale, cudaStream_t st);
cudaError_t launch_compress_e4m3(const ssconv_desc_t& d, const void* w, const uint8_t* pattern, void* w_comp, void* meta,
                                 cudaStream_t st);
cudaError_t launch_decompress_e4m3(const ssconv_desc_t& d, const void* w_comp, const void* meta, void* w_out,
                                   uint8_t* pattern_out, cudaStream_t st);
int nm_pattern_count(int N, int M);
cudaError_t launch_nm_select(int mode, const void* scores, int64_t G, int N, int M, uint8_t* pattern, cudaStream_t st);
cudaError_t launch_nm_apply(const void* w, const uint8_t* pattern, int64_t G, int N, int M, void* w_masked,
                            cudaStream_t st);
int32_t launch_forward_grouped(const ssconv_desc_t& d, int groups, bool sparse, const void* x, const void* weights,
                               const void* meta, const float* bias, void* y, void* ws, size_t ws_bytes,
                               int32_t* dev_status, cudaStream_t stream);
cudaError_t launch_depthwise(const void* x, const void* w, const float* bias, void* y, int N, int H, int W, int C, int Ho,
                             int Wo, int KH, int KW, int stride, int pad, int dil, uint32_t flags, cudaStream_t st);
cudaError_t launch_layernorm(const void* x, const float* gamma, const float* beta, void* y, long long pixels, int C,
                             float eps, cudaStream_t st);
size_t workspace_bytes();
int32_t set_tuning(int32_t option, int32_t value);
cudaError_t launch_maxpool(const void* x, void* y, int N, int H, int W, int C, int k, int stride, int pad,
                           cudaStream_t st);
cudaError_t launch_pad_channels(const void* x, void* y, long long pixels, int C, int C_pad, cudaStream_t st);
cudaError_t launch_fold_weights(const void* w, void* out, int C_out, int KH, int KW, int KWf, int s, int d, int f,
                                long long tap_bytes, const float* bias, float* bias_out, cudaStream_t st);
cudaError_t launch_unfold_w(const void* x, void* y, long long rows, int W, int C, int KW, int stride, int pad, int dil,
                            int C_pad, cudaStream_t st);
int32_t plan_query(const ssconv_desc_t& d, bool sparse, int32_t* bn, int32_t* split, int32_t* ctas,
                   int32_t* ring_groups, int32_t* pair);
int32_t launch_forward_static_ws(const ssconv_desc_t& d, const void* x, const void* w_comp, const void* meta,
                                 const float* bias, void* y, int32_t* dev_status, cudaStream_t stream);
cudaError_t launch_soft_mask(const float* logits, const float* noise, float tau, const void* w, int64_t G, float* z,
                             void* w_eff, cudaStream_t st);
cudaError_t launch_dgrad_weights(const void* w, void* w_t, int C_out, int KH, int KW, int C_in, cudaStream_t st);
cudaError_t launch_dgrad_class_weights(const void* w, void* w_c, int C_out, int KH, int KW, int C_in, int a, int b,
                                       int Ja, int Jb, int sh, int sw, cudaStream_t st);
cudaError_t launch_dgrad_gather(const DgradClasses& cls, void* dx, int N, int H, int W, int C, int pitch, int sh, int sw,
                                int ph, int pw, cudaStream_t st);
cudaError_t launch_dgrad_fused_weights(const void* w, void* w_all, int C_out, int KH, int KW, int C_in, int Jh, int Jw,
                                       int sh, int sw, cudaStream_t st);
cudaError_t launch_mask_grad(const float* z, float tau, const void* w, const float* g_w_eff, int64_t G,
                             float* g_logits, cudaStream_t st);
cudaError_t launch_adamw(float* theta, const float* g, float* m, float* v, int64_t n, float lr, float beta1,
                         float beta2, float eps, float wd, float c1, float c2, cudaStream_t st);
cudaError_t launch_mask_norms(const void* w, const uint8_t* pattern, int C_out, int64_t K, float* out, cudaStream_t st);
cudaError_t launch_absmax(const void* x, int64_t n, float* out, cudaStream_t st);
cudaError_t launch_dgrad_weights(const void* w, void* w_t, int C_out, int KH, int KW, int C_in, cudaStream_t st);
cudaError_t launch_dgrad_spread(const void* dy, void* dyz, int N, int Ho, int Wo, int C, int Hz, int Wz, int sh, int sw,
                                cudaStream_t st);
int32_t launch_wgrad(const ssconv_desc_t& d, const void* x, const void* dy, float* dw, void* ws, size_t ws_bytes,
                     int32_t* dev_status, cudaStream_t stream);
int32_t wgrad_workspace_bytes(const ssconv_desc_t& d, size_t* bytes);
}  // namespace ssconv

#include <atomic>
#include <cmath>
namespace ssconv {
static std::atomic<unsigned long long> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
}  // namespace ssconv

namespace {

using ssconv::Geometry;
using ssconv::make_geometry;

int out_extent(int in, int k, int stride, int pad, int dil) {
  long long span = (long long)in + 2LL * pad - (long long)dil * (k - 1) - 1;
  return span < 0 ? 0 : (int)(span / stride + 1);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks every shape rule both forward kernels share; `sparse` adds the 2:4 ones.
int32_t check_desc(const ssconv_desc_t* d, bool need_tma_shape) {
  if (!d) return SSCONV_ERR_NULL;
  if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->C_in <= 0 || d->C_out <= 0 || d->KH <= 0 || d->KW <= 0)
    return SSCONV_ERR_BAD_DESC;
  if (d->stride_h <= 0 || d->stride_w <= 0 || d->dil_h <= 0 || d->dil_w <= 0 || d->pad_h < 0 || d->pad_w < 0)
    return SSCONV_ERR_BAD_DESC;
  if (d->flags & ~(SSCONV_FLAG_BIAS | SSCONV_FLAG_RELU | SSCONV_FLAG_GELU)) return SSCONV_ERR_BAD_DESC;
  if ((d->flags & SSCONV_FLAG_RELU) && (d->flags & SSCONV_FLAG_GELU)) return SSCONV_ERR_BAD_DESC;  // one activation
  int Ho = out_extent(d->H, d->KH, d->stride_h, d->pad_h, d->dil_h);
  int Wo = out_extent(d->W, d->KW, d->stride_w, d->pad_w, d->dil_w);
  if (Ho <= 0 || Wo <= 0) return SSCONV_ERR_BAD_DESC;
  if ((long long)d->N * Ho * Wo > 0x7FFFFF00LL) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if ((long long)d->C_out * d->KH * d->KW * d->C_in > 0x7FFFFFFFLL) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (need_tma_shape) {
    if (d->C_in % 8 != 0 || d->C_out % 8 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
    if (d->pad_h > 127 || d->pad_w > 127) return SSCONV_ERR_UNSUPPORTED_SHAPE;
    if ((d->KH - 1) * d->dil_h > 255 || (d->KW - 1) * d->dil_w > 255) return SSCONV_ERR_UNSUPPORTED_SHAPE;
    // lower corner -pad and upper corner pad - (K-1)*dil of the filter-placement box are 8-bit fields
    if (d->pad_h - (d->KH - 1) * d->dil_h < -128 || d->pad_w - (d->KW - 1) * d->dil_w < -128)
      return SSCONV_ERR_UNSUPPORTED_SHAPE;
    if (d->stride_h > 8 || d->stride_w > 8) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  }
  return SSCONV_OK;
}

}  // namespace

extern "C" {

int32_t ssconv_version(void) { return 100; }

uint64_t ssconv_launch_count(void) { return ssconv::g_launches.load(std::memory_order_relaxed); }

const char* ssconv_status_string(int32_t status) {
  switch (status) {
    case SSCONV_OK: return "ok";
    case SSCONV_ERR_NULL: return "null pointer";
    case SSCONV_ERR_BAD_DESC: return "bad descriptor";
    case SSCONV_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case SSCONV_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case SSCONV_ERR_WORKSPACE: return "workspace missing or too small";
    case SSCONV_ERR_ARCH: return "device is not sm_100";
    case SSCONV_ERR_CUDA: return "CUDA call or launch failed";
    case SSCONV_ERR_TIMEOUT: return "kernel wait timed out";
    default: return "unknown status";
  }
}

int32_t ssconv_out_shape(const ssconv_desc_t* desc, int32_t* H_out, int32_t* W_out) {
  if (!desc || !H_out || !W_out) return SSCONV_ERR_NULL;
  int32_t rc = check_desc(desc, false);
  if (rc != SSCONV_OK) return rc;
  *H_out = out_extent(desc->H, desc->KH, desc->stride_h, desc->pad_h, desc->dil_h);
  *W_out = out_extent(desc->W, desc->KW, desc->stride_w, desc->pad_w, desc->dil_w);
  return SSCONV_OK;
}

int32_t ssconv_sizes(const ssconv_desc_t* desc, int64_t* G, size_t* w_comp_bytes, size_t* meta_bytes,
                     size_t* ws_bytes_sparse, size_t* ws_bytes_dense) {
  int32_t rc = check_desc(desc, false);
  if (rc != SSCONV_OK) return rc;
  if (desc->C_in % 4 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  Geometry geo = make_geometry(*desc);
  if (G) *G = (int64_t)desc->C_out * geo.taps * (desc->C_in / 4);
  if (w_comp_bytes) *w_comp_bytes = (size_t)geo.Mp * geo.KC * 2;
  if (meta_bytes) *meta_bytes = (size_t)geo.m_tiles * geo.stages * ssconv::kMetaImageBytes;
  if (ws_bytes_sparse) *ws_bytes_sparse = ssconv::workspace_bytes();
  if (ws_bytes_dense) *ws_bytes_dense = ssconv::workspace_bytes();
  return SSCONV_OK;
}

int32_t ssconv_plan(const ssconv_desc_t* desc, int32_t sparse, int32_t* tile_positions, int32_t* split,
                    int32_t* ctas, int32_t* ring_groups, int32_t* pair) {
  int32_t st = check_desc(desc, true);
  if (st != SSCONV_OK) return st;
  return ssconv::plan_query(*desc, sparse != 0, tile_positions, split, ctas, ring_groups, pair);
}

int32_t ssconv_plan_for_sms(const ssconv_desc_t* desc, int32_t sparse, int32_t sm_count, int32_t* tile_positions,
                            int32_t* split, int32_t* ctas, int32_t* ring_groups, int32_t* pair) {
  int32_t st = check_desc(desc, true);
  if (st != SSCONV_OK) return st;
  return ssconv::plan_query_sms(*desc, sparse != 0, sm_count, tile_positions, split, ctas, ring_groups, pair);
}

int32_t ssconv_window_extent(int32_t in, int32_t k, int32_t stride, int32_t pad, int32_t dil) {
  if (in <= 0 || k <= 0 || stride <= 0 || pad < 0 || dil <= 0) return 0;
  return out_extent(in, k, stride, pad, dil);
}

int32_t ssconv_selftest_wait_timeout(int64_t limit_cycles, int32_t* dev_status, void* stream) {
  if (!dev_status) return SSCONV_ERR_NULL;
  if (limit_cycles < 1000 || limit_cycles > 2000000000LL) return SSCONV_ERR_BAD_DESC;
  return ssconv::launch_wait_timeout_selftest(limit_cycles, dev_status, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_tune(int32_t option, int32_t value) { return ssconv::set_tuning(option, value); }

int32_t ssconv_select_mask(int32_t mode, const void* scores, int64_t G, uint8_t* pattern, void* stream) {
  if (mode != SSCONV_MASK_LOGITS_F32 && mode != SSCONV_MASK_MAGNITUDE_BF16 && mode != SSCONV_MASK_MAGNITUDE_E4M3)
    return SSCONV_ERR_BAD_DESC;
  if (G < 0) return SSCONV_ERR_BAD_DESC;
  if (G == 0) return SSCONV_OK;
  if (!scores || !pattern) return SSCONV_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(scores) & (mode == SSCONV_MASK_MAGNITUDE_E4M3 ? 3u : 7u)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_select(mode, scores, G, pattern, (cudaStream_t)stream) == cudaSuccess ? SSCONV_OK
                                                                                              : SSCONV_ERR_CUDA;
}

int32_t ssconv_nm_patterns(int32_t N, int32_t M) { return ssconv::nm_pattern_count(N, M); }

int32_t ssconv_select_mask_nm(int32_t mode, const void* scores, int64_t G, int32_t N, int32_t M, uint8_t* pattern,
                              void* stream) {
  if (mode != SSCONV_MASK_LOGITS_F32 && mode != SSCONV_MASK_MAGNITUDE_BF16) return SSCONV_ERR_BAD_DESC;
  if (G < 0 || ssconv::nm_pattern_count(N, M) == 0) return SSCONV_ERR_BAD_DESC;
  if (G == 0) return SSCONV_OK;
  if (!scores || !pattern) return SSCONV_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(scores) & (mode == SSCONV_MASK_LOGITS_F32 ? 3u : 1u)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_nm_select(mode, scores, G, N, M, pattern, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_apply_mask_nm(const void* w_bf16, const uint8_t* pattern, int64_t G, int32_t N, int32_t M,
                             void* w_masked_bf16, void* stream) {
  if (G < 0 || ssconv::nm_pattern_count(N, M) == 0) return SSCONV_ERR_BAD_DESC;
  if (G == 0) return SSCONV_OK;
  if (!w_bf16 || !pattern || !w_masked_bf16) return SSCONV_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(w_bf16) | reinterpret_cast<uintptr_t>(w_masked_bf16)) & 1u) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_nm_apply(w_bf16, pattern, G, N, M, w_masked_bf16, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_compress(const ssconv_desc_t* desc, const void* w_bf16, const uint8_t* pattern, void* w_comp,
                        void* meta, void* stream) {
  int32_t rc = check_desc(desc, false);
  if (rc != SSCONV_OK) return rc;
  if (desc->C_in % 8 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (!w_bf16 || !pattern || !w_comp || !meta) return SSCONV_ERR_NULL;
  if (!aligned16(w_bf16) || !aligned16(w_comp) || !aligned16(meta)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_compress(*desc, w_bf16, pattern, w_comp, meta, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_decompress(const ssconv_desc_t* desc, const void* w_comp, const void* meta, void* w_masked_bf16,
                          uint8_t* pattern_out, void* stream) {
  int32_t rc = check_desc(desc, false);
  if (rc != SSCONV_OK) return rc;
  if (desc->C_in % 8 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (!w_comp || !meta || !w_masked_bf16) return SSCONV_ERR_NULL;
  if (!aligned16(w_comp) || !aligned16(meta) || !aligned16(w_masked_bf16)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_decompress(*desc, w_comp, meta, w_masked_bf16, pattern_out, (cudaStream_t)stream) ==
                 cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_maxpool(const void* x, void* y, int32_t N, int32_t H, int32_t W, int32_t C, int32_t k, int32_t stride,
                       int32_t pad, void* stream) {
  if (!x || !y) return SSCONV_ERR_NULL;
  if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || k <= 0 || stride <= 0 || pad < 0) return SSCONV_ERR_BAD_DESC;
  if (2 * pad >= 2 * k || H + 2 * pad < k || W + 2 * pad < k) return SSCONV_ERR_BAD_DESC;  // every window meets the image
  if (C % 8 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(x) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  if ((long long)N * H * W * C > 0x7FFFFFFFFFLL) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  return ssconv::launch_maxpool(x, y, N, H, W, C, k, stride, pad, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_pad_channels(const void* x, void* y, int64_t pixels, int32_t C, int32_t C_pad, void* stream) {
  if (!x || !y) return SSCONV_ERR_NULL;
  if (pixels <= 0 || C <= 0 || C_pad < C) return SSCONV_ERR_BAD_DESC;
  if (C_pad % 8 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x) & 1u) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  if (pixels > 0x7FFFFFFFFFLL / C_pad) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  return ssconv::launch_pad_channels(x, y, pixels, C, C_pad, (cudaStream_t)stream) == cudaSuccess ? SSCONV_OK
                                                                                                  : SSCONV_ERR_CUDA;
}

int32_t ssconv_unfold_w(const void* x, void* y, int64_t rows, int32_t W, int32_t C, int32_t KW, int32_t stride_w,
                        int32_t pad_w, int32_t dil_w, int32_t C_pad, void* stream) {
  if (!x || !y) return SSCONV_ERR_NULL;
  if (rows <= 0 || W <= 0 || C <= 0 || KW <= 0 || stride_w <= 0 || dil_w <= 0 || pad_w < 0) return SSCONV_ERR_BAD_DESC;
  if (C % 8 != 0 || C_pad % 8 != 0 || (long long)KW * C > C_pad) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if ((long long)W + 2LL * pad_w - (long long)dil_w * (KW - 1) - 1 < 0) return SSCONV_ERR_BAD_DESC;
  if (!aligned16(x) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  if (rows > 0x7FFFFFFFLL) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  return ssconv::launch_unfold_w(x, y, rows, W, C, KW, stride_w, pad_w, dil_w, C_pad, (cudaStream_t)stream) ==
                 cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_forward(const ssconv_desc_t* desc, const void* x, const void* w_comp, const void* meta,
                       const float* bias, void* y, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream) {
  int32_t rc = check_desc(desc, true);
  if (rc != SSCONV_OK) return rc;
  if (!x || !w_comp || !meta || !y) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_comp) || !aligned16(meta) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_forward_sparse(*desc, x, w_comp, meta, bias, nullptr, y, ws, ws_bytes, dev_status,
                                       (cudaStream_t)stream);
}

int32_t ssconv_forward_res(const ssconv_desc_t* desc, const void* x, const void* w_comp, const void* meta,
                           const float* bias, const void* residual, void* y, void* ws, size_t ws_bytes,
                           int32_t* dev_status, void* stream) {
  int32_t rc = check_desc(desc, true);
  if (rc != SSCONV_OK) return rc;
  if (!x || !w_comp || !meta || !y || !residual) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_comp) || !aligned16(meta) || !aligned16(y) || !aligned16(residual))
    return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_forward_sparse(*desc, x, w_comp, meta, bias, residual, y, ws, ws_bytes, dev_status,
                                       (cudaStream_t)stream);
}


int32_t ssconv_forward_dense(const ssconv_desc_t* desc, const void* x, const void* w_bf16, const float* bias,
                             void* y, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream) {
  int32_t rc = check_desc(desc, true);
  if (rc != SSCONV_OK) return rc;
  if (!x || !w_bf16 || !y) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_bf16) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_forward_dense(*desc, x, w_bf16, bias, nullptr, y, ws, ws_bytes, dev_status,
                                      (cudaStream_t)stream);
}

int32_t ssconv_forward_dense_strided(const ssconv_desc_t* desc, const void* x, int64_t stride_w, int64_t stride_h,
                                     int64_t stride_n, const void* w_bf16, const float* bias, void* y, void* ws,
                                     size_t ws_bytes, int32_t* dev_status, void* stream) {
  int32_t rc = check_desc(desc, true);
  if (rc != SSCONV_OK) return rc;
  if (!x || !w_bf16 || !y) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_bf16) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  if (desc->C_in == 8) return SSCONV_ERR_UNSUPPORTED_SHAPE;  // the 8-channel mode reads packed pixels
  // tensor-map strides are multiples of 16 bytes below 2^40
  if (stride_w <= 0 || stride_h <= 0 || stride_n <= 0 || stride_w % 8 || stride_h % 8 || stride_n % 8)
    return SSCONV_ERR_BAD_DESC;
  if (stride_n >= (1LL << 38) || stride_h >= (1LL << 38) || stride_w >= (1LL << 38)) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  const int64_t strides[3] = {stride_w, stride_h, stride_n};
  return ssconv::launch_forward_dense(*desc, x, w_bf16, bias, nullptr, y, ws, ws_bytes, dev_status,
                                      (cudaStream_t)stream, strides);
}

int32_t ssconv_space_to_depth(const void* x, void* y, int32_t N, int32_t H, int32_t W, int32_t C, int32_t block,
                              int32_t pad, int32_t Hb, int32_t Wb, int32_t C_pad, void* stream) {
  if (!x || !y) return SSCONV_ERR_NULL;
  if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || block <= 0 || pad < 0 || Hb <= 0 || Wb <= 0) return SSCONV_ERR_BAD_DESC;
  if (C_pad % 4 != 0 || (long long)block * block * C > C_pad) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x) & 1u) || (reinterpret_cast<uintptr_t>(y) & (C_pad % 8 == 0 ? 15u : 7u)))
    return SSCONV_ERR_ALIGNMENT;
  if ((long long)N * Hb > 0x7FFFFFFFLL || (long long)Wb * C_pad > 0x7FFFFFFFLL) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if ((long long)Wb * (C_pad / 4) > 65535LL * 256) return SSCONV_ERR_UNSUPPORTED_SHAPE;  // grid limit along a row
  return ssconv::launch_space_to_depth(x, y, N, H, W, C, block, pad, Hb, Wb, C_pad, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

// ---- folding of neighbouring output pixels into the output channels
static int32_t fold_geometry(const ssconv_desc_t* d, int32_t f, int* KWf, int* Wo) {
  if (!d) return SSCONV_ERR_NULL;
  if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->C_in <= 0 || d->C_out <= 0 || d->KH <= 0 || d->KW <= 0 ||
      d->stride_w <= 0 || d->stride_h <= 0 || d->dil_w <= 0 || d->dil_h <= 0 || d->pad_w < 0 || d->pad_h < 0)
    return SSCONV_ERR_BAD_DESC;
  if (f < 1 || f > 16) return SSCONV_ERR_BAD_DESC;
  const long long span = (long long)d->W + 2LL * d->pad_w - (long long)d->dil_w * (d->KW - 1) - 1;
  if (span < 0) return SSCONV_ERR_BAD_DESC;
  *Wo = (int)(span / d->stride_w) + 1;
  if (*Wo % f != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  const long long kwf = (long long)(f - 1) * d->stride_w + (long long)(d->KW - 1) * d->dil_w + 1;
  if (kwf > 0x7FFF || (long long)f * d->C_out > 0x7FFFFFFFLL || (long long)f * d->stride_w > 0x7FFF)
    return SSCONV_ERR_UNSUPPORTED_SHAPE;
  *KWf = (int)kwf;
  return SSCONV_OK;
}

int32_t ssconv_fold_desc(const ssconv_desc_t* desc, int32_t f, ssconv_desc_t* folded) {
  if (!folded) return SSCONV_ERR_NULL;
  int KWf = 0, Wo = 0;
  const int32_t rc = fold_geometry(desc, f, &KWf, &Wo);
  if (rc != SSCONV_OK) return rc;
  *folded = *desc;
  folded->C_out = desc->C_out * f;
  folded->KW = KWf;
  folded->stride_w = desc->stride_w * f;
  folded->dil_w = 1;
  return SSCONV_OK;
}

int32_t ssconv_fold_factor(const ssconv_desc_t* desc) {
  int KWf = 0, Wo = 0;
  if (fold_geometry(desc, 2, &KWf, &Wo) != SSCONV_OK) return 1;
  // Tiles have 128 accumulator rows whatever C_out is: with two pixels per row block the multiply-adds
  // issued per output change by KW' / (2 KW); worth it from 15 % on.
  if (desc->C_out > 64 || desc->C_out % 8 != 0) return 1;
  return (20LL * KWf <= 17LL * 2 * desc->KW) ? 2 : 1;
}

int32_t ssconv_fold_weights(const ssconv_desc_t* desc, int32_t f, const void* w, void* w_folded, int64_t tap_bytes,
                            const float* bias, float* bias_folded, void* stream) {
  int KWf = 0, Wo = 0;
  const int32_t rc = fold_geometry(desc, f, &KWf, &Wo);
  if (rc != SSCONV_OK) return rc;
  if ((w == nullptr) != (w_folded == nullptr) || (bias == nullptr) != (bias_folded == nullptr)) return SSCONV_ERR_NULL;
  if (w != nullptr && (tap_bytes <= 0 || tap_bytes > 0x7FFFFFFFLL)) return SSCONV_ERR_BAD_DESC;
  if ((long long)f * desc->C_out * desc->KH * KWf > (0x7FFFFFFFLL * 256) / (tap_bytes > 0 ? tap_bytes : 1))
    return SSCONV_ERR_UNSUPPORTED_SHAPE;
  return ssconv::launch_fold_weights(w, w_folded, desc->C_out, desc->KH, desc->KW, KWf, desc->stride_w, desc->dil_w, f,
                                     tap_bytes, bias, bias_folded, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

// Shape rules of the 8-bit entry points on top of check_desc: rows of 16 bytes for the copies.
static int32_t check_fp8(const ssconv_desc_t* desc, float out_scale) {
  int32_t rc = check_desc(desc, true);
  if (rc != SSCONV_OK) return rc;
  if (desc->C_in % 16 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (!(out_scale > 0.0f) || !(out_scale < 3.0e38f)) return SSCONV_ERR_BAD_DESC;
  return SSCONV_OK;
}

// ---- grouped convolutions
static int32_t check_groups(const ssconv_desc_t* desc, int32_t groups, ssconv_desc_t* sub) {
  int32_t rc = check_desc(desc, true);
  if (rc != SSCONV_OK) return rc;
  if (groups < 1 || desc->C_in % groups != 0 || desc->C_out % groups != 0) return SSCONV_ERR_BAD_DESC;
  *sub = *desc;
  sub->C_in = desc->C_in / groups;
  sub->C_out = desc->C_out / groups;
  if (sub->C_in % 8 != 0 || sub->C_out % 8 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;  // (one channel per group: ssconv_depthwise)
  return SSCONV_OK;
}

int32_t ssconv_sizes_grouped(const ssconv_desc_t* desc, int32_t groups, int64_t* G, size_t* w_comp_bytes,
                             size_t* meta_bytes) {
  ssconv_desc_t sub;
  int32_t rc = check_groups(desc, groups, &sub);
  if (rc != SSCONV_OK) return rc;
  int64_t g1 = 0;
  size_t a = 0, b = 0;
  rc = ssconv_sizes(&sub, &g1, &a, &b, nullptr, nullptr);
  if (rc != SSCONV_OK) return rc;
  if (G) *G = g1 * groups;
  if (w_comp_bytes) *w_comp_bytes = a * groups;
  if (meta_bytes) *meta_bytes = b * groups;
  return SSCONV_OK;
}

int32_t ssconv_compress_grouped(const ssconv_desc_t* desc, int32_t groups, const void* w_bf16, const uint8_t* pattern,
                                void* w_comp, void* meta, void* stream) {
  ssconv_desc_t sub;
  int32_t rc = check_groups(desc, groups, &sub);
  if (rc != SSCONV_OK) return rc;
  int64_t g1 = 0;
  size_t a = 0, b = 0;
  rc = ssconv_sizes(&sub, &g1, &a, &b, nullptr, nullptr);
  if (rc != SSCONV_OK) return rc;
  if (!w_bf16 || !pattern || !w_comp || !meta) return SSCONV_ERR_NULL;
  if (!aligned16(w_bf16) || !aligned16(w_comp) || !aligned16(meta)) return SSCONV_ERR_ALIGNMENT;
  const size_t w_step = (size_t)sub.C_out * sub.KH * sub.KW * sub.C_in * 2;
  for (int32_t i = 0; i < groups; ++i) {
    rc = ssconv_compress(&sub, static_cast<const char*>(w_bf16) + i * w_step, pattern + (size_t)i * g1,
                         static_cast<char*>(w_comp) + i * a, static_cast<char*>(meta) + i * b, stream);
    if (rc != SSCONV_OK) return rc;
  }
  return SSCONV_OK;
}

int32_t ssconv_forward_grouped(const ssconv_desc_t* desc, int32_t groups, const void* x, const void* w_comp,
                               const void* meta, const float* bias, void* y, void* ws, size_t ws_bytes,
                               int32_t* dev_status, void* stream) {
  ssconv_desc_t sub;
  int32_t rc = check_groups(desc, groups, &sub);
  if (rc != SSCONV_OK) return rc;
  if (!x || !w_comp || !meta || !y) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_comp) || !aligned16(meta) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_forward_grouped(*desc, groups, true, x, w_comp, meta, bias, y, ws, ws_bytes, dev_status,
                                        (cudaStream_t)stream);
}

int32_t ssconv_forward_dense_grouped(const ssconv_desc_t* desc, int32_t groups, const void* x, const void* w_bf16,
                                     const float* bias, void* y, void* ws, size_t ws_bytes, int32_t* dev_status,
                                     void* stream) {
  ssconv_desc_t sub;
  int32_t rc = check_groups(desc, groups, &sub);
  if (rc != SSCONV_OK) return rc;
  if (!x || !w_bf16 || !y) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_bf16) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_forward_grouped(*desc, groups, false, x, w_bf16, nullptr, bias, y, ws, ws_bytes, dev_status,
                                        (cudaStream_t)stream);
}

int32_t ssconv_depthwise(const ssconv_desc_t* desc, const void* x, const void* w_bf16, const float* bias, void* y,
                         void* stream) {
  int32_t rc = check_desc(desc, false);
  if (rc != SSCONV_OK) return rc;
  if (desc->C_in != desc->C_out) return SSCONV_ERR_BAD_DESC;
  if (desc->C_in % 8 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (desc->flags & SSCONV_FLAG_GELU) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (!x || !w_bf16 || !y) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_bf16) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  const int Ho = out_extent(desc->H, desc->KH, desc->stride_h, desc->pad_h, desc->dil_h);
  const int Wo = out_extent(desc->W, desc->KW, desc->stride_w, desc->pad_w, desc->dil_w);
  if (desc->stride_h != desc->stride_w || desc->pad_h != desc->pad_w || desc->dil_h != desc->dil_w)
    return SSCONV_ERR_UNSUPPORTED_SHAPE;
  return ssconv::launch_depthwise(x, w_bf16, bias, y, desc->N, desc->H, desc->W, desc->C_in, Ho, Wo, desc->KH, desc->KW,
                                  desc->stride_h, desc->pad_h, desc->dil_h, desc->flags, (cudaStream_t)stream) ==
                 cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_layernorm(const void* x_bf16, const float* gamma, const float* beta, float eps, void* y_bf16,
                         int64_t pixels, int32_t C, void* stream) {
  if (pixels < 0 || C <= 0 || !(eps >= 0.0f)) return SSCONV_ERR_BAD_DESC;
  if (pixels == 0) return SSCONV_OK;
  if (!x_bf16 || !gamma || !beta || !y_bf16) return SSCONV_ERR_NULL;
  if (pixels > 0x3FFFFFFLL * 8) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  return ssconv::launch_layernorm(x_bf16, gamma, beta, y_bf16, pixels, C, eps, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_quantize_e4m3(const void* x_bf16, void* y_e4m3, int64_t n, float scale, void* stream) {
  if (n < 0 || n % 2 != 0 || !(scale > 0.0f) || !(scale < 3.0e38f)) return SSCONV_ERR_BAD_DESC;
  if (n == 0) return SSCONV_OK;
  if (!x_bf16 || !y_e4m3) return SSCONV_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(x_bf16) & 3u) || (reinterpret_cast<uintptr_t>(y_e4m3) & 1u)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_quantize_e4m3(x_bf16, y_e4m3, n, scale, (cudaStream_t)stream) == cudaSuccess ? SSCONV_OK
                                                                                                      : SSCONV_ERR_CUDA;
}

int32_t ssconv_sizes_fp8(const ssconv_desc_t* desc, int64_t* G, size_t* w_comp_bytes, size_t* meta_bytes) {
  int32_t rc = check_desc(desc, false);
  if (rc != SSCONV_OK) return rc;
  if (desc->C_in % 16 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  Geometry geo = make_geometry(*desc, 128);
  if (G) *G = (int64_t)desc->C_out * geo.taps * (desc->C_in / 4);
  if (w_comp_bytes) *w_comp_bytes = (size_t)geo.Mp * geo.kblocks_pad * 64;
  if (meta_bytes) *meta_bytes = (size_t)geo.m_tiles * geo.stages * 2 * ssconv::kMetaImageBytes;
  return SSCONV_OK;
}

int32_t ssconv_compress_fp8(const ssconv_desc_t* desc, const void* w_e4m3, const uint8_t* pattern, void* w_comp,
                            void* meta, void* stream) {
  int32_t rc = check_desc(desc, false);
  if (rc != SSCONV_OK) return rc;
  if (desc->C_in % 16 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (!w_e4m3 || !pattern || !w_comp || !meta) return SSCONV_ERR_NULL;
  if (!aligned16(w_e4m3) || !aligned16(w_comp) || !aligned16(meta)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_compress_e4m3(*desc, w_e4m3, pattern, w_comp, meta, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_decompress_fp8(const ssconv_desc_t* desc, const void* w_comp, const void* meta, void* w_masked_e4m3,
                              uint8_t* pattern_out, void* stream) {
  int32_t rc = check_desc(desc, false);
  if (rc != SSCONV_OK) return rc;
  if (desc->C_in % 16 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (!w_comp || !meta || !w_masked_e4m3) return SSCONV_ERR_NULL;
  if (!aligned16(w_comp) || !aligned16(meta) || !aligned16(w_masked_e4m3)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_decompress_e4m3(*desc, w_comp, meta, w_masked_e4m3, pattern_out, (cudaStream_t)stream) ==
                 cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_forward_fp8(const ssconv_desc_t* desc, const void* x_e4m3, const void* w_comp, const void* meta,
                           const float* bias, float out_scale, void* y, int32_t* dev_status, void* stream) {
  int32_t rc = check_fp8(desc, out_scale);
  if (rc != SSCONV_OK) return rc;
  if (!x_e4m3 || !w_comp || !meta || !y) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x_e4m3) || !aligned16(w_comp) || !aligned16(meta) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_forward_fp8(*desc, true, x_e4m3, w_comp, meta, bias, out_scale, y, dev_status,
                                    (cudaStream_t)stream);
}

int32_t ssconv_forward_dense_fp8(const ssconv_desc_t* desc, const void* x_e4m3, const void* w_e4m3, const float* bias,
                                 float out_scale, void* y, int32_t* dev_status, void* stream) {
  int32_t rc = check_fp8(desc, out_scale);
  if (rc != SSCONV_OK) return rc;
  if (!x_e4m3 || !w_e4m3 || !y) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x_e4m3) || !aligned16(w_e4m3) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_forward_fp8(*desc, false, x_e4m3, w_e4m3, nullptr, bias, out_scale, y, dev_status,
                                    (cudaStream_t)stream);
}

int32_t ssconv_forward_dense_res(const ssconv_desc_t* desc, const void* x, const void* w_bf16, const float* bias,
                                 const void* residual, void* y, void* ws, size_t ws_bytes, int32_t* dev_status,
                                 void* stream) {
  int32_t rc = check_desc(desc, true);
  if (rc != SSCONV_OK) return rc;
  if (!x || !w_bf16 || !y || !residual) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_bf16) || !aligned16(y) || !aligned16(residual)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_forward_dense(*desc, x, w_bf16, bias, residual, y, ws, ws_bytes, dev_status,
                                      (cudaStream_t)stream);
}

int32_t ssconv_soft_mask(const float* logits, const float* noise, float tau, const void* w_bf16, int64_t G, float* z,
                         void* w_eff_bf16, void* stream) {
  if (G < 0 || !(tau > 0.0f)) return SSCONV_ERR_BAD_DESC;
  if (G == 0) return SSCONV_OK;
  if (!logits || (w_eff_bf16 && !w_bf16) || (!z && !w_eff_bf16)) return SSCONV_ERR_NULL;
  const uintptr_t all = reinterpret_cast<uintptr_t>(logits) | reinterpret_cast<uintptr_t>(noise) |
                        reinterpret_cast<uintptr_t>(w_bf16) | reinterpret_cast<uintptr_t>(z) |
                        reinterpret_cast<uintptr_t>(w_eff_bf16);
  if (all & 7u) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_soft_mask(logits, noise, tau, w_bf16, G, z, w_eff_bf16, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_mask_grad(const float* z, float tau, const void* w_bf16, const float* g_w_eff, int64_t G,
                         float* g_logits, void* stream) {
  if (G < 0 || !(tau > 0.0f)) return SSCONV_ERR_BAD_DESC;
  if (G == 0) return SSCONV_OK;
  if (!z || !w_bf16 || !g_w_eff || !g_logits) return SSCONV_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(z) | reinterpret_cast<uintptr_t>(w_bf16) | reinterpret_cast<uintptr_t>(g_logits)) & 7u)
    return SSCONV_ERR_ALIGNMENT;
  if (!aligned16(g_w_eff)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_mask_grad(z, tau, w_bf16, g_w_eff, G, g_logits, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_adamw(float* theta, const float* g, float* m, float* v, int64_t n, int32_t step, float lr, float beta1,
                     float beta2, float eps, float weight_decay, void* stream) {
  if (n < 0 || step < 1) return SSCONV_ERR_BAD_DESC;
  if (!(beta1 >= 0.0f && beta1 < 1.0f && beta2 >= 0.0f && beta2 < 1.0f) || !(eps >= 0.0f)) return SSCONV_ERR_BAD_DESC;
  if (n == 0) return SSCONV_OK;
  if (!theta || !g || !m || !v) return SSCONV_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(theta) | reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(m) |
       reinterpret_cast<uintptr_t>(v)) & 15u)
    return SSCONV_ERR_ALIGNMENT;
  const double c1 = 1.0 / (1.0 - std::pow((double)beta1, (double)step));
  const double c2 = 1.0 / (1.0 - std::pow((double)beta2, (double)step));
  return ssconv::launch_adamw(theta, g, m, v, n, lr, beta1, beta2, eps, weight_decay, (float)c1, (float)c2,
                              (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_mask_norms(const void* w_bf16, const uint8_t* pattern, int32_t C_out, int64_t K, float* out3,
                          void* stream) {
  if (C_out <= 0 || K <= 0) return SSCONV_ERR_BAD_DESC;
  if (K % 4 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  if (!w_bf16 || !pattern || !out3) return SSCONV_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(w_bf16) & 7u) || (reinterpret_cast<uintptr_t>(out3) & 3u)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_mask_norms(w_bf16, pattern, C_out, K, out3, (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_absmax(const void* x_bf16, int64_t n, float* out, void* stream) {
  if (n < 0) return SSCONV_ERR_BAD_DESC;
  if (!out || (n > 0 && !x_bf16)) return SSCONV_ERR_NULL;
  if (!aligned16(x_bf16) || (reinterpret_cast<uintptr_t>(out) & 3u)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_absmax(x_bf16, n, out, (cudaStream_t)stream) == cudaSuccess ? SSCONV_OK : SSCONV_ERR_CUDA;
}

double ssconv_stability_threshold(int32_t lemma, double L, const double* layer_norms, int32_t depth, int32_t j,
                                  double extra_norm, double x_norm) {
  if (!layer_norms || depth <= 0 || j < 0 || j >= depth) return -1.0;
  if (lemma != SSCONV_LEMMA_PERTURBATION && lemma != SSCONV_LEMMA_ANY_MASK && lemma != SSCONV_LEMMA_MASKED_UPDATE)
    return -1.0;
  double others = 1.0;
  for (int32_t i = 0; i < depth; ++i)
    if (i != j) others *= layer_norms[i];
  const double lip = std::pow(L, (double)depth);
  const double own = lemma == SSCONV_LEMMA_PERTURBATION   ? extra_norm
                     : lemma == SSCONV_LEMMA_ANY_MASK     ? layer_norms[j]
                                                          : layer_norms[j] + extra_norm;
  return lip * own * x_norm * others;
}

int32_t ssconv_dgrad_spread(const ssconv_desc_t* desc, const void* dy, void* dy_spread, void* stream) {
  ssconv_desc_t d;
  if (desc) {
    d = *desc;
    d.flags = 0;
  }
  int32_t rc = check_desc(desc ? &d : nullptr, true);
  if (rc != SSCONV_OK) return rc;
  if (!dy || !dy_spread) return SSCONV_ERR_NULL;
  if (!aligned16(dy) || !aligned16(dy_spread)) return SSCONV_ERR_ALIGNMENT;
  const int Hz = d.H + 2 * d.pad_h - d.dil_h * (d.KH - 1), Wz = d.W + 2 * d.pad_w - d.dil_w * (d.KW - 1);
  const int Ho = out_extent(d.H, d.KH, d.stride_h, d.pad_h, d.dil_h);
  const int Wo = out_extent(d.W, d.KW, d.stride_w, d.pad_w, d.dil_w);
  return ssconv::launch_dgrad_spread(dy, dy_spread, d.N, Ho, Wo, d.C_out, Hz, Wz, d.stride_h, d.stride_w,
                                     (cudaStream_t)stream) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_dgrad_prepare(const ssconv_desc_t* desc, const void* w_bf16, void* w_t_bf16, ssconv_desc_t* desc_dx,
                             void* stream) {
  ssconv_desc_t d;
  if (desc) {
    d = *desc;
    d.flags = 0;
  }
  int32_t rc = check_desc(desc ? &d : nullptr, true);
  if (rc != SSCONV_OK) return rc;
  if (!desc_dx) return SSCONV_ERR_NULL;
  const int pad_h = d.dil_h * (d.KH - 1) - d.pad_h, pad_w = d.dil_w * (d.KW - 1) - d.pad_w;
  if (pad_h < 0 || pad_w < 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;  // padding wider than the filter's reach
  ssconv_desc_t t = d;
  // Extents of the (spread) gradient: all filter placements at unit stride.  With unit stride this is
  // the layer's own output extent.
  t.H = d.H + 2 * d.pad_h - d.dil_h * (d.KH - 1);
  t.W = d.W + 2 * d.pad_w - d.dil_w * (d.KW - 1);
  t.stride_h = t.stride_w = 1;
  t.C_in = d.C_out;
  t.C_out = d.C_in;
  t.pad_h = pad_h;
  t.pad_w = pad_w;
  t.flags = 0;
  rc = check_desc(&t, true);
  if (rc != SSCONV_OK) return rc;
  *desc_dx = t;
  if (w_bf16 == nullptr && w_t_bf16 == nullptr) return SSCONV_OK;  // descriptor only
  if (!w_bf16 || !w_t_bf16) return SSCONV_ERR_NULL;
  if (!aligned16(w_bf16) || !aligned16(w_t_bf16)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_dgrad_weights(w_bf16, w_t_bf16, d.C_out, d.KH, d.KW, d.C_in, (cudaStream_t)stream) ==
                 cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

// ---- input gradient in one call
namespace {
struct DgradPlan {
  bool strided;
  bool spread;                      // strided with a dilation, or a stride above 4: zero-spread dy, one convolution
  int Hz, Wz;                       // extents of the spread gradient
  size_t spread_off;
  int classes;                      // stride_h * stride_w
  int Ja[4], Jb[4];                 // taps per residue of the padded row / column
  int Ho, Wo;
  bool fused;                       // all classes in one convolution (three or more of them have taps)
  int Jh, Jw;                       // its window: ceil(KH / s_h) x ceil(KW / s_w)
  size_t w_off[ssconv::kMaxDgradClasses], t_off[ssconv::kMaxDgradClasses];
  size_t fwd_off, fwd_bytes;        // scratch of the convolution(s) themselves (K split)
  size_t bytes;
};
size_t round256(size_t v) { return (v + 255) & ~size_t(255); }

// Shape rules and workspace layout: per class its weights [C_in, Ja, Jb, C_out] and its tensor
// [N, Ho + Ja - 1, Wo + Jb - 1, C_in]; with unit stride only the reversed weights.
int32_t dgrad_plan(const ssconv_desc_t& d, DgradPlan* p) {
  if (d.C_out % 8 != 0) return SSCONV_ERR_UNSUPPORTED_SHAPE;  // dy's channels are the convolutions' input channels
  if (d.dil_h * (d.KH - 1) < d.pad_h || d.dil_w * (d.KW - 1) < d.pad_w) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  p->strided = d.stride_h > 1 || d.stride_w > 1;
  p->Ho = (d.H + 2 * d.pad_h - d.dil_h * (d.KH - 1) - 1) / d.stride_h + 1;
  p->Wo = (d.W + 2 * d.pad_w - d.dil_w * (d.KW - 1) - 1) / d.stride_w + 1;
  const size_t w_bytes = (size_t)d.C_in * d.KH * d.KW * d.C_out * 2;
  p->fwd_bytes = ssconv::workspace_bytes();
  p->spread = false;
  if (!p->strided) {
    p->classes = 1;
    p->fwd_off = round256(w_bytes);
    p->bytes = p->fwd_off + p->fwd_bytes;
    return SSCONV_OK;
  }
  p->spread = d.dil_h != 1 || d.dil_w != 1 || d.stride_h > 4 || d.stride_w > 4;
  if (p->spread) {
    // The residue classes are built for undilated filters and strides up to 4.  The rest (rare shapes) take
    // the plain route: dy spread out by the stride with zeros in between, then the unit-stride convolution
    // with the reversed filter; its multiplications by the zeros are the price.
    p->classes = 1;
    p->Hz = d.H + 2 * d.pad_h - d.dil_h * (d.KH - 1);
    p->Wz = d.W + 2 * d.pad_w - d.dil_w * (d.KW - 1);
    p->spread_off = round256(w_bytes);
    p->fwd_off = p->spread_off + round256((size_t)d.N * p->Hz * p->Wz * d.C_out * 2);
    p->bytes = p->fwd_off + p->fwd_bytes;
    return SSCONV_OK;
  }
  p->classes = d.stride_h * d.stride_w;
  for (int a = 0; a < d.stride_h; ++a) p->Ja[a] = a < d.KH ? (d.KH - 1 - a) / d.stride_h + 1 : 0;
  for (int b = 0; b < d.stride_w; ++b) p->Jb[b] = b < d.KW ? (d.KW - 1 - b) / d.stride_w + 1 : 0;
  int with_taps = 0;
  for (int a = 0; a < d.stride_h; ++a)
    for (int b = 0; b < d.stride_w; ++b) with_taps += (p->Ja[a] > 0 && p->Jb[b] > 0) ? 1 : 0;
  p->Jh = (d.KH + d.stride_h - 1) / d.stride_h;
  p->Jw = (d.KW + d.stride_w - 1) / d.stride_w;
  p->fused = with_taps >= 3;
  if (p->fused) {  // weights [classes C_in, Jh, Jw, C_out], tensor [N, Ho + Jh - 1, Wo + Jw - 1, classes C_in]
    p->w_off[0] = 0;
    p->t_off[0] = round256((size_t)p->classes * d.C_in * p->Jh * p->Jw * d.C_out * 2);
    p->fwd_off = p->t_off[0] + round256((size_t)d.N * (p->Ho + p->Jh - 1) * (p->Wo + p->Jw - 1) * p->classes * d.C_in * 2);
    p->bytes = p->fwd_off + p->fwd_bytes;
    return SSCONV_OK;
  }
  size_t off = 0;
  for (int a = 0; a < d.stride_h; ++a)
    for (int b = 0; b < d.stride_w; ++b) {
      const int k = a * d.stride_w + b;
      const int Ja = p->Ja[a], Jb = p->Jb[b];
      p->w_off[k] = off;
      off += round256((size_t)d.C_in * Ja * Jb * d.C_out * 2);
      p->t_off[k] = off;
      if (Ja > 0 && Jb > 0) off += round256((size_t)d.N * (p->Ho + Ja - 1) * (p->Wo + Jb - 1) * d.C_in * 2);
    }
  p->fwd_off = off;
  p->bytes = off + p->fwd_bytes;
  return SSCONV_OK;
}
}  // namespace

int32_t ssconv_dgrad_ws_bytes(const ssconv_desc_t* desc, size_t* bytes) {
  if (!bytes) return SSCONV_ERR_NULL;
  ssconv_desc_t d;
  if (desc) {
    d = *desc;
    d.flags = 0;
  }
  int32_t rc = check_desc(desc ? &d : nullptr, true);
  if (rc != SSCONV_OK) return rc;
  DgradPlan p;
  rc = dgrad_plan(d, &p);
  if (rc != SSCONV_OK) return rc;
  *bytes = p.bytes;
  return SSCONV_OK;
}

int32_t ssconv_dgrad(const ssconv_desc_t* desc, const void* dy, const void* w_bf16, void* dx, void* ws, size_t ws_bytes,
                     int32_t* dev_status, void* stream) {
  ssconv_desc_t d;
  if (desc) {
    d = *desc;
    d.flags = 0;
  }
  int32_t rc = check_desc(desc ? &d : nullptr, true);
  if (rc != SSCONV_OK) return rc;
  if (!dy || !w_bf16 || !dx) return SSCONV_ERR_NULL;
  if (!aligned16(dy) || !aligned16(w_bf16) || !aligned16(dx) || !aligned16(ws)) return SSCONV_ERR_ALIGNMENT;
  DgradPlan p;
  rc = dgrad_plan(d, &p);
  if (rc != SSCONV_OK) return rc;
  if (ws == nullptr || ws_bytes < p.bytes) return SSCONV_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* base = static_cast<uint8_t*>(ws);
  ssconv_desc_t c = d;  // the convolution(s) of dy: channels exchanged, unit stride
  c.H = p.Ho;
  c.W = p.Wo;
  c.C_in = d.C_out;
  c.C_out = d.C_in;
  c.stride_h = c.stride_w = 1;
  c.dil_h = d.dil_h;
  c.dil_w = d.dil_w;
  c.flags = 0;
  if (!p.strided) {
    c.pad_h = d.dil_h * (d.KH - 1) - d.pad_h;
    c.pad_w = d.dil_w * (d.KW - 1) - d.pad_w;
    rc = check_desc(&c, true);
    if (rc != SSCONV_OK) return rc;
    // (the reversed, channel-exchanged filter = the one class of a unit stride, written by the tiled transpose)
    if (ssconv::launch_dgrad_fused_weights(w_bf16, base, d.C_out, d.KH, d.KW, d.C_in, d.KH, d.KW, 1, 1, st) != cudaSuccess)
      return SSCONV_ERR_CUDA;
    return ssconv::launch_forward_dense(c, dy, base, nullptr, nullptr, dx, base + p.fwd_off, p.fwd_bytes, dev_status, st);
  }
  if (p.spread) {
    c.H = p.Hz;
    c.W = p.Wz;
    c.pad_h = d.dil_h * (d.KH - 1) - d.pad_h;
    c.pad_w = d.dil_w * (d.KW - 1) - d.pad_w;
    rc = check_desc(&c, true);
    if (rc != SSCONV_OK) return rc;
    if (ssconv::launch_dgrad_fused_weights(w_bf16, base, d.C_out, d.KH, d.KW, d.C_in, d.KH, d.KW, 1, 1, st) != cudaSuccess)
      return SSCONV_ERR_CUDA;
    if (ssconv::launch_dgrad_spread(dy, base + p.spread_off, d.N, p.Ho, p.Wo, d.C_out, p.Hz, p.Wz, d.stride_h, d.stride_w,
                                    st) != cudaSuccess)
      return SSCONV_ERR_CUDA;
    return ssconv::launch_forward_dense(c, base + p.spread_off, base, nullptr, nullptr, dx, base + p.fwd_off, p.fwd_bytes,
                                        dev_status, st);
  }
  ssconv::DgradClasses cls;
  for (int k = 0; k < ssconv::kMaxDgradClasses; ++k) {
    cls.t[k] = nullptr;
    cls.rows[k] = cls.cols[k] = 0;
  }
  if (p.fused) {
    c.KH = p.Jh;
    c.KW = p.Jw;
    c.pad_h = p.Jh - 1;
    c.pad_w = p.Jw - 1;
    c.C_out = p.classes * d.C_in;
    rc = check_desc(&c, true);
    if (rc != SSCONV_OK) return rc;
    if (ssconv::launch_dgrad_fused_weights(w_bf16, base, d.C_out, d.KH, d.KW, d.C_in, p.Jh, p.Jw, d.stride_h, d.stride_w,
                                           st) != cudaSuccess)
      return SSCONV_ERR_CUDA;
    rc = ssconv::launch_forward_dense(c, dy, base, nullptr, nullptr, base + p.t_off[0], base + p.fwd_off, p.fwd_bytes,
                                      dev_status, st);
    if (rc != SSCONV_OK) return rc;
    for (int k = 0; k < p.classes; ++k) {
      cls.t[k] = base + p.t_off[0] + (size_t)k * d.C_in * 2;
      cls.rows[k] = p.Ho + p.Jh - 1;
      cls.cols[k] = p.Wo + p.Jw - 1;
    }
    return ssconv::launch_dgrad_gather(cls, dx, d.N, d.H, d.W, d.C_in, p.classes * d.C_in, d.stride_h, d.stride_w,
                                       d.pad_h, d.pad_w, st) == cudaSuccess
               ? SSCONV_OK
               : SSCONV_ERR_CUDA;
  }
  for (int a = 0; a < d.stride_h; ++a)
    for (int b = 0; b < d.stride_w; ++b) {
      const int k = a * d.stride_w + b;
      const int Ja = p.Ja[a], Jb = p.Jb[b];
      if (Ja == 0 || Jb == 0) continue;
      c.KH = Ja;
      c.KW = Jb;
      c.pad_h = Ja - 1;
      c.pad_w = Jb - 1;
      rc = check_desc(&c, true);
      if (rc != SSCONV_OK) return rc;
      if (ssconv::launch_dgrad_class_weights(w_bf16, base + p.w_off[k], d.C_out, d.KH, d.KW, d.C_in, a, b, Ja, Jb,
                                             d.stride_h, d.stride_w, st) != cudaSuccess)
        return SSCONV_ERR_CUDA;
      rc = ssconv::launch_forward_dense(c, dy, base + p.w_off[k], nullptr, nullptr, base + p.t_off[k], base + p.fwd_off,
                                        p.fwd_bytes, dev_status, st);
      if (rc != SSCONV_OK) return rc;
      cls.t[k] = base + p.t_off[k];
      cls.rows[k] = p.Ho + Ja - 1;
      cls.cols[k] = p.Wo + Jb - 1;
    }
  return ssconv::launch_dgrad_gather(cls, dx, d.N, d.H, d.W, d.C_in, d.C_in, d.stride_h, d.stride_w, d.pad_h, d.pad_w,
                                     st) == cudaSuccess
             ? SSCONV_OK
             : SSCONV_ERR_CUDA;
}

int32_t ssconv_wgrad_ws_bytes(const ssconv_desc_t* desc, size_t* bytes) {
  if (!bytes) return SSCONV_ERR_NULL;
  ssconv_desc_t d;
  if (desc) {
    d = *desc;
    d.flags = 0;
  }
  int32_t rc = check_desc(desc ? &d : nullptr, true);
  if (rc != SSCONV_OK) return rc;
  return ssconv::wgrad_workspace_bytes(d, bytes);
}

int32_t ssconv_wgrad(const ssconv_desc_t* desc, const void* x, const void* dy, float* dw, void* ws, size_t ws_bytes,
                     int32_t* dev_status, void* stream) {
  ssconv_desc_t d;
  if (desc) {
    d = *desc;
    d.flags = 0;  // bias and activation play no part in this gradient
  }
  int32_t rc = check_desc(desc ? &d : nullptr, true);
  if (rc != SSCONV_OK) return rc;
  if (!x || !dy || !dw) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(dy) || !aligned16(dw) || !aligned16(ws)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_wgrad(d, x, dy, dw, ws, ws_bytes, dev_status, (cudaStream_t)stream);
}

int32_t ssconv_forward_static_ws(const ssconv_desc_t* desc, const void* x, const void* w_comp, const void* meta,
                                 const float* bias, void* y, int32_t* dev_status, void* stream) {
  int32_t rc = check_desc(desc, true);
  if (rc != SSCONV_OK) return rc;
  if (!x || !w_comp || !meta || !y) return SSCONV_ERR_NULL;
  if ((desc->flags & SSCONV_FLAG_BIAS) && !bias) return SSCONV_ERR_NULL;
  if (!aligned16(x) || !aligned16(w_comp) || !aligned16(meta) || !aligned16(y)) return SSCONV_ERR_ALIGNMENT;
  return ssconv::launch_forward_static_ws(*desc, x, w_comp, meta, bias, y, dev_status, (cudaStream_t)stream);
}

}  // extern "C"
