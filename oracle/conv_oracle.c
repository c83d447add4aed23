/*
 * CPU oracle for the masked convolution (TEST INFRASTRUCTURE, not a product path).
 *
 * Plain fp64 direct convolution written from the definition in the paper:
 *   Eq. 4  (Sec. 3.3): y_ij = sum_c sum_u sum_s H_cus * X_{c, f(i,u), g(j,s)},
 *          where f and g return the index sum, or "padding" (a zero contribution)
 *          when that sum falls outside the input.  An index SUM means the kernel
 *          is not flipped (cross-correlation).
 *   Eq. 6  (Sec. 3.3): Y = (M .* W) U(X): the masked convolution is the dense
 *          convolution of the element-wise masked weights.
 *
 * Inputs are bf16 bit patterns; they are widened exactly to fp64, all products and
 * sums are fp64, the fp32 bias is widened exactly, ReLU is applied in fp64, and the
 * result is NOT rounded.  Loop order is n, ho, wo, co, kh, kw, ci with one scalar
 * accumulator; there is no blocking, fusion or reordering.  OpenMP only distributes
 * whole output pixels over threads (each output element is still one sequential sum).
 *
 * Layouts: x [N,H,W,C_in], w [C_out,KH,KW,C_in], mask [C_out,KH,KW,C_in] (0/1 bytes,
 * may be NULL = all ones), bias [C_out] (may be NULL), y [N,H_out,W_out,C_out].
 *
 * Nothing here is shared with the CUDA library: no header, no helper, no table.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int32_t N, H, W, C_in;
  int32_t C_out, KH, KW;
  int32_t stride_h, stride_w;
  int32_t pad_h, pad_w;
  int32_t dil_h, dil_w;
  int32_t relu;
} oracle_conv_shape;

/* bf16 is the upper half of an IEEE binary32: widening is exact. */
static double bf16_bits_to_f64(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* Output extent of one spatial dimension: the number of filter placements whose
 * top-left tap index ho*stride - pad + (K-1)*dil stays within the padded input.
 * (Sec. 3.3 prints L with garbled signs; its own special case "full padding gives
 * L = b*d" fixes this reading.) */
static int32_t out_extent(int32_t in, int32_t k, int32_t stride, int32_t pad, int32_t dil) {
  int32_t span = in + 2 * pad - dil * (k - 1) - 1;
  if (span < 0) return 0;
  return span / stride + 1;
}

int32_t oracle_out_shape(const oracle_conv_shape* s, int32_t* H_out, int32_t* W_out) {
  *H_out = out_extent(s->H, s->KH, s->stride_h, s->pad_h, s->dil_h);
  *W_out = out_extent(s->W, s->KW, s->stride_w, s->pad_w, s->dil_w);
  return 0;
}

int32_t oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* One output element by Eq. 4 over the masked weights of Eq. 6. */
static double one_output(const oracle_conv_shape* s, const double* xd, const double* wd,
                         const uint8_t* mask, const float* bias,
                         int64_t n, int64_t ho, int64_t wo, int64_t co) {
  double acc = 0.0;
  for (int32_t kh = 0; kh < s->KH; ++kh) {
    int64_t hi = ho * s->stride_h - s->pad_h + (int64_t)kh * s->dil_h;
    for (int32_t kw = 0; kw < s->KW; ++kw) {
      int64_t wi = wo * s->stride_w - s->pad_w + (int64_t)kw * s->dil_w;
      if (hi < 0 || hi >= s->H || wi < 0 || wi >= s->W) continue; /* zero padding */
      const double* xp = xd + ((n * s->H + hi) * s->W + wi) * s->C_in;
      int64_t woff = ((co * s->KH + kh) * s->KW + kw) * (int64_t)s->C_in;
      const double* wp = wd + woff;
      if (mask) {
        const uint8_t* mp = mask + woff;
        for (int32_t ci = 0; ci < s->C_in; ++ci)
          if (mp[ci]) acc += wp[ci] * xp[ci];
      } else {
        for (int32_t ci = 0; ci < s->C_in; ++ci) acc += wp[ci] * xp[ci];
      }
    }
  }
  if (bias) acc += (double)bias[co];
  if (s->relu && acc < 0.0) acc = 0.0;
  return acc;
}

static double* widen(const uint16_t* src, int64_t count) {
  double* d = (double*)malloc(sizeof(double) * (size_t)(count > 0 ? count : 1));
  if (!d) return NULL;
  for (int64_t i = 0; i < count; ++i) d[i] = bf16_bits_to_f64(src[i]);
  return d;
}

/* Full output tensor. Returns 0, or 1 when memory for the widened copies is missing. */
int32_t oracle_conv2d_f64(const oracle_conv_shape* s, const uint16_t* x_bf16,
                          const uint16_t* w_bf16, const uint8_t* mask, const float* bias,
                          double* y) {
  int32_t H_out, W_out;
  oracle_out_shape(s, &H_out, &W_out);
  int64_t nx = (int64_t)s->N * s->H * s->W * s->C_in;
  int64_t nw = (int64_t)s->C_out * s->KH * s->KW * s->C_in;
  double* xd = widen(x_bf16, nx);
  double* wd = widen(w_bf16, nw);
  if (!xd || !wd) { free(xd); free(wd); return 1; }
  int64_t pixels = (int64_t)s->N * H_out * W_out;
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < pixels; ++p) {
    int64_t n = p / ((int64_t)H_out * W_out);
    int64_t r = p % ((int64_t)H_out * W_out);
    int64_t ho = r / W_out, wo = r % W_out;
    for (int64_t co = 0; co < s->C_out; ++co)
      y[p * s->C_out + co] = one_output(s, xd, wd, mask, bias, n, ho, wo, co);
  }
  free(xd);
  free(wd);
  return 0;
}

/* Selected output elements only: idx holds flat indices into y [N,H_out,W_out,C_out].
 * Used where the full tensor would take too long.  It has a loop of its own (the same sum of Eq. 4,
 * term by term in the same order, over bf16 inputs widened on the fly instead of a widened copy of
 * the whole input); a test pins it equal to the full-tensor routine. */
int32_t oracle_conv2d_f64_sample(const oracle_conv_shape* s, const uint16_t* x_bf16,
                                 const uint16_t* w_bf16, const uint8_t* mask,
                                 const float* bias, const int64_t* idx, int64_t n_idx,
                                 double* out) {
  int32_t H_out, W_out;
  oracle_out_shape(s, &H_out, &W_out);
  int64_t nw = (int64_t)s->C_out * s->KH * s->KW * s->C_in;
  double* wd = widen(w_bf16, nw);
  if (!wd) return 1;
  int32_t C_in = s->C_in;
#pragma omp parallel
  {
    /* per-thread scratch for the input pixels one output touches */
    double* xs = (double*)malloc(sizeof(double) * (size_t)C_in);
#pragma omp for schedule(static)
    for (int64_t t = 0; t < n_idx; ++t) {
      int64_t f = idx[t];
      int64_t co = f % s->C_out; f /= s->C_out;
      int64_t wo = f % W_out;    f /= W_out;
      int64_t ho = f % H_out;    f /= H_out;
      int64_t n = f;
      double acc = 0.0;
      for (int32_t kh = 0; kh < s->KH; ++kh) {
        int64_t hi = ho * s->stride_h - s->pad_h + (int64_t)kh * s->dil_h;
        for (int32_t kw = 0; kw < s->KW; ++kw) {
          int64_t wi = wo * s->stride_w - s->pad_w + (int64_t)kw * s->dil_w;
          if (hi < 0 || hi >= s->H || wi < 0 || wi >= s->W) continue;
          const uint16_t* xp = x_bf16 + ((n * s->H + hi) * s->W + wi) * C_in;
          for (int32_t ci = 0; ci < C_in; ++ci) xs[ci] = bf16_bits_to_f64(xp[ci]);
          int64_t woff = ((co * s->KH + kh) * s->KW + kw) * (int64_t)C_in;
          for (int32_t ci = 0; ci < C_in; ++ci)
            if (!mask || mask[woff + ci]) acc += wd[woff + ci] * xs[ci];
        }
      }
      if (bias) acc += (double)bias[co];
      if (s->relu && acc < 0.0) acc = 0.0;
      out[t] = acc;
    }
    free(xs);
  }
  free(wd);
  return 0;
}
