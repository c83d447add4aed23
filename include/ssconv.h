/*
 * ssconv: 2:4 semi-structured sparse convolution for NVIDIA B200 (sm_100a).
 *
 * C ABI of the inference path of "Inducing Semi-Structured Sparsity by Masking for
 * Efficient Model Inference in Convolutional Networks": a convolution whose weight
 * matrix carries a 2:4 mask (Sec. 3.1, Sec. 3.3), executed as an implicit GEMM on the
 * sparse tensor cores.
 *
 * Conventions shared by every entry point
 *  - All tensor pointers are DEVICE pointers owned by the caller; the library keeps
 *    nothing between calls, allocates no device memory and never synchronises.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *    Work is enqueued on it and the call returns immediately.
 *  - Every function returns an ssconv_status_t.  Errors the host can see (null
 *    pointers, bad descriptor, unsupported shape, misalignment, wrong device) are
 *    returned before anything is launched.
 *  - Activations x, y: bf16, NHWC.  Weights: bf16 [C_out, KH, KW, C_in], read as the
 *    row-major matrix W in R^{C_out x K}, K = KH*KW*C_in ordered (kh, kw, c_in)
 *    (Eq. 5).  Bias: fp32 [C_out].
 *  - Group g = ((c_out*KH + kh)*KW + kw)*(C_in/4) + q covers the 4 consecutive input
 *    channels 4q..4q+3 of one filter tap: 4 contiguous entries of a row of W (Eq. 2,
 *    Eq. 6).  `pattern[g]` in 0..5 names the kept pair of positions in lexicographic
 *    order: {0,1},{0,2},{0,3},{1,2},{1,3},{2,3} (the columns of the pattern matrix D).
 */
#ifndef SSCONV_H_
#define SSCONV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SSCONV_OK = 0,
  SSCONV_ERR_NULL = 1,              /* a required pointer is NULL */
  SSCONV_ERR_BAD_DESC = 2,          /* non-positive extent, stride or dilation; negative pad; empty output */
  SSCONV_ERR_UNSUPPORTED_SHAPE = 3, /* shape outside what the kernels cover (see each call) */
  SSCONV_ERR_ALIGNMENT = 4,         /* a tensor pointer is not 16-byte aligned */
  SSCONV_ERR_WORKSPACE = 5,         /* workspace missing or too small */
  SSCONV_ERR_ARCH = 6,              /* current device is not compute capability 10.x */
  SSCONV_ERR_CUDA = 7,              /* a CUDA runtime/driver call or a launch failed */
  SSCONV_ERR_TIMEOUT = 8            /* written to *dev_status by a kernel whose bounded wait ran out */
} ssconv_status_t;

typedef struct {
  int32_t N, H, W, C_in;
  int32_t C_out, KH, KW;
  int32_t stride_h, stride_w;
  int32_t pad_h, pad_w;
  int32_t dil_h, dil_w;
  uint32_t flags; /* SSCONV_FLAG_* */
} ssconv_desc_t;

/* GELU (exact form, x Phi(x)) is not part of the paper's method: it is the activation of the
 * ConvNeXt point-wise layers the paper evaluates on (Sec. 4).  At most one of RELU and GELU. */
enum { SSCONV_FLAG_BIAS = 1u, SSCONV_FLAG_RELU = 2u, SSCONV_FLAG_GELU = 4u };

enum {
  SSCONV_MASK_LOGITS_F32 = 0,    /* scores: float [G,6], one score per pattern            */
  SSCONV_MASK_MAGNITUDE_BF16 = 1,/* scores: bf16 weights [C_out,KH,KW,C_in] = [G,4]       */
  SSCONV_MASK_MAGNITUDE_E4M3 = 2 /* scores: e4m3 weights [C_out,KH,KW,C_in] = [G,4] (bytes; 4-byte aligned) */
};

/* Library version (major*10000 + minor*100 + patch). */
int32_t ssconv_version(void);

/* Number of GPU kernels this library has launched in this process so far (all devices and
 * threads; memsets and copies are not counted).  A diagnostic with no counterpart in the paper:
 * it lets a caller verify that a call ran on the GPU and how many kernels it took (a layer whose
 * K range is split launches two, see ssconv_forward).  Host only, never fails. */
uint64_t ssconv_launch_count(void);

/* Static string for a status code. */
const char* ssconv_status_string(int32_t status);

/* Output extent, H_out = floor((H + 2*pad - dil*(KH-1) - 1)/stride) + 1 (same for W):
 * the count of filter placements of Eq. 4 under zero padding (Sec. 3.3; with
 * pad = floor(k/2), stride 1, this gives H_out*W_out = H*W as the paper states). */
int32_t ssconv_out_shape(const ssconv_desc_t* desc, int32_t* H_out, int32_t* W_out);

/* Sizes for a layer: number of groups G = C_out*K/4, bytes of the compressed value
 * blob and of the metadata blob written by ssconv_compress, and workspace bytes the two
 * forward calls may need.  Any output pointer may be NULL.  The blobs are padded to whole
 * tiles, so they can be slightly larger than C_out*K and C_out*K/8 bytes.  The workspace
 * size is the same for every layer (about 47 MB), so one buffer serves a whole network. */
int32_t ssconv_sizes(const ssconv_desc_t* desc, int64_t* G, size_t* w_comp_bytes,
                     size_t* meta_bytes, size_t* ws_bytes_sparse, size_t* ws_bytes_dense);

/* How ssconv_forward (sparse != 0) or ssconv_forward_dense (sparse == 0) would run this layer on
 * the current device: positions per output tile (the N of the tensor-core instruction, a multiple
 * of 16 up to 240, chosen so that the tiles fill the SMs), whether the K range is split across
 * thread blocks (then a second, finishing kernel runs and ws is used), the number of thread
 * blocks, the depth of the shared-memory ring in pairs of 64-column k-blocks, and whether the layer
 * runs on pairs of thread blocks that share tiles of 256 output channels (layers with more than 128
 * output channels and enough tiles; ctas is then twice the number of pairs).  A tuning aid with no
 * counterpart in the paper; nothing is launched.  Needs a device of compute capability 10.x to be
 * current (SSCONV_ERR_ARCH / SSCONV_ERR_CUDA otherwise).  Any output may be NULL. */
int32_t ssconv_plan(const ssconv_desc_t* desc, int32_t sparse, int32_t* tile_positions, int32_t* split,
                    int32_t* ctas, int32_t* ring_groups, int32_t* pair);

/* Process-wide overrides of the choices ssconv_plan reports, for tuning sweeps and tests (no
 * counterpart in the paper).  SSCONV_TUNE_TILE_POSITIONS: 0 lets the planner choose (default), or a
 * multiple of 16 in [48, 240] that every later forward call uses as its tile width where the layer
 * allows it (calls with a residual are limited to 208 sparse / 160 dense and ignore a wider setting;
 * the pair kernel takes 64 and up).  SSCONV_TUNE_PAIR: -1 lets the planner choose (default), 0 never
 * uses pairs of thread blocks, 1 uses them wherever they apply.  SSCONV_TUNE_WGRAD_RANGES: 0 lets
 * ssconv_wgrad choose into how many position ranges it cuts a layer (default), otherwise an upper limit
 * (ssconv_wgrad_ws_bytes follows).  SSCONV_TUNE_WGRAD_PAIR: as SSCONV_TUNE_PAIR, for ssconv_wgrad.
 * SSCONV_TUNE_RESIDENT_WEIGHTS: 1 (default) keeps the weights of dense layers with one channel tile and
 * at most four k-blocks in shared memory, 0 sends them through the ring like every other layer's.
 * SSCONV_TUNE_PAIR_TILES: -1 lets the planner choose (default) whether a work item of the pair kernel is two
 * neighbouring position tiles that share every group's weights, 0 never, 1 wherever the ring still holds two
 * groups (tiles of at most 192 positions keep three).  Not
 * thread-safe against concurrent calls.  Returns SSCONV_ERR_BAD_DESC for an unknown option or a value
 * out of range. */
enum {
  SSCONV_TUNE_TILE_POSITIONS = 1,
  SSCONV_TUNE_PAIR = 2,
  SSCONV_TUNE_WGRAD_RANGES = 3,
  SSCONV_TUNE_WGRAD_PAIR = 4,
  SSCONV_TUNE_RESIDENT_WEIGHTS = 5,
  SSCONV_TUNE_PAIR_TILES = 6
};
int32_t ssconv_tune(int32_t option, int32_t value);

/* ssconv_plan for a device with `sm_count` SMs, without looking at any device (host arithmetic
 * only; usable where no GPU is present, e.g. to pin the planner's choices in a test). */
int32_t ssconv_plan_for_sms(const ssconv_desc_t* desc, int32_t sparse, int32_t sm_count, int32_t* tile_positions,
                            int32_t* split, int32_t* ctas, int32_t* ring_groups, int32_t* pair);

/* Extent of a sliding window: the number of placements of a window of k taps with the given stride,
 * padding and dilation along an axis of `in` elements, floor((in + 2 pad - dil (k-1) - 1)/stride) + 1
 * (0 if the window does not fit): the output-extent formula of Sec. 3.3 as the library computes it
 * for the convolutions, the max-pool, the width unfold and the spread-out gradient.  Host only. */
int32_t ssconv_window_extent(int32_t in, int32_t k, int32_t stride, int32_t pad, int32_t dil);

/* Self-test of the bounded waits every kernel of this library relies on (no counterpart in the
 * paper): launches a one-block kernel that waits, with a limit of `limit_cycles` SM clock cycles, on
 * an mbarrier nobody ever arrives at.  The wait gives up, the kernel stores SSCONV_ERR_TIMEOUT to
 * *dev_status (device int32, required) exactly as the convolution kernels do, and returns normally,
 * so the context stays usable.  limit_cycles in [1000, 2e9]. */
int32_t ssconv_selftest_wait_timeout(int64_t limit_cycles, int32_t* dev_status, void* stream);

/* Hard pattern choice per group (Eq. 1 of Sec. 3.1 without the one-hot: the index of the
 * winning pattern).
 *   mode LOGITS:    pattern[g] = argmax_i scores[g][i]; the caller has already added any
 *                   Gumbel noise g_i to log pi_i.  Ties: lowest index.  Scores must be
 *                   finite.
 *   mode MAGNITUDE: pattern[g] keeps the two entries of largest |w| of the group (the
 *                   magnitude heuristic of Sec. 2); equal magnitudes: lower position
 *                   first; +0 and -0 are equal.
 * scores: device, 8-byte aligned.  pattern: device uint8 [G].  G >= 0 (0 is a no-op). */
int32_t ssconv_select_mask(int32_t mode, const void* scores, int64_t G, uint8_t* pattern,
                           void* stream);

/* General N:M masks (Sec. 3.1: blocks of M consecutive entries of a row of W of which N are kept;
 * the n = C(M, N) possible blocks are the columns of D in Eq. 2), 1 <= N <= M <= 8.  Patterns are
 * numbered lexicographically in the kept positions (for 2:4 the numbering of ssconv_select_mask).
 * ssconv_nm_patterns returns n (0 for an N, M out of range).  ssconv_select_mask_nm: mode LOGITS takes
 * float scores [G, n] (Eq. 1: first maximum), mode MAGNITUDE_BF16 takes bf16 weights [G, M] and keeps
 * the N largest |w| of each block (equal magnitudes: the lower position).  ssconv_apply_mask_nm writes
 * M .* W (Eq. 6): kept values bit for bit, +0 elsewhere; a pattern index >= n counts as pattern 0.  The
 * sparse tensor-core operation exists for 2:4 only: weights masked with another N:M go through
 * ssconv_forward_dense.  scores / w: device, 4- / 2-byte aligned; pattern: device uint8 [G]. */
int32_t ssconv_nm_patterns(int32_t N, int32_t M);
int32_t ssconv_select_mask_nm(int32_t mode, const void* scores, int64_t G, int32_t N, int32_t M, uint8_t* pattern,
                              void* stream);
int32_t ssconv_apply_mask_nm(const void* w_bf16, const uint8_t* pattern, int64_t G, int32_t N, int32_t M,
                             void* w_masked_bf16, void* stream);

/* Apply the mask (M .* W of Eq. 6) and pack the result in the structured form of Fig. 1:
 * the two kept bf16 values of each group, in ascending position order, bit-exact, plus
 * two 2-bit position indices per group, laid out in the tile order the sparse tensor-core
 * instruction reads.  Needs C_in % 8 == 0 (else SSCONV_ERR_UNSUPPORTED_SHAPE: run such a
 * layer through ssconv_forward_dense).  w_comp / meta: device, 16-byte aligned, of the
 * sizes ssconv_sizes reports; every byte of both blobs is written.  pattern[g] must be in 0..5;
 * the array lives on the device and is not checked: a value outside that range is treated as
 * pattern 0, so the blobs stay well-formed whatever the array holds. */
int32_t ssconv_compress(const ssconv_desc_t* desc, const void* w_bf16, const uint8_t* pattern,
                        void* w_comp, void* meta, void* stream);

/* Inverse of ssconv_compress: w_masked [C_out,KH,KW,C_in] bf16 = M .* W with +0 in the
 * dropped positions; pattern_out (nullable) [G] receives the pattern read back from the
 * metadata. */
int32_t ssconv_decompress(const ssconv_desc_t* desc, const void* w_comp, const void* meta,
                          void* w_masked_bf16, uint8_t* pattern_out, void* stream);

/* Max-pooling of NHWC bf16 activations with a k x k window, given stride and padding (padding
 * never wins): y[n,ho,wo,c] = max over the window of x.  H_out = (H + 2 pad - k)/stride + 1.  Not
 * part of the paper's method: the pooling step between the stem and the first block of the
 * ResNet-shaped convolution stacks the paper evaluates on (Sec. 4), here so that such a stack runs
 * without any other library.  x, y: device, 16-byte aligned; C % 8 == 0; pad < k. */
int32_t ssconv_maxpool(const void* x, void* y, int32_t N, int32_t H, int32_t W, int32_t C, int32_t k,
                       int32_t stride, int32_t pad, void* stream);

/* Channel padding of NHWC bf16 activations: y[p, c] = x[p, c] for c < C and 0 for C <= c < C_pad,
 * for `pixels` pixels.  Not part of the paper's method: the forward entry points want C_in % 8 == 0,
 * and the networks of Sec. 4 start from 3-channel images; the zero channels meet zero-extended
 * weights, so the convolution (Eq. 4) is unchanged.  x: device, 2-byte aligned; y: device, 16-byte
 * aligned; C_pad % 8 == 0, C_pad >= C. */
int32_t ssconv_pad_channels(const void* x, void* y, int64_t pixels, int32_t C, int32_t C_pad, void* stream);

/* Space to depth of NHWC bf16 images: blocks of `block` x `block` pixels of the zero-padded image
 * become the channels of one pixel,
 *   y[n, r, q, (bh*block + bw)*C + c] = x[n, block*r - pad + bh, block*q - pad + bw, c],
 * zero outside the image and in the channels [block*block*C, C_pad); y: bf16 [N, Hb, Wb, C_pad].
 * Not part of the paper's method; it is how a strided convolution over very few channels (the
 * 7x7 stride-2 stem of the ResNets of Sec. 4 on RGB images) reaches the tensor-core path: with
 * T = ceil(K/block), Hb = H_out + T - 1 and Wb = W_out + T - 1, the K x K convolution of stride
 * `block` and padding `pad` over x (Eq. 4) equals a T x T convolution of unit stride and no padding
 * over y, and, reading T neighbouring pixels of y as one pixel of T*C_pad channels through
 * ssconv_forward_dense_strided, a T x 1 convolution.  The weights are rearranged by the same call:
 * [C_out, K, K, C] as C_out "images" with pad 0 and Hb = Wb = T gives [C_out, T, T, C_pad].
 * x: device, 2-byte aligned; y: device, 16-byte aligned (8-byte when C_pad % 8 != 0); C_pad % 4 == 0,
 * C_pad >= block*block*C. */
int32_t ssconv_space_to_depth(const void* x, void* y, int32_t N, int32_t H, int32_t W, int32_t C, int32_t block,
                              int32_t pad, int32_t Hb, int32_t Wb, int32_t C_pad, void* stream);

/* Partial unfold along the width: the unfold U(X) of Eq. 5 restricted to one filter row.  For every
 * row of pixels (rows = N*H of them, each W pixels of C channels, bf16) and every horizontal filter
 * placement wo:
 *   y[row, wo, kw*C + c] = x[row, wo*stride_w - pad_w + kw*dil_w, c],   0 <= kw < KW,
 * zero outside the row and in the padding channels [KW*C, C_pad).  y: bf16 [rows, W_out, C_pad] with
 * W_out = (W + 2 pad_w - dil_w (KW-1) - 1)/stride_w + 1.  A KH x KW convolution over x then equals a
 * KH x 1 convolution over y with horizontal stride 1, no horizontal padding and C_pad input channels,
 * with weights unfolded by the same call (weights [C_out,KH,KW,C] are rows = C_out*KH "pixel rows" of
 * width KW: stride 1, pad 0 gives [C_out,KH,1,C_pad]).  Meant for dense layers with very few input
 * channels (an RGB stem padded to C = 8: KW = 7 gives C_pad = 64), whose 16-byte pixels the
 * convolution kernels load slowly.  x, y: device, 16-byte aligned; C % 8 == 0, C_pad % 8 == 0,
 * C_pad >= KW*C. */
int32_t ssconv_unfold_w(const void* x, void* y, int64_t rows, int32_t W, int32_t C, int32_t KW,
                        int32_t stride_w, int32_t pad_w, int32_t dil_w, int32_t C_pad, void* stream);

/* Masked convolution forward (Eq. 6 with the direct definition Eq. 4):
 *   y[n,ho,wo,co] = act( bias[co] + sum_{kh,kw,ci} x[n, ho*s-p+kh*d, wo*s-p+kw*d, ci]
 *                                                  * (M .* W)[co,kh,kw,ci] ),
 * taps outside the image contribute 0, products are exact, accumulation is fp32, the
 * result is rounded once to bf16 (nearest even).  act = ReLU if SSCONV_FLAG_RELU, GELU if SSCONV_FLAG_GELU, bias is
 * read only if SSCONV_FLAG_BIAS.
 * x, y, w_comp, meta: device, 16-byte aligned.  Needs C_in % 8 == 0, C_out % 8 == 0,
 * pad <= 127, dil*(K-1) <= 255, stride <= 8.
 * ws: device scratch of at least the size ssconv_sizes reports, 16-byte aligned.  It is used
 * only by layers with too few output tiles to fill the GPU, whose K range is then split over
 * several thread blocks that park fp32 partial results there; a second small kernel, launched
 * by the same call, sums them in a fixed order, so results are reproducible.  ws needs no
 * initialisation: every part is written before it is read.  Calls issued one after another on
 * one stream may share it; calls that may overlap on the GPU need separate workspaces.
 * If ws is NULL or too small
 * the K range is never split: such layers then run on whole tiles (correct, slower where a layer has
 * few tiles and a deep K), so a caller without scratch memory can pass ws = NULL for any layer.
 * dev_status (nullable): device int32; a kernel whose bounded wait expires stores
 * SSCONV_ERR_TIMEOUT there and drains instead of hanging; it is never written on success,
 * so the caller zeroes it once and reads it after its own synchronisation. */
int32_t ssconv_forward(const ssconv_desc_t* desc, const void* x, const void* w_comp,
                       const void* meta, const float* bias, void* y, void* ws, size_t ws_bytes,
                       int32_t* dev_status, void* stream);

/* Dense counterpart (Eq. 5, the unmasked reformulation): same formula with the dense
 * weights w_bf16 [C_out,KH,KW,C_in], same tiling and pipeline, dense tensor-core
 * instruction.  Needs C_in % 8 == 0 and C_out % 8 == 0. */
int32_t ssconv_forward_dense(const ssconv_desc_t* desc, const void* x, const void* w_bf16,
                             const float* bias, void* y, void* ws, size_t ws_bytes,
                             int32_t* dev_status, void* stream);

/* Both forward calls with a residual tensor added before the activation:
 *   y = act(bias + conv(x, .) + residual),   residual: bf16 NHWC, the shape of y,
 * the sum taken in fp32 and rounded once.  This is the last convolution of a ResNet bottleneck
 * fused with the block's skip connection (the architectures of Sec. 4); the paper's method itself
 * has no such step.  residual may be y's own buffer only if nothing else reads y concurrently (each
 * element is read before it is written, by the same thread block).  Otherwise as the calls above;
 * residual: device, 16-byte aligned, not NULL. */
int32_t ssconv_forward_res(const ssconv_desc_t* desc, const void* x, const void* w_comp,
                           const void* meta, const float* bias, const void* residual, void* y,
                           void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);
int32_t ssconv_forward_dense_res(const ssconv_desc_t* desc, const void* x, const void* w_bf16,
                                 const float* bias, const void* residual, void* y, void* ws,
                                 size_t ws_bytes, int32_t* dev_status, void* stream);

/* ---- Learning the mask (Sec. 3.1): one training step's kernels for one layer ----------------
 * Only the choice weights (one logit per pattern and group) are trained; the pretrained weights W
 * stay as they are (Sec. 4.1).  A step for one layer is: ssconv_soft_mask -> ssconv_forward_dense
 * with the effective weights -> (the caller's loss and its gradient dL/dy) -> ssconv_wgrad ->
 * ssconv_mask_grad -> ssconv_adamw on the logits; ssconv_dgrad_prepare (+ ssconv_dgrad_spread for a
 * strided layer) + ssconv_forward_dense hand dL/dx to the layer before. */

/* Relaxed choice and soft mask of every group:
 *   z[g][i]   = softmax_i((logits[g][i] + noise[g][i]) / tau)                      (Eq. 3)
 *   b[g][j]   = sum_i D[j][i] z[g][i],   D the 4 x 6 pattern matrix of Eq. 2       (b = D z)
 *   w_eff     = b .* w  (Eq. 6 with the soft mask), rounded once to bf16 (nearest even).
 * logits = log pi up to a constant per group; noise = the caller's Gumbel(0,1) sample per logit
 * (NULL: none); tau > 0.  All arithmetic is fp32.  Pattern order as in ssconv_select_mask.
 * logits, noise, z: device fp32 [G][6], 8-byte aligned; w, w_eff: device bf16 [C_out,KH,KW,C_in]
 * read as G groups of 4, 8-byte aligned.  z (nullable) is kept for ssconv_mask_grad; w_eff
 * (nullable, then w may be NULL too) feeds ssconv_forward_dense.  G >= 0 (0 is a no-op). */
int32_t ssconv_soft_mask(const float* logits, const float* noise, float tau, const void* w_bf16,
                         int64_t G, float* z, void* w_eff_bf16, void* stream);

/* Gradient of the loss with respect to the choice weights, from G = dL/dw_eff (chain rule through
 * Eq. 6, Eq. 2 and Eq. 3; the paper prints no gradient):
 *   dL/db[g][j] = G[g][j] w[g][j],   dL/dz[g][i] = sum_j D[j][i] dL/db[g][j],
 *   g_logits[g][i] = z[g][i] (dL/dz[g][i] - sum_k z[g][k] dL/dz[g][k]) / tau.
 * z: what ssconv_soft_mask stored; g_w_eff: device fp32 [C_out,KH,KW,C_in] (what ssconv_wgrad
 * writes), 16-byte aligned; g_logits: device fp32 [G][6], 8-byte aligned.  fp32 arithmetic. */
int32_t ssconv_mask_grad(const float* z, float tau, const void* w_bf16, const float* g_w_eff,
                         int64_t G, float* g_logits, void* stream);

/* Gradient with respect to a layer's input.  With unit stride, dL/dx is the convolution of dL/dy with
 * the filter taps reversed and input and output channels exchanged,
 *   dx[n,h,w,ci] = sum_{kh,kw,co} dy[n, h + pad - kh*dil, w + pad - kw*dil, co] * w[co,kh,kw,ci]
 * (Eq. 4 differentiated in the input), so it runs on the dense forward kernel.  With a stride s above 1
 * the same sum runs over the gradient spread out with zeros, dyz[n, ho*s, wo*s, :] = dy[n, ho, wo, :],
 * of extents Hz = H + 2 pad - dil (KH - 1) and Wz likewise (ssconv_dgrad_spread below writes it).
 * This call prepares the convolution: it writes w_t [C_in,KH,KW,C_out] bf16 with
 * w_t[ci][KH-1-kh][KW-1-kw][co] = w[co][kh][kw][ci] (for the mask-learning step w is the effective
 * weights of ssconv_soft_mask) and fills *desc_dx with the descriptor of the equivalent convolution
 * (input = dy, or dyz for a strided layer, [N,Hz,Wz,C_out]; output = dx [N,H,W,C_in]; unit stride,
 * padding dil*(K-1) - pad, no bias, no activation).  Then
 *   ssconv_forward_dense(desc_dx, dy or dyz, w_t, NULL, dx, ws, ws_bytes, dev_status, stream)
 * computes dx in bf16.  w_bf16 = w_t_bf16 = NULL fills only the descriptor.  Layers with padding
 * beyond dil*(K-1) return SSCONV_ERR_UNSUPPORTED_SHAPE.  w, w_t: device, 16-byte aligned. */
int32_t ssconv_dgrad_prepare(const ssconv_desc_t* desc, const void* w_bf16, void* w_t_bf16,
                             ssconv_desc_t* desc_dx, void* stream);

/* The output gradient of a strided layer spread out for ssconv_dgrad_prepare's convolution:
 *   dy_spread[n, hz, wz, :] = dy[n, hz / stride_h, wz / stride_w, :] where both divisions are exact and
 *   land inside dy, zero elsewhere;  dy_spread is [N, Hz, Wz, C_out] with Hz = H + 2 pad_h - dil_h (KH - 1),
 *   Wz = W + 2 pad_w - dil_w (KW - 1)  (desc_dx->H and desc_dx->W of ssconv_dgrad_prepare).
 * desc is the layer's own descriptor.  dy: device bf16 [N,H_out,W_out,C_out]; dy_spread: device bf16,
 * caller-owned, every element written; both 16-byte aligned.  With unit stride it is a plain copy and
 * not needed.  Values are moved bit-exactly. */
int32_t ssconv_dgrad_spread(const ssconv_desc_t* desc, const void* dy, void* dy_spread, void* stream);

/* One AdamW update (decoupled weight decay; the optimiser of the Appendix's training details, there
 * with learning rate 1.0, momentum 0.9, weight decay 1e-4) of n fp32 parameters in place:
 *   m <- beta1 m + (1 - beta1) g,   v <- beta2 v + (1 - beta2) g^2,
 *   theta <- theta - lr ( (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps) + weight_decay theta ).
 * step counts from 1.  theta (the logits), g (from ssconv_mask_grad), m, v: device fp32 [n]; m and v
 * start as zeros and belong to the caller; all four 16-byte aligned.  fp32 arithmetic. */
int32_t ssconv_adamw(float* theta, const float* g, float* m, float* v, int64_t n, int32_t step, float lr,
                     float beta1, float beta2, float eps, float weight_decay, void* stream);

/* Weight gradient of the convolution (Eq. 4 differentiated in the weights):
 *   dw[co,kh,kw,ci] = sum_{n,ho,wo} dy[n,ho,wo,co] * x[n, ho*s-p+kh*d, wo*s-p+kw*d, ci],
 * pixels outside the image contributing nothing.  x: bf16 NHWC input of the layer; dy: bf16 NHWC
 * gradient of its output [N,H_out,W_out,C_out]; dw: fp32 [C_out,KH,KW,C_in], every element written.
 * Products are exact, accumulation is fp32 on the tensor cores.  flags of desc are ignored.
 * Shape rules as ssconv_forward_dense.  x, dy, dw, ws: device, 16-byte aligned.
 * ws: scratch of at least ssconv_wgrad_ws_bytes, always needed: thread blocks store partial
 * gradients there (one slice per range of positions; layers with few weights and many positions
 * split the positions over thread blocks), and a second kernel adds the slices in a fixed order
 * and writes dw.  Needs no initialisation.  dev_status: as in ssconv_forward. */
int32_t ssconv_wgrad(const ssconv_desc_t* desc, const void* x, const void* dy, float* dw, void* ws,
                     size_t ws_bytes, int32_t* dev_status, void* stream);
/* The gradient with respect to the layer's input in one call (Eq. 4 differentiated in x; the paper prints
 * no gradient):  dx[n,h,w,ci] = sum over (kh,kw,co) of dy[n,ho,wo,co] * w[co,kh,kw,ci]  for the outputs
 * (ho,wo) whose tap (kh,kw) read pixel (h,w).  dy: bf16 [N,H_out,W_out,C_out], w: bf16 [C_out,KH,KW,C_in],
 * dx: bf16 [N,H,W,C_in] (every element is written), all device, 16-byte aligned; one rounding to bf16.
 * With unit stride it is one convolution of dy with the reversed, channel-exchanged filter (as
 * ssconv_dgrad_prepare + ssconv_forward_dense).  With a stride s > 1 the input pixels are split into the
 * s_h x s_w residue classes of their padded position: a pixel with (h + pad) mod s = a only met the taps
 * kh = a, a + s, ..., so each class is a unit-stride convolution of dy with its own few taps (all classes
 * together carry the layer's KH x KW taps, where ssconv_dgrad_spread makes every input pixel meet all of
 * them, s_h s_w - 1 of every s_h s_w products being zeros), written to scratch and interleaved into dx
 * by a gather kernel.  Strided layers with a dilation other than 1 or a stride above 4 take the plain route
 * instead (dy spread out with zeros as by ssconv_dgrad_spread, into scratch, then one convolution).
 * The flags of desc are ignored (no bias, no activation).
 * ws: device scratch of ssconv_dgrad_ws_bytes(desc) bytes (reversed weights; per class its weights and
 * tensor, or the spread gradient), too small -> SSCONV_ERR_WORKSPACE.  SSCONV_ERR_UNSUPPORTED_SHAPE: padding
 * beyond the filter's reach, C_out % 8 != 0. */
int32_t ssconv_dgrad_ws_bytes(const ssconv_desc_t* desc, size_t* bytes);
int32_t ssconv_dgrad(const ssconv_desc_t* desc, const void* dy, const void* w_bf16, void* dx, void* ws, size_t ws_bytes,
                     int32_t* dev_status, void* stream);

/* Scratch bytes ssconv_wgrad needs for this layer on the current device. */
int32_t ssconv_wgrad_ws_bytes(const ssconv_desc_t* desc, size_t* bytes);

/* ---- Stability quantities (Sec. 3.2) -----------------------------------------------------------
 * A masking B of a weight matrix W is the additive perturbation dW = (B - 1) .* W (Lemma 3.3).  In the
 * maximum-absolute-row-sum norm over W in R^{C_out x K} (a row is one output channel):
 *   out3[0] = ||W||_inf,   out3[1] = ||(B - 1) .* W||_inf  (<= out3[0], Lemma 3.3),   out3[2] = ||B .* W||_inf.
 * w_bf16: device bf16 [C_out][K], 8-byte aligned; pattern: device uint8 [C_out*K/4], as from
 * ssconv_select_mask; out3: device fp32 [3] (cleared and written by the call).  K % 4 == 0.
 * Magnitudes are summed in fp32 in a fixed order. */
int32_t ssconv_mask_norms(const void* w_bf16, const uint8_t* pattern, int32_t C_out, int64_t K,
                          float* out3, void* stream);

/* ||x||_inf = the largest magnitude among n bf16 values (exact).  x: device, 16-byte aligned; out:
 * device fp32 [1] (cleared and written by the call).  n >= 0 (0 gives 0). */
int32_t ssconv_absmax(const void* x_bf16, int64_t n, float* out, void* stream);

/* The confidence above which a depth-`depth` classifier with L-Lipschitz activations keeps its
 * prediction on a sample of norm x_norm (host arithmetic in double; returns a negative value for bad
 * arguments).  layer_norms[i] = ||W_i||, j = the layer that is masked or perturbed:
 *   SSCONV_LEMMA_PERTURBATION  (Lemma 3.4): L^depth * extra_norm * x_norm * prod_{i != j} ||W_i||,
 *                              extra_norm = ||dW_j|| (e.g. out3[1] of ssconv_mask_norms);
 *   SSCONV_LEMMA_ANY_MASK      (Lemma 3.5): L^depth * x_norm * prod_i ||W_i||  (extra_norm unused);
 *   SSCONV_LEMMA_MASKED_UPDATE (Lemma 3.6): L^depth * (||W_j|| + extra_norm) * x_norm * prod_{i != j} ||W_i||,
 *                              extra_norm = ||U_j||, the norm of the weight update. */
enum { SSCONV_LEMMA_PERTURBATION = 34, SSCONV_LEMMA_ANY_MASK = 35, SSCONV_LEMMA_MASKED_UPDATE = 36 };
double ssconv_stability_threshold(int32_t lemma, double L, const double* layer_norms, int32_t depth,
                                  int32_t j, double extra_norm, double x_norm);

/* ---- Grouped convolutions (Sec. 4: the paper leaves grouped convolutions dense; here both forms
 * exist).  The layer is `groups` independent convolutions on channel slices: group g reads input
 * channels [g C_in/groups, (g+1) C_in/groups) and writes output channels [g C_out/groups, ...).  desc
 * names the whole layer; weights are [C_out, KH, KW, C_in/groups] (each output channel sees its group's
 * inputs); the 2:4 groups of four are four consecutive input channels *of the group's slice*, the
 * pattern array follows the weight order, and the compressed operand is the concatenation of the
 * per-group blobs (ssconv_sizes_grouped gives the totals; each part is what ssconv_sizes reports for the
 * per-group layer and can be read back with ssconv_decompress).  Needs (C_in/groups) % 8 == 0 and
 * (C_out/groups) % 8 == 0; one launch per group on strided views of x and y.  ws as for
 * ssconv_forward (NULL allowed). */
int32_t ssconv_sizes_grouped(const ssconv_desc_t* desc, int32_t groups, int64_t* G, size_t* w_comp_bytes,
                             size_t* meta_bytes);
int32_t ssconv_compress_grouped(const ssconv_desc_t* desc, int32_t groups, const void* w_bf16, const uint8_t* pattern,
                                void* w_comp, void* meta, void* stream);
int32_t ssconv_forward_grouped(const ssconv_desc_t* desc, int32_t groups, const void* x, const void* w_comp,
                               const void* meta, const float* bias, void* y, void* ws, size_t ws_bytes,
                               int32_t* dev_status, void* stream);
int32_t ssconv_forward_dense_grouped(const ssconv_desc_t* desc, int32_t groups, const void* x, const void* w_bf16,
                                     const float* bias, void* y, void* ws, size_t ws_bytes, int32_t* dev_status,
                                     void* stream);

/* Depthwise convolution (groups = C_in = C_out), dense, as the paper leaves it (Sec. 4):
 *   y[n,ho,wo,c] = act( bias[c] + sum_{kh,kw} x[n, ho*s-p+kh*d, wo*s-p+kw*d, c] * w[kh,kw,c] ),
 * weights tap-major [KH, KW, C] bf16, fp32 accumulation, one rounding to bf16; act = ReLU or none.
 * Equal strides, paddings and dilations in both directions; C % 8 == 0; 16-byte aligned pointers. */
int32_t ssconv_depthwise(const ssconv_desc_t* desc, const void* x, const void* w_bf16, const float* bias, void* y,
                         void* stream);

/* Layer normalisation over the channels of each pixel, y = (x - mean) / sqrt(var + eps) * gamma + beta
 * (biased variance; fp32 arithmetic, one rounding to bf16): the normalisation between the depthwise and
 * the point-wise convolutions of a ConvNeXt block (Sec. 4 evaluates on ConvNeXt); no counterpart in the
 * paper's method.  x, y: bf16 [pixels, C]; gamma, beta: float [C]. */
int32_t ssconv_layernorm(const void* x_bf16, const float* gamma, const float* beta, float eps, void* y_bf16,
                         int64_t pixels, int32_t C, void* stream);

/* ---- 8-bit (e4m3) operands.  The paper's method is stated for any operand type the 2:4 hardware
 * operation supports (Sec. 2: the sparse operation halves storage and time; Sec. 3.1 defines the
 * N:M masks on the weight matrix regardless of its number format); these calls run Eq. 6 / Eq. 4
 * with activations and weights in the 8-bit floating-point format e4m3 (1 sign, 4 exponent bits of
 * bias 7, 3 mantissa bits, no infinities, largest magnitude 448), fp32 accumulation and bf16
 * output:   y = act( bias + out_scale * sum x_q * (M .* W)_q ),
 * where x_q, W_q are the values the codes stand for and out_scale (> 0) undoes whatever scales the
 * caller applied when quantising (ssconv_quantize_e4m3).  Layouts as for bf16 with one byte per
 * element; C_in % 16 == 0; no residual form, no K split (no workspace), one-block tiles only. */

/* y[i] = the e4m3 value nearest to x[i] * scale (the product rounded to fp32 first; ties to the even
 * mantissa; magnitudes beyond 448 saturate to 448; the sign is kept).  x: bf16, 4-byte aligned;
 * y: bytes, 2-byte aligned; n even. */
int32_t ssconv_quantize_e4m3(const void* x_bf16, void* y_e4m3, int64_t n, float scale, void* stream);

/* ssconv_sizes / ssconv_compress / ssconv_decompress for e4m3 weights [C_out,KH,KW,C_in] (bytes).
 * The blobs differ from the bf16 ones (k-blocks of 128 channels, one byte per kept value, twice the
 * metadata per pair of k-blocks) and only ssconv_forward_fp8 / ssconv_decompress_fp8 read them. */
int32_t ssconv_sizes_fp8(const ssconv_desc_t* desc, int64_t* G, size_t* w_comp_bytes, size_t* meta_bytes);
int32_t ssconv_compress_fp8(const ssconv_desc_t* desc, const void* w_e4m3, const uint8_t* pattern, void* w_comp,
                            void* meta, void* stream);
int32_t ssconv_decompress_fp8(const ssconv_desc_t* desc, const void* w_comp, const void* meta, void* w_masked_e4m3,
                              uint8_t* pattern_out, void* stream);

/* The masked convolution on e4m3 operands (sparse tcgen05.mma kind::f8f6f4) and its dense counterpart. */
int32_t ssconv_forward_fp8(const ssconv_desc_t* desc, const void* x_e4m3, const void* w_comp, const void* meta,
                           const float* bias, float out_scale, void* y, int32_t* dev_status, void* stream);
int32_t ssconv_forward_dense_fp8(const ssconv_desc_t* desc, const void* x_e4m3, const void* w_e4m3, const float* bias,
                                 float out_scale, void* y, int32_t* dev_status, void* stream);

/* Folding of f neighbouring output pixels of a row into the output channels.  A tile of the forward
 * kernels always spends 128 accumulator rows on output channels, so a layer with C_out <= 64 wastes
 * half of every multiply-add it issues.  The convolution of Eq. 4 with KW taps of stride s and
 * dilation d along the width equals, output pixel (h, f i + j) <-> channel block j of pixel (h, i), a
 * convolution with f C_out output channels, KW' = (f-1) s + (KW-1) d + 1 undilated taps and stride f s,
 *   W'[j C_out + c, kh, kw', :] = W[c, kh, kw, :]  where kw' = j s + kw d, and 0 elsewhere,
 * whose NHWC output [N, H_out, W_out / f, f C_out] is byte for byte the output [N, H_out, W_out, C_out]
 * of the original.  Groups of four input channels stay together, so a 2:4 pattern folds with its
 * weights (all-zero groups take pattern 0) and the folded layer goes through ssconv_compress /
 * ssconv_forward, or ssconv_forward_dense, like any other; bias and residual keep their meaning (the
 * bias is repeated f times, the residual tensor is read through the same byte identity).
 *   ssconv_fold_factor: the factor (1 or 2) the planner suggests for a layer: 2 when C_out <= 64,
 *     W_out is even and the folded layer issues at least 15 % fewer multiply-adds per output.
 *   ssconv_fold_desc: the folded descriptor; W_out % f != 0 -> SSCONV_ERR_UNSUPPORTED_SHAPE.
 *   ssconv_fold_weights: w (nullable) is [C_out, KH, KW] vectors of tap_bytes bytes each (bf16 weights:
 *     2 C_in; e4m3 weights: C_in; patterns: C_in / 4), w_folded [f C_out, KH, KW'] such vectors;
 *     bias (nullable) [C_out] floats, bias_folded [f C_out].  Device pointers, no alignment rule. */
int32_t ssconv_fold_factor(const ssconv_desc_t* desc);
int32_t ssconv_fold_desc(const ssconv_desc_t* desc, int32_t f, ssconv_desc_t* folded);
int32_t ssconv_fold_weights(const ssconv_desc_t* desc, int32_t f, const void* w, void* w_folded, int64_t tap_bytes,
                            const float* bias, float* bias_folded, void* stream);

/* ssconv_forward_dense on a strided view of the input: pixel (n, h, w) of the H x W x C_in input the
 * descriptor names starts stride_n*n + stride_h*h + stride_w*w elements into x.  The strides are
 * multiples of 8 elements and need not exceed C_in: with stride_w < C_in neighbouring pixels
 * overlap, i.e. the input is a sliding window of C_in channels over a narrower tensor (the unfold of
 * Eq. 5 along the width, taken by the loads themselves instead of being written out; see
 * ssconv_space_to_depth).  Everything else as ssconv_forward_dense; C_in == 8 is not accepted. */
int32_t ssconv_forward_dense_strided(const ssconv_desc_t* desc, const void* x, int64_t stride_w, int64_t stride_h,
                                     int64_t stride_n, const void* w_bf16, const float* bias, void* y, void* ws,
                                     size_t ws_bytes, int32_t* dev_status, void* stream);

/* ssconv_forward for callers that have no way to provide scratch memory.  (The paper has no
 * counterpart to this call; it exists for integration only.)
 *
 * Some hosts of this library may not allocate on the device at all once they are running: an
 * inference server that hands every component a fixed arena at start-up, a real-time loop where
 * cudaMalloc's implicit synchronisation is unacceptable, a plug-in inside a process whose memory
 * pool is owned by someone else.  For them the scratch that ssconv_forward takes as `ws` is
 * compiled into the library: a fixed device array of about 15.7 MB (room for 64 thread blocks),
 * which every GPU that loads the library holds until the process exits.  The call allocates
 * nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 *
 * Same arguments, formula, layouts and error codes as ssconv_forward, without ws.  Differences:
 *  - Only small layers are accepted, the ones whose K range is worth splitting across thread
 *    blocks: at most 64 output tiles (a tile is 128 output channels x 240 pixels); larger layers
 *    return SSCONV_ERR_UNSUPPORTED_SHAPE and should go through ssconv_forward, which needs no
 *    scratch for them (ws = NULL is accepted there).
 *  - The K range is always split, over at most 64 thread blocks, so the fp32 summation order,
 *    and with it the last bits of y, can differ from ssconv_forward's.
 *  - The first call on each device looks up the array's device address (with that device
 *    current); make that first call outside any stream capture.  The array itself comes into
 *    being when the CUDA module that holds the forward kernels is loaded on the device, which
 *    under CUDA's default lazy loading is the first forward call of any kind on that device:
 *    until then its 15.7 MB are not yet taken.
 *  - All calls share the one array, and it keeps what the previous call left in it.  Nothing in
 *    it has to be cleared (every partial sum is written before it is read), so calls issued one
 *    after another on one stream are safe; two calls that can overlap on the GPU
 *    (different streams, no dependency) race on the array and give wrong results. */
int32_t ssconv_forward_static_ws(const ssconv_desc_t* desc, const void* x, const void* w_comp,
                                 const void* meta, const float* bias, void* y, int32_t* dev_status,
                                 void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SSCONV_H_ */
