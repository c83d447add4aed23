// Masked (2:4 sparse) and dense NHWC bf16 convolution forward as an implicit GEMM on the
// sm_100a tensor cores (Eq. 5 / Eq. 6 of the paper; the unfold U(X) is never materialised).
//
//   D[C_out x Q] = A[C_out x K] * B[K x Q],   Q = output positions, K = KH*KW*C_in
//
// A = weights (the only operand tcgen05.mma.sp accepts in 2:4 form), B = activations.  A CTA
// owns a 128 (output channels) x BN (positions) tile of D at a time and walks a static list of
// tiles (persistent kernel).  BN is chosen per layer by the host, a multiple of 16 up to 240: 240
// is as wide as two fp32 accumulators plus the metadata columns allow in the 512 TMEM columns, and
// wide MMAs amortise the cost of issuing them; narrower tiles are used when 240-wide ones would
// leave most SMs without work.
//
// Positions are the output pixels (n, ho, wo) in row-major order.  K is cut into k-blocks of 64
// input channels at one filter tap; per k-block one im2col-mode TMA load brings the tile's pixels'
// channels at that tap, zero-filled outside the image.  The shared-memory ring's unit is a group
// of two k-blocks (see Cfg).  Dense layers with 8 input channels pack 8 taps into a k-block instead
// (see producer_role).
//
// Warp roles: warps 0, 10 and 11 TMA producers (one thread each: the activations of a group's
// first k-block, of its second, the weights), warp 1 MMA issuer (one thread; owns TMEM), warps 2-9
// epilogue in two groups of four warps that each own half of a tile's positions.  The accumulator
// has channels on TMEM lanes and positions on columns, NHWC wants the transpose: the epilogue reads
// TMEM in the MMA-fragment layout (tcgen05.ld 16x256b), adds the bias, converts pairs to bf16
// (with ReLU in the conversion), and stmatrix.trans writes 8x8 blocks transposed into a 128-byte
// swizzled staging buffer [position][channel], which TMA stores write to NHWC asynchronously.
// That is about 2.5 instructions per thread and element pair; an epilogue of scalar shared-memory
// stores or lane shuffles is issue-bound at several times that.
//
// What paces the main loop (measured): the issuing warp pays about 200 cycles per mbarrier wait,
// even on a complete barrier, and 60-80 per tcgen05 instruction, and the tensor pipe's queue is
// shallow, so every instruction between MMAs is exposed: hence one handshake per group and nothing
// else in that loop.  The other bound is the rate at which an SM takes
// loads in from L2, about 68 bytes per cycle when all SMs load.  Staging one run of padded input per
// channel chunk and serving all taps of a 3x3 filter from it through row-shifted descriptors (which
// would cut the activation loads ninefold) was built and measured before the issue loop was lean,
// and dropped; it remains the way past the fill bound for large feature maps.
//
// Work partition: the unit of work is one group's worth of K for one output tile.  Either every CTA
// takes a contiguous block of whole output tiles, or (when whole tiles would leave many SMs idle)
// the units are dealt out evenly, so a CTA's range may start and end inside an output tile
// ("stream-K").  A CTA writes a partly computed tile (fp32) to a scratch region of its own in
// global memory; a second, small kernel (ssconv_split_finish_kernel) then sums the regions of
// every split tile in a fixed order on all SMs and applies the same epilogue.  No CTA ever waits
// for another, and the result does not depend on timing.
// All mbarrier waits are bounded; when one runs out the CTA raises a flag, every role leaves
// its loop, TMEM is freed and SSCONV_ERR_TIMEOUT is stored to *dev_status.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <type_traits>

#include "layout.cuh"
#include "sm100_ptx.cuh"
#include "ssconv.h"

namespace ssconv {

constexpr int kBN = 240;                 // most positions per tile (N of the MMA); a layer's tile may be narrower
constexpr int kGroups = 2;               // epilogue warp groups, each owning half of a tile's positions
constexpr int kGroupCols = kBN / kGroups;
constexpr int kPiece = 40;               // positions per epilogue piece (one staging buffer)
constexpr int kFirstExtraProducerWarp = 2 + 4 * kGroups;  // warps 10 and 11: two more TMA producers
constexpr int kThreads = 64 + 128 * kGroups + 64;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kAccCol1 = 256;       // second accumulator; the first starts at column 0
constexpr uint32_t kMetaCol = kBN;       // metadata: 2 slots x 4 columns in [240, 248)
constexpr long long kWaitLimitCycles = 4000000000LL;  // ~2 s at 1.9 GHz
constexpr uint32_t kATileBytes = 128 * 128;          // 128 rows x 128 B
constexpr uint32_t kHalfPieceBytes = kPiece * 128;    // 40 positions x 64 channels bf16, 128-byte swizzled
constexpr uint32_t kPieceBytes = 2 * kHalfPieceBytes; // channels [0,64) then [64,128) of the tile
__host__ __device__ constexpr uint32_t staging_bytes(int bufs) { return (uint32_t)bufs * kGroups * kPieceBytes; }  // per group 2 or 4 buffers
constexpr uint32_t kBarrierBytes = 256;

// The ring's unit is a group: the operands of one pair of k-blocks (128 dense columns of K).
// Layout of a group in shared memory: weights (sparse: one 128 x 128 B tile of kept values, which
// spans both k-blocks, + its metadata image; dense: two tiles), then the two activation tiles of
// BN x 128 B.  One full and one empty barrier per group: the issuing thread pays about 200 cycles
// per wait and 80 per tcgen05 instruction, so the handshake is per pair of k-blocks, not per k-block.
// FP8: e4m3 operands (tcgen05 kind::f8f6f4).  A 128-byte row then holds 128 channels, so a k-block is
// 128 channels of one tap; in bytes every tile is what it is for bf16, only the metadata of a 2:4 group
// of two k-blocks doubles (512 dense columns instead of 256: two images of 2048 bytes).
template <bool SPARSE, bool FP8 = false>
struct Cfg {
  static constexpr uint32_t kMetaBytes = (FP8 ? 2u : 1u) * (uint32_t)kMetaImageBytes;
  static constexpr uint32_t kAGroupBytes = SPARSE ? kATileBytes + kMetaBytes : 2 * kATileBytes;
  static constexpr int kKbChannels = FP8 ? 2 * kBlockK : kBlockK;  // input channels per k-block
};
constexpr int kMaxGroups = 4;                  // groups in the ring: as many as fit, 2 to 4
constexpr uint32_t kMaxSmemBytes = 232448;     // 227 KB per CTA
__host__ __device__ constexpr uint32_t group_bytes(uint32_t a_group_bytes, int BN) {
  return a_group_bytes + 2u * (uint32_t)BN * 128u;
}

struct FwdParams {
  int C_in, C_out;
  int Ho, Wo;               // output extent
  int Q;                    // positions = N * Ho * Wo
  int BN;                   // positions per tile, a multiple of 16, at most kBN
  int pieces;               // epilogue pieces per group: ceil(BN / 2 / kPiece)
  int tail_cols;            // positions in a group's last piece (a multiple of 8, at most kPiece)
  int ring_groups;          // groups in the shared-memory ring
  int stage_bufs;           // staging buffers per epilogue group: 2, or 4 when residual pieces are prefetched
  int small_c;              // dense layers with C_in == 8: a k-block is 8 filter taps (see producer_role)
  uint32_t a_grp_bytes;     // bytes of weights (and metadata) at the head of a ring group; 0: weights resident
  uint32_t a_res_bytes;     // dense layers of one channel tile and at most four k-blocks: the whole weight
                            // tile stays in shared memory after the ring (loaded once per CTA), groups hold
                            // activations only
  int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, KW;
  int taps, cblocks, kblocks;
  int m_tiles, num_tiles;   // (pair kernel: m_tiles counts pairs of 128-channel tiles, m_real the tiles themselves)
  int m_real;
  int a_tiles;              // pairs of k-blocks (groups) per output tile
  int dual;                 // pair kernel: a work item is two neighbouring position tiles sharing the group's weights
  int split;                // 1: units dealt out evenly across CTAs (stream-K); 0: whole tiles per CTA
  int work_quot, work_rem;  // work items per CTA: quotient and remainder of (tiles or units) / grid
  float out_scale;          // 8-bit operands: factor applied to the accumulators before the bias
  float4* ws_regions;       // [2 * gridDim.x] regions of 128 x 240 fp32: a CTA's partial tiles
  uint32_t flags;
  const float* bias;
  const uint8_t* meta;
  __nv_bfloat16* y;
  int32_t* dev_status;
};

// Range [a0, a1) of groups (pairs of k-blocks) of one output tile: what a CTA computes in one
// accumulator pass.
struct Segment {
  int tile, a0, a1;
};

// The W work items (whole tiles, or (tile, group) units when K is split) are dealt out to the G
// CTAs in contiguous, near-equal ranges: CTA c gets [c q + min(c, r), ...) of length q + (c < r)
// with q = W / G, r = W % G, both computed on the host: the device needs no division for it.
struct WorkIter {
  int tile, a0, left, A;  // next tile, first group of it, units left in this CTA's range, groups per tile
  __device__ explicit WorkIter(const FwdParams& p) : WorkIter(p, blockIdx.x) {}
  __device__ WorkIter(const FwdParams& p, uint32_t c) {  // c: this worker's number (CTA, or CTA pair)
    A = p.a_tiles;
    const uint32_t start = c * (uint32_t)p.work_quot + (c < (uint32_t)p.work_rem ? c : (uint32_t)p.work_rem);
    const int count = p.work_quot + (c < (uint32_t)p.work_rem ? 1 : 0);
    if (p.split) {
      tile = (int)(start / (uint32_t)A);  // the one division of the split path
      a0 = (int)(start - (uint32_t)tile * (uint32_t)A);
      left = count;
    } else {
      tile = (int)start;
      a0 = 0;
      left = count * A;
    }
  }
  __device__ bool next(Segment& s) {
    if (left <= 0) return false;
    s.tile = tile;
    s.a0 = a0;
    s.a1 = (left >= A - a0) ? A : a0 + left;
    left -= s.a1 - s.a0;
    ++tile;
    a0 = 0;
    return true;
  }
};

// Walks the epilogue pieces of this CTA's whole tiles in the order the epilogue meets them, ahead of
// it: used to prefetch residual pieces.
struct PieceAhead {
  WorkIter it;
  Segment seg;
  int piece, pieces, a_tiles;
  bool have;
  __device__ PieceAhead(const FwdParams& p) : it(p), piece(0), pieces(p.pieces), a_tiles(p.a_tiles), have(false) {}
  __device__ PieceAhead(const FwdParams& p, uint32_t worker)
      : it(p, worker), piece(0), pieces(p.pieces), a_tiles(p.a_tiles), have(false) {}
  __device__ bool next(int& tile, int& piece_out) {
    while (!have || piece == pieces) {
      if (!it.next(seg)) return false;
      have = (seg.a0 == 0 && seg.a1 == a_tiles);
      piece = 0;
    }
    tile = seg.tile;
    piece_out = piece++;
    return true;
  }
};

// CTA that owns work unit u under that dealing: inverse of start(c) = c q + min(c, r).
__device__ __forceinline__ int unit_owner(uint32_t u, uint32_t q, uint32_t r) {
  const uint32_t big = r * (q + 1);  // units held by the r CTAs with one extra
  return (u < big) ? (int)(u / (q + 1)) : (int)(r + (u - big) / q);
}

// A scratch region holds one 128 x 240 fp32 partial tile in the order the epilogue threads hold it:
// float4 number j (of 10) of piece `piece` of thread `gtid` of group `grp`, consecutive threads
// adjacent, so that a warp reads or writes 512 contiguous bytes at a time.
constexpr int kRegionVecs = kTileM * kBN / 4;
constexpr int kPiecesPerGroup = kGroupCols / kPiece;
__device__ __forceinline__ int region_vec(int grp, int piece, int j, int gtid) {
  return ((grp * kPiecesPerGroup + piece) * (kPiece / 4) + j) * 128 + gtid;
}
// Region of CTA c for a split tile: its range starts inside the tile (0) or the tile starts inside
// its range (1).  A range has at most one segment of each kind.
__device__ __forceinline__ size_t region_index(int c, bool tile_starts_here) {
  return 2 * (size_t)c + (tile_starts_here ? 1 : 0);
}

// Named barriers: 1 and 2 for the epilogue groups, 3 for the setup (warp 0 arrives without waiting).
__device__ __forceinline__ void epilogue_bar_sync(int group) {
  asm volatile("bar.sync %0, 128;" ::"r"(group + 1) : "memory");
}
__device__ __forceinline__ void setup_bar_arrive() {
  __threadfence_block();
  asm volatile("bar.arrive 3, %0;" ::"n"(kThreads) : "memory");
}
__device__ __forceinline__ void setup_bar_sync() { asm volatile("bar.sync 3, %0;" ::"n"(kThreads) : "memory"); }
// One epilogue piece of this warp's 32 lanes x 40 columns in fragment layout: register
// r[20 h + 4 k + 2 s + e] = lane (16 h + 8 s + t/4), column (8 k + 2 (t%4) + e).  No wait.
__device__ __forceinline__ void tc_ld_piece(uint32_t taddr, uint32_t (&r)[kPiece]) {
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint32_t a = taddr + ((uint32_t)(16 * h) << 16);
    tc_ld_16x256b_x4(a, &r[20 * h]);
    tc_ld_16x256b_x1(a + 32, &r[20 * h + 16]);
  }
}
// bias, activation and bf16 for one piece, written transposed to its staging buffer.  st_addr is
// this thread's address for the first 8 positions; each further 8 positions are 1024 bytes on.
// With RES the staging buffer already holds the residual tile (bf16, same layout): it is read back
// in fragment layout (ldmatrix.trans, the inverse of the store), added in fp32 before the one
// rounding, and overwritten in place (a warp only touches its own 16-byte columns).
// ACT: 0 identity, 1 ReLU (inside the bf16 conversion), 2 GELU in its erf form x Phi(x) =
// 0.5 x (1 + erf(x / sqrt 2)), evaluated in fp32 before the rounding.
// erf without branches: erf(z) = 1 - 2^R(z) for z >= 0 with R a degree-6 polynomial (no constant term)
// fitted to log2(erfc(z)) on [0, 4] (beyond 4, erfc < 2e-8 and z is clamped), odd extension by the sign of
// x; the factor 1 / sqrt 2 of z = |x| / sqrt 2 is folded into the coefficients, so the polynomial takes
// |x| clamped at 4 sqrt 2.  The difference 1 - 2^R loses relative accuracy near 0, which x Phi(x) does not
// need.  Against fp64 over every bf16 input up to 8: |R - log2 erfc| <= 4.8e-5, i.e. 3.3e-5 relative in
// exact arithmetic; evaluated in fp32 the result is within 5.1e-6 absolute, and within 3e-4 relative
// wherever |x Phi(x)| > 1e-4 (the largest ratio sits in the far negative tail, where 0.5 x and |x| t
// cancel), a seventh of the rounding to bf16 that follows (2^-9).  A degree-8 fit bought nothing after that
// rounding and cost two more multiply-adds per value, which matters because shallow layers with this
// activation are bound by the epilogue's arithmetic.
constexpr int kActNone = 0, kActRelu = 1, kActGelu = 2;
constexpr float kGeluClamp = 5.656854152679443f;  // 4 sqrt 2
constexpr float kGeluC1 = -1.1506847143173218f, kGeluC2 = -0.46029916405677795f, kGeluC3 = -0.05191940814256668f,
                kGeluC4 = 0.00745233241468668f, kGeluC5 = -0.0006528479279950261f, kGeluC6 = 2.5540923161315732e-05f;
// Two values at once, the polynomial on fp32 pairs (fma.rn.f32x2); the result is formed as
// x (0.5 + sign(x) (0.5 - 0.5 e)) = 0.5 x + |x| (0.5 - 0.5 e) with e = 2^R.
__device__ __forceinline__ unsigned long long f32x2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ unsigned long long horner2(unsigned long long r, unsigned long long z, float c) {
  asm("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(r) : "l"(z), "l"(f32x2(c, c)));
  return r;
}
__device__ __forceinline__ void split2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// GELU of the pair x, returned as a pair; everything that has a paired form is done on pairs (the polynomial,
// 0.5 - 0.5 e, 0.5 x and the final multiply-add), so that the eight epilogue warps issue as few instructions as
// possible: the result is x s + 0.5 x with s = sign(x) (0.5 - 0.5 e).
__device__ __forceinline__ unsigned long long gelu_f32x2(unsigned long long x) {
  float lo, hi;
  split2(x, lo, hi);
  const unsigned long long a = f32x2(fminf(fabsf(lo), kGeluClamp), fminf(fabsf(hi), kGeluClamp));
  unsigned long long r = f32x2(kGeluC6, kGeluC6);
  r = horner2(r, a, kGeluC5);
  r = horner2(r, a, kGeluC4);
  r = horner2(r, a, kGeluC3);
  r = horner2(r, a, kGeluC2);
  r = horner2(r, a, kGeluC1);
  asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(r) : "l"(a));
  float r0, r1, e0, e1;
  split2(r, r0, r1);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(r0));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(r1));
  unsigned long long t = f32x2(e0, e1);
  asm("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(t) : "l"(f32x2(-0.5f, -0.5f)), "l"(f32x2(0.5f, 0.5f)));
  float t0, t1;
  split2(t, t0, t1);
  const unsigned long long sgn = f32x2(copysignf(t0, lo), copysignf(t1, hi));
  unsigned long long y;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(y) : "l"(x), "l"(f32x2(0.5f, 0.5f)));
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(y) : "l"(x), "l"(sgn));
  return y;
}
template <int ACT>
__device__ __forceinline__ uint32_t activate_pack(float lo, float hi) {
  if (ACT == kActGelu) split2(gelu_f32x2(f32x2(lo, hi)), lo, hi);
  return pack_bf16x2<ACT == kActRelu>(lo, hi);
}
__host__ __device__ inline int activation_of(uint32_t flags) {
  return (flags & SSCONV_FLAG_GELU) ? kActGelu : (flags & SSCONV_FLAG_RELU) ? kActRelu : kActNone;
}
template <int ACT, bool RES>
__device__ __forceinline__ void stage_piece(const uint32_t (&r)[kPiece], const float (&bias)[4], uint32_t st_addr) {
#pragma unroll
  for (int k = 0; k < kPiece / 8; ++k) {
    uint32_t w[4];
    uint32_t res[4] = {0u, 0u, 0u, 0u};
    if (RES) ldmatrix_x4_trans(st_addr + 1024u * k, res);
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // channel block i = 2 h + s of the warp's 32 channels
      const int at = 20 * (i >> 1) + 4 * k + 2 * (i & 1);
      if (ACT == kActGelu && !RES) {
        // (the bias goes in as a pair too)
        unsigned long long x = f32x2(__uint_as_float(r[at]), __uint_as_float(r[at + 1]));
        asm("add.rn.f32x2 %0, %0, %1;" : "+l"(x) : "l"(f32x2(bias[i], bias[i])));
        float lo, hi;
        split2(gelu_f32x2(x), lo, hi);
        w[i] = pack_bf16x2<false>(lo, hi);
        continue;
      }
      float lo = __uint_as_float(r[at]) + bias[i], hi = __uint_as_float(r[at + 1]) + bias[i];
      if (RES) {
        lo += bf16_lo(res[i]);
        hi += bf16_hi(res[i]);
      }
      w[i] = activate_pack<ACT>(lo, hi);
    }
    stmatrix_x4_trans(st_addr + 1024u * k, w[0], w[1], w[2], w[3]);
  }
}

// Position q -> (image, output row, output column).
struct Pos {
  int n, r, c;
};
__device__ __forceinline__ Pos decode_pos(int q, int Wq, int Hq) {
  Pos s;
  const int rho = q / Wq;
  s.c = q - rho * Wq;
  s.n = rho / Hq;
  s.r = rho - s.n * Hq;
  return s;
}

// Filter tap and channel chunk of a k-block (numbered chunk * taps + tap), advanced incrementally.
struct TapIter {
  int cc, tap, kw, off_w, off_h;
  __device__ void init(int kb, const FwdParams& p) {
    cc = kb / p.taps;
    tap = kb - cc * p.taps;
    const int kh = tap / p.KW;
    kw = tap - kh * p.KW;
    off_w = kw * p.dil_w;
    off_h = kh * p.dil_h;
  }
  __device__ void advance(const FwdParams& p) {
    ++tap;
    off_w += p.dil_w;
    if (++kw == p.KW) {
      kw = 0;
      off_w = 0;
      off_h += p.dil_h;
      if (tap == p.taps) {  // next channel chunk
        tap = 0;
        off_h = 0;
        ++cc;
      }
    }
  }
};

// One of the three TMA producer warps.  All of them walk the same sequence of groups; role 0
// loads the activation tile of each group's first k-block, role 1 that of the second, role 2 the
// weights (with their metadata).  A TMA instruction occupies its issuing thread for a few hundred
// cycles, so one thread issuing everything cannot keep up with the tensor pipe; three can.
constexpr int kRoleActFirst = 0, kRoleActSecond = 1, kRoleWeights = 2;
template <bool SPARSE, int ROLE, bool FP8 = false>
__device__ __forceinline__ void producer_role(const CUtensorMap* tm_a, const CUtensorMap* tm_b, const FwdParams& p,
                                              uint32_t full0, uint32_t empty0, uint32_t ring0, uint32_t res_bar,
                                              volatile int* abort_flag) {
  using C = Cfg<SPARSE, FP8>;
  constexpr int kKb = C::kKbChannels;
  const uint32_t b_bytes = (uint32_t)p.BN * 128u;  // one activation tile: BN positions x 64 channels
  const uint32_t grp_bytes = p.a_grp_bytes + 2u * b_bytes;
  const bool resident = !SPARSE && !FP8 && p.a_res_bytes != 0;
  uint32_t g = 0, ph = 0;  // group slot and its phase parity
  bool ok = true;
  bool first_segment = true;
  WorkIter work(p);
  Segment seg;
  while (ok && work.next(seg)) {
    const int pt = seg.tile / p.m_tiles;
    const int m = seg.tile - pt * p.m_tiles;
    const Pos q0 = decode_pos(pt * p.BN, p.Wo, p.Ho);
    const int base_w = q0.c * p.stride_w - p.pad_w;
    const int base_h = q0.r * p.stride_h - p.pad_h;
    const uint8_t* meta_src = p.meta + ((size_t)m * p.a_tiles + seg.a0) * C::kMetaBytes;
    TapIter it;
    it.init(2 * seg.a0 + (ROLE == kRoleActSecond ? 1 : 0), p);
    if (first_segment) {
      // everything above ran concurrently with the tail of the previous grid in the stream; its
      // results (our inputs) are complete from here on
      grid_dependency_wait();
      first_segment = false;
      if (ROLE == kRoleWeights && resident) {
        // the layer's whole weight tile, once: k-block b at b * kATileBytes after the ring
        const uint32_t res0 = ring0 + (uint32_t)p.ring_groups * grp_bytes;
        mbar_expect_tx_w(res_bar, (uint32_t)p.kblocks * kATileBytes);
        TapIter rit;
        rit.init(0, p);
        for (int b = 0; b < p.kblocks; ++b) {
          tma_load_3d_w(res0 + (uint32_t)b * kATileBytes, tm_a, res_bar, rit.cc * kKb, rit.tap, m * kTileM);
          rit.advance(p);
        }
      }
    }
    for (int a = seg.a0; a < seg.a1; ++a) {
      if (!mbar_wait_a(empty0 + 8u * g, ph ^ 1u, abort_flag, kWaitLimitCycles)) { ok = false; break; }
      const uint32_t full = full0 + 8u * g;
      const uint32_t dst = ring0 + g * grp_bytes;
      const bool has_second = 2 * a + 1 < p.kblocks;
      if (!SPARSE && p.small_c) {
        // 8 input channels (16 bytes per pixel): a k-block is 8 filter taps, held in shared memory as
        // 8 unswizzled chunks, each 16 bytes wide (chunk after chunk, rows every 16 bytes).
        // One load per tap and operand (im2col for the activations, a 8 x 1 x 128 box for the
        // weights; a single box over 8 taps was measured slower).  MMAs take chunks in pairs, so an
        // odd tail is padded with a tap beyond the filter, whose channel coordinate lies outside
        // the tensor: TMA fills zeros on both operands.
        const int first_tap = 16 * a + (ROLE == kRoleActSecond ? 8 : 0);
        int left_taps = p.taps - first_tap;
        const int most = (ROLE == kRoleWeights) ? 16 : 8;
        left_taps = left_taps < 0 ? 0 : (left_taps > most ? most : left_taps);
        const int chunks = (left_taps + 1) & ~1;
        it.init(first_tap, p);  // counted in taps here
        if (chunks == 0) {
          mbar_arrive_w(full);
        } else if (ROLE == kRoleWeights) {
          mbar_expect_tx_w(full, (uint32_t)chunks * 2048u);
          for (int j = 0; j < chunks; ++j) {  // chunks 8.. belong to the second k-block: 16 KB further on = 8 x 2048
            tma_load_3d_w(dst + (uint32_t)j * 2048u, tm_a, full, it.cc * kKb, it.tap, m * kTileM);
            it.advance(p);
          }
        } else {
          const uint32_t chunk_bytes = (uint32_t)p.BN * 16u;
          mbar_expect_tx_w(full, (uint32_t)chunks * chunk_bytes);
          const uint32_t b_dst = dst + p.a_grp_bytes + (ROLE == kRoleActSecond ? b_bytes : 0u);
          for (int j = 0; j < chunks; ++j) {
            tma_load_im2col_4d_w(b_dst + (uint32_t)j * chunk_bytes, tm_b, full, it.cc * kKb, base_w, base_h,
                                 q0.n, (uint16_t)it.off_w, (uint16_t)it.off_h);
            it.advance(p);
          }
        }
      } else if (ROLE == kRoleWeights && resident) {
        mbar_arrive_w(full);  // nothing to load per group: only keep the barrier's count
      } else if (ROLE == kRoleWeights) {
        if (SPARSE) {
          mbar_expect_tx_w(full, C::kAGroupBytes);
          tma_load_2d_w(dst, tm_a, full, a * (FP8 ? 128 : 64), m * kTileM);  // 128 bytes of kept values per group
          bulk_load_w(dst + kATileBytes, meta_src, C::kMetaBytes, full);
          meta_src += C::kMetaBytes;
        } else {
          mbar_expect_tx_w(full, has_second ? 2 * kATileBytes : kATileBytes);
          tma_load_3d_w(dst, tm_a, full, it.cc * kKb, it.tap, m * kTileM);
          it.advance(p);
          if (has_second) tma_load_3d_w(dst + kATileBytes, tm_a, full, it.cc * kKb, it.tap, m * kTileM);
          it.advance(p);
        }
      } else if (ROLE == kRoleActFirst || has_second) {
        mbar_expect_tx_w(full, b_bytes);
        tma_load_im2col_4d_w(dst + p.a_grp_bytes + (ROLE == kRoleActSecond ? b_bytes : 0u), tm_b, full,
                             it.cc * kKb, base_w, base_h, q0.n, (uint16_t)it.off_w, (uint16_t)it.off_h);
        it.advance(p);
        it.advance(p);
      } else {
        mbar_arrive_w(full);  // the group has no second k-block: only keep the barrier's count
      }
      if (++g == (uint32_t)p.ring_groups) {
        g = 0;
        ph ^= 1u;
      }
    }
  }
}

// RES: a residual tensor is added in the epilogue (its own instantiation, so that the plain kernel's
// epilogue loop carries none of that code).
template <bool SPARSE, bool RES, bool FP8 = false>
__global__ void __launch_bounds__(kThreads, 1)
ssconv_fwd_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                  const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_y_tail,
                  const __grid_constant__ CUtensorMap tm_r, const __grid_constant__ CUtensorMap tm_r_tail,
                  const FwdParams p) {
  using C = Cfg<SPARSE, FP8>;
  static_assert(!(FP8 && RES), "the residual epilogue is not built for 8-bit operands");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* ring = smem;                                                    // ring_groups groups
  // (then the resident weight tile, if any), then per epilogue group two buffers
  uint8_t* out_stage = ring + p.ring_groups * (p.a_grp_bytes + 2u * (uint32_t)p.BN * 128u) + p.a_res_bytes;
  // barrier slots: [0,4) group full, [4,8) group empty, [8,10) accumulator full, [10,12) accumulator empty,
  // [12,20) residual piece landed (per epilogue group and staging buffer), [20,24) first k-block of a
  // group consumed (two-slot rings only: its activation tile may be refilled ahead of the rest)
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_stage + staging_bytes(p.stage_bufs));
  uint64_t* bar_full = bars;
  uint64_t* bar_empty = bars + 4;
  uint64_t* bar_acc_full = bars + 8;
  uint64_t* bar_acc_empty = bars + 10;
  uint64_t* bar_res = bars + 12;
  uint64_t* bar_empty_first = bars + 20;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 24);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* epi_go = abort_flag + 1;         // per group two slots: the leader's go/stop verdict per tile

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // Warp 0 initialises the barriers and goes straight on to load; everybody else also waits for
  // the TMEM allocation (which the producer does not need).
  if (warp == 0) {
    // barrier slots in memory order: 4 group full (3 arrivals: the three producers), 4 group empty (one
    // commit by the MMA thread), 2 accumulator full, 2 accumulator empty (one arrival per epilogue
    // warp), 8 residual (one arrival with bytes), 4 first-k-block empty (one commit); lane i
    // initialises slot i
    if (lane < 24) {
      const uint32_t count = (lane < 4) ? 3u : (lane < 10) ? 1u : (lane < 12) ? (uint32_t)(4 * kGroups) : 1u;
      mbar_init(&bars[lane], count);
    }
    if (lane == 0) {
      grid_launch_dependents();  // the next grid in the stream may set itself up as SMs become free
      *abort_flag = 0;
    }
    __syncwarp();
    if (lane == 0) {
      mbar_fence_init();
      fence_proxy_async_smem();
    }
    __syncwarp();
    setup_bar_arrive();
  } else {
    if (warp == 1) {
      tmem_alloc(tmem_slot, kTmemCols);
      tmem_relinquish();
    }
    if (lane == 0) {  // tensor maps are fetched while thread 0 initialises the barriers
      if (warp == kFirstExtraProducerWarp) prefetch_tensormap(&tm_b);
      if (warp == kFirstExtraProducerWarp + 1) prefetch_tensormap(&tm_a);
      if (warp == 2) {
        prefetch_tensormap(&tm_y);
        prefetch_tensormap(&tm_y_tail);
        if (RES) {
          prefetch_tensormap(&tm_r);
          prefetch_tensormap(&tm_r_tail);
        }
      }
    }
    tc_fence_before();
    setup_bar_sync();
    tc_fence_after();
  }
  const uint32_t tmem_base = (warp == 0) ? 0u : *tmem_slot;

  if (warp == 0 || warp >= kFirstExtraProducerWarp) {
    // ------------------------------------------------------------------ TMA producers
    // (each a whole warp in lock step, one elected lane issuing: see the warp-wide forms)
    {
      const uint32_t full0 = smem_u32(bar_full), empty0 = smem_u32(bar_empty), ring0 = smem_u32(ring);
      if (warp == 0)
        producer_role<SPARSE, kRoleActFirst, FP8>(&tm_a, &tm_b, p, full0,
                                             p.ring_groups == 2 ? smem_u32(bar_empty_first) : empty0, ring0,
                                             smem_u32(bar_res), abort_flag);
      else if (warp == kFirstExtraProducerWarp)
        producer_role<SPARSE, kRoleActSecond, FP8>(&tm_a, &tm_b, p, full0, empty0, ring0, smem_u32(bar_res), abort_flag);
      else
        producer_role<SPARSE, kRoleWeights, FP8>(&tm_a, &tm_b, p, full0, empty0, ring0, smem_u32(bar_res), abort_flag);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // All 32 lanes run this loop in lock step and wait on the barriers together; the tcgen05
    // instructions are issued by one elected lane (see the warp-wide forms in sm100_ptx.cuh).
    {
      const uint32_t idesc = FP8 ? make_idesc_e4m3(kTileM, (uint32_t)p.BN, SPARSE)
                                 : make_idesc_bf16(kTileM, (uint32_t)p.BN, SPARSE);
      constexpr int kKb = C::kKbChannels;
      // descriptor address units are 16 B
      const uint32_t grp_desc = (p.a_grp_bytes + 2u * (uint32_t)p.BN * 128u) >> 4;
      const uint32_t b_desc = ((uint32_t)p.BN * 128u) >> 4;
      const uint32_t ring_lo0 = desc_lo(smem_u32(ring));
      const uint32_t a_off_desc = p.a_grp_bytes >> 4;
      // resident weights (dense, bf16 only): the tile's k-blocks lie after the ring and arrive once
      const bool resident = !SPARSE && !FP8 && p.a_res_bytes != 0;
      const uint32_t res_lo0 = ring_lo0 + (uint32_t)p.ring_groups * grp_desc;
      bool ok = true;
      if (resident && !mbar_wait_bounded(&bar_res[0], 0u, abort_flag, kWaitLimitCycles)) ok = false;
      const uint32_t full0 = smem_u32(bar_full), empty0 = smem_u32(bar_empty);
      // With two ring slots the ring's depth bounds the main loop: the first k-block's activation
      // tile is then released on its own, so that its reload starts one k-block earlier.
      const uint32_t empty_first0 = smem_u32(bar_empty_first);
      const bool early_release = p.ring_groups == 2;
      const uint32_t meta_tmem0 = tmem_base + kMetaCol;
      // channels left in the last chunk decide how many MMAs its k-blocks need
      const int tail_c = p.C_in - (p.cblocks - 1) * kKb;
      const int mma_full = SPARSE ? 2 : 4;
      // channels per MMA: bf16 32 sparse / 16 dense, e4m3 64 / 32
      const int mma_tail = SPARSE ? ((tail_c + kKb / 2 - 1) / (kKb / 2)) : ((tail_c + kKb / 4 - 1) / (kKb / 4));
      const int tail_start = (tail_c == kKb) ? p.kblocks : (p.cblocks - 1) * p.taps;  // first k-block of the tail
      const int a_lean_end = tail_start >> 1;  // groups before this one hold two full k-blocks
      uint32_t g = 0, ph = 0;  // group slot and its phase parity
      uint32_t tcount = 0;
      uint32_t mslot = 0;
      WorkIter work(p);
      Segment seg;
      for (; ok && work.next(seg); ++tcount) {
        const uint32_t buf = tcount & 1u;
        const uint32_t aph = (tcount >> 1) & 1u;
        if (!mbar_wait_bounded(&bar_acc_empty[buf], aph ^ 1u, abort_flag, kWaitLimitCycles)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * kAccCol1;
        uint32_t accumulate = 0;
        // This thread's instruction stream paces the tensor pipe (its queue is shallow): per group
        // one wait, the MMAs, one commit, and as little else as possible.
        // The loop exists twice, with and without the early release, so that rings of more than two
        // slots pay no branch for it in this thread's instruction stream.
        auto run_groups = [&](auto early_tag) {
          constexpr bool kEarly = decltype(early_tag)::value;
          for (int a = seg.a0; a < seg.a1; ++a) {
            if (!mbar_wait_a(full0 + 8u * g, ph, abort_flag, kWaitLimitCycles)) { ok = false; break; }
            const uint32_t grp_lo = ring_lo0 + g * grp_desc;
            const uint32_t a_lo = resident ? res_lo0 + (uint32_t)a * ((2u * kATileBytes) >> 4) : grp_lo;
            const uint32_t b0_lo = grp_lo + a_off_desc;
            const uint32_t b1_lo = b0_lo + b_desc;
            if (SPARSE && FP8) {
              // two metadata images -> 8 TMEM columns: 2 per MMA of 64 dense columns; operand steps in
              // bytes as for bf16 (A 32 kept bytes, B 64 bytes per MMA)
              const uint32_t meta_tmem = meta_tmem0 + 8u * mslot;
              mslot ^= 1u;
              tc_cp_128x128b_w(meta_tmem, a_lo + (kATileBytes >> 4));
              tc_cp_128x128b_w(meta_tmem + 4u, a_lo + ((kATileBytes + (uint32_t)kMetaImageBytes) >> 4));
              const int n0 = (2 * a >= tail_start) ? mma_tail : mma_full;
              const int n1 = (2 * a + 1 >= p.kblocks) ? 0 : ((2 * a + 1 >= tail_start) ? mma_tail : mma_full);
              tc_mma_f8_sparse_w(d_tmem, a_lo, b0_lo, meta_tmem, idesc, accumulate);
              if (n0 > 1) tc_mma_f8_sparse_w(d_tmem, a_lo + 2u, b0_lo + 4u, meta_tmem + 2u, idesc, 1u);
              if (kEarly) tc_commit_w(empty_first0 + 8u * g);
              if (n1 > 0) tc_mma_f8_sparse_w(d_tmem, a_lo + 4u, b1_lo, meta_tmem + 4u, idesc, 1u);
              if (n1 > 1) tc_mma_f8_sparse_w(d_tmem, a_lo + 6u, b1_lo + 4u, meta_tmem + 6u, idesc, 1u);
            } else if (SPARSE) {
              // metadata image -> 4 TMEM columns: 2 per k-block.  Kept values of the second k-block
              // start 64 B into the tile's rows; per MMA A advances 16 kept values = 32 B, B 32
              // channels = 64 B (descriptor units of 16 B).
              const uint32_t meta_tmem = meta_tmem0 + 4u * mslot;
              mslot ^= 1u;
              tc_cp_128x128b_w(meta_tmem, a_lo + (kATileBytes >> 4));
              if (a < a_lean_end) {
                tc_mma_sparse_w(d_tmem, a_lo, b0_lo, meta_tmem, idesc, accumulate);
                tc_mma_sparse_w(d_tmem, a_lo + 2u, b0_lo + 4u, meta_tmem, idesc | 1u, 1u);
                if (kEarly) tc_commit_w(empty_first0 + 8u * g);
                tc_mma_sparse_w(d_tmem, a_lo + 4u, b1_lo, meta_tmem + 2u, idesc, 1u);
                tc_mma_sparse_w(d_tmem, a_lo + 6u, b1_lo + 4u, meta_tmem + 2u, idesc | 1u, 1u);
              } else {
                const int n0 = (2 * a >= tail_start) ? mma_tail : mma_full;
                const int n1 = (2 * a + 1 >= p.kblocks) ? 0 : ((2 * a + 1 >= tail_start) ? mma_tail : mma_full);
                tc_mma_sparse_w(d_tmem, a_lo, b0_lo, meta_tmem, idesc, accumulate);
                if (n0 > 1) tc_mma_sparse_w(d_tmem, a_lo + 2u, b0_lo + 4u, meta_tmem, idesc | 1u, 1u);
                if (kEarly) tc_commit_w(empty_first0 + 8u * g);
                if (n1 > 0) tc_mma_sparse_w(d_tmem, a_lo + 4u, b1_lo, meta_tmem + 2u, idesc, 1u);
                if (n1 > 1) tc_mma_sparse_w(d_tmem, a_lo + 6u, b1_lo + 4u, meta_tmem + 2u, idesc | 1u, 1u);
              }
            } else if (p.small_c) {
              // chunked operands (see producer_role): chunk stride 2048 B for the weights, 16 BN for the
              // activations; an MMA takes two chunks (K = 16) of each
              const uint32_t a_ns = (a_lo & 0xFFFFu) | (128u << 16);
              const uint32_t b_ns = (b0_lo & 0xFFFFu) | ((uint32_t)p.BN << 16);
  #pragma unroll 1
              for (int kb = 0; kb < 2; ++kb) {
                int left_taps = p.taps - (16 * a + 8 * kb);
                left_taps = left_taps < 0 ? 0 : (left_taps > 8 ? 8 : left_taps);
                const int n_mma = (left_taps + 1) >> 1;
                for (int i = 0; i < n_mma; ++i) {
                  tc_mma_dense_w(d_tmem, a_ns + (uint32_t)kb * (kATileBytes >> 4) + (uint32_t)i * 256u,
                                 b_ns + (uint32_t)kb * b_desc + (uint32_t)i * (uint32_t)(2 * p.BN), idesc, accumulate,
                                 kDescHiNoSwizzle128);
                  accumulate = 1;
                }
                if (kEarly && kb == 0) tc_commit_w(empty_first0 + 8u * g);
              }
            } else if (FP8) {
              const uint32_t a1_lo = a_lo + (kATileBytes >> 4);
              const int n0 = (2 * a >= tail_start) ? mma_tail : mma_full;
              const int n1 = (2 * a + 1 >= p.kblocks) ? 0 : ((2 * a + 1 >= tail_start) ? mma_tail : mma_full);
              for (int kk = 0; kk < n0; ++kk)
                tc_mma_f8_dense_w(d_tmem, a_lo + 2u * kk, b0_lo + 2u * kk, idesc, (kk > 0) ? 1u : accumulate);
              if (kEarly) tc_commit_w(empty_first0 + 8u * g);
              for (int kk = 0; kk < n1; ++kk) tc_mma_f8_dense_w(d_tmem, a1_lo + 2u * kk, b1_lo + 2u * kk, idesc, 1u);
            } else {
              const uint32_t a1_lo = a_lo + (kATileBytes >> 4);
              if (a < a_lean_end) {
                tc_mma_dense_w(d_tmem, a_lo, b0_lo, idesc, accumulate);
                tc_mma_dense_w(d_tmem, a_lo + 2u, b0_lo + 2u, idesc, 1u);
                tc_mma_dense_w(d_tmem, a_lo + 4u, b0_lo + 4u, idesc, 1u);
                tc_mma_dense_w(d_tmem, a_lo + 6u, b0_lo + 6u, idesc, 1u);
                if (kEarly) tc_commit_w(empty_first0 + 8u * g);
                tc_mma_dense_w(d_tmem, a1_lo, b1_lo, idesc, 1u);
                tc_mma_dense_w(d_tmem, a1_lo + 2u, b1_lo + 2u, idesc, 1u);
                tc_mma_dense_w(d_tmem, a1_lo + 4u, b1_lo + 4u, idesc, 1u);
                tc_mma_dense_w(d_tmem, a1_lo + 6u, b1_lo + 6u, idesc, 1u);
              } else {
                const int n0 = (2 * a >= tail_start) ? mma_tail : mma_full;
                const int n1 = (2 * a + 1 >= p.kblocks) ? 0 : ((2 * a + 1 >= tail_start) ? mma_tail : mma_full);
                for (int kk = 0; kk < n0; ++kk)
                  tc_mma_dense_w(d_tmem, a_lo + 2u * kk, b0_lo + 2u * kk, idesc, (kk > 0) ? 1u : accumulate);
                if (kEarly) tc_commit_w(empty_first0 + 8u * g);
                for (int kk = 0; kk < n1; ++kk) tc_mma_dense_w(d_tmem, a1_lo + 2u * kk, b1_lo + 2u * kk, idesc, 1u);
              }
            }
            accumulate = 1;
            tc_commit_w(empty0 + 8u * g);
            if (++g == (uint32_t)p.ring_groups) {
              g = 0;
              ph ^= 1u;
            }
          }
        };
        if (early_release) run_groups(std::true_type{}); else run_groups(std::false_type{});
        if (ok) tc_commit_w(smem_u32(&bar_acc_full[buf]));
      }
    }
  } else if (warp < kFirstExtraProducerWarp) {
    // ------------------------------------------------------------------ epilogue
    // Two independent groups of four warps; group g owns positions [g BN/2, (g + 1) BN/2) of every
    // tile, with its own staging buffers and named barrier, and handles them 40 at a time (the last
    // piece of a group may hold fewer).
    const int grp = (warp - 2) >> 2;
    const int q = warp & 3;  // TMEM lane quadrant this warp may read: channels [32 q, 32 q + 32) of the tile
    const int gtid = q * 32 + lane;
    const bool leader = (q == 2 && lane == 0);  // first warp of each group
    const int act = activation_of(p.flags);
    const int col_base = grp * (p.BN >> 1);
    const uint32_t nbuf = (uint32_t)p.stage_bufs;  // 2 or 4
    const uint32_t nbuf_shift = nbuf == 4 ? 2u : 1u;
    uint8_t* my_stage = out_stage + grp * nbuf * kPieceBytes;
    volatile int* my_go = epi_go + 2 * grp;
    // stmatrix duty of this thread: 16 bytes = 8 channels of block (lane / 8) of the warp's four, at
    // position (lane % 8) of each run of 8 positions; the 16-byte chunks of a 128-byte staging row
    // are permuted by the row number (the swizzle the TMA store undoes)
    const uint32_t st_offset = (uint32_t)(q >> 1) * kHalfPieceBytes + (uint32_t)(lane & 7) * 128u +
                               ((((uint32_t)(q & 1) * 4u + (uint32_t)(lane >> 3)) ^ (uint32_t)(lane & 7)) << 4);
    uint32_t tcount = 0;
    uint32_t piece_count = 0;
    grid_dependency_wait();  // before the first access to global memory (bias, scratch, output)
    // Residual pieces are brought into the staging buffers by TMA, nbuf - 1 pieces ahead of the
    // epilogue (they come from HBM: one piece of latency would be exposed on every piece).  The
    // leader walks the same sequence of pieces with an iterator of its own.
    PieceAhead ahead(p);
    auto load_residual = [&](uint32_t count) {  // leader only; count = running number of the piece to load
      int tile_a, piece_a;
      if (!ahead.next(tile_a, piece_a)) return;  // no such piece: nobody will wait for it
      const uint32_t b = count & (nbuf - 1u);
      const uint32_t bar = smem_u32(&bar_res[4 * grp + b]);
      const int pt_a = tile_a / p.m_tiles;
      const int m_a = tile_a - pt_a * p.m_tiles;
      const int q_piece = pt_a * p.BN + col_base + piece_a * kPiece;
      if (q_piece >= p.Q) {  // nothing of this piece is stored: only keep the barrier's phases in step
        mbar_arrive_a(bar);
        return;
      }
      const bool tail = (piece_a == p.pieces - 1 && p.tail_cols != kPiece);
      const CUtensorMap* map = tail ? &tm_r_tail : &tm_r;
      const uint32_t half_bytes = (uint32_t)(tail ? p.tail_cols : kPiece) * 128u;
      const bool two = m_a * kTileM + 64 < p.C_out;
      const uint32_t dst = smem_u32(my_stage + b * kPieceBytes);
      mbar_expect_tx_a(bar, two ? 2u * half_bytes : half_bytes);
      tma_load_2d_a(dst, map, bar, m_a * kTileM, q_piece);
      if (two) tma_load_2d_a(dst + kHalfPieceBytes, map, bar, m_a * kTileM + 64, q_piece);
    };
    if (RES && leader)
      for (uint32_t c = 0; c + 1 < nbuf; ++c) load_residual(c);
    WorkIter work(p);
    Segment seg;
    for (; work.next(seg); ++tcount) {
      const int pt = seg.tile / p.m_tiles;
      const int m = seg.tile - pt * p.m_tiles;
      const uint32_t buf = tcount & 1u;
      const uint32_t aph = (tcount >> 1) & 1u;
      const bool got = mbar_wait_bounded(&bar_acc_full[buf], aph, abort_flag, kWaitLimitCycles, 64);
      // All threads of a group must take the same branch (they meet at named barriers below):
      // the leader publishes one verdict, everybody reads it after the barrier.
      if (leader) my_go[tcount & 1u] = (got && *abort_flag == 0) ? 1 : 0;
      epilogue_bar_sync(grp);
      if (my_go[tcount & 1u] == 0) break;
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kAccCol1 + col_base;
      const bool whole = (seg.a0 == 0 && seg.a1 == p.a_tiles);
      if (!whole) {
        // ---- partial tile: park this CTA's share in its own scratch region; the finishing kernel
        // sums the shares of all contributors
        float4* mine = p.ws_regions + region_index(blockIdx.x, seg.a0 == 0) * kRegionVecs;
#pragma unroll 1
        for (int piece = 0; piece < p.pieces; ++piece) {  // (a short last piece is parked whole)
          uint32_t r[kPiece];
          tc_ld_piece(t_row + piece * kPiece, r);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < kPiece / 4; ++j)
            __stcg(mine + region_vec(grp, piece, j, gtid),
                   make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                               __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3])));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
        continue;
      }
      // ---- finish the tile: bias, activation, bf16, transposed staging, TMA stores ---------------
      // the four channels whose accumulators this thread receives: 8 i + lane / 4 of the warp's 32
      float bias_v[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int co = m * kTileM + q * 32 + 8 * i + (lane >> 2);
        bias_v[i] = ((p.flags & SSCONV_FLAG_BIAS) && co < p.C_out) ? p.bias[co] : 0.0f;
      }
#pragma unroll 1
      for (int piece = 0; piece < p.pieces; ++piece, ++piece_count) {
        const uint32_t sbuf = piece_count & (nbuf - 1u);
        uint8_t* stage = my_stage + sbuf * kPieceBytes;
        uint32_t r[kPiece];
        // (a short last piece still reads and stages 40 columns; the surplus is never stored)
        tc_ld_piece(t_row + piece * kPiece, r);
        tc_wait_ld();
        if (piece == p.pieces - 1) {
          // this warp's part of the accumulator is read: hand it back to the MMA thread
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
        }
        // The buffer was last the source of the store issued two pieces ago; the leader saw that
        // store finish reading before it entered the barrier of the previous piece.
        const uint32_t st_addr = smem_u32(stage) + st_offset;
        if (FP8) {  // the accumulators are sums of products of quantised values: undo the operands' scales
#pragma unroll
          for (int i = 0; i < kPiece; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * p.out_scale);
        }
        if (RES) {
          // the residual piece has landed in this buffer (a wait that runs out raises the abort flag;
          // the group still goes on to its barrier and stops at the next tile)
          mbar_wait_bounded(&bar_res[4 * grp + sbuf], (piece_count >> nbuf_shift) & 1u, abort_flag, kWaitLimitCycles);
          if (act == kActRelu)
            stage_piece<kActRelu, true>(r, bias_v, st_addr);
          else if (act == kActGelu)
            stage_piece<kActGelu, true>(r, bias_v, st_addr);
          else
            stage_piece<kActNone, true>(r, bias_v, st_addr);
        } else if (act == kActRelu) {
          stage_piece<kActRelu, false>(r, bias_v, st_addr);
        } else if (act == kActGelu) {
          stage_piece<kActGelu, false>(r, bias_v, st_addr);
        } else {
          stage_piece<kActNone, false>(r, bias_v, st_addr);
        }
        fence_proxy_async_smem();  // generic-proxy writes -> visible to the TMA store
        // Without a residual the next piece overwrites the other buffer: its store (the previous
        // piece's) must have read it.  With one, the buffers are refilled by the residual loads
        // below, which wait for the stores themselves.
        if (leader && !RES) bulk_wait_group_read0();
        epilogue_bar_sync(grp);
        if (leader) {
          const int q_piece = pt * p.BN + col_base + piece * kPiece;
          if (q_piece < p.Q) {
            // positions beyond Q and channels beyond C_out fall outside the tensor map and are dropped;
            // a short last piece goes through the map whose box holds just its positions
            const CUtensorMap* map = (piece == p.pieces - 1 && p.tail_cols != kPiece) ? &tm_y_tail : &tm_y;
            tma_store_2d(map, stage, m * kTileM, q_piece);
            if (m * kTileM + 64 < p.C_out) tma_store_2d(map, stage + kHalfPieceBytes, m * kTileM + 64, q_piece);
          }
          bulk_commit_group();
          if (RES) {
            // refill the buffer the previous piece's store read: residual piece (count + nbuf - 1)
            bulk_wait_group_read1();
            load_residual(piece_count + nbuf - 1u);
          }
        }
      }
    }
    // the stores have read their staging buffers before shared memory is released; the writes
    // themselves complete with the grid
    if (leader) bulk_wait_group_read0();
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag != 0) {
    // give copies and MMAs still in flight time to land before shared memory and TMEM go away
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    if (threadIdx.x == 0 && p.dev_status != nullptr) atomicExch(p.dev_status, (int)SSCONV_ERR_TIMEOUT);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------
// Finishing kernel of the split-K path
// ---------------------------------------------------------------------------------------
// One CTA of 128 threads finishes 128 channels x 8 positions of one split tile: thread gtid sums,
// in CTA order, the two float4s it would have held in the main kernel's epilogue (fragment
// layout, see region_vec), applies bias / ReLU / bf16, and the block is transposed through shared
// memory by stmatrix.trans exactly as in the main kernel before 16-byte stores write NHWC.
struct FinishParams {
  int C_out, Q;
  int BN, pieces, tail_cols;  // the main kernel's tile width and epilogue pieces per group
  int m_tiles, a_tiles;
  int work_quot, work_rem;  // the main kernel's dealing of (tile, group) units to its CTAs
  const float4* ws_regions;
  uint32_t flags;
  const float* bias;
  const __nv_bfloat16* residual;  // nullable
  __nv_bfloat16* y;
  int y_pitch;  // elements between consecutive positions of y (and of the residual): C_out, or more for a channel slice
};
constexpr int kFinishThreads = 128;
// work items per tile: epilogue groups x pieces per group x blocks of 8 positions per piece
__host__ __device__ constexpr int finish_items_per_tile(int pieces) { return kGroups * pieces * (kPiece / 8); }
constexpr int kFinishBatch = 8;  // contributors whose loads are in flight together

__global__ void __launch_bounds__(kFinishThreads) ssconv_split_finish_kernel(const FinishParams f) {
  __shared__ __align__(128) uint8_t stage[8 * 256];  // [position][128 channels], 16-byte chunks permuted per row
  const int gtid = threadIdx.x, lane = gtid & 31, q = gtid >> 5;
  int item = blockIdx.x;
  const int k = item % (kPiece / 8);
  item /= (kPiece / 8);
  const int piece = item % f.pieces;
  item /= f.pieces;
  const int grp = item % kGroups;
  const int tile = item / kGroups;
  if (gtid == 0) grid_launch_dependents();
  const uint32_t u_first = (uint32_t)tile * (uint32_t)f.a_tiles;
  const int c_first = unit_owner(u_first, f.work_quot, f.work_rem);
  const int c_last = unit_owner(u_first + f.a_tiles - 1, f.work_quot, f.work_rem);
  if (c_first == c_last) return;  // the tile was computed whole by one CTA, which also finished it
  if (piece == f.pieces - 1 && 8 * k >= f.tail_cols) return;  // beyond a short last piece
  const int pt = tile / f.m_tiles;
  const int m = tile - pt * f.m_tiles;
  grid_dependency_wait();  // the main kernel's partial tiles are complete and visible

  float4 acc0 = make_float4(0.f, 0.f, 0.f, 0.f), acc1 = acc0;
  const int at0 = region_vec(grp, piece, k, gtid);               // lanes 0-15 of the warp's quadrant
  const int at1 = region_vec(grp, piece, kPiece / 8 + k, gtid);  // lanes 16-31
  for (int c0 = c_first; c0 <= c_last; c0 += kFinishBatch) {
    float4 v0[kFinishBatch], v1[kFinishBatch];
#pragma unroll
    for (int i = 0; i < kFinishBatch; ++i) {
      const int c = c0 + i;
      if (c <= c_last) {
        const float4* src = f.ws_regions + region_index(c, c == c_first) * kRegionVecs;
        v0[i] = __ldcg(src + at0);
        v1[i] = __ldcg(src + at1);
      }
    }
#pragma unroll
    for (int i = 0; i < kFinishBatch; ++i) {
      if (c0 + i <= c_last) {
        acc0.x += v0[i].x; acc0.y += v0[i].y; acc0.z += v0[i].z; acc0.w += v0[i].w;
        acc1.x += v1[i].x; acc1.y += v1[i].y; acc1.z += v1[i].z; acc1.w += v1[i].w;
      }
    }
  }
  float bias_v[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int co = m * kTileM + q * 32 + 8 * i + (lane >> 2);
    bias_v[i] = ((f.flags & SSCONV_FLAG_BIAS) && co < f.C_out) ? f.bias[co] : 0.0f;
  }
  // thread 8 i + j of a warp addresses position j of channel block i of the warp's four
  const uint32_t row = (uint32_t)(lane & 7);
  const uint32_t chunk = (uint32_t)(4 * q + (lane >> 3));
  const uint32_t st_addr = smem_u32(stage) + row * 256u + ((chunk ^ row) << 4);
  const int pos = gtid >> 4, ch16 = gtid & 15;  // 16 threads cover the 256 contiguous bytes of one position
  const int q_pos = pt * f.BN + grp * (f.BN >> 1) + piece * kPiece + 8 * k + pos;
  const int co16 = m * kTileM + 8 * ch16;
  const bool in_range = q_pos < f.Q && co16 < f.C_out;
  if (f.residual != nullptr) {
    // residual block -> staging buffer (same layout), read back in fragment layout, added in fp32
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (in_range) v = *reinterpret_cast<const uint4*>(f.residual + (size_t)q_pos * f.y_pitch + co16);
    *reinterpret_cast<uint4*>(stage + pos * 256 + ((ch16 ^ pos) << 4)) = v;
    __syncthreads();
    uint32_t res[4];
    ldmatrix_x4_trans(st_addr, res);
    acc0.x += bf16_lo(res[0]); acc0.y += bf16_hi(res[0]); acc0.z += bf16_lo(res[1]); acc0.w += bf16_hi(res[1]);
    acc1.x += bf16_lo(res[2]); acc1.y += bf16_hi(res[2]); acc1.z += bf16_lo(res[3]); acc1.w += bf16_hi(res[3]);
  }
  uint32_t w[4];
  const float v[8] = {acc0.x + bias_v[0], acc0.y + bias_v[0], acc0.z + bias_v[1], acc0.w + bias_v[1],
                      acc1.x + bias_v[2], acc1.y + bias_v[2], acc1.z + bias_v[3], acc1.w + bias_v[3]};
  const int act = activation_of(f.flags);
#pragma unroll
  for (int i = 0; i < 4; ++i)
    w[i] = (act == kActRelu)   ? activate_pack<kActRelu>(v[2 * i], v[2 * i + 1])
           : (act == kActGelu) ? activate_pack<kActGelu>(v[2 * i], v[2 * i + 1])
                               : activate_pack<kActNone>(v[2 * i], v[2 * i + 1]);
  stmatrix_x4_trans(st_addr, w[0], w[1], w[2], w[3]);
  __syncthreads();
  if (in_range) {
    const uint4 v = *reinterpret_cast<const uint4*>(stage + pos * 256 + ((ch16 ^ pos) << 4));
    *reinterpret_cast<uint4*>(f.y + (size_t)q_pos * f.y_pitch + co16) = v;
  }
}


// ---------------------------------------------------------------------------------------
// Pair kernel: a tile of 256 output channels x BN positions on two CTAs (tcgen05 cta_group::2)
// ---------------------------------------------------------------------------------------
// What bounds the one-CTA kernel on compute-bound layers is shared-memory bandwidth: per k-block an
// SM writes its weight and activation tiles once (TMA) and the MMAs read them once, 17 KB + 256 BN
// bytes at about 140 bytes per cycle, against 240 cycles of sparse tensor time at BN = 240.  Two CTAs
// of a cluster sharing one MMA of M = 256 halve the activation part: each CTA loads and holds its own
// 128 weight rows (and their metadata) and only half of the tile's positions, and the tensor cores of
// both SMs read both halves.  Per CTA nothing else changes: its TMEM holds its 128 channels x BN
// positions, so the epilogue is the one-CTA kernel's.  Roles as there (three producer warps, one
// issuing warp, eight epilogue warps), except that only the even CTA of a pair (the leader) issues
// tcgen05.cp / mma / commit, for both.  Barriers: "full" lives in the leader and collects the bytes
// of both CTAs' loads (the peer's copies signal it directly, the leader announces the sum); "empty"
// and "accumulator full" exist in each CTA and the leader commits to both; "accumulator empty" lives
// in the leader and counts the epilogue warps of both CTAs.  No load is multicast: each CTA fetches
// what it needs itself.  Whole tiles only (no K split), no 8-channel mode.  RES: the fused residual, as in
// the one-CTA kernel (each CTA prefetches the residual pieces of its own channels into four staging buffers
// per epilogue group, on barriers of its own).
template <bool SPARSE, int ROLE, bool FP8 = false>
__device__ __forceinline__ void pair_producer_role(const CUtensorMap* tm_a, const CUtensorMap* tm_b,
                                                   const CUtensorMap* tm_meta, const FwdParams& p, uint32_t rank,
                                                   uint32_t pair, uint32_t full0_leader, uint32_t full0_local,
                                                   uint32_t empty0, uint32_t ring0, volatile int* abort_flag) {
  using C = Cfg<SPARSE, FP8>;
  constexpr int kKb = C::kKbChannels;
  const uint32_t half_bytes = (uint32_t)(p.BN >> 1) * 128u;  // this CTA's half of an activation tile
  const uint32_t tiles_per = p.dual ? 2u : 1u;                // position tiles per work item
  const uint32_t grp_bytes = C::kAGroupBytes + 2u * tiles_per * half_bytes;
  const bool leader = rank == 0;
  uint32_t g = 0, ph = 0;
  bool ok = true;
  bool first_segment = true;
  WorkIter work(p, pair);
  Segment seg;
  while (ok && work.next(seg)) {
    const int pu = seg.tile / p.m_tiles;  // (m_tiles counts pairs of 128-channel tiles here)
    const int pt = pu * (int)tiles_per;   // the item's first position tile
    const int m = 2 * (seg.tile - pu * p.m_tiles) + (int)rank;
    const int m_meta = m < p.m_real ? m : p.m_real - 1;  // a CTA beyond the last channel tile multiplies zeros
    const Pos q0 = decode_pos(pt * p.BN + (int)rank * (p.BN >> 1), p.Wo, p.Ho);
    const int base_w = q0.c * p.stride_w - p.pad_w;
    const int base_h = q0.r * p.stride_h - p.pad_h;
    // second tile of the item (a tile past the last position reads zeros: its pixels lie outside the tensor)
    const Pos q1 = decode_pos((pt + 1) * p.BN + (int)rank * (p.BN >> 1), p.Wo, p.Ho);
    const int base_w1 = q1.c * p.stride_w - p.pad_w;
    const int base_h1 = q1.r * p.stride_h - p.pad_h;
    TapIter it;
    it.init(ROLE == kRoleActSecond ? 1 : 0, p);
    if (first_segment) {
      grid_dependency_wait();
      first_segment = false;
    }
    for (int a = 0; a < p.a_tiles; ++a) {
      if (!mbar_wait_a(empty0 + 8u * g, ph ^ 1u, abort_flag, kWaitLimitCycles)) { ok = false; break; }
      const uint32_t full = full0_leader + 8u * g;  // cluster address of the leader's barrier
      const uint32_t dst = ring0 + g * grp_bytes;
      const bool has_second = 2 * a + 1 < p.kblocks;
      if (ROLE == kRoleWeights) {
        if (SPARSE) {
          if (leader) mbar_expect_tx_w(full0_local + 8u * g, 2u * C::kAGroupBytes);
          tma2_load_2d_w(dst, tm_a, full, a * (FP8 ? 128 : 64), m * kTileM);  // 128 bytes of kept values per group
          tma2_load_2d_w(dst + kATileBytes, tm_meta, full, 0, (m_meta * p.a_tiles + a) * (int)(C::kMetaBytes / 16));
        } else {
          if (leader) mbar_expect_tx_w(full0_local + 8u * g, (has_second ? 4u : 2u) * kATileBytes);
          tma2_load_3d_w(dst, tm_a, full, it.cc * kKb, it.tap, m * kTileM);
          it.advance(p);
          if (has_second) tma2_load_3d_w(dst + kATileBytes, tm_a, full, it.cc * kKb, it.tap, m * kTileM);
          it.advance(p);
        }
      } else if (ROLE == kRoleActFirst || has_second) {
        if (leader) mbar_expect_tx_w(full0_local + 8u * g, 2u * tiles_per * half_bytes);
        const uint32_t b_dst = dst + C::kAGroupBytes + (ROLE == kRoleActSecond ? half_bytes : 0u);
        tma2_load_im2col_4d_w(b_dst, tm_b, full, it.cc * kKb, base_w, base_h, q0.n, (uint16_t)it.off_w, (uint16_t)it.off_h);
        if (p.dual)
          tma2_load_im2col_4d_w(b_dst + 2u * half_bytes, tm_b, full, it.cc * kKb, base_w1, base_h1, q1.n,
                                (uint16_t)it.off_w, (uint16_t)it.off_h);
        it.advance(p);
        it.advance(p);
      } else if (leader) {
        mbar_arrive_w(full0_local + 8u * g);  // the group has no second k-block: only keep the barrier's count
      }
      if (++g == (uint32_t)p.ring_groups) {
        g = 0;
        ph ^= 1u;
      }
    }
  }
}

template <bool SPARSE, bool FP8 = false, bool RES = false>
__global__ void __launch_bounds__(kThreads, 1)
ssconv_fwd_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                       const __grid_constant__ CUtensorMap tm_meta, const __grid_constant__ CUtensorMap tm_y,
                       const __grid_constant__ CUtensorMap tm_y_tail, const __grid_constant__ CUtensorMap tm_r,
                       const __grid_constant__ CUtensorMap tm_r_tail, const FwdParams p) {
  using C = Cfg<SPARSE, FP8>;
  static_assert(!FP8 || SPARSE, "the pair kernel takes 8-bit operands only in the 2:4 form");
  static_assert(!(FP8 && RES), "the residual epilogue is not built for 8-bit operands");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t half_bytes = (uint32_t)(p.BN >> 1) * 128u;
  const uint32_t grp_bytes = C::kAGroupBytes + (p.dual ? 4u : 2u) * half_bytes;
  uint8_t* ring = smem;
  uint8_t* out_stage = ring + p.ring_groups * grp_bytes;
  // barrier slots: [0,4) group full (used in the leader), [4,8) group empty, [8,10) accumulator full,
  // [10,12) accumulator empty (used in the leader), [12,20) residual piece landed (per epilogue group and
  // staging buffer, each block its own)
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_stage + staging_bytes(p.stage_bufs));
  uint64_t* bar_full = bars;
  uint64_t* bar_empty = bars + 4;
  uint64_t* bar_acc_full = bars + 8;
  uint64_t* bar_acc_empty = bars + 10;
  uint64_t* bar_res = bars + 12;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 20);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* epi_go = abort_flag + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t pair = blockIdx.x >> 1;
  const bool leader_cta = rank == 0;

  if (warp == 0) {
    if (lane < 20) {
      // full: the leader's three producers; empty, accumulator full: one commit; accumulator empty: the
      // epilogue warps of both CTAs; residual: one arrival with bytes
      const uint32_t count = (lane < 4) ? 3u : (lane < 10) ? 1u : (lane < 12) ? (uint32_t)(2 * 4 * kGroups) : 1u;
      mbar_init(&bars[lane], count);
    }
    if (lane == 0) {
      grid_launch_dependents();
      *abort_flag = 0;
    }
    __syncwarp();
    if (lane == 0) {
      mbar_fence_init();
      fence_proxy_async_smem();
    }
  } else if (warp == 1) {
    tmem_alloc2(tmem_slot, kTmemCols);
    tmem_relinquish2();
  } else if (lane == 0) {
    if (warp == kFirstExtraProducerWarp) prefetch_tensormap(&tm_b);
    if (warp == kFirstExtraProducerWarp + 1) {
      prefetch_tensormap(&tm_a);
      if (SPARSE) prefetch_tensormap(&tm_meta);
    }
    if (warp == 2) {
      prefetch_tensormap(&tm_y);
      prefetch_tensormap(&tm_y_tail);
      if (RES) {
        prefetch_tensormap(&tm_r);
        prefetch_tensormap(&tm_r_tail);
      }
    }
  }
  // both CTAs' barriers and TMEM exist before either touches the other's
  tc_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 || warp >= kFirstExtraProducerWarp) {
    // ------------------------------------------------------------------ TMA producers (whole warps)
    const uint32_t full0_local = smem_u32(bar_full);
    const uint32_t full0_leader = map_to_cta(full0_local, 0);
    const uint32_t empty0 = smem_u32(bar_empty), ring0 = smem_u32(ring);
    if (warp == 0)
      pair_producer_role<SPARSE, kRoleActFirst, FP8>(&tm_a, &tm_b, &tm_meta, p, rank, pair, full0_leader, full0_local, empty0,
                                                ring0, abort_flag);
    else if (warp == kFirstExtraProducerWarp)
      pair_producer_role<SPARSE, kRoleActSecond, FP8>(&tm_a, &tm_b, &tm_meta, p, rank, pair, full0_leader, full0_local,
                                                 empty0, ring0, abort_flag);
    else
      pair_producer_role<SPARSE, kRoleWeights, FP8>(&tm_a, &tm_b, &tm_meta, p, rank, pair, full0_leader, full0_local, empty0,
                                               ring0, abort_flag);
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (leader_cta) {
      const uint32_t idesc = FP8 ? make_idesc_e4m3(2 * kTileM, (uint32_t)p.BN, SPARSE)
                                 : make_idesc_bf16(2 * kTileM, (uint32_t)p.BN, SPARSE);
      constexpr int kKb = C::kKbChannels;
      const uint32_t grp_desc = grp_bytes >> 4;
      const uint32_t half_desc = half_bytes >> 4;
      const uint32_t ring_lo0 = desc_lo(smem_u32(ring));
      const uint32_t full0 = smem_u32(bar_full);
      const uint32_t empty0 = smem_u32(bar_empty), accf0 = smem_u32(bar_acc_full);
      const uint32_t meta_tmem0 = tmem_base + kMetaCol;
      const int tail_c = p.C_in - (p.cblocks - 1) * kKb;
      const int mma_full = SPARSE ? 2 : 4;
      // channels per MMA: bf16 32 sparse / 16 dense, e4m3 64 sparse
      const int mma_tail = SPARSE ? ((tail_c + kKb / 2 - 1) / (kKb / 2)) : ((tail_c + 15) >> 4);
      const int tail_start = (tail_c == kKb) ? p.kblocks : (p.cblocks - 1) * p.taps;  // first k-block of the tail
      uint32_t g = 0, ph = 0, tcount = 0, mslot = 0;
      uint32_t ready = 0;  // the look-ahead saw the group in hand complete
      bool ok = true;
      WorkIter work(p, pair);
      Segment seg;
      const bool dual = p.dual != 0;
      const uint32_t tile1_desc = 2u * half_desc;  // the item's second tile lies behind the first one's two k-blocks
      for (; ok && work.next(seg); ++tcount) {
        // one accumulator per tile: alternating between the two buffers, or (two tiles per item) both at once
        const uint32_t buf = dual ? 0u : (tcount & 1u);
        const uint32_t aph = dual ? (tcount & 1u) : ((tcount >> 1) & 1u);
        if (!mbar_wait_bounded(&bar_acc_empty[buf], aph ^ 1u, abort_flag, kWaitLimitCycles)) { ok = false; break; }
        if (dual && !mbar_wait_bounded(&bar_acc_empty[1], aph ^ 1u, abort_flag, kWaitLimitCycles)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * kAccCol1;
        const uint32_t d_tmem1 = tmem_base + kAccCol1;
        uint32_t accumulate = 0;
        for (int a = 0; a < p.a_tiles; ++a) {
          if (!ready && !mbar_wait_a(full0 + 8u * g, ph, abort_flag, kWaitLimitCycles)) { ok = false; break; }
          {  // look ahead at the next group's barrier (the ring runs on across tiles) while this group's
             // MMAs are issued; the answer is used at the top of the next iteration
            const uint32_t g_next = (g + 1u == (uint32_t)p.ring_groups) ? 0u : g + 1u;
            ready = mbar_test_a(full0 + 8u * g_next, g_next == 0u ? ph ^ 1u : ph);
          }
          tc_fence_after();
          const uint32_t a_lo = ring_lo0 + g * grp_desc;
          const uint32_t b0_lo = a_lo + (C::kAGroupBytes >> 4);
          const uint32_t b1_lo = b0_lo + half_desc;
          const int n0 = (2 * a >= tail_start) ? mma_tail : mma_full;
          const int n1 = (2 * a + 1 >= p.kblocks) ? 0 : ((2 * a + 1 >= tail_start) ? mma_tail : mma_full);
          if (SPARSE && FP8) {
            // two metadata images -> 8 TMEM columns, 2 per MMA of 64 dense columns (as in the one-block kernel)
            const uint32_t meta_tmem = meta_tmem0 + 8u * mslot;
            mslot ^= 1u;
            tc2_cp_128x128b_w(meta_tmem, a_lo + (kATileBytes >> 4));
            tc2_cp_128x128b_w(meta_tmem + 4u, a_lo + ((kATileBytes + (uint32_t)kMetaImageBytes) >> 4));
            for (uint32_t t = 0; t < (dual ? 2u : 1u); ++t) {  // (the second tile: same weights and metadata)
              const uint32_t d = t ? d_tmem1 : d_tmem, tb = t * tile1_desc;
              tc2_mma_f8_sparse_w(d, a_lo, b0_lo + tb, meta_tmem, idesc, accumulate);
              if (n0 > 1) tc2_mma_f8_sparse_w(d, a_lo + 2u, b0_lo + tb + 4u, meta_tmem + 2u, idesc, 1u);
              if (n1 > 0) tc2_mma_f8_sparse_w(d, a_lo + 4u, b1_lo + tb, meta_tmem + 4u, idesc, 1u);
              if (n1 > 1) tc2_mma_f8_sparse_w(d, a_lo + 6u, b1_lo + tb + 4u, meta_tmem + 6u, idesc, 1u);
            }
          } else if (SPARSE) {
            const uint32_t meta_tmem = meta_tmem0 + 4u * mslot;
            mslot ^= 1u;
            tc2_cp_128x128b_w(meta_tmem, a_lo + (kATileBytes >> 4));
            tc2_mma_sparse_w(d_tmem, a_lo, b0_lo, meta_tmem, idesc, accumulate);
            if (n0 > 1) tc2_mma_sparse_w(d_tmem, a_lo + 2u, b0_lo + 4u, meta_tmem, idesc | 1u, 1u);
            if (n1 > 0) tc2_mma_sparse_w(d_tmem, a_lo + 4u, b1_lo, meta_tmem + 2u, idesc, 1u);
            if (n1 > 1) tc2_mma_sparse_w(d_tmem, a_lo + 6u, b1_lo + 4u, meta_tmem + 2u, idesc | 1u, 1u);
            if (dual) {  // the second tile: same weights and metadata
              const uint32_t c0_lo = b0_lo + tile1_desc, c1_lo = b1_lo + tile1_desc;
              tc2_mma_sparse_w(d_tmem1, a_lo, c0_lo, meta_tmem, idesc, accumulate);
              if (n0 > 1) tc2_mma_sparse_w(d_tmem1, a_lo + 2u, c0_lo + 4u, meta_tmem, idesc | 1u, 1u);
              if (n1 > 0) tc2_mma_sparse_w(d_tmem1, a_lo + 4u, c1_lo, meta_tmem + 2u, idesc, 1u);
              if (n1 > 1) tc2_mma_sparse_w(d_tmem1, a_lo + 6u, c1_lo + 4u, meta_tmem + 2u, idesc | 1u, 1u);
            }
          } else {
            const uint32_t a1_lo = a_lo + (kATileBytes >> 4);
            for (uint32_t t = 0; t < (dual ? 2u : 1u); ++t) {
              const uint32_t d = t ? d_tmem1 : d_tmem, tb = t * tile1_desc;
              for (int kk = 0; kk < n0; ++kk)
                tc2_mma_dense_w(d, a_lo + 2u * kk, b0_lo + tb + 2u * kk, idesc, (kk > 0) ? 1u : accumulate);
              for (int kk = 0; kk < n1; ++kk) tc2_mma_dense_w(d, a1_lo + 2u * kk, b1_lo + tb + 2u * kk, idesc, 1u);
            }
          }
          accumulate = 1;
          tc2_commit_both_w(empty0 + 8u * g);
          if (++g == (uint32_t)p.ring_groups) {
            g = 0;
            ph ^= 1u;
          }
        }
        if (ok) tc2_commit_both_w(accf0 + 8u * buf);
        if (ok && dual) tc2_commit_both_w(accf0 + 8u);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (as in the one-CTA kernel)
    const int grp = (warp - 2) >> 2;
    const int q = warp & 3;
    const bool leader = (q == 2 && lane == 0);
    const int act = activation_of(p.flags);
    const int col_base = grp * (p.BN >> 1);
    // one or two staging buffers per group (one where the K loop is long enough to hide the wait for the
    // previous piece's store, which then leaves room for another ring group)
    const bool one_buffer = p.stage_bufs == 1;
    const uint32_t nbuf = (uint32_t)p.stage_bufs;  // 1 or 2; 4 with a residual (pieces prefetched three ahead)
    uint8_t* my_stage = out_stage + grp * p.stage_bufs * kPieceBytes;
    volatile int* my_go = epi_go + 2 * grp;
    const uint32_t acc_empty0_leader = map_to_cta(smem_u32(bar_acc_empty), 0);
    const uint32_t st_offset = (uint32_t)(q >> 1) * kHalfPieceBytes + (uint32_t)(lane & 7) * 128u +
                               ((((uint32_t)(q & 1) * 4u + (uint32_t)(lane >> 3)) ^ (uint32_t)(lane & 7)) << 4);
    uint32_t tcount = 0, piece_count = 0, icount = 0;
    const uint32_t tiles_per = p.dual ? 2u : 1u;
    bool go_on = true;
    grid_dependency_wait();
    // Residual pieces come into the staging buffers by TMA, nbuf - 1 pieces ahead of the epilogue, as in the
    // one-block kernel; each block loads its own channels' pieces on its own barriers.
    PieceAhead ahead(p, pair);
    auto load_residual = [&](uint32_t count) {  // leader only; count = running number of the piece to load
      int tile_a, piece_a;
      if (!ahead.next(tile_a, piece_a)) return;
      const uint32_t b = count & (nbuf - 1u);
      const uint32_t bar = smem_u32(&bar_res[4 * grp + b]);
      const int pt_a = tile_a / p.m_tiles;
      const int m_a = 2 * (tile_a - pt_a * p.m_tiles) + (int)rank;
      const int q_piece = pt_a * p.BN + col_base + piece_a * kPiece;
      if (q_piece >= p.Q || m_a >= p.m_real) {  // nothing of this piece is stored: only keep the barrier's phases in step
        mbar_arrive_a(bar);
        return;
      }
      const bool tail = (piece_a == p.pieces - 1 && p.tail_cols != kPiece);
      const CUtensorMap* map = tail ? &tm_r_tail : &tm_r;
      const uint32_t half_res = (uint32_t)(tail ? p.tail_cols : kPiece) * 128u;
      const bool two = m_a * kTileM + 64 < p.C_out;
      const uint32_t dst = smem_u32(my_stage + b * kPieceBytes);
      mbar_expect_tx_a(bar, two ? 2u * half_res : half_res);
      tma_load_2d_a(dst, map, bar, m_a * kTileM, q_piece);
      if (two) tma_load_2d_a(dst + kHalfPieceBytes, map, bar, m_a * kTileM + 64, q_piece);
    };
    if (RES && leader)
      for (uint32_t c = 0; c + 1 < nbuf; ++c) load_residual(c);
    WorkIter work(p, pair);
    Segment seg;
    for (; go_on && work.next(seg); ++icount)
    for (uint32_t t = 0; t < tiles_per; ++t, ++tcount) {  // the item's tiles, one accumulator each
      const int pu = seg.tile / p.m_tiles;
      const int pt = pu * (int)tiles_per + (int)t;
      const int m = 2 * (seg.tile - pu * p.m_tiles) + (int)rank;
      const uint32_t buf = p.dual ? t : (icount & 1u);
      const uint32_t aph = p.dual ? (icount & 1u) : ((icount >> 1) & 1u);
      const bool got = mbar_wait_bounded(&bar_acc_full[buf], aph, abort_flag, kWaitLimitCycles, 64);
      if (leader) my_go[tcount & 1u] = (got && *abort_flag == 0) ? 1 : 0;
      epilogue_bar_sync(grp);
      if (my_go[tcount & 1u] == 0) {
        go_on = false;
        break;
      }
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kAccCol1 + col_base;
      const bool real = m < p.m_real;  // (the odd CTA of the last pair may have no channels at all)
      float bias_v[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int co = m * kTileM + q * 32 + 8 * i + (lane >> 2);
        bias_v[i] = ((p.flags & SSCONV_FLAG_BIAS) && co < p.C_out) ? p.bias[co] : 0.0f;
      }
#pragma unroll 1
      for (int piece = 0; piece < p.pieces; ++piece, ++piece_count) {
        const uint32_t sbuf = RES ? (piece_count & (nbuf - 1u)) : (one_buffer ? 0u : (piece_count & 1u));
        uint8_t* stage = my_stage + sbuf * kPieceBytes;
        uint32_t r[kPiece];
        tc_ld_piece(t_row + piece * kPiece, r);
        tc_wait_ld();
        if (piece == p.pieces - 1) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acc_empty0_leader + 8u * buf);
        }
        if (FP8) {
#pragma unroll
          for (int i = 0; i < kPiece; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * p.out_scale);
        }
        if (!RES && one_buffer) {  // the previous piece's store has read the buffer before anyone overwrites it
          if (leader) bulk_wait_group_read0();
          epilogue_bar_sync(grp);
        }
        const uint32_t st_addr = smem_u32(stage) + st_offset;
        if (RES) {
          // the residual piece has landed in this buffer (a wait that runs out raises the abort flag; the
          // group still goes on to its barrier and stops at the next tile)
          mbar_wait_bounded(&bar_res[4 * grp + sbuf], (piece_count >> 2) & 1u, abort_flag, kWaitLimitCycles);
          if (act == kActRelu)
            stage_piece<kActRelu, true>(r, bias_v, st_addr);
          else if (act == kActGelu)
            stage_piece<kActGelu, true>(r, bias_v, st_addr);
          else
            stage_piece<kActNone, true>(r, bias_v, st_addr);
        } else if (act == kActRelu) {
          stage_piece<kActRelu, false>(r, bias_v, st_addr);
        } else if (act == kActGelu) {
          stage_piece<kActGelu, false>(r, bias_v, st_addr);
        } else {
          stage_piece<kActNone, false>(r, bias_v, st_addr);
        }
        fence_proxy_async_smem();
        if (leader && !RES) bulk_wait_group_read0();
        epilogue_bar_sync(grp);
        if (leader) {
          const int q_piece = pt * p.BN + col_base + piece * kPiece;
          if (real && q_piece < p.Q) {
            const CUtensorMap* map = (piece == p.pieces - 1 && p.tail_cols != kPiece) ? &tm_y_tail : &tm_y;
            tma_store_2d(map, stage, m * kTileM, q_piece);
            if (m * kTileM + 64 < p.C_out) tma_store_2d(map, stage + kHalfPieceBytes, m * kTileM + 64, q_piece);
          }
          bulk_commit_group();
          if (RES) {
            // refill the buffer the previous piece's store read: residual piece (count + nbuf - 1)
            bulk_wait_group_read1();
            load_residual(piece_count + nbuf - 1u);
          }
        }
      }
    }
    if (leader) bulk_wait_group_read0();
  }

  // ------------------------------------------------------------------ teardown
  // Neither CTA may leave while the other can still signal its barriers or read its shared memory.
  tc_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  if (*abort_flag != 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    if (threadIdx.x == 0 && p.dev_status != nullptr) atomicExch(p.dev_status, (int)SSCONV_ERR_TIMEOUT);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, kTmemCols);
  }
}


// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn g_encode_tiled = nullptr;
static EncodeIm2colFn g_encode_im2col = nullptr;

static bool load_driver_entry_points() {
  if (g_encode_tiled && g_encode_im2col) return true;
  void* f1 = nullptr;
  void* f2 = nullptr;
  cudaDriverEntryPointQueryResult q1, q2;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f1, cudaEnableDefault, &q1) != cudaSuccess) return false;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f2, cudaEnableDefault, &q2) != cudaSuccess) return false;
  if (q1 != cudaDriverEntryPointSuccess || q2 != cudaDriverEntryPointSuccess || !f1 || !f2) return false;
  g_encode_tiled = reinterpret_cast<EncodeTiledFn>(f1);
  g_encode_im2col = reinterpret_cast<EncodeIm2colFn>(f2);
  return true;
}

static int out_extent(int in, int k, int stride, int pad, int dil) {
  int span = in + 2 * pad - dil * (k - 1) - 1;
  return span < 0 ? 0 : span / stride + 1;
}

// Scratch for partly computed tiles: two fp32 regions (128 x 240) per CTA.  The grid is one CTA per SM
// of the device the call runs on; this is only the largest grid the scratch size (which is fixed
// without looking at a device, see ssconv_sizes) provides for.
constexpr int kMaxWorkers = 192;
constexpr size_t kRegionBytes = (size_t)kTileM * kBN * sizeof(float);
// Cost model behind the choice of tile width and of splitting K (cycles, measured on B200).
// A k-block of 64 dense columns takes the longest of four things.  The issuing thread: per pair
// of k-blocks one wait (about 200 cycles even on a complete barrier), about 76 per tcgen05
// instruction (metadata copy, MMAs, commit) and some loop overhead: 365 per k-block sparse, 480
// dense, whatever the tile width BN.  The tensor pipe: MMAs of about 35 + 0.5 BN (sparse, two per
// k-block) or 5 + 0.49 BN (dense, four).  The fill of shared memory from L2: the weight tile's
// share plus 128 BN bytes of activations at 56 bytes per cycle and SM (a probe with all SMs
// loading reached 68; sweeps of forced tile widths over 27 layers fit 50-56 best).  The depth of
// the ring: see kblock_cycles (load latency of about 1000 cycles, fitted by the same sweeps).  An
// epilogue that nothing overlaps takes about 900 cycles per 40 positions of a group, and every
// parked partial tile costs the chip about 90 cycles of L2 traffic (123 KB written by the main
// kernel and read again by the finishing kernel).
constexpr double kFillBytesPerCycle = 56.0;
constexpr double kLoadLatencyCycles = 1000.0;
constexpr double kIssueSparse = 365.0, kIssueDense = 480.0;
constexpr double kEpiloguePieceCycles = 900.0;
constexpr double kCyclesPerParkedTile = 90.0;
constexpr double kSplitAdvantage = 1.1;  // split only if the model predicts at least this gain

static int ring_groups_for(uint32_t a_group_bytes, int BN, int stage_bufs) {
  // as many groups in the ring as fit beside the staging buffers, at most kMaxGroups
  const int n =
      (int)((kMaxSmemBytes - 1024 - kBarrierBytes - staging_bytes(stage_bufs)) / group_bytes(a_group_bytes, BN));
  return n > kMaxGroups ? kMaxGroups : n;
}

template <bool SPARSE>
static double kblock_cycles(int BN, int stage_bufs, bool steady_ring = true) {
  const double a_bytes = Cfg<SPARSE>::kAGroupBytes / 2.0;
  const double fill = (a_bytes + 128.0 * BN) / kFillBytesPerCycle;
  const double issue = SPARSE ? kIssueSparse : kIssueDense;
  const double pipe = SPARSE ? 2.0 * (35.0 + 0.5 * BN) + 11.0 : 4.0 * (5.0 + 0.49 * BN);
  // A ring slot is refilled only once both of its k-blocks are consumed, so a slot's cycle is its
  // MMAs plus the latency and transfer of its loads, and the ring completes one slot per
  // (that cycle / slots): wide tiles with two slots are bound by this.
  const int groups = ring_groups_for(Cfg<SPARSE>::kAGroupBytes, BN, stage_bufs);
  const double ring = (kLoadLatencyCycles + 2.0 * fill + 2.0 * issue) / (2.0 * (groups < 1 ? 1 : groups));
  double t = fill > issue ? fill : issue;
  t = t > pipe ? t : pipe;
  // (a CTA of a split layer works through a handful of groups per tile and never reaches that
  // steady state: forced split plans measured fastest at the widths the other three terms choose)
  return (steady_ring && ring > t) ? ring : t;
}

// Process-wide overrides of the planner (ssconv_tune): tile width (0 lets the model choose) and the
// use of the pair kernel.
int32_t wgrad_set_tuning(int32_t option, int32_t value);  // (wgrad.cu)
static int g_tune_bn = 0;
static int g_tune_resident = 1;  // 0: weights always travel through the ring
static int g_tune_pair = -1;  // -1: the model chooses; 0: never the pair kernel; 1: wherever it applies
static int g_tune_pair_dual = -1;  // pair kernel, two position tiles per work item: -1 the model, 0 never, 1 always
int32_t set_tuning(int32_t option, int32_t value) {
  if (option == SSCONV_TUNE_PAIR) {
    if (value < -1 || value > 1) return SSCONV_ERR_BAD_DESC;
    g_tune_pair = value;
    return SSCONV_OK;
  }
  if (option == SSCONV_TUNE_PAIR_TILES) {
    if (value < -1 || value > 1) return SSCONV_ERR_BAD_DESC;
    g_tune_pair_dual = value;
    return SSCONV_OK;
  }
  if (option == SSCONV_TUNE_RESIDENT_WEIGHTS) {
    if (value < 0 || value > 1) return SSCONV_ERR_BAD_DESC;
    g_tune_resident = value;
    return SSCONV_OK;
  }
  if (option == SSCONV_TUNE_TILE_POSITIONS) {
    if (value != 0 && (value < 48 || value > kBN || value % 16 != 0)) return SSCONV_ERR_BAD_DESC;
    g_tune_bn = value;
    return SSCONV_OK;
  }
  return wgrad_set_tuning(option, value);
}

// Tile width and partition of a layer.
struct Plan {
  int BN;
  bool split;
  double cost = 0.0;  // the model's cycles for the layer
  bool pair = false;  // 256-channel tiles on CTA pairs (ssconv_fwd_pair_kernel)
  bool dual = false;  // ... with two position tiles per work item
};
template <bool SPARSE>
static Plan plan_layer(long long Q, const Geometry& geo, int workers, bool force_split, int max_bn = kBN,
                       int stage_bufs = 2, bool allow_split = true) {
  if (force_split) return Plan{kBN, true};
  int min_bn = 48;
  if (g_tune_bn != 0 && g_tune_bn <= max_bn) max_bn = min_bn = g_tune_bn;
  Plan best{max_bn, false};
  double best_cost = 0.0;
  for (int BN = max_bn; BN >= min_bn; BN -= 16) {
    const long long tiles = ((Q + BN - 1) / BN) * geo.m_tiles;
    const long long per_cta = (tiles + workers - 1) / workers;
    const int pieces = (BN / 2 + kPiece - 1) / kPiece;
    // (with at most three groups per tile the ring never reaches its steady state: such layers are paced
    // by their output stream, and measured fastest at the width the other terms choose)
    const double cost = (double)per_cta * geo.kblocks * kblock_cycles<SPARSE>(BN, stage_bufs, geo.stages >= 4) +
                        pieces * kEpiloguePieceCycles;
    if (BN == max_bn || cost < 0.97 * best_cost) {  // a narrower tile has to earn its extra weight traffic
      best_cost = cost;
      best.BN = BN;
    }
  }
  best.cost = best_cost;
  // Even split of K ("stream-K"), when many SMs would still idle and K is deep: every CTA gets the
  // same number of groups; parked partial tiles cost L2 traffic in proportion to the tile width.
  const int a_tiles = geo.stages;
  if (a_tiles > 1 && allow_split) {
    Plan best_split{kBN, true};
    double best_split_cost = 0.0;
    for (int BN = max_bn; BN >= min_bn; BN -= 16) {
      const long long tiles = ((Q + BN - 1) / BN) * geo.m_tiles;
      const double units = (double)tiles * a_tiles;
      const double ctas = units < workers ? units : (double)workers;
      const int pieces = (BN / 2 + kPiece - 1) / kPiece;
      const double cost = units / ctas * 2.0 * kblock_cycles<SPARSE>(BN, stage_bufs, false) +
                          (ctas + tiles) * kCyclesPerParkedTile * (pieces * 2.0 * kPiece / kBN);
      if (BN == max_bn || cost < 0.97 * best_split_cost) {
        best_split_cost = cost;
        best_split.BN = BN;
      }
    }
    best_split.cost = best_split_cost;
    if (best_cost > kSplitAdvantage * best_split_cost) return best_split;
  }
  return best;
}

// Pair kernel: a CTA holds the group's weights and half of each activation tile.
// Staging buffers per epilogue group in the pair kernel: with a deep K (its loop hides the epilogue)
// one buffer, which leaves room for one more ring group at the widest tiles; two otherwise.
constexpr int kPairOneBufferKBlocks = 24;
static int pair_stage_bufs(int kblocks) { return kblocks >= kPairOneBufferKBlocks ? 1 : 2; }
static int pair_ring_groups_with(uint32_t a_group_bytes, int BN, int stage_bufs) {
  const int n = (int)((kMaxSmemBytes - 1024 - kBarrierBytes - staging_bytes(stage_bufs)) /
                      (a_group_bytes + (uint32_t)BN * 128u));
  return n > kMaxGroups ? kMaxGroups : n;
}
static int pair_ring_groups(uint32_t a_group_bytes, int BN, int kblocks) {
  return pair_ring_groups_with(a_group_bytes, BN, pair_stage_bufs(kblocks));
}
// Plan for the pair kernel (whole tiles of 256 channels x BN positions dealt out to workers / 2
// pairs), or BN = 0 where it does not apply.  Per k-block a CTA of a pair takes in its weights and
// 64 BN bytes of activations (at a fitted 48 bytes per cycle) and the issuing warp does the work of
// one CTA for two.  Measured on the ResNet-50 and ConvNeXt layer sets: layers with a deep K and
// several tiles per pair gain 1.2-1.5x; layers with fewer than 12 k-blocks are bound by their
// epilogues and output traffic, where two CTAs in lock step do worse than two independent ones
// (0.6-0.9x), and with about one tile per pair the fixed costs decide: neither kind is paired
// unless the override forces it.
constexpr double kFillBytesPerCyclePair = 48.0;
constexpr int kPairMinKBlocks = 12;
constexpr double kPairMinTilesPerPair = 1.25;  // counted at the widest tile
constexpr int kPairDualMinKBlocks = 48;
constexpr int kPairDualMaxBN = 192;
constexpr double kPairDualGain = 0.92;         // measured 0.88-0.95 where it applies
template <bool SPARSE>
static Plan plan_pair(long long Q, const Geometry& geo, int workers, bool forced) {
  Plan best{0, false};
  best.pair = true;
  const int pairs = workers / 2;
  if (geo.m_tiles < 2 || pairs < 1) return best;
  if (!forced && geo.kblocks < kPairMinKBlocks) return best;
  const int mp_tiles = (geo.m_tiles + 1) / 2;
  if (!forced && (double)(((Q + kBN - 1) / kBN) * mp_tiles) < kPairMinTilesPerPair * pairs) return best;
  int max_bn = kBN, min_bn = 64;
  if (g_tune_bn != 0) max_bn = min_bn = g_tune_bn < 64 ? 64 : g_tune_bn;
  const double a_bytes = Cfg<SPARSE>::kAGroupBytes / 2.0;
  const double issue = SPARSE ? kIssueSparse : kIssueDense;
  for (int BN = max_bn; BN >= min_bn; BN -= 16) {
    const int groups = pair_ring_groups(Cfg<SPARSE>::kAGroupBytes, BN, geo.kblocks);
    if (groups < 2) continue;
    const long long tiles = ((Q + BN - 1) / BN) * mp_tiles;
    const long long per_pair = (tiles + pairs - 1) / pairs;
    const int pieces = (BN / 2 + kPiece - 1) / kPiece;
    const double fill = (a_bytes + 64.0 * BN) / kFillBytesPerCyclePair;
    const double pipe = SPARSE ? 2.0 * (35.0 + 0.5 * BN) + 11.0 : 4.0 * (5.0 + 0.49 * BN);
    const double ring = (kLoadLatencyCycles + 2.0 * fill + 2.0 * issue) / (2.0 * groups);
    double t = fill > issue ? fill : issue;
    t = t > pipe ? t : pipe;
    t = t > ring ? t : ring;
    const double cost = (double)per_pair * geo.kblocks * t + pieces * kEpiloguePieceCycles;
    if (best.BN == 0 || cost < 0.97 * best.cost) {
      best.BN = BN;
      best.cost = cost;
    }
  }
  // Two position tiles per work item (the pair's ring group then holds the weights once and both tiles'
  // halves, one accumulator each): measured at batch 256 / 128 on the layer sets, it pays where K is deep,
  // the layer has at least two pairs of channel tiles and about one item per pair or more (3x3 512 channels
  // at 7x7: 37 -> 33 us; 3072 -> 768 at 7x7: 24.5 -> 22.7; 2048 -> 512 at 7x7, 32 k-blocks: no difference in
  // the stack) and costs elsewhere (one pair of channel tiles, 16 k-blocks, few items: 1.1-1.5x slower; the
  // dense form never gains).  Tiles of at most 192 positions, so that the ring keeps three groups.
  best.dual = false;
  if (best.BN != 0 && g_tune_pair_dual != 0 && best.BN <= kPairDualMaxBN) {
    const long long items = (((Q + best.BN - 1) / best.BN + 1) / 2) * mp_tiles;
    const bool pays = SPARSE && geo.kblocks >= kPairDualMinKBlocks && mp_tiles >= 2 && 4 * items >= 3 * (long long)pairs;
    if ((pays || g_tune_pair_dual == 1) && pair_ring_groups(Cfg<SPARSE>::kAGroupBytes, 2 * best.BN, geo.kblocks) >= 2) {
      best.dual = true;
      best.cost *= kPairDualGain;
    }
  }
  return best;
}
constexpr double kPairAdvantage = 1.05;  // the pair kernel only if the model predicts at least this gain

constexpr size_t scratch_bytes(int workers) {
  return 2 * (size_t)workers * kRegionBytes;
}
size_t workspace_bytes() { return scratch_bytes(kMaxWorkers); }

static int g_sm_count[64] = {0};
static bool g_attr_set[64][2][2] = {{{false}}};
static bool g_pair_attr_set[64][2] = {{false}};
static bool g_pair_res_attr_set[64][2] = {{false}};
static bool g_fp8_attr_set[64][2] = {{false}};
static bool g_pair_fp8_attr_set[64] = {false};

// Dense layers with 8 input channels (a channel-padded RGB stem): a k-block of 64 K-elements is 8
// filter taps instead of 64 channels of one tap, which would be 7/8 padding.
static bool small_channel_mode(const ssconv_desc_t& d, bool sparse) { return !sparse && d.C_in == 8; }
static Geometry layer_geometry(const ssconv_desc_t& d, bool sparse, bool fp8 = false) {
  Geometry g = make_geometry(d, fp8 ? 2 * kBlockK : kBlockK);
  if (small_channel_mode(d, sparse)) {
    g.kblocks = (g.taps + 7) / 8;
    g.kblocks_pad = (g.kblocks + 1) & ~1;
    g.stages = g.kblocks_pad / 2;
  }
  return g;
}

// Current device and its SM count (checked once per device: must be compute capability 10.x).
static int32_t current_device(int* dev_out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SSCONV_ERR_CUDA;
  if (g_sm_count[dev] == 0) {
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SSCONV_ERR_CUDA;
    if (major != 10) return SSCONV_ERR_ARCH;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
      return SSCONV_ERR_CUDA;
    g_sm_count[dev] = sms;
  }
  *dev_out = dev;
  return SSCONV_OK;
}

// Widest tile for which two groups fit beside the staging buffers.
static int widest_tile(uint32_t a_group_bytes, int stage_bufs) {
  int BN = kBN;
  while (BN > 48 && ring_groups_for(a_group_bytes, BN, stage_bufs) < 2) BN -= 16;
  return BN;
}

// The plan for a layer without a residual: one-CTA tiles (whole or K split) or the pair kernel.
template <bool SPARSE>
static Plan choose_plan(const ssconv_desc_t& d, long long Q, const Geometry& geo, int workers, bool force_split,
                        bool allow_split = true) {
  const Plan plan = plan_layer<SPARSE>(Q, geo, workers, force_split, kBN, 2, allow_split);
  if (force_split || small_channel_mode(d, SPARSE) || g_tune_pair == 0) return plan;
  const Plan pair = plan_pair<SPARSE>(Q, geo, workers, g_tune_pair == 1);
  if (pair.BN != 0 && (g_tune_pair == 1 || plan.cost > kPairAdvantage * pair.cost)) return pair;
  return plan;
}

int32_t plan_query_sms(const ssconv_desc_t& d, bool sparse, int sm_count, int32_t* bn, int32_t* split, int32_t* ctas,
                       int32_t* ring_groups, int32_t* pair);
// What launch_forward_impl would do for this layer on the current device.
int32_t plan_query(const ssconv_desc_t& d, bool sparse, int32_t* bn, int32_t* split, int32_t* ctas,
                   int32_t* ring_groups, int32_t* pair) {
  int dev = 0;
  const int32_t st = current_device(&dev);
  if (st != SSCONV_OK) return st;
  return plan_query_sms(d, sparse, g_sm_count[dev], bn, split, ctas, ring_groups, pair);
}
int32_t plan_query_sms(const ssconv_desc_t& d, bool sparse, int sm_count, int32_t* bn, int32_t* split, int32_t* ctas,
                       int32_t* ring_groups, int32_t* pair) {
  if (sm_count <= 0) return SSCONV_ERR_BAD_DESC;
  const Geometry geo = layer_geometry(d, sparse);
  const long long Q = (long long)d.N * out_extent(d.H, d.KH, d.stride_h, d.pad_h, d.dil_h) *
                      out_extent(d.W, d.KW, d.stride_w, d.pad_w, d.dil_w);
  const int workers = sm_count < kMaxWorkers ? sm_count : kMaxWorkers;
  const Plan plan = sparse ? choose_plan<true>(d, Q, geo, workers, false) : choose_plan<false>(d, Q, geo, workers, false);
  const uint32_t a_group_bytes = sparse ? Cfg<true>::kAGroupBytes : Cfg<false>::kAGroupBytes;
  const long long q_tiles = (Q + plan.BN - 1) / plan.BN;
  if (bn) *bn = plan.BN;
  if (pair) *pair = plan.pair ? 1 : 0;
  if (plan.pair) {
    const long long tiles = (plan.dual ? (q_tiles + 1) / 2 : q_tiles) * ((geo.m_tiles + 1) / 2);  // work items
    const long long pairs = workers / 2;
    if (split) *split = 0;
    if (ctas) *ctas = (int32_t)(2 * (tiles < pairs ? tiles : pairs));
    if (ring_groups) *ring_groups = pair_ring_groups(a_group_bytes, plan.dual ? 2 * plan.BN : plan.BN, geo.kblocks);
    return SSCONV_OK;
  }
  const long long tiles = q_tiles * geo.m_tiles;
  const bool do_split = plan.split && geo.stages > 1;
  const long long work = do_split ? tiles * geo.stages : tiles;
  if (split) *split = do_split ? 1 : 0;
  if (ctas) *ctas = (int32_t)(work < workers ? work : workers);
  if (ring_groups) *ring_groups = ring_groups_for(a_group_bytes, plan.BN, 2);
  return SSCONV_OK;
}

template <bool SPARSE, bool FP8 = false>
static int32_t launch_forward_impl(const ssconv_desc_t& d, const void* x, const void* weights, const void* meta,
                                   const float* bias, const void* residual, void* y, void* ws, size_t ws_bytes,
                                   int32_t* dev_status, cudaStream_t stream, int worker_cap = kMaxWorkers,
                                   bool force_split = false, const int64_t* x_strides = nullptr,
                                   float out_scale = 1.0f, int64_t y_pitch = 0) {
  using C = Cfg<SPARSE, FP8>;
  constexpr int kKb = C::kKbChannels;
  constexpr size_t kElem = FP8 ? 1 : 2;  // bytes per operand element
  constexpr CUtensorMapDataType kOperandType = FP8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  if (FP8 && residual != nullptr) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  const int64_t y_pitch_el = y_pitch > 0 ? y_pitch : d.C_out;
  if (!load_driver_entry_points()) return SSCONV_ERR_CUDA;
  int dev = 0;
  {
    const int32_t st = current_device(&dev);
    if (st != SSCONV_OK) return st;
  }
  for (int res = 0; res < 2; ++res) {
    if (g_attr_set[dev][SPARSE ? 1 : 0][res]) continue;
    const cudaError_t e = res ? cudaFuncSetAttribute(ssconv_fwd_kernel<SPARSE, true>,
                                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmemBytes)
                              : cudaFuncSetAttribute(ssconv_fwd_kernel<SPARSE, false>,
                                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmemBytes);
    if (e != cudaSuccess) return SSCONV_ERR_CUDA;
    g_attr_set[dev][SPARSE ? 1 : 0][res] = true;
  }
  if (FP8 && !g_fp8_attr_set[dev][SPARSE ? 1 : 0]) {
    if (cudaFuncSetAttribute(ssconv_fwd_kernel<SPARSE, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kMaxSmemBytes) != cudaSuccess)
      return SSCONV_ERR_CUDA;
    g_fp8_attr_set[dev][SPARSE ? 1 : 0] = true;
  }
  const Geometry geo = layer_geometry(d, SPARSE, FP8);
  const bool small_c = !FP8 && small_channel_mode(d, SPARSE);
  const int Ho = out_extent(d.H, d.KH, d.stride_h, d.pad_h, d.dil_h);
  const int Wo = out_extent(d.W, d.KW, d.stride_w, d.pad_w, d.dil_w);
  const long long Q = (long long)d.N * Ho * Wo;  // positions
  if (Q > 0x7FFFFF00LL) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  const int workers = g_sm_count[dev] < worker_cap ? g_sm_count[dev] : worker_cap;
  // With a residual the epilogue prefetches residual pieces three ahead into four staging buffers
  // per group, which narrows the widest tile that still leaves room for two ring groups.  (When K
  // is split the finishing kernel adds the residual to the split tiles; the main kernel then keeps
  // two buffers and one piece of lookahead for the whole tiles it may also own.)
  // Without a usable workspace the K range is not split: the best plan of whole tiles runs instead
  // (slower on layers with few tiles and a deep K, never wrong).
  const bool have_ws = !FP8 && ws != nullptr && ws_bytes >= scratch_bytes(worker_cap);  // (8-bit: whole tiles only)
  if (have_ws && (reinterpret_cast<uintptr_t>(ws) & 15u)) return SSCONV_ERR_ALIGNMENT;
  if (force_split && !have_ws) return SSCONV_ERR_WORKSPACE;
  // (8-bit operands: the pair kernel exists for the 2:4 form only; the dense counterpart stays on one-block tiles)
  Plan plan = (residual != nullptr || (FP8 && !SPARSE)) ? plan_layer<SPARSE>(Q, geo, workers, force_split, kBN, 2, have_ws)
                                                        : choose_plan<SPARSE>(d, Q, geo, workers, force_split, have_ws);
  int stage_bufs = 2;
  if (residual != nullptr && !plan.split) {
    stage_bufs = 4;
    plan = plan_layer<SPARSE>(Q, geo, workers, false, widest_tile(C::kAGroupBytes, 4), 4);
    if (plan.split) {  // the narrower limit made splitting look better: stay unsplit at the limit
      plan.split = false;
      plan.BN = widest_tile(C::kAGroupBytes, 4);
    }
    // The pair kernel takes a residual too (four staging buffers per group there as well): where its model
    // wins and the ring still holds two groups, one work item is one tile.
    if (!FP8 && !force_split && !small_c && g_tune_pair != 0) {
      Plan pp = plan_pair<SPARSE>(Q, geo, workers, g_tune_pair == 1);
      if (pp.BN != 0 && pair_ring_groups_with(C::kAGroupBytes, pp.BN, 4) >= 2 &&
          (g_tune_pair == 1 || plan.cost > kPairAdvantage * pp.cost)) {
        pp.dual = false;
        plan = pp;
      }
    }
  }
  const int BN = plan.BN;
  const int pieces = (BN / 2 + kPiece - 1) / kPiece;
  const int tail_cols = BN / 2 - (pieces - 1) * kPiece;
  const bool pair = plan.pair;  // a CTA of a pair holds half of each activation tile
  // Dense layers of one channel tile and at most four k-blocks (a stem run as a T x 1 convolution over 64
  // channels): every tile needs the same 16-64 KB of weights, which then stay in shared memory for the
  // life of the CTA instead of travelling through the ring with every tile; the groups hold activations
  // only, and more of them fit.
  const bool resident = !SPARSE && !FP8 && !small_c && !pair && !plan.split && residual == nullptr && geo.m_tiles == 1 &&
                        geo.kblocks <= 4 && g_tune_resident != 0;
  const uint32_t a_grp_bytes = resident ? 0u : C::kAGroupBytes;
  const uint32_t a_res_bytes = resident ? (uint32_t)geo.stages * 2u * kATileBytes : 0u;
  if (pair) stage_bufs = residual != nullptr ? 4 : pair_stage_bufs(geo.kblocks);
  // pair kernel: two neighbouring position tiles per work item share every group's weights (its ring group
  // then holds both tiles' halves) where that still leaves a ring of two groups
  const bool dual = pair && plan.dual && residual == nullptr && pair_ring_groups(C::kAGroupBytes, 2 * BN, geo.kblocks) >= 2;
  const uint32_t grp_bytes = pair ? C::kAGroupBytes + (dual ? 2u : 1u) * (uint32_t)BN * 128u : group_bytes(a_grp_bytes, BN);
  int ring_groups = pair ? pair_ring_groups_with(C::kAGroupBytes, dual ? 2 * BN : BN, stage_bufs)
                         : ring_groups_for(C::kAGroupBytes, BN, stage_bufs);
  if (resident) {
    ring_groups = (int)((kMaxSmemBytes - 1024 - kBarrierBytes - staging_bytes(stage_bufs) - a_res_bytes) / grp_bytes);
    if (ring_groups > kMaxGroups) ring_groups = kMaxGroups;
  }
  const uint32_t smem_bytes =
      1024 + (uint32_t)ring_groups * grp_bytes + a_res_bytes + staging_bytes(stage_bufs) + kBarrierBytes;
  if (pair && !FP8 && !g_pair_attr_set[dev][SPARSE ? 1 : 0]) {
    if (cudaFuncSetAttribute(ssconv_fwd_pair_kernel<SPARSE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kMaxSmemBytes) != cudaSuccess)
      return SSCONV_ERR_CUDA;
    g_pair_attr_set[dev][SPARSE ? 1 : 0] = true;
  }
  if (pair && !FP8 && residual != nullptr && !g_pair_res_attr_set[dev][SPARSE ? 1 : 0]) {
    if (cudaFuncSetAttribute(ssconv_fwd_pair_kernel<SPARSE, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kMaxSmemBytes) != cudaSuccess)
      return SSCONV_ERR_CUDA;
    g_pair_res_attr_set[dev][SPARSE ? 1 : 0] = true;
  }
  if (pair && FP8 && !g_pair_fp8_attr_set[dev]) {
    if (cudaFuncSetAttribute(ssconv_fwd_pair_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kMaxSmemBytes) != cudaSuccess)
      return SSCONV_ERR_CUDA;
    g_pair_fp8_attr_set[dev] = true;
  }

  CUtensorMap tm_a, tm_b, tm_y, tm_y_tail, tm_r, tm_r_tail;
  // activations: NHWC seen as (c, w, h, n), im2col mode; elements outside the image read as zero
  // (= the zero padding of Eq. 4); base pixels are the filter placements, each load adds a tap offset
  {
    cuuint64_t dims[4] = {(cuuint64_t)d.C_in, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.N};
    cuuint64_t strides[3] = {(cuuint64_t)d.C_in * kElem, (cuuint64_t)d.W * d.C_in * kElem,
                             (cuuint64_t)d.H * d.W * d.C_in * kElem};
    if (x_strides != nullptr)  // a strided (possibly overlapping) view: element strides of w, h, n
      for (int i = 0; i < 3; ++i) strides[i] = (cuuint64_t)x_strides[i] * kElem;
    int lower[2] = {-d.pad_w, -d.pad_h};
    int upper[2] = {d.pad_w - (d.KW - 1) * d.dil_w, d.pad_h - (d.KH - 1) * d.dil_h};
    cuuint32_t estr[4] = {1, (cuuint32_t)d.stride_w, (cuuint32_t)d.stride_h, 1};
    // (8-channel mode: 16-byte-wide unswizzled chunks, one per filter tap)
    // L2 fetches 256 bytes per miss where a pixel is at least that long and every pixel is read
    // (measured: up to 4 % faster on such layers, 4 % slower on a strided one, nothing elsewhere)
    const bool wide_pixels = d.C_in * kElem >= 256 && d.stride_h == 1 && d.stride_w == 1 && x_strides == nullptr;
    CUresult r = g_encode_im2col(&tm_b, kOperandType, 4, const_cast<void*>(x), dims, strides,
                                 lower, upper, small_c ? 8u : (cuuint32_t)kKb,
                                 (cuuint32_t)(pair ? BN / 2 : BN), estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE,
                                 small_c ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                                 wide_pixels ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return SSCONV_ERR_CUDA;
  }
  if (SPARSE) {
    // kept values: 64 bytes per row and k-block (KC counts 2-byte units); a box is 128 rows x 128 bytes
    cuuint64_t dims[2] = {(cuuint64_t)geo.KC * 2 / kElem, (cuuint64_t)geo.Mp};
    cuuint64_t strides[1] = {(cuuint64_t)geo.KC * 2};
    cuuint32_t box[2] = {(cuuint32_t)(128 / kElem), (cuuint32_t)kTileM};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode_tiled(&tm_a, kOperandType, 2, const_cast<void*>(weights), dims, strides,
                                box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return SSCONV_ERR_CUDA;
  } else {
    // dense weights [C_out][taps][C_in] seen as (c, tap, output channel); 8-channel mode: one tap's
    // 8 channels of 128 rows per load, unswizzled
    cuuint64_t dims[3] = {(cuuint64_t)d.C_in, (cuuint64_t)geo.taps, (cuuint64_t)d.C_out};
    cuuint64_t strides[2] = {(cuuint64_t)d.C_in * kElem, (cuuint64_t)geo.taps * d.C_in * kElem};
    cuuint32_t box[3] = {small_c ? 8u : (cuuint32_t)kKb, 1, (cuuint32_t)kTileM};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode_tiled(&tm_a, kOperandType, 3, const_cast<void*>(weights), dims, strides,
                                box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                small_c ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return SSCONV_ERR_CUDA;
  }
  // pair kernel: the metadata images as rows of 16 bytes, one box per image (128 rows), so that they
  // come in by a tensor copy, which unlike the plain bulk copy can signal a barrier in the peer CTA
  CUtensorMap tm_meta = tm_a;
  if (pair && SPARSE) {
    // (8-bit operands: two images per group = 256 rows)
    const cuuint32_t rows = C::kMetaBytes / 16;
    cuuint64_t dims[2] = {16, (cuuint64_t)geo.m_tiles * geo.stages * rows};
    cuuint64_t strides[1] = {16};
    cuuint32_t box[2] = {16, rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode_tiled(&tm_meta, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(meta), dims, strides, box,
                                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return SSCONV_ERR_CUDA;
  }
  // output: NHWC seen as (c, position); a box is one staging half piece, 64 channels x 40 positions
  {
    cuuint64_t dims[2] = {(cuuint64_t)d.C_out, (cuuint64_t)Q};
    cuuint64_t strides[1] = {(cuuint64_t)y_pitch_el * 2};  // (channels beyond C_out are clipped: a slice stays a slice)
    cuuint32_t box[2] = {64, (cuuint32_t)kPiece};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode_tiled(&tm_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, y, dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return SSCONV_ERR_CUDA;
    // the last piece of a group may hold fewer positions: same view, shorter box
    box[1] = (cuuint32_t)tail_cols;
    r = g_encode_tiled(&tm_y_tail, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, y, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return SSCONV_ERR_CUDA;
    // the residual tensor, when there is one, is read through the same two views
    tm_r = tm_y;
    tm_r_tail = tm_y_tail;
    if (residual != nullptr) {
      void* res = const_cast<void*>(residual);
      box[1] = (cuuint32_t)kPiece;
      r = g_encode_tiled(&tm_r, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, res, dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return SSCONV_ERR_CUDA;
      box[1] = (cuuint32_t)tail_cols;
      r = g_encode_tiled(&tm_r_tail, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, res, dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return SSCONV_ERR_CUDA;
    }
  }

  FwdParams p;
  p.C_in = d.C_in;
  p.C_out = d.C_out;
  p.Ho = Ho;
  p.Wo = Wo;
  p.Q = (int)Q;
  p.BN = BN;
  p.pieces = pieces;
  p.tail_cols = tail_cols;
  p.ring_groups = ring_groups;
  p.small_c = small_c ? 1 : 0;
  p.a_grp_bytes = a_grp_bytes;
  p.a_res_bytes = a_res_bytes;
  p.stage_bufs = stage_bufs;
  p.stride_h = d.stride_h;
  p.stride_w = d.stride_w;
  p.pad_h = d.pad_h;
  p.pad_w = d.pad_w;
  p.dil_h = d.dil_h;
  p.dil_w = d.dil_w;
  p.KW = d.KW;
  p.taps = geo.taps;
  p.cblocks = geo.cblocks;
  p.kblocks = geo.kblocks;
  p.m_real = geo.m_tiles;
  p.m_tiles = pair ? (geo.m_tiles + 1) / 2 : geo.m_tiles;
  const long long q_tiles = (Q + BN - 1) / BN;
  p.dual = dual ? 1 : 0;
  p.num_tiles = (int)((dual ? (q_tiles + 1) / 2 : q_tiles) * p.m_tiles);  // (work items, where they hold two tiles)
  p.a_tiles = geo.stages;
  p.flags = d.flags;
  p.bias = bias;
  p.meta = static_cast<const uint8_t*>(meta);
  p.y = static_cast<__nv_bfloat16*>(y);
  p.dev_status = dev_status;
  p.out_scale = out_scale;

  const long long units = q_tiles * geo.m_tiles * geo.stages;
  if (units >= (1LL << 31)) return SSCONV_ERR_UNSUPPORTED_SHAPE;  // 32-bit work indices on the device
  p.split = (plan.split && p.a_tiles > 1) ? 1 : 0;
  int grid;
  if (p.split) {
    grid = units < workers ? (int)units : workers;
    p.ws_regions = static_cast<float4*>(ws);
  } else if (pair) {
    const int pairs = workers / 2;
    grid = 2 * (p.num_tiles < pairs ? p.num_tiles : pairs);  // the tiles are dealt out to the pairs
    p.ws_regions = nullptr;
  } else {
    grid = p.num_tiles < workers ? p.num_tiles : workers;
    p.ws_regions = nullptr;
  }
  {
    const long long work = p.split ? units : (long long)p.num_tiles;
    const int dealt_to = pair ? grid / 2 : grid;
    p.work_quot = (int)(work / dealt_to);
    p.work_rem = (int)(work % dealt_to);
  }
  // Programmatic stream serialisation: this grid's set-up (barriers, TMEM, tensor-map fetch, index
  // arithmetic) may overlap the tail of the previous kernel in the stream; the kernel itself
  // waits for that kernel's completion before it touches global memory.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)kThreads);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;  // pair kernel: clusters of two CTAs
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pair ? 2 : 1;
  const cudaError_t launched =
      (FP8 && pair) ? cudaLaunchKernelEx(&cfg, ssconv_fwd_pair_kernel<true, true>, tm_a, tm_b, tm_meta, tm_y, tm_y_tail, tm_r,
                                         tm_r_tail, p)
      : FP8 ? cudaLaunchKernelEx(&cfg, ssconv_fwd_kernel<SPARSE, false, FP8>, tm_a, tm_b, tm_y, tm_y_tail, tm_r, tm_r_tail, p)
      : (pair && residual != nullptr)
          ? cudaLaunchKernelEx(&cfg, ssconv_fwd_pair_kernel<SPARSE, false, true>, tm_a, tm_b, tm_meta, tm_y, tm_y_tail, tm_r,
                               tm_r_tail, p)
      : pair ? cudaLaunchKernelEx(&cfg, ssconv_fwd_pair_kernel<SPARSE>, tm_a, tm_b, tm_meta, tm_y, tm_y_tail, tm_r, tm_r_tail, p)
      : residual != nullptr
          ? cudaLaunchKernelEx(&cfg, ssconv_fwd_kernel<SPARSE, true>, tm_a, tm_b, tm_y, tm_y_tail, tm_r, tm_r_tail, p)
          : cudaLaunchKernelEx(&cfg, ssconv_fwd_kernel<SPARSE, false>, tm_a, tm_b, tm_y, tm_y_tail, tm_r, tm_r_tail, p);
  if (launched != cudaSuccess) return SSCONV_ERR_CUDA;
  count_launch();
  if (p.split) {
    FinishParams f;
    f.C_out = d.C_out;
    f.Q = (int)Q;
    f.BN = BN;
    f.pieces = pieces;
    f.tail_cols = tail_cols;
    f.m_tiles = geo.m_tiles;
    f.a_tiles = p.a_tiles;
    f.work_quot = p.work_quot;
    f.work_rem = p.work_rem;
    f.ws_regions = p.ws_regions;
    f.flags = d.flags;
    f.bias = bias;
    f.residual = static_cast<const __nv_bfloat16*>(residual);
    f.y = p.y;
    f.y_pitch = (int)y_pitch_el;
    cfg.gridDim = dim3((unsigned)p.num_tiles * finish_items_per_tile(pieces));
    cfg.blockDim = dim3((unsigned)kFinishThreads);
    cfg.dynamicSmemBytes = 0;
    if (cudaLaunchKernelEx(&cfg, ssconv_split_finish_kernel, f) != cudaSuccess) return SSCONV_ERR_CUDA;
    count_launch();
  }
  return SSCONV_OK;
}

int32_t launch_forward_sparse(const ssconv_desc_t& d, const void* x, const void* w_comp, const void* meta,
                              const float* bias, const void* residual, void* y, void* ws, size_t ws_bytes,
                              int32_t* dev_status, cudaStream_t stream) {
  return launch_forward_impl<true>(d, x, w_comp, meta, bias, residual, y, ws, ws_bytes, dev_status, stream);
}
int32_t launch_forward_dense(const ssconv_desc_t& d, const void* x, const void* w, const float* bias,
                             const void* residual, void* y, void* ws, size_t ws_bytes, int32_t* dev_status,
                             cudaStream_t stream, const int64_t* x_strides) {
  return launch_forward_impl<false>(d, x, w, nullptr, bias, residual, y, ws, ws_bytes, dev_status, stream, kMaxWorkers,
                                    false, x_strides);
}

// Grouped convolution: `groups` independent convolutions on channel slices, group g reading input
// channels [g C_in/groups, ...) and writing output channels [g C_out/groups, ...); one launch per group
// on strided views of x and y.  The compressed operand of a grouped layer is the concatenation of the
// groups' blobs (each of the size ssconv_sizes reports for the per-group layer).
int32_t launch_forward_grouped(const ssconv_desc_t& d, int groups, bool sparse, const void* x, const void* weights,
                               const void* meta, const float* bias, void* y, void* ws, size_t ws_bytes,
                               int32_t* dev_status, cudaStream_t stream) {
  ssconv_desc_t g = d;
  g.C_in = d.C_in / groups;
  g.C_out = d.C_out / groups;
  const Geometry geo = make_geometry(g);
  const size_t w_step = sparse ? (size_t)geo.Mp * geo.KC * 2 : (size_t)g.C_out * geo.taps * g.C_in * 2;
  const size_t m_step = (size_t)geo.m_tiles * geo.stages * kMetaImageBytes;
  const int64_t xs[3] = {d.C_in, (int64_t)d.W * d.C_in, (int64_t)d.H * d.W * d.C_in};
  for (int i = 0; i < groups; ++i) {
    const char* xg = static_cast<const char*>(x) + (size_t)i * g.C_in * 2;
    char* yg = static_cast<char*>(y) + (size_t)i * g.C_out * 2;
    const float* bg = bias ? bias + (size_t)i * g.C_out : nullptr;
    const char* wg = static_cast<const char*>(weights) + (size_t)i * w_step;
    const int32_t rc =
        sparse ? launch_forward_impl<true>(g, xg, wg, static_cast<const char*>(meta) + (size_t)i * m_step, bg, nullptr, yg,
                                           ws, ws_bytes, dev_status, stream, kMaxWorkers, false, xs, 1.0f, d.C_out)
               : launch_forward_impl<false>(g, xg, wg, nullptr, bg, nullptr, yg, ws, ws_bytes, dev_status, stream,
                                            kMaxWorkers, false, xs, 1.0f, d.C_out);
    if (rc != SSCONV_OK) return rc;
  }
  return SSCONV_OK;
}

int32_t launch_forward_fp8(const ssconv_desc_t& d, bool sparse, const void* x, const void* weights, const void* meta,
                           const float* bias, float out_scale, void* y, int32_t* dev_status, cudaStream_t stream) {
  return sparse ? launch_forward_impl<true, true>(d, x, weights, meta, bias, nullptr, y, nullptr, 0, dev_status, stream,
                                                  kMaxWorkers, false, nullptr, out_scale)
                : launch_forward_impl<false, true>(d, x, weights, nullptr, bias, nullptr, y, nullptr, 0, dev_status,
                                                   stream, kMaxWorkers, false, nullptr, out_scale);
}

// ---------------------------------------------------------------------------------------
// Variant with built-in scratch, for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------
// The scratch of the split-K path lives in this file-scope device array instead of a caller
// buffer.  It is sized for kStaticWorkers thread blocks; every GPU that loads the library keeps
// it (about 15.7 MB) until the process exits.  In host code the array's name is only a handle:
// the device address comes from cudaGetSymbolAddress, once per device.
constexpr int kStaticWorkers = 64;
constexpr int kStaticMaxTiles = 64;
static __device__ __align__(256) unsigned char g_static_scratch[scratch_bytes(kStaticWorkers)];
static unsigned char* g_static_scratch_ptr[64] = {nullptr};

int32_t launch_forward_static_ws(const ssconv_desc_t& d, const void* x, const void* w_comp, const void* meta,
                                 const float* bias, void* y, int32_t* dev_status, cudaStream_t stream) {
  const Geometry geo = make_geometry(d);
  const long long P = (long long)d.N * out_extent(d.H, d.KH, d.stride_h, d.pad_h, d.dil_h) *
                      out_extent(d.W, d.KW, d.stride_w, d.pad_w, d.dil_w);
  const long long tiles = ((P + kBN - 1) / kBN) * geo.m_tiles;
  if (tiles > kStaticMaxTiles) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SSCONV_ERR_CUDA;
  if (g_static_scratch_ptr[dev] == nullptr) {
    unsigned char* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess || ptr == nullptr)
      return SSCONV_ERR_CUDA;
    g_static_scratch_ptr[dev] = ptr;
  }
  unsigned char* scratch = g_static_scratch_ptr[dev];
  // Nothing in the array has to be cleared: it keeps whatever the previous call left, and every
  // partial-sum region is written by this call's main kernel before its finishing kernel reads it.
  return launch_forward_impl<true>(d, x, w_comp, meta, bias, nullptr, y, scratch, scratch_bytes(kStaticWorkers), dev_status,
                                   stream, kStaticWorkers, true);
}

// ---------------------------------------------------------------------------------------
// Self-test of the bounded wait
// ---------------------------------------------------------------------------------------
// One block; thread 0 waits on an mbarrier that nobody arrives at, with the same helper and the same
// give-up path as the convolution kernels (abort flag, status word), only with a short limit.
__global__ void wait_timeout_selftest_kernel(long long limit_cycles, int32_t* dev_status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool done = mbar_wait_bounded(&bar, 0, &abort_flag, limit_cycles);
    if (!done && abort_flag != 0) atomicExch(dev_status, (int)SSCONV_ERR_TIMEOUT);
  }
}
cudaError_t launch_wait_timeout_selftest(long long limit_cycles, int32_t* dev_status, cudaStream_t st) {
  count_launch();
  wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(limit_cycles, dev_status);
  return cudaGetLastError();
}

}  // namespace ssconv
