// Weight gradient of the NHWC bf16 convolution (Eq. 4 differentiated in W) as an implicit GEMM on
// the sm_100a tensor cores: the backward half of the mask-learning step (Sec. 3.1), whose result
// ssconv_mask_grad turns into the gradient of the choice weights.
//
//   dW[C_out x K] = dY^T[C_out x Q] * U(X)^T[Q x K],   Q = output positions, K = KH*KW*C_in
//
// The contraction runs over positions.  Both operands arrive position-major, exactly as the forward
// kernel's loads leave them in shared memory: a tile of 64 positions x 64 channels with 128-byte
// rows (one position each) in the 128-byte swizzle.  For this product the rows are the K dimension,
// so both operands are "MN-major" and the matrix descriptors say so: 8 rows (positions) of one
// 64-channel block form a swizzle atom, groups of 8 positions lie 1024 B apart (stride-dimension
// offset), and the next block of 64 channels lies one tile (8 KB) further on (leading-dimension
// offset).  A = dY tile (128 output channels = two blocks), B = up to four activation tiles, one
// per k-block (a filter tap x a chunk of 64 input channels, numbered chunk * taps + tap as in the
// forward kernel): N = 64 to 256 columns of dW per CTA, so the gradient tile is loaded once for up
// to four taps.
//
// A CTA owns one work item: 128 output channels x T k-blocks x one range of positions, and walks
// its positions 64 at a time through a 4-stage TMA ring (four producer threads, one MMA thread,
// four epilogue warps, fp32 accumulator of 64 T columns in TMEM).  The accumulator has output
// channels on TMEM lanes, so an epilogue thread holds one row of dW: it writes to a scratch slice
// laid out [tile of 128 output channels][K][128], where the 32 lanes of a warp store 128 contiguous
// bytes and a CTA's whole output is one contiguous block.  A second kernel
// adds the slices of all position ranges in a fixed order (the result does not depend on timing)
// and transposes 32 x 32 tiles through shared memory into dW [C_out][K].  All mbarrier waits are
// bounded (see sm100_ptx.cuh).
#include <cuda.h>
#include <cuda_runtime.h>

#include "layout.cuh"
#include "sm100_ptx.cuh"
#include "ssconv.h"

namespace ssconv {

constexpr int kWgThreads = 288;        // warps 0, 6, 7, 8: TMA producers, warp 1: MMA, warps 2-5: epilogue
constexpr int kWgPos = 64;             // positions per ring stage
constexpr int kWgMaxT = 4;             // k-blocks per work item (N = 64 T <= 256)
constexpr int kWgStages = 4;
constexpr uint32_t kWgTileBytes = kWgPos * 128;                  // 64 positions x 64 channels bf16
constexpr uint32_t kWgStageBytes = (2 + kWgMaxT) * kWgTileBytes;  // two gradient halves + T activation tiles
constexpr uint32_t kWgTmemCols = 256;
constexpr uint32_t kWgSmemBytes = 1024 + kWgStages * kWgStageBytes + 256;
constexpr long long kWgWaitLimitCycles = 4000000000LL;

struct WgParams {
  int C_in, C_out, Ho, Wo, Q;
  int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, KW;
  int taps, kblocks;       // k-blocks = channel chunks x taps, numbered chunk * taps + tap
  int T, items_b;          // k-blocks per item, items along K = ceil(kblocks / T)
  int m_tiles;
  int splits;              // position ranges
  int ksteps, ksteps_per_split;  // steps of 64 positions: in all, per range
  int dy_one_load;         // C_out % 64 == 0: both halves of a gradient tile come with one 3-D load
  float* out;              // `splits` slices [m_tiles][taps * C_in][128] of partial gradients
  int32_t* dev_status;
};

// This warp's 32 TMEM lanes x 32 consecutive columns: register j = column j of the thread's lane.
__device__ __forceinline__ void tc_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

// Low word of the descriptor of a position-major (MN-major) operand: address and the distance
// between 64-channel blocks (one tile) as the leading-dimension offset.
__device__ __forceinline__ uint32_t wg_desc_lo(uint32_t smem_addr) {
  return ((smem_addr & 0x3FFFFu) >> 4) | ((kWgTileBytes >> 4) << 16);
}

struct WgItem {
  int m, b0, nb, ks0, ks1, split;
};
__device__ __forceinline__ WgItem wg_item(const WgParams& p) {
  WgItem it;
  int i = blockIdx.x;
  const int ib = i % p.items_b;
  i /= p.items_b;
  it.m = i % p.m_tiles;
  it.split = i / p.m_tiles;
  it.b0 = ib * p.T;
  it.nb = min(p.T, p.kblocks - it.b0);
  it.ks0 = it.split * p.ksteps_per_split;
  it.ks1 = min(p.ksteps, it.ks0 + p.ksteps_per_split);
  return it;
}

__global__ void __launch_bounds__(kWgThreads, 1)
ssconv_wgrad_kernel(const __grid_constant__ CUtensorMap tm_dy, const __grid_constant__ CUtensorMap tm_x,
                    const WgParams p) {
  extern __shared__ uint8_t wg_smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(wg_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kWgStages * kWgStageBytes);
  uint64_t* bar_full = bars;                 // [kWgStages]
  uint64_t* bar_empty = bars + kWgStages;    // [kWgStages]
  uint64_t* bar_acc = bars + 2 * kWgStages;  // accumulator complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kWgStages + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const WgItem item = wg_item(p);
  const uint32_t producers = 1u + (uint32_t)min(item.nb, 3);  // roles that load something

  if (warp == 0) {
    if (lane == 0) {
      for (int s = 0; s < kWgStages; ++s) {
        mbar_init(&bar_full[s], producers);
        mbar_init(&bar_empty[s], 1u);
      }
      mbar_init(bar_acc, 1u);
      *abort_flag = 0;
      mbar_fence_init();
      fence_proxy_async_smem();
      prefetch_tensormap(&tm_dy);
      prefetch_tensormap(&tm_x);
    }
    __syncwarp();
  } else if (warp == 1) {
    tmem_alloc(tmem_slot, kWgTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t full0 = smem_u32(bar_full), empty0 = smem_u32(bar_empty), ring0 = smem_u32(smem);

  if (warp == 0 || warp >= 6) {
    // ------------------------------------------------------------------ TMA producers
    // A TMA instruction occupies its thread for a few hundred cycles, so the loads of a stage are
    // spread over four threads: role 0 the gradient tile, roles 1-3 the activation tiles
    // (role 1 also the fourth one).
    const int role = (warp == 0) ? 0 : warp - 5;
    if (lane == 0 && role < (int)producers) {
      uint32_t s = 0, ph = 0;
      for (int ks = item.ks0; ks < item.ks1; ++ks) {
        if (!mbar_wait_a(empty0 + 8u * s, ph ^ 1u, abort_flag, kWgWaitLimitCycles)) break;
        const uint32_t full = full0 + 8u * s;
        const uint32_t dst = ring0 + s * kWgStageBytes;
        const int q0 = ks * kWgPos;
        if (role == 0) {
          // channels beyond C_out and positions beyond Q lie outside the tensor map: zeros
          mbar_expect_tx_a(full, 2u * kWgTileBytes);
          if (p.dy_one_load) {
            tma_load_3d_a(dst, &tm_dy, full, 0, q0, 2 * item.m);
          } else {
            tma_load_2d_a(dst, &tm_dy, full, item.m * kTileM, q0);
            tma_load_2d_a(dst + kWgTileBytes, &tm_dy, full, item.m * kTileM + 64, q0);
          }
        } else {
          const int rho = q0 / p.Wo;
          const int wo = q0 - rho * p.Wo;
          const int n = rho / p.Ho;
          const int ho = rho - n * p.Ho;
          const int base_w = wo * p.stride_w - p.pad_w;
          const int base_h = ho * p.stride_h - p.pad_h;
          const bool two = (role == 1 && item.nb > 3);
          mbar_expect_tx_a(full, two ? 2u * kWgTileBytes : kWgTileBytes);
          for (int t = role - 1; t < item.nb; t += 3) {
            const int b = item.b0 + t;
            const int cc = b / p.taps;
            const int tap = b - cc * p.taps;
            const int kh = tap / p.KW;
            const int kw = tap - kh * p.KW;
            tma_load_im2col_4d_a(dst + (uint32_t)(2 + t) * kWgTileBytes, &tm_x, full, cc * kBlockK, base_w, base_h,
                                 n, (uint16_t)(kw * p.dil_w), (uint16_t)(kh * p.dil_h));
          }
        }
        if (++s == kWgStages) {
          s = 0;
          ph ^= 1u;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // both operands MN-major: bits 15 and 16 of the instruction descriptor
      const uint32_t idesc = make_idesc_bf16(kTileM, (uint32_t)(64 * item.nb), false) | (1u << 15) | (1u << 16);
      uint32_t s = 0, ph = 0, accumulate = 0;
      bool ok = true;
      for (int ks = item.ks0; ks < item.ks1; ++ks) {
        if (!mbar_wait_a(full0 + 8u * s, ph, abort_flag, kWgWaitLimitCycles)) { ok = false; break; }
        const uint32_t a_lo = wg_desc_lo(ring0 + s * kWgStageBytes);
        const uint32_t b_lo = a_lo + ((2u * kWgTileBytes) >> 4);
        // 16 positions per MMA = two groups of 8 rows = 2048 B
#pragma unroll
        for (int i = 0; i < kWgPos / 16; ++i) {
          tc_mma_dense_lo(tmem_base, a_lo + (uint32_t)i * 128u, b_lo + (uint32_t)i * 128u, idesc, accumulate);
          accumulate = 1;
        }
        tc_commit_a(empty0 + 8u * s);
        if (++s == kWgStages) {
          s = 0;
          ph ^= 1u;
        }
      }
      if (ok) tc_commit(bar_acc);
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ epilogue
    const int qd = warp & 3;  // TMEM lane quadrant of this warp
    // the TMEM loads below are warp-wide: the warp goes on only if every lane saw the barrier complete
    const bool got =
        __all_sync(0xFFFFFFFFu, mbar_wait_bounded(bar_acc, 0u, abort_flag, kWgWaitLimitCycles, 64) ? 1 : 0) != 0;
    if (got) {
      tc_fence_after();
      const size_t K = (size_t)p.taps * p.C_in;
      float* out = p.out + ((size_t)item.split * p.m_tiles + item.m) * K * kTileM + qd * 32 + lane;
      for (int t = 0; t < item.nb; ++t) {
        const int b = item.b0 + t;
        const int cc = b / p.taps;
        const int tap = b - cc * p.taps;
        // column c of this k-block is row tap * C_in + 64 cc + c of the tile's [K][128] block
        // (rows of output channels beyond C_out hold zeros: their gradient rows were zero-filled)
        float* col0 = out + ((size_t)tap * p.C_in + cc * kBlockK) * kTileM;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          uint32_t r[32];
          tc_ld_32x32b_x32(tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)(64 * t + 32 * half), r);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int c = 32 * half + j;
            if (cc * kBlockK + c < p.C_in) col0[(size_t)c * kTileM] = __uint_as_float(r[j]);
          }
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag != 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    if (threadIdx.x == 0 && p.dev_status != nullptr) atomicExch(p.dev_status, (int)SSCONV_ERR_TIMEOUT);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kWgTmemCols);
  }
}

// ---------------------------------------------------------------------------------------
// The same product on CTA pairs (tcgen05.mma cta_group::2), transposed:
//
//   dW^T[K x C_out] = U(X)[K x Q] * dY[Q x C_out]
//
// A pair owns four k-blocks (M = 256 rows of dW^T: each CTA loads the activation tiles of its two
// k-blocks, 128 rows) x one tile of NT = 128 or 256 output channels (each CTA loads the gradient
// tiles of its half of them) x one range of positions, walked 128 positions at a time through a
// three-stage ring.  Against the one-CTA kernel above, every byte staged in shared memory serves
// twice the multiply-adds (the other CTA's tensor core reads it too), which is what that kernel is
// bound by; and since the accumulator's lanes now run along K, a warp's 32 lanes write 128 contiguous
// bytes of dW [C_out][K] itself: the slices of the position ranges have the layout of the result (a
// CTA's part of the tile is staged in shared memory and leaves as two-dimensional bulk copies) and the
// second kernel only adds them, in slice order.
// Layout of a stage in each CTA: two activation tiles, then two gradient tiles, 128 positions x 64
// channels (16 KB) each, position-major in the 128-byte swizzle as above.  Barriers as in the forward
// pair kernel: "full" lives in the even CTA (the leader) and collects the bytes of both CTAs' loads,
// "empty" and "accumulator complete" exist in both and the leader commits to both.  No load is
// multicast.  Tiles that lie outside the tensors (k-blocks past the last one, channels past C_out,
// positions past Q) are loaded all the same and arrive as zeros.
constexpr int kWpThreads = 256;        // warp 0: activation loads, warp 1: MMA (leader), warp 2: gradient loads, 4-7: epilogue
constexpr int kWpPos = 128;            // positions per ring stage
constexpr int kWpStages = 3;
constexpr uint32_t kWpTileBytes = kWpPos * 128;
constexpr uint32_t kWpStageBytes = 4 * kWpTileBytes;
constexpr uint32_t kWpTmemCols = 256;
constexpr uint32_t kWpSmemBytes = 1024 + kWpStages * kWpStageBytes + 256;

struct WpParams {
  int C_in, C_out, Ho, Wo;
  int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, KW;
  int taps, kblocks, cblocks;
  int kgroups, n_tiles, NT;
  int ksteps, ksteps_per_split;
  int32_t* dev_status;
};

__device__ __forceinline__ uint32_t wp_desc_lo(uint32_t smem_addr) {
  return ((smem_addr & 0x3FFFFu) >> 4) | ((kWpTileBytes >> 4) << 16);
}

__global__ void __launch_bounds__(kWpThreads, 1)
ssconv_wgrad_pair_kernel(const __grid_constant__ CUtensorMap tm_dy, const __grid_constant__ CUtensorMap tm_x,
                         const __grid_constant__ CUtensorMap tm_dw, const WpParams p) {
  extern __shared__ uint8_t wp_smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(wp_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kWpStages * kWpStageBytes);
  uint64_t* bar_full = bars;                  // [kWpStages], used in the leader
  uint64_t* bar_empty = bars + kWpStages;     // [kWpStages]
  uint64_t* bar_acc = bars + 2 * kWpStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kWpStages + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  // item of this pair: (range of positions, tile of output channels, group of four k-blocks)
  int i = (int)(blockIdx.x >> 1);
  const int kg = i % p.kgroups;
  i /= p.kgroups;
  const int nt = i % p.n_tiles;
  const int split = i / p.n_tiles;
  const int ks0 = split * p.ksteps_per_split;
  const int ks1 = min(p.ksteps, ks0 + p.ksteps_per_split);
  const int b_first = 4 * kg + 2 * (int)rank;   // this CTA's two k-blocks
  const int n_half = p.NT >> 1;                 // this CTA's gradient channels: n_first .. n_first + n_half
  const int n_first = nt * p.NT + (int)rank * n_half;

  if (warp == 0) {
    if (lane == 0) {
      for (int s = 0; s < kWpStages; ++s) {
        mbar_init(&bar_full[s], 2u);   // the leader's two producer warps
        mbar_init(&bar_empty[s], 1u);
      }
      mbar_init(bar_acc, 1u);
      *abort_flag = 0;
      mbar_fence_init();
      fence_proxy_async_smem();
      prefetch_tensormap(&tm_dy);
      prefetch_tensormap(&tm_x);
      prefetch_tensormap(&tm_dw);
      grid_launch_dependents();   // (the adding kernel waits for this grid's completion itself)
    }
    __syncwarp();
  } else if (warp == 1) {
    tmem_alloc2(tmem_slot, kWpTmemCols);
    tmem_relinquish2();
  }
  // both CTAs' barriers and TMEM exist before either touches the other's
  tc_fence_before();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t full0_local = smem_u32(bar_full), empty0 = smem_u32(bar_empty), ring0 = smem_u32(smem);
  const uint32_t full0_leader = map_to_cta(full0_local, 0);

  if (warp == 0 || warp == 2) {
    // ------------------------------------------------------------------ TMA producers (whole warps)
    uint32_t s = 0, ph = 0;
    int cc[2], kh[2], kw[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int b = b_first + t;
      // (a k-block past the last one reads the channel chunk after the last: zeros)
      cc[t] = b < p.kblocks ? b / p.taps : p.cblocks;
      const int tap = b < p.kblocks ? b - cc[t] * p.taps : 0;
      kh[t] = tap / p.KW;
      kw[t] = tap - kh[t] * p.KW;
    }
    grid_dependency_wait();   // everything above may overlap the tail of the kernel before this one
    for (int ks = ks0; ks < ks1; ++ks) {
      if (!mbar_wait_a(empty0 + 8u * s, ph ^ 1u, abort_flag, kWgWaitLimitCycles)) break;
      const uint32_t full = full0_leader + 8u * s;
      const uint32_t dst = ring0 + s * kWpStageBytes;
      const int q0 = ks * kWpPos;
      if (warp == 0) {
        if (rank == 0) mbar_expect_tx_w(full0_local + 8u * s, 4u * kWpTileBytes);   // both CTAs' activation tiles
        const int rho = q0 / p.Wo;
        const int wo = q0 - rho * p.Wo;
        const int n = rho / p.Ho;
        const int ho = rho - n * p.Ho;
        const int base_w = wo * p.stride_w - p.pad_w;
        const int base_h = ho * p.stride_h - p.pad_h;
#pragma unroll
        for (int t = 0; t < 2; ++t)
          tma2_load_im2col_4d_w(dst + (uint32_t)t * kWpTileBytes, &tm_x, full, cc[t] * kBlockK, base_w, base_h, n,
                                (uint16_t)(kw[t] * p.dil_w), (uint16_t)(kh[t] * p.dil_h));
      } else {
        const uint32_t tiles = (uint32_t)(n_half >> 6);
        if (rank == 0) mbar_expect_tx_w(full0_local + 8u * s, 2u * tiles * kWpTileBytes);
        for (uint32_t t = 0; t < tiles; ++t)
          tma2_load_2d_w(dst + (2u + t) * kWpTileBytes, &tm_dy, full, n_first + 64 * (int)t, q0);
      }
      if (++s == kWpStages) {
        s = 0;
        ph ^= 1u;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only, whole warp)
    if (rank == 0) {
      const uint32_t idesc = make_idesc_bf16(2 * kTileM, (uint32_t)p.NT, false) | (1u << 15) | (1u << 16);
      uint32_t s = 0, ph = 0, accumulate = 0;
      bool ok = true;
      for (int ks = ks0; ks < ks1; ++ks) {
        if (!mbar_wait_a(full0_local + 8u * s, ph, abort_flag, kWgWaitLimitCycles)) { ok = false; break; }
        tc_fence_after();
        const uint32_t a_lo = wp_desc_lo(ring0 + s * kWpStageBytes);
        const uint32_t b_lo = a_lo + ((2u * kWpTileBytes) >> 4);
        // 16 positions per MMA = two groups of 8 rows = 2048 B
#pragma unroll
        for (int k = 0; k < kWpPos / 16; ++k) {
          tc2_mma_dense_w(tmem_base, a_lo + (uint32_t)k * 128u, b_lo + (uint32_t)k * 128u, idesc, accumulate);
          accumulate = 1;
        }
        tc2_commit_both_w(empty0 + 8u * s);
        if (++s == kWpStages) {
          s = 0;
          ph ^= 1u;
        }
      }
      if (ok) tc2_commit_both_w(smem_u32(bar_acc));
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ epilogue
    const int qd = warp & 3;  // TMEM lane quadrant of this warp
    const bool got =
        __all_sync(0xFFFFFFFFu, mbar_wait_bounded(bar_acc, 0u, abort_flag, kWgWaitLimitCycles, 64) ? 1 : 0) != 0;
    if (got) {
      tc_fence_after();
      // Lane row 32 qd + lane of this CTA = channel (32 qd + lane) % 64 of its k-block (32 qd + lane) / 64.
      // The tile goes through shared memory (the ring is idle by now: every load has been consumed), as
      // [k-block][output channel][64 channels] fp32, and from there to dW [C_out][taps][C_in] as boxes of
      // 128 output channels x 64 channels: per-lane stores of 4 bytes would take several times the
      // main loop of a short position range.  Rows and columns outside the tensor are clipped by the copy.
      const uint32_t stage = ring0 + (uint32_t)(qd >> 1) * (uint32_t)p.NT * 256u + (uint32_t)((qd & 1) * 32 + lane) * 4u;
      const int n0 = nt * p.NT;
#pragma unroll 1
      for (int j0 = 0; j0 < p.NT; j0 += 128) {
        if (n0 + j0 >= p.C_out) break;   // (uniform over the warp)
        uint32_t r[4][32];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          tc_ld_32x32b_x32(tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)(j0 + 32 * u), r[u]);
        tc_wait_ld();
#pragma unroll
        for (int u = 0; u < 4; ++u) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            asm volatile("st.shared.b32 [%0], %1;" ::"r"(stage + (uint32_t)(j0 + 32 * u + j) * 256u), "r"(r[u][j]) : "memory");
        }
      }
      fence_proxy_async_smem();
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");   // the four epilogue warps
    if (got && warp == 4 && lane == 0 && *abort_flag == 0) {
      const int n0 = nt * p.NT;
      grid_dependency_wait();
      for (int t = 0; t < 2; ++t) {
        const int b = b_first + t;
        if (b >= p.kblocks) break;
        const int ccb = b / p.taps;
        const int tap = b - ccb * p.taps;
        for (int j0 = 0; j0 < p.NT && n0 + j0 < p.C_out; j0 += 128)
          tma_store_4d(&tm_dw, ring0 + (uint32_t)t * (uint32_t)p.NT * 256u + (uint32_t)j0 * 256u, ccb * kBlockK, tap,
                       n0 + j0, split);
      }
      bulk_commit_group();
      bulk_wait_group_read0();   // shared memory is released below; the writes complete with the grid
    }
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
    tmem_dealloc2(tmem_base, kWpTmemCols);
  }
}

// dW = the sum, in slice order, of `splits` slices of the same layout (four elements per thread).
__global__ void __launch_bounds__(256) wgrad_sum_kernel(const float4* __restrict__ slices, int splits, size_t slice_vec,
                                                        float4* __restrict__ dw) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  grid_dependency_wait();   // launched while the kernel that writes the slices is still running
  if (i >= slice_vec) return;
  float4 acc = slices[i];
  for (int s = 1; s < splits; ++s) {
    const float4 v = slices[(size_t)s * slice_vec + i];
    acc.x += v.x;
    acc.y += v.y;
    acc.z += v.z;
    acc.w += v.w;
  }
  dw[i] = acc;
}

// dW [C_out][K] = transpose of the sum, in slice order, of the slices [m_tiles][K][128].  A block
// of 32 x 8 threads handles 32 output channels x 8 columns of K, one element per thread: reads are
// contiguous along the output channels, writes go out as 32-byte runs along K.  With many slices
// the sums are latency-bound, hence the small tiles (many blocks) and eight loads in flight.
__global__ void wgrad_reduce_kernel(const float* __restrict__ slices, int splits, int K, int C_out, int m_tiles,
                                    float* __restrict__ dw) {
  __shared__ float tile[8][33];
  const int k0 = blockIdx.x * 8, c0 = blockIdx.y * 32;
  const size_t slice = (size_t)m_tiles * K * kTileM;
  const int c = c0 + threadIdx.x, k = k0 + threadIdx.y;
  float acc = 0.0f;
  if (k < K && c < C_out) {
    const float* src = slices + ((size_t)(c / kTileM) * K + k) * kTileM + (c % kTileM);
    int s = 0;
    for (; s + 8 <= splits; s += 8) {  // eight loads in flight, added in slice order
      float v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = src[(size_t)(s + j) * slice];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc += v[j];
    }
    for (; s < splits; ++s) acc += src[(size_t)s * slice];
  }
  tile[threadIdx.y][threadIdx.x] = acc;
  __syncthreads();
  const int t = threadIdx.y * 32 + threadIdx.x;
  const int cl = t >> 3, kl = t & 7;
  if (k0 + kl < K && c0 + cl < C_out) dw[(size_t)(c0 + cl) * K + k0 + kl] = tile[kl][cl];
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
namespace {

typedef CUresult (*WgEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*WgEncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                     const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t,
                                     const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                     CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
WgEncodeTiledFn wg_encode_tiled = nullptr;
WgEncodeIm2colFn wg_encode_im2col = nullptr;

bool wg_load_encoders() {
  if (wg_encode_tiled && wg_encode_im2col) return true;
  void* f1 = nullptr;
  void* f2 = nullptr;
  cudaDriverEntryPointQueryResult q1, q2;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f1, cudaEnableDefault, &q1) != cudaSuccess) return false;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f2, cudaEnableDefault, &q2) != cudaSuccess) return false;
  if (q1 != cudaDriverEntryPointSuccess || q2 != cudaDriverEntryPointSuccess || !f1 || !f2) return false;
  wg_encode_tiled = reinterpret_cast<WgEncodeTiledFn>(f1);
  wg_encode_im2col = reinterpret_cast<WgEncodeIm2colFn>(f2);
  return true;
}

int wg_out_extent(int in, int k, int stride, int pad, int dil) {
  const int span = in + 2 * pad - dil * (k - 1) - 1;
  return span < 0 ? 0 : span / stride + 1;
}

bool g_wg_attr_set[64] = {false};
int g_tune_wg_ranges = 0;   // 0: the planner chooses; otherwise an upper limit on the position ranges
int g_tune_wg_pair = -1;    // -1: the planner chooses; 0: one-CTA kernel only; 1: the pair kernel wherever it applies

// How a layer's weight gradient is cut into work items.
struct WgPlan {
  int taps, kblocks, T, items_b, m_tiles, ksteps, splits, ksteps_per_split;
  long long Q;
  bool pair;                 // the CTA-pair kernel
  int kgroups, n_tiles, NT;  // its items: groups of four k-blocks x tiles of NT output channels
};
WgPlan wg_plan(const ssconv_desc_t& d, int sms) {
  WgPlan w;
  w.taps = d.KH * d.KW;
  w.kblocks = w.taps * ((d.C_in + kBlockK - 1) / kBlockK);
  w.Q = (long long)d.N * wg_out_extent(d.H, d.KH, d.stride_h, d.pad_h, d.dil_h) *
        wg_out_extent(d.W, d.KW, d.stride_w, d.pad_w, d.dil_w);
  // CTA pairs whenever at least three of a pair's four k-blocks exist (its 256 accumulator rows run
  // along K); layers with one or two k-blocks (1 x 1 convolutions over at most 128 channels) keep
  // the one-CTA kernel, whose 128 rows run along C_out.
  w.pair = (g_tune_wg_pair < 0 ? w.kblocks >= 3 : g_tune_wg_pair == 1) && sms >= 2;
  if (w.pair) {
    w.kgroups = (w.kblocks + 3) / 4;
    w.NT = d.C_out > 128 ? 256 : 128;
    w.n_tiles = (d.C_out + w.NT - 1) / w.NT;
    w.ksteps = (int)((w.Q + kWpPos - 1) / kWpPos);
    w.T = 4;
    w.items_b = w.kgroups;
    w.m_tiles = w.n_tiles;
    const int items = w.kgroups * w.n_tiles;
    int splits = (sms / 2) / items;
    if (splits > w.ksteps / 4) splits = w.ksteps / 4;   // at least four steps of 128 positions per range
    if (g_tune_wg_ranges > 0 && splits > g_tune_wg_ranges) splits = g_tune_wg_ranges;
    if (splits < 1) splits = 1;
    w.ksteps_per_split = (w.ksteps + splits - 1) / splits;
    w.splits = (w.ksteps + w.ksteps_per_split - 1) / w.ksteps_per_split;
    return w;
  }
  w.kgroups = w.n_tiles = w.NT = 0;
  const int groups = (w.kblocks + kWgMaxT - 1) / kWgMaxT;
  w.T = (w.kblocks + groups - 1) / groups;
  w.items_b = (w.kblocks + w.T - 1) / w.T;
  w.m_tiles = (d.C_out + kTileM - 1) / kTileM;
  w.ksteps = (int)((w.Q + kWgPos - 1) / kWgPos);
  // Split the positions when the items alone would leave SMs idle, but keep at least 8 steps per
  // range so that the pipeline's ramp and the epilogue stay small against the loop.
  const int items = w.m_tiles * w.items_b;
  int splits = sms / items;
  if (splits > w.ksteps / 8) splits = w.ksteps / 8;
  if (g_tune_wg_ranges > 0 && splits > g_tune_wg_ranges) splits = g_tune_wg_ranges;
  if (splits < 1) splits = 1;
  w.ksteps_per_split = (w.ksteps + splits - 1) / splits;
  w.splits = (w.ksteps + w.ksteps_per_split - 1) / w.ksteps_per_split;  // no empty range
  return w;
}

int wg_sm_count(int* sms) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SSCONV_ERR_CUDA;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SSCONV_ERR_CUDA;
  if (major != 10) return SSCONV_ERR_ARCH;
  if (cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || *sms <= 0)
    return SSCONV_ERR_CUDA;
  return SSCONV_OK;
}

}  // namespace

int32_t wgrad_set_tuning(int32_t option, int32_t value) {
  if (option == SSCONV_TUNE_WGRAD_RANGES) {
    if (value < 0 || value > 1024) return SSCONV_ERR_BAD_DESC;
    g_tune_wg_ranges = value;
    return SSCONV_OK;
  }
  if (option == SSCONV_TUNE_WGRAD_PAIR) {
    if (value < -1 || value > 1) return SSCONV_ERR_BAD_DESC;
    g_tune_wg_pair = value;
    return SSCONV_OK;
  }
  return SSCONV_ERR_BAD_DESC;
}

// Scratch the layer's weight gradient needs on the current device: one slice per position range.
int32_t wgrad_workspace_bytes(const ssconv_desc_t& d, size_t* bytes) {
  int sms = 0;
  const int32_t st = wg_sm_count(&sms);
  if (st != SSCONV_OK) return st;
  const WgPlan w = wg_plan(d, sms);
  if (w.pair)
    *bytes = w.splits > 1 ? (size_t)w.splits * d.C_out * w.taps * d.C_in * sizeof(float) : 0;
  else
    *bytes = (size_t)w.splits * w.m_tiles * kTileM * w.taps * d.C_in * sizeof(float);
  return SSCONV_OK;
}

namespace {
bool g_wp_attr_set[64] = {false};

int32_t launch_wgrad_pair(const ssconv_desc_t& d, const WgPlan& w, int Ho, int Wo, const void* x, const void* dy,
                          float* dw, void* ws, size_t ws_bytes, int32_t* dev_status, cudaStream_t stream) {
  int dev = 0;
  cudaGetDevice(&dev);
  if (!g_wp_attr_set[dev]) {
    if (cudaFuncSetAttribute(ssconv_wgrad_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kWpSmemBytes) != cudaSuccess)
      return SSCONV_ERR_CUDA;
    g_wp_attr_set[dev] = true;
  }
  const size_t slice_elems = (size_t)d.C_out * w.taps * d.C_in;
  if (w.splits > 1 && (ws == nullptr || ws_bytes < (size_t)w.splits * slice_elems * sizeof(float)))
    return SSCONV_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(dw) & 15u) || (w.splits > 1 && (reinterpret_cast<uintptr_t>(ws) & 15u)))
    return SSCONV_ERR_ALIGNMENT;
  CUtensorMap tm_dy, tm_x;
  {
    // gradient of the output, NHWC seen as (c, position); a box is 64 channels x 128 positions
    cuuint64_t dims[2] = {(cuuint64_t)d.C_out, (cuuint64_t)w.Q};
    cuuint64_t strides[1] = {(cuuint64_t)d.C_out * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kWpPos};
    cuuint32_t estr[2] = {1, 1};
    if (wg_encode_tiled(&tm_dy, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(dy), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SSCONV_ERR_CUDA;
  }
  {
    // activations in im2col mode as in the one-CTA kernel, 128 positions per load
    cuuint64_t dims[4] = {(cuuint64_t)d.C_in, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.N};
    cuuint64_t strides[3] = {(cuuint64_t)d.C_in * 2, (cuuint64_t)d.W * d.C_in * 2,
                             (cuuint64_t)d.H * d.W * d.C_in * 2};
    int lower[2] = {-d.pad_w, -d.pad_h};
    int upper[2] = {d.pad_w - (d.KW - 1) * d.dil_w, d.pad_h - (d.KH - 1) * d.dil_h};
    cuuint32_t estr[4] = {1, (cuuint32_t)d.stride_w, (cuuint32_t)d.stride_h, 1};
    if (wg_encode_im2col(&tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(x), dims, strides, lower,
                         upper, (cuuint32_t)kBlockK, (cuuint32_t)kWpPos, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SSCONV_ERR_CUDA;
  }
  CUtensorMap tm_dw;
  {
    // the result (or its slices, one per position range) as (c_in, tap, c_out, range) fp32; a box is 64
    // channels of one tap x 128 output channels, unswizzled
    float* out = w.splits > 1 ? static_cast<float*>(ws) : dw;
    cuuint64_t dims[4] = {(cuuint64_t)d.C_in, (cuuint64_t)w.taps, (cuuint64_t)d.C_out, (cuuint64_t)w.splits};
    cuuint64_t strides[3] = {(cuuint64_t)d.C_in * 4, (cuuint64_t)w.taps * d.C_in * 4, (cuuint64_t)slice_elems * 4};
    cuuint32_t box[4] = {64, 1, 128, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (wg_encode_tiled(&tm_dw, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, out, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SSCONV_ERR_CUDA;
  }
  WpParams p;
  p.C_in = d.C_in;
  p.C_out = d.C_out;
  p.Ho = Ho;
  p.Wo = Wo;
  p.stride_h = d.stride_h;
  p.stride_w = d.stride_w;
  p.pad_h = d.pad_h;
  p.pad_w = d.pad_w;
  p.dil_h = d.dil_h;
  p.dil_w = d.dil_w;
  p.KW = d.KW;
  p.taps = w.taps;
  p.kblocks = w.kblocks;
  p.cblocks = (d.C_in + kBlockK - 1) / kBlockK;
  p.kgroups = w.kgroups;
  p.n_tiles = w.n_tiles;
  p.NT = w.NT;
  p.ksteps = w.ksteps;
  p.ksteps_per_split = w.ksteps_per_split;
  p.dev_status = dev_status;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * w.splits * w.n_tiles * w.kgroups));
  cfg.blockDim = dim3(kWpThreads);
  cfg.dynamicSmemBytes = kWpSmemBytes;
  cfg.stream = stream;
  // Programmatic stream serialisation on both kernels: a grid's set-up overlaps the tail of the grid
  // before it; each waits for that grid's completion before it touches global memory.
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  count_launch();
  if (cudaLaunchKernelEx(&cfg, ssconv_wgrad_pair_kernel, tm_dy, tm_x, tm_dw, p) != cudaSuccess) return SSCONV_ERR_CUDA;
  if (w.splits > 1) {
    const size_t vec = slice_elems / 4;
    cudaLaunchConfig_t cs = {};
    cs.gridDim = dim3((unsigned)((vec + 255) / 256));
    cs.blockDim = dim3(256);
    cs.stream = stream;
    cs.attrs = attr;
    cs.numAttrs = 1;
    count_launch();
    if (cudaLaunchKernelEx(&cs, wgrad_sum_kernel, static_cast<const float4*>(ws), (int)w.splits, vec,
                           reinterpret_cast<float4*>(dw)) != cudaSuccess)
      return SSCONV_ERR_CUDA;
  }
  return SSCONV_OK;
}
}  // namespace

int32_t launch_wgrad(const ssconv_desc_t& d, const void* x, const void* dy, float* dw, void* ws, size_t ws_bytes,
                     int32_t* dev_status, cudaStream_t stream) {
  if (!wg_load_encoders()) return SSCONV_ERR_CUDA;
  int sms = 0;
  {
    const int32_t st = wg_sm_count(&sms);
    if (st != SSCONV_OK) return st;
  }
  int dev = 0;
  cudaGetDevice(&dev);
  if (!g_wg_attr_set[dev]) {
    if (cudaFuncSetAttribute(ssconv_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWgSmemBytes) !=
        cudaSuccess)
      return SSCONV_ERR_CUDA;
    g_wg_attr_set[dev] = true;
  }
  const WgPlan w = wg_plan(d, sms);
  if (w.Q > 0x7FFFFF00LL) return SSCONV_ERR_UNSUPPORTED_SHAPE;
  const int Ho = wg_out_extent(d.H, d.KH, d.stride_h, d.pad_h, d.dil_h);
  const int Wo = wg_out_extent(d.W, d.KW, d.stride_w, d.pad_w, d.dil_w);
  if (w.pair) return launch_wgrad_pair(d, w, Ho, Wo, x, dy, dw, ws, ws_bytes, dev_status, stream);
  const size_t slice_bytes = (size_t)w.m_tiles * kTileM * w.taps * d.C_in * sizeof(float);
  if (ws == nullptr || ws_bytes < (size_t)w.splits * slice_bytes) return SSCONV_ERR_WORKSPACE;

  CUtensorMap tm_dy, tm_x;
  {
    // gradient of the output, NHWC seen as (c, position); a box is 64 channels x 64 positions.  When
    // C_out is a multiple of 64 the view is (64 channels, position, block of 64 channels) instead, so
    // that one box of 64 x 64 x 2 brings both halves of a 128-channel tile, half after half.
    const bool one_load = d.C_out % 64 == 0;
    CUresult r;
    if (one_load) {
      cuuint64_t dims[3] = {64, (cuuint64_t)w.Q, (cuuint64_t)(d.C_out / 64)};
      cuuint64_t strides[2] = {(cuuint64_t)d.C_out * 2, 128};
      cuuint32_t box[3] = {64, (cuuint32_t)kWgPos, 2};
      cuuint32_t estr[3] = {1, 1, 1};
      r = wg_encode_tiled(&tm_dy, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(dy), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
      cuuint64_t dims[2] = {(cuuint64_t)d.C_out, (cuuint64_t)w.Q};
      cuuint64_t strides[1] = {(cuuint64_t)d.C_out * 2};
      cuuint32_t box[2] = {64, (cuuint32_t)kWgPos};
      cuuint32_t estr[2] = {1, 1};
      r = wg_encode_tiled(&tm_dy, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(dy), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return SSCONV_ERR_CUDA;
  }
  {
    // activations: NHWC seen as (c, w, h, n) in im2col mode, as in the forward kernel: base pixels
    // are the filter placements of 64 consecutive output positions, each load adds a tap offset,
    // pixels outside the image read as zero (the zero padding of Eq. 4)
    cuuint64_t dims[4] = {(cuuint64_t)d.C_in, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.N};
    cuuint64_t strides[3] = {(cuuint64_t)d.C_in * 2, (cuuint64_t)d.W * d.C_in * 2,
                             (cuuint64_t)d.H * d.W * d.C_in * 2};
    int lower[2] = {-d.pad_w, -d.pad_h};
    int upper[2] = {d.pad_w - (d.KW - 1) * d.dil_w, d.pad_h - (d.KH - 1) * d.dil_h};
    cuuint32_t estr[4] = {1, (cuuint32_t)d.stride_w, (cuuint32_t)d.stride_h, 1};
    if (wg_encode_im2col(&tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(x), dims, strides, lower,
                         upper, (cuuint32_t)kBlockK, (cuuint32_t)kWgPos, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SSCONV_ERR_CUDA;
  }

  WgParams p;
  p.C_in = d.C_in;
  p.C_out = d.C_out;
  p.Ho = Ho;
  p.Wo = Wo;
  p.Q = (int)w.Q;
  p.stride_h = d.stride_h;
  p.stride_w = d.stride_w;
  p.pad_h = d.pad_h;
  p.pad_w = d.pad_w;
  p.dil_h = d.dil_h;
  p.dil_w = d.dil_w;
  p.KW = d.KW;
  p.taps = w.taps;
  p.kblocks = w.kblocks;
  p.T = w.T;
  p.items_b = w.items_b;
  p.m_tiles = w.m_tiles;
  p.splits = w.splits;
  p.ksteps = w.ksteps;
  p.ksteps_per_split = w.ksteps_per_split;
  p.dy_one_load = (d.C_out % 64 == 0) ? 1 : 0;
  p.out = static_cast<float*>(ws);
  p.dev_status = dev_status;

  const unsigned grid = (unsigned)(w.splits * w.m_tiles * w.items_b);
  ssconv_wgrad_kernel<<<grid, kWgThreads, kWgSmemBytes, stream>>>(tm_dy, tm_x, p);
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return SSCONV_ERR_CUDA;
  {
    const int K = w.taps * d.C_in;
    const dim3 rgrid((unsigned)((K + 7) / 8), (unsigned)((d.C_out + 31) / 32));
    wgrad_reduce_kernel<<<rgrid, dim3(32, 8), 0, stream>>>(static_cast<const float*>(ws), w.splits, K, d.C_out,
                                                           w.m_tiles, dw);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return SSCONV_ERR_CUDA;
  }
  return SSCONV_OK;
}

}  // namespace ssconv
