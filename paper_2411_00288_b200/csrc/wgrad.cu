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

// How a layer's weight gradient is cut into work items.
struct WgPlan {
  int taps, kblocks, T, items_b, m_tiles, ksteps, splits, ksteps_per_split;
  long long Q;
};
WgPlan wg_plan(const ssconv_desc_t& d, int sms) {
  WgPlan w;
  w.taps = d.KH * d.KW;
  w.kblocks = w.taps * ((d.C_in + kBlockK - 1) / kBlockK);
  const int groups = (w.kblocks + kWgMaxT - 1) / kWgMaxT;
  w.T = (w.kblocks + groups - 1) / groups;
  w.items_b = (w.kblocks + w.T - 1) / w.T;
  w.m_tiles = (d.C_out + kTileM - 1) / kTileM;
  w.Q = (long long)d.N * wg_out_extent(d.H, d.KH, d.stride_h, d.pad_h, d.dil_h) *
        wg_out_extent(d.W, d.KW, d.stride_w, d.pad_w, d.dil_w);
  w.ksteps = (int)((w.Q + kWgPos - 1) / kWgPos);
  // Split the positions when the items alone would leave SMs idle, but keep at least 8 steps per
  // range so that the pipeline's ramp and the epilogue stay small against the loop.
  const int items = w.m_tiles * w.items_b;
  int splits = sms / items;
  if (splits > w.ksteps / 8) splits = w.ksteps / 8;
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

// Scratch the layer's weight gradient needs on the current device: one slice per position range.
int32_t wgrad_workspace_bytes(const ssconv_desc_t& d, size_t* bytes) {
  int sms = 0;
  const int32_t st = wg_sm_count(&sms);
  if (st != SSCONV_OK) return st;
  const WgPlan w = wg_plan(d, sms);
  *bytes = (size_t)w.splits * w.m_tiles * kTileM * w.taps * d.C_in * sizeof(float);
  return SSCONV_OK;
}

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
  const size_t slice_bytes = (size_t)w.m_tiles * kTileM * w.taps * d.C_in * sizeof(float);
  if (ws == nullptr || ws_bytes < (size_t)w.splits * slice_bytes) return SSCONV_ERR_WORKSPACE;
  const int Ho = wg_out_extent(d.H, d.KH, d.stride_h, d.pad_h, d.dil_h);
  const int Wo = wg_out_extent(d.W, d.KW, d.stride_w, d.pad_w, d.dil_w);

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
