// Thin inline-PTX wrappers for the sm_100a features the convolution kernels use:
// mbarrier, TMA (tiled, im2col, bulk), tcgen05 (alloc, mma, mma.sp, cp, ld, commit).
// Every wait in here is bounded: see mbar_wait_bounded.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ssconv {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Spin on a phase of an mbarrier for at most `spins` tries, entirely inside one asm block: the
// common short wait costs a few instructions and no call.  Returns whether the phase completed.
__device__ __forceinline__ bool mbar_spin_a(uint32_t bar_addr, uint32_t parity, uint32_t spins) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .u32 n;\n\t"
      "mov.u32 n, %3;\n"
      "SPIN:\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "@p bra DONE;\n\t"
      "sub.u32 n, n, 1;\n\t"
      "setp.ne.u32 q, n, 0;\n\t"
      "@q bra SPIN;\n"
      "DONE:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar_addr), "r"(parity), "r"(spins)
      : "memory");
  return ok != 0;
}

// Out-of-line continuation of a wait that outlasted the fast spin: polls on, but never forever.
// After `limit_cycles` SM clock cycles without completion, or as soon as another thread of the
// CTA has raised *abort_flag, it gives up and returns false.
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar_addr, uint32_t parity, volatile int* abort_flag,
                                            long long limit_cycles, uint32_t backoff_ns) {
  const long long t0 = clock64();
  while (true) {
    if (mbar_spin_a(bar_addr, parity, 64)) return true;
    if (*abort_flag != 0) return false;
    if (clock64() - t0 > limit_cycles) {
      *abort_flag = 1;
      return false;
    }
    if (backoff_ns) __nanosleep(backoff_ns);
  }
}

// Wait for a phase of an mbarrier, but never forever (see mbar_wait_slow).  The caller then leaves
// its loop and the CTA drains (see the kernels' tail).  `backoff_ns` > 0 makes a long wait sleep
// between polls: for roles whose waits are long and not latency critical.
constexpr uint32_t kFastSpins = 2048;
__device__ __forceinline__ bool mbar_wait_a(uint32_t bar_addr, uint32_t parity, volatile int* abort_flag,
                                            long long limit_cycles, uint32_t backoff_ns = 0) {
  if (mbar_spin_a(bar_addr, parity, kFastSpins)) return true;
  return mbar_wait_slow(bar_addr, parity, abort_flag, limit_cycles, backoff_ns);
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                  long long limit_cycles, uint32_t backoff_ns = 0) {
  return mbar_wait_a(smem_u32(bar), parity, abort_flag, limit_cycles, backoff_ns);
}

// ---------------------------------------------------------------- proxies / fences
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------- TMA loads

// ---------------------------------------------------------------- fragment -> shared memory
// Four 8x8 matrices of 16-bit elements, each stored transposed: register i of thread t holds
// elements (row t/4, columns 2(t%4), 2(t%4)+1) of matrix i; thread 8i+j supplies the address of
// the 16 bytes that receive column j of matrix i.
__device__ __forceinline__ void stmatrix_x4_trans(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(r0), "r"(r1),
               "r"(r2), "r"(r3)
               : "memory");
}
// The inverse: thread t receives in register i elements (row t/4, columns 2(t%4), 2(t%4)+1) of
// matrix i, read transposed from the 16-byte rows whose addresses threads 8i+j supply.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
// Low and high bf16 of a packed pair as floats (exact).
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }
// Two floats -> packed bf16 pair (lo in the low half), round to nearest even, optionally max(., 0).
template <bool RELU>
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  if (RELU)
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  else
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// Programmatic dependent launch: a grid launched with programmatic stream serialisation may start
// while the grid before it in the stream is still running.  grid_dependency_wait() returns once
// that grid has completed and its memory operations are visible; until then this grid must not
// touch global memory the earlier grid may read or write.  grid_launch_dependents() lets the grid
// after this one start as soon as every CTA of this grid has called it or exited.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Start fetching a tensor map (a kernel parameter) so that the first copy through it does not wait.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---------------------------------------------------------------- TMA store
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* smem_src, int32_t x, int32_t y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t smem_src, int32_t x, int32_t y, int32_t z,
                                             int32_t w) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(map), "r"(smem_src), "r"(x), "r"(y), "r"(z), "r"(w)
               : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_group_read0() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
// Wait until at most one committed bulk group is still reading its shared-memory source.
__device__ __forceinline__ void bulk_wait_group_read1() {
  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
}

// ---------------------------------------------------------------- tcgen05: TMEM management
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
               ::"r"(smem_u32(smem_result)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Arrive (count 1) on an mbarrier once every tcgen05 operation this thread issued so far
// has completed.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(smem_u32(bar))
               : "memory");
}

// ---------------------------------------------------------------- tcgen05: descriptors

// Instruction descriptor of tcgen05.mma kind::f16 with bf16 A and B (both K-major) and an
// fp32 accumulator:
//   bits 0-1 sparsity selector, bit 2 sparse flag, bits 4-5 D format (1 = f32),
//   bits 7-9 A format (1 = bf16), bits 10-12 B format (1 = bf16), bits 15/16 A/B major (0 = K),
//   bits 17-22 N >> 3, bits 24-28 M >> 4.
__host__ __device__ constexpr uint32_t make_idesc_bf16(uint32_t M, uint32_t N, bool sparse) {
  return (sparse ? (1u << 2) : 0u) | (1u << 4) | (1u << 7) | (1u << 10) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

// Instruction descriptor of tcgen05.mma kind::f8f6f4 with e4m3 A and B (format code 0 in bits 7-9 and
// 10-12; both K-major) and an fp32 accumulator; the other fields as above.
__host__ __device__ constexpr uint32_t make_idesc_e4m3(uint32_t M, uint32_t N, bool sparse) {
  return (sparse ? (1u << 2) : 0u) | (1u << 4) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

// ---------------------------------------------------------------- tcgen05: mma / cp / ld

// 16 lanes x 8N consecutive 32-bit columns in the layout of an MMA accumulator fragment: per
// group of 8 columns thread t receives 4 registers: lane (base + t/4), columns 2(t%4) and 2(t%4)+1,
// then lane (base + t/4 + 8), same columns.  base is the first or the 17th lane of the warp's quadrant.
__device__ __forceinline__ void tc_ld_16x256b_x4(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_ld_16x256b_x1(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x1.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- lean forms for the hot loops
// The producer and the MMA issuer are single threads whose instruction streams sit on the critical
// path of every k-block, so their helpers take 32-bit shared-memory addresses and 32-bit descriptor
// halves that the caller keeps in registers, and the slow path of a wait is kept out of line.
__device__ __forceinline__ void mbar_expect_tx_a(uint32_t bar_addr, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_a(uint32_t bar_addr) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_addr) : "memory");
}
__device__ __forceinline__ void tc_commit_a(uint32_t bar_addr) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_addr)
               : "memory");
}
// TMA loads with shared addresses already converted.
__device__ __forceinline__ void tma_load_2d_a(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t x, int32_t y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_a(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t x, int32_t y,
                                              int32_t z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tma_load_im2col_4d_a(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t c,
                                                     int32_t w, int32_t h, int32_t n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}
__device__ __forceinline__ void bulk_load_a(uint32_t dst, const void* gsrc, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(gsrc), "r"(bytes), "r"(bar)
      : "memory");
}

// A shared-memory matrix descriptor is 64 bits:
//   bits  0-13  start address >> 4
//   bits 16-29  leading-dimension byte offset >> 4 (distance between 16-byte K-chunks of an
//               unswizzled tile; not used by swizzled K-major tiles, set to 1)
//   bits 32-45  stride-dimension byte offset >> 4 = distance between groups of 8 rows
//   bits 46-47  descriptor version (1 on sm_100)
//   bits 61-63  swizzle mode (0 = none, 2 = 128 B)
// The kernels build it from two 32-bit halves.  The high half is one of two constants: for a
// K-major tile with 128-byte rows in the 128-byte swizzle (what a TMA load with SWIZZLE_128B
// produces; 8-row groups 1024 B apart), and for an unswizzled tile of 16-byte-wide chunks (8 rows =
// one 128-byte core matrix).  The low half is (address >> 4) | (leading-dimension offset << 16).
constexpr uint32_t kDescHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);
constexpr uint32_t kDescHiNoSwizzle128 = (128u >> 4) | (1u << 14);
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr) { return ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16); }

// D[128 x N] (+)= A[128 x 16] B[N x 16]^T, bf16 operands in swizzled K-major shared-memory tiles, fp32
// accumulator at TMEM address d_tmem; `accumulate` == 0 overwrites D.  Issued by one thread.
__device__ __forceinline__ void tc_mma_dense_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                                uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %5};\n\t"
      "mov.b64 db, {%2, %5};\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
      : "memory");
}
// The 2:4 sparse form (warp-wide, below): A holds the 16 kept values of 32 dense K-columns per row, B
// the 32 columns; meta_tmem is the TMEM column with the 2-bit indices of those columns (bit 0 of the
// column address is passed in the instruction descriptor's selector bits by the caller).
// tcgen05.cp 128x128b copies 128 rows x 128 bits from shared memory (unswizzled, 16-byte rows) into 4
// TMEM columns, row r to lane r: one weight tile's metadata image; it is ordered with the MMAs of the
// issuing thread.

// ---------------------------------------------------------------- warp-wide forms
// The same tcgen05 instructions for a loop that all 32 lanes of a warp execute in lock step, with one
// elected lane issuing: the operands (descriptors, TMEM and barrier addresses) are then uniform over
// the warp, which lets the compiler keep them in the uniform register file that these instructions
// read; inside a branch taken by a single lane every operand has to be moved there per instruction
// (measured on the forward kernel's issuing loop: 80 -> 62 cycles per tcgen05 instruction, 256 -> 205
// per wait on a complete barrier).
// desc_hi = kDescHiNoSwizzle128 selects unswizzled K-major operands: 16-byte chunks of 8 K-elements;
// within a chunk the rows follow each other every 16 bytes (8 rows = one 128-byte core matrix), chunks
// follow each other every `chunk stride` bytes, which goes into bits 16-29 of the low word as the
// leading-dimension offset: lo = (address >> 4) | ((chunk stride >> 4) << 16).
__device__ __forceinline__ void tc_mma_dense_w(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                               uint32_t accumulate, uint32_t desc_hi = kDescHiSw128) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b64 da, {%1, %5};\n\t"
      "mov.b64 db, {%2, %5};\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(desc_hi)
      : "memory");
}
__device__ __forceinline__ void tc_mma_sparse_w(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t meta_tmem,
                                                uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b64 da, {%1, %6};\n\t"
      "mov.b64 db, {%2, %6};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "@e tcgen05.mma.sp.cta_group::1.kind::f16 [%0], da, db, [%3], %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(meta_tmem), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
      : "memory");
}
__device__ __forceinline__ void tc_cp_128x128b_w(uint32_t dst_tmem, uint32_t src_lo) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t.reg .b64 ds;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b64 ds, {%1, %2};\n\t"
      "@e tcgen05.cp.cta_group::1.128x128b [%0], ds;\n\t}"
      ::"r"(dst_tmem), "r"(src_lo), "r"(kDescHiNoSwizzle128)
      : "memory");
}
__device__ __forceinline__ void tc_commit_w(uint32_t bar_addr) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar_addr)
      : "memory");
}

// Producer side, warp-wide: the whole warp waits and walks the loop, one elected lane arrives on the
// barrier and issues the copies (their tensor-map, shared-memory and barrier operands are uniform).
__device__ __forceinline__ void mbar_expect_tx_w(uint32_t bar_addr, uint32_t bytes) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t}" ::"r"(bar_addr), "r"(bytes)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_w(uint32_t bar_addr) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}" ::"r"(bar_addr)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_w(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t x, int32_t y) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];\n\t}"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_w(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t x, int32_t y,
                                              int32_t z) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];\n\t}"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tma_load_im2col_4d_w(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t c,
                                                     int32_t w, int32_t h, int32_t n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};\n\t}"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}
__device__ __forceinline__ void bulk_load_w(uint32_t dst, const void* gsrc, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n\t}"
      ::"r"(dst), "l"(gsrc), "r"(bytes), "r"(bar)
      : "memory");
}

// 8-bit operands (kind::f8f6f4, here e4m3): a dense MMA covers K = 32 elements, a 2:4 sparse one K = 64
// (A holds the 32 kept bytes per row); in bytes per row the operand steps are those of the 16-bit forms.
__device__ __forceinline__ void tc_mma_f8_dense_w(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                                  uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b64 da, {%1, %5};\n\t"
      "mov.b64 db, {%2, %5};\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
      : "memory");
}
__device__ __forceinline__ void tc_mma_f8_sparse_w(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t meta_tmem,
                                                   uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b64 da, {%1, %6};\n\t"
      "mov.b64 db, {%2, %6};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "@e tcgen05.mma.sp.cta_group::1.kind::f8f6f4 [%0], da, db, [%3], %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(meta_tmem), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
      : "memory");
}

// ---------------------------------------------------------------- CTA pairs (cta_group::2)
// Two CTAs of a cluster work on one MMA: M = 256 (each CTA holds 128 rows of A and of the
// accumulator in its own shared memory and TMEM), each CTA supplies half of B's N rows; the
// instructions are issued by a thread of the even CTA (the leader) with shared-memory offsets that
// are the same in both CTAs.  Every tcgen05 instruction of such a kernel uses cta_group::2, and the
// TMEM allocation is made by one warp in each of the two CTAs.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address, in the cluster's shared window, of the same shared-memory location in CTA `rank`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// Arrive (count 1) on an mbarrier anywhere in the cluster (address from map_to_cta).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t* smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
               ::"r"(smem_u32(smem_result)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Warp-wide forms (one elected lane issues), as above.
__device__ __forceinline__ void tc2_mma_dense_w(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                                uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b64 da, {%1, %5};\n\t"
      "mov.b64 db, {%2, %5};\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
      : "memory");
}
__device__ __forceinline__ void tc2_mma_sparse_w(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t meta_tmem,
                                                 uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b64 da, {%1, %6};\n\t"
      "mov.b64 db, {%2, %6};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "@e tcgen05.mma.sp.cta_group::2.kind::f16 [%0], da, db, [%3], %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(meta_tmem), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
      : "memory");
}
__device__ __forceinline__ void tc2_mma_f8_sparse_w(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t meta_tmem,
                                                    uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b64 da, db;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b64 da, {%1, %6};\n\t"
      "mov.b64 db, {%2, %6};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "@e tcgen05.mma.sp.cta_group::2.kind::f8f6f4 [%0], da, db, [%3], %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(meta_tmem), "r"(idesc), "r"(accumulate), "r"(kDescHiSw128)
      : "memory");
}
// In both CTAs: 128 rows x 128 bits from the CTA's own shared memory into its own TMEM.
__device__ __forceinline__ void tc2_cp_128x128b_w(uint32_t dst_tmem, uint32_t src_lo) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t.reg .b64 ds;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b64 ds, {%1, %2};\n\t"
      "@e tcgen05.cp.cta_group::2.128x128b [%0], ds;\n\t}"
      ::"r"(dst_tmem), "r"(src_lo), "r"(kDescHiNoSwizzle128)
      : "memory");
}
// Arrive on one mbarrier (cluster address: it may be the peer's) once the pair's MMAs issued so far are done.
__device__ __forceinline__ void tc2_commit_w(uint32_t cluster_bar_addr) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "@e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(cluster_bar_addr)
      : "memory");
}
// The same arrival delivered to the mbarrier at this shared-memory offset in both CTAs of the pair.
// (A commit, not a copy: no data is multicast.)
__device__ __forceinline__ void tc2_commit_both_w(uint32_t bar_addr) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t.reg .b16 m;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "mov.b16 m, 3;\n\t"
      "@e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}"
      ::"r"(bar_addr)
      : "memory");
}
// One non-blocking look at a phase of an mbarrier.  Issued when a ring slot is taken up, for the slot
// after it, its latency hides behind the MMAs in between, where a wait that starts only when the data
// is needed stalls the issuing warp for some 200 cycles even on a complete barrier.
__device__ __forceinline__ uint32_t mbar_test_a(uint32_t bar_addr, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar_addr), "r"(parity)
      : "memory");
  return ok;
}
// TMA loads into this CTA's shared memory whose completion is signalled on an mbarrier that may live
// in the peer CTA (cluster address).
__device__ __forceinline__ void tma2_load_2d_w(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t x, int32_t y) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];\n\t}"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tma2_load_3d_w(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t x, int32_t y,
                                               int32_t z) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];\n\t}"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tma2_load_im2col_4d_w(uint32_t dst, const CUtensorMap* map, uint32_t bar, int32_t c,
                                                      int32_t w, int32_t h, int32_t n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
      "@e cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};\n\t}"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}

}  // namespace ssconv
