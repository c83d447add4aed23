// Geometry of the compressed 2:4 operand as the forward kernel consumes it.
//
// The weight matrix W [C_out x K], K ordered (kh, kw, c_in), is cut along K into "k-blocks"
// of 64 dense columns that never straddle a filter tap: a k-block is 64 consecutive input
// channels (a "channel chunk", the last one possibly partly padding) at one tap.  K-blocks are
// numbered chunk-major, b = chunk * taps + tap, so that all taps of one channel chunk are
// consecutive: the forward kernel can then serve them from one staged run of activations.
// The block count is rounded up to even (the extra block is padding).  Two consecutive
// k-blocks share one weight tile of the sparse kernel (128 dense columns = 64 kept values
// per row).
//
// Value blob:    bf16 [Mp][KC], Mp = C_out rounded up to 128, KC = 32 * n_kblocks_padded.
//                Column 32*b + 2*q + s holds kept value s (0 = lower position) of the q-th
//                group of k-block b; padding is +0.
// Metadata blob: [Mp/128][n_stages] images of 2048 bytes.  An image is what one
//                tcgen05.cp 128x128b moves into 4 TMEM columns: 128 lanes x 4 words.
//                Word j of lane L belongs to the j-th sparse MMA of the stage (32 dense
//                columns each): its low half describes row (L%8) + 16*(L/16), its high half
//                that row + 8, both for the 16 dense columns starting at 32*j + 16*((L/8)%2):
//                four 4-bit codes, lowest group in the lowest nibble, code = pos0 | pos1<<2.
//                Padding groups carry the legal code 0x4.
#pragma once

#include <stdint.h>

#include "ssconv.h"

namespace ssconv {

constexpr int kTileM = 128;          // rows of W (output channels) per CTA tile
constexpr int kBlockK = 64;          // dense columns per k-block
constexpr int kMetaImageBytes = 2048;

struct Geometry {
  int taps;          // KH*KW
  int cblocks;       // k-blocks per tap = ceil(C_in/64)
  int kblocks;       // taps*cblocks, numbered chunk * taps + tap
  int kblocks_pad;   // rounded up to even
  int stages;        // kblocks_pad/2 (sparse pipeline stages per tile)
  int m_tiles;       // ceil(C_out/128)
  int Mp;            // m_tiles*128
  int KC;            // 32*kblocks_pad: kept values per padded row
};

// kb_channels: input channels per k-block: 64 for bf16 (a 128-byte row of 16-bit elements), 128 for
// 8-bit operands.  The byte sizes (KC kept values of 2 bytes, or 2 KC kept bytes... per row) work out
// the same: 64 bytes of kept values per row and k-block either way.
__host__ __device__ inline Geometry make_geometry(const ssconv_desc_t& d, int kb_channels = kBlockK) {
  Geometry g;
  g.taps = d.KH * d.KW;
  g.cblocks = (d.C_in + kb_channels - 1) / kb_channels;
  g.kblocks = g.taps * g.cblocks;
  g.kblocks_pad = (g.kblocks + 1) & ~1;
  g.stages = g.kblocks_pad / 2;
  g.m_tiles = (d.C_out + kTileM - 1) / kTileM;
  g.Mp = g.m_tiles * kTileM;
  g.KC = 32 * g.kblocks_pad;
  return g;
}

// 4-bit position code (pos0 | pos1 << 2) of the six patterns, lexicographic in the kept
// positions: {0,1},{0,2},{0,3},{1,2},{1,3},{2,3}.  A pattern index outside 0..5 (the array comes
// from the caller's device memory and cannot be checked on the host) is treated as pattern 0, so that
// whatever is in the array the metadata stays legal for the sparse MMA (two ascending positions).
__host__ __device__ inline uint32_t pattern_code(uint32_t p) {
  const uint32_t codes = 0x4u | (0x8u << 4) | (0xCu << 8) | (0x9u << 12) | (0xDu << 16) | (0xEu << 20);
  return p < 6u ? (codes >> (4 * p)) & 0xFu : 0x4u;
}
// Inverse: 4-bit code -> pattern index, 0xFF for a code that is not two ascending positions.
__host__ __device__ inline uint32_t code_pattern(uint32_t code) {
  switch (code & 0xFu) {
    case 0x4: return 0;
    case 0x8: return 1;
    case 0xC: return 2;
    case 0x9: return 3;
    case 0xD: return 4;
    case 0xE: return 5;
    default: return 0xFFu;
  }
}

// Kernels launched by this library in this process (all devices, all threads); see ssconv_launch_count.
void count_launch();

// The residue classes of a strided layer's input gradient (at most 4 x 4): per class the tensor its
// convolution wrote, [N, rows, cols, C_in] bf16, or null for a class that meets no filter tap.
constexpr int kMaxDgradClasses = 16;
struct DgradClasses {
  const void* t[kMaxDgradClasses];
  int rows[kMaxDgradClasses];
  int cols[kMaxDgradClasses];
};

}  // namespace ssconv
