// Packed layouts of the quantized KV cache (this library's choice; the paper
// does not discuss packing).  One stream per (sequence, kv head).  The layouts
// are made for the decode kernel, which expands codes into fp16 tensor-core
// operands held in tensor memory, one matrix row per thread:
//
// Key codes -- a thread owns a TOKEN and needs all of its channels.  A token's
// D codes fill W = D*bits/32 words; word j holds channels [j*cpw, (j+1)*cpw),
// cpw = 32/bits: channel j*cpw + 2s in the low 16 bits and j*cpw + 2s + 1 in the
// high 16 bits, both at bit bits*s, so that `word & (mask << bits*s)` is an
// fp16x2 pair (channel 2c, 2c+1) = one 32-bit column of a K-major fp16 operand
// row (a code in the low mantissa bits of an fp16 is the subnormal c * 2^(pos-24)).
// Words are stored per 32-token unit as [W/CW][32 tokens][CW words], CW = min(4, W),
// so that the 32 threads of a warp read consecutive 16-byte chunks.
//
// Value codes -- a thread owns a CHANNEL and needs the tokens of a 128-token
// block.  Per block and channel WB = 128*bits/32 words; word j holds tokens
// [j*cpw, (j+1)*cpw) of the block, token j*cpw + 2s low, j*cpw + 2s + 1 high, at
// bit bits*s.  Stored per block as [WB/4][D channels][4 words].
//
// Key scale/zero: per stream two planes of [groups][D] fp16 in channel order,
// all scale blocks first, then all zero-point blocks.
// Value scale/zero: per token [2][NG] fp16 (NG = D/g): scales, then zero-points.
//
// Capacities of the quantized regions are rounded up to whole 128-token blocks.
#pragma once
#include <stdint.h>

namespace xq {

struct CodePos {
  int word;  // index within the stream
  int bit;   // bit offset of the code's least significant bit
};

__host__ __device__ inline int k_words_per_token(int bits, int D) { return D * bits / 32; }
__host__ __device__ inline int v_words_per_block_channel(int bits) { return 128 * bits / 32; }

__host__ __device__ inline CodePos k_code_position(int t, int d, int bits, int D) {
  const int W = k_words_per_token(bits, D), cpw = 32 / bits, CW = W < 4 ? W : 4;
  const int j = d / cpw, r = d % cpw;
  CodePos p;
  p.word = (t / 32) * (32 * W) + ((j / CW) * 32 + (t % 32)) * CW + (j % CW);
  p.bit = 16 * (r & 1) + bits * (r >> 1);
  return p;
}

__host__ __device__ inline CodePos v_code_position(int t, int d, int bits, int D) {
  const int WB = v_words_per_block_channel(bits), cpw = 32 / bits;
  const int tb = t % 128, j = tb / cpw, r = tb % cpw;
  CodePos p;
  p.word = (t / 128) * (D * WB) + ((j / 4) * D + d) * 4 + (j % 4);
  p.bit = 16 * (r & 1) + bits * (r >> 1);
  return p;
}

// index (in fp16 units) of the value scale (which = 0) or zero-point (which = 1) of token t, channel group gi
__host__ __device__ inline size_t v_meta_index(int t, int gi, int which, int n_g) {
  return (size_t)t * (2 * n_g) + which * n_g + gi;
}

__host__ __device__ inline int round_up_128(int x) { return (x + 127) / 128 * 128; }

}  // namespace xq
