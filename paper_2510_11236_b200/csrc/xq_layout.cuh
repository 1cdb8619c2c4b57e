// Packed layouts of the quantized KV cache (this library's choice; the paper
// does not discuss packing).  One stream per (sequence, kv head).
//
// Code tile = 128 uint32 words (512 bytes).  Each 16-bit half of a word is cut
// into NSLOT = 16/bits slots, slot 0 in the least significant bits.  The D/16
// channel blocks of a token share the slots of a word; when slots remain,
// consecutive 16-token sub-tiles fill them, so a tile spans
// TPT = 16 * NSLOT / (D/16) tokens.  Inside a 16x16 (row, col) block the element
// (row, col) sits in word 4*lane + i, half hf, with
//     lane = (row % 8) * 4 + (col % 8) / 2,  i = row / 8 + 2 * (col / 8),  hf = col % 2.
// Keys: row = token, col = channel.  Values: row = channel, col = token.
// This is the A-operand register layout of mma.sync.m16n8k16: thread `lane`
// loads one 128-bit vector {word 4*lane .. 4*lane+3}, and `word & (mask << slot)`
// is, for every slot, a ready fp16x2 fragment register whose two halves hold the
// integer code times 2^(bits*slot) as fp16 subnormals (value * 2^-24).
//
// Key scale/zero: per stream two planes of [groups][D] fp16, all scale blocks
// first, then all zero-point blocks (plane stride = group capacity * D), so that
// the zero-point blocks of consecutive token groups are contiguous.  Inside a
// block the D values are cut into 16-byte chunks, chunk (d/32)*4 + ((d%16)%8)/2
// holding, for the two 16-channel blocks 2*(d/32) and 2*(d/32)+1, the four
// values (d%16 in {2t, 2t+1, 2t+8, 2t+9}) that B-operand thread t of an
// mma.sync.m16n8k16 needs: index ((d/16)%2)*4 + ((d%16)/8)*2 + d%2 in the chunk.
// The four threads of a quad then read 64 contiguous bytes per load.
// Value scale/zero: per 16 tokens two blocks of 16*NG fp16 (NG = D/g), entry
// (token tk, group gi) at ((tk%8)/2) * (4*NG) + gi*4 + (tk/8)*2 + tk%2.
#pragma once
#include <stdint.h>

namespace xq {

__host__ __device__ inline int tokens_per_code_tile(int bits, int D) { return 16 * ((16 / bits) / (D / 16)); }

struct CodePos {
  int word;  // index within the stream
  int bit;   // bit offset of the code's least significant bit
};

// (row, col) of a 16x16 block, sub-tile tt, channel block cb -> position in tile
__host__ __device__ inline CodePos block_position(int tile, int tt, int cb, int row, int col, int bits, int D) {
  int lane = (row & 7) * 4 + ((col & 7) >> 1);
  int i = (row >> 3) + 2 * (col >> 3);
  int slot = tt * (D / 16) + cb;
  CodePos p;
  p.word = tile * 128 + lane * 4 + i;
  p.bit = 16 * (col & 1) + bits * slot;
  return p;
}

__host__ __device__ inline CodePos k_code_position(int t, int d, int bits, int D) {
  int tpt = tokens_per_code_tile(bits, D);
  int tile = t / tpt, tl = t % tpt;
  return block_position(tile, tl / 16, d / 16, tl % 16, d % 16, bits, D);
}

__host__ __device__ inline CodePos v_code_position(int t, int d, int bits, int D) {
  int tpt = tokens_per_code_tile(bits, D);
  int tile = t / tpt, tl = t % tpt;
  return block_position(tile, tl / 16, d / 16, d % 16, tl % 16, bits, D);
}

__host__ __device__ inline int k_meta_position(int d, int D) {
  (void)D;
  int cb = d / 16, kk = d % 16;
  int chunk = (cb >> 1) * 4 + ((kk & 7) >> 1);
  return chunk * 8 + (cb & 1) * 4 + (kk >> 3) * 2 + (kk & 1);
}

__host__ __device__ inline int v_meta_position(int tk, int gi, int n_g) {
  return ((tk & 7) >> 1) * (4 * n_g) + gi * 4 + (tk >> 3) * 2 + (tk & 1);
}

}  // namespace xq
