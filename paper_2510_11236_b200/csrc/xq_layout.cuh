// Packed layouts of the quantized KV cache (this library's choice; the paper
// does not discuss packing).  One stream per (sequence, kv head).
//
// The layouts serve a decode kernel in which one thread owns one row of a
// tensor-core A operand held in tensor memory: a token's channels for the keys,
// a channel's tokens for the values.  A row is expanded from its packed words
// with one AND per four codes: the codes of four consecutive row elements sit at
// the same bit offset of the four bytes of a word, so `word & (mask << s)` is four
// 8-bit operand elements at once (the code times 2^s).
//
// Key codes.  Token t, channel d, B bits.  A token's row is D*B/32 words; rows
// are grouped by units of 32 tokens, a unit being stored as chunks of up to 16
// bytes per token ([chunk][token][bytes]) so that the 32 threads of a warp read
// consecutive 16-byte vectors.  Word i of the row holds the channels
// [i*32/B, (i+1)*32/B); inside it channel d sits in byte d % 4 at bit
// B * ((d % (32/B)) / 4) of that byte.
//
// Value codes.  Same with the roles swapped, per batch of 128 tokens: channel d
// owns a row of 128*B/32 words, stored [chunk][channel][16 bytes]; word i holds
// the tokens [i*32/B, (i+1)*32/B) of the batch, token t in byte t % 4 at bit
// B * ((t % (32/B)) / 4).
//
// Key scale / zero-point: per token group 2*D fp16: the D scales, then the D
// zero-points, each in the order pos(d) = (d % 32) * (D/32) + d / 32 (a lane of
// the decode kernel owns the channels lane, lane + 32, ... and reads them as one
// vector).  Value scale / zero-point: per token 2*NG fp16 (NG = D/g): the NG
// scales, then the NG zero-points.
#pragma once
#include <stdint.h>

namespace xq {

constexpr int XQ_BATCH = 128;  // tokens per value-code batch (and per decode tile)

struct CodePos {
  size_t word;  // 32-bit word index within the stream
  int bit;      // bit offset of the code's least significant bit
};

// words per token row (keys) / per channel row of one batch (values)
__host__ __device__ inline int k_row_words(int bits, int D) { return D * bits / 32; }
__host__ __device__ inline int v_row_words(int bits) { return XQ_BATCH * bits / 32; }

__host__ __device__ inline CodePos k_code_position(int t, int d, int bits, int D) {
  const int per_word = 32 / bits;
  const int i = d / per_word;               // word of the row
  const int row_bytes = D * bits / 8;
  const int chunk_bytes = row_bytes < 16 ? row_bytes : 16;
  const int chunk = (i * 4) / chunk_bytes, in_chunk = (i * 4) % chunk_bytes;
  const size_t unit = (size_t)(t / 32) * (32 * row_bytes);
  CodePos p;
  p.word = (unit + (size_t)chunk * (32 * chunk_bytes) + (size_t)(t % 32) * chunk_bytes + in_chunk) / 4;
  p.bit = 8 * (d % 4) + bits * ((d % per_word) / 4);
  return p;
}

__host__ __device__ inline CodePos v_code_position(int t, int d, int bits, int D) {
  const int per_word = 32 / bits;
  const int tl = t % XQ_BATCH;
  const int i = tl / per_word;              // word of the channel's row
  const size_t batch = (size_t)(t / XQ_BATCH) * ((size_t)D * 16 * bits);
  CodePos p;
  p.word = (batch + (size_t)(i / 4) * (D * 16) + (size_t)d * 16 + (i % 4) * 4) / 4;
  p.bit = 8 * (tl % 4) + bits * ((tl % per_word) / 4);
  return p;
}

// index of channel d inside the D scales (or the D zero-points) of a key token group
__host__ __device__ inline int k_meta_position(int d, int D) { return (d % 32) * (D / 32) + d / 32; }

// fp16 index, within a stream's value scale / zero-point region, of token t, channel group gi
__host__ __device__ inline size_t v_scale_index(int t, int gi, int n_g) { return (size_t)t * 2 * n_g + gi; }
__host__ __device__ inline size_t v_zero_index(int t, int gi, int n_g) { return (size_t)t * 2 * n_g + n_g + gi; }

// tokens of capacity the code and value-parameter regions are sized for (whole batches)
__host__ __device__ inline int padded_capacity(int nq_cap) { return (nq_cap + XQ_BATCH - 1) / XQ_BATCH * XQ_BATCH; }

}  // namespace xq
