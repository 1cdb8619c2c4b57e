// Quantize-and-pack of residual-window blocks (Eq. 1, 2, 12; Algorithm 2) and
// the window append.  One CTA quantizes a tile of T (32 or 64) tokens x D channels of
// one (sequence, kv head) for keys or for values.
//
// The fp32 arithmetic uses the *_rn intrinsics so that no multiply-add is ever
// contracted: codes, scales and zero-points are compared bit for bit with a CPU
// evaluation of the same formulas.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "xq_internal.h"
#include "xq_layout.cuh"

namespace xq {

__device__ __forceinline__ float bf16_bits(uint16_t u) { return __uint_as_float(((uint32_t)u) << 16); }

// The 16-bit input type: widening to fp32 (exact) and packed min / max of two elements.
template <bool F16>
struct In16;
template <>
struct In16<false> {
  using V2 = __nv_bfloat162;
  static __device__ __forceinline__ float lo(uint32_t w) { return __uint_as_float(w << 16); }
  static __device__ __forceinline__ float hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
  static __device__ __forceinline__ float one(uint16_t u) { return bf16_bits(u); }
  // pattern of the nearest 16-bit value (of x itself when it is one)
  static __device__ __forceinline__ uint32_t bits(float x) { return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x)); }
  // the nearest 16-bit value at or above / at or below x
  static __device__ __forceinline__ uint32_t bits_up(float x) { return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_ru(x)); }
  static __device__ __forceinline__ uint32_t bits_down(float x) { return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rd(x)); }
};
template <>
struct In16<true> {
  using V2 = __half2;
  static __device__ __forceinline__ float lo(uint32_t w) { return __half2float(__ushort_as_half((unsigned short)(w & 0xffffu))); }
  static __device__ __forceinline__ float hi(uint32_t w) { return __half2float(__ushort_as_half((unsigned short)(w >> 16))); }
  static __device__ __forceinline__ float one(uint16_t u) { return __half2float(__ushort_as_half(u)); }
  static __device__ __forceinline__ uint32_t bits(float x) { return (uint32_t)__half_as_ushort(__float2half_rn(x)); }
  static __device__ __forceinline__ uint32_t bits_up(float x) { return (uint32_t)__half_as_ushort(__float2half_ru(x)); }
  static __device__ __forceinline__ uint32_t bits_down(float x) { return (uint32_t)__half_as_ushort(__float2half_rd(x)); }
};

// Merged words of a sharing pair (Appendix F): field by field, the code of (e0, e1) from the table.
template <int BITS>
__device__ __forceinline__ uint32_t merge_words(uint32_t w0, uint32_t w1, uint32_t lut) {
  uint32_t out = 0u;
#pragma unroll
  for (int f = 0; f < 32; f += BITS) {
    const uint32_t e0 = (w0 >> f) & ((1u << BITS) - 1u), e1 = (w1 >> f) & ((1u << BITS) - 1u);
    out |= ((lut >> (2u * (4u * e0 + e1))) & ((1u << BITS) - 1u)) << f;
  }
  return out;
}

// Eq. 1 and Eq. 12 for one group: z = min, s = (max - min)/(2^B - 1),
// z_hat = z + (eta * s) * (2^B - 1), s_hat = (1 - 2 eta) * s.
__device__ __forceinline__ void group_params(float mn, float mx, int bits, float eta, float& z, float& s,
                                             __half& zh, __half& sh) {
  const float qmax = (float)((1 << bits) - 1);
  s = __fdiv_rn(__fsub_rn(mx, mn), qmax);
  z = mn;
  float t = __fmul_rn(__fmul_rn(eta, s), qmax);
  zh = __float2half_rn(__fadd_rn(z, t));
  float k = __fsub_rn(1.0f, __fmul_rn(2.0f, eta));
  sh = __float2half_rn(__fmul_rn(k, s));
}

constexpr int PACK_THREADS = 128;
constexpr int PACK_ROW_PAD = 16;  // bytes added to each staged row: 8 consecutive rows then fall in 8 different bank groups

// 1/s for the quotient sequence of `quotient`: 0 for a constant group (every code 0), NaN where that sequence is
// not known to round correctly -- a scale whose significand is all ones, or one so small or large that an
// intermediate could leave the normal range -- which sends the group to the division.
__device__ __forceinline__ float safe_rcp(float s) {
  if (s == 0.0f) return 0.0f;
  const uint32_t b = __float_as_uint(s);
  const uint32_t e = (b >> 23) & 0xffu;
  if ((b & 0x7fffffu) == 0x7fffffu || e < 40u || e > 210u) return __uint_as_float(0x7fc00000u);
  return __frcp_rn(s);
}

// Codes by comparison (Eq. 2).  The code of x in a group, c(x) = clamp(rint(RN(RN(x - z) / s)), 0, 2^B - 1), never
// decreases with x, and x is a 16-bit float, so the group's codes are fixed by B-bit-many thresholds on the input
// lattice: X_k = the smallest 16-bit value with c(X_k) >= k, and c(x) = #{k : x >= X_k}.  One thread per group
// finds the X_k: next to z + (k - 1/2) s, from the rounding bounds of the quotient where they decide, else by
// evaluating c itself (the quotient exactly as the division gives it, ties of rint to even) at lattice points; the
// elements are then coded two at a time with packed 16-bit compares.

// 16-bit float pattern <-> integer that orders like the value (sign-magnitude to two's complement; -0 and +0 -> 0)
__device__ __forceinline__ int ord16(uint32_t h) {
  const int m = (int)(h & 0x7fffu);
  return (h & 0x8000u) ? -m : m;
}
__device__ __forceinline__ uint32_t pat16(int o) { return o >= 0 ? (uint32_t)o : (0x8000u | (uint32_t)(-o)); }

// A group's uncalibrated parameters for the quotient RN(RN(x - z) / s).  With y = RN(1/s): q = RN(a y),
// r = a - q s (exact in one fused multiply-add), q' = RN(q + r y) is the correctly rounded quotient (the classical
// correction step of division by a correctly rounded reciprocal; the scales it can miss get a NaN from safe_rcp
// and take the division).
struct Quot {
  float z, s, y;
  bool fast;
};
__device__ __forceinline__ float quotient(const Quot& g, float x) {
  const float a = __fsub_rn(x, g.z);
  if (g.fast) {
    const float q = __fmul_rn(a, g.y);
    const float r = __fmaf_rn(-q, g.s, a);
    return __fmaf_rn(r, g.y, q);
  }
  return __fdiv_rn(a, g.s);
}

// X_k as a 16-bit pattern for a group with minimum mn and maximum mx.  In real numbers the threshold is
// tau = z + (k - 1/2) s.  The computed quotient differs from (x - z) / s by less than 2^-23 relative (two
// roundings), i.e. by less than 3.1 * 2^-23 s in x, and t = RN(tau) from tau by at most 2^-24 |t|: a lattice point
// at or above t + eps certainly has c >= k, one below t - eps certainly has not, for eps = 2^-22 |t| + 2^-20 s
// (twice what is needed).  Where the lattice is coarser than eps -- almost always -- no lattice point lies between
// the bounds and nothing is evaluated; otherwise (a threshold next to zero under a large |z|, an exact tie on the
// lattice) c itself decides, by bisection between the bounds.  Groups whose scale takes the division (safe_rcp)
// are bisected from the group's ends (c(mn) = 0, c(mx) = 2^B - 1).
template <bool F16>
__device__ __forceinline__ uint32_t threshold16(const Quot& g, int k, float mn, float mx) {
  const float kk = (float)k - 0.5f;
  int lo, hi;  // ordered integers of lattice points with c(lo) < k <= c(hi)
  if (g.fast) {
    const float t = __fmaf_rn(kk, g.s, g.z);
    const float eps = __fmaf_rn(fabsf(t), 0x1p-22f, __fmul_rn(g.s, 0x1p-20f));
    // the smallest lattice points at or above t + eps and at or above t - eps: the same point when no lattice
    // point lies between the two bounds, and then it is X_k (mn lies below t - eps, mx above t + eps: the
    // thresholds are half a step and more away from both)
    const uint32_t up = In16<F16>::bits_up(__fadd_ru(t, eps)), up_lo = In16<F16>::bits_up(__fadd_rd(t, -eps));
    constexpr uint32_t INF16 = F16 ? 0x7c00u : 0x7f80u;
    if (up == up_lo && up != INF16) return up;
    hi = up != INF16 ? ord16(up) : ord16(In16<F16>::bits(mx));  // (a bound beyond the largest finite value)
    lo = ord16(up_lo) - 1;  // below t - eps
  } else {
    lo = ord16(In16<F16>::bits(mn));
    hi = ord16(In16<F16>::bits(mx));
  }
  const bool even = (k & 1) == 0;  // rint takes a tie to the even neighbour: k - 1/2 counts as >= k only for even k
  while (hi - lo > 1) {
    const int mid = lo + ((hi - lo) >> 1);
    const float q = quotient(g, In16<F16>::one((uint16_t)pat16(mid)));
    if (even ? q >= kk : q > kk) hi = mid; else lo = mid;
  }
  return pat16(hi);
}

// The thresholds of a group with minimum mn and maximum mx (16-bit values, widened) into thr[k * stride]; unused
// ones (k beyond 2^B - 1, or a constant group: every code 0) are +infinity.
template <bool F16>
__device__ __forceinline__ void group_thresholds(float mn, float mx, float z, float sc, int bits, uint16_t* thr, int stride) {
  constexpr uint16_t INF16 = F16 ? 0x7c00u : 0x7f80u;
  const float y = safe_rcp(sc);
  const Quot g{z, sc, y, y == y};
  const int qmax = (1 << bits) - 1;
#pragma unroll
  for (int k = 1; k <= 3; ++k)
    thr[(k - 1) * stride] = (k <= qmax && sc != 0.0f) ? (uint16_t)threshold16<F16>(g, k, mn, mx) : INF16;
}

// Codes of two packed 16-bit elements against their groups' packed thresholds: code of the low element at bit 0,
// of the high element at bit 16.
template <int BITS, typename V2>
__device__ __forceinline__ uint32_t code_pair(uint32_t x, uint32_t t1, uint32_t t2, uint32_t t3) {
  const V2 xv = *reinterpret_cast<const V2*>(&x);
  const uint32_t m1 = __hge2_mask(xv, *reinterpret_cast<const V2*>(&t1));
  if constexpr (BITS == 1) {
    return m1 & 0x00010001u;
  } else {
    const uint32_t m2 = __hge2_mask(xv, *reinterpret_cast<const V2*>(&t2));
    const uint32_t m3 = __hge2_mask(xv, *reinterpret_cast<const V2*>(&t3));
    // A mask is 0xffff per element that passed.  n = -(m1 + m2 + m3) holds the low element's count in its low
    // half and (high count - low count) in its high half (the low half borrows); n * 0x10001 adds the low count
    // back to the high half.
    const uint32_t n = 0u - m1 - m2 - m3;
    return n * 0x10001u;
  }
}

// Adds to hist[d] the number of fields of the two words whose codes differ by d.
template <int BITS>
__device__ __forceinline__ void delta_count(uint32_t w0, uint32_t w1, uint32_t (&hist)[4]) {
#pragma unroll
  for (int f = 0; f < 32; f += BITS) {
    const int e0 = (int)((w0 >> f) & ((1u << BITS) - 1u)), e1 = (int)((w1 >> f) & ((1u << BITS) - 1u));
    const int d = e0 > e1 ? e0 - e1 : e1 - e0;
#pragma unroll
    for (int k = 0; k < (1 << BITS); ++k) hist[k] += d == k;
  }
}

// One CTA: T tokens x D channels of one (sequence, kv head), keys (blockIdx.x even) or values (odd).  Staged
// rows are padded.  Keys: a thread builds whole words of a token's row (four consecutive channels per bit
// offset), the words are collected in shared memory in stream order and leave in 16-byte vectors.  Values: a
// thread builds whole words of a channel's row over the tile's tokens and stores them itself.
// G: group size; T = p.tb: a multiple of G and of 32; F16: the 16-bit type is IEEE half precision.
// blockIdx.y is the (sequence, kv head) stream, blockIdx.z the layer of the launch.  With p.win_count > 0 the CTAs of the first block also copy
// the new window rows that replace the rows they staged.
template <int D, int G, int T, bool F16>
__global__ void __launch_bounds__(PACK_THREADS) pack_kernel(const __grid_constant__ PackParams p) {
  using I16 = In16<F16>;
  using V2 = typename I16::V2;
  constexpr int ROWB = D * 2 + PACK_ROW_PAD;
  constexpr int NG = D / G;
  constexpr int CB = D / 16;
  constexpr int NPAR = (T * NG > (T / G) * D) ? T * NG : (T / G) * D;  // groups of the tile, either kind
  constexpr int KP = PACK_THREADS / ((T / G) * (D / 2));               // token parts of a key group in the statistics
  static_assert(KP >= 1 && G % KP == 0, "key statistics: 128 threads over (group, channel pair, token part)");
  __shared__ __align__(16) uint8_t tile[T * ROWB];
  // thresholds X_1..X_3 of a group: [k][group]; keys: group = [token group][channel], values: [channel group][token]
  __shared__ __align__(16) uint16_t thr[3 * NPAR];
  // packed words (at most T * D * 2 / 32); before that, the key statistics' partial (min, max) pairs, two words per thread
  constexpr int NWBUF = (T * D * 2 / 32) > 2 * PACK_THREADS ? (T * D * 2 / 32) : 2 * PACK_THREADS;
  __shared__ __align__(16) uint32_t wbuf[NWBUF];

  const Dims& dm = p.dm;
  const int R = dm.R;
  const int kind = blockIdx.x & 1;  // 0 keys, 1 values
  const int tile_idx = blockIdx.x >> 1;
  const PackLayer pl = p.layer[blockIdx.z];  // by value: its fields are read in every loop below
  const int bh = blockIdx.y;                  // (sequence, kv head) stream
  const int tid = threadIdx.x;
  const int tq0 = p.nq_old + tile_idx * T;  // absolute index of the tile's first token

  {
    const uint16_t* win = kind ? pl.L.win_v : pl.L.win_k;
    const uint16_t* in = kind ? pl.V_in : pl.K_in;
    constexpr int VPR = D / 8;
    // row `pabs` (absolute token) of the stream: in the old window while pabs < s_old, else in the input
    const uint16_t* const win_rows = win + ((size_t)bh * R - p.nq_old) * D;
    const uint16_t* const in_rows = in + ((size_t)bh * p.n_in - p.s_old) * D;
#pragma unroll
    for (int k = 0; k < T * VPR / PACK_THREADS; ++k) {
      const int idx = tid + k * PACK_THREADS;
      const int tl = idx / VPR, c8 = idx % VPR;
      const int pabs = tq0 + tl;
      const uint16_t* src = (pabs < p.s_old ? win_rows : in_rows) + (size_t)pabs * D;
      *reinterpret_cast<uint4*>(tile + tl * ROWB + c8 * 16) = reinterpret_cast<const uint4*>(src)[c8];
    }
  }
  __syncthreads();
  // the window rows this CTA staged are free: the tokens that follow the quantized blocks take them
  if (p.win_count > 0 && tile_idx * T < p.win_count) {
    uint16_t* win = kind ? pl.L.win_v : pl.L.win_k;
    const uint16_t* in = kind ? pl.V_in : pl.K_in;
    constexpr int VPR = D / 8;
    const int rows = min(T, p.win_count - tile_idx * T);
    for (int idx = tid; idx < rows * VPR; idx += PACK_THREADS) {
      const int r = tile_idx * T + idx / VPR, c8 = idx % VPR;
      const uint4* src = reinterpret_cast<const uint4*>(in + ((size_t)bh * p.n_in + (p.nq_new + r - p.s_old)) * D) + c8;
      reinterpret_cast<uint4*>(win + ((size_t)bh * R + r) * D)[c8] = *src;
    }
  }

  const int bits = kind ? pl.L.bv : pl.L.bk;
  const float eta = kind ? pl.eta_v : pl.eta_k;
  const int own = kind ? pl.own_v : pl.own_k;

  if (kind == 0) {
    // keys: one group per (channel, run of G tokens).  First bf16x2 min / max of a channel pair over a part of the
    // group's tokens (consecutive threads take consecutive pairs), then one thread per (group, channel).
    {
      const int dp = tid % (D / 2), rest = tid / (D / 2);
      const int gl = rest / KP, part = rest % KP;
      const uint8_t* col = tile + (gl * G + part * (G / KP)) * ROWB + dp * 4;
      V2 mn2 = *reinterpret_cast<const V2*>(col), mx2 = mn2;
#pragma unroll
      for (int j = 1; j < G / KP; ++j) {
        const V2 v = *reinterpret_cast<const V2*>(col + j * ROWB);
        mn2 = __hmin2(mn2, v);
        mx2 = __hmax2(mx2, v);
      }
      wbuf[(rest * (D / 2) + dp) * 2] = *reinterpret_cast<uint32_t*>(&mn2);
      wbuf[(rest * (D / 2) + dp) * 2 + 1] = *reinterpret_cast<uint32_t*>(&mx2);
    }
    __syncthreads();
    __half* meta = reinterpret_cast<__half*>(pl.L.k_meta);
    const size_t cap_g = (size_t)(dm.nq_cap / G);
#pragma unroll
    for (int k = 0; k < ((T / G) * D + PACK_THREADS - 1) / PACK_THREADS; ++k) {
      const int item = tid + k * PACK_THREADS;
      if (item < (T / G) * D) {
        const int gl = item / D, d = item % D;
        float mn = 0.f, mx = 0.f;
#pragma unroll
        for (int part = 0; part < KP; ++part) {
          const uint32_t a2 = wbuf[((gl * KP + part) * (D / 2) + d / 2) * 2], b2 = wbuf[((gl * KP + part) * (D / 2) + d / 2) * 2 + 1];
          const float lo = (d & 1) ? I16::hi(a2) : I16::lo(a2);
          const float hi = (d & 1) ? I16::hi(b2) : I16::lo(b2);
          mn = part == 0 ? lo : fminf(mn, lo);
          mx = part == 0 ? hi : fmaxf(mx, hi);
        }
        float z, sc;
        __half zh, sh;
        group_params(mn, mx, bits, eta, z, sc, zh, sh);
        if (own) group_thresholds<F16>(mn, mx, z, sc, bits, thr + item, NPAR);
        const size_t grp = (size_t)bh * cap_g + (tq0 / G + gl);  // per group: D scales, then D zero-points
        const int pos = k_meta_position(d, D);
        meta[grp * 2 * D + pos] = sh;
        meta[grp * 2 * D + D + pos] = zh;
      }
    }
  } else {
    // values: one group per (token, run of G channels); consecutive threads take consecutive tokens
    __half* meta = reinterpret_cast<__half*>(pl.L.v_meta);
#pragma unroll
    for (int k = 0; k < (T * NG + PACK_THREADS - 1) / PACK_THREADS; ++k) {
      const int item = tid + k * PACK_THREADS;
      if (item < T * NG) {
        const int tl = item % T, gi = item / T;
        const uint4* row = reinterpret_cast<const uint4*>(tile + tl * ROWB + gi * G * 2);
        V2 mn2, mx2;
        {
          uint4 v = row[0];
          const V2* e = reinterpret_cast<const V2*>(&v);
          mn2 = __hmin2(__hmin2(e[0], e[1]), __hmin2(e[2], e[3]));
          mx2 = __hmax2(__hmax2(e[0], e[1]), __hmax2(e[2], e[3]));
        }
#pragma unroll
        for (int j = 1; j < G / 8; ++j) {
          uint4 v = row[j];
          const V2* e = reinterpret_cast<const V2*>(&v);
          mn2 = __hmin2(mn2, __hmin2(__hmin2(e[0], e[1]), __hmin2(e[2], e[3])));
          mx2 = __hmax2(mx2, __hmax2(__hmax2(e[0], e[1]), __hmax2(e[2], e[3])));
        }
        const uint32_t mnw = *reinterpret_cast<const uint32_t*>(&mn2), mxw = *reinterpret_cast<const uint32_t*>(&mx2);
        const float mn = fminf(I16::lo(mnw), I16::hi(mnw));
        const float mx = fmaxf(I16::lo(mxw), I16::hi(mxw));
        float z, sc;
        __half zh, sh;
        group_params(mn, mx, bits, eta, z, sc, zh, sh);
        if (own) group_thresholds<F16>(mn, mx, z, sc, bits, thr + gi * T + tl, NPAR);
        const int tabs = tq0 + tl;
        __half* mine = meta + (size_t)bh * dm.nq_cap * 2 * NG;
        mine[v_scale_index(tabs, gi, NG)] = sh;
        mine[v_zero_index(tabs, gi, NG)] = zh;
      }
    }
  }
  if (!own) return;  // PseudoQuantize: parameters only
  __syncthreads();

  // codes
  uint32_t* codes = kind ? pl.L.v_codes : pl.L.k_codes;
  const bool merge = (own & 2) != 0, stats = (own & 4) != 0, store = (own & 3) != 0;
  uint32_t hist[4] = {0u, 0u, 0u, 0u};
  const size_t stream_words = (size_t)dm.nq_cap * D * bits / 32;
  auto build = [&](auto bits_c) {
    constexpr int BITS = decltype(bits_c)::value;
    constexpr int N = 32 / BITS;        // codes per word
    if (kind == 0) {
      constexpr int NW = D * BITS / 32;  // words per token row
      const size_t w0 = k_code_position(tq0, 0, BITS, D).word;  // the tile's words are one contiguous run
#pragma unroll
      for (int k = 0; k < (T * NW + PACK_THREADS - 1) / PACK_THREADS; ++k) {
        const int item = tid + k * PACK_THREADS;
        if (item < T * NW) {
          const int tl = item % T, i = item / T, gl = tl / G;
          const uint8_t* row = tile + tl * ROWB;
          uint32_t word = 0u;
#pragma unroll
          for (int s4 = 0; s4 < N / 4; ++s4) {
            const int d = i * N + 4 * s4;  // four consecutive channels: four groups
            const uint2 xx = *reinterpret_cast<const uint2*>(row + d * 2);
            const uint2 t1 = *reinterpret_cast<const uint2*>(thr + gl * D + d);
            uint2 t2 = t1, t3 = t1;
            if constexpr (BITS == 2) {
              t2 = *reinterpret_cast<const uint2*>(thr + NPAR + gl * D + d);
              t3 = *reinterpret_cast<const uint2*>(thr + 2 * NPAR + gl * D + d);
            }
            const uint32_t lo = code_pair<BITS, V2>(xx.x, t1.x, t2.x, t3.x), hi = code_pair<BITS, V2>(xx.y, t1.y, t2.y, t3.y);
            word |= __byte_perm(lo, hi, 0x6420) << (BITS * s4);
          }
          wbuf[k_code_position(tq0 + tl, i * N, BITS, D).word - w0] = word;
        }
      }
      __syncthreads();
      uint4* dst = reinterpret_cast<uint4*>(codes + (size_t)bh * stream_words + w0);
      for (int v = tid; v < T * NW / 4; v += PACK_THREADS) {
        uint4 w = reinterpret_cast<const uint4*>(wbuf)[v];
        if (merge || stats) {  // the dominant layer's codes of these positions are in place
          const uint4 o = dst[v];
          if (stats) {
            delta_count<BITS>(o.x, w.x, hist); delta_count<BITS>(o.y, w.y, hist);
            delta_count<BITS>(o.z, w.z, hist); delta_count<BITS>(o.w, w.w, hist);
          }
          const uint32_t lut = p.merge_lut[BITS - 1];
          w = make_uint4(merge_words<BITS>(o.x, w.x, lut), merge_words<BITS>(o.y, w.y, lut),
                         merge_words<BITS>(o.z, w.z, lut), merge_words<BITS>(o.w, w.w, lut));
        }
        if (store) dst[v] = w;
      }
    } else {
      constexpr int WPC = T / N;  // words per channel over the tile's tokens
#pragma unroll
      for (int k = 0; k < (D * WPC + PACK_THREADS - 1) / PACK_THREADS; ++k) {
        const int item = tid + k * PACK_THREADS;
        if (item < D * WPC) {
          const int d = item % D, wi = item / D, gi = d / G;
          uint32_t word = 0u;
#pragma unroll
          for (int s4 = 0; s4 < N / 4; ++s4) {
            const int tl = wi * N + 4 * s4;  // four consecutive tokens: four groups
            const uint8_t* src = tile + tl * ROWB + d * 2;
            const uint32_t x0 = *reinterpret_cast<const uint16_t*>(src), x1 = *reinterpret_cast<const uint16_t*>(src + ROWB);
            const uint32_t x2 = *reinterpret_cast<const uint16_t*>(src + 2 * ROWB), x3 = *reinterpret_cast<const uint16_t*>(src + 3 * ROWB);
            const uint2 t1 = *reinterpret_cast<const uint2*>(thr + gi * T + tl);
            uint2 t2 = t1, t3 = t1;
            if constexpr (BITS == 2) {
              t2 = *reinterpret_cast<const uint2*>(thr + NPAR + gi * T + tl);
              t3 = *reinterpret_cast<const uint2*>(thr + 2 * NPAR + gi * T + tl);
            }
            const uint32_t lo = code_pair<BITS, V2>(x0 | (x1 << 16), t1.x, t2.x, t3.x);
            const uint32_t hi = code_pair<BITS, V2>(x2 | (x3 << 16), t1.y, t2.y, t3.y);
            word |= __byte_perm(lo, hi, 0x6420) << (BITS * s4);
          }
          uint32_t* dst = codes + (size_t)bh * stream_words + v_code_position(tq0 + wi * N, d, BITS, D).word;
          if (merge || stats) {
            const uint32_t o = *dst;
            if (stats) delta_count<BITS>(o, word, hist);
            word = merge_words<BITS>(o, word, p.merge_lut[BITS - 1]);
          }
          if (store) *dst = word;
        }
      }
    }
  };
  if (bits == 2) build(std::integral_constant<int, 2>{}); else build(std::integral_constant<int, 1>{});
  if (stats) {
    unsigned long long* out = kind ? pl.delta_v : pl.delta_k;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t tot = __reduce_add_sync(0xffffffffu, hist[k]);
      if ((tid & 31) == 0 && tot) atomicAdd(out + k, (unsigned long long)tot);
    }
  }
}

template <bool F16>
cudaError_t launch_pack_t(const PackParams& p, cudaStream_t st) {
  int tiles = p.n_blocks * (p.dm.R / p.tb);
  dim3 grid(2 * tiles, p.dm.B * p.dm.Hkv, p.n_layers);
  const int key = p.dm.D * 10000 + p.dm.g * 100 + p.tb;
  switch (key) {
    case 1283232: pack_kernel<128, 32, 32, F16><<<grid, PACK_THREADS, 0, st>>>(p); break;
    case 1286464: pack_kernel<128, 64, 64, F16><<<grid, PACK_THREADS, 0, st>>>(p); break;
    case 643232: pack_kernel<64, 32, 32, F16><<<grid, PACK_THREADS, 0, st>>>(p); break;
    case 646464: pack_kernel<64, 64, 64, F16><<<grid, PACK_THREADS, 0, st>>>(p); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_pack(const PackParams& p, cudaStream_t st) {
  if (p.n_layers < 1 || p.n_layers > PACK_MAX_LAYERS) return cudaErrorInvalidValue;
  return p.f16 ? launch_pack_t<true>(p, st) : launch_pack_t<false>(p, st);
}

// Copies new tokens into the 16-bit window, keys and values in one launch.
__global__ void __launch_bounds__(256) window_append_kernel(WindowParams p) {
  const Dims& dm = p.dm;
  const int vec_per_row = dm.D / 8;
  const size_t per_kind = (size_t)dm.B * dm.Hkv * p.count * vec_per_row;
  size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  grid_dependents_go();    // the next kernel may get its CTAs placed; it waits for this one before it reads the window
  grid_dependency_wait();  // the inputs come from the preceding kernel, and earlier kernels may still read the window
  if (idx >= 2 * per_kind) return;
  int kind = idx >= per_kind;
  size_t r = idx - (kind ? per_kind : 0);
  int c8 = r % vec_per_row;
  r /= vec_per_row;
  int tok = r % p.count;
  int bh = r / p.count;
  int pabs = p.first + tok;
  const uint16_t* in = kind ? p.V_in : p.K_in;
  uint16_t* win = kind ? p.L.win_v : p.L.win_k;
  const uint4* src = reinterpret_cast<const uint4*>(in + ((size_t)bh * p.n_in + (pabs - p.s_old)) * dm.D) + c8;
  uint4* dst = reinterpret_cast<uint4*>(win + ((size_t)bh * dm.R + (pabs - p.nq_new)) * dm.D) + c8;
  *dst = *src;
}

cudaError_t launch_window_append(const WindowParams& p, cudaStream_t st) {
  size_t total = 2 * (size_t)p.dm.B * p.dm.Hkv * p.count * (p.dm.D / 8);
  unsigned blocks = (unsigned)((total + 255) / 256);
  return launch_dependent(window_append_kernel, dim3(blocks), dim3(256), 0, st, p);
}

}  // namespace xq
