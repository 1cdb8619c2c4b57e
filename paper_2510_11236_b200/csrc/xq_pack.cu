// Quantize-and-pack of residual-window blocks (Eq. 1, 2, 12; Algorithm 2) and
// the window append.  One CTA quantizes a tile of `tb` tokens x D channels of
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

// Eq. 2 with the uncalibrated z, s; ties to even; clamped; constant group -> 0.
__device__ __forceinline__ uint32_t code_of(float x, float z, float s, float qmax) {
  if (s == 0.0f) return 0u;
  float c = rintf(__fdiv_rn(__fsub_rn(x, z), s));
  c = fminf(fmaxf(c, 0.0f), qmax);
  return (uint32_t)c;
}

constexpr int PACK_THREADS = 128;
constexpr int PACK_MAX_TB = 64;
constexpr int PACK_ROW_PAD = 16;  // bytes added to each staged row: 8 consecutive rows then fall in 8 different bank groups

// The quantizer's parameters of one group as the code loop wants them.
struct GroupPar {
  float z, s, inv, unused;  // inv = 1/s rounded to nearest (0 for a constant group)
};

__device__ __forceinline__ GroupPar make_par(float z, float s) {
  GroupPar r;
  r.z = z;
  r.s = s;
  r.inv = (s == 0.0f) ? 0.0f : __frcp_rn(s);
  r.unused = 0.0f;
  return r;
}

// Eq. 2 through the reciprocal.  (x - z) * inv differs from the correctly
// rounded quotient (x - z) / s by at most three roundings of a value below
// 2^B, i.e. by less than 6e-7, so both round to the same integer unless the
// product lies within 1e-5 of a tie; `doubt` collects that case (and any
// non-finite product of a subnormal scale), and the caller then recomputes the
// word with the division.  0 <= (x - z) / s < 2^B - 1/2 holds for every member
// of the group, so the fast path needs no clamp.
__device__ __forceinline__ uint32_t code_fast(float x, const GroupPar& g, bool& doubt) {
  float t = __fmul_rn(__fsub_rn(x, g.z), g.inv);
  float c = rintf(t);
  doubt |= !(fabsf(__fsub_rn(t, c)) <= 0.49999f);
  return (uint32_t)(int)c;
}

// One CTA: T = p.tb tokens x D channels of one (sequence, kv head), keys
// (blockIdx.x even) or values (odd).  Staged rows are padded; the statistics
// and the codes read them without bank conflicts; the packed words are
// collected in shared memory and leave in 16-byte vectors.
template <int D, int G>
__global__ void __launch_bounds__(PACK_THREADS) pack_kernel(PackParams p) {
  constexpr int ROWB = D * 2 + PACK_ROW_PAD;
  constexpr int NG = D / G;
  constexpr int CB = D / 16;
  __shared__ __align__(16) uint8_t tile[PACK_MAX_TB * ROWB];
  __shared__ __align__(16) GroupPar par[PACK_MAX_TB * NG > (PACK_MAX_TB / G) * D ? PACK_MAX_TB * NG : (PACK_MAX_TB / G) * D];
  __shared__ __align__(16) uint32_t wbuf[PACK_MAX_TB * D * 2 / 32];

  const Dims& dm = p.dm;
  const int R = dm.R, T = p.tb;
  const int kind = blockIdx.x & 1;  // 0 keys, 1 values
  const int tile_idx = blockIdx.x >> 1;
  const int h = blockIdx.y, b = blockIdx.z;
  const int bh = b * dm.Hkv + h;
  const int tid = threadIdx.x;
  const int tq0 = p.nq_old + tile_idx * T;  // absolute index of the tile's first token

  {
    const uint16_t* win = kind ? p.L.win_v : p.L.win_k;
    const uint16_t* in = kind ? p.V_in : p.K_in;
    constexpr int VPR = D / 8;
    for (int idx = tid; idx < T * VPR; idx += PACK_THREADS) {
      int tl = idx / VPR, c8 = idx % VPR;
      int pabs = tq0 + tl;
      const uint16_t* src = (pabs < p.s_old) ? win + ((size_t)bh * R + (pabs - p.nq_old)) * D
                                             : in + ((size_t)bh * p.n_in + (pabs - p.s_old)) * D;
      *reinterpret_cast<uint4*>(tile + tl * ROWB + c8 * 16) = reinterpret_cast<const uint4*>(src)[c8];
    }
  }
  __syncthreads();

  const int bits = kind ? p.L.bv : p.L.bk;
  const float eta = kind ? p.eta_v : p.eta_k;
  const int own = kind ? p.own_v : p.own_k;

  if (kind == 0) {
    // keys: one group per (channel, run of G tokens); consecutive threads take consecutive channels
    __half* meta = reinterpret_cast<__half*>(p.L.k_meta);
    const size_t cap_g = (size_t)(dm.nq_cap / G);
    for (int item = tid; item < (T / G) * D; item += PACK_THREADS) {
      int gl = item / D, d = item % D;
      const uint8_t* col = tile + (gl * G) * ROWB + d * 2;
      float mn = bf16_bits(*reinterpret_cast<const uint16_t*>(col)), mx = mn;
#pragma unroll 8
      for (int j = 1; j < G; ++j) {
        float x = bf16_bits(*reinterpret_cast<const uint16_t*>(col + j * ROWB));
        mn = fminf(mn, x);
        mx = fmaxf(mx, x);
      }
      float z, s;
      __half zh, sh;
      group_params(mn, mx, bits, eta, z, s, zh, sh);
      par[item] = make_par(z, s);
      size_t grp = (size_t)bh * 2 * cap_g + (tq0 / G + gl);  // scale plane, then zero-point plane
      int pos = k_meta_position(d, D);
      meta[grp * D + pos] = sh;
      meta[(grp + cap_g) * D + pos] = zh;
    }
  } else {
    // values: one group per (token, run of G channels); consecutive threads take consecutive tokens
    __half* meta = reinterpret_cast<__half*>(p.L.v_meta);
    for (int item = tid; item < T * NG; item += PACK_THREADS) {
      int tl = item % T, gi = item / T;
      const uint4* row = reinterpret_cast<const uint4*>(tile + tl * ROWB + gi * G * 2);
      __nv_bfloat162 mn2, mx2;
      {
        uint4 v = row[0];
        const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&v);
        mn2 = __hmin2(__hmin2(e[0], e[1]), __hmin2(e[2], e[3]));
        mx2 = __hmax2(__hmax2(e[0], e[1]), __hmax2(e[2], e[3]));
      }
#pragma unroll
      for (int j = 1; j < G / 8; ++j) {
        uint4 v = row[j];
        const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&v);
        mn2 = __hmin2(mn2, __hmin2(__hmin2(e[0], e[1]), __hmin2(e[2], e[3])));
        mx2 = __hmax2(mx2, __hmax2(__hmax2(e[0], e[1]), __hmax2(e[2], e[3])));
      }
      float mn = fminf(__low2float(mn2), __high2float(mn2));
      float mx = fmaxf(__low2float(mx2), __high2float(mx2));
      float z, s;
      __half zh, sh;
      group_params(mn, mx, bits, eta, z, s, zh, sh);
      par[tl * NG + gi] = make_par(z, s);
      int tabs = tq0 + tl;
      size_t t16 = (size_t)bh * (dm.nq_cap / 16) + tabs / 16;
      int pos = v_meta_position(tabs % 16, gi, NG);
      meta[(t16 * 2 + 0) * (16 * NG) + pos] = sh;
      meta[(t16 * 2 + 1) * (16 * NG) + pos] = zh;
    }
  }
  if (!own) return;  // PseudoQuantize: parameters only
  __syncthreads();

  // codes: thread -> (tile, fragment lane, word of the lane); lanes of a warp
  // differ in the fragment lane, so they read 8 rows x 4 column pairs (keys)
  // or 4 token pairs x 8 channels (values) of the padded tile
  const int n_words = T * D * bits / 32;
  auto build = [&](auto bits_c) {
    constexpr int BITS = decltype(bits_c)::value;
    constexpr int NSLOT = 16 / BITS;
    constexpr int TPT = 16 * (NSLOT / CB);
    constexpr float QMAX = (float)((1 << BITS) - 1);
    for (int it = tid; it < n_words; it += PACK_THREADS) {
      const int lane = it & 31, i = (it >> 5) & 3, tile_l = it >> 7;
      const int row = (lane >> 2) + 8 * (i & 1);
      const int col = 2 * (lane & 3) + 8 * (i >> 1);
      uint32_t word = 0;
      bool doubt = false;
      if (kind == 0) {
#pragma unroll
        for (int slot = 0; slot < NSLOT; ++slot) {
          const int tt = slot / CB, cb = slot % CB;
          const int tl = tile_l * TPT + tt * 16 + row, d = cb * 16 + col;
          uint32_t xx = *reinterpret_cast<const uint32_t*>(tile + tl * ROWB + d * 2);
          const GroupPar* gp = par + ((tile_l * TPT + tt * 16) / G) * D + d;
          GroupPar g0 = gp[0], g1 = gp[1];
          uint32_t c0 = code_fast(__uint_as_float(xx << 16), g0, doubt);
          uint32_t c1 = code_fast(__uint_as_float(xx & 0xffff0000u), g1, doubt);
          word |= (c0 | (c1 << 16)) << (BITS * slot);
        }
        if (doubt) {
          word = 0;
#pragma unroll 1
          for (int slot = 0; slot < NSLOT; ++slot) {
            const int tt = slot / CB, cb = slot % CB;
            const int tl = tile_l * TPT + tt * 16 + row, d = cb * 16 + col;
            uint32_t xx = *reinterpret_cast<const uint32_t*>(tile + tl * ROWB + d * 2);
            const GroupPar* gp = par + ((tile_l * TPT + tt * 16) / G) * D + d;
            uint32_t c0 = code_of(__uint_as_float(xx << 16), gp[0].z, gp[0].s, QMAX);
            uint32_t c1 = code_of(__uint_as_float(xx & 0xffff0000u), gp[1].z, gp[1].s, QMAX);
            word |= (c0 | (c1 << 16)) << (BITS * slot);
          }
        }
      } else {
#pragma unroll
        for (int slot = 0; slot < NSLOT; ++slot) {
          const int tt = slot / CB, cb = slot % CB;
          const int tl = tile_l * TPT + tt * 16 + col, d = cb * 16 + row;
          const uint8_t* src = tile + tl * ROWB + d * 2;
          float x0 = bf16_bits(*reinterpret_cast<const uint16_t*>(src));
          float x1 = bf16_bits(*reinterpret_cast<const uint16_t*>(src + ROWB));
          const GroupPar* gp = par + tl * NG + (cb * 16) / G;
          GroupPar g0 = gp[0], g1 = gp[NG];
          uint32_t c0 = code_fast(x0, g0, doubt);
          uint32_t c1 = code_fast(x1, g1, doubt);
          word |= (c0 | (c1 << 16)) << (BITS * slot);
        }
        if (doubt) {
          word = 0;
#pragma unroll 1
          for (int slot = 0; slot < NSLOT; ++slot) {
            const int tt = slot / CB, cb = slot % CB;
            const int tl = tile_l * TPT + tt * 16 + col, d = cb * 16 + row;
            const uint8_t* src = tile + tl * ROWB + d * 2;
            float x0 = bf16_bits(*reinterpret_cast<const uint16_t*>(src));
            float x1 = bf16_bits(*reinterpret_cast<const uint16_t*>(src + ROWB));
            const GroupPar* gp = par + tl * NG + (cb * 16) / G;
            uint32_t c0 = code_of(x0, gp[0].z, gp[0].s, QMAX);
            uint32_t c1 = code_of(x1, gp[NG].z, gp[NG].s, QMAX);
            word |= (c0 | (c1 << 16)) << (BITS * slot);
          }
        }
      }
      wbuf[tile_l * 128 + lane * 4 + i] = word;
    }
  };
  if (bits == 2)
    build(std::integral_constant<int, 2>{});
  else
    build(std::integral_constant<int, 1>{});
  __syncthreads();

  uint32_t* codes = kind ? p.L.v_codes : p.L.k_codes;
  const size_t stream_words = (size_t)dm.nq_cap * D * bits / 32;
  uint4* dst = reinterpret_cast<uint4*>(codes + (size_t)bh * stream_words + (size_t)(tq0 / 32) * (D * bits));
  for (int v = tid; v < n_words / 4; v += PACK_THREADS) dst[v] = reinterpret_cast<const uint4*>(wbuf)[v];
}

cudaError_t launch_pack(const PackParams& p, cudaStream_t st) {
  int tiles = p.n_blocks * (p.dm.R / p.tb);
  dim3 grid(2 * tiles, p.dm.Hkv, p.dm.B);
  if (p.dm.D == 128 && p.dm.g == 32)
    pack_kernel<128, 32><<<grid, PACK_THREADS, 0, st>>>(p);
  else if (p.dm.D == 128)
    pack_kernel<128, 64><<<grid, PACK_THREADS, 0, st>>>(p);
  else if (p.dm.g == 32)
    pack_kernel<64, 32><<<grid, PACK_THREADS, 0, st>>>(p);
  else
    pack_kernel<64, 64><<<grid, PACK_THREADS, 0, st>>>(p);
  return cudaGetLastError();
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
