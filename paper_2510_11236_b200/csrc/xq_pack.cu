// Quantize-and-pack of residual-window blocks (Eq. 1, 2, 12; Algorithm 2) and
// the window append.  One CTA quantizes a tile of `tb` tokens x D channels of
// one (sequence, kv head) for keys or for values.
//
// The fp32 arithmetic uses the *_rn intrinsics so that no multiply-add is ever
// contracted: codes, scales and zero-points are compared bit for bit with a CPU
// evaluation of the same formulas.
#include <cuda_fp16.h>

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

constexpr int PACK_THREADS = 256;
constexpr int PACK_MAX_TB = 64;
constexpr int PACK_MAX_D = 128;

__global__ void __launch_bounds__(PACK_THREADS) pack_kernel(PackParams p) {
  __shared__ __align__(16) uint16_t tile[PACK_MAX_TB * PACK_MAX_D];
  __shared__ float z_arr[256];
  __shared__ float s_arr[256];

  const Dims& dm = p.dm;
  const int D = dm.D, g = dm.g, R = dm.R, NG = dm.NG, tb = p.tb;
  const int kind = blockIdx.x & 1;  // 0 keys, 1 values
  const int tile_idx = blockIdx.x >> 1;
  const int h = blockIdx.y, b = blockIdx.z;
  const int bh = b * dm.Hkv + h;
  const int tid = threadIdx.x;
  const int tq0 = p.nq_old + tile_idx * tb;  // absolute index of the tile's first token

  const uint16_t* win = kind ? p.L.win_v : p.L.win_k;
  const uint16_t* in = kind ? p.V_in : p.K_in;
  const int vec_per_row = D / 8;
  for (int idx = tid; idx < tb * vec_per_row; idx += PACK_THREADS) {
    int tl = idx / vec_per_row, c8 = idx % vec_per_row;
    int pabs = tq0 + tl;
    const uint16_t* src = (pabs < p.s_old) ? win + ((size_t)bh * R + (pabs - p.nq_old)) * D
                                           : in + ((size_t)bh * p.n_in + (pabs - p.s_old)) * D;
    reinterpret_cast<uint4*>(tile)[idx] = reinterpret_cast<const uint4*>(src)[c8];
  }
  __syncthreads();

  const int bits = kind ? p.L.bv : p.L.bk;
  const float eta = kind ? p.eta_v : p.eta_k;
  const float qmax = (float)((1 << bits) - 1);
  const int own = kind ? p.own_v : p.own_k;

  if (kind == 0) {
    // keys: one group per (channel, run of g tokens)
    const int n_gl = tb / g;
    __half* meta = reinterpret_cast<__half*>(p.L.k_meta);
    for (int item = tid; item < n_gl * D; item += PACK_THREADS) {
      int gl = item / D, d = item % D;
      float mn = bf16_bits(tile[(gl * g) * D + d]), mx = mn;
      for (int j = 1; j < g; ++j) {
        float x = bf16_bits(tile[(gl * g + j) * D + d]);
        mn = fminf(mn, x);
        mx = fmaxf(mx, x);
      }
      float z, s;
      __half zh, sh;
      group_params(mn, mx, bits, eta, z, s, zh, sh);
      z_arr[item] = z;
      s_arr[item] = s;
      const size_t cap_g = (size_t)(dm.nq_cap / g);
      size_t grp = (size_t)bh * 2 * cap_g + (tq0 / g + gl);  // scale plane, then zero-point plane
      int pos = k_meta_position(d, D);
      meta[grp * D + pos] = sh;
      meta[(grp + cap_g) * D + pos] = zh;
    }
  } else {
    // values: one group per (token, run of g channels)
    __half* meta = reinterpret_cast<__half*>(p.L.v_meta);
    for (int item = tid; item < tb * NG; item += PACK_THREADS) {
      int tl = item / NG, gi = item % NG;
      const uint16_t* row = tile + tl * D + gi * g;
      float mn = bf16_bits(row[0]), mx = mn;
      for (int j = 1; j < g; ++j) {
        float x = bf16_bits(row[j]);
        mn = fminf(mn, x);
        mx = fmaxf(mx, x);
      }
      float z, s;
      __half zh, sh;
      group_params(mn, mx, bits, eta, z, s, zh, sh);
      z_arr[item] = z;
      s_arr[item] = s;
      int tabs = tq0 + tl;
      size_t t16 = (size_t)bh * (dm.nq_cap / 16) + tabs / 16;
      int pos = v_meta_position(tabs % 16, gi, NG);
      meta[(t16 * 2 + 0) * (16 * NG) + pos] = sh;
      meta[(t16 * 2 + 1) * (16 * NG) + pos] = zh;
    }
  }
  if (!own) return;  // PseudoQuantize: parameters only
  __syncthreads();

  // codes: each thread assembles whole 32-bit words of the packed layout
  const int nslot = 16 / bits;
  const int CB = D / 16;
  const int tpt = tokens_per_code_tile(bits, D);
  const int words_per_token_x32 = D * bits;  // words per 32 tokens
  const int n_words = tb * D * bits / 32;
  uint32_t* codes = kind ? p.L.v_codes : p.L.k_codes;
  const size_t stream_words = (size_t)dm.nq_cap * D * bits / 32;
  uint32_t* dst = codes + (size_t)bh * stream_words + (size_t)(tq0 / 32) * words_per_token_x32;
  for (int wl = tid; wl < n_words; wl += PACK_THREADS) {
    int tile_l = wl >> 7, w = wl & 127;
    int lane = w >> 2, i = w & 3;
    uint32_t word = 0;
    for (int hf = 0; hf < 2; ++hf) {
      int row = (lane >> 2) + 8 * (i & 1);
      int col = 2 * (lane & 3) + hf + 8 * (i >> 1);
      for (int slot = 0; slot < nslot; ++slot) {
        int tt = slot / CB, cb = slot % CB;
        int tl, d;
        if (kind == 0) {
          tl = tile_l * tpt + tt * 16 + row;
          d = cb * 16 + col;
        } else {
          tl = tile_l * tpt + tt * 16 + col;
          d = cb * 16 + row;
        }
        float x = bf16_bits(tile[tl * D + d]);
        int gidx = (kind == 0) ? (tl / g) * D + d : tl * NG + d / g;
        uint32_t c = code_of(x, z_arr[gidx], s_arr[gidx], qmax);
        word |= c << (16 * hf + bits * slot);
      }
    }
    dst[wl] = word;
  }
}

cudaError_t launch_pack(const PackParams& p, cudaStream_t st) {
  int tiles = p.n_blocks * (p.dm.R / p.tb);
  dim3 grid(2 * tiles, p.dm.Hkv, p.dm.B);
  pack_kernel<<<grid, PACK_THREADS, 0, st>>>(p);
  return cudaGetLastError();
}

// Copies new tokens into the 16-bit window, keys and values in one launch.
__global__ void __launch_bounds__(256) window_append_kernel(WindowParams p) {
  const Dims& dm = p.dm;
  const int vec_per_row = dm.D / 8;
  const size_t per_kind = (size_t)dm.B * dm.Hkv * p.count * vec_per_row;
  size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
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
  window_append_kernel<<<blocks, 256, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace xq
