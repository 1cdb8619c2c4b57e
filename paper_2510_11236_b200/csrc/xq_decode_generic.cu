// Scalar decode-attention kernel over the packed cache plus the 16-bit window,
// and the split-K merge kernel.  This kernel handles every supported shape by
// walking the layout index functions element by element; it is the slow path
// and the on-device cross-check of the tensor-core kernel.
//
// Grid (split, kv head, sequence); 4 warps per CTA; each warp takes every 4th
// token of the split's range, lanes cover channels (d = lane + 32 j), and keeps
// an online softmax (running max m in log2 units, sum l, accumulator) per query
// head of the group.  The warps' states are combined in shared memory and the
// CTA writes one partial (m, l, acc[D]) per query head.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <math_constants.h>

#include "xq_internal.h"
#include "xq_layout.cuh"

namespace xq {

__device__ __forceinline__ float bf16_bits_f(uint16_t u) { return __uint_as_float(((uint32_t)u) << 16); }
__device__ __forceinline__ float f16_bits_f(uint16_t u) { return __half2float(__ushort_as_half(u)); }
// an element of q, K, V or the window: IEEE half precision or bfloat16
__device__ __forceinline__ float io_bits_f(uint16_t u, int f16) { return f16 ? f16_bits_f(u) : bf16_bits_f(u); }

constexpr int GEN_WARPS = 4;
constexpr int GEN_HEADS = 8;  // query heads processed per pass

template <int DPL>
__global__ void __launch_bounds__(GEN_WARPS * 32) decode_generic_kernel(DecodeParams p) {
  constexpr int D = DPL * 32;
  __shared__ float sm_acc[GEN_WARPS][GEN_HEADS][D];
  __shared__ float sm_ml[GEN_WARPS][GEN_HEADS][2];

  const Dims& dm = p.dm;
  const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int bh = b * dm.Hkv + hk;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ns = p.ns_q + p.ns_w;
  const int g = dm.g, NG = dm.NG;

  bool quant = split < p.ns_q;
  int t0, t1;
  if (quant) {
    int units = (p.n_q + 31) / 32;  // the last unit is ragged when a visibility limit cuts the packed region
    share_of(units, p.ns_q, split, t0, t1);
    t0 *= 32;
    t1 = min(t1 * 32, p.n_q);
  } else {
    int sw = split - p.ns_q;
    int tiles = (p.r + 15) / 16;
    share_of(tiles, p.ns_w, sw, t0, t1);
    t0 *= 16;
    t1 = min(t1 * 16, p.r);
  }

  const int bk = p.L.bk, bv = p.L.bv;
  const uint32_t* kc = p.L.k_codes + (size_t)bh * ((size_t)dm.nq_cap * D * bk / 32);
  const uint32_t* vc = p.L.v_codes + (size_t)bh * ((size_t)dm.nq_cap * D * bv / 32);
  const uint16_t* km = p.L.k_meta + (size_t)bh * (dm.nq_cap / g) * 2 * D;
  const uint16_t* vm = p.L.v_meta + (size_t)bh * dm.nq_cap * 2 * NG;
  const uint16_t* wk = p.L.win_k + (size_t)bh * dm.R * D;
  const uint16_t* wv = p.L.win_v + (size_t)bh * dm.R * D;
  const float scale2 = p.scale * 1.4426950408889634f;

  for (int g0 = 0; g0 < dm.G; g0 += GEN_HEADS) {
    const int nh = min(GEN_HEADS, dm.G - g0);
    float q[GEN_HEADS][DPL], acc[GEN_HEADS][DPL], m[GEN_HEADS], l[GEN_HEADS];
#pragma unroll
    for (int a = 0; a < GEN_HEADS; ++a) {
      m[a] = -CUDART_INF_F;
      l[a] = 0.f;
#pragma unroll
      for (int j = 0; j < DPL; ++j) {
        acc[a][j] = 0.f;
        q[a][j] = (a < nh) ? io_bits_f(p.q[((size_t)b * dm.Hq + hk * dm.G + g0 + a) * D + lane + 32 * j], p.f16) : 0.f;
      }
    }
    for (int t = t0 + warp; t < t1; t += GEN_WARPS) {
      float kx[DPL], vx[DPL];
#pragma unroll
      for (int j = 0; j < DPL; ++j) {
        int d = lane + 32 * j;
        if (quant) {
          CodePos pk = k_code_position(t, d, bk, D);
          float c = (float)((kc[pk.word] >> pk.bit) & ((1u << bk) - 1));
          const uint16_t* mk = km + (size_t)(t / g) * 2 * D;  // the group's D scales, then its D zero-points
          int pos = k_meta_position(d, D);
          kx[j] = fmaf(c, f16_bits_f(mk[pos]), f16_bits_f(mk[D + pos]));
          CodePos pv = v_code_position(t, d, bv, D);
          float cv = (float)((vc[pv.word] >> pv.bit) & ((1u << bv) - 1));
          vx[j] = fmaf(cv, f16_bits_f(vm[v_scale_index(t, d / g, NG)]), f16_bits_f(vm[v_zero_index(t, d / g, NG)]));
        } else {
          kx[j] = io_bits_f(wk[(size_t)t * D + d], p.f16);
          vx[j] = io_bits_f(wv[(size_t)t * D + d], p.f16);
        }
      }
#pragma unroll
      for (int a = 0; a < GEN_HEADS; ++a) {
        if (a < nh) {
          float dot = 0.f;
#pragma unroll
          for (int j = 0; j < DPL; ++j) dot = fmaf(q[a][j], kx[j], dot);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
          float x = dot * scale2;
          float mn = fmaxf(m[a], x);
          float corr = exp2f(m[a] - mn);
          float pe = exp2f(x - mn);
          l[a] = l[a] * corr + pe;
#pragma unroll
          for (int j = 0; j < DPL; ++j) acc[a][j] = acc[a][j] * corr + pe * vx[j];
          m[a] = mn;
        }
      }
    }
    // combine the warps
#pragma unroll
    for (int a = 0; a < GEN_HEADS; ++a) {
#pragma unroll
      for (int j = 0; j < DPL; ++j) sm_acc[warp][a][lane + 32 * j] = acc[a][j];
      if (lane == 0) {
        sm_ml[warp][a][0] = m[a];
        sm_ml[warp][a][1] = l[a];
      }
    }
    __syncthreads();
    for (int item = threadIdx.x; item < nh * D; item += GEN_WARPS * 32) {
      int a = item / D, d = item % D;
      float M = -CUDART_INF_F;
      for (int w = 0; w < GEN_WARPS; ++w) M = fmaxf(M, sm_ml[w][a][0]);
      float Lsum = 0.f, A = 0.f;
      for (int w = 0; w < GEN_WARPS; ++w) {
        float mw = sm_ml[w][a][0];
        float f = (mw == -CUDART_INF_F) ? 0.f : exp2f(mw - M);
        Lsum += sm_ml[w][a][1] * f;
        A += sm_acc[w][a][d] * f;
      }
      size_t hq = (size_t)b * dm.Hq + hk * dm.G + g0 + a;
      p.part_acc[(hq * ns + split) * D + d] = A;
      if (d == 0) {
        p.part_ml[(hq * ns + split) * 2 + 0] = M;
        p.part_ml[(hq * ns + split) * 2 + 1] = Lsum;
      }
    }
    __syncthreads();
  }
}

cudaError_t launch_decode_generic(const DecodeParams& p, cudaStream_t st) {
  dim3 grid(p.ns_q + p.ns_w, p.dm.Hkv, p.dm.B);
  if (p.dm.D == 128)
    decode_generic_kernel<4><<<grid, GEN_WARPS * 32, 0, st>>>(p);
  else
    decode_generic_kernel<2><<<grid, GEN_WARPS * 32, 0, st>>>(p);
  return cudaGetLastError();
}

// Split-K merge: out[d] = sum_s acc_s[d] 2^(m_s - M) / sum_s l_s 2^(m_s - M).
// Grid (query head, sequence), D threads.
__global__ void merge_kernel(MergeParams p) {
  const Dims& dm = p.dm;
  const int hq = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
  const int D = dm.D, ns = p.ns;
  const size_t base = ((size_t)b * dm.Hq + hq) * ns;
  float M = -CUDART_INF_F;
  for (int s = 0; s < ns; ++s) M = fmaxf(M, p.part_ml[(base + s) * 2]);
  float Lsum = 0.f, A = 0.f;
  for (int s = 0; s < ns; ++s) {
    float ms = p.part_ml[(base + s) * 2];
    float f = (ms == -CUDART_INF_F) ? 0.f : exp2f(ms - M);
    Lsum += p.part_ml[(base + s) * 2 + 1] * f;
    A += p.part_acc[(base + s) * D + d] * f;
  }
  float o = A / Lsum;
  size_t oi = ((size_t)b * dm.Hq + hq) * D + d;
  if (p.out_f32)
    reinterpret_cast<float*>(p.out)[oi] = o;
  else if (p.f16)
    reinterpret_cast<__half*>(p.out)[oi] = __float2half_rn(o);
  else
    reinterpret_cast<__nv_bfloat16*>(p.out)[oi] = __float2bfloat16_rn(o);
}

cudaError_t launch_merge(const MergeParams& p, cudaStream_t st) {
  dim3 grid(p.dm.Hq, p.dm.B);
  merge_kernel<<<grid, p.dm.D, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace xq
