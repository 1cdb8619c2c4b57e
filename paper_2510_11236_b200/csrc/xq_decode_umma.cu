// Tensor-core decode attention over the packed cache (head_dim 128, up to 8
// query heads per kv head) on the 5th-generation tensor cores: tcgen05.mma with
// the code matrices in tensor memory.
//
// The packed cache delivers ~1.8e13 quantized elements/s at the HBM roofline, so
// a code may cost about one ALU instruction per two elements and nothing else.
// A code sitting in the low mantissa bits of an fp16 IS the subnormal
// c * 2^(pos-24), so `word & mask` is a ready fp16x2 operand; scale and
// zero-point are folded out of the inner products,
//
//   q . k_hat_t = sum_d (q_d s_d) c_td + sum_d q_d z_d        (keys, per channel)
//   sum_t p_t v_hat_td = sum_t (p_t s_tg) c_td + sum_t p_t z_tg  (values, per token)
//
// and the products over raw codes run on the tensor cores.  Registers cannot feed
// tcgen05.mma and shared memory is too slow for expanded codes (2 bytes per
// element each way), but tensor memory can: every thread owns one lane (matrix
// row), writes its row of masked words with tcgen05.st, and the MMA reads A from
// there.  The small B operands (q folded with the key scales; softmax numerators
// folded with the value scales) live in shared memory.
//
// One CTA (4 warps = 128 tensor-memory lanes) walks a range of 128-token batches
// of one (sequence, kv head):
//   keys:    A_K[128 tokens x 128 channels] (thread = token),   B_K[(group, head) x channel]
//            S[token][(group, head)]; a token reads the columns of its own group.
//   values:  A_V[128 channels x 128 tokens] (thread = channel), B_P[token x (channel group, head)]
//            O[channel][(channel group, head)] accumulates over all batches in tensor memory.
// The q . z bias of every token group of the range comes from one more set of
// MMAs in the prologue (A = zero-point rows, B = q).  Softmax uses one reference
// per head for the whole CTA, raised only when a logit exceeds it by more than
// TAU; raising it rescales O in tensor memory (rare).  Batches are staged with
// cp.async through a ring.  MMAs are issued by one thread and tracked with
// mbarriers; the key MMAs of batch i+1 run while batch i's softmax and value
// expansion execute.  Split-K partials are merged by the last CTA of a stream
// (atomic ticket; nobody waits for another CTA).
//
// Every wait on an mbarrier is bounded: a CTA that gives up sets the status word,
// frees its tensor memory and leaves.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <math_constants.h>

#include "xq_internal.h"

namespace xq {

namespace {

constexpr int UT = 128;  // threads = tensor-memory lanes = tokens per batch = channels
constexpr int UW = 4;
constexpr int HD = 128;
constexpr int BT = 128;    // tokens per batch
constexpr int NSTB = 6;    // staged batches
constexpr float TAU = 4.0f;
constexpr int WAIT_LIMIT = 1 << 22;
constexpr uint32_t TM_COLS = 256, COL_AK = 0, COL_AV = 64, COL_S = 128, COL_O = 160;

// ---------------------------------------------------------------------------
// small PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void cp_async16_if(uint32_t smem_addr, const void* gmem, bool on) {
  asm volatile(
      "{\n"
      ".reg .pred q;\n"
      "setp.ne.b32 q, %2, 0;\n"
      "@q cp.async.cg.shared.global [%0], [%1], 16;\n"
      "}\n" ::"r"(smem_addr),
      "l"(gmem), "r"((int)on)
      : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t hmul2_u(uint32_t a, uint32_t b) {
  __half2 r = __hmul2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<__half2*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ float2 half2_to_float2(uint32_t a) { return __half22float2(*reinterpret_cast<__half2*>(&a)); }
__device__ __forceinline__ float bf16_to_f(uint16_t u) { return __uint_as_float(((uint32_t)u) << 16); }
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait; false if the phase did not complete within WAIT_LIMIT polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (int i = 0; i < WAIT_LIMIT; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st4(uint32_t taddr, const float* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(taddr), "f"(r[0]), "f"(r[1]),
               "f"(r[2]), "f"(r[3])
               : "memory");
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, float* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];\n"
               : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3])
               : "r"(taddr)
               : "memory");
}
template <int GP>
__device__ __forceinline__ void tmem_ld_row(uint32_t taddr, float (&r)[GP]) {
#pragma unroll
  for (int i = 0; i < GP; i += 4) tmem_ld4(taddr + i, r + i);
}
template <int GP>
__device__ __forceinline__ void tmem_st_row(uint32_t taddr, const float (&r)[GP]) {
#pragma unroll
  for (int i = 0; i < GP; i += 4) tmem_st4(taddr + i, r + i);
}

// shared-memory matrix descriptor, no swizzle: core matrices of 8 rows x 16 bytes;
// lbo / sbo: byte distance between core matrices along the leading / the other dimension
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3fff);
  d |= (uint64_t)((lbo >> 4) & 0x3fff) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3fff) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version of this architecture
  return d;
}
// kind::f16 instruction descriptor: fp16 A and B, fp32 accumulate, M = 128, A K-major (tensor memory)
__host__ __device__ constexpr uint32_t idesc_f16(int n, int b_mn_major) {
  return (1u << 4) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// D[128 x N] (+)= A[128 x 16] (tensor memory) * B[16 x N] (shared memory); one thread issues
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5,%5,%5,%5}, p;\n"
      "}\n" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}

// ---------------------------------------------------------------------------
// stage of one 128-token batch and the slot arithmetic of the code words
// ---------------------------------------------------------------------------
template <int BK, int BV, int GS>
struct Stage {
  static constexpr int NG = HD / GS;     // channel groups of a value row
  static constexpr int NGRP = BT / GS;   // key token groups per batch
  static constexpr int KU = 512 * BK;    // key codes of one 32-token unit
  static constexpr int KC = 4 * KU;
  static constexpr int KS = NGRP * 256;  // key scale rows of the batch's groups
  static constexpr int VC = 2048 * BV;   // value codes of the block: [chunk][128 channels][16 B]
  static constexpr int VM = BT * 4 * NG; // value scale / zero-point: per token [2][NG] fp16
  static constexpr int OFF_KS = KC;
  static constexpr int OFF_VC = KC + KS;
  static constexpr int OFF_VM = KC + KS + VC;
  static constexpr int BYTES = KC + KS + VC + VM;
};

// key codes: log2 of the weight channel d's code carries in its operand element
template <int BK>
__host__ __device__ constexpr int k_weight_log2(int d) {
  return BK == 2 ? ((((d % 16) / 2) < 5) ? 2 * ((d % 16) / 2) : 2 * (((d % 16) / 2) - 5)) : (((d % 32) / 2) % 8);
}
// value codes: same for token t of a block
template <int BV>
__host__ __device__ constexpr int v_weight_log2(int t) {
  return BV == 2 ? 2 * (((t % 16) / 2) % 2) : (((t % 32) / 2) % 4);
}

// Expands this thread's token (lane of unit `warp`) into its A_K row: 64 columns of fp16x2.
template <int BK>
__device__ __forceinline__ void expand_keys(uint32_t unit_smem, int lane, uint32_t row_taddr) {
  if (BK == 2) {
    const uint4 c0 = lds128(unit_smem + lane * 16), c1 = lds128(unit_smem + 512 + lane * 16);
    const uint32_t w[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t r[16];
#pragma unroll
      for (int jj = 0; jj < 2; ++jj) {
        const uint32_t wj = w[2 * q + jj], ws = wj >> 10;
#pragma unroll
        for (int s = 0; s < 8; ++s) r[8 * jj + s] = (s < 5) ? (wj & (0x00030003u << (2 * s))) : (ws & (0x00030003u << (2 * (s - 5))));
      }
      tmem_st16(row_taddr + 16 * q, r);
    }
  } else {
    const uint4 c0 = lds128(unit_smem + lane * 16);
    const uint32_t w[4] = {c0.x, c0.y, c0.z, c0.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t r[16];
      const uint32_t wj = w[q], ws = wj >> 8;
#pragma unroll
      for (int s = 0; s < 16; ++s) r[s] = ((s < 8) ? wj : ws) & (0x00010001u << (s & 7));
      tmem_st16(row_taddr + 16 * q, r);
    }
  }
}

// Expands this thread's channel d into its A_V row: 64 columns of fp16x2 over the block's 128 tokens.
template <int BV>
__device__ __forceinline__ void expand_values(uint32_t vc_smem, int d, uint32_t row_taddr) {
  if (BV == 1) {
    const uint4 c0 = lds128(vc_smem + d * 16);
    const uint32_t w[4] = {c0.x, c0.y, c0.z, c0.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t r[16];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t wk = w[q] >> (4 * k);
#pragma unroll
        for (int s = 0; s < 4; ++s) r[4 * k + s] = wk & (0x00010001u << s);
      }
      tmem_st16(row_taddr + 16 * q, r);
    }
  } else {
    const uint4 c0 = lds128(vc_smem + d * 16), c1 = lds128(vc_smem + (128 + d) * 16);
    const uint32_t w[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t r[16];
#pragma unroll
      for (int jj = 0; jj < 2; ++jj) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t wk = w[2 * q + jj] >> (4 * k);
          r[8 * jj + 2 * k] = wk & 0x00030003u;
          r[8 * jj + 2 * k + 1] = wk & 0x000C000Cu;
        }
      }
      tmem_st16(row_taddr + 16 * q, r);
    }
  }
}

constexpr int MS = HD + 4;  // state row: acc[HD], m, l, padding (keeps rows 16-byte aligned)

// ---------------------------------------------------------------------------
// window path: plain fp32 over 16-bit tokens [t0, t1); warp w takes tokens
// t0 + w, t0 + w + 4, ... four at a time.  The loads of q and of the first four
// tokens are issued by window_preload, later rounds load one round ahead.  Each
// warp leaves its state (acc, m, l per head) in `ws`.
// ---------------------------------------------------------------------------
struct WindowRegs {
  uint2 q[8];   // this lane's 4 channels of each query head of the group
  uint2 k[4];   // this lane's 4 channels of up to four window tokens
  uint2 v[4];
};

__device__ __forceinline__ void window_load_round(const DecodeParams& p, int tb, int t1, int hk, int b, uint2 (&k)[4],
                                                  uint2 (&v)[4]) {
  const Dims& dm = p.dm;
  const int lane = threadIdx.x & 31;
  const size_t row0 = (size_t)(b * dm.Hkv + hk) * dm.R;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int t = tb + i * UW;
    k[i] = v[i] = make_uint2(0u, 0u);
    if (t < t1) {
      k[i] = *reinterpret_cast<const uint2*>(p.L.win_k + (row0 + t) * HD + lane * 4);
      v[i] = *reinterpret_cast<const uint2*>(p.L.win_v + (row0 + t) * HD + lane * 4);
    }
  }
}

__device__ __forceinline__ void window_preload(const DecodeParams& p, int t0, int t1, int hk, int b, WindowRegs& w) {
  const Dims& dm = p.dm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int a = 0; a < 8; ++a)
    w.q[a] = *reinterpret_cast<const uint2*>(p.q + ((size_t)b * dm.Hq + hk * dm.G + (a < dm.G ? a : 0)) * HD + lane * 4);
  window_load_round(p, t0 + warp, t1, hk, b, w.k, w.v);
}

__device__ __forceinline__ void window_tokens(const DecodeParams& p, int t0, int t1, int hk, int b, float* ws,
                                              WindowRegs& w) {
  const Dims& dm = p.dm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = dm.G;
  const float scale2 = p.scale * 1.4426950408889634f;
  float q[8][4], acc[8][4], m[8], l[8];
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    m[a] = -CUDART_INF_F;
    l[a] = 0.f;
    q[a][0] = bf16_to_f(w.q[a].x & 0xffff) * scale2; q[a][1] = bf16_to_f(w.q[a].x >> 16) * scale2;
    q[a][2] = bf16_to_f(w.q[a].y & 0xffff) * scale2; q[a][3] = bf16_to_f(w.q[a].y >> 16) * scale2;
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[a][j] = 0.f;
  }
  for (int tb = t0 + warp; tb < t1; tb += 4 * UW) {
    uint2 kn[4], vn[4];
    window_load_round(p, tb + 4 * UW, t1, hk, b, kn, vn);  // next round, in flight during this one
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (tb + i * UW < t1) {
        const float kx[4] = {bf16_to_f(w.k[i].x & 0xffff), bf16_to_f(w.k[i].x >> 16), bf16_to_f(w.k[i].y & 0xffff),
                             bf16_to_f(w.k[i].y >> 16)};
        const float vx[4] = {bf16_to_f(w.v[i].x & 0xffff), bf16_to_f(w.v[i].x >> 16), bf16_to_f(w.v[i].y & 0xffff),
                             bf16_to_f(w.v[i].y >> 16)};
#pragma unroll
        for (int a = 0; a < 8; ++a) {
          if (a < G) {
            float x = q[a][0] * kx[0];
            x = fmaf(q[a][1], kx[1], x);
            x = fmaf(q[a][2], kx[2], x);
            x = fmaf(q[a][3], kx[3], x);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            float mn = fmaxf(m[a], x);
            float corr = ex2(m[a] - mn);
            float pe = ex2(x - mn);
            l[a] = l[a] * corr + pe;
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[a][j] = acc[a][j] * corr + pe * vx[j];
            m[a] = mn;
          }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      w.k[i] = kn[i];
      w.v[i] = vn[i];
    }
  }
  float* mine = ws + (size_t)warp * G * MS;
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    if (a < G) {
      float* row = mine + a * MS;
      *reinterpret_cast<float4*>(row + lane * 4) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
      if (lane == 0) {
        row[HD] = m[a];
        row[HD + 1] = l[a];
      }
    }
  }
}

// Combines the CTA's packed-region state (mb: G rows of MS floats, may be absent)
// with the four warps' window states (ws: G rows per warp, may be absent) and
// writes the CTA's partial for each head.
__device__ __forceinline__ void write_partial(const DecodeParams& p, const float* mb, const float* ws, int split,
                                              int ns, int hk, int b) {
  const Dims& dm = p.dm;
  const int d = threadIdx.x;  // UT == HD
  const int G = dm.G;
  for (int a = 0; a < G; ++a) {
    float M = mb ? mb[a * MS + HD] : -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < UW; ++w)
      if (ws) M = fmaxf(M, ws[(w * G + a) * MS + HD]);
    float Lsum = 0.f, A = 0.f;
    if (mb) {
      const float* row = mb + a * MS;
      float f = ex2(row[HD] - M);  // 2^-inf = 0 for an empty state; M is finite whenever any state is not empty
      Lsum = row[HD + 1] * f;
      A = row[d] * f;
    }
#pragma unroll
    for (int w = 0; w < UW; ++w) {
      if (ws) {
        const float* row = ws + (w * G + a) * MS;
        float f = ex2(row[HD] - M);
        Lsum = fmaf(row[HD + 1], f, Lsum);
        A = fmaf(row[d], f, A);
      }
    }
    size_t hq = (size_t)b * dm.Hq + hk * G + a;
    p.part_acc[(hq * ns + split) * HD + d] = A;
    if (d == 0) *reinterpret_cast<float2*>(p.part_ml + (hq * ns + split) * 2) = make_float2(M, Lsum);
  }
}

__device__ __forceinline__ float ld_cg(const float* p) {
  float v;
  asm volatile("ld.global.cg.f32 %0, [%1];\n" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ float4 ld_cg4(const float* p) {
  float4 v;
  asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

// Split-K merge by the last CTA of a (sequence, kv head): takes a ticket after
// its partials are visible device-wide; the CTA that draws the last ticket reads
// all partials from L2 and writes out = sum_s acc_s 2^(m_s-M) / sum_s l_s 2^(m_s-M).
// No CTA ever waits for another.
__device__ __forceinline__ void ticket_merge(const DecodeParams& p, int ns, int hk, int b, int* s_flag) {
  const Dims& dm = p.dm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = b * dm.Hkv + hk;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned t = atomicAdd(p.tickets + bh, 1u);
    *s_flag = (t == (unsigned)(ns - 1));
  }
  __syncthreads();
  if (!*s_flag) return;
  __threadfence();
  for (int a = warp; a < dm.G; a += UW) {
    const size_t hq = (size_t)b * dm.Hq + hk * dm.G + a;
    const float* ml = p.part_ml + hq * ns * 2;
    const float* pa = p.part_acc + hq * ns * HD + lane * 4;
    float M = -CUDART_INF_F;
    for (int s = lane; s < ns; s += 32) M = fmaxf(M, ld_cg(ml + 2 * s));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float Ls = 0.f;
#pragma unroll 4
    for (int s = 0; s < ns; ++s) {
      float f = ex2(ld_cg(ml + 2 * s) - M);
      Ls = fmaf(ld_cg(ml + 2 * s + 1), f, Ls);
      float4 v = ld_cg4(pa + (size_t)s * HD);
      acc.x = fmaf(v.x, f, acc.x); acc.y = fmaf(v.y, f, acc.y);
      acc.z = fmaf(v.z, f, acc.z); acc.w = fmaf(v.w, f, acc.w);
    }
    const float inv = 1.0f / Ls;
    acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    if (p.out_f32) {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + hq * HD + lane * 4) = acc;
    } else {
      __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
      uint2 pk = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + hq * HD + lane * 4) = pk;
    }
  }
  if (threadIdx.x == 0) p.tickets[bh] = 0u;  // ready for the next launch on this stream
}

// ---------------------------------------------------------------------------
// shared memory plan (dynamic):
//   [NSTB stages]  (the merge buffer aliases the start after the loop)
//   [B_K: N_S x 128 fp16, K-major] [B_P: 128 x N_O fp16, N-major; B_Q of the bias MMAs aliases it]
//   [bias: 128 groups x 8 fp32] [reduction scratch: 4 warps x 32 fp32] [window states]
// ---------------------------------------------------------------------------
template <int BK, int BV, int GS, int GP>
struct Plan {
  using St = Stage<BK, BV, GS>;
  static constexpr int N_S = (St::NGRP * GP) < 16 ? 16 : St::NGRP * GP;  // columns of S: (token group, head)
  static constexpr int N_O = (St::NG * GP) < 16 ? 16 : St::NG * GP;      // columns of O: (channel group, head)
  static constexpr int OFF_BK = NSTB * St::BYTES;
  static constexpr int BK_BYTES = N_S * HD * 2;
  static constexpr int OFF_BP = OFF_BK + BK_BYTES;
  static constexpr int BP_BYTES = (BT * N_O * 2) > (16 * HD * 2) ? (BT * N_O * 2) : (16 * HD * 2);
  static constexpr int OFF_BIAS = OFF_BP + BP_BYTES;
  static constexpr int BIAS_BYTES = 128 * 8 * 4;
  static constexpr int OFF_RED = OFF_BIAS + BIAS_BYTES;
  static constexpr int RED_BYTES = UW * 32 * 4;
  static constexpr int OFF_WS = OFF_RED + RED_BYTES;
  static constexpr int MERGE_BYTES = 8 * MS * 4;
  static_assert(OFF_BK >= MERGE_BYTES, "the merge buffer aliases the stages");
};
__host__ __device__ inline int wstate_bytes(int G) { return UW * G * MS * 4; }

// ---------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------
template <int BK, int BV, int GS, int GP>
__global__ void __launch_bounds__(UT, 2) decode_umma_kernel(DecodeParams p) {
  using St = Stage<BK, BV, GS>;
  using Pl = Plan<BK, BV, GS, GP>;
  constexpr int NG = St::NG, NGRP = St::NGRP, N_S = Pl::N_S, N_O = Pl::N_O;
  constexpr int WPG = GS / 32;                  // warps whose tokens share a key group
  constexpr int NITEM = (GP * 16) / (32 * WPG); // (head, 8-channel chunk) rows of B_K per lane
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) unsigned long long bar_mem[2];
  __shared__ uint32_t tmem_base_sm;
  __shared__ int s_flag;
  float* mb = reinterpret_cast<float*>(smem);
  float* bias_sm = reinterpret_cast<float*>(smem + Pl::OFF_BIAS);
  float* red = reinterpret_cast<float*>(smem + Pl::OFF_RED);
  float* ws = reinterpret_cast<float*>(smem + Pl::OFF_WS);

  const Dims& dm = p.dm;
  const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = dm.G;

  if (p.ns_q == 0) {  // nothing is quantized yet: window-only splits
    const int ns = p.ns_w;
    const int tiles = (p.r + 15) / 16;
    const int t0 = (int)(((long long)split * tiles) / ns) * 16;
    const int t1 = min((int)(((long long)(split + 1) * tiles) / ns) * 16, p.r);
    WindowRegs wr;
    window_preload(p, t0, t1, hk, b, wr);
    window_tokens(p, t0, t1, hk, b, ws, wr);
    __syncthreads();
    write_partial(p, nullptr, ws, split, ns, hk, b);
    ticket_merge(p, ns, hk, b, &s_flag);
    return;
  }

  const int ns = p.ns_q;
  const int nb_total = (p.n_q + BT - 1) / BT;
  const int b0 = (int)(((long long)split * nb_total) / ns);
  const int nb = (int)(((long long)(split + 1) * nb_total) / ns) - b0;  // this CTA's batches: [b0, b0 + nb), 1 <= nb <= GS
  const int bh = b * dm.Hkv + hk;

  // the four streams at this CTA's first batch
  const uint8_t* gk = reinterpret_cast<const uint8_t*>(p.L.k_codes) + (size_t)bh * ((size_t)dm.nq_cap * (HD * BK / 8)) +
                      (size_t)b0 * St::KC;
  const uint8_t* gv = reinterpret_cast<const uint8_t*>(p.L.v_codes) + (size_t)bh * ((size_t)dm.nq_cap * (HD * BV / 8)) +
                      (size_t)b0 * St::VC;
  const uint8_t* gvm = reinterpret_cast<const uint8_t*>(p.L.v_meta) + (size_t)bh * ((size_t)dm.nq_cap * 4 * NG) +
                       (size_t)b0 * St::VM;
  const size_t plane = (size_t)(dm.nq_cap / GS) * 256;  // bytes of the key scale plane (= of the zero-point plane)
  const uint8_t* gks = reinterpret_cast<const uint8_t*>(p.L.k_meta) + (size_t)bh * 2 * plane + (size_t)b0 * St::KS;
  const uint8_t* gkz = gks + plane;

  const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(smem);
  const uint32_t barS = (uint32_t)__cvta_generic_to_shared(&bar_mem[0]);
  const uint32_t barO = (uint32_t)__cvta_generic_to_shared(&bar_mem[1]);

  // ---- loads the prologue waits for go out first ----
  const int wt0 = (int)(((long long)split * p.r) / ns), wt1 = (int)(((long long)(split + 1) * p.r) / ns);
  WindowRegs wr;
  window_preload(p, wt0, wt1, hk, b, wr);

  // stage batch jj of this CTA into ring slot `slot`, if it exists (no commit, no branch)
  auto issue_batch = [&](int jj, int slot) {
    const bool on = jj < nb;
    const uint32_t s = sm_base + slot * St::BYTES + tid * 16;
    const uint8_t* k = gk + (size_t)(uint32_t)jj * St::KC + tid * 16;
#pragma unroll
    for (int i = 0; i < St::KC / 2048; ++i) cp_async16_if(s + i * 2048, k + i * 2048, on);
    cp_async16_if(s + St::OFF_KS, gks + (size_t)(uint32_t)jj * St::KS + tid * 16, on && tid * 16 < St::KS);
    const uint8_t* v = gv + (size_t)(uint32_t)jj * St::VC + tid * 16;
#pragma unroll
    for (int i = 0; i < St::VC / 2048; ++i) cp_async16_if(s + St::OFF_VC + i * 2048, v + i * 2048, on);
    cp_async16_if(s + St::OFF_VM, gvm + (size_t)(uint32_t)jj * St::VM + tid * 16, on && tid * 16 < St::VM);
  };
#pragma unroll
  for (int jj = 0; jj < NSTB - 1; ++jj) {
    issue_batch(jj, jj);
    cp_async_commit();
  }

  // ---- set-up: barriers, tensor memory, zeroed B operands ----
  if (tid == 0) {
    mbar_init(barS, 1);
    mbar_init(barO, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(
                     (uint32_t)__cvta_generic_to_shared(&tmem_base_sm)),
                 "r"(TM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  for (int i = tid; i < (Pl::BK_BYTES + Pl::BP_BYTES) / 16; i += UT) sts128(sm_base + Pl::OFF_BK + i * 16, 0u, 0u, 0u, 0u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = tmem_base_sm;
  const uint32_t lane_base = tbase + ((uint32_t)(warp * 32) << 16);
  uint32_t phS = 0, phO = 0;  // parities of the next completions of barS / barO
  bool dead = false;          // a bounded wait gave up

  // ---- q: B operand of the bias MMAs (unscaled, rows = heads) and this lane's pre-weighted chunks for B_K ----
  // B_Q[n][k] K-major, N = 16: byte offset (k/8)*256 + (n/8)*128 + (n%8)*16 + (k%8)*2
  {
    const int h = tid >> 4, ck = tid & 15;  // 8 heads x 16 chunks of 8 channels
    if (h < G) {
      const uint4 raw = *reinterpret_cast<const uint4*>(p.q + ((size_t)b * dm.Hq + hk * G + h) * HD + ck * 8);
      const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) o[i] = pack_half2(bf16_to_f(rw[i] & 0xffff), bf16_to_f(rw[i] >> 16));
      sts128(sm_base + Pl::OFF_BP + ck * 256 + (h >> 3) * 128 + (h & 7) * 16, o[0], o[1], o[2], o[3]);
    }
  }
  const int my_gl = (warp * 32) / GS;  // token group (within the batch) of this warp's tokens
  uint32_t qk[NITEM][4];               // q chunks of this lane's B_K rows, times 2^-weight of each channel's slot
  int item_h[NITEM], item_ck[NITEM];
#pragma unroll
  for (int it = 0; it < NITEM; ++it) {
    const int item = (warp % WPG) * 32 + lane + it * 32 * WPG;
    const int h = item >> 4, ck = item & 15;
    item_h[it] = h;
    item_ck[it] = ck;
    uint4 raw = make_uint4(0u, 0u, 0u, 0u);
    if (h < G) raw = *reinterpret_cast<const uint4*>(p.q + ((size_t)b * dm.Hq + hk * G + h) * HD + ck * 8);
    const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = (BK == 2) ? ((((ck & 1) * 4 + i) < 5) ? 2 * ((ck & 1) * 4 + i) : 2 * ((ck & 1) * 4 + i - 5))
                              : ((((ck & 3) * 4 + i)) % 8);
      // channels 8 ck + 2 i, 8 ck + 2 i + 1 share a slot
      const float sc = __int_as_float((127 - e) << 23);
      qk[it][i] = pack_half2(bf16_to_f(rw[i] & 0xffff) * sc, bf16_to_f(rw[i] >> 16) * sc);
    }
  }

  // ---- bias of every key token group of this CTA's range: bias_sm[group][head] = scale2 * sum_d q_d z_d ----
  const float scale2 = p.scale * 1.4426950408889634f;
  const int n_grp = nb * NGRP;  // <= 128
  {
    // thread = group row: its 128 zero-points are already fp16 pairs in channel order = one A row
    const int gr = min(tid, n_grp - 1);
    const uint4* zrow = reinterpret_cast<const uint4*>(gkz + (size_t)gr * 256);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint4 z[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) z[i] = zrow[4 * q + i];
      const uint32_t r[16] = {z[0].x, z[0].y, z[0].z, z[0].w, z[1].x, z[1].y, z[1].z, z[1].w,
                              z[2].x, z[2].y, z[2].z, z[2].w, z[3].x, z[3].y, z[3].z, z[3].w};
      tmem_st16(lane_base + COL_AK + 16 * q, r);
    }
    tc_wait_st();
    proxy_fence();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      constexpr uint32_t idesc = idesc_f16(16, 0);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        umma_ts(tbase + COL_S, tbase + COL_AK + 8 * ks, smem_desc(sm_base + Pl::OFF_BP + ks * 512, 256, 128), idesc, ks > 0);
      umma_commit(barS);
    }
  }
  // the window share, while the bias MMAs and the first copies fly
  window_tokens(p, wt0, wt1, hk, b, ws, wr);
  dead = __syncthreads_or(!mbar_wait(barS, phS));
  phS ^= 1;
  if (!dead) {
    tc_fence_after();
    float bz[8];
    tmem_ld4(lane_base + COL_S, bz);
    tmem_ld4(lane_base + COL_S + 4, bz + 4);
    tc_wait_ld();
#pragma unroll
    for (int h = 0; h < 8; ++h) bias_sm[tid * 8 + h] = bz[h] * scale2;
    // B_Q is dead: clear its place for B_P (padding columns must read as zero)
    for (int i = tid; i < Pl::BP_BYTES / 16; i += UT) sts128(sm_base + Pl::OFF_BP + i * 16, 0u, 0u, 0u, 0u);
  }

  const float c1 = scale2 * 16777216.0f;  // undoes the 2^-24 of the subnormal code operand
  float m[GP], L[GP], zacc[NG][GP];
#pragma unroll
  for (int h = 0; h < GP; ++h) {
    m[h] = -CUDART_INF_F;
    L[h] = 0.f;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) zacc[gi][h] = 0.f;
  }
  const float vw = __int_as_float((127 - v_weight_log2<BV>(lane)) << 23);  // 2^-weight of this lane's token slot (values)
  constexpr uint32_t idescS = idesc_f16(N_S, 0), idescO = idesc_f16(N_O, 1);
  constexpr uint32_t LBO_K = (N_S / 8) * 128, LBO_P = (N_O / 8) * 128;

  // B_K rows of this warp's group for the batch staged at `st`
  auto build_bk = [&](uint32_t st) {
#pragma unroll
    for (int it = 0; it < NITEM; ++it) {
      const int h = item_h[it], ck = item_ck[it];
      if (h < G) {
        const uint4 sv = lds128(st + St::OFF_KS + my_gl * 256 + ck * 16);
        const int n = my_gl * GP + h;
        sts128(sm_base + Pl::OFF_BK + ck * LBO_K + (n >> 3) * 128 + (n & 7) * 16, hmul2_u(qk[it][0], sv.x),
               hmul2_u(qk[it][1], sv.y), hmul2_u(qk[it][2], sv.z), hmul2_u(qk[it][3], sv.w));
      }
    }
  };
  auto issue_key_mmas = [&]() {  // one thread
    tc_fence_after();
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
      umma_ts(tbase + COL_S, tbase + COL_AK + 8 * ks, smem_desc(sm_base + Pl::OFF_BK + ks * 2 * LBO_K, LBO_K, 128), idescS,
              ks > 0);
    umma_commit(barS);
  };

  // ---- first batch: keys expanded and their MMAs issued ----
  cp_async_wait<NSTB - 3>();  // batches 0 and 1 have landed (for this thread)
  __syncthreads();
  if (!dead) {
    expand_keys<BK>(sm_base + warp * St::KU, lane, lane_base + COL_AK);
    build_bk(sm_base);
    tc_wait_st();
    proxy_fence();
    tc_fence_before();
  }
  __syncthreads();
  if (tid == 0 && !dead) issue_key_mmas();

  int slot = 0;  // ring slot of batch i
  for (int i = 0; i < nb && !dead; ++i) {
    const uint32_t st = sm_base + slot * St::BYTES;
    const int slot_next = (slot + 1 == NSTB) ? 0 : slot + 1;
    const int slot_prev = (slot == 0) ? NSTB - 1 : slot - 1;
    const int tok = (b0 + i) * BT + tid;  // this thread's token (keys, softmax)
    const bool valid = tok < p.n_q;
    const int gidx = i * NGRP + my_gl;     // its key group within this CTA's range

    // 1. logits of batch i
    bool lost = !mbar_wait(barS, phS);
    phS ^= 1;
    tc_fence_after();
    float x[GP];
    tmem_ld_row<GP>(lane_base + COL_S + my_gl * GP, x);
    tc_wait_ld();
    bool raise = false;
#pragma unroll
    for (int h = 0; h < GP; ++h) {
      x[h] = (valid && h < G) ? fmaf(x[h], c1, bias_sm[gidx * 8 + h]) : -CUDART_INF_F;
      raise |= x[h] > m[h] + TAU;
    }
    // 2. keys of batch i + 1 (their stage became visible at the previous barrier)
    if (i + 1 < nb) {
      const uint32_t sn = sm_base + slot_next * St::BYTES;
      expand_keys<BK>(sn + warp * St::KU, lane, lane_base + COL_AK);
      build_bk(sn);
      tc_wait_st();
      proxy_fence();
    }
    tc_fence_before();
    // 3. barrier: S has been read by everyone, A_K / B_K of batch i + 1 are complete
    const int votes = __syncthreads_or((raise ? 1 : 0) | (lost ? 2 : 0));
    if (votes & 2) {
      dead = true;
      break;
    }
    if (tid == 0 && i + 1 < nb) issue_key_mmas();
    // the slot of batch i - 1 is free now: refill it
    issue_batch(i + NSTB - 1, slot_prev);
    cp_async_commit();

    // the value MMAs of batch i - 1 must be done before A_V, B_P (and O, when rescaling) are touched
    if (i > 0) {
      lost = !mbar_wait(barO, phO);
      phO ^= 1;
      tc_fence_after();
    }
    // 4. raise the softmax reference (rare): CTA-wide maximum per head, rescale O, L, the zero-point sums
    if (votes & 1) {
      float xm[GP];
#pragma unroll
      for (int h = 0; h < GP; ++h) {
        xm[h] = x[h];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) xm[h] = fmaxf(xm[h], __shfl_xor_sync(0xffffffffu, xm[h], o));
        if (lane == 0) red[warp * 32 + h] = xm[h];
      }
      __syncthreads();
      float f[GP];
#pragma unroll
      for (int h = 0; h < GP; ++h) {
        const float mn = fmaxf(fmaxf(m[h], fmaxf(red[h], red[32 + h])), fmaxf(red[64 + h], red[96 + h]));
        f[h] = ex2(m[h] - mn);  // 0 on the first batch (m = -inf); padded heads: -inf - -inf = NaN, never used
        m[h] = mn;
        L[h] *= f[h];
#pragma unroll
        for (int gi = 0; gi < NG; ++gi) zacc[gi][h] *= f[h];
      }
      if (i > 0) {  // this thread's channel row of O: the columns of its own channel group
        const uint32_t oaddr = lane_base + COL_O + ((warp * 32) / GS) * GP;
        float o[GP];
        tmem_ld_row<GP>(oaddr, o);
        tc_wait_ld();
#pragma unroll
        for (int h = 0; h < GP; ++h) o[h] *= f[h];
        tmem_st_row<GP>(oaddr, o);
      }
      __syncthreads();  // `red` may be reused
    }

    // 5. numerators of batch i, P' rows, zero-point and normaliser sums; values of batch i
    {
      uint32_t sv[NG / 2], zv[NG / 2];  // this token's value scales and zero-points, fp16 pairs
      if (NG == 4) {
        uint4 mt = lds128(st + St::OFF_VM + tid * 16);
        sv[0] = mt.x; sv[NG / 2 - 1] = mt.y; zv[0] = mt.z; zv[NG / 2 - 1] = mt.w;
      } else {
        uint2 mt = lds64(st + St::OFF_VM + tid * 8);
        sv[0] = mt.x; zv[0] = mt.y;
      }
      if (!valid) {
#pragma unroll
        for (int i2 = 0; i2 < NG / 2; ++i2) sv[i2] = zv[i2] = 0u;
      }
      float pe[GP];
#pragma unroll
      for (int h = 0; h < GP; ++h) {
        pe[h] = (valid && h < G) ? ex2(x[h] - m[h]) * vw : 0.f;  // carries 2^-weight of the token's value slot
        L[h] += pe[h];
      }
#pragma unroll
      for (int g2 = 0; g2 < NG / 2; ++g2) {
        const float2 zf = half2_to_float2(zv[g2]);
#pragma unroll
        for (int h = 0; h < GP; ++h) {
          zacc[2 * g2][h] = fmaf(pe[h], zf.x, zacc[2 * g2][h]);
          zacc[2 * g2 + 1][h] = fmaf(pe[h], zf.y, zacc[2 * g2 + 1][h]);
        }
      }
      uint32_t ph[GP / 2];
#pragma unroll
      for (int h = 0; h < GP / 2; ++h) ph[h] = pack_half2(pe[2 * h], pe[2 * h + 1]);
      // row `tid` of B_P: columns gi * GP + h, 8 columns per 16-byte chunk
      const uint32_t prow = sm_base + Pl::OFF_BP + (tid >> 3) * LBO_P + (tid & 7) * 16;
#pragma unroll
      for (int gi = 0; gi < NG; ++gi) {
        const uint32_t sb = __byte_perm(sv[gi >> 1], 0u, (gi & 1) ? 0x3232 : 0x1010);  // (s, s)
        if (GP == 4) {
          if ((gi & 1) == 0) {
            const uint32_t sb1 = __byte_perm(sv[gi >> 1], 0u, 0x3232);
            sts128(prow + (gi >> 1) * 128, hmul2_u(ph[0], sb), hmul2_u(ph[1], sb), hmul2_u(ph[0], sb1), hmul2_u(ph[1], sb1));
          }
        } else {
          sts128(prow + gi * 128, hmul2_u(ph[0], sb), hmul2_u(ph[1], sb), hmul2_u(ph[GP / 2 - 2], sb),
                 hmul2_u(ph[GP / 2 - 1], sb));
        }
      }
    }
    expand_values<BV>(st + St::OFF_VC, tid, lane_base + COL_AV);
    tc_wait_st();
    proxy_fence();
    tc_fence_before();
    cp_async_wait<NSTB - 3>();  // batch i + 2 has landed (for this thread); visible to all after the barrier
    // 6. barrier: A_V and B_P are complete
    if (__syncthreads_or(lost ? 1 : 0)) {
      dead = true;
      break;
    }
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        umma_ts(tbase + COL_O, tbase + COL_AV + 8 * ks, smem_desc(sm_base + Pl::OFF_BP + ks * 2 * LBO_P, LBO_P, 128), idescO,
                (i > 0 || ks > 0) ? 1u : 0u);
      umma_commit(barO);
    }
    slot = slot_next;
  }

  // ---- epilogue ----
  cp_async_wait<0>();
  if (!dead) dead = !mbar_wait(barO, phO);  // the last value MMAs
  dead = __syncthreads_or(dead ? 1 : 0) != 0;
  tc_fence_after();
  if (dead && tid == 0) atomicExch(p.status, 1);
  if (!dead) {
    // L and the zero-point sums were accumulated with the per-lane factor 2^-weight; undo it, then reduce
    const float uw = __int_as_float((127 + v_weight_log2<BV>(lane)) << 23);
    float* wsum = reinterpret_cast<float*>(smem + Pl::OFF_BK);  // [warp][64]; B_K is dead
#pragma unroll
    for (int r = 0; r <= NG; ++r) {
#pragma unroll
      for (int h = 0; h < GP; ++h) {
        float v = ((r < NG) ? zacc[r < NG ? r : 0][h] : L[h]) * uw;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) wsum[warp * 64 + r * GP + h] = v;
      }
    }
  }
  __syncthreads();  // all stages are dead: the memory becomes the merge buffer
  if (!dead) {
    const float* wsum = reinterpret_cast<const float*>(smem + Pl::OFF_BK);
    const int gi = (warp * 32) / GS;  // channel group of this thread's channel
    float o[GP];
    tmem_ld_row<GP>(lane_base + COL_O + gi * GP, o);
    tc_wait_ld();
#pragma unroll
    for (int h = 0; h < GP; ++h) {
      if (h < G) {
        const float z = wsum[gi * GP + h] + wsum[64 + gi * GP + h] + wsum[128 + gi * GP + h] + wsum[192 + gi * GP + h];
        mb[h * MS + tid] = fmaf(o[h], 16777216.0f, z);  // the code operands carried 2^-24
        if (tid == 0) {
          mb[h * MS + HD] = m[h];
          mb[h * MS + HD + 1] = wsum[NG * GP + h] + wsum[64 + NG * GP + h] + wsum[128 + NG * GP + h] + wsum[192 + NG * GP + h];
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tbase), "r"(TM_COLS) : "memory");
  if (dead) {  // leave a neutral partial so that the merge stays finite; the status word tells the host
    for (int a = 0; a < G; ++a) {
      mb[a * MS + tid] = 0.f;
      if (tid == 0) {
        mb[a * MS + HD] = -CUDART_INF_F;
        mb[a * MS + HD + 1] = 0.f;
      }
    }
    __syncthreads();
  }
  write_partial(p, mb, ws, split, ns, hk, b);
  ticket_merge(p, ns, hk, b, &s_flag);
}

template <int BK, int BV, int GS, int GP>
int smem_bytes(int G) {
  return Plan<BK, BV, GS, GP>::OFF_WS + wstate_bytes(G);
}

template <int BK, int BV, int GS, int GP>
cudaError_t launch_t(const DecodeParams& p, cudaStream_t st) {
  const int smem = smem_bytes<BK, BV, GS, GP>(p.dm.G);
  static int configured = 0;
  if (configured < smem) {
    cudaError_t e = cudaFuncSetAttribute(decode_umma_kernel<BK, BV, GS, GP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  const int ns = p.ns_q > 0 ? p.ns_q : p.ns_w;
  dim3 grid(ns, p.dm.Hkv, p.dm.B);
  decode_umma_kernel<BK, BV, GS, GP><<<grid, UT, smem, st>>>(p);
  return cudaGetLastError();
}

template <int BK, int BV, int GS, int GP>
int ctas_per_sm_t(int G) {
  const int smem = smem_bytes<BK, BV, GS, GP>(G);
  if (cudaFuncSetAttribute(decode_umma_kernel<BK, BV, GS, GP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=
      cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_umma_kernel<BK, BV, GS, GP>, UT, smem) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n < 2 ? n : 2;  // 512 tensor-memory columns per SM, 256 per CTA
}

}  // namespace

bool decode_mma_supported(const Dims& dm, int bk, int bv) {
  (void)bk; (void)bv;
  return dm.D == HD && dm.G <= 8 && (dm.g == 32 || dm.g == 64);
}

// Most batches one CTA may take: its bias table holds 128 key token groups.
int decode_mma_max_batches(const Dims& dm) { return dm.g; }

#define XQ_DISPATCH(FN, ...)                                                         \
  switch (bk * 1000 + bv * 100 + (g == 64) * 10 + (G > 4)) {                          \
    case 2200: return FN<2, 2, 32, 4>(__VA_ARGS__); case 2201: return FN<2, 2, 32, 8>(__VA_ARGS__); \
    case 2210: return FN<2, 2, 64, 4>(__VA_ARGS__); case 2211: return FN<2, 2, 64, 8>(__VA_ARGS__); \
    case 2100: return FN<2, 1, 32, 4>(__VA_ARGS__); case 2101: return FN<2, 1, 32, 8>(__VA_ARGS__); \
    case 2110: return FN<2, 1, 64, 4>(__VA_ARGS__); case 2111: return FN<2, 1, 64, 8>(__VA_ARGS__); \
    case 1200: return FN<1, 2, 32, 4>(__VA_ARGS__); case 1201: return FN<1, 2, 32, 8>(__VA_ARGS__); \
    case 1210: return FN<1, 2, 64, 4>(__VA_ARGS__); case 1211: return FN<1, 2, 64, 8>(__VA_ARGS__); \
    case 1100: return FN<1, 1, 32, 4>(__VA_ARGS__); case 1101: return FN<1, 1, 32, 8>(__VA_ARGS__); \
    case 1110: return FN<1, 1, 64, 4>(__VA_ARGS__); case 1111: return FN<1, 1, 64, 8>(__VA_ARGS__); \
  }

// Resident CTAs per SM of the kernel variant for these bit-widths (0 if unknown: no device).
int decode_mma_ctas_per_sm(const Dims& dm, int bk, int bv) {
  const int g = dm.g, G = dm.G;
  XQ_DISPATCH(ctas_per_sm_t, dm.G)
  return 0;
}

cudaError_t launch_decode_mma(const DecodeParams& p, cudaStream_t st) {
  const int bk = p.L.bk, bv = p.L.bv, g = p.dm.g, G = p.dm.G;
  XQ_DISPATCH(launch_t, p, st)
  return cudaErrorInvalidValue;
}

}  // namespace xq
