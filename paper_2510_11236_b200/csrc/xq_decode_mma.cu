// Tensor-core decode attention over the packed cache (head_dim 128, up to 8
// query heads per kv head).
//
// Why mma.sync from registers: the packed cache delivers ~1.8e13 quantized
// elements/s at the HBM roofline, so an element may cost about one instruction
// per two elements and no trip through on-chip memory in expanded form.  The
// packed word layout is the A-fragment layout of mma.sync.m16n8k16, so
// `word & mask` IS an fp16x2 operand register (the code sits in the mantissa
// bits of an fp16 subnormal: value c * 2^(pos-24)), and scale / zero-point are
// folded into the other operand.  (tcgen05.mma takes A from shared or tensor
// memory: the codes would have to be expanded there first -- the same masks plus
// tcgen05.st -- and with N = 8..16 columns one tcgen05.mma costs its issuing
// thread ~67 cycles on this part; a version built that way ran slower.)
//
//   q . k_hat_t = sum_d (q_d s_d) c_td + sum_d q_d z_d        (keys, per channel)
//   sum_t p_t v_hat_td = sum_t (p_t s_tg) c_td + sum_t p_t z_tg  (values, per token)
//
// Tokens are the M dimension of both products (S^T = Kc * Q'^T, O^T = Vc^T * P'),
// so a GQA group of up to 8 query heads fills the N = 8 columns.
//
// Work split: grid (split, kv head, sequence), sized by the host to one wave of
// long-lived CTAs.  Every split takes a contiguous range of 32-token units of the
// packed region, cut into four contiguous warp ranges, plus an equal share of the
// 16-bit window tokens, which one of its warps takes as tiles of 16 tokens (bf16
// tensor-core operands loaded with ldmatrix) before its packed units.  Each warp stages its own units in
// shared memory with cp.async (a ring of NST stages: key codes, key scales, value
// codes, value scale / zero-point of one unit) and, once per 16 units, the key
// zero-point rows of the next 16 units, from which the q . z biases of those
// units are computed with one set of MMAs.  The loop is software-pipelined:
// iteration j computes the logits of unit j + 1 and, from the logits of unit j,
// the softmax numerators and the value product, so that the two MMA chains
// overlap.  The softmax reference is only raised when a logit exceeds it by more
// than TAU (checked with one vote, no shuffles), which keeps every numerator
// below 2^TAU.  The warps' states are merged at the end and the CTA writes one
// partial (m, l, acc[D]) per query head.  The CTA that finishes last for a
// (sequence, kv head) -- found with an atomic ticket, never by waiting -- merges
// the partials and writes the output.  No thread ever spins on memory.
//
// Launch: programmatic dependent launch.  The kernel lets its successor start
// at once and waits for its predecessor only after it has queued its first
// packed units (when the host says that no pack kernel wrote them since the
// layer's last decode), so its set-up hides under the predecessor's tail.
// Variants: SP (groups of <= 4 heads in the even columns, odd columns padding),
// HP (the padding column carries what the fp16 rounding of q_d s_d lost), and
// the fused append of xq_decode_step (the newest window row comes from the
// step's input and is stored into the window by the CTA that reads it).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>
#include <math_constants.h>

#include "xq_internal.h"

namespace xq {

namespace {

constexpr int MMA_WARPS = 4;
constexpr int MMA_THREADS = MMA_WARPS * 32;
constexpr int NST = 4;       // stages per warp: two being consumed, two in flight
constexpr int HD = 128;
constexpr int ZROWS = 16;    // units per zero-point bias batch
constexpr float TAU = 4.0f;  // log2 units a logit may exceed the softmax reference before it is raised

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// D = A * B (accumulator input zero)
__device__ __forceinline__ void mma16816_z(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                           uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}

// 2^x, approximate (relative error ~2^-22), flushes denormals; 2^-inf = 0
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
  return d;
}

__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_addr), "l"(gmem) : "memory");
}
// the same, issued only where `on` is true (a predicated instruction, no branch)
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
// a * b - c in one rounding, per half
__device__ __forceinline__ uint32_t hfms2_u(uint32_t a, uint32_t b, uint32_t c) {
  __half2 r = __hfma2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<__half2*>(&b), __hneg2(*reinterpret_cast<__half2*>(&c)));
  return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ uint32_t hmul2_u(uint32_t a, uint32_t b) {
  __half2 r = __hmul2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<__half2*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}
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
__device__ __forceinline__ float2 lds64f(uint32_t a) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];\n" : "=f"(v.x), "=f"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts64f(uint32_t a, float x, float y) {
  asm volatile("st.shared.v2.f32 [%0], {%1,%2};\n" ::"r"(a), "f"(x), "f"(y) : "memory");
}

// Slot s (0..7) of a word holds, per 16-bit half, a BITS-bit code at bit BITS*s
// (1-bit words carry a second sub-tile in slots 8..15, reached by a shift of 8).
// Slots whose bits fall outside the fp16 mantissa are reached by one shift.
template <int BITS>
struct Slots;
template <>
struct Slots<2> {
  static constexpr int SHIFT = 10;                                   // slots 5..7 -> bit 0, 2, 4
  __host__ __device__ static constexpr int e(int s) { return s < 5 ? 2 * s : 2 * (s - 5); }  // log2 weight
  __device__ static constexpr uint32_t mask(int s) { return 0x00030003u << e(s); }
  __device__ static constexpr bool shifted(int s) { return s >= 5; }
};
template <>
struct Slots<1> {
  static constexpr int SHIFT = 8;  // second sub-tile
  __host__ __device__ static constexpr int e(int s) { return s; }
  __device__ static constexpr uint32_t mask(int s) { return 0x00010001u << s; }
  __device__ static constexpr bool shifted(int) { return false; }
};

template <int BK, int BV, int GS>
struct Stage {
  static constexpr int NG = HD / GS;
  static constexpr int KC = 512 * BK;  // key codes of one 32-token unit
  static constexpr int KS = 256;       // key scale block of the unit's token group
  static constexpr int VC = 512 * BV;
  static constexpr int VM = 128 * NG;  // value scale + zero blocks of the unit's two 16-token tiles
  static constexpr int OFF_KS = KC;
  static constexpr int OFF_VC = KC + KS;
  static constexpr int OFF_VM = KC + KS + VC;
  static constexpr int BYTES = KC + KS + VC + VM;
};

constexpr int ZBUF_BYTES = ZROWS * 256;    // key zero-point rows of one batch
constexpr int ZTAB_BYTES = ZROWS * 8 * 4;  // q . z biases [unit][head], fp32, log2 units
constexpr int MS = HD + 4;                 // state row: acc[HD], m, l, padding (keeps rows 16-byte aligned)
constexpr int MERGE_BYTES = MMA_WARPS * 8 * MS * 4;
constexpr int Q_BYTES = 32 * 64;

// dynamic shared memory:
//   [per warp: NST stages | zero-point rows | bias table]   (the merge buffer aliases the start after the loop)
//   [q in B-operand order] [window states]
template <int BK, int BV, int GS>
constexpr int warp_bytes() {
  return NST * Stage<BK, BV, GS>::BYTES + ZBUF_BYTES + ZTAB_BYTES;
}
template <int BK, int BV, int GS>
constexpr int pipe_bytes() {
  static_assert(MMA_WARPS * warp_bytes<BK, BV, GS>() >= MERGE_BYTES, "the merge buffer aliases the stages");
  return MMA_WARPS * warp_bytes<BK, BV, GS>();
}

// ---------------------------------------------------------------------------
// window path: plain fp32 over 16-bit tokens [t0, t1); warp w takes tokens
// t0 + w, t0 + w + 4, ... four at a time.  The loads of q and of the first four
// tokens are issued by window_preload (before the packed stream's copies are
// queued), later rounds load one round ahead.  Each warp leaves its state
// (acc, m, l per head) in `ws`.
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
    const int t = tb + i * MMA_WARPS;
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
  for (int tb = t0 + warp; tb < t1; tb += 4 * MMA_WARPS) {
    uint2 kn[4], vn[4];
    window_load_round(p, tb + 4 * MMA_WARPS, t1, hk, b, kn, vn);  // next round, in flight during this one
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (tb + i * MMA_WARPS < t1) {
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

// ---------------------------------------------------------------------------
// window tiles on the tensor cores: 16 tokens of the 16-bit window are staged
// row by row (rows padded to WROW bytes against bank conflicts) and enter the
// same softmax state as the packed units, as bf16 operands.
// ---------------------------------------------------------------------------
constexpr int WROW = 2 * HD + 16;        // bytes per staged window row
constexpr int WIN_BYTES = 2 * 16 * WROW;  // 16 key rows, then 16 value rows

__device__ __forceinline__ void mma16816_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// One warp stages window tokens [tb, tb + 16) (rows at or beyond t1 are zero-filled); no commit.
__device__ __forceinline__ void window_stage(const DecodeParams& p, int tb, int t1, int hk, int b, uint32_t wbuf, int lane) {
  const Dims& dm = p.dm;
  const size_t row0 = (size_t)(b * dm.Hkv + hk) * dm.R;
  const uint8_t* wk = reinterpret_cast<const uint8_t*>(p.L.win_k);
  const uint8_t* wv = reinterpret_cast<const uint8_t*>(p.L.win_v);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int chunk = lane + 32 * i, row = chunk >> 4, c = chunk & 15;
    const uint32_t dk = wbuf + row * WROW + c * 16, dv = dk + 16 * WROW;
    if (tb + row < t1) {
      const size_t off = (row0 + tb + row) * (2 * HD) + c * 16;
      if (p.K_new != nullptr && tb + row == p.r - 1) {  // the token of this step: not in the window yet
        const size_t noff = (size_t)(b * dm.Hkv + hk) * (2 * HD) + c * 16;
        cp_async16(dk, reinterpret_cast<const uint8_t*>(p.K_new) + noff);
        cp_async16(dv, reinterpret_cast<const uint8_t*>(p.V_new) + noff);
      } else {
        cp_async16(dk, wk + off);
        cp_async16(dv, wv + off);
      }
    } else {
      asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};\n" ::"r"(dk), "r"(0u) : "memory");
      asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};\n" ::"r"(dv), "r"(0u) : "memory");
    }
  }
}

// Fused append: the staged tile [tb, tb + 16) holds the token of this step (row r - 1); one warp stores it into
// the window, keys by lanes 0..15, values by lanes 16..31.
__device__ __forceinline__ void window_store_new(const DecodeParams& p, int tb, int hk, int b, uint32_t wbuf, int lane) {
  const Dims& dm = p.dm;
  const int row = p.r - 1 - tb, c = lane & 15;
  const uint4 v = lds128(wbuf + (lane >> 4) * 16 * WROW + row * WROW + c * 16);
  uint8_t* win = reinterpret_cast<uint8_t*>(lane < 16 ? p.L.win_k : p.L.win_v);
  *reinterpret_cast<uint4*>(win + ((size_t)(b * dm.Hkv + hk) * dm.R + (p.r - 1)) * (2 * HD) + c * 16) = v;
}

// One warp folds the staged tile (n_valid of its 16 tokens exist) into its softmax state.  accO is kept in true
// units here (the caller applies the slot weights of the packed path once all window tiles are in).
// qb: q of head gid as bf16 pairs in B-operand order (as loaded), scale2: softmax scale in log2 units.
template <bool SP>
__device__ __forceinline__ void window_tile(uint32_t wbuf, int n_valid, const uint32_t (&qb)[16], float scale2,
                                            float (&accO)[8][4], float (&accZ)[4], float& m0, float& m1, int lane) {
  const int gid = lane >> 2;
  float s[4] = {0.f, 0.f, 0.f, 0.f};  // rows = tokens gid, gid + 8; cols = heads 2 tig, 2 tig + 1
  const uint32_t ka = wbuf + ((lane & 7) + 8 * ((lane >> 3) & 1)) * WROW + (lane >> 4) * 16;
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    uint32_t a0, a1, a2, a3;
    ldmatrix_x4(ka + ks * 32, a0, a1, a2, a3);
    mma16816_bf16(s, a0, a1, a2, a3, qb[2 * ks], qb[2 * ks + 1]);
  }
  const bool va = gid < n_valid, vb = gid + 8 < n_valid;
  // SP: the odd columns are padding (q = 0 there): they keep reference 0 and numerators 0
  const float x00 = va ? s[0] * scale2 : -CUDART_INF_F, x01 = SP ? 0.f : (va ? s[1] * scale2 : -CUDART_INF_F);
  const float x10 = vb ? s[2] * scale2 : -CUDART_INF_F, x11 = SP ? 0.f : (vb ? s[3] * scale2 : -CUDART_INF_F);
  float r0 = fmaxf(x00, x10), r1 = fmaxf(x01, x11);
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    r0 = fmaxf(r0, __shfl_xor_sync(0xffffffffu, r0, o));
    if (!SP) r1 = fmaxf(r1, __shfl_xor_sync(0xffffffffu, r1, o));
  }
  const float mn0 = fmaxf(m0, r0), mn1 = SP ? m1 : fmaxf(m1, r1);  // finite: token 0 of the tile exists
  const float f0 = ex2(m0 - mn0), f1 = SP ? 1.f : ex2(m1 - mn1);
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    accO[mt][0] *= f0; accO[mt][2] *= f0;
    if (!SP) { accO[mt][1] *= f1; accO[mt][3] *= f1; }
  }
  accZ[0] *= f0; accZ[2] *= f0;
  if (!SP) { accZ[1] *= f1; accZ[3] *= f1; }
  m0 = mn0; m1 = mn1;
  const float p00 = ex2(x00 - m0), p10 = ex2(x10 - m0);
  const float p01 = SP ? 0.f : ex2(x01 - m1), p11 = SP ? 0.f : ex2(x11 - m1);
  // numerators as bf16 hi + lo (16 bits of precision), transposed into B-operand order
  const uint32_t h0 = pack_bf16x2(p00, p01), h1 = pack_bf16x2(p10, p11);
  const uint32_t l0 = pack_bf16x2(p00 - bf16_to_f(h0 & 0xffff), p01 - bf16_to_f(h0 >> 16));
  const uint32_t l1 = pack_bf16x2(p10 - bf16_to_f(h1 & 0xffff), p11 - bf16_to_f(h1 >> 16));
  const uint32_t bh0 = movmatrix_trans(h0), bh1 = movmatrix_trans(h1), bl0 = movmatrix_trans(l0), bl1 = movmatrix_trans(l1);
  const uint32_t ones = (gid == 0) ? 0x3F803F80u : 0u;  // row 8 of the sums tile: sum_t p_t
  mma16816_bf16(accZ, 0u, ones, 0u, ones, bh0, bh1);
  mma16816_bf16(accZ, 0u, ones, 0u, ones, bl0, bl1);
  // O^T += V^T P: A fragments are transposed 8x8 blocks of the row-major value rows
  const int mi = lane >> 3;
  const uint32_t va_addr = wbuf + 16 * WROW + ((lane & 7) + 8 * (mi >> 1)) * WROW + (mi & 1) * 16;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    uint32_t a0, a1, a2, a3;
    ldmatrix_x4_trans(va_addr + mt * 32, a0, a1, a2, a3);
    mma16816_bf16(accO[mt], a0, a1, a2, a3, bh0, bh1);
    mma16816_bf16(accO[mt], a0, a1, a2, a3, bl0, bl1);
  }
}

// Combines warp states (rows of MS floats: mb has 8 rows per warp, ws has G rows
// per warp; either may be absent) and writes the CTA's partial for each head.
__device__ __forceinline__ void write_partial(const DecodeParams& p, const float* mb, const float* ws, int split,
                                              int stride, int hk, int b) {
  const Dims& dm = p.dm;
  const int d = threadIdx.x;  // MMA_THREADS == HD
  const int G = dm.G;
  for (int a = 0; a < G; ++a) {
    float M = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < MMA_WARPS; ++w) {
      if (mb) M = fmaxf(M, mb[(w * 8 + a) * MS + HD]);
      if (ws) M = fmaxf(M, ws[(w * G + a) * MS + HD]);
    }
    float Lsum = 0.f, A = 0.f;
#pragma unroll
    for (int w = 0; w < MMA_WARPS; ++w) {
      if (mb) {
        const float* row = mb + (w * 8 + a) * MS;
        float f = ex2(row[HD] - M);  // 2^-inf = 0 for an empty state; M is finite whenever any state is not empty
        Lsum = fmaf(row[HD + 1], f, Lsum);
        A = fmaf(row[d], f, A);
      }
      if (ws) {
        const float* row = ws + (w * G + a) * MS;
        float f = ex2(row[HD] - M);
        Lsum = fmaf(row[HD + 1], f, Lsum);
        A = fmaf(row[d], f, A);
      }
    }
    size_t hq = (size_t)b * dm.Hq + hk * G + a;
    p.part_acc[(hq * stride + split) * HD + d] = A;
    if (d == 0) *reinterpret_cast<float2*>(p.part_ml + (hq * stride + split) * 2) = make_float2(M, Lsum);
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
__device__ __forceinline__ void ticket_merge(const DecodeParams& p, int ns, int stride, int hk, int b, int* s_flag) {
  const Dims& dm = p.dm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = b * dm.Hkv + hk;
  // The CTA's barrier orders every thread's partial stores before thread 0's ticket; the ticket is a release
  // (cumulative over what the barrier ordered) and an acquire at device scope, so the CTA that draws the last
  // ticket sees all partials after its second barrier.  The partials are then read from L2 (ld.global.cg).
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned t;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;\n" : "=r"(t) : "l"(p.tickets + bh) : "memory");
    *s_flag = (t == (unsigned)(ns - 1));
  }
  __syncthreads();
  if (!*s_flag) return;
  for (int a = warp; a < dm.G; a += MMA_WARPS) {
    const size_t hq = (size_t)b * dm.Hq + hk * dm.G + a;
    const float* ml = p.part_ml + hq * stride * 2;
    const float* pa = p.part_acc + hq * stride * HD + lane * 4;
    // every load of a round is issued before anything waits for one: the merge costs one L2 round trip per 16
    // partials instead of one per partial
    float4 v[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = (i < ns) ? ld_cg4(pa + (size_t)i * HD) : make_float4(0.f, 0.f, 0.f, 0.f);
    float M = -CUDART_INF_F;
    for (int s = lane; s < ns; s += 32) M = fmaxf(M, ld_cg(ml + 2 * s));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float Ls = 0.f;
    for (int s0 = 0; s0 < ns; s0 += 16) {
      if (s0 > 0) {
#pragma unroll
        for (int i = 0; i < 16; ++i)
          v[i] = (s0 + i < ns) ? ld_cg4(pa + (size_t)(s0 + i) * HD) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      float f = 0.f;  // lane i < 16: weight of partial s0 + i
      if (lane < 16 && s0 + lane < ns) {
        f = ex2(ld_cg(ml + 2 * (s0 + lane)) - M);
        Ls = fmaf(ld_cg(ml + 2 * (s0 + lane) + 1), f, Ls);
      }
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float fi = __shfl_sync(0xffffffffu, f, i);
        acc.x = fmaf(v[i].x, fi, acc.x); acc.y = fmaf(v[i].y, fi, acc.y);
        acc.z = fmaf(v[i].z, fi, acc.z); acc.w = fmaf(v[i].w, fi, acc.w);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Ls += __shfl_xor_sync(0xffffffffu, Ls, o);
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

// S^T = Kc (q s)^T for the 32 tokens of the unit staged at `st`:
// accS[mt] rows = tokens 16 mt + gid (+8), cols = heads 2 tig (+1); values carry a factor 2^-24.
// HP (with the spread column layout only): column 2h carries fp16(q_d s_d) of head h and column 2h + 1 what that
// rounding lost, q_d s_d - fp16(q_d s_d) (one fused multiply-add; alpha is 1 in the odd columns and 0 in the even
// ones, where the same instruction reproduces the rounded product).  The caller adds the two columns' sums.
template <int BK, int BV, int GS, bool HP>
__device__ __forceinline__ void unit_logits(uint32_t st, const uint32_t (&qe)[16], uint32_t alpha, float (&accS)[2][4],
                                            int lane, int tig) {
  using St = Stage<BK, BV, GS>;
  uint4 w[2];
  if (BK == 2) {
    w[0] = lds128(st + lane * 16);
    w[1] = lds128(st + 512 + lane * 16);
  } else {
    w[0] = lds128(st + lane * 16);
    w[1] = make_uint4(w[0].x >> 8, w[0].y >> 8, w[0].z >> 8, w[0].w >> 8);
  }
  uint4 wsft[2];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
    wsft[mt] = make_uint4(w[mt].x >> Slots<BK>::SHIFT, w[mt].y >> Slots<BK>::SHIFT, w[mt].z >> Slots<BK>::SHIFT,
                          w[mt].w >> Slots<BK>::SHIFT);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 sv = lds128(st + St::OFF_KS + i * 64 + tig * 16);  // scales of k-steps 2i, 2i+1
    uint32_t bq[4] = {hmul2_u(qe[4 * i + 0], sv.x), hmul2_u(qe[4 * i + 1], sv.y),
                      hmul2_u(qe[4 * i + 2], sv.z), hmul2_u(qe[4 * i + 3], sv.w)};
    if (HP) {
      bq[0] = hfms2_u(qe[4 * i + 0], sv.x, hmul2_u(bq[0], alpha));
      bq[1] = hfms2_u(qe[4 * i + 1], sv.y, hmul2_u(bq[1], alpha));
      bq[2] = hfms2_u(qe[4 * i + 2], sv.z, hmul2_u(bq[2], alpha));
      bq[3] = hfms2_u(qe[4 * i + 3], sv.w, hmul2_u(bq[3], alpha));
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int s = 2 * i + h;
      const uint32_t mk = Slots<BK>::mask(s);
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const uint4& src = Slots<BK>::shifted(s) ? wsft[mt] : w[mt];
        if (s == 0)
          mma16816_z(accS[mt], src.x & mk, src.y & mk, src.z & mk, src.w & mk, bq[2 * h], bq[2 * h + 1]);
        else
          mma16816(accS[mt], src.x & mk, src.y & mk, src.z & mk, src.w & mk, bq[2 * h], bq[2 * h + 1]);
      }
    }
  }
  if (HP) {
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      accS[mt][0] += accS[mt][1];
      accS[mt][2] += accS[mt][3];
    }
  }
}

// O^T += Vc^T (p s) for the unit staged at `st`, plus the zero-point and normaliser sums.
// pb: P as B operand, [16-token tile][b0, b1].
template <int BK, int BV, int GS>
__device__ __forceinline__ void unit_values(uint32_t st, const uint32_t (&pb)[2][2], float (&accO)[8][4],
                                            float (&accZ)[4], int lane, int gid, int tig) {
  using St = Stage<BK, BV, GS>;
  constexpr int NG = St::NG;
  uint4 wv1 = make_uint4(0, 0, 0, 0);
  if (BV == 1) wv1 = lds128(st + St::OFF_VC + lane * 16);
#pragma unroll
  for (int tt = 0; tt < 2; ++tt) {
    const uint32_t vmeta = st + St::OFF_VM + tt * (64 * NG);
    uint32_t sv[2 * NG];
    if (NG == 4) {
      uint4 x0 = lds128(vmeta + tig * 32), x1 = lds128(vmeta + tig * 32 + 16);
      sv[0] = x0.x; sv[1] = x0.y; sv[2] = x0.z; sv[3] = x0.w;
      sv[4 % (2 * NG)] = x1.x; sv[5 % (2 * NG)] = x1.y; sv[6 % (2 * NG)] = x1.z; sv[7 % (2 * NG)] = x1.w;
    } else {
      uint4 x0 = lds128(vmeta + tig * 16);
      sv[0] = x0.x; sv[1] = x0.y; sv[2] = x0.z; sv[3] = x0.w;
    }
    uint32_t za0 = 0, za2 = 0;
    if (gid < NG) {
      uint2 zz = lds64(vmeta + 32 * NG + tig * (8 * NG) + gid * 8);
      za0 = zz.x; za2 = zz.y;
    }
    const uint32_t ones = (gid == 0) ? 0x3C003C00u : 0u;
    mma16816(accZ, za0, ones, za2, ones, pb[tt][0], pb[tt][1]);
    uint32_t pg[NG][2];
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
      pg[gi][0] = hmul2_u(pb[tt][0], sv[2 * gi]);
      pg[gi][1] = hmul2_u(pb[tt][1], sv[2 * gi + 1]);
    }
    uint4 w;
    if (BV == 2) {
      w = lds128(st + St::OFF_VC + tt * 512 + lane * 16);
    } else {
      w = wv1;
      if (tt == 1) { w.x >>= 8; w.y >>= 8; w.z >>= 8; w.w >>= 8; }
    }
    uint4 wsft = make_uint4(w.x >> Slots<BV>::SHIFT, w.y >> Slots<BV>::SHIFT, w.z >> Slots<BV>::SHIFT,
                            w.w >> Slots<BV>::SHIFT);
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const uint32_t mk = Slots<BV>::mask(mt);
      const uint4& src = Slots<BV>::shifted(mt) ? wsft : w;
      const int gi = (16 * mt) / GS;
      mma16816(accO[mt], src.x & mk, src.y & mk, src.z & mk, src.w & mk, pg[gi][0], pg[gi][1]);
    }
  }
}

// ---------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------
// SP ("spread"): groups of at most 4 query heads put head h in column 2h of the N = 8 tiles and leave the odd
// columns as padding, so that each thread's accumulator pairs hold one real head: half the softmax work.
// HP: q_d s_d as an fp16 pair in the two columns of a head (see unit_logits); needs SP.
template <int BK, int BV, int GS, bool SP, bool HP>
__global__ void __launch_bounds__(MMA_THREADS, 3) decode_mma_kernel(DecodeParams p) {
  static_assert(SP || !HP, "the residual column is the padding column of the spread layout");
  using St = Stage<BK, BV, GS>;
  constexpr int NG = St::NG;
  constexpr int WARP_BYTES = warp_bytes<BK, BV, GS>();
  constexpr int PIPE = pipe_bytes<BK, BV, GS>();
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ int s_flag;
  float* mb = reinterpret_cast<float*>(smem);                   // merge buffer (after the loop)
  uint32_t* q_sm = reinterpret_cast<uint32_t*>(smem + PIPE);     // [4 chunks][lane][4] half2
  float* ws = reinterpret_cast<float*>(smem);                  // window states of the window-only path

  const Dims& dm = p.dm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int G = dm.G;

  if (p.ns_q == 0) {  // nothing is quantized yet: window-only splits, grid (splits, kv heads, sequences)
    grid_dependents_go();
    grid_dependency_wait();
    const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int ns = p.ns_w;
    const int tiles = (p.r + 15) / 16;
    int t0, t1;
    share_of(tiles, ns, split, t0, t1);
    t0 *= 16;
    t1 = min(t1 * 16, p.r);
    WindowRegs wr;
    window_preload(p, t0, t1, hk, b, wr);
    window_tokens(p, t0, t1, hk, b, ws, wr);
    __syncthreads();
    write_partial(p, nullptr, ws, split, ns, hk, b);
    ticket_merge(p, ns, ns, hk, b, &s_flag);
    return;
  }

  // Packed path: a one-dimensional grid of p.n_ctas CTAs dealt to the streams in order; the first
  // n_ctas % streams streams get one split more than the others (the host only chooses such a count when the
  // splits are many, so the CTAs' sizes differ by a few percent), which lets the grid fill every resident slot.
  int split, ns, hk, b;
  {
    const unsigned n_streams = (unsigned)(dm.B * dm.Hkv), c = blockIdx.x;
    const unsigned base = (unsigned)p.n_ctas / n_streams, rem = (unsigned)p.n_ctas - base * n_streams;
    const unsigned big = rem * (base + 1u);
    unsigned stream;
    if (c < big) {
      stream = c / (base + 1u);
      split = (int)(c - stream * (base + 1u));
      ns = (int)base + 1;
    } else {
      const unsigned c2 = c - big;
      stream = rem + c2 / base;
      split = (int)(c2 - (c2 / base) * base);
      ns = (int)base;
    }
    hk = (int)(stream % (unsigned)dm.Hkv);
    b = (int)(stream / (unsigned)dm.Hkv);
  }
  const int units = p.n_q / 32;
  int u0, u1;
  share_of(units, ns, split, u0, u1);
  const int n_cta = u1 - u0;
  const int uw = u0 + (warp * n_cta) / MMA_WARPS;  // this warp's units: [uw, uw + n_my)
  const int n_my = u0 + ((warp + 1) * n_cta) / MMA_WARPS - uw;
  const int bh = b * dm.Hkv + hk;

  // this lane's 16-byte column of this warp's first unit in the four streams
  const uint8_t* gk = reinterpret_cast<const uint8_t*>(p.L.k_codes) + (size_t)bh * ((size_t)dm.nq_cap * (HD * BK / 8)) +
                      (size_t)uw * St::KC + lane * 16;
  const uint8_t* gv = reinterpret_cast<const uint8_t*>(p.L.v_codes) + (size_t)bh * ((size_t)dm.nq_cap * (HD * BV / 8)) +
                      (size_t)uw * St::VC + lane * 16;
  const uint8_t* gvm = reinterpret_cast<const uint8_t*>(p.L.v_meta) + (size_t)bh * (dm.nq_cap / 16) * (64 * NG) +
                       (size_t)uw * St::VM + lane * 16;
  const size_t plane = (size_t)(dm.nq_cap / GS) * 256;  // bytes of the key scale plane (= of the zero-point plane)
  const uint8_t* gks = reinterpret_cast<const uint8_t*>(p.L.k_meta) + (size_t)bh * 2 * plane + lane * 16;
  const uint8_t* gkz = gks + plane;

  const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(smem);
  const uint32_t my = sm_base + warp * WARP_BYTES;  // this warp's stages
  const uint32_t zbuf = my + NST * St::BYTES;
  const uint32_t ztab = zbuf + ZBUF_BYTES;

  // stage unit jj of this warp at byte offset `soff` of its ring, if it exists (no commit, no branch)
  auto issue_unit = [&](int jj, uint32_t soff) {
    const bool on = jj < n_my;
    const uint32_t s = my + soff + lane * 16;
    const uint8_t* k = gk + (size_t)(uint32_t)jj * St::KC;
    cp_async16_if(s, k, on);
    if (St::KC == 1024) cp_async16_if(s + 512, k + 512, on);
    cp_async16_if(s + St::OFF_KS, gks + (size_t)(uint32_t)(((uw + jj) * 32) / GS) * 256, on && lane < 16);
    const uint8_t* v = gv + (size_t)(uint32_t)jj * St::VC;
    cp_async16_if(s + St::OFF_VC, v, on);
    if (St::VC == 1024) cp_async16_if(s + St::OFF_VC + 512, v + 512, on);
    cp_async16_if(s + St::OFF_VM, gvm + (size_t)(uint32_t)jj * St::VM, on && lane * 16 < St::VM);
  };
  // the same for a unit that is known to exist: no predicates beyond the two lane masks
  auto issue_unit_always = [&](int jj, uint32_t soff) {
    const uint32_t s = my + soff + lane * 16;
    const uint8_t* k = gk + (size_t)(uint32_t)jj * St::KC;
    cp_async16(s, k);
    if (St::KC == 1024) cp_async16(s + 512, k + 512);
    if (lane < 16) cp_async16(s + St::OFF_KS, gks + (size_t)(uint32_t)(((uw + jj) * 32) / GS) * 256);
    const uint8_t* v = gv + (size_t)(uint32_t)jj * St::VC;
    cp_async16(s + St::OFF_VC, v);
    if (St::VC == 1024) cp_async16(s + St::OFF_VC + 512, v + 512);
    if (lane * 16 < St::VM) cp_async16(s + St::OFF_VM, gvm + (size_t)(uint32_t)jj * St::VM);
  };
  // stage the key zero-point rows of the groups of units [jb, jb + ZROWS) (no commit)
  auto issue_zero_rows = [&](int jb) {
    const int rows = min(ZROWS, n_my - jb);
    const int g_first = ((uw + jb) * 32) / GS, g_last = ((uw + jb + rows - 1) * 32) / GS;
    const int bytes = (g_last - g_first + 1) * 256;
    const uint8_t* src = gkz + (size_t)g_first * 256;
#pragma unroll
    for (int i = 0; i < ZBUF_BYTES / 512; ++i)
      if (i * 512 + lane * 16 < bytes) cp_async16(zbuf + i * 512 + lane * 16, src + i * 512);
  };

  // The first units of the packed streams may be on their way while the preceding kernel in the stream (which
  // wrote q and the newest window rows, and whose predecessors may still use the split-K scratch) is finishing:
  // with early_fetch the whole ring is queued before this kernel waits for that one (groups 0, 1, 2 = units 0, 1,
  // 2; the window tile gets a group of its own).  Without it, group 0 holds unit 0, the first zero-point rows and
  // the window tile, and the rest of the ring follows once q is here: a launch-wide burst of three units per warp
  // would sit in the memory queues in front of the q loads.
  const bool early = p.early_fetch != 0;
  grid_dependents_go();
  if (!early) grid_dependency_wait();
  issue_unit(0, 0);
  if (n_my > 0) issue_zero_rows(0);
  if (early) {
    cp_async_commit();
#pragma unroll
    for (int jj = 1; jj < NST - 1; ++jj) {
      issue_unit(jj, jj * St::BYTES);
      cp_async_commit();
    }
    grid_dependency_wait();
  }

  // Loads the prologue waits for go out next: q in B-operand order and the first rows of this split's share of
  // the window.
  int wt0, wt1;
  share_of(p.r, ns, split, wt0, wt1);
  uint32_t raw[16];  // q of head gid: (q[16s + 2tig + 8j], q[16s + 2tig + 8j + 1]), j = 0, 1
  {
    const int hcol = SP ? (gid >> 1) : gid;  // the head of column gid
    const bool real = SP ? ((gid & 1) == 0 && hcol < G) : (gid < G);
    const uint16_t* qp = p.q + ((size_t)b * dm.Hq + hk * G + (real ? hcol : 0)) * HD + 2 * tig;
#pragma unroll
    for (int i = 0; i < 16; ++i) raw[i] = real ? *reinterpret_cast<const uint32_t*>(qp + 16 * (i >> 1) + 8 * (i & 1)) : 0u;
  }
  // the CTA's share of the window, in tiles of 16 tokens, goes to one warp (rotating with the split index)
  const int ww = split & (MMA_WARPS - 1);
  const uint32_t wbuf = sm_base + PIPE + Q_BYTES;
  if (warp == ww && wt0 < wt1) window_stage(p, wt0, wt1, hk, b, wbuf, lane);

  cp_async_commit();  // group 0, or the window tile's group (empty for the other warps)

  const uint32_t alpha = (HP && (gid & 1)) ? 0x3C003C00u : 0u;  // (1, 1) in the residual columns
  uint32_t qe[16];  // q as fp16 B operand, pre-scaled by 2^-e(s), the weight the code's slot carries
#pragma unroll
  for (int s = 0; s < 8; ++s) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      float lo = bf16_to_f(raw[2 * s + j] & 0xffff), hi = bf16_to_f(raw[2 * s + j] >> 16);
      if (warp == 0) q_sm[((s >> 1) * 32 + lane) * 4 + (s & 1) * 2 + j] = pack_half2(lo, hi);
      if (HP) {  // the odd column of a head multiplies the same q (its raw[] stays zero: bias and window use it)
        const uint32_t left = __shfl_up_sync(0xffffffffu, raw[2 * s + j], 4);
        if ((gid & 1) && (gid >> 1) < G) {
          lo = bf16_to_f(left & 0xffff);
          hi = bf16_to_f(left >> 16);
        }
      }
      const float sc = 1.0f / (float)(1 << Slots<BK>::e(s));
      qe[2 * s + j] = pack_half2(lo * sc, hi * sc);
    }
  }
  __syncthreads();
  if (!early) {  // q is here: the rest of the ring (group jj holds unit jj)
#pragma unroll
    for (int jj = 1; jj < NST - 1; ++jj) {
      issue_unit(jj, jj * St::BYTES);
      cp_async_commit();
    }
  }

  const float scale2 = p.scale * 1.4426950408889634f;
  const float c1 = scale2 * 16777216.0f;  // undoes the 2^-24 of the subnormal code operand
  float accO[8][4];                        // O^T: rows = channels 16 mt + gid (+8), cols = heads 2 tig (+1)
  float accZ[4] = {0.f, 0.f, 0.f, 0.f};    // rows 0..NG-1: sum_t p_t z_tg ; row 8: sum_t p_t
#pragma unroll
  for (int mt = 0; mt < 8; ++mt)
#pragma unroll
    for (int i = 0; i < 4; ++i) accO[mt][i] = 0.f;
  // softmax reference (log2 units) of columns 2 tig, 2 tig + 1 (SP: the odd column is padding, reference 0)
  float m0 = -CUDART_INF_F, m1 = SP ? 0.f : -CUDART_INF_F;
  float accS[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};

  // unit 0, the first zero-point rows and (for its warp) the first window tile have landed
  if (!early)
    cp_async_wait<NST - 2>();
  else if (warp == ww && wt0 < wt1)
    cp_async_wait<0>();
  else
    cp_async_wait<NST - 1>();
  __syncwarp();
  if (warp == ww && wt0 < wt1) {
    // window tokens first (the accumulators are empty): true units, then the slot weights of the packed path
    for (int tb = wt0; tb < wt1; tb += 16) {
      if (tb > wt0) {  // a share of more than 16 tokens (few splits): stage the next tile and wait for it
        __syncwarp();
        window_stage(p, tb, wt1, hk, b, wbuf, lane);
        cp_async_commit();
        cp_async_wait<0>();
        __syncwarp();
      }
      if (p.K_new != nullptr && tb + 16 > p.r - 1 && wt1 == p.r) window_store_new(p, tb, hk, b, wbuf, lane);
      window_tile<SP>(wbuf, wt1 - tb, raw, scale2, accO, accZ, m0, m1, lane);
    }
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const float wgt = 1.0f / (float)(1u << (24 - Slots<BV>::e(mt)));
#pragma unroll
      for (int i = 0; i < 4; ++i) accO[mt][i] *= wgt;
    }
  }
  if (n_my > 0) unit_logits<BK, BV, GS, HP>(my, qe, alpha, accS, lane, tig);

  // One iteration: bias table every ZROWS units, refill of the stage unit j - 1 used, softmax reference,
  // numerators of unit j, then (MORE) logits of unit j + 1 next to the value product of unit j.
  // off_prev / off_cur / off_next: ring offsets of the stages of units j - 1 (free, refilled), j and j + 1.
  // refill: unit j + NST - 1 exists (then so does unit j + 1, and `more` is true)
  auto step = [&](auto refill, int j, bool more, uint32_t off_prev, uint32_t off_cur, uint32_t off_next) {
    const int jr = j & (ZROWS - 1);
    if (jr == 0) {
      // bias table of units [j, j + 16): ztab[row][head] = scale * sum_d q_d z_d (log2 units)
      const int rows = min(ZROWS, n_my - j);
      const int g_first = ((uw + j) * 32) / GS;
      const int ra_row = ((uw + j + min(gid, rows - 1)) * 32) / GS - g_first;
      const int rb_row = ((uw + j + min(gid + 8, rows - 1)) * 32) / GS - g_first;
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint4 ra = lds128(zbuf + ra_row * 256 + i * 64 + tig * 16);
        const uint4 rb = lds128(zbuf + rb_row * 256 + i * 64 + tig * 16);
        const uint4 qq = *reinterpret_cast<const uint4*>(q_sm + (i * 32 + lane) * 4);  // k-steps 2i, 2i+1
        mma16816(acc, ra.x, rb.x, ra.y, rb.y, qq.x, qq.y);
        mma16816(acc, ra.z, rb.z, ra.w, rb.w, qq.z, qq.w);
      }
      sts64f(ztab + gid * 32 + tig * 8, acc[0] * scale2, acc[1] * scale2);
      sts64f(ztab + (gid + 8) * 32 + tig * 8, acc[2] * scale2, acc[3] * scale2);
      __syncwarp();  // table visible; every lane is done with the rows
      if (j + ZROWS < n_my) issue_zero_rows(j + ZROWS);  // lands with this iteration's group, 16 units early
    }

    __syncwarp();  // every lane is done with the stage of unit j - 1
    if (decltype(refill)::value) issue_unit_always(j + NST - 1, off_prev);
    cp_async_commit();  // (an empty group once the stream's end is near: the waits below count groups)

    // ---- softmax reference: raise it only when a logit of unit j exceeds it by more than TAU ----
    const float2 bz = lds64f(ztab + jr * 32 + tig * 8);
    {
      const float lm0 = fmaxf(fmaxf(accS[0][0], accS[0][2]), fmaxf(accS[1][0], accS[1][2]));
      const float lm1 = SP ? 0.f : fmaxf(fmaxf(accS[0][1], accS[0][3]), fmaxf(accS[1][1], accS[1][3]));
      float x0 = fmaf(lm0, c1, bz.x), x1 = SP ? 0.f : fmaf(lm1, c1, bz.y);
      if (__any_sync(0xffffffffu, SP ? (x0 > m0 + TAU) : ((x0 > m0 + TAU) | (x1 > m1 + TAU)))) {
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
          x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, o));
          if (!SP) x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, o));
        }
        const float mn0 = fmaxf(m0, x0), mn1 = SP ? m1 : fmaxf(m1, x1);
        const float f0 = ex2(m0 - mn0), f1 = SP ? 1.f : ex2(m1 - mn1);
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          accO[mt][0] *= f0; accO[mt][2] *= f0;
          if (!SP) { accO[mt][1] *= f1; accO[mt][3] *= f1; }
        }
        accZ[0] *= f0; accZ[2] *= f0;
        if (!SP) { accZ[1] *= f1; accZ[3] *= f1; }
        m0 = mn0; m1 = mn1;
      }
    }

    cp_async_wait<NST - 2>();  // unit j + 1 has landed
    __syncwarp();

    // ---- softmax numerators of unit j (log2 domain; the unit's key bias is common to its 32 tokens) ----
    const float t0 = bz.x - m0, t1 = bz.y - m1;
    uint32_t pb[2][2];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      float p0 = ex2(fmaf(accS[mt][0], c1, t0)), p1 = SP ? 0.f : ex2(fmaf(accS[mt][1], c1, t1));
      float p2 = ex2(fmaf(accS[mt][2], c1, t0)), p3 = SP ? 0.f : ex2(fmaf(accS[mt][3], c1, t1));
      pb[mt][0] = movmatrix_trans(pack_half2(p0, p1));
      pb[mt][1] = movmatrix_trans(pack_half2(p2, p3));
    }
    if (more) unit_logits<BK, BV, GS, HP>(my + off_next, qe, alpha, accS, lane, tig);
    unit_values<BK, BV, GS>(my + off_cur, pb, accO, accZ, lane, gid, tig);
  };

  // main loop: two copies of the body, one that refills and one that does not (four unrolled copies with constant
  // stage offsets save address arithmetic but cost more in instruction-cache misses than they save)
  static_assert(NST == 4, "ring of four stages");
  int j = 0;
#pragma unroll 1
  for (; j + NST - 1 < n_my; ++j)  // steady state: every refill exists
    step(std::true_type{}, j, true, ((j + 3) & 3) * St::BYTES, (j & 3) * St::BYTES, ((j + 1) & 3) * St::BYTES);
#pragma unroll 1
  for (; j < n_my; ++j)  // the last NST - 1 units: nothing left to fetch; the very last unit has no successor
    step(std::false_type{}, j, j + 1 < n_my, ((j + 3) & 3) * St::BYTES, (j & 3) * St::BYTES, ((j + 1) & 3) * St::BYTES);
  cp_async_wait<0>();
  __syncthreads();  // all warps are done with their stages: the memory becomes the merge buffer

  // ---- epilogue: undo slot weights, add the zero-point sums, hand the state to the merge buffer ----
  const float l0 = __shfl_sync(0xffffffffu, accZ[2], tig), l1 = __shfl_sync(0xffffffffu, accZ[3], tig);
  float* mine = mb + (size_t)warp * 8 * MS;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    const int gi = (16 * mt) / GS;
    const float z0 = __shfl_sync(0xffffffffu, accZ[0], 4 * gi + tig), z1 = __shfl_sync(0xffffffffu, accZ[1], 4 * gi + tig);
    const float wgt = (float)(1u << (24 - Slots<BV>::e(mt)));
    const int ch = 16 * mt + gid;
    const int h0 = SP ? tig : 2 * tig;  // the head of this thread's even column
    if (h0 < G) {
      float* row = mine + h0 * MS;
      row[ch] = fmaf(accO[mt][0], wgt, z0);
      row[ch + 8] = fmaf(accO[mt][2], wgt, z0);
    }
    if (!SP && 2 * tig + 1 < G) {
      float* row = mine + (2 * tig + 1) * MS;
      row[ch] = fmaf(accO[mt][1], wgt, z1);
      row[ch + 8] = fmaf(accO[mt][3], wgt, z1);
    }
  }
  if (gid == 0) {
    const int h0 = SP ? tig : 2 * tig;
    if (h0 < G) {
      mine[h0 * MS + HD] = m0;
      mine[h0 * MS + HD + 1] = l0;
    }
    if (!SP && 2 * tig + 1 < G) {
      mine[(2 * tig + 1) * MS + HD] = m1;
      mine[(2 * tig + 1) * MS + HD + 1] = l1;
    }
  }
  __syncthreads();
  write_partial(p, mb, nullptr, split, p.ns_q, hk, b);
  ticket_merge(p, ns, p.ns_q, hk, b, &s_flag);
}

template <int BK, int BV, int GS>
int smem_bytes(int G) {
  (void)G;
  return pipe_bytes<BK, BV, GS>() + Q_BYTES + WIN_BYTES;
}

template <int BK, int BV, int GS, bool SP, bool HP>
cudaError_t launch_sp(const DecodeParams& p, cudaStream_t st) {
  const int smem = smem_bytes<BK, BV, GS>(p.dm.G);
  static int configured = 0;
  if (configured < smem) {
    cudaError_t e = cudaFuncSetAttribute(decode_mma_kernel<BK, BV, GS, SP, HP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  const dim3 grid = p.ns_q > 0 ? dim3(p.n_ctas) : dim3(p.ns_w, p.dm.Hkv, p.dm.B);
  return launch_dependent(decode_mma_kernel<BK, BV, GS, SP, HP>, grid, dim3(MMA_THREADS), (size_t)smem, st, p);
}

template <int BK, int BV, int GS>
cudaError_t launch_t(const DecodeParams& p, cudaStream_t st) {
  if (p.dm.G > 4) return p.precise ? cudaErrorInvalidValue : launch_sp<BK, BV, GS, false, false>(p, st);
  return p.precise ? launch_sp<BK, BV, GS, true, true>(p, st) : launch_sp<BK, BV, GS, true, false>(p, st);
}

template <int BK, int BV, int GS, bool SP, bool HP>
int ctas_per_sm_sp(int G) {
  const int smem = smem_bytes<BK, BV, GS>(G);
  if (cudaFuncSetAttribute(decode_mma_kernel<BK, BV, GS, SP, HP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=
      cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_mma_kernel<BK, BV, GS, SP, HP>, MMA_THREADS, smem) !=
      cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

template <int BK, int BV, int GS>
int ctas_per_sm_t(int G) {
  return G <= 4 ? ctas_per_sm_sp<BK, BV, GS, true, false>(G) : ctas_per_sm_sp<BK, BV, GS, false, false>(G);
}

}  // namespace

bool decode_mma_supported(const Dims& dm, int bk, int bv) {
  (void)bk; (void)bv;
  return dm.D == HD && dm.G <= 8 && (dm.g == 32 || dm.g == 64);
}

#define XQ_DISPATCH(FN, ...)                    \
  switch (bk * 100 + bv * 10 + (g == 64)) {     \
    case 220: return FN<2, 2, 32>(__VA_ARGS__); \
    case 221: return FN<2, 2, 64>(__VA_ARGS__); \
    case 210: return FN<2, 1, 32>(__VA_ARGS__); \
    case 211: return FN<2, 1, 64>(__VA_ARGS__); \
    case 120: return FN<1, 2, 32>(__VA_ARGS__); \
    case 121: return FN<1, 2, 64>(__VA_ARGS__); \
    case 110: return FN<1, 1, 32>(__VA_ARGS__); \
    case 111: return FN<1, 1, 64>(__VA_ARGS__); \
  }

// Resident CTAs per SM of the kernel variant for these bit-widths (0 if unknown: no device).
int decode_mma_ctas_per_sm(const Dims& dm, int bk, int bv) {
  const int g = dm.g;
  XQ_DISPATCH(ctas_per_sm_t, dm.G)
  return 0;
}

cudaError_t launch_decode_mma(const DecodeParams& p, cudaStream_t st) {
  const int bk = p.L.bk, bv = p.L.bv, g = p.dm.g;
  XQ_DISPATCH(launch_t, p, st)
  return cudaErrorInvalidValue;
}

}  // namespace xq
