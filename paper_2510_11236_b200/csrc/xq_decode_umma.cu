// Tensor-core decode attention over the packed cache (head_dim 128, up to 8
// query heads per kv head): tcgen05.mma kind::i8 with the code matrices in
// tensor memory.
//
// Why integers.  The packed cache delivers ~1.8e13 quantized elements/s at the
// HBM roofline, so a code may cost a quarter of an ALU instruction and no trip
// through shared memory in expanded form.  Four codes of a row sit at one bit
// offset of the four bytes of a packed word, so `word & mask` is four unsigned
// 8-bit operand elements at once; every thread owns one row of the A operand
// (a token's channels for the keys, a channel's tokens for the values), expands
// it with one AND per four codes and writes it to its lane of tensor memory
// (tcgen05.st).  Scale and zero-point are folded out of the inner products,
//
//   q . k_hat_t = sum_d (q_d s_d) c_td + sum_d q_d z_d        (keys, per channel)
//   sum_t p_t v_hat_td = sum_t (p_t s_tg) c_td + sum_t p_t z_tg  (values, per token)
//
// and the other operand (q_d s_d, or p_t s_tg) goes to shared memory as 24-bit
// fixed point: one fused multiply-add with the constant 2^23 (+ an offset for
// signed values) leaves the rounded integer in the low three bytes of the fp32
// result, which are stored as they are -- three operand columns (weights 1, 2^8,
// 2^16) and a constant fourth column (0x4B) whose product gives the row sum that
// removes the offset.  The s32 accumulators are exact; the columns are recombined
// with shifts and adds (keys, per token) or once per CTA in fp32 (values).
//
// One CTA walks a range of 128-token batches of one (sequence, kv head):
//   keys:    A_K[128 tokens x 128 channels],  B_K[channel x (token group, head, byte)]
//            S[token][(group, head, byte)]: a token reads the columns of its own group (its warp's);
//   values:  A_V[128 channels x 128 tokens],  B_V[token x (channel group, head, byte)]
//            O[channel][(channel group, head, byte)] accumulates over all batches in tensor memory.
// Warps: the compute warps (thread = tensor-memory lane; four, or two teams of four that split the heads and
// the columns of every expansion -- measured slower, kept as a template parameter), one warp that folds the
// CTA's share of the 16-bit window (bf16 or f16 mma.sync over 16-token tiles), one that turns the staged key
// zero-points into the logit biases sigma * sum_d q_d z_d (one row of mma.sync products per batch), and one that
// issues the bulk copies of the stage ring (cp.async.bulk + mbarrier transaction counts) and, from one elected
// lane, the matrix products.  The loop is software-pipelined: while the tensor core multiplies the keys of batch
// i + 1, the compute warps run the softmax of batch i and expand its values.  Softmax keeps one integer reference
// per head for the whole team, raised only when a logit exceeds it by more than TAU; the value scales are
// normalised by a power of two per channel group, raised the same way; raising either rescales O in tensor
// memory (rare).  Split-K partials are merged by the last CTA of a stream (atomic ticket; nobody waits for
// another CTA).
//
// What bounds it (32k context, four heads per kv head): tensor memory holds two CTAs per SM (64 + 3 * 64 columns
// each), and a batch takes a CTA about 1600 cycles whether or not it shares its SM.  That time is the latency of
// the compute warps' own instruction chain (expand keys ~190 cycles, B_K ~270, read S ~130, logits and the team's
// vote ~250, exponentials and sums ~70, B_V and expand values ~290) plus 100 to 200 cycles for every hand-over on
// it (a wait on an mbarrier, tcgen05.wait, proxy fence and arrive); the SM's units are far from busy (issue slots
// 40 %, tensor pipe 20 %, DRAM 25 %).  So the loop keeps the hand-overs few: the bias barrier of a batch also
// stands for the arrival of its stage, one wait for S of batch i + 1 also covers the value products of batch i - 1
// (a commit covers everything its thread issued before), and a wait first tests its barrier without suspending
// (most are complete by then).  A raise of the references costs ~1200 cycles, so a raised reference leaves three
// units of room.  A CTA lives ~31 us for ~25 us of loop; consecutive launches of a decode step overlap
// (late_wait), so the next launch's CTAs take the slots as this one's leave.
// Variants built and measured on that shape, per launch, back to back (the kept loop: 40 us before the hand-overs
// were thinned out, 34.4 us now): two teams of four compute warps 50 us; separate expansion and softmax warps with
// their own hand-overs 50 us; the last arriving compute warp issuing the products itself 63 us (a tcgen05.mma
// costs its issuing thread ~50 cycles); every load of an iteration issued at its top with the team's vote cast
// early and read late 46 us; four (72 registers) or three (80) CTAs per SM for a single head per kv head 45 us
// and 44 us against 36 us with two; one S buffer read before the keys are handed over, with two buffers for A_V
// and B_V instead, 42.5 us; polling warps that sleep between polls: no change; polling warps that never suspend:
// 0.7 us slower (they take issue slots from the compute warp of their sub-partition); B_K and the logit scales of
// all four groups written a batch ahead by the bias warp (two B_K buffers) 42 us, only the groups' exponents and
// logit scales from the bias warp: 1.3 us slower; the team's votes cast a batch ahead through an mbarrier instead
// of the hardware barrier (logits of batch i + 1 at the end of iteration i) 42.6 us; a warp of its own for the
// bulk copies: no change; the first copies, or q, fetched before the tensor-memory allocation: no change; the
// four bulk copies of a batch issued from four lanes instead of one: 40.5 us.
// For one head per kv head at 4k context (27.5 us with two CTAs per SM): three CTAs per SM at 96 registers, no
// spills, 41.5 us -- a third chain on an SM slows all three.
//
// Every wait on an mbarrier is bounded: a thread that gives up sets the status
// word in global memory and a flag in shared memory that makes every other wait
// of the CTA give up too; the CTA then frees its tensor memory and leaves
// without writing a result.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <math_constants.h>

#include "xq_internal.h"

namespace xq {

namespace {

constexpr int HD = 128;
constexpr int BT = 128;          // tokens per batch
constexpr int NSTG = 4;          // staged batches
constexpr int TAU = 3;           // log2 units a logit may exceed the softmax reference before it is raised
constexpr int MREF = 0;           // a raised reference is the largest logit rounded up: three more units before the next raise
constexpr int FRAC_V = 23 - TAU; // fraction bits of the value-side fixed point
constexpr int WAIT_LIMIT = 1 << 20;     // polls of a wait before it gives up
constexpr uint32_t WAIT_HINT_NS = 10000;  // longest suspension of one poll (it ends at once when the phase completes)
constexpr float MAGIC_V = 8388608.0f;              // 2^23: x + MAGIC_V holds rint(x) in its mantissa, 0 <= x < 2^23
constexpr float MAGIC_K = 8388608.0f + 1228800.0f;  // offset 75 * 2^14: signed x, |x| <= 2^20
constexpr int MS = HD + 4;       // state row: acc[HD], m, l, padding

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float bf16_to_f(uint32_t u16) { return __uint_as_float(u16 << 16); }
__device__ __forceinline__ float f16_to_f(uint32_t u16) { return __half2float(__ushort_as_half((unsigned short)u16)); }
// an element of q: IEEE half precision or bfloat16
__device__ __forceinline__ float io_to_f(uint32_t u16, int f16) { return f16 ? f16_to_f(u16) : bf16_to_f(u16); }
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
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void sts64(uint32_t a, uint32_t x, uint32_t y) {
  asm volatile("st.shared.v2.u32 [%0], {%1,%2};\n" ::"r"(a), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t x) {
  asm volatile("st.shared.u32 [%0], %1;\n" ::"r"(a), "r"(x) : "memory");
}
__device__ __forceinline__ int redux_max_s32(int v) {
  int r;
  asm volatile("redux.sync.max.s32 %0, %1, 0xffffffff;\n" : "=r"(r) : "r"(v));
  return r;
}
__device__ __forceinline__ uint32_t redux_max_u32(uint32_t v) {
  uint32_t r;
  asm volatile("redux.sync.max.u32 %0, %1, 0xffffffff;\n" : "=r"(r) : "r"(v));
  return r;
}
__device__ __forceinline__ int redux_add_s32(int v) {
  int r;
  asm volatile("redux.sync.add.s32 %0, %1, 0xffffffff;\n" : "=r"(r) : "r"(v));
  return r;
}
// float -> int whose signed order is the float order (finite values and infinities)
__device__ __forceinline__ int float_key(float x) {
  const int b = __float_as_int(x);
  return b ^ ((b >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float key_float(int k) { return __int_as_float(k ^ ((k >> 31) & 0x7fffffff)); }
// 2^e as a float, e clamped to the normal range
__device__ __forceinline__ float pow2i(int e) {
  e = max(-126, min(127, e));
  return __int_as_float((e + 127) << 23);
}
// floor(log2 x) of a positive normal float (its exponent)
__device__ __forceinline__ int exponent_of(float x) { return (int)((__float_as_uint(x) >> 23) & 0xffu) - 127; }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// Bounded wait; gives up as well when another thread of the CTA has (dead flag in shared memory).
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* dead) {
  if (mbar_test_wait(bar, parity)) return true;  // the usual case on the loop's path: already complete
  for (int i = 0; i < WAIT_LIMIT; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*dead) return false;
  }
  *dead = 1;
  return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
// global -> shared bulk copy (16-byte aligned, size a multiple of 16) that reports to an mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// barriers of a team of 128 compute threads (hardware barrier `id` >= 1; barrier 0 is __syncthreads of the whole CTA)
__device__ __forceinline__ void bar_sync_team(uint32_t id) { asm volatile("bar.sync %0, 128;\n" ::"r"(id) : "memory"); }
__device__ __forceinline__ void bar_sync_compute() { bar_sync_team(1); }
__device__ __forceinline__ bool bar_or_team(uint32_t id, bool v) {
  uint32_t r;
  asm volatile(
      "{\n.reg .pred p, q;\nsetp.ne.b32 p, %2, 0;\nbar.red.or.pred q, %1, 128, p;\nselp.u32 %0, 1, 0, q;\n}\n"
      : "=r"(r) : "r"(id), "r"((int)v) : "memory");
  return r != 0;
}
// running count in shared memory; release of what this thread (and, through __syncwarp, its warp) wrote before,
// acquire of what the earlier arrivals released
__device__ __forceinline__ unsigned atom_add_acq_rel(unsigned int* counter) {
  unsigned old;
  asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], 1;\n"
               : "=r"(old) : "r"((uint32_t)__cvta_generic_to_shared(counter)) : "memory");
  return old;
}
__device__ __forceinline__ uint32_t elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred P;\nelect.sync _|P, 0xffffffff;\nselp.u32 %0, 1, 0, P;\n}\n" : "=r"(pred));
  return pred;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
// NC (16 or 32) consecutive columns of this thread's lane
template <int NC>
__device__ __forceinline__ void tmem_st_cols(uint32_t taddr, const uint32_t (&r)[NC]) {
  if constexpr (NC == 32) tmem_st32(taddr, r);
  else tmem_st16(taddr, r);
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st4(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
               "r"(r[2]), "r"(r[3]) : "memory");
}
// NC (a multiple of 4) consecutive columns of this thread's lane
template <int NC>
__device__ __forceinline__ void tmem_ld_row(uint32_t taddr, uint32_t (&r)[NC]) {
  if constexpr (NC == 16) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
  } else {
#pragma unroll
    for (int i = 0; i < NC; i += 4) tmem_ld4(taddr + i, r + i);
  }
}
template <int NC>
__device__ __forceinline__ void tmem_st_row(uint32_t taddr, const uint32_t (&r)[NC]) {
#pragma unroll
  for (int i = 0; i < NC; i += 4) tmem_st4(taddr + i, r + i);
}

// shared-memory matrix descriptor, no swizzle: core matrices of 8 rows x 16 bytes;
// lbo / sbo: byte distance between core matrices along K / along N
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3fff);
  d |= (uint64_t)((lbo >> 4) & 0x3fff) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3fff) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version of this architecture
  return d;
}
// kind::i8 instruction descriptor: unsigned 8-bit A and B, s32 accumulate, M = 128, A K-major (tensor memory),
// B N-major (a token's or a channel's columns are contiguous in shared memory)
__host__ __device__ constexpr uint32_t idesc_i8(int n) {
  return (2u << 4) | (1u << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// D[128 x N] (+)= A[128 x 32] (tensor memory) * B[32 x N] (shared memory); issued by one thread
template <bool ACC>
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc) {
  if constexpr (ACC) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.eq.b32 p, 0, 0;\n"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%4,%4,%4,%4}, p;\n}\n" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(0u) : "memory");
  } else {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, 0, 0;\n"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%4,%4,%4,%4}, p;\n}\n" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(0u) : "memory");
  }
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}

// ---------------------------------------------------------------------------
// stage of one 128-token batch, shared-memory plan, tensor-memory columns
// ---------------------------------------------------------------------------
template <int BK, int BV, int GS>
struct Stage {
  static constexpr int NGB = BT / GS;        // key token groups per batch = channel groups of a value row
  static constexpr int KC = 2048 * BK;       // key codes: 4 units of [chunk][32 tokens][16 B]
  static constexpr int KM = NGB * 512;       // key scales and zero-points of the batch's groups
  static constexpr int VC = 2048 * BV;       // value codes: [chunk][128 channels][16 B]
  static constexpr int VM = BT * 4 * NGB;    // value scales and zero-points: per token [NGB][NGB] fp16
  static constexpr int OFF_KM = KC;
  static constexpr int OFF_VC = KC + KM;
  static constexpr int OFF_VM = KC + KM + VC;
  static constexpr int BYTES = KC + KM + VC + VM;
};

constexpr int WROW = 2 * HD + 16;         // bytes per staged window row (padded against bank conflicts)
constexpr int WIN_BYTES = 2 * 16 * WROW;  // 16 key rows, then 16 value rows

// GP: query heads per kv head, padded to a power of two
template <int BK, int BV, int GS, int GP>
struct Plan {
  using St = Stage<BK, BV, GS>;
  static constexpr int NGB = St::NGB;
  static constexpr int NCOL = 4 * GP;                                   // operand columns of one (group, head set)
  static constexpr int N = (NGB * NCOL) < 16 ? 16 : NGB * NCOL;         // MMA N: (group, head, byte)
  static constexpr uint32_t LBO = (N / 16) * 128;                       // 8 K-rows of N bytes
  static constexpr int B_BYTES = BT * N;
  static constexpr int OFF_BK = NSTG * St::BYTES;
  static constexpr int OFF_BV = OFF_BK + B_BYTES;
  static constexpr int OFF_WIN = OFF_BV + B_BYTES;
  static constexpr int OFF_RED = OFF_WIN + WIN_BYTES;                    // reductions: [2 teams][4 warps][64] words
  static constexpr int META_SLOT = NGB * GP * 4;                         // logit biases of a batch: [group][head] fp32
  static constexpr int OFF_META = OFF_RED + 2 * 4 * 64 * 4;              // one slot per stage
  static constexpr int OFF_WST = OFF_META + NSTG * META_SLOT;            // window state rows [GP][MS]
  static constexpr int OFF_MST = OFF_WST + GP * MS * 4;                  // main state rows [GP][MS]
  static constexpr int TOTAL = OFF_MST + GP * MS * 4;
  // tensor memory columns: A_K, A_V, S of even and odd batches, O
  static constexpr uint32_t COL_AK = 0, COL_AV = 32, COL_S = 64, COL_O = 64 + 2 * N;
  static constexpr uint32_t COLS_USED = 64 + 3 * N;
  static constexpr uint32_t TM_COLS = COLS_USED <= 128 ? 128 : (COLS_USED <= 256 ? 256 : 512);
  static_assert(COLS_USED <= 512, "tensor memory has 512 columns");
};

// key codes: the weight channel d's code carries in its operand byte is 2^k_weight_log2
template <int BK>
__device__ __forceinline__ int k_weight_log2(int d) { return BK == 2 ? 2 * (((d % 16) / 4) & 1) : ((d % 32) / 4) % 4; }
// value codes: same for token t of a batch
template <int BV>
__device__ __forceinline__ int v_weight_log2(int t) { return BV == 2 ? 0 : ((t % 32) / 4) & 1; }

// ---------------------------------------------------------------------------
// window tiles on the legacy tensor-core path: 16 tokens of the 16-bit window are staged row by row and folded
// into a softmax state held in registers by one warp (bf16 operands, fp32 accumulate).
// ---------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_addr), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::: "memory"); }
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
  return d;
}
// 16-bit operands of the window's type (F16: IEEE half precision, else bfloat16), fp32 accumulate
template <bool F16>
__device__ __forceinline__ void mma16816_io(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                            uint32_t b0, uint32_t b1) {
  if constexpr (F16) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  } else {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
template <bool F16>
__device__ __forceinline__ uint32_t pack_io2(float lo, float hi) {
  if constexpr (F16) {
    __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
  } else {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
  }
}
template <bool F16>
__device__ __forceinline__ float io2_lo(uint32_t w) { return F16 ? f16_to_f(w & 0xffffu) : bf16_to_f(w & 0xffffu); }
template <bool F16>
__device__ __forceinline__ float io2_hi(uint32_t w) { return F16 ? f16_to_f(w >> 16) : bf16_to_f(w >> 16); }

// One warp stages window tokens [tb, tb + 16) (rows at or beyond t1 are zero-filled); no commit.  With a fused
// append the newest row (index r - 1) is not in the window yet: it comes from the step's input.
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
      if (p.K_new != nullptr && tb + row == p.r - 1) {
        const size_t noff = (size_t)(b * dm.Hkv + hk) * (2 * HD) + c * 16;
        cp_async16(dk, reinterpret_cast<const uint8_t*>(p.K_new) + noff);
        cp_async16(dv, reinterpret_cast<const uint8_t*>(p.V_new) + noff);
      } else {
        cp_async16(dk, wk + off);
        cp_async16(dv, wv + off);
      }
    } else {
      sts128(dk, 0u, 0u, 0u, 0u);
      sts128(dv, 0u, 0u, 0u, 0u);
    }
  }
}

// Fused append: the staged tile [tb, tb + 16) holds the token of this step (row r - 1); the warp stores it into
// the window, keys by lanes 0..15, values by lanes 16..31.
__device__ __forceinline__ void window_store_new(const DecodeParams& p, int tb, int hk, int b, uint32_t wbuf, int lane) {
  const Dims& dm = p.dm;
  const int row = p.r - 1 - tb, c = lane & 15;
  const uint4 v = lds128(wbuf + (lane >> 4) * 16 * WROW + row * WROW + c * 16);
  uint8_t* win = reinterpret_cast<uint8_t*>(lane < 16 ? p.L.win_k : p.L.win_v);
  *reinterpret_cast<uint4*>(win + ((size_t)(b * dm.Hkv + hk) * dm.R + (p.r - 1)) * (2 * HD) + c * 16) = v;
}

// One warp folds the staged tile (n_valid of its 16 tokens exist) into its softmax state: S^T = K q^T with tokens
// as rows and the heads in the eight columns (SP: head h in column 2h, odd columns padding), O^T += V^T P.
// qb: q of the head of column lane/4 as bf16 pairs in B-operand order; accZ row 8 carries sum_t p_t.
template <bool SP, bool F16>
__device__ __forceinline__ void window_tile(uint32_t wbuf, int n_valid, const uint32_t (&qb)[16], float scale2,
                                            float (&accO)[8][4], float (&accZ)[4], float& m0, float& m1, int lane) {
  const int gid = lane >> 2;
  float s[4] = {0.f, 0.f, 0.f, 0.f};  // rows = tokens gid, gid + 8; cols = 2 tig, 2 tig + 1
  const uint32_t ka = wbuf + ((lane & 7) + 8 * ((lane >> 3) & 1)) * WROW + (lane >> 4) * 16;
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    uint32_t a0, a1, a2, a3;
    ldmatrix_x4(ka + ks * 32, a0, a1, a2, a3);
    mma16816_io<F16>(s, a0, a1, a2, a3, qb[2 * ks], qb[2 * ks + 1]);
  }
  const bool va = gid < n_valid, vb = gid + 8 < n_valid;
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
  // numerators as a 16-bit pair hi + lo (at least 16 bits of precision), transposed into B-operand order
  const uint32_t h0 = pack_io2<F16>(p00, p01), h1 = pack_io2<F16>(p10, p11);
  const uint32_t l0 = pack_io2<F16>(p00 - io2_lo<F16>(h0), p01 - io2_hi<F16>(h0));
  const uint32_t l1 = pack_io2<F16>(p10 - io2_lo<F16>(h1), p11 - io2_hi<F16>(h1));
  const uint32_t bh0 = movmatrix_trans(h0), bh1 = movmatrix_trans(h1), bl0 = movmatrix_trans(l0), bl1 = movmatrix_trans(l1);
  const uint32_t ones = (gid == 0) ? (F16 ? 0x3C003C00u : 0x3F803F80u) : 0u;  // row 8 of the sums tile: sum_t p_t
  mma16816_io<F16>(accZ, 0u, ones, 0u, ones, bh0, bh1);
  mma16816_io<F16>(accZ, 0u, ones, 0u, ones, bl0, bl1);
  const int mi = lane >> 3;
  const uint32_t va_addr = wbuf + 16 * WROW + ((lane & 7) + 8 * (mi >> 1)) * WROW + (mi & 1) * 16;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    uint32_t a0, a1, a2, a3;
    ldmatrix_x4_trans(va_addr + mt * 32, a0, a1, a2, a3);
    mma16816_io<F16>(accO[mt], a0, a1, a2, a3, bh0, bh1);
    mma16816_io<F16>(accO[mt], a0, a1, a2, a3, bl0, bl1);
  }
}

// The window warp: this CTA's share [wt0, wt1) of the window, tile by tile; leaves one state row per head
// (acc[HD], m, l) in `wst` (heads without tokens: m = -inf, l = 0).
template <bool SP, bool F16>
__device__ __forceinline__ void window_warp(const DecodeParams& p, int wt0, int wt1, int hk, int b, uint32_t wbuf,
                                            float* wst, int lane) {
  const Dims& dm = p.dm;
  const int G = dm.G, gid = lane >> 2, tig = lane & 3;
  const float scale2 = p.scale * 1.4426950408889634f;
  uint32_t raw[16];  // q of the head of column gid: (q[16s + 2tig + 8j], q[16s + 2tig + 8j + 1])
  {
    const int hcol = SP ? (gid >> 1) : gid;
    const bool real = SP ? ((gid & 1) == 0 && hcol < G) : (gid < G);
    const uint16_t* qp = p.q + ((size_t)b * dm.Hq + hk * G + (real ? hcol : 0)) * HD + 2 * tig;
#pragma unroll
    for (int i = 0; i < 16; ++i) raw[i] = real ? *reinterpret_cast<const uint32_t*>(qp + 16 * (i >> 1) + 8 * (i & 1)) : 0u;
  }
  float accO[8][4], accZ[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int mt = 0; mt < 8; ++mt)
#pragma unroll
    for (int i = 0; i < 4; ++i) accO[mt][i] = 0.f;
  float m0 = -CUDART_INF_F, m1 = SP ? 0.f : -CUDART_INF_F;
  for (int tb = wt0; tb < wt1; tb += 16) {
    __syncwarp();
    window_stage(p, tb, wt1, hk, b, wbuf, lane);
    cp_async_commit();
    cp_async_wait_all();
    __syncwarp();
    if (p.K_new != nullptr && tb + 16 > p.r - 1 && wt1 == p.r) window_store_new(p, tb, hk, b, wbuf, lane);
    window_tile<SP, F16>(wbuf, wt1 - tb, raw, scale2, accO, accZ, m0, m1, lane);
  }
  const float l0 = __shfl_sync(0xffffffffu, accZ[2], tig), l1 = __shfl_sync(0xffffffffu, accZ[3], tig);
  const int h0 = SP ? tig : 2 * tig, h1 = 2 * tig + 1;
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    const int ch = 16 * mt + gid;
    if (h0 < G) { wst[h0 * MS + ch] = accO[mt][0]; wst[h0 * MS + ch + 8] = accO[mt][2]; }
    if (!SP && h1 < G) { wst[h1 * MS + ch] = accO[mt][1]; wst[h1 * MS + ch + 8] = accO[mt][3]; }
  }
  if (gid == 0) {
    if (h0 < G) { wst[h0 * MS + HD] = m0; wst[h0 * MS + HD + 1] = l0; }
    if (!SP && h1 < G) { wst[h1 * MS + HD] = m1; wst[h1 * MS + HD + 1] = l1; }
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

// Split-K merge by the last CTA of a (sequence, kv head), run by the 128 compute threads: the CTA takes a ticket
// after its partials are visible device-wide; the CTA that draws the last ticket reads all partials from L2 and
// writes out = sum_s acc_s 2^(m_s-M) / sum_s l_s 2^(m_s-M).  No CTA ever waits for another.
__device__ __forceinline__ void ticket_merge(const DecodeParams& p, int ns, int stride, int hk, int b, int* s_flag) {
  const Dims& dm = p.dm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = b * dm.Hkv + hk;
  // The barrier orders every thread's partial stores before thread 0's ticket; the ticket is a release (cumulative
  // over what the barrier ordered) and an acquire at device scope, so the CTA that draws the last ticket sees all
  // partials after its second barrier.  The partials are then read from L2 (ld.global.cg).
  bar_sync_compute();
  if (threadIdx.x == 0) {
    unsigned t;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;\n" : "=r"(t) : "l"(p.tickets + bh) : "memory");
    *s_flag = (t == (unsigned)(ns - 1));
  }
  bar_sync_compute();
  if (!*s_flag) return;
  for (int a = warp; a < dm.G; a += 4) {
    const size_t hq = (size_t)b * dm.Hq + hk * dm.G + a;
    const float* ml = p.part_ml + hq * stride * 2;
    const float* pa = p.part_acc + hq * stride * HD + lane * 4;
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
      uint2 pk;
      if (p.f16) {
        __half2 lo = __floats2half2_rn(acc.x, acc.y), hi = __floats2half2_rn(acc.z, acc.w);
        pk = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      } else {
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        pk = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      }
      *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(p.out) + hq * HD + lane * 4) = pk;
    }
  }
  if (threadIdx.x == 0) p.tickets[bh] = 0u;  // ready for the next launch on this stream
}

// stores NCOL consecutive operand bytes of a row (inside one 16-byte block, or two whole blocks); words[h] holds
// the four bytes of head h
template <int NCOL>
__device__ __forceinline__ void store_slice(uint32_t addr, const uint32_t* words) {
  if constexpr (NCOL == 4) sts32(addr, words[0]);
  else if constexpr (NCOL == 8) sts64(addr, words[0], words[1]);
  else if constexpr (NCOL == 16) sts128(addr, words[0], words[1], words[2], words[3]);
  else {
    sts128(addr, words[0], words[1], words[2], words[3]);
    sts128(addr + 128, words[4], words[5], words[6], words[7]);
  }
}
// Expands this thread's share of its token's packed key row into A_K columns: team t of NT takes the columns
// [t * 32 / NT, (t + 1) * 32 / NT).  `unit` is the token's 32-token unit of the staged batch.
template <int BK, int NT>
__device__ __forceinline__ void expand_keys(uint32_t kc_smem, int unit, int lane, int team, uint32_t row_taddr) {
  constexpr int NW = (BK == 2 ? 8 : 4) / NT;  // packed words this thread expands
  uint32_t w[NW];
  if constexpr (BK == 2) {
    // [chunk][token][16 bytes]: chunk c holds words 4c .. 4c + 3
    if constexpr (NT == 1) {
      const uint4 c0 = lds128(kc_smem + unit * 1024 + lane * 16), c1 = lds128(kc_smem + unit * 1024 + 512 + lane * 16);
      w[0] = c0.x; w[1] = c0.y; w[2] = c0.z; w[3] = c0.w; w[4] = c1.x; w[5] = c1.y; w[6] = c1.z; w[7] = c1.w;
    } else {
      const uint4 c0 = lds128(kc_smem + unit * 1024 + team * 512 + lane * 16);
      w[0] = c0.x; w[1] = c0.y; w[2] = c0.z; w[3] = c0.w;
    }
  } else {
    if constexpr (NT == 1) {
      const uint4 c0 = lds128(kc_smem + unit * 512 + lane * 16);
      w[0] = c0.x; w[1] = c0.y; w[2] = c0.z; w[3] = c0.w;
    } else {
      const uint2 c0 = lds64(kc_smem + unit * 512 + lane * 16 + team * 8);
      w[0] = c0.x; w[1] = c0.y;
    }
  }
  uint32_t r[32 / NT];
#pragma unroll
  for (int i = 0; i < NW; ++i) {
    const uint32_t hi = w[i] >> 4;
    if constexpr (BK == 2) {
      r[4 * i + 0] = w[i] & 0x03030303u;
      r[4 * i + 1] = w[i] & 0x0C0C0C0Cu;
      r[4 * i + 2] = hi & 0x03030303u;
      r[4 * i + 3] = hi & 0x0C0C0C0Cu;
    } else {
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        r[8 * i + m] = w[i] & (0x01010101u << m);
        r[8 * i + 4 + m] = hi & (0x01010101u << m);
      }
    }
  }
  tmem_st_cols<32 / NT>(row_taddr + team * (32 / NT), r);
}

// Expands this thread's share of channel d's packed row into A_V columns (32 columns over the batch's 128 tokens).
// The values keep small weights (1-bit: 1 or 2; 2-bit: 1): every rounding of the other operand is multiplied by them.
template <int BV, int NT>
__device__ __forceinline__ void expand_values(uint32_t vc_smem, int d, int team, uint32_t row_taddr) {
  constexpr int NW = (BV == 2 ? 8 : 4) / NT;
  uint32_t w[NW];
  if constexpr (BV == 2) {
    if constexpr (NT == 1) {
      const uint4 c0 = lds128(vc_smem + d * 16), c1 = lds128(vc_smem + 2048 + d * 16);
      w[0] = c0.x; w[1] = c0.y; w[2] = c0.z; w[3] = c0.w; w[4] = c1.x; w[5] = c1.y; w[6] = c1.z; w[7] = c1.w;
    } else {
      const uint4 c0 = lds128(vc_smem + team * 2048 + d * 16);
      w[0] = c0.x; w[1] = c0.y; w[2] = c0.z; w[3] = c0.w;
    }
  } else {
    if constexpr (NT == 1) {
      const uint4 c0 = lds128(vc_smem + d * 16);
      w[0] = c0.x; w[1] = c0.y; w[2] = c0.z; w[3] = c0.w;
    } else {
      const uint2 c0 = lds64(vc_smem + d * 16 + team * 8);
      w[0] = c0.x; w[1] = c0.y;
    }
  }
  uint32_t r[32 / NT];
#pragma unroll
  for (int i = 0; i < NW; ++i) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t s = w[i] >> (2 * k);
      if constexpr (BV == 1) {
        r[8 * i + 2 * k] = s & 0x01010101u;
        r[8 * i + 2 * k + 1] = s & 0x02020202u;
      } else {
        r[4 * i + k] = s & 0x03030303u;
      }
    }
  }
  tmem_st_cols<32 / NT>(row_taddr + team * (32 / NT), r);
}

// byte offset, within a row of a B operand, of column n
__device__ __forceinline__ uint32_t column_offset(int n) { return (uint32_t)((n >> 4) * 128 + (n & 15)); }

// ---------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------
// GP: heads per kv head padded to a power of two; SP: window tiles with the heads in the even columns (G <= 4);
// NT: teams of four compute warps (a team takes GP / NT heads and 32 / NT columns of every expansion).
template <int BK, int BV, int GS, int GP, bool SP, int NT>
__global__ void __launch_bounds__((4 * NT + 3) * 32, GP <= 4 ? 2 : 1) decode_umma_kernel(DecodeParams p) {
  using St = Stage<BK, BV, GS>;
  using Pl = Plan<BK, BV, GS, GP>;
  constexpr int NGB = St::NGB, N = Pl::N, NCOL = Pl::NCOL;
  constexpr int WPG = GS / 32;        // warps of a team whose rows share a group
  constexpr int NCW = 4 * NT;         // compute warps
  constexpr int W_WIN = NCW, W_BIAS = NCW + 1, W_MMA = NCW + 2;
  constexpr int HT = GP / NT;         // heads of a team
  constexpr int TCOL = 4 * HT;        // operand columns (bytes) of a team within a (row, group) slice
  constexpr uint32_t LBO = Pl::LBO;
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) unsigned long long bar_mem[2 * NSTG + 5];
  __shared__ uint32_t tmem_base_sm;
  __shared__ int tma_issued;              // batches whose copies have been issued
  __shared__ int s_flag;
  __shared__ volatile int dead_sm;

  const Dims& dm = p.dm;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = dm.G;

  // The next kernel in the stream may be scheduled at once when all work before this kernel's own predecessor is
  // known to be complete (a chained launch); otherwise only after this kernel's own wait (below), so that a chained
  // successor never starts before the work this kernel waited for has completed.
  if (p.late_wait) grid_dependents_go();

  // CTA -> (stream, split): p.n_ctas CTAs dealt to the streams in order; the first n_ctas % streams streams get one
  // split more than the others
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
  const int bh = b * dm.Hkv + hk;
  const int nbt = (p.n_q + BT - 1) / BT;  // batches of the stream (the last one may be ragged)
  int b0, b1;
  share_of(nbt, ns, split, b0, b1);
  const int nb = b1 - b0;                 // >= 1: the host never asks for more splits than batches

  const uint32_t sm_base = (uint32_t)__cvta_generic_to_shared(smem);
  const uint32_t bars = (uint32_t)__cvta_generic_to_shared(&bar_mem[0]);
  const uint32_t bar_full = bars;                     // [NSTG] the bulk copies of a batch have landed
  const uint32_t bar_bias = bar_full + 8 * NSTG;      // [NSTG] the logit biases of a batch are written
  const uint32_t bar_sready = bar_bias + 8 * NSTG;    // [2] the key products of a batch are complete
  const uint32_t bar_odone = bar_sready + 16;         // the value products of a batch are complete
  const uint32_t bar_kready = bar_odone + 8;          // every compute warp has written its part of A_K and B_K
  const uint32_t bar_vready = bar_kready + 8;         // the same for A_V and B_V (and the batch's stage is free)
  float* wst = reinterpret_cast<float*>(smem + Pl::OFF_WST);
  float* mst = reinterpret_cast<float*>(smem + Pl::OFF_MST);

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < NSTG; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_bias + 8 * s, 1);
    }
    mbar_init(bar_sready, 1);
    mbar_init(bar_sready + 8, 1);
    mbar_init(bar_odone, 1);
    mbar_init(bar_kready, NCW);
    mbar_init(bar_vready, NCW);
    tma_issued = 0;
    dead_sm = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == W_MMA) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(
                     (uint32_t)__cvta_generic_to_shared(&tmem_base_sm)), "r"(Pl::TM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = tmem_base_sm;

  // Copies of batch j of this CTA's range into its stage (one thread; the stage is free)
  auto issue_batch = [&](int j) {
    const int s = j % NSTG;
    const size_t bj = (size_t)(b0 + j);
    const uint8_t* gk = reinterpret_cast<const uint8_t*>(p.L.k_codes) + (size_t)bh * ((size_t)dm.nq_cap * (HD * BK / 8)) + bj * St::KC;
    const uint8_t* gkm = reinterpret_cast<const uint8_t*>(p.L.k_meta) + (size_t)bh * ((size_t)(dm.nq_cap / GS) * 512) + bj * St::KM;
    const uint8_t* gv = reinterpret_cast<const uint8_t*>(p.L.v_codes) + (size_t)bh * ((size_t)dm.nq_cap * (HD * BV / 8)) + bj * St::VC;
    const uint8_t* gvm = reinterpret_cast<const uint8_t*>(p.L.v_meta) + (size_t)bh * ((size_t)dm.nq_cap * 4 * NGB) + bj * St::VM;
    const uint32_t dst = sm_base + s * St::BYTES, fb = bar_full + 8 * s;
    mbar_expect_tx(fb, St::BYTES);
    bulk_load(dst, gk, St::KC, fb);
    bulk_load(dst + St::OFF_KM, gkm, St::KM, fb);
    bulk_load(dst + St::OFF_VC, gv, St::VC, fb);
    bulk_load(dst + St::OFF_VM, gvm, St::VM, fb);
    tma_issued = j + 1;
  };

  if (warp == W_MMA) {
    // ================= MMA warp: copies and products (the loop is warp-uniform, one elected lane issues) ============
    // Packed data that earlier calls completed may be fetched while the preceding kernel still runs; when a pack
    // kernel may have written it since this layer's last decode, the first copies wait for that kernel.
    if (!p.early_fetch) grid_dependency_wait();
    if (lane == 0) {
      for (int j = 0; j < nb && j < NSTG; ++j) issue_batch(j);
    }
    __syncwarp();
    const uint64_t dK = smem_desc(sm_base + Pl::OFF_BK, LBO, 128), dV = smem_desc(sm_base + Pl::OFF_BV, LBO, 128);
    constexpr uint32_t KSTEP = (4 * LBO) >> 4;  // descriptor units per 32 rows of K
    constexpr uint32_t IDESC = idesc_i8(N);
    for (int i = 0; i <= nb; ++i) {
      if (i < nb) {  // keys of batch i
        const bool ok = mbar_wait(bar_kready, i & 1, &dead_sm);
        tc_fence_after();
        if (ok && elect_one()) {
          const uint32_t dS = tbase + Pl::COL_S + (uint32_t)(i & 1) * N, aK = tbase + Pl::COL_AK;
          umma_i8<false>(dS, aK, dK, IDESC);
          umma_i8<true>(dS, aK + 8, dK + KSTEP, IDESC);
          umma_i8<true>(dS, aK + 16, dK + 2 * KSTEP, IDESC);
          umma_i8<true>(dS, aK + 24, dK + 3 * KSTEP, IDESC);
          umma_commit(bar_sready + 8 * (i & 1));
        }
        __syncwarp();
      }
      if (i > 0) {  // values of batch i - 1; its stage is free
        const int k = i - 1;
        const bool ok = mbar_wait(bar_vready, k & 1, &dead_sm);
        tc_fence_after();
        if (ok && elect_one()) {
          const uint32_t dO = tbase + Pl::COL_O, aV = tbase + Pl::COL_AV;
          if (k == 0) umma_i8<false>(dO, aV, dV, IDESC);
          else umma_i8<true>(dO, aV, dV, IDESC);
          umma_i8<true>(dO, aV + 8, dV + KSTEP, IDESC);
          umma_i8<true>(dO, aV + 16, dV + 2 * KSTEP, IDESC);
          umma_i8<true>(dO, aV + 24, dV + 3 * KSTEP, IDESC);
          umma_commit(bar_odone);
          if (k + NSTG < nb) issue_batch(k + NSTG);
        }
        __syncwarp();
      }
    }
  } else if (warp == W_WIN) {
    // ================= window warp: this CTA's share of the 16-bit window =================
    if (!p.late_wait) grid_dependency_wait();
    int wt0, wt1;
    share_of(p.r, ns, split, wt0, wt1);
    if (wt0 < wt1) {
      if (p.f16) window_warp<SP, true>(p, wt0, wt1, hk, b, sm_base + Pl::OFF_WIN, wst, lane);
      else window_warp<SP, false>(p, wt0, wt1, hk, b, sm_base + Pl::OFF_WIN, wst, lane);
    } else {
      for (int h = 0; h < G; ++h) {
        for (int c = lane; c < HD; c += 32) wst[h * MS + c] = 0.f;
        if (lane == 0) { wst[h * MS + HD] = -CUDART_INF_F; wst[h * MS + HD + 1] = 0.f; }
      }
    }
  } else if (warp == W_BIAS) {
    // ================= bias warp: sigma * sum_d q_d z_d per (token group, head) of a batch =================
    if (!p.late_wait) grid_dependency_wait();  // q may come from the preceding kernel
    // One row of legacy tensor-core products per batch: rows = the batch's token groups (zero-points read as they
    // are staged, fp16), columns = heads (q as fp16: exact for bf16 inputs of ordinary magnitude), fp32 accumulate.
    const int gid = lane >> 2, tig = lane & 3;
    const float scale2 = p.scale * 1.4426950408889634f;
    uint32_t qf[16];  // B fragments: head gid, staged positions 16 ks + 2 tig (+1) and + 8
    {
      const bool real = gid < G;
      const uint16_t* qp = p.q + ((size_t)b * dm.Hq + hk * G + (real ? gid : 0)) * HD;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int pos = 16 * (i >> 1) + 8 * (i & 1) + 2 * tig;  // staged position -> channel (pos % 4) * 32 + pos / 4
        const float q0 = real ? io_to_f(qp[(pos & 3) * 32 + (pos >> 2)], p.f16) : 0.f;
        const float q1 = real ? io_to_f(qp[((pos + 1) & 3) * 32 + ((pos + 1) >> 2)], p.f16) : 0.f;
        const __half2 h2 = __floats2half2_rn(q0, q1);
        qf[i] = *reinterpret_cast<const uint32_t*>(&h2);
      }
    }
    for (int i = 0; i < nb; ++i) {
      const int s = i % NSTG;
      mbar_wait(bar_full + 8 * s, (i / NSTG) & 1, &dead_sm);
      const uint32_t zrow = sm_base + s * St::BYTES + St::OFF_KM + (gid < NGB ? gid : 0) * 512 + 256 + 4 * tig;
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint32_t a0 = gid < NGB ? lds32(zrow + 32 * ks) : 0u, a2 = gid < NGB ? lds32(zrow + 32 * ks + 16) : 0u;
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(qf[2 * ks]), "r"(qf[2 * ks + 1]));
      }
      if (gid < NGB) {
        float* slot = reinterpret_cast<float*>(smem + Pl::OFF_META + s * Pl::META_SLOT) + gid * GP;
        if (2 * tig < GP) slot[2 * tig] = c[0] * scale2;
        if (2 * tig + 1 < GP) slot[2 * tig + 1] = c[1] * scale2;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_bias + 8 * s);
    }
  } else {
    // ================= compute warps: thread = tensor-memory lane =================
    const int team = NT == 1 ? 0 : warp >> 2, qw = warp & 3;  // qw: lane quarter
    const int ctid = qw * 32 + lane;                          // row: token of the batch / channel
    const int h0 = team * HT;                                 // first head of the team
    if (!p.late_wait) {
      grid_dependency_wait();  // q may come from the preceding kernel
      grid_dependents_go();    // whatever this kernel waited for is complete for its successor too
    }
    const int gam = qw / WPG;  // this warp's rows: key token group of the batch / channel group of O
    const uint32_t row_t = tbase + ((uint32_t)(qw * 32) << 16);
    const float scale2 = p.scale * 1.4426950408889634f;
    const uint32_t bar_team = 1 + team;  // hardware barrier of the team's 128 threads

    // ---- q: this lane's channels lane + 32 j of the team's heads, pre-scaled for the B_K operand ----
    // B_K holds rint(q_d s_d 2^(Eq + Es) / w_d): w_d is the weight the code of channel d carries in its A byte,
    // Eq puts the head's largest |q| and Es the group's largest scale just below 2^10 (|product| < 2^20).
    float qp[HT][4], cq[HT];
    {
      const int wl = k_weight_log2<BK>(lane);  // the same for lane + 32 j
#pragma unroll
      for (int h = 0; h < HT; ++h) {
        float qv[4], am = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          qv[j] = h0 + h < G ? io_to_f(p.q[((size_t)b * dm.Hq + hk * G + h0 + h) * HD + lane + 32 * j], p.f16) : 0.f;
          am = fmaxf(am, fabsf(qv[j]));
        }
        const float qmax = __uint_as_float(redux_max_u32(__float_as_uint(am)));
        const int Eq = qmax > 0.f ? max(-100, min(100, 9 - exponent_of(qmax))) : 0;
        const float e2 = pow2i(Eq - wl);
#pragma unroll
        for (int j = 0; j < 4; ++j) qp[h][j] = qv[j] * e2;
        cq[h] = scale2 * pow2i(-Eq);
      }
    }

    // softmax state of the team (the same in each of its threads) and this thread's partial sums
    float m[HT], l[HT], zacc[NGB][HT];
    int Ev[NGB];        // value scales of channel group gi are taken relative to 2^Ev[gi]
    float vsc[NGB];     // 2^(FRAC_V - Ev[gi]) / (weight of this thread's token in its A_V byte)
    const float wv_inv = pow2i(-v_weight_log2<BV>(ctid));
#pragma unroll
    for (int h = 0; h < HT; ++h) {
      m[h] = -CUDART_INF_F;
      l[h] = 0.f;
#pragma unroll
      for (int gi = 0; gi < NGB; ++gi) zacc[gi][h] = 0.f;
    }
#pragma unroll
    for (int gi = 0; gi < NGB; ++gi) { Ev[gi] = -24; vsc[gi] = pow2i(FRAC_V + 24) * wv_inv; }

    // A_K row and B_K slice of the batch staged at `st` for this warp's token group; returns the logit scales
    auto prep_keys = [&](uint32_t st, float (&ck)[HT]) {
      expand_keys<BK, NT>(st, qw, lane, team, row_t + Pl::COL_AK);
      const uint32_t km = st + St::OFF_KM + gam * 512 + lane * 8;
      const uint2 sraw = lds64(km);
      const float2 s01 = __half22float2(*reinterpret_cast<const __half2*>(&sraw.x));
      const float2 s23 = __half22float2(*reinterpret_cast<const __half2*>(&sraw.y));
      const float sf[4] = {s01.x, s01.y, s23.x, s23.y};
      const float smx = fmaxf(fmaxf(sf[0], sf[1]), fmaxf(sf[2], sf[3]));
      const float smax = __uint_as_float(redux_max_u32(__float_as_uint(smx)));
      const int Es = smax > 0.f ? 9 - exponent_of(smax) : 0;
      const float e2 = pow2i(Es), e2i = pow2i(-Es);
      const uint32_t bk = sm_base + Pl::OFF_BK + (lane >> 3) * LBO + (lane & 7) * 16 + column_offset(gam * NCOL + team * TCOL);
#pragma unroll
      for (int jj = 0; jj < 4 / WPG; ++jj) {
        const int j = WPG == 1 ? jj : 2 * (qw % WPG) + jj;  // with two warps per group each takes half the channels
        const float sp = sf[j] * e2;
        uint32_t words[HT];
#pragma unroll
        for (int h = 0; h < HT; ++h) words[h] = __float_as_uint(fmaf(qp[h][j], sp, MAGIC_K));
        store_slice<TCOL>(bk + 4 * j * LBO, words);
      }
#pragma unroll
      for (int h = 0; h < HT; ++h) ck[h] = cq[h] * e2i;
    };
    // this warp's part of the key (value) operands is written: hand it to the MMA warp
    auto publish = [&](uint32_t bar) {
      tc_wait_st();
      proxy_fence();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar);
    };

    // Raises the team's softmax references and / or value-scale exponents so that every numerator of this batch
    // is at most 2^TAU and every normalised value scale below 1, and rescales what has been accumulated.
    auto raise = [&](int i, const float (&x)[HT], const float (&sv)[NGB]) {
      int* red = reinterpret_cast<int*>(smem + Pl::OFF_RED) + team * 256;  // [4 warps][64]
#pragma unroll
      for (int h = 0; h < HT; ++h) {
        const int k = redux_max_s32(float_key(x[h]));
        if (lane == 0) red[qw * 64 + h] = k;
      }
#pragma unroll
      for (int gi = 0; gi < NGB; ++gi) {
        const uint32_t u = redux_max_u32(__float_as_uint(sv[gi]));
        if (lane == 0) red[qw * 64 + 8 + gi] = (int)u;
      }
      bar_sync_team(bar_team);
      float dmh[HT];
      int dE_row = 0;
#pragma unroll
      for (int h = 0; h < HT; ++h) {
        const int k = max(max(red[h], red[64 + h]), max(red[128 + h], red[192 + h]));
        const float xm = key_float(k);
        float mn = m[h];
        if (xm > m[h] + (float)(TAU - 1)) mn = fmaxf(m[h], ceilf(xm) - (float)MREF);
        dmh[h] = mn - m[h];  // +inf on the first batch (nothing accumulated yet)
        const float f = ex2(-dmh[h]);
        l[h] *= f;
#pragma unroll
        for (int gi = 0; gi < NGB; ++gi) zacc[gi][h] *= f;
        m[h] = mn;
      }
#pragma unroll
      for (int gi = 0; gi < NGB; ++gi) {
        const uint32_t u = (uint32_t)max(max(red[8 + gi], red[64 + 8 + gi]), max(red[128 + 8 + gi], red[192 + 8 + gi]));
        int En = Ev[gi];
        if ((int)u >= ((Ev[gi] + 127) << 23)) En = min(exponent_of(__uint_as_float(u)) + 1, 64);
        if (gi == gam) dE_row = En - Ev[gi];
        Ev[gi] = En;
        vsc[gi] = pow2i(FRAC_V - En) * wv_inv;
      }
      if (i > 0) {  // O of this thread's channel: its group's columns of the team's heads, three byte planes per head
        mbar_wait(bar_odone, (i - 1) & 1, &dead_sm);
        tc_fence_after();
        uint32_t o[TCOL];
        tmem_ld_row<TCOL>(row_t + Pl::COL_O + gam * NCOL + team * TCOL, o);
        tc_wait_ld();
#pragma unroll
        for (int h = 0; h < HT; ++h) {
          const int k = (int)fminf(dmh[h], 64.f) + dE_row;
          unsigned long long T = (unsigned long long)o[4 * h] + ((unsigned long long)o[4 * h + 1] << 8) +
                                 ((unsigned long long)o[4 * h + 2] << 16);
          T = k >= 63 ? 0ull : (T >> k);
          o[4 * h] = (uint32_t)(T & 0xffffull);
          o[4 * h + 1] = 0u;
          o[4 * h + 2] = (uint32_t)(T >> 16);
        }
        tmem_st_row<TCOL>(row_t + Pl::COL_O + gam * NCOL + team * TCOL, o);
        tc_wait_st();
      }
      bar_sync_team(bar_team);  // the reduction scratch may be written again
    };

    // ---- prologue: keys of the first batch ----
    float ck[HT], ck_n[HT];
    mbar_wait(bar_bias, 0, &dead_sm);  // the biases of a batch are written once its stage has landed
    prep_keys(sm_base, ck);
    publish(bar_kready);
#pragma unroll
    for (int h = 0; h < HT; ++h) ck_n[h] = ck[h];
    mbar_wait(bar_sready, 0, &dead_sm);  // S of the first batch
    tc_fence_after();

    // ---- main loop: keys of batch i + 1 go to the tensor core, then softmax and values of batch i ----
#pragma unroll 1
    for (int i = 0; i < nb; ++i) {
      const int s = i % NSTG;
      const uint32_t st = sm_base + s * St::BYTES;
      // S of batch i is complete and A_K and B_K are free (waited for in the iteration before)
      if (i + 1 < nb) {
        const int sn = (i + 1) % NSTG;
        mbar_wait(bar_bias + 8 * sn, ((i + 1) / NSTG) & 1, &dead_sm);  // stage and biases of batch i + 1
        prep_keys(sm_base + sn * St::BYTES, ck_n);
        publish(bar_kready);
      }

      // logits of this thread's token: its group's columns of S for the team's heads
      uint32_t d[TCOL];
      tmem_ld_row<TCOL>(row_t + Pl::COL_S + (uint32_t)(i & 1) * N + gam * NCOL + team * TCOL, d);
      // value scale / zero-point of this thread's token
      float sv[NGB], zv[NGB];
      if constexpr (NGB == 4) {
        const uint4 raw = lds128(st + St::OFF_VM + ctid * 16);
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
        const float2 c = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
        const float2 e = __half22float2(*reinterpret_cast<const __half2*>(&raw.z));
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&raw.w));
        sv[0] = a.x; sv[1] = a.y; sv[2] = c.x; sv[3] = c.y;
        zv[0] = e.x; zv[1] = e.y; zv[2] = f.x; zv[3] = f.y;
      } else {
        const uint2 raw = lds64(st + St::OFF_VM + ctid * 8);
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
        const float2 e = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
        sv[0] = a.x; sv[1] = a.y;
        zv[0] = e.x; zv[1] = e.y;
      }
      float bias[HT];
      {
        const float* slot = reinterpret_cast<const float*>(smem + Pl::OFF_META + s * Pl::META_SLOT) + gam * GP + h0;
#pragma unroll
        for (int h = 0; h < HT; ++h) bias[h] = slot[h];
      }
      const bool valid = (b0 + i) * BT + ctid < p.n_q;  // only the stream's last batch can be ragged
      if (!valid) {
#pragma unroll
        for (int gi = 0; gi < NGB; ++gi) { sv[gi] = 0.f; zv[gi] = 0.f; }
      }
      tc_wait_ld();
      float x[HT];
      bool need = false;
#pragma unroll
      for (int h = 0; h < HT; ++h) {
        // sum_d c_d w_d X_d = D0 + 2^8 D1 + 2^16 D2 - 2^14 D3 (D3 = 75 * row sum undoes the offset 75 * 2^14 of X_d)
        const int S = (int)(d[4 * h] + (d[4 * h + 1] << 8) + (d[4 * h + 2] << 16) - (d[4 * h + 3] << 14));
        x[h] = valid ? fmaf((float)S, ck[h], bias[h]) : -CUDART_INF_F;
        need |= x[h] > m[h] + (float)TAU;
      }
#pragma unroll
      for (int gi = 0; gi < NGB; ++gi) need |= __float_as_int(sv[gi]) >= ((Ev[gi] + 127) << 23);
      if (bar_or_team(bar_team, need)) raise(i, x, sv);

      float pe[HT];
#pragma unroll
      for (int h = 0; h < HT; ++h) {
        pe[h] = ex2(x[h] - m[h]);
        l[h] += pe[h];
#pragma unroll
        for (int gi = 0; gi < NGB; ++gi) zacc[gi][h] = fmaf(pe[h], zv[gi], zacc[gi][h]);
      }
      // The value products of batch i - 1 must be done with A_V and B_V.  They were issued before the key products
      // of batch i + 1, and a commit covers everything its thread issued before it: S of batch i + 1 being complete
      // says both, in one wait.
      if (i + 1 < nb) mbar_wait(bar_sready + 8 * ((i + 1) & 1), ((i + 1) >> 1) & 1, &dead_sm);
      else if (i > 0) mbar_wait(bar_odone, (i - 1) & 1, &dead_sm);
      tc_fence_after();
      {
        const uint32_t bv = sm_base + Pl::OFF_BV + (ctid >> 3) * LBO + (ctid & 7) * 16;
#pragma unroll
        for (int gi = 0; gi < NGB; ++gi) {
          const float sp = sv[gi] * vsc[gi];
          uint32_t words[HT];
#pragma unroll
          for (int h = 0; h < HT; ++h) words[h] = __float_as_uint(fmaf(pe[h], sp, MAGIC_V));
          store_slice<TCOL>(bv + column_offset(gi * NCOL + team * TCOL), words);
        }
      }
      expand_values<BV, NT>(st + St::OFF_VC, ctid, team, row_t + Pl::COL_AV);
      publish(bar_vready);
#pragma unroll
      for (int h = 0; h < HT; ++h) ck[h] = ck_n[h];
    }

    // ---- epilogue: O of this thread's channel, the team's sums, one state row per head ----
    mbar_wait(bar_odone, (nb - 1) & 1, &dead_sm);
    tc_fence_after();
    uint32_t o[TCOL];
    tmem_ld_row<TCOL>(row_t + Pl::COL_O + gam * NCOL + team * TCOL, o);
    float* redf = reinterpret_cast<float*>(smem + Pl::OFF_RED) + team * 256;  // [4 warps][64]: l[HT], then zacc[NGB][HT]
#pragma unroll
    for (int h = 0; h < HT; ++h) {
      float v = l[h];
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
      if (lane == 0) redf[qw * 64 + h] = v;
#pragma unroll
      for (int gi = 0; gi < NGB; ++gi) {
        float z = zacc[gi][h];
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) z += __shfl_xor_sync(0xffffffffu, z, s);
        if (lane == 0) redf[qw * 64 + HT + gi * HT + h] = z;
      }
    }
    tc_wait_ld();
    bar_sync_team(bar_team);
    int Erow = Ev[0];
#pragma unroll
    for (int gi = 1; gi < NGB; ++gi) Erow = gi == gam ? Ev[gi] : Erow;
    const float unit = pow2i(Erow - FRAC_V);
#pragma unroll
    for (int h = 0; h < HT; ++h) {
      if (h0 + h < G) {
        const float T = fmaf(__uint2float_rn(o[4 * h + 2]), 65536.f, fmaf(__uint2float_rn(o[4 * h + 1]), 256.f, __uint2float_rn(o[4 * h])));
        const int zi = HT + gam * HT + h;
        const float zs = (redf[zi] + redf[64 + zi]) + (redf[128 + zi] + redf[192 + zi]);
        mst[(h0 + h) * MS + ctid] = fmaf(T, unit, zs);
        if (ctid == 0) {
          mst[(h0 + h) * MS + HD] = m[h];
          mst[(h0 + h) * MS + HD + 1] = (redf[h] + redf[64 + h]) + (redf[128 + h] + redf[192 + h]);
        }
      }
    }
  }

  // ---- all warps: combine the main state with the window state, write the partial, merge ----
  tc_fence_before();
  __syncthreads();
  if (p.late_wait) grid_dependency_wait();  // the preceding launch still reads and writes the scratch and its result
  const bool dead = dead_sm != 0;
  if (warp < 4 && !dead) {
    const int stride = p.ns_q;
    for (int h = 0; h < G; ++h) {
      const float m1 = mst[h * MS + HD], m2 = wst[h * MS + HD];
      const float M = fmaxf(m1, m2);  // finite: the packed range of this CTA is not empty
      const float f1 = ex2(m1 - M), f2 = ex2(m2 - M);
      const size_t hq = (size_t)b * dm.Hq + hk * G + h;
      p.part_acc[(hq * stride + split) * HD + tid] = fmaf(mst[h * MS + tid], f1, wst[h * MS + tid] * f2);
      if (tid == 0)
        *reinterpret_cast<float2*>(p.part_ml + (hq * stride + split) * 2) =
            make_float2(M, fmaf(mst[h * MS + HD + 1], f1, wst[h * MS + HD + 1] * f2));
    }
    ticket_merge(p, ns, stride, hk, b, &s_flag);
  }
  if (dead && tid == 0) {
    // leaving early: no copy of this CTA may still be in flight when its shared memory is released
    const int issued = tma_issued;
    for (int j = max(0, issued - NSTG); j < issued; ++j) {
      bool done = false;
      for (int it = 0; it < WAIT_LIMIT && !done; ++it) done = mbar_try_wait(bar_full + 8 * (j % NSTG), (j / NSTG) & 1);
    }
    atomicExch(p.status, 1);
  }
  __syncthreads();
  if (warp == W_MMA)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tbase), "r"(Pl::TM_COLS) : "memory");
}

template <int BK, int BV, int GS, int GP>
struct Variant {
  static constexpr bool SP = GP <= 4;
  // two teams of four compute warps where one CTA has the SM to itself (groups of 5..8 heads); with two CTAs per SM
  // two teams were measured slower on every shape (50 us against 40 us per launch at 32k, four heads)
  static constexpr int NT = GP == 8 ? 2 : 1;
  static constexpr int THREADS = (4 * NT + 3) * 32;
  static auto kernel() { return decode_umma_kernel<BK, BV, GS, GP, SP, NT>; }
};

template <int BK, int BV, int GS, int GP>
cudaError_t launch_gp(const DecodeParams& p, cudaStream_t st) {
  using Pl = Plan<BK, BV, GS, GP>;
  using Va = Variant<BK, BV, GS, GP>;
  auto kernel = Va::kernel();
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Pl::TOTAL);
    // the largest shared-memory carve-out: several CTAs of this size are to share an SM
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  return launch_dependent(kernel, dim3(p.n_ctas), dim3(Va::THREADS), (size_t)Pl::TOTAL, st, p);
}

template <int BK, int BV, int GS, int GP>
int ctas_per_sm_gp() {
  using Pl = Plan<BK, BV, GS, GP>;
  using Va = Variant<BK, BV, GS, GP>;
  auto kernel = Va::kernel();
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Pl::TOTAL) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  // Residency from the kernel's own figures (the occupancy calculator answers 1 for this kernel although two
  // CTAs do share an SM): registers, shared memory with the 1 KB the system keeps per CTA, threads.
  cudaFuncAttributes fa;
  int dev = 0, regs_sm = 0, smem_sm = 0, thr_sm = 0;
  if (cudaFuncGetAttributes(&fa, kernel) != cudaSuccess || cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&regs_sm, cudaDevAttrMaxRegistersPerMultiprocessor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&thr_sm, cudaDevAttrMaxThreadsPerMultiProcessor, dev) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  const int warps = Va::THREADS / 32;
  const int regs_cta = warps * ((fa.numRegs * 32 + 511) / 512 * 512);  // allocated per warp in units of 512
  const int smem_cta = (int)Pl::TOTAL + (int)fa.sharedSizeBytes + 1024;
  int n = regs_sm / regs_cta;
  if (smem_sm / smem_cta < n) n = smem_sm / smem_cta;
  if (thr_sm / Va::THREADS < n) n = thr_sm / Va::THREADS;
  const int by_tmem = 512 / (int)Pl::TM_COLS;  // a CTA beyond this would wait for tensor memory
  return n < by_tmem ? n : by_tmem;
}

template <int BK, int BV, int GS>
cudaError_t launch_t(const DecodeParams& p, cudaStream_t st) {
  if (p.dm.G == 1) return launch_gp<BK, BV, GS, 1>(p, st);
  if (p.dm.G <= 4) return launch_gp<BK, BV, GS, 4>(p, st);
  return launch_gp<BK, BV, GS, 8>(p, st);
}
template <int BK, int BV, int GS>
int ctas_per_sm_t(int G) {
  if (G == 1) return ctas_per_sm_gp<BK, BV, GS, 1>();
  if (G <= 4) return ctas_per_sm_gp<BK, BV, GS, 4>();
  return ctas_per_sm_gp<BK, BV, GS, 8>();
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
