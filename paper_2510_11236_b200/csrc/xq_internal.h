// Internal declarations shared by the host state machine and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace xq {

struct Dims {
  int B, Hq, Hkv, G, D, g, R, NG;
  int nq_cap;  // capacity of the quantized region in tokens, padded to whole 128-token batches
};

// Device addresses of one layer's regions (codes: of the layer that owns them).
struct LayerPtrs {
  uint16_t* win_k;   // [B,Hkv,R,D] bf16
  uint16_t* win_v;
  uint16_t* k_meta;  // [B,Hkv,nq_cap/g,2,D] fp16 (per token group: scales, then zero-points)
  uint16_t* v_meta;  // [B,Hkv,nq_cap,2,NG] fp16 (per token: scales, then zero-points)
  uint32_t* k_codes; // [B,Hkv,nq_cap*D*bk/32]
  uint32_t* v_codes;
  int bk, bv;
};

// One layer of a quantize-and-pack launch.
struct PackLayer {
  LayerPtrs L;
  const uint16_t* K_in;  // [B,Hkv,n_in,D] new tokens (absolute positions s_old ..)
  const uint16_t* V_in;
  // codes of a cache kind: 0 = none (the layer keeps scale and zero-point only), 1 = written, 2 = merged into the
  // codes the dominant layer wrote (weighted average, Appendix F); 4 = computed for the statistic only; 6 = both
  int own_k, own_v;
  float eta_k, eta_v;
  // with bit 2 set in own_*: count the elements by |own code - stored code| into these four counters (before the
  // codes are merged, if they are)
  unsigned long long* delta_k;
  unsigned long long* delta_v;
};

constexpr int PACK_MAX_LAYERS = 32;  // layers one launch can take (they share every length below)

struct PackParams {
  Dims dm;
  int n_layers;
  int n_in;
  int s_old;     // tokens cached before this append
  int nq_old;    // quantized tokens before this append
  int n_blocks;  // R-token blocks to quantize, starting at absolute token nq_old
  int tb;        // tokens per CTA tile (32 or 64)
  int f16;       // inputs and window are IEEE half precision (else bfloat16)
  // tokens nq_new .. s_new - 1 of the input go into window rows 0 .. win_count - 1 (the CTAs that staged those rows
  // of the old window copy them); 0: the caller copies
  int win_count;
  int nq_new;
  // merged code of (e0, e1) at bits 2 * (4 e0 + e1), for 1-bit and 2-bit codes
  uint32_t merge_lut[2];
  PackLayer layer[PACK_MAX_LAYERS];
};

struct WindowParams {
  Dims dm;
  LayerPtrs L;
  const uint16_t* K_in;
  const uint16_t* V_in;
  int n_in;
  int s_old;
  int first;   // first absolute token to copy
  int count;   // tokens to copy
  int nq_new;  // window slot = absolute token - nq_new
};

struct DecodeParams {
  Dims dm;
  LayerPtrs L;
  const uint16_t* q;  // [B,Hq,D] bf16
  int n_q;            // quantized tokens
  int r;              // window tokens
  int ns_q, ns_w;     // splits over the quantized region (most of any stream) / over the window
  int n_ctas;         // tensor-core kernel: CTAs over all streams (n_ctas / streams splits per stream, or one more)
  float scale;
  float* part_acc;    // [B,Hq,ns,D]
  float* part_ml;     // [B,Hq,ns,2]  (running max in log2 units, sum)
  // used by kernels that merge the partials themselves (last CTA of a stream):
  void* out;              // [B,Hq,D] bf16 or f32
  int out_f32;
  unsigned int* tickets;  // [B*Hkv], zero between launches
  // 1: the packed streams were complete before the preceding kernel in the stream started, so their first
  // copies may be issued before this kernel has waited for that kernel (programmatic dependent launch)
  int early_fetch;
  // 1: the preceding kernel in the stream is a decode launch of the same call that itself started only after all
  // earlier work in the stream had completed, so nothing this launch reads is still being written: it reads at
  // once and waits for that launch only before its first write that the launch could see (partials, tickets,
  // result, status).  Implies early_fetch.
  int late_wait;
  // Fused append of one token per stream (tensor-core kernel with quantized tokens only; else null): the newest
  // window row, index r - 1, is not in the window yet but here, [B,Hkv,D] bf16.  The CTA whose share of the
  // window holds that row reads it from here and stores it into the window.
  const uint16_t* K_new;
  const uint16_t* V_new;
  int* status;  // device word the tensor-core kernel sets when one of its bounded waits gave up
  int f16;      // q, the window and the 16-bit output are IEEE half precision (else bfloat16)
};

struct MergeParams {
  Dims dm;
  int ns;
  int f16;
  const float* part_acc;
  const float* part_ml;
  void* out;
  int out_f32;
};

// Part `part` of `parts` nearly equal shares of n items: [lo, hi), sizes differ by at most one.
// (32-bit arithmetic: a 64-bit division costs a device thread hundreds of instructions.)
__host__ __device__ inline void share_of(int n, int parts, int part, int& lo, int& hi) {
  const unsigned base = (unsigned)n / (unsigned)parts, rem = (unsigned)n - base * (unsigned)parts;
  lo = (int)((unsigned)part * base + ((unsigned)part < rem ? (unsigned)part : rem));
  hi = lo + (int)base + ((unsigned)part < rem ? 1 : 0);
}

// Programmatic dependent launch (sm_90 and later).  A kernel launched with launch_dependent() may start while
// the preceding kernel in the stream is still running, provided that kernel has called grid_dependents_go() (or
// when it ends); it must call grid_dependency_wait() before it touches anything the preceding kernels wrote or
// still read.  After the wait all earlier work in the stream is complete and visible, as at a kernel boundary.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void grid_dependents_go() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

template <typename P>
cudaError_t launch_dependent(void (*kernel)(P), dim3 grid, dim3 block, size_t smem, cudaStream_t st, const P& params) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, params);
}
#endif

cudaError_t launch_pack(const PackParams& p, cudaStream_t st);
cudaError_t launch_window_append(const WindowParams& p, cudaStream_t st);
cudaError_t launch_decode_generic(const DecodeParams& p, cudaStream_t st);
cudaError_t launch_decode_mma(const DecodeParams& p, cudaStream_t st);
bool decode_mma_supported(const Dims& dm, int bk, int bv);
int decode_mma_ctas_per_sm(const Dims& dm, int bk, int bv);
cudaError_t launch_merge(const MergeParams& p, cudaStream_t st);

}  // namespace xq
