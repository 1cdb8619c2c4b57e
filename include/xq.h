/* xq.h -- C ABI of the XQuant KV-cache library for NVIDIA B200 (sm_100a).
 *
 * The library keeps, for every transformer layer, a KV cache made of
 *   - a quantized region: 1- or 2-bit integer codes plus one fp16 scale and one
 *     fp16 zero-point per group (keys: one group per channel and run of
 *     `group_size` tokens; values: one group per token and run of `group_size`
 *     channels) -- the min-max group quantizer of Section 3.1 (Eq. 1-3) with
 *     the data-free calibration of Section 3.2 (Eq. 12);
 *   - a 16-bit residual window holding the most recent tokens unquantized
 *     (Section 4.1, residual length);
 * and, for each adjacent layer pair (2p, 2p+1) at or above the sharing start,
 * stores the integer codes once, in layer 2p, while both layers keep their own
 * scale and zero-point (Section 3.3.3 / 3.3.4 with group size G = 2 and dominant
 * layer k = 0; Algorithms 1 and 2).  The configuration also takes the paper's
 * other sharing patterns: groups of three and four layers, another dominant
 * layer, and a pair's codes merged by a weighted average (Tables group, gamma).
 *
 * Two operations form the hot path: xq_append_kv (window append, and
 * quantize-and-pack of every window block that fills) and xq_decode_attention
 * (one query per head against the packed cache plus the window);
 * xq_decode_step runs both for every layer of a model, xq_attention_chunk
 * takes several query tokens.
 *
 * Conventions that hold for every entry point:
 *   - "device" pointers are CUDA device addresses valid on the device that was
 *     current when xq_create ran; "host" pointers are ordinary host addresses.
 *   - The caller owns every device byte (inputs, outputs, the workspace) and the
 *     stream.  The library never allocates or frees device memory and never
 *     synchronizes the device, except where a function says otherwise.  All
 *     kernels are launched asynchronously on the given stream
 *     (a cudaStream_t passed as void*; NULL is the default stream).
 *     The decode and window-append kernels are launched as programmatic
 *     dependents: their thread blocks may be placed, and packed cache data that
 *     earlier calls completed may be fetched, while the preceding kernel in the
 *     stream is still running; they wait for that kernel to complete before
 *     they touch q, new tokens, the window, the split scratch or any output, so
 *     stream order holds for everything a caller can observe.
 *   - Every function returns XQ_OK (0) or a negative XQ_ERR_* code; a failing
 *     call leaves the cache unchanged.  Nothing is thrown across the boundary.
 *   - A cache handle is not thread-safe; use one host thread per handle.
 *   - 16-bit inputs, outputs and the residual window have the type io_dtype
 *     names: bfloat16 (XQ_BF16, where a comment below says "bfloat16" read
 *     "io_dtype") or IEEE half precision (XQ_F16).
 */
#ifndef XQ_H_
#define XQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define XQ_OK 0
#define XQ_ERR_CONFIG (-1)   /* invalid xq_config                                        */
#define XQ_ERR_ARG (-2)      /* null / misaligned pointer, layer or token count invalid   */
#define XQ_ERR_CAPACITY (-3) /* would exceed max_seq, or the workspace is too small       */
#define XQ_ERR_ORDER (-4)    /* a code-borrowing layer is ahead of the layer owning codes */
#define XQ_ERR_CUDA (-5)     /* a CUDA call failed; xq_last_cuda_error gives the code     */
#define XQ_ERR_NOMEM (-6)    /* host allocation failed                                    */
#define XQ_ERR_DEVICE (-7)   /* a kernel gave up a bounded wait (xq_check_device)         */

#define XQ_BF16 0 /* bfloat16 */
#define XQ_F16 1  /* IEEE half precision */

#define XQ_KERNEL_AUTO 0    /* tensor-core kernel when the shape allows it, else generic   */
#define XQ_KERNEL_GENERIC 1 /* scalar kernel: any supported shape, slow, used as cross-check */
/* Tensor-core kernel (tcgen05, integer operands): head_dim 128, group of <= 8 query
 * heads, layers that hold quantized tokens.  The products q_d * s_d (query times
 * key scale) and p_t * s_t (softmax numerator times value scale) enter the matrix
 * products as 21- and 23-bit fixed point relative to their largest member, the
 * accumulation is exact (32-bit integers), everything else is fp32. */
#define XQ_KERNEL_MMA 2

#define XQ_MEM_DEVICE 0
#define XQ_MEM_HOST 1

/* Problem statement of Algorithm 1 (inputs kq, vq, km, vm, eta[2]) plus the
 * group size and residual length of Section 4.1 and the tensor shapes. */
typedef struct xq_config {
  int32_t n_layers;     /* L >= 1                                                         */
  int32_t batch;        /* sequences, all of the same length                              */
  int32_t n_q_heads;    /* query heads; a multiple of n_kv_heads (GQA; equal = MHA)       */
  int32_t n_kv_heads;   /* KV heads; query head h reads KV head h / (n_q_heads/n_kv_heads) */
  int32_t head_dim;     /* D: 64 or 128                                                   */
  int32_t max_seq;      /* capacity in tokens per sequence                                */
  int32_t group_size;   /* g: tokens per key group, channels per value group; 32 or 64   */
  int32_t residual_len; /* R: window capacity; a multiple of g and of 32                  */
  int32_t kq, vq;       /* key / value layers [0,kq) / [0,vq) use 2 bits, the rest 1 bit
                           (Appendix E)                                                   */
  int32_t km, vm;       /* from layer km / vm on, layers share integer codes in groups
                           (Algorithm 1, dequantize loop: odd layer l reads the codes of
                           l-1); km = vm = n_layers: no sharing.  The layers of a sharing
                           group must have equal bit-width.                               */
  float eta1, eta2;     /* calibration parameter eta_B for B = 1, 2, in [0, 0.5] (Eq. 5)  */
  float sm_scale;       /* softmax scale; 0 selects 1/sqrt(head_dim)                      */
  int32_t n_splits;     /* sequence splits per (sequence, KV head) in decode; 0 = library
                           chooses; at most XQ_MAX_SPLITS                                 */
  int32_t io_dtype;     /* type of K, V, q, out and of the residual window: XQ_BF16 or
                           XQ_F16                                                         */
  int32_t kernel;       /* XQ_KERNEL_*                                                    */
  /* Cross-layer sharing pattern (Section 3.3.3, 3.3.4; ablations of Tables gamma and
   * group).  All zero selects the accelerated scheme of the paper's main results:
   * pairs, first layer dominant, its codes shared as they are. */
  int32_t share_group;    /* G: layers per sharing group, 2, 3 or 4; 0 = 2.  G = 2 follows
                             Algorithm 1 (layer l >= km pairs with its neighbour of the
                             other parity); G = 3, 4: contiguous groups counted from km
                             (vm), and (n_layers - km) % G == 0 is required (likewise vm) */
  int32_t share_dominant; /* k in [0, G): the group's layer whose codes all its layers read
                             (Section 3.3.4); the others keep scale and zero-point only.
                             A layer ahead of its dominant layer can decode only once that
                             layer has appended (xq_decode_step: pass a layer_order that
                             names the dominant layer first)                              */
  float gamma1;           /* weighted-average merging (Section 3.3.3, Appendix F), G = 2 and
                             k = 0 only: weight of the pair's second layer, in [0, 1];
                             gamma_0 = 1 - gamma1.  0: no merging.  Otherwise the second
                             layer's append quantizes its own block too and replaces the
                             pair's codes by round(gamma_0 e_0 + gamma1 e_1), ties to even
                             (evaluated in double precision); until then the block holds
                             the first layer's codes e_0                                  */
  int32_t delta_stats;    /* 1: every layer that reads another layer's codes also quantizes
                             its own blocks (codes not stored) and counts, per cache kind,
                             the elements by |own code - shared code| -- the statistic of
                             Section 3.3.1 (Figure delta) on the caller's own data, read
                             with xq_delta_histogram.  Costs the code computation the
                             accelerated scheme saves; 0 (default): off                  */
} xq_config;

#define XQ_MAX_SPLITS 256

typedef struct xq_cache xq_cache; /* opaque; owns host memory only */

/* Validates a configuration (rules above; head_dim % group_size == 0).
 * XQ_OK or XQ_ERR_CONFIG. */
int xq_config_check(const xq_config* cfg);

/* Device bytes xq_create needs for `cfg`: windows, scale / zero-point, codes of
 * code-owning layers, split-K partials and the host-staging area.  0 if invalid. */
size_t xq_workspace_bytes(const xq_config* cfg);

/* Creates a cache over the caller's device buffer `dev_workspace` (256-byte
 * aligned, at least xq_workspace_bytes(cfg) bytes, contents arbitrary).  The
 * buffer must outlive the handle and must not be written by the caller while
 * the handle lives.  Uses the current CUDA device.  All layers start empty. */
int xq_create(const xq_config* cfg, void* dev_workspace, size_t bytes, xq_cache** out);

/* Frees the host-side handle (and its timing events).  Device memory is the caller's. */
int xq_destroy(xq_cache* c);

/* All layers back to length 0.  No device work. */
int xq_reset(xq_cache* c);

/* Appends n_tokens >= 1 tokens to `layer` (Algorithm 1, quantize loop, with the
 * residual window of Section 4.1).  K, V: device, [batch, n_kv_heads, n_tokens,
 * head_dim] contiguous bfloat16, 16-byte aligned, read-only, must stay valid
 * until the stream has run the call.  Tokens enter the window; when the window
 * already holds R tokens and a further token arrives, that block of R tokens is
 * quantized (Eq. 1, 2, 12): scale and zero-point always, integer codes only if
 * the layer owns codes (Quantize), not if it borrows them (PseudoQuantize); with
 * gamma1 > 0 the second layer of a pair quantizes too and merges its codes into
 * the pair's (Appendix F), which needs the first layer's blocks in place.
 * After S tokens the window holds ((S-1) mod R)+1 tokens.  One kernel launch:
 * the quantize-and-pack launch also refills the window.
 * Errors: XQ_ERR_ARG, XQ_ERR_CAPACITY (S would exceed max_seq), XQ_ERR_ORDER (a
 * merging or difference-counting layer ahead of its dominant layer), XQ_ERR_CUDA. */
int xq_append_kv(xq_cache* c, int layer, const void* K, const void* V, int n_tokens, void* stream);

/* One decode query per head against everything cached in `layer` (Algorithm 1,
 * dequantize loop, followed by softmax attention): K_hat = codes * s_hat + z_hat
 * (Eq. 3 with the calibrated parameters of `layer`, codes of the pair's owning
 * layer), logits = sm_scale * q . K_hat over quantized then window tokens,
 * out = softmax(logits) . V_hat.  No mask.  q, out: device, [batch, n_q_heads,
 * head_dim] bfloat16, 16-byte aligned.  fp32 accumulation.
 * Errors: XQ_ERR_ARG (also: empty layer), XQ_ERR_ORDER (the owning layer holds
 * fewer quantized tokens than `layer`), XQ_ERR_CUDA. */
int xq_decode_attention(xq_cache* c, int layer, const void* q, void* out, void* stream);

/* Same as xq_decode_attention with out: device float32 [batch, n_q_heads,
 * head_dim] (the accumulator before the final rounding to bfloat16). */
int xq_decode_attention_f32(xq_cache* c, int layer, const void* q, float* out, void* stream);

/* Attention of the last n_q_tokens tokens of `layer` as queries (a prefill chunk,
 * or the prompt / output workload of Appendix D), causal inside the chunk: the
 * keys and values of these tokens are already in the cache (xq_append_kv), and
 * query token j (0 .. n_q_tokens - 1) attends to the tokens 0 .. S - n_q_tokens + j,
 * S the layer's length -- packed tokens through their codes, window tokens as they
 * are, exactly as xq_decode_attention does for the tokens it sees; n_q_tokens = 1
 * is xq_decode_attention.  q, out: device, [n_q_tokens, batch, n_q_heads, head_dim]
 * contiguous (token-major: one token's slice is a decode call's q), io_dtype;
 * 16-byte aligned.  The _f32 variant writes float results (tests).  Errors as
 * xq_decode_attention; 1 <= n_q_tokens <= S. */
int xq_attention_chunk(xq_cache* c, int layer, const void* q, void* out, int n_q_tokens, void* stream);
int xq_attention_chunk_f32(xq_cache* c, int layer, const void* q, float* out, int n_q_tokens, void* stream);

/* xq_decode_attention for callers that cannot provide scratch memory of their
 * own.  (The paper has no counterpart: this is a deployment variant, not part of
 * the method.)  Some hosts hand every byte of device memory to their own pools at
 * start-up and forbid cudaMalloc afterwards -- an inference server that runs this
 * library as a plug-in, a real-time loop that must not enter the allocator, a
 * process whose memory budget was fixed before this library was loaded.  Such a
 * caller still passes q and out (device, [batch, n_q_heads, head_dim] bfloat16,
 * 16-byte aligned) but the split-K partials and merge tickets, which
 * xq_decode_attention keeps in the caller's workspace, live here in a
 * XQ_STATIC_SCRATCH_BYTES array that is part of the library image: every GPU
 * that the library's image is loaded on holds that much device memory until the
 * process exits.  The call allocates and frees nothing, on the host side of CUDA
 * or through any library.  Result: identical to xq_decode_attention.
 * Limits: the partials of the call (batch * n_q_heads * splits * (head_dim + 2)
 * floats, plus one ticket per (sequence, kv head) and a status word) must fit the array, else
 * XQ_ERR_CAPACITY and nothing is launched; a smaller n_splits in xq_config
 * shrinks them.  The array is shared by every handle and every call on a device
 * and keeps the previous call's contents; the call clears the part that must
 * start at zero (the tickets) on `stream` before its kernel.  Two such calls
 * whose kernels may overlap on the GPU (different streams without an ordering
 * between them) race on the array: keep them on one stream or order them.
 * xq_create looks up the array's device address (a short synchronous CUDA
 * runtime query that also makes the driver place the library's image, the array
 * included, on the device: create the handle at start-up, before the host fills
 * its pools and outside any stream capture); the call itself only checks that
 * the current device is the handle's (else XQ_ERR_ARG).  Unlike
 * xq_decode_attention this call never fetches packed data ahead of the kernel
 * that precedes it in the stream.  Other errors as xq_decode_attention. */
#define XQ_STATIC_SCRATCH_BYTES (8u << 20)
int xq_decode_attention_static(xq_cache* c, int layer, const void* q, void* out, void* stream);

/* One decode step of a whole model: for each layer, append one token and run
 * decode attention.  K_new, V_new: [n_layers, batch, n_kv_heads, 1, head_dim];
 * q, out: [n_layers, batch, n_q_heads, head_dim]; bfloat16; slice l belongs to
 * layer l.  layer_order: host array of n_layers distinct layer indices giving
 * the order in which layers are processed, or NULL for ascending order; a
 * code-owning layer must come before the layer that borrows its codes.
 * mem = XQ_MEM_DEVICE: device pointers, used in place.
 * mem = XQ_MEM_HOST: host pointers (pinned memory for the copies to be
 * asynchronous); inputs are copied to the workspace's staging area on `stream`,
 * the result is copied back to `out` on `stream`; the caller synchronizes the
 * stream before reading `out` or reusing the host buffers.
 * The result equals xq_append_kv followed by xq_decode_attention per layer, bit
 * for bit; where the tensor-core kernel serves the layer and the token fills no
 * window block, that kernel stores the token into the window itself (one launch
 * per layer); on the step on which every layer's window block fills (all layers
 * of equal length, no merging or difference counting), one quantize-and-pack
 * launch serves all layers before the decode launches.  K_new and V_new must
 * stay unchanged until the step's kernels have run.  The tensor-core decode
 * launches of a step overlap: the first waits for all earlier work in `stream`
 * before it reads anything; each later one starts while its predecessor still
 * runs, reads at once (everything before the first launch is complete by then,
 * and a decode launch writes only its own window row, scratch and result) and
 * waits for the predecessor before its own first write to scratch or result.
 * Every layer's capacity, order and kernel are checked before the first copy or
 * launch: a call refused with XQ_ERR_ARG / CAPACITY / ORDER / CONFIG changes
 * nothing.  After XQ_ERR_CUDA the cache's state is undefined. */
int xq_decode_step(xq_cache* c, const void* K_new, const void* V_new, const void* q, void* out,
                   const int32_t* layer_order, int mem, void* stream);

/* Waits for `stream` and reports whether a kernel launched through this handle
 * gave up one of its bounded waits (XQ_ERR_DEVICE; the outputs of that call are
 * then invalid and the handle should be reset) -- every wait inside the kernels
 * has an iteration limit instead of the ability to hang the GPU.  XQ_OK otherwise.
 * Synchronizes; not for the hot path. */
int xq_check_device(xq_cache* c, void* stream);

/* Code-similarity statistic of Section 3.3.1 (needs delta_stats = 1 in the
 * configuration): counts[d], d = 0..3, is the number of quantized elements of
 * `layer` (kind 0: keys, 1: values; all sequences and heads, every block packed
 * since xq_create or xq_reset) whose own code differs by d from the code it reads
 * from its group's dominant layer (before any merging of that block).  Zero for a
 * layer that keeps its own codes.  Waits for `stream`; not for the hot path.
 * XQ_ERR_CONFIG without delta_stats. */
int xq_delta_histogram(xq_cache* c, int layer, int kind, unsigned long long counts[4], void* stream);

/* Equivalent bit-width of Appendix C: stored code bits per cached element,
 * averaged over layers and over keys and values; scale / zero-point excluded,
 * a code-borrowing layer counts zero.  Negative if cfg is invalid. */
double xq_equiv_bits(const xq_config* cfg);

/* Tokens cached in `layer` (negative error code on bad arguments). */
int xq_seq_len(const xq_cache* c, int layer);
/* Of those, tokens in the quantized region (a multiple of residual_len). */
int xq_quantized_len(const xq_cache* c, int layer);
/* Splits per (sequence, kv head) stream (quantized-region, window) the next decode
 * call on `layer` would use; where the library's own choice gives some streams one
 * split more than others to fill the GPU, the larger number. */
int xq_split_plan(const xq_cache* c, int layer, int* n_splits_quantized, int* n_splits_window);

/* Where a layer's data lives inside the workspace, for tests and snapshots.
 * which: 0 key codes, 1 value codes (of the layer that owns them), 2 key
 * scale/zero, 3 value scale/zero, 4 key window, 5 value window.  Returns byte
 * offset from the workspace start and the byte stride between consecutive
 * (sequence, kv head) streams.
 * Layouts (all little-endian, one stream per (sequence, kv head); bit map and
 * index functions: csrc/xq_layout.cuh):
 *   key codes: per 32 tokens [chunk][token][<= 16 bytes] of the tokens' rows;
 *   value codes: per 128 tokens [chunk][channel][16 bytes] of the channels' rows
 *     (the words of a last, partly filled batch that no token has reached yet are
 *     undefined);
 *   key scale/zero: per token group [2][head_dim] fp16 (scales, then zero-points),
 *     channel d at index (d % 32) * (head_dim / 32) + d / 32;
 *   value scale/zero: per token [2][head_dim/group_size] fp16;
 *   windows: [R][head_dim] bfloat16. */
int xq_region(const xq_cache* c, int layer, int which, size_t* offset, size_t* stream_stride);

/* Kernel launches issued through this handle since creation (all kinds). */
long long xq_launch_count(const xq_cache* c);

/* Optional per-kernel timing with CUDA events recorded on the launching stream
 * around each kernel.  xq_timing_enable(c, 1) allocates an event pool (host
 * call, not on the hot path) and clears the records; (c, 0) stops recording.
 * xq_timing_read synchronizes on the recorded events and returns, per kind
 * (0 decode split kernel, 1 merge kernel, 2 quantize-and-pack kernel, 3 window
 * append kernel), the launch count and total milliseconds. */
int xq_timing_enable(xq_cache* c, int on);
int xq_timing_read(xq_cache* c, int kind, int* launches, double* total_ms);

/* CUDA error code (cudaError_t) of the last XQ_ERR_CUDA on this handle, else 0. */
int xq_last_cuda_error(const xq_cache* c);

/* Static text for an XQ_* code. */
const char* xq_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* XQ_H_ */
