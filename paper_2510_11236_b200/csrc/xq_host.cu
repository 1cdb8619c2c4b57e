// Host side of the library: configuration checks, workspace carving, the
// per-layer sequence counters (Algorithm 1's bookkeeping), split planning and
// the C entry points.  No device memory is allocated here.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../include/xq.h"
#include "xq_internal.h"
#include "xq_layout.cuh"

using namespace xq;

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline int layer_bits(int l, int q) { return l < q ? 2 : 1; }

// The layer whose integer codes layer l reads (l itself when it keeps its own), for one cache kind with sharing
// from layer m on.  Groups of two follow Algorithm 1's dequantize loop (the layers of a pair differ in parity;
// the dominant one has parity k), larger groups are contiguous runs counted from m (Section 3.3.4, Table group).
inline int code_owner(int l, int m, int group, int k) {
  if (l < m) return l;
  if (group == 2) return l - (l % 2) + k;
  return l - (l - m) % group + k;
}
inline int share_group_of(const xq_config* c) { return c->share_group == 0 ? 2 : c->share_group; }
inline int k_owner(const xq_config* c, int l) { return code_owner(l, c->km, share_group_of(c), c->share_dominant); }
inline int v_owner(const xq_config* c, int l) { return code_owner(l, c->vm, share_group_of(c), c->share_dominant); }
// Weighted-average merging (Appendix F): the pair's second layer rewrites the shared codes of a cache kind
inline bool merges_codes(const xq_config* c, int l, int m) { return c->gamma1 > 0.f && l >= m && (l % 2) == 1; }

struct LayerRegions {
  size_t win_k, win_v, k_meta, v_meta, k_codes, v_codes;  // byte offsets; codes: of the owning layer
  size_t stride[6];                                       // per (sequence, kv head) stream, bytes
};

struct Plan {
  Dims dm;
  std::vector<LayerRegions> layers;
  size_t part_acc, part_ml, tickets, status, delta, staging, total;
  size_t staging_kv_bytes, staging_q_bytes;
};

bool check(const xq_config* c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1) return false;
  if (c->n_q_heads % c->n_kv_heads) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->group_size != 32 && c->group_size != 64) return false;
  if (c->head_dim % c->group_size) return false;
  if (c->residual_len < 32 || c->residual_len % c->group_size || c->residual_len % 32) return false;
  if (c->residual_len > 4096) return false;
  if (c->max_seq < 1) return false;
  if (c->kq < 0 || c->kq > c->n_layers || c->vq < 0 || c->vq > c->n_layers) return false;
  if (c->km < 0 || c->km > c->n_layers || c->vm < 0 || c->vm > c->n_layers) return false;
  if (!(c->eta1 >= 0.f && c->eta1 <= 0.5f) || !(c->eta2 >= 0.f && c->eta2 <= 0.5f)) return false;
  if (!(c->sm_scale >= 0.f) || isinf(c->sm_scale)) return false;
  if (c->n_splits < 0 || c->n_splits > XQ_MAX_SPLITS) return false;
  if (c->io_dtype != XQ_BF16 && c->io_dtype != XQ_F16) return false;
  if (c->kernel < XQ_KERNEL_AUTO || c->kernel > XQ_KERNEL_MMA) return false;
  const int group = share_group_of(c);
  if (group < 2 || group > 4) return false;
  if (c->share_dominant < 0 || c->share_dominant >= group) return false;
  if (!(c->gamma1 >= 0.f && c->gamma1 <= 1.f)) return false;
  if (c->gamma1 > 0.f && (group != 2 || c->share_dominant != 0)) return false;
  if (c->delta_stats != 0 && c->delta_stats != 1) return false;
  if (group > 2 && ((c->n_layers - c->km) % group || (c->n_layers - c->vm) % group)) return false;
  // every layer reads the codes of a layer that exists and has its bit-width
  for (int l = 0; l < c->n_layers; ++l) {
    const int ok = k_owner(c, l), ov = v_owner(c, l);
    if (ok < 0 || ok >= c->n_layers || ov < 0 || ov >= c->n_layers) return false;
    if (layer_bits(l, c->kq) != layer_bits(ok, c->kq) || layer_bits(l, c->vq) != layer_bits(ov, c->vq)) return false;
  }
  return true;
}

void make_plan(const xq_config* c, Plan& pl) {
  Dims& dm = pl.dm;
  dm.B = c->batch; dm.Hq = c->n_q_heads; dm.Hkv = c->n_kv_heads; dm.G = dm.Hq / dm.Hkv;
  dm.D = c->head_dim; dm.g = c->group_size; dm.R = c->residual_len; dm.NG = dm.D / dm.g;
  // quantized tokens never exceed ((max_seq - 1) / R) * R; the regions hold whole 128-token batches
  dm.nq_cap = padded_capacity(c->max_seq > 1 ? ((c->max_seq - 1) / dm.R) * dm.R : 0);
  const size_t BH = (size_t)dm.B * dm.Hkv;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  pl.layers.resize(c->n_layers);
  for (int l = 0; l < c->n_layers; ++l) {
    LayerRegions& r = pl.layers[l];
    int bk = layer_bits(l, c->kq), bv = layer_bits(l, c->vq);
    r.stride[4] = r.stride[5] = (size_t)dm.R * dm.D * 2;
    r.win_k = take(BH * r.stride[4]);
    r.win_v = take(BH * r.stride[5]);
    r.stride[2] = (size_t)(dm.nq_cap / dm.g) * 2 * dm.D * 2;
    r.stride[3] = (size_t)dm.nq_cap * 2 * dm.NG * 2;
    r.k_meta = take(BH * r.stride[2]);
    r.v_meta = take(BH * r.stride[3]);
    r.stride[0] = (size_t)dm.nq_cap * dm.D * bk / 8;
    r.stride[1] = (size_t)dm.nq_cap * dm.D * bv / 8;
    r.k_codes = k_owner(c, l) == l ? take(BH * r.stride[0]) : 0;
    r.v_codes = v_owner(c, l) == l ? take(BH * r.stride[1]) : 0;
  }
  for (int l = 0; l < c->n_layers; ++l) {  // the other layers of a group read the dominant layer's codes
    if (k_owner(c, l) != l) pl.layers[l].k_codes = pl.layers[k_owner(c, l)].k_codes;
    if (v_owner(c, l) != l) pl.layers[l].v_codes = pl.layers[v_owner(c, l)].v_codes;
  }
  pl.part_acc = take((size_t)dm.B * dm.Hq * XQ_MAX_SPLITS * dm.D * 4);
  pl.part_ml = take((size_t)dm.B * dm.Hq * XQ_MAX_SPLITS * 2 * 4);
  pl.tickets = take(BH * 4);
  pl.status = take(4);
  pl.delta = take((size_t)c->n_layers * 2 * 4 * 8);  // per layer and cache kind: elements by code difference 0..3
  pl.staging_kv_bytes = (size_t)c->n_layers * BH * dm.D * 2;
  pl.staging_q_bytes = (size_t)c->n_layers * dm.B * dm.Hq * dm.D * 2;
  pl.staging = take(2 * align_up(pl.staging_kv_bytes, 256) + 2 * align_up(pl.staging_q_bytes, 256));
  pl.total = off;
}

constexpr int N_KINDS = 4;
constexpr int TIMING_POOL = 1 << 15;

struct EventPair { cudaEvent_t a, b; int kind; };

}  // namespace

// Scratch of xq_decode_attention_static: part of the library image, one copy per
// GPU that loads it.  In host code this name is only a handle for the runtime's
// symbol table, never a device address: kernels get the address that
// cudaGetSymbolAddress returns for the current device.
static __device__ __align__(256) unsigned char g_static_scratch[XQ_STATIC_SCRATCH_BYTES];

namespace {

// Device address of g_static_scratch on the current device (a synchronous runtime query that also makes the
// driver load this module's image, array included, on that device).
cudaError_t static_scratch_address(uint8_t** out) {
  void* p = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
  if (e != cudaSuccess) return e;
  if (!p || ((uintptr_t)p & 255)) return cudaErrorInvalidSymbol;
  *out = (uint8_t*)p;
  return cudaSuccess;
}

}  // namespace

struct xq_cache {
  xq_config cfg;
  Plan plan;
  uint8_t* ws;
  std::vector<int> seq;  // tokens cached per layer
  long long launches;
  int last_cuda;
  float scale;
  int sm_count;
  int device;            // CUDA device the handle was created on (-1: none)
  uint8_t* static_base;  // device address of the library's static scratch array on that device (null: not resolved)
  bool tickets_clean;  // the ticket counters have been zeroed on a stream
  bool delta_clean;    // the code-difference counters have been zeroed on a stream
  std::vector<uint8_t> repacked;  // per layer: codes or parameters it reads were written since its last decode
  int mma_ctas[2][2];  // resident CTAs per SM of the tensor-core kernel by (key bits - 1, value bits - 1); 0 = not asked yet
  // timing
  bool timing;
  std::vector<EventPair> pool;
  size_t used;
};

namespace {

inline int residual_count(int S, int R) { return S > 0 ? ((S - 1) % R) + 1 : 0; }

LayerPtrs layer_ptrs(const xq_cache* c, int l) {
  const LayerRegions& r = c->plan.layers[l];
  LayerPtrs p;
  p.win_k = (uint16_t*)(c->ws + r.win_k);
  p.win_v = (uint16_t*)(c->ws + r.win_v);
  p.k_meta = (uint16_t*)(c->ws + r.k_meta);
  p.v_meta = (uint16_t*)(c->ws + r.v_meta);
  p.k_codes = (uint32_t*)(c->ws + r.k_codes);
  p.v_codes = (uint32_t*)(c->ws + r.v_codes);
  p.bk = layer_bits(l, c->cfg.kq);
  p.bv = layer_bits(l, c->cfg.vq);
  return p;
}

// Bytes one quantized token / one window token costs a (sequence, kv head) stream.
void token_bytes(const xq_cache* c, int l, double& q_bytes, double& w_bytes) {
  const Dims& dm = c->plan.dm;
  int bk = layer_bits(l, c->cfg.kq), bv = layer_bits(l, c->cfg.vq);
  q_bytes = dm.D * (bk + bv) / 8.0 + 4.0 * dm.D / dm.g + 4.0 * dm.NG;
  w_bytes = 4.0 * dm.D;
}

bool layer_uses_mma(const xq_cache* c, int l) {
  if (c->cfg.kernel == XQ_KERNEL_GENERIC) return false;
  return decode_mma_supported(c->plan.dm, layer_bits(l, c->cfg.kq), layer_bits(l, c->cfg.vq));
}

int mma_ctas_per_sm(const xq_cache* c, int l) {
  int bk = layer_bits(l, c->cfg.kq), bv = layer_bits(l, c->cfg.vq);
  int& slot = const_cast<xq_cache*>(c)->mma_ctas[bk - 1][bv - 1];
  if (slot == 0) {
    slot = decode_mma_ctas_per_sm(c->plan.dm, bk, bv);
    if (slot <= 0) slot = 2;  // no device to ask
  }
  return slot;
}

// Splits per (sequence, kv head) stream.  Tensor-core kernel (layers with quantized
// tokens): every split takes whole batches of the packed region and a share of the
// window (ns_w = 0), sized towards whole waves of resident CTAs.  Generic kernel:
// separate splits for the packed region and for the window, in proportion to their bytes.
// nq packed tokens and r window tokens are visible to the call.
void plan_splits(const xq_cache* c, int l, int nq, int r, int& ns_q, int& ns_w, int* n_ctas_out = nullptr) {
  const Dims& dm = c->plan.dm;
  int units = (nq + 31) / 32, tiles = (r + 15) / 16;
  const int streams = dm.B * dm.Hkv;
  if (layer_uses_mma(c, l) && nq > 0) {
    // the tensor-core kernel: whole 128-token batches per CTA, every CTA also takes a share of the window
    const int batches = (nq + XQ_BATCH - 1) / XQ_BATCH;
    ns_w = 0;
    if (c->cfg.n_splits > 0) {
      ns_q = c->cfg.n_splits < batches ? c->cfg.n_splits : batches;
      if (n_ctas_out) *n_ctas_out = ns_q * streams;
      return;
    }
    const long long slot_count = (long long)c->sm_count * mma_ctas_per_sm(c, l);
    int best = 1;
    double best_score = -1.0;
    for (int ns = 1; ns <= XQ_MAX_SPLITS && ns <= batches; ++ns) {
      double ctas = (double)ns * streams;
      double waves = ceil(ctas / (double)slot_count);
      double fill = ctas / (waves * (double)slot_count);
      double bpc = (double)batches / ns;         // batches per CTA
      double score = fill * bpc / (bpc + 5.0);   // ~5 batches' worth of fixed cost per CTA
      if (score > best_score) { best_score = score; best = ns; }
    }
    ns_q = best;
    if (n_ctas_out) *n_ctas_out = best * streams;
    // One wave that does not fill every resident slot: give some streams one split more, if the splits are many
    // enough for the CTAs' sizes to stay within a few percent of each other.
    if ((long long)best * streams < slot_count && slot_count < (long long)(best + 1) * streams && best >= 8 &&
        best + 1 <= batches && best + 1 <= XQ_MAX_SPLITS) {
      ns_q = best + 1;
      if (n_ctas_out) *n_ctas_out = (int)slot_count;
    }
    return;
  }
  double qb, wb;
  token_bytes(c, l, qb, wb);
  double bytes_q = qb * nq, bytes_w = wb * r;
  int total;
  if (c->cfg.n_splits > 0) {
    total = c->cfg.n_splits;
  } else {
    double per_stream = bytes_q + bytes_w;
    int want = (int)ceil(per_stream / 49152.0);
    if (want < 1) want = 1;
    long long ctas = (long long)want * streams;
    long long wave = 2LL * c->sm_count;
    if (ctas > wave) {
      long long waves = (ctas + wave / 2) / wave;
      if (waves < 1) waves = 1;
      want = (int)((waves * wave) / streams);
      if (want < 1) want = 1;
    }
    total = want;
  }
  if (total > XQ_MAX_SPLITS) total = XQ_MAX_SPLITS;
  if (units == 0) {
    ns_q = 0;
    ns_w = total < tiles ? total : tiles;
    if (ns_w < 1) ns_w = 1;
    return;
  }
  int w = (int)floor(total * bytes_w / (bytes_q + bytes_w) + 0.5);
  if (w < 1) w = 1;
  if (w > tiles) w = tiles;
  int q = total - w;
  if (q < 1) q = 1;
  if (q > units) q = units;
  ns_q = q;
  ns_w = w;
}

struct Timer {
  xq_cache* c; cudaStream_t st; EventPair* ev;
  Timer(xq_cache* c_, cudaStream_t st_, int kind) : c(c_), st(st_), ev(nullptr) {
    if (c->timing && c->used < c->pool.size()) {
      ev = &c->pool[c->used++];
      ev->kind = kind;
      cudaEventRecord(ev->a, st);
    }
  }
  ~Timer() { if (ev) cudaEventRecord(ev->b, st); }
};

int fail_cuda(xq_cache* c, cudaError_t e) { c->last_cuda = (int)e; return XQ_ERR_CUDA; }

// Where the split-K partials, the merge tickets and the kernel status word of a decode call live.
struct Scratch {
  float* part_acc;
  float* part_ml;
  unsigned int* tickets;
  int* status;
};

// Checks a decode call and fills the kernel parameters (everything but the scratch).  Touches no state.
// K_new / V_new: one new token per stream that the tensor-core kernel appends itself; S_eff is the layer's
// length with that token counted.  vis >= 0: only the first vis tokens are visible to the query (a query token of
// a chunk that is followed by later tokens in the cache).
int prepare_decode(const xq_cache* c, int layer, const void* q, void* out, int out_f32, const void* K_new,
                   const void* V_new, int S_eff, DecodeParams& p, bool& use_mma, int vis = -1) {
  if (!c || !q || !out) return XQ_ERR_ARG;
  if (layer < 0 || layer >= c->cfg.n_layers) return XQ_ERR_ARG;
  if (((uintptr_t)q & 15) || ((uintptr_t)out & 15)) return XQ_ERR_ARG;
  if (((uintptr_t)K_new & 15) || ((uintptr_t)V_new & 15)) return XQ_ERR_ARG;
  const Dims& dm = c->plan.dm;
  const int S = S_eff;
  if (S < 1) return XQ_ERR_ARG;
  int r = residual_count(S, dm.R), nq = S - r;
  if (vis >= 0) {
    if (vis < 1 || vis > S) return XQ_ERR_ARG;
    if (vis < nq) { nq = vis; r = 0; } else { r = vis - nq; }
  }
  // a code-borrowing layer needs the owning layer's codes for all of its quantized tokens
  for (int o : {k_owner(&c->cfg, layer), v_owner(&c->cfg, layer)}) {
    if (o != layer && c->seq[o] - residual_count(c->seq[o], dm.R) < nq) return XQ_ERR_ORDER;
  }
  use_mma = layer_uses_mma(c, layer) && nq > 0;
  if (c->cfg.kernel >= XQ_KERNEL_MMA && !layer_uses_mma(c, layer)) return XQ_ERR_CONFIG;
  if (K_new && !use_mma) return XQ_ERR_ARG;
  p.dm = dm;
  p.L = layer_ptrs(c, layer);
  p.q = (const uint16_t*)q;
  p.n_q = nq;
  p.r = r;
  p.n_ctas = 0;
  plan_splits(c, layer, nq, r, p.ns_q, p.ns_w, &p.n_ctas);
  p.scale = c->scale;
  p.out = out;
  p.out_f32 = out_f32;
  p.early_fetch = 0;
  p.late_wait = 0;
  p.f16 = c->cfg.io_dtype == XQ_F16;
  p.K_new = (const uint16_t*)K_new;
  p.V_new = (const uint16_t*)V_new;
  return XQ_OK;
}

// Launches a prepared decode call.  The tensor-core kernel merges its partials itself.
int launch_decode(xq_cache* c, DecodeParams& p, bool use_mma, const Scratch& s, cudaStream_t st) {
  p.part_acc = s.part_acc;
  p.part_ml = s.part_ml;
  p.tickets = s.tickets;
  p.status = s.status;
  cudaError_t e;
  {
    Timer t(c, st, 0);
    e = use_mma ? launch_decode_mma(p, st) : launch_decode_generic(p, st);
  }
  c->launches++;
  if (e != cudaSuccess) return fail_cuda(c, e);
  if (use_mma) return XQ_OK;
  MergeParams m;
  m.dm = p.dm;
  m.ns = p.ns_q + p.ns_w;
  m.f16 = p.f16;
  m.part_acc = p.part_acc;
  m.part_ml = p.part_ml;
  m.out = p.out;
  m.out_f32 = p.out_f32;
  {
    Timer t(c, st, 1);
    e = launch_merge(m, st);
  }
  c->launches++;
  if (e != cudaSuccess) return fail_cuda(c, e);
  return XQ_OK;
}

Scratch workspace_scratch(const xq_cache* c) {
  Scratch s;
  s.part_acc = (float*)(c->ws + c->plan.part_acc);
  s.part_ml = (float*)(c->ws + c->plan.part_ml);
  s.tickets = (unsigned int*)(c->ws + c->plan.tickets);
  s.status = (int*)(c->ws + c->plan.status);
  return s;
}

// The ticket counters and the status word start at zero: cleared once per handle on the first stream used.
int ensure_clean_scratch(xq_cache* c, cudaStream_t st) {
  if (c->tickets_clean) return XQ_OK;
  const Dims& dm = c->plan.dm;
  cudaError_t e = cudaMemsetAsync(c->ws + c->plan.tickets, 0, (size_t)dm.B * dm.Hkv * 4, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + c->plan.status, 0, 4, st);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->tickets_clean = true;
  return XQ_OK;
}

// Merged code of (e0, e1) for every pair of B-bit codes, at bits 2 * (4 e0 + e1): round(gamma_0 e0 + gamma_1 e1) in
// double precision, ties to even (Appendix F).
uint32_t merge_table(float gamma1, int bits) {
  const double g1 = (double)gamma1, g0 = 1.0 - g1;
  uint32_t lut = 0u;
  for (int e0 = 0; e0 < (1 << bits); ++e0)
    for (int e1 = 0; e1 < (1 << bits); ++e1) {
      const double v = g0 * (double)e0 + g1 * (double)e1;
      lut |= ((uint32_t)nearbyint(v) & 3u) << (2 * (4 * e0 + e1));
    }
  return lut;
}

// One quantize-and-pack launch for `n` layers of equal length that each receive n_tokens new tokens (layer i's at
// K + i * layer_stride bytes), at least one window block of which fills.  The launch also moves the tokens that
// follow the quantized blocks into the window.  Layers that merge codes (gamma1 > 0) need their dominant layer's
// blocks in place: they go one per launch, after it.
int pack_layers(xq_cache* c, const int* layers, int n, const void* K, const void* V, size_t layer_stride, int n_tokens,
                cudaStream_t st) {
  const Dims& dm = c->plan.dm;
  const int s_old = c->seq[layers[0]], s_new = s_old + n_tokens;
  const int nq_old = s_old - residual_count(s_old, dm.R), nq_new = s_new - residual_count(s_new, dm.R);
  PackParams p;
  p.dm = dm;
  p.n_layers = n;
  p.n_in = n_tokens; p.s_old = s_old; p.nq_old = nq_old; p.n_blocks = (nq_new - nq_old) / dm.R;
  p.tb = dm.g > 32 ? dm.g : 32;  // tokens per CTA: whole key groups, whole words of either kind
  p.f16 = c->cfg.io_dtype == XQ_F16;
  p.win_count = s_new - nq_new;
  p.nq_new = nq_new;
  p.merge_lut[0] = merge_table(c->cfg.gamma1, 1);
  p.merge_lut[1] = merge_table(c->cfg.gamma1, 2);
  for (int i = 0; i < n; ++i) {
    const int l = layers[i];
    if (c->seq[l] != s_old) return XQ_ERR_ARG;
    PackLayer& pl = p.layer[i];
    pl.L = layer_ptrs(c, l);
    pl.K_in = (const uint16_t*)((const uint8_t*)K + (size_t)i * layer_stride);
    pl.V_in = (const uint16_t*)((const uint8_t*)V + (size_t)i * layer_stride);
    const int ok = k_owner(&c->cfg, l), ov = v_owner(&c->cfg, l);
    const int stat = c->cfg.delta_stats ? 4 : 0;
    pl.own_k = ok == l ? 1 : ((merges_codes(&c->cfg, l, c->cfg.km) ? 2 : 0) | stat);
    pl.own_v = ov == l ? 1 : ((merges_codes(&c->cfg, l, c->cfg.vm) ? 2 : 0) | stat);
    pl.delta_k = (unsigned long long*)(c->ws + c->plan.delta) + (size_t)(l * 2 + 0) * 4;
    pl.delta_v = (unsigned long long*)(c->ws + c->plan.delta) + (size_t)(l * 2 + 1) * 4;
    if (pl.own_k > 1 || pl.own_v > 1) {
      // the layer reads the codes its dominant layer wrote for these blocks: that layer must hold them, and the
      // launch that wrote them must be another one
      if (n != 1) return XQ_ERR_ARG;
      for (int o : {ok, ov})
        if (o != l && c->seq[o] - residual_count(c->seq[o], dm.R) < nq_new) return XQ_ERR_ORDER;
    }
    pl.eta_k = pl.L.bk == 1 ? c->cfg.eta1 : c->cfg.eta2;
    pl.eta_v = pl.L.bv == 1 ? c->cfg.eta1 : c->cfg.eta2;
  }
  cudaError_t e;
  if (c->cfg.delta_stats && !c->delta_clean) {
    e = cudaMemsetAsync(c->ws + c->plan.delta, 0, (size_t)c->cfg.n_layers * 2 * 4 * 8, st);
    if (e != cudaSuccess) return fail_cuda(c, e);
    c->delta_clean = true;
  }
  {
    Timer t(c, st, 2);
    e = launch_pack(p, st);
  }
  c->launches++;
  if (e != cudaSuccess) return fail_cuda(c, e);
  // every layer that reads what this launch wrote must wait for it before its next decode fetches packed data
  for (int i = 0; i < n; ++i)
    for (int l2 = 0; l2 < c->cfg.n_layers; ++l2)
      if (l2 == layers[i] || k_owner(&c->cfg, l2) == layers[i] || v_owner(&c->cfg, l2) == layers[i] ||
          k_owner(&c->cfg, layers[i]) == l2 || v_owner(&c->cfg, layers[i]) == l2)
        c->repacked[l2] = 1;
  return XQ_OK;
}

// chained: the launch before this one in the stream is a tensor-core decode launch of the same call, so nothing this
// launch reads (q, the new token, the window, the packed streams) can still be written when its CTAs start; it
// waits for that launch only before it writes.  *was_mma tells the caller whether this launch can head such a chain.
int decode_impl(xq_cache* c, int layer, const void* q, void* out, int out_f32, cudaStream_t st,
                const void* K_new = nullptr, const void* V_new = nullptr, int vis = -1, bool chained = false,
                bool* was_mma = nullptr) {
  if (was_mma) *was_mma = false;
  if (!c) return XQ_ERR_ARG;
  if (layer < 0 || layer >= c->cfg.n_layers) return XQ_ERR_ARG;
  DecodeParams p;
  bool use_mma = false;
  int rc = prepare_decode(c, layer, q, out, out_f32, K_new, V_new, c->seq[layer] + (K_new ? 1 : 0), p, use_mma, vis);
  if (rc != XQ_OK) return rc;
  if (use_mma) {
    rc = ensure_clean_scratch(c, st);
    if (rc != XQ_OK) return rc;
    // the packed streams may be fetched ahead of the preceding kernel unless a pack kernel wrote them since
    // this layer's last decode (then that kernel may be the writer, or only just behind it)
    p.early_fetch = c->repacked[layer] ? 0 : 1;
    if (chained) p.early_fetch = p.late_wait = 1;
  }
  rc = launch_decode(c, p, use_mma, workspace_scratch(c), st);
  if (rc != XQ_OK) {
    if (use_mma) c->tickets_clean = false;
    return rc;
  }
  if (use_mma) c->repacked[layer] = 0;
  if (K_new) c->seq[layer] += 1;
  if (was_mma) *was_mma = use_mma;
  return XQ_OK;
}

}  // namespace

extern "C" {

int xq_config_check(const xq_config* cfg) { return check(cfg) ? XQ_OK : XQ_ERR_CONFIG; }

size_t xq_workspace_bytes(const xq_config* cfg) {
  if (!check(cfg)) return 0;
  Plan pl;
  make_plan(cfg, pl);
  return pl.total;
}

int xq_create(const xq_config* cfg, void* dev_workspace, size_t bytes, xq_cache** out) {
  if (!out) return XQ_ERR_ARG;
  *out = nullptr;
  if (!check(cfg)) return XQ_ERR_CONFIG;
  if (!dev_workspace || ((uintptr_t)dev_workspace & 255)) return XQ_ERR_ARG;
  xq_cache* c = new (std::nothrow) xq_cache();
  if (!c) return XQ_ERR_NOMEM;
  c->cfg = *cfg;
  make_plan(cfg, c->plan);
  if (bytes < c->plan.total) { delete c; return XQ_ERR_CAPACITY; }
  c->ws = (uint8_t*)dev_workspace;
  c->seq.assign(cfg->n_layers, 0);
  c->repacked.assign(cfg->n_layers, 1);
  c->launches = 0;
  c->last_cuda = 0;
  c->scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.0f / sqrtf((float)cfg->head_dim);
  c->timing = false;
  c->used = 0;
  c->sm_count = 148;
  c->tickets_clean = false;
  c->delta_clean = false;
  c->device = -1;
  c->static_base = nullptr;
  memset(c->mma_ctas, 0, sizeof(c->mma_ctas));
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) {
    c->sm_count = sms;
    c->device = dev;
    // Set-up, not the hot path: the address of the static scratch array of xq_decode_attention_static.  The query
    // makes the driver place the library's image (the array included) on this device now.
    if (static_scratch_address(&c->static_base) != cudaSuccess) {
      cudaGetLastError();
      c->static_base = nullptr;
    }
  } else {
    cudaGetLastError();  // no device (host-only use of the handle): keep the defaults
  }
  *out = c;
  return XQ_OK;
}

int xq_destroy(xq_cache* c) {
  if (!c) return XQ_ERR_ARG;
  for (auto& e : c->pool) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
  delete c;
  return XQ_OK;
}

int xq_reset(xq_cache* c) {
  if (!c) return XQ_ERR_ARG;
  for (auto& s : c->seq) s = 0;
  for (auto& r : c->repacked) r = 1;  // as after xq_create: the first decode of a layer waits for its predecessor
  c->tickets_clean = false;           // tickets and status are cleared again before their next use
  c->delta_clean = false;             // and so are the code-difference counters
  return XQ_OK;
}

int xq_append_kv(xq_cache* c, int layer, const void* K, const void* V, int n_tokens, void* stream) {
  if (!c || !K || !V) return XQ_ERR_ARG;
  if (layer < 0 || layer >= c->cfg.n_layers || n_tokens < 1) return XQ_ERR_ARG;
  if (((uintptr_t)K & 15) || ((uintptr_t)V & 15)) return XQ_ERR_ARG;
  const Dims& dm = c->plan.dm;
  cudaStream_t st = (cudaStream_t)stream;
  int s_old = c->seq[layer];
  if ((long long)s_old + n_tokens > c->cfg.max_seq) return XQ_ERR_CAPACITY;
  int s_new = s_old + n_tokens;
  int nq_old = s_old - residual_count(s_old, dm.R);
  int nq_new = s_new - residual_count(s_new, dm.R);
  int n_blocks = (nq_new - nq_old) / dm.R;
  if (n_blocks > 0) {
    int rc = pack_layers(c, &layer, 1, K, V, 0, n_tokens, st);
    if (rc != XQ_OK) return rc;
  } else {
    WindowParams w;
    w.dm = dm; w.L = layer_ptrs(c, layer);
    w.K_in = (const uint16_t*)K; w.V_in = (const uint16_t*)V;
    w.n_in = n_tokens; w.s_old = s_old;
    w.first = s_old;
    w.count = n_tokens;
    w.nq_new = nq_new;
    cudaError_t e;
    {
      Timer t(c, st, 3);
      e = launch_window_append(w, st);
    }
    c->launches++;
    if (e != cudaSuccess) return fail_cuda(c, e);
  }
  c->seq[layer] = s_new;
  return XQ_OK;
}

int xq_decode_attention(xq_cache* c, int layer, const void* q, void* out, void* stream) {
  return decode_impl(c, layer, q, out, 0, (cudaStream_t)stream);
}

int xq_decode_attention_f32(xq_cache* c, int layer, const void* q, float* out, void* stream) {
  return decode_impl(c, layer, q, out, 1, (cudaStream_t)stream);
}

namespace {
// Query token j of n sees the cache up to its own position; one decode launch per token (their visible ranges
// differ), all on the same stream.
int chunk_impl(xq_cache* c, int layer, const void* q, void* out, int n, int out_f32, void* stream) {
  if (!c || !q || !out) return XQ_ERR_ARG;
  if (layer < 0 || layer >= c->cfg.n_layers) return XQ_ERR_ARG;
  const int S = c->seq[layer];
  if (n < 1 || n > S) return XQ_ERR_ARG;
  if (((uintptr_t)q & 15) || ((uintptr_t)out & 15)) return XQ_ERR_ARG;
  const Dims& dm = c->plan.dm;
  // everything that can be refused is the same for every token: check the first and the last before any launch
  {
    DecodeParams p;
    bool use_mma;
    int rc = prepare_decode(c, layer, q, out, out_f32, nullptr, nullptr, S, p, use_mma, S - n + 1);
    if (rc == XQ_OK) rc = prepare_decode(c, layer, q, out, out_f32, nullptr, nullptr, S, p, use_mma, S);
    if (rc != XQ_OK) return rc;
  }
  const size_t row = (size_t)dm.B * dm.Hq * dm.D;  // elements of one token's queries: [batch, heads, head_dim]
  bool chain = false;  // launches after the first read what the first one waited for and write their own rows
  for (int j = 0; j < n; ++j) {
    const uint8_t* qj = (const uint8_t*)q + (size_t)j * row * 2;
    uint8_t* oj = (uint8_t*)out + (size_t)j * row * (out_f32 ? 4 : 2);
    const int rc = decode_impl(c, layer, qj, oj, out_f32, (cudaStream_t)stream, nullptr, nullptr, S - n + 1 + j, chain, &chain);
    if (rc != XQ_OK) return rc;
  }
  return XQ_OK;
}
}  // namespace

int xq_attention_chunk(xq_cache* c, int layer, const void* q, void* out, int n_q_tokens, void* stream) {
  return chunk_impl(c, layer, q, out, n_q_tokens, 0, stream);
}

int xq_attention_chunk_f32(xq_cache* c, int layer, const void* q, float* out, int n_q_tokens, void* stream) {
  return chunk_impl(c, layer, q, out, n_q_tokens, 1, stream);
}

int xq_decode_attention_static(xq_cache* c, int layer, const void* q, void* out, void* stream) {
  if (!c) return XQ_ERR_ARG;
  if (layer < 0 || layer >= c->cfg.n_layers) return XQ_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  DecodeParams p;
  bool use_mma = false;
  int rc = prepare_decode(c, layer, q, out, 0, nullptr, nullptr, c->seq[layer], p, use_mma);
  if (rc != XQ_OK) return rc;
  // the array belongs to the device the handle was created on
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return fail_cuda(c, cudaGetLastError());
  if (dev != c->device) return XQ_ERR_ARG;
  if (!c->static_base) return fail_cuda(c, cudaErrorInvalidSymbol);
  // carve the static array: [partial accumulators | partial (max, sum) | tickets | status]
  const Dims& dm = c->plan.dm;
  const size_t ns = (size_t)p.ns_q + (size_t)p.ns_w;
  const size_t acc_bytes = align_up((size_t)dm.B * dm.Hq * ns * dm.D * 4, 256);
  const size_t ml_bytes = align_up((size_t)dm.B * dm.Hq * ns * 2 * 4, 256);
  const size_t ticket_bytes = align_up((size_t)dm.B * dm.Hkv * 4, 256);
  if (acc_bytes + ml_bytes + ticket_bytes + 256 > (size_t)XQ_STATIC_SCRATCH_BYTES) return XQ_ERR_CAPACITY;
  Scratch s;
  s.part_acc = (float*)c->static_base;
  s.part_ml = (float*)(c->static_base + acc_bytes);
  s.tickets = (unsigned int*)(c->static_base + acc_bytes + ml_bytes);
  s.status = (int*)(c->static_base + acc_bytes + ml_bytes + ticket_bytes);
  if (use_mma) {
    // the array keeps whatever the previous call (of any handle) left: tickets and status must start at zero
    cudaError_t e = cudaMemsetAsync(s.tickets, 0, ticket_bytes + 256, st);
    if (e != cudaSuccess) return fail_cuda(c, e);
  }
  return launch_decode(c, p, use_mma, s, st);  // early_fetch stays 0: this call never fetches ahead of its predecessor
}

int xq_decode_step(xq_cache* c, const void* K_new, const void* V_new, const void* q, void* out,
                   const int32_t* layer_order, int mem, void* stream) {
  if (!c || !K_new || !V_new || !q || !out) return XQ_ERR_ARG;
  if (mem != XQ_MEM_DEVICE && mem != XQ_MEM_HOST) return XQ_ERR_ARG;
  if (mem == XQ_MEM_DEVICE &&
      (((uintptr_t)K_new & 15) || ((uintptr_t)V_new & 15) || ((uintptr_t)q & 15) || ((uintptr_t)out & 15)))
    return XQ_ERR_ARG;
  const Dims& dm = c->plan.dm;
  const int L = c->cfg.n_layers;
  // Everything that can be refused is checked before the first copy or launch, on a copy of the layer lengths
  // advanced in processing order, so that a refused call leaves the cache as it was.
  {
    std::vector<char> seen(L, 0);
    std::vector<int> len(c->seq);
    for (int i = 0; i < L; ++i) {
      const int l = layer_order ? layer_order[i] : i;
      if (l < 0 || l >= L || seen[l]) return XQ_ERR_ARG;
      seen[l] = 1;
      if (len[l] + 1 > c->cfg.max_seq) return XQ_ERR_CAPACITY;
      len[l] += 1;
      for (int o : {k_owner(&c->cfg, l), v_owner(&c->cfg, l)}) {
        if (o == l) continue;
        if (!seen[o]) return XQ_ERR_ORDER;
        const int nq = len[l] - residual_count(len[l], dm.R), nqo = len[o] - residual_count(len[o], dm.R);
        if (nqo < nq) return XQ_ERR_ORDER;
      }
      if (c->cfg.kernel >= XQ_KERNEL_MMA && !layer_uses_mma(c, l)) return XQ_ERR_CONFIG;
    }
  }
  cudaStream_t st = (cudaStream_t)stream;
  const size_t kv_layer = (size_t)dm.B * dm.Hkv * dm.D * 2;
  const size_t q_layer = (size_t)dm.B * dm.Hq * dm.D * 2;
  const uint8_t *dk = (const uint8_t*)K_new, *dv = (const uint8_t*)V_new, *dq = (const uint8_t*)q;
  uint8_t* dout = (uint8_t*)out;
  if (mem == XQ_MEM_HOST) {
    uint8_t* s = c->ws + c->plan.staging;
    size_t kvb = align_up(c->plan.staging_kv_bytes, 256), qb = align_up(c->plan.staging_q_bytes, 256);
    uint8_t *sk = s, *sv = s + kvb, *sq = s + 2 * kvb, *so = s + 2 * kvb + qb;
    cudaError_t e = cudaMemcpyAsync(sk, K_new, c->plan.staging_kv_bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sv, V_new, c->plan.staging_kv_bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sq, q, c->plan.staging_q_bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return fail_cuda(c, e);
    dk = sk; dv = sv; dq = sq; dout = so;
  }
  // Only a CUDA error can stop what follows (the cache is then in an undefined state, as after any XQ_ERR_CUDA).
  // The step on which every layer's window block fills: one quantize-and-pack launch for all layers (it also moves
  // the new token into the emptied windows), then the decode launches.
  bool appended = false;
  {
    bool same = true;
    for (int l = 1; l < L; ++l) same = same && c->seq[l] == c->seq[0];
    const int s_old = c->seq[0];
    const int nq_old = s_old - residual_count(s_old, dm.R), nq_new = s_old + 1 - residual_count(s_old + 1, dm.R);
    if (same && nq_new > nq_old && c->cfg.gamma1 == 0.f && !c->cfg.delta_stats) {
      for (int c0 = 0; c0 < L; c0 += PACK_MAX_LAYERS) {
        int idx[PACK_MAX_LAYERS];
        const int n = L - c0 < PACK_MAX_LAYERS ? L - c0 : PACK_MAX_LAYERS;
        for (int i = 0; i < n; ++i) idx[i] = c0 + i;
        const int rc = pack_layers(c, idx, n, dk + c0 * kv_layer, dv + c0 * kv_layer, kv_layer, 1, st);
        if (rc != XQ_OK) return rc;
      }
      for (int l = 0; l < L; ++l) c->seq[l] += 1;
      appended = true;
    }
  }
  bool chain = false;  // the launch before the next one is a tensor-core decode launch of this call
  for (int i = 0; i < L; ++i) {
    const int l = layer_order ? layer_order[i] : i;
    if (appended) {
      const int rc = decode_impl(c, l, dq + l * q_layer, dout + l * q_layer, 0, st, nullptr, nullptr, -1, chain, &chain);
      if (rc != XQ_OK) return rc;
      continue;
    }
    // One token that neither fills a window block nor is the layer's first quantized step goes into the window
    // inside the tensor-core decode kernel; every other case appends with its own kernels first.
    const int s_old = c->seq[l];
    const int nq_old = s_old - residual_count(s_old, dm.R), nq_new = s_old + 1 - residual_count(s_old + 1, dm.R);
    int rc;
    if (nq_new == nq_old && nq_old > 0 && layer_uses_mma(c, l)) {
      rc = decode_impl(c, l, dq + l * q_layer, dout + l * q_layer, 0, st, dk + l * kv_layer, dv + l * kv_layer, -1, chain,
                       &chain);
    } else {
      rc = xq_append_kv(c, l, dk + l * kv_layer, dv + l * kv_layer, 1, stream);
      if (rc != XQ_OK) return rc;
      rc = decode_impl(c, l, dq + l * q_layer, dout + l * q_layer, 0, st, nullptr, nullptr, -1, false, &chain);
    }
    if (rc != XQ_OK) return rc;
  }
  if (mem == XQ_MEM_HOST) {
    cudaError_t e = cudaMemcpyAsync(out, dout, c->plan.staging_q_bytes, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return fail_cuda(c, e);
  }
  return XQ_OK;
}

int xq_check_device(xq_cache* c, void* stream) {
  if (!c) return XQ_ERR_ARG;
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(c, e);
  if (!c->tickets_clean) return XQ_OK;  // the status word has not been used yet
  int status = 0;
  e = cudaMemcpy(&status, c->ws + c->plan.status, 4, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(c, e);
  return status ? XQ_ERR_DEVICE : XQ_OK;
}

int xq_delta_histogram(xq_cache* c, int layer, int kind, unsigned long long counts[4], void* stream) {
  if (!c || !counts) return XQ_ERR_ARG;
  if (layer < 0 || layer >= c->cfg.n_layers || kind < 0 || kind > 1) return XQ_ERR_ARG;
  if (!c->cfg.delta_stats) return XQ_ERR_CONFIG;
  for (int k = 0; k < 4; ++k) counts[k] = 0ull;
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(c, e);
  if (!c->delta_clean) return XQ_OK;  // nothing has been counted yet
  e = cudaMemcpy(counts, c->ws + c->plan.delta + (size_t)(layer * 2 + kind) * 4 * 8, 4 * 8, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(c, e);
  return XQ_OK;
}

double xq_equiv_bits(const xq_config* cfg) {
  if (!check(cfg)) return -1.0;
  long long k = 0, v = 0;
  for (int l = 0; l < cfg->n_layers; ++l) {
    if (k_owner(cfg, l) == l) k += layer_bits(l, cfg->kq);
    if (v_owner(cfg, l) == l) v += layer_bits(l, cfg->vq);
  }
  return 0.5 * ((double)k + (double)v) / (double)cfg->n_layers;
}

int xq_seq_len(const xq_cache* c, int layer) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return XQ_ERR_ARG;
  return c->seq[layer];
}

int xq_quantized_len(const xq_cache* c, int layer) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return XQ_ERR_ARG;
  int S = c->seq[layer];
  return S - residual_count(S, c->plan.dm.R);
}

int xq_split_plan(const xq_cache* c, int layer, int* nsq, int* nsw) {
  if (!c || !nsq || !nsw || layer < 0 || layer >= c->cfg.n_layers) return XQ_ERR_ARG;
  if (c->seq[layer] < 1) return XQ_ERR_ARG;
  {
    const int S = c->seq[layer], r = residual_count(S, c->plan.dm.R);
    plan_splits(c, layer, S - r, r, *nsq, *nsw);
  }
  return XQ_OK;
}

int xq_region(const xq_cache* c, int layer, int which, size_t* offset, size_t* stream_stride) {
  if (!c || !offset || !stream_stride || layer < 0 || layer >= c->cfg.n_layers) return XQ_ERR_ARG;
  if (which < 0 || which > 5) return XQ_ERR_ARG;
  const LayerRegions& r = c->plan.layers[layer];
  const size_t offs[6] = {r.k_codes, r.v_codes, r.k_meta, r.v_meta, r.win_k, r.win_v};
  *offset = offs[which];
  *stream_stride = r.stride[which];
  return XQ_OK;
}

long long xq_launch_count(const xq_cache* c) { return c ? c->launches : 0; }

int xq_timing_enable(xq_cache* c, int on) {
  if (!c) return XQ_ERR_ARG;
  if (on && c->pool.empty()) {
    c->pool.reserve(TIMING_POOL);
    for (int i = 0; i < TIMING_POOL; ++i) {
      EventPair e;
      if (cudaEventCreate(&e.a) != cudaSuccess || cudaEventCreate(&e.b) != cudaSuccess)
        return fail_cuda(c, cudaGetLastError());
      e.kind = -1;
      c->pool.push_back(e);
    }
  }
  c->timing = on != 0;
  if (on) c->used = 0;
  return XQ_OK;
}

int xq_timing_read(xq_cache* c, int kind, int* launches, double* total_ms) {
  if (!c || !launches || !total_ms || kind < 0 || kind >= N_KINDS) return XQ_ERR_ARG;
  int n = 0;
  double tot = 0.0;
  for (size_t i = 0; i < c->used; ++i) {
    EventPair& e = c->pool[i];
    if (e.kind != kind) continue;
    cudaError_t err = cudaEventSynchronize(e.b);
    float ms = 0.f;
    if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e.a, e.b);
    if (err != cudaSuccess) return fail_cuda(c, err);
    tot += ms;
    ++n;
  }
  *launches = n;
  *total_ms = tot;
  return XQ_OK;
}

int xq_last_cuda_error(const xq_cache* c) { return c ? c->last_cuda : 0; }

const char* xq_strerror(int code) {
  switch (code) {
    case XQ_OK: return "ok";
    case XQ_ERR_CONFIG: return "invalid configuration";
    case XQ_ERR_ARG: return "invalid argument";
    case XQ_ERR_CAPACITY: return "capacity exceeded";
    case XQ_ERR_ORDER: return "code-owning layer is behind the layer that borrows its codes";
    case XQ_ERR_CUDA: return "CUDA error (see xq_last_cuda_error)";
    case XQ_ERR_NOMEM: return "out of host memory";
    case XQ_ERR_DEVICE: return "a kernel gave up a bounded wait (results of that call are invalid)";
    default: return "unknown error";
  }
}

}  // extern "C"
