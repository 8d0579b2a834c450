// Host side of the C ABI: argument checks, cache layout, call sequencing.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <new>
#include <vector>
#include <algorithm>
#include "zc_internal.h"
#include "zc_layout.cuh"

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int n_salient(double r, int n) { return (int)floor(r * (double)n); }
inline bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

int check_config(const zc_config* cfg) {
  if (!cfg || cfg->struct_size != (int)sizeof(zc_config)) return ZC_EINVAL;
  if (cfg->dtype != ZC_F16 && cfg->dtype != ZC_BF16) return ZC_EINVAL;
  if (cfg->batch < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads < 1) return ZC_EINVAL;
  if (cfg->n_q_heads % cfg->n_kv_heads) return ZC_EINVAL;
  if (cfg->n_q_heads / cfg->n_kv_heads > ZC_MAX_G) return ZC_EINVAL;
  if (cfg->head_dim != ZC_D) return ZC_EINVAL;
  if (cfg->max_prefill < 1 || cfg->max_prefill > (1 << 20)) return ZC_EINVAL;
  if (cfg->max_new_tokens < 0) return ZC_EINVAL;
  if (cfg->window < 8 || cfg->window > ZC_MAX_WINDOW) return ZC_EINVAL;
  if (cfg->bits_hi != 4 && cfg->bits_hi != 2 && cfg->bits_hi != 8 && cfg->bits_hi != 16) return ZC_EINVAL;
  if (cfg->bits_lo != 4 && cfg->bits_lo != 2 && cfg->bits_lo != 8 && cfg->bits_lo != 16) return ZC_EINVAL;
  // an 8-bit class and a class kept at 16 bits have separate builds of the decode kernel
  if ((cfg->bits_hi == 8 || cfg->bits_lo == 8) && (cfg->bits_hi == 16 || cfg->bits_lo == 16)) return ZC_EINVAL;
  if (cfg->flags & ~(ZC_FLAG_DEFER_APPEND | ZC_FLAG_OVERLAP_CALLS | ZC_FLAG_OUT_F32 | ZC_FLAG_PARAMS_F16 |
                     ZC_FLAG_GROUP_ALL_HEADS))
    return ZC_EINVAL;
  if (cfg->flags & ZC_FLAG_GROUP_ALL_HEADS) {   // one (s, z) per token for all heads: one split per token, quantised classes
    if (cfg->scope != ZC_SCOPE_TOKEN) return ZC_EINVAL;
    if (cfg->bits_hi == 16 || cfg->bits_lo == 16) return ZC_EINVAL;
  }
  if (cfg->flags & ZC_FLAG_PARAMS_F16) {   // 16-bit parameters: CSTQuant at 2 or 4 bits, every call waits for what precedes it
    if (cfg->flags & ZC_FLAG_OVERLAP_CALLS) return ZC_EINVAL;
    if (cfg->k_scheme != ZC_K_CST) return ZC_EINVAL;
    if ((cfg->bits_hi != 2 && cfg->bits_hi != 4) || (cfg->bits_lo != 2 && cfg->bits_lo != 4)) return ZC_EINVAL;
  }
  if (!(cfg->saliency_ratio >= 0.0 && cfg->saliency_ratio <= 1.0)) return ZC_EINVAL;
  if (cfg->k_scheme != ZC_K_CST && cfg->k_scheme != ZC_K_CHANNEL) return ZC_EINVAL;
  if (cfg->scope != ZC_SCOPE_KV_HEAD && cfg->scope != ZC_SCOPE_TOKEN) return ZC_EINVAL;
  // token scope re-compresses a window by kernels that follow the decode kernel: every call must
  // then wait for what precedes it on the stream
  if (cfg->scope == ZC_SCOPE_TOKEN && (cfg->flags & ZC_FLAG_OVERLAP_CALLS)) return ZC_EINVAL;
  if ((long long)cfg->batch * cfg->n_kv_heads > 65535) return ZC_EINVAL;
  // every re-compressed window adds two items to a decode call
  if (2 * (cfg->max_new_tokens / cfg->window) + 2 + 2 > ZC_MAX_ITEMS) return ZC_EINVAL;
  return ZC_OK;
}

void make_layout(const zc_config* cfg, ZcLayout* lay, size_t* cache_bytes, size_t* ws_bytes) {
  const int elt = 2;
  lay->units = cfg->batch * cfg->n_kv_heads;
  lay->G = cfg->n_q_heads / cfg->n_kv_heads;
  lay->n_kv = cfg->n_kv_heads;
  lay->window = cfg->window;
  lay->dtype = cfg->dtype;
  lay->out_f32 = (cfg->flags & ZC_FLAG_OUT_F32) ? 1 : 0;
  lay->kch = cfg->k_scheme == ZC_K_CHANNEL ? 1 : 0;
  lay->p16 = (cfg->flags & ZC_FLAG_PARAMS_F16) ? 1 : 0;
  lay->grp_all = (cfg->flags & ZC_FLAG_GROUP_ALL_HEADS) ? 1 : 0;
  lay->bits[0] = cfg->bits_hi;
  lay->bits[1] = cfg->bits_lo;
  const int max_flush = cfg->max_new_tokens / cfg->window;
  const int ns_max = n_salient(cfg->saliency_ratio, cfg->max_prefill);
  const int nr_max = cfg->max_prefill - ns_max;  // l - floor(r l) is non-decreasing in l
  const int ns_w = n_salient(cfg->saliency_ratio, cfg->window);
  const int nr_w = cfg->window - ns_w;
  // floor(r l) for l < max_prefill never exceeds ns_max; l - floor(r l) never exceeds nr_max.
  lay->cap_tiles[0] = zc_ceil_div(ns_max, ZC_TILE) + max_flush * zc_ceil_div(ns_w, ZC_TILE);
  lay->cap_tiles[1] = zc_ceil_div(nr_max, ZC_TILE) + max_flush * zc_ceil_div(nr_w, ZC_TILE);
  lay->max_runs = 2 * (1 + max_flush);
  lay->idx_cap0 = cfg->max_prefill;
  size_t off = 0;
  for (int c = 0; c < 2; ++c) {
    lay->tile_bytes[c] = zc_tile_bytes(lay->bits[c], lay->kch, lay->p16);
    lay->off_tiles[c] = (long long)off;
    off = align_up(off + (size_t)lay->cap_tiles[c] * lay->tile_bytes[c], 256);
  }
  lay->off_fac = (long long)off;
  off = align_up(off + (size_t)lay->max_runs * ZC_FAC_FLOATS * 4, 256);
  lay->off_cmax = (long long)off;
  off = align_up(off + 2 * 3 * ZC_D * 4, 256);
  lay->off_tailK = (long long)off;
  off = align_up(off + (size_t)cfg->window * ZC_D * elt, 256);
  lay->off_tailV = (long long)off;
  off = align_up(off + (size_t)cfg->window * ZC_D * elt, 256);
  lay->off_colsum = (long long)off;
  off = align_up(off + ZC_MAX_WINDOW * 4, 256);
  lay->off_sync = (long long)off;   // directly after colsum: both are cleared together
  off = align_up(off + ZC_EPOCH_CALLS * 4, 256);
  lay->off_scores = (long long)off;
  off = align_up(off + (size_t)std::max(cfg->max_prefill, cfg->window) * 4, 256);
  lay->off_idx = (long long)off;
  off = align_up(off + ((size_t)cfg->max_prefill + (size_t)max_flush * cfg->window) * 4, 256);
  lay->off_tokmm = (long long)off;   // only with token groups over all heads (the other layouts stay as they were)
  if (lay->grp_all) off = align_up(off + (size_t)std::max(cfg->max_prefill, cfg->window) * 16, 256);
  lay->unit_stride = (long long)off;
  if (cache_bytes) *cache_bytes = off * (size_t)lay->units;
  if (ws_bytes) {
    // prefill: probe positions + per-row log-sum-exp for every query head
    const int np_max = cfg->max_prefill;
    size_t pre = align_up((size_t)np_max * 4, 256) +
                 align_up((size_t)cfg->batch * cfg->n_q_heads * (size_t)np_max * 4, 256);
    // ... and a dense copy of the probe rows for probe sets of up to an eighth of the context
    // (larger sets are gathered tile by tile instead)
    pre += (size_t)cfg->batch * cfg->n_q_heads * (size_t)std::max(512, cfg->max_prefill / 8) * ZC_D * 2;
    // decode: partials [unit][items + tail tiles][G][ZC_PART_STRIDE] + tail logits
    // [unit][G][ZC_MAX_WINDOW] per call.  Calls in flight together take separate regions: room
    // for kCallsInFlight calls of the largest plan this configuration produces, and never less
    // than twice the worst case of any plan.
    const int max_items = std::min(ZC_MAX_ITEMS, 2 * ZC_MAX_SPLIT_HOST + 2 * max_flush);
    auto per_call = [&](int items) {
      return align_up((size_t)lay->units * (items + ZC_MAX_WINDOW / ZC_SUB) * lay->G * ZC_PART_STRIDE * 4, 256) +
             align_up((size_t)lay->units * lay->G * ZC_MAX_WINDOW * 4, 256);
    };
    zc_cache probe;   // the cache at its fullest, for the planner
    memset(&probe, 0, sizeof(probe));
    probe.cfg = *cfg;
    probe.lay = *lay;
    probe.l0 = cfg->max_prefill;
    probe.n0[0] = ns_max;
    probe.n0[1] = cfg->max_prefill - n_salient(cfg->saliency_ratio, cfg->max_prefill);
    probe.nw[0] = ns_w;
    probe.nw[1] = nr_w;
    probe.n_seg = 1 + max_flush;
    probe.n_sm = 148;
    constexpr int kCallsInFlight = 16;
    const size_t dec = std::max(2 * per_call(max_items), kCallsInFlight * per_call(zc_make_plan(&probe).items));
    *ws_bytes = align_up(std::max(pre, dec), 512);
  }
}

const char* kMsgs[] = {"ok", "invalid argument", "capacity exceeded", "call out of order",
                       "pointer not 16-byte aligned", "CUDA error",
                       "the call needs more scratch than the built-in buffer of "
                       "zc_decode_attention_noalloc holds: pass a workspace to zc_decode_attention"};
thread_local char g_cuda_msg[256] = "CUDA error";

int cuda_fail(cudaError_t e) {
  snprintf(g_cuda_msg, sizeof(g_cuda_msg), "CUDA error: %s", cudaGetErrorString(e));
  return ZC_ECUDA;
}

#define ZC_CUDA(expr)                              \
  do {                                             \
    cudaError_t e__ = (cudaError_t)(expr);         \
    if (e__ != cudaSuccess) return cuda_fail(e__); \
  } while (0)

}  // namespace

// Performs a deferred append as its own launch (a call other than decode attention came first).
static int flush_pending(zc_cache* c) {
  if (!c->pend_k) return ZC_OK;
  const void* k = c->pend_k;
  const void* v = c->pend_v;
  c->pend_k = c->pend_v = nullptr;
  ZC_CUDA(zc_launch_append(c, k, v, c->n_tail - 1, c->pend_stream));
  return ZC_OK;
}

ZcSeg zc_segment(const zc_cache* c, int seg) {
  ZcSeg s;
  for (int k = 0; k < 2; ++k) {
    const int t0 = zc_ceil_div(c->n0[k], ZC_TILE), tw = zc_ceil_div(c->nw[k], ZC_TILE);
    s.n_tok[k] = seg == 0 ? c->n0[k] : c->nw[k];
    s.tile0[k] = seg == 0 ? 0 : t0 + (seg - 1) * tw;
  }
  s.idx_off = seg == 0 ? 0 : c->lay.idx_cap0 + (seg - 1) * c->cfg.window;
  s.run0 = 2 * seg;
  return s;
}

ZcDecodePlan zc_make_plan(const zc_cache* c) {
  ZcDecodePlan p;
  memset(&p, 0, sizeof(p));
  p.n_seg = c->n_seg;
  p.n_tail = c->n_tail;
  p.l0 = c->l0;
  for (int k = 0; k < 2; ++k) {
    p.n0[k] = c->n0[k];
    p.nw[k] = c->nw[k];
    p.tiles0[k] = zc_ceil_div(c->n0[k], ZC_TILE);
    p.tilesw[k] = zc_ceil_div(c->nw[k], ZC_TILE);
  }
  // How finely to cut segment 0.  Two things cost time: CTAs that do not fill a whole wave of
  // the GPU (slots = SMs x resident CTAs), and the fixed set-up and merge of every CTA, worth
  // about ZC_ITEM_OVERHEAD sub-tiles of streaming.  Each candidate item size is scored by
  // (share of the slot-time its waves use) x (share of a CTA's life spent streaming).  Calls
  // of many waves use the build with 4 CTAs per SM.
  const int extras = 2 * (c->n_seg - 1);
  const int zs = zc_ceil_div(c->lay.G, 4);
  const int cap = std::max(1, (ZC_MAX_ITEMS - extras) / 2);
  int subs[2];
  for (int k = 0; k < 2; ++k) subs[k] = std::max(1, zc_ceil_div(c->n0[k], ZC_SUB));
  static const int kCand[] = {256, 192, 128, 96, 80, 64, 56, 48, 40, 32};
  auto choose = [&](int per_sm) -> double {
    const int slots = c->n_sm * per_sm;
    double best = -1.0, best_ctas = 0.0;
    for (int target : kCand) {
      int spi[2], split[2];
      for (int k = 0; k < 2; ++k) {
        const int want = std::min(std::min(zc_ceil_div(subs[k], target), std::min(ZC_MAX_SPLIT_HOST, cap)),
                                  subs[k]);
        // an even number of sub-tiles per item: the kernel consumes them in pairs
        spi[k] = (zc_ceil_div(subs[k], std::max(1, want)) + 1) & ~1;
        split[k] = zc_ceil_div(subs[k], spi[k]);
      }
      // items of every head group, one tail CTA per unit, the one CTA that only waits
      const double n_ctas = ((double)(split[0] + split[1] + extras) * zs + 1) * c->lay.units + 1;
      const double waves = n_ctas / slots;
      // a handful of CTAs beyond a whole wave start as soon as the first ones retire
      const double whole = std::max(1.0, (waves - floor(waves) <= ZC_WAVE_SLACK) ? floor(waves) : ceil(waves));
      const double fill = std::min(1.0, n_ctas / (whole * slots));
      const double per_item = (double)(subs[0] + subs[1]) / (split[0] + split[1]);
      const double score = fill * per_item / (per_item + ZC_ITEM_OVERHEAD);
      if (score > best) {
        best = score;
        best_ctas = n_ctas;
        for (int k = 0; k < 2; ++k) { p.spi0[k] = spi[k]; p.split0[k] = split[k]; }
      }
    }
    return best_ctas;
  };
  p.ctas_per_sm = 3;
  if (choose(4) >= ZC_MANY_WAVES * c->n_sm * 4) p.ctas_per_sm = 4;
  else choose(3);
  // One CTA per unit and head group, one item per class of the prompt's segment: for calls that run side by
  // side with their neighbours (wave fill is then no concern, only the fixed cost per CTA), and
  // for a call alone whose units by themselves fill every slot of the GPU (workload 4: 1024 units
  // on 592 slots; 115 us per call against 134 us with one CTA per item).
  const bool overlap_calls = (c->cfg.flags & ZC_FLAG_OVERLAP_CALLS) != 0;
  const bool unit_ctas = overlap_calls || (long long)c->lay.units * zs >= (long long)c->n_sm * 4;
  if (unit_ctas) {
    p.ctas_per_sm = 4;
    p.fold_tail = 1;
    for (int k = 0; k < 2; ++k) {   // one item per class, however long: every further item costs a set-up and a merge
      p.spi0[k] = (subs[k] + 1) & ~1;
      p.split0[k] = 1;
    }
  }
  p.chain_free = overlap_calls ? 1 : 0;
  p.items = p.split0[0] + p.split0[1] + 2 * (p.n_seg - 1);
  p.cta_items = 1;
  if (unit_ctas) p.cta_items = p.items;   // one CTA per unit and head group
  return p;
}

extern "C" {

const char* zc_strerror(int status) {
  if (status == ZC_ECUDA) return g_cuda_msg;
  if (status > 0 || status < -6) return "unknown status";
  return kMsgs[-status];
}

int zc_cache_bytes(const zc_config* cfg, size_t* cache_bytes, size_t* workspace_bytes) {
  int rc = check_config(cfg);
  if (rc) return rc;
  ZcLayout lay;
  make_layout(cfg, &lay, cache_bytes, workspace_bytes);
  return ZC_OK;
}

int zc_cache_init(void* dev_mem, size_t bytes, const zc_config* cfg, zc_cache** out) {
  if (!out) return ZC_EINVAL;
  *out = nullptr;
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!dev_mem) return ZC_EINVAL;
  if ((uintptr_t)dev_mem & 255) return ZC_EALIGN;
  zc_cache* c = new (std::nothrow) zc_cache();
  if (!c) return ZC_EINVAL;
  memset(c, 0, sizeof(*c));
  c->cfg = *cfg;
  size_t need = 0;
  make_layout(cfg, &c->lay, &need, &c->ws_bytes);
  if (bytes < need) {
    delete c;
    return ZC_ECAPACITY;
  }
  c->base = (char*)dev_mem;
  c->bytes = bytes;
  c->l0 = -1;
  c->n_seg = 0;
  c->fence.rec = -1;
  int dev = 0, n_sm = 148;
  if (cudaGetDevice(&dev) == cudaSuccess)
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  else
    cudaGetLastError();
  c->n_sm = n_sm > 0 ? n_sm : 148;
  // the address look-ups the decode launches need are done here, outside any stream capture
  if (zc_order_words(nullptr) != (int)cudaSuccess) cudaGetLastError();
  if (zc_static_scratch(nullptr) != (int)cudaSuccess) cudaGetLastError();
  *out = c;
  return ZC_OK;
}

void zc_cache_free(zc_cache* c) { delete c; }

int zc_probe_count(int l, double rho_recent, double rho_random) {
  if (l < 1 || !(rho_recent >= 0.0 && rho_recent <= 1.0) ||
      !(rho_random >= 0.0 && rho_random <= 1.0))
    return ZC_EINVAL;
  int n_rec = std::min(l, std::max(1, (int)floor(rho_recent * (double)l)));
  int n_rnd = std::min(l - n_rec, (int)floor(rho_random * (double)l));
  return n_rec + n_rnd;
}

int zc_default_probes(int l, double rho_recent, double rho_random, uint64_t seed, int32_t* out,
                      int* n_out) {
  int total = zc_probe_count(l, rho_recent, rho_random);
  if (total < 0 || !out) return ZC_EINVAL;
  const int n_rec = std::min(l, std::max(1, (int)floor(rho_recent * (double)l)));
  const int n_rnd = total - n_rec;
  const int pool = l - n_rec;
  std::vector<int32_t> perm((size_t)pool);
  for (int i = 0; i < pool; ++i) perm[i] = i;
  uint64_t state = seed;
  for (int i = 0; i < n_rnd; ++i) {
    state += 0x9E3779B97F4A7C15ull;
    uint64_t z = state;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    int j = i + (int)(z % (uint64_t)(pool - i));
    std::swap(perm[i], perm[j]);
  }
  std::sort(perm.begin(), perm.begin() + n_rnd);
  for (int i = 0; i < n_rnd; ++i) out[i] = perm[i];
  for (int i = 0; i < n_rec; ++i) out[n_rnd + i] = pool + i;
  if (n_out) *n_out = total;
  return ZC_OK;
}

}  // extern "C"

static int prefill_compress(zc_cache* c, const void* Q, const void* K, const void* V, int l,
                            const int64_t q_strides[3], const int64_t kv_strides[3],
                            const int32_t* probe_pos, int n_probe, const int32_t* salient_idx,
                            const float* row_lse, void* workspace, size_t workspace_bytes,
                            zc_stream_t stream) {
  if (!c || !K || !V || !kv_strides) return ZC_EINVAL;
  if (l < 1) return ZC_EINVAL;
  if (l > c->cfg.max_prefill) return ZC_ECAPACITY;
  if (!aligned16(K) || !aligned16(V)) return ZC_EALIGN;
  for (int i = 0; i < 3; ++i)
    if (kv_strides[i] < 0 || (kv_strides[i] % 8)) return ZC_EINVAL;
  if (kv_strides[2] < ZC_D) return ZC_EINVAL;
  if (!salient_idx) {
    if (!Q || !q_strides || !probe_pos || !workspace) return ZC_EINVAL;
    if (!aligned16(Q) || !aligned16(workspace)) return ZC_EALIGN;
    for (int i = 0; i < 3; ++i)
      if (q_strides[i] < 0 || (q_strides[i] % 8)) return ZC_EINVAL;
    if (q_strides[2] < ZC_D) return ZC_EINVAL;
    if (n_probe < 1 || n_probe > l) return ZC_EINVAL;
    for (int i = 0; i < n_probe; ++i) {
      if (probe_pos[i] < 0 || probe_pos[i] >= l) return ZC_EINVAL;
      if (i && probe_pos[i] <= probe_pos[i - 1]) return ZC_EINVAL;
    }
    if (probe_pos[n_probe - 1] != l - 1) return ZC_EINVAL;
    size_t need = align_up((size_t)n_probe * 4, 256) +
                  (size_t)c->cfg.batch * c->cfg.n_q_heads * (size_t)n_probe * 4;
    if (workspace_bytes < need) return ZC_ECAPACITY;
  } else if (!aligned16(salient_idx)) {
    return ZC_EALIGN;
  }
  cudaStream_t st = (cudaStream_t)stream;
  c->pend_k = c->pend_v = nullptr;   // a prefill starts the cache over
  c->l0 = l;
  c->n0[0] = n_salient(c->cfg.saliency_ratio, l);
  c->n0[1] = l - c->n0[0];
  c->nw[0] = n_salient(c->cfg.saliency_ratio, c->cfg.window);
  c->nw[1] = c->cfg.window - c->nw[0];
  c->n_seg = 1;
  c->n_tail = 0;
  c->step_i = 0;
  c->fresh = 0;
  c->n_new = 0;
  memset(c->tail_nnz, 0, sizeof(c->tail_nnz));
  c->last_scores_n = l;
  // window statistics and the decode kernel's arrival counter start at zero
  ZC_CUDA(cudaMemset2DAsync(c->base + c->lay.off_colsum, (size_t)c->lay.unit_stride, 0,
                            (size_t)(c->lay.off_sync + ZC_EPOCH_CALLS * 4 - c->lay.off_colsum),
                            (size_t)c->lay.units, st));
  if (!salient_idx) {
    int32_t* P_dev = (int32_t*)workspace;
    float* lse = (float*)((char*)workspace + align_up((size_t)n_probe * 4, 256));
    ZC_CUDA(cudaMemcpyAsync(P_dev, probe_pos, (size_t)n_probe * 4, cudaMemcpyHostToDevice, st));
    const size_t used = align_up((size_t)n_probe * 4, 256) +
                        align_up((size_t)c->cfg.batch * c->cfg.n_q_heads * (size_t)n_probe * 4, 256);
    void* qp = used < workspace_bytes ? (char*)workspace + used : nullptr;
    ZC_CUDA(zc_launch_probe_scores(c, Q, K, l, q_strides, kv_strides, P_dev, n_probe, lse, qp,
                                   qp ? workspace_bytes - used : 0, row_lse, st));
    // one decision per token of a batch row: the mean of its KV heads' scores, for every head
    if (c->cfg.scope == ZC_SCOPE_TOKEN) ZC_CUDA(zc_launch_share_scores(c, l, st));
  }
  ZC_CUDA(zc_launch_topk(c, l, c->n0[0], 0, salient_idx, st));
  ZcSrc src{K, V, kv_strides[0], kv_strides[1], kv_strides[2], l};
  ZC_CUDA(zc_launch_quantize(c, src, zc_segment(c, 0), st));
  return ZC_OK;
}

extern "C" {

int zc_prefill_compress(zc_cache* c, const void* Q, const void* K, const void* V, int l,
                        const int64_t q_strides[3], const int64_t kv_strides[3],
                        const int32_t* probe_pos, int n_probe, const int32_t* salient_idx,
                        void* workspace, size_t workspace_bytes, zc_stream_t stream) {
  return prefill_compress(c, Q, K, V, l, q_strides, kv_strides, probe_pos, n_probe, salient_idx, nullptr,
                          workspace, workspace_bytes, stream);
}

int zc_prefill_compress_lse(zc_cache* c, const void* Q, const void* K, const void* V, int l,
                            const int64_t q_strides[3], const int64_t kv_strides[3],
                            const int32_t* probe_pos, int n_probe, const float* row_lse,
                            void* workspace, size_t workspace_bytes, zc_stream_t stream) {
  if (!row_lse) return ZC_EINVAL;
  if (!aligned16(row_lse)) return ZC_EALIGN;
  return prefill_compress(c, Q, K, V, l, q_strides, kv_strides, probe_pos, n_probe, nullptr, row_lse,
                          workspace, workspace_bytes, stream);
}

int zc_prefill_attention(zc_cache* c, const void* Q, const void* K, const void* V, int l,
                         const int64_t q_strides[3], const int64_t kv_strides[3], void* O, float* row_lse,
                         zc_stream_t stream) {
  if (!c || !Q || !K || !V || !O || !row_lse || !q_strides || !kv_strides) return ZC_EINVAL;
  if (l < 1) return ZC_EINVAL;
  if (l > c->cfg.max_prefill) return ZC_ECAPACITY;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(row_lse)) return ZC_EALIGN;
  for (int i = 0; i < 3; ++i)
    if (q_strides[i] < 0 || (q_strides[i] % 8) || kv_strides[i] < 0 || (kv_strides[i] % 8)) return ZC_EINVAL;
  if (q_strides[2] < ZC_D || kv_strides[2] < ZC_D) return ZC_EINVAL;
  ZC_CUDA(zc_launch_prefill_attention(c, Q, K, V, l, q_strides, kv_strides, O, row_lse, (cudaStream_t)stream));
  return ZC_OK;
}

int zc_append(zc_cache* c, const void* k_new, const void* v_new, zc_stream_t stream) {
  if (!c || !k_new || !v_new) return ZC_EINVAL;
  if (c->l0 < 0) return ZC_ESTATE;
  if (!aligned16(k_new) || !aligned16(v_new)) return ZC_EALIGN;
  if (c->n_new >= c->cfg.max_new_tokens) return ZC_ECAPACITY;
  if (c->n_tail >= c->cfg.window) return ZC_ESTATE;
  int rc = flush_pending(c);
  if (rc) return rc;
  if (c->cfg.flags & ZC_FLAG_DEFER_APPEND) {
    c->pend_k = k_new;
    c->pend_v = v_new;
    c->pend_stream = (cudaStream_t)stream;
  } else {
    ZC_CUDA(zc_launch_append(c, k_new, v_new, c->n_tail, (cudaStream_t)stream));
  }
  c->n_tail += 1;
  c->n_new += 1;
  c->fresh = 1;
  return ZC_OK;
}

// need_worst: check the workspace against the worst case of the cache's whole life (the public
// contract) rather than against what this call touches.
static int decode_attention(zc_cache* c, const void* q, void* out, int is_probe_step, void* workspace,
                            size_t workspace_bytes, bool need_worst, zc_stream_t stream) {
  if (!c || !q || !out || !workspace) return ZC_EINVAL;
  if (c->l0 < 0) return ZC_ESTATE;
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return ZC_EALIGN;
  if (need_worst && workspace_bytes < c->ws_bytes) return ZC_ECAPACITY;
  cudaStream_t st = (cudaStream_t)stream;
  if (c->pend_k && c->pend_stream != st) {
    int rc = flush_pending(c);
    if (rc) return rc;
  }
  ZcDecodePlan plan = zc_make_plan(c);
  // Alg. 3 counts one step per generated token: a call that follows an append takes the step
  // (probe-row collection, the window's completion); a further call on the same tail (a
  // re-query) attends the cache as it is and leaves the window's bookkeeping alone.
  const bool fresh = c->fresh != 0;
  c->fresh = 0;
  const int i_next = c->step_i + 1;
  const int collect =
      fresh && (c->n_tail > 0) && (is_probe_step || i_next > c->cfg.window - 5) ? 1 : 0;
  const void* pk = c->pend_k;
  const void* pv = c->pend_v;
  c->pend_k = c->pend_v = nullptr;
  // Alg. 3: the call that completes the window also re-compresses it (inside its kernel)
  const bool completes = fresh && c->n_tail == c->cfg.window;
  ZcFlushArgs fl;
  memset(&fl, 0, sizeof(fl));
  const bool token_scope = c->cfg.scope == ZC_SCOPE_TOKEN;
  // the heads' statistics must meet first (token scope), or the tiles carry 16-bit parameters,
  // which only the prefill quantiser writes: the window is re-compressed by kernels of their own
  const bool host_flush = token_scope || c->lay.p16 != 0;
  if (completes) {
    fl.on = host_flush ? 0 : 1;
    fl.seg = zc_segment(c, c->n_seg);
    for (int j = 0; j < c->n_tail; ++j) fl.nnz[j] = (unsigned char)(c->tail_nnz[j] + (collect ? 1 : 0));
  }
  ZC_CUDA(zc_launch_decode(c, plan, q, out, collect, (char*)workspace, workspace_bytes, pk, pv,
                           completes ? &fl : nullptr, st));
  if (completes && host_flush) {
    // The window's scores of all KV heads of a batch row meet before the split: scores from
    // the statistics the decode kernels collected, their mean over the row's heads, then the
    // prompt's own split and quantise kernels with the tail as their source.
    ZC_CUDA(zc_launch_window_scores(c, fl, st));
    if (token_scope) ZC_CUDA(zc_launch_share_scores(c, c->cfg.window, st));
    ZC_CUDA(zc_launch_topk(c, c->cfg.window, c->nw[0], fl.seg.idx_off, nullptr, st));
    const int64_t sh = (int64_t)(c->lay.unit_stride / 2);   // elements from one unit's tail to the next
    ZcSrc src{c->base + c->lay.off_tailK, c->base + c->lay.off_tailV, sh * c->lay.n_kv, sh, ZC_D, c->cfg.window};
    ZC_CUDA(zc_launch_quantize(c, src, fl.seg, st));
  }
  // Alg. 3 bookkeeping: the step counter follows the tokens of the current window
  if (fresh && c->n_tail > 0) {
    c->step_i = i_next;
    if (collect)
      for (int j = 0; j < c->n_tail; ++j) c->tail_nnz[j] += 1;
    if (completes) {
      c->last_scores_n = c->cfg.window;
      c->n_seg += 1;
      c->n_tail = 0;
      c->step_i = 0;
      memset(c->tail_nnz, 0, sizeof(c->tail_nnz));
    }
  }
  return ZC_OK;
}

int zc_decode_attention(zc_cache* c, const void* q, void* out, int is_probe_step,
                        void* workspace, size_t workspace_bytes, zc_stream_t stream) {
  return decode_attention(c, q, out, is_probe_step, workspace, workspace_bytes, true, stream);
}

int zc_decode_attention_noalloc(zc_cache* c, const void* q, void* out, int is_probe_step,
                                zc_stream_t stream) {
  if (!c || !q || !out) return ZC_EINVAL;
  if (c->l0 < 0) return ZC_ESTATE;
  // what this call really writes: partials and tail logits for the cache's present number of
  // items (calls that follow take further room in the buffer, or wait for this one)
  const ZcDecodePlan plan = zc_make_plan(c);
  const size_t need = zc_decode_scratch_bytes(c, plan.items);
  if (need > (size_t)ZC_NOALLOC_SCRATCH_BYTES) return ZC_ESCRATCH;
  void* scratch = nullptr;
  ZC_CUDA(zc_static_scratch(&scratch));   // first call per device: a synchronous address query
  return decode_attention(c, q, out, is_probe_step, scratch, (size_t)ZC_NOALLOC_SCRATCH_BYTES, false, stream);
}

int zc_num_segments(const zc_cache* c) { return c ? c->n_seg : ZC_EINVAL; }
int zc_tail_tokens(const zc_cache* c) { return c ? c->n_tail : ZC_EINVAL; }

int zc_segment_tokens(const zc_cache* c, int segment, int subset) {
  if (!c || segment < 0 || segment >= c->n_seg || subset < 0 || subset > 1) return ZC_EINVAL;
  return segment == 0 ? c->n0[subset] : c->nw[subset];
}

int zc_export_scores(zc_cache* c, float* p_tilde, zc_stream_t stream) {
  if (!c || !p_tilde) return ZC_EINVAL;
  if (c->l0 < 0) return ZC_ESTATE;
  { int rc = flush_pending(c); if (rc) return rc; }
  ZC_CUDA(zc_launch_export_scores(c, p_tilde, c->last_scores_n, (cudaStream_t)stream));
  return ZC_OK;
}

int zc_export_segment(zc_cache* c, int segment, int tensor, int subset, int32_t* idx,
                      uint8_t* codes, float* sz, float* cf, zc_stream_t stream) {
  if (!c || tensor < 0 || tensor > 1 || subset < 0 || subset > 1) return ZC_EINVAL;
  if (c->l0 < 0) return ZC_ESTATE;
  if (segment < 0 || segment >= c->n_seg) return ZC_EINVAL;
  { int rc = flush_pending(c); if (rc) return rc; }
  ZC_CUDA(zc_launch_export_segment(c, zc_segment(c, segment), tensor, subset, idx, codes, sz, cf,
                                   (cudaStream_t)stream));
  return ZC_OK;
}

int64_t zc_decode_bytes(const zc_cache* c) {
  if (!c || c->l0 < 0) return 0;
  int64_t per_unit = 0;
  for (int k = 0; k < 2; ++k) {
    const bool raw = c->lay.bits[k] == 16;   // tokens kept at full precision: rows only
    const int64_t per_tok = raw ? 2 * ZC_D * 2 : 32 * c->lay.bits[k] + ((c->lay.kch ? 8 : 16) >> c->lay.p16);  // K+V codes, (s,z) pairs
    const int64_t toks = (int64_t)c->n0[k] + (int64_t)(c->n_seg - 1) * c->nw[k];
    per_unit += toks * per_tok;
    const int runs = (c->n0[k] > 0 ? 1 : 0) + (c->nw[k] > 0 ? c->n_seg - 1 : 0);
    if (!raw) per_unit += (int64_t)runs * (c->lay.kch ? 3 : 2) * ZC_D * 4;   // channel factors of V; of K, or its (s, z) per channel
  }
  per_unit += (int64_t)c->n_tail * 2 * ZC_D * 2;     // full-precision tail
  per_unit += (int64_t)c->lay.G * ZC_D * 2 * 2;      // q in, out
  return per_unit * c->lay.units;
}

int64_t zc_launch_count(const zc_cache* c) { return c ? c->launches : 0; }

int zc_device_status(int* code) {
  if (!code) return ZC_EINVAL;
  ZC_CUDA(cudaDeviceSynchronize());
  ZC_CUDA(zc_device_error_code(code));
  int probe = 0, att = 0;
  ZC_CUDA(zc_probe_error_code(&probe));
  ZC_CUDA(zc_attention_error_code(&att));
  if (*code == 0 && (probe || att)) *code = 3;
  int dbg_c = 0, dbg_d = 0;   // bounds-checked build only: 100 + the first failed check
  ZC_CUDA(zc_debug_code_compress(&dbg_c));
  ZC_CUDA(zc_debug_code_decode(&dbg_d));
  if (*code == 0 && (dbg_c || dbg_d)) *code = 100 + (dbg_c ? dbg_c : dbg_d);
  return ZC_OK;
}

}  // extern "C"
