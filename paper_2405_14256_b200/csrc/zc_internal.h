// Internal declarations shared by the host API and the kernels of the library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "zipcache.h"

#define ZC_D 128            // head_dim
#define ZC_TILE 64          // tokens per cache tile
#define ZC_SUB 16           // tokens per MMA sub-tile inside a tile
#define ZC_FAC_FLOATS 400   // per-run factor block: cK[128] (channelwise keys: their scales), cV[128],
                            // smaxV, pad to 272, then the zero points of channelwise keys [128]
#define ZC_FAC_ZK 272
#define ZC_PART_STRIDE 132  // split-K partial per head: m, l, pad, pad, acc[128]
#define ZC_MAX_G 8
#define ZC_MAX_SPLIT_HOST 32      // most items one class of segment 0 is split into
#define ZC_MAX_ITEMS 128          // most items of one unit in one decode call
#define ZC_EPOCH_CALLS 64          // most decode calls in flight together on a stream (arrival counters per unit)
#define ZC_ITEM_OVERHEAD 24       // fixed cost of one split-K item, in 16-token sub-tiles of streaming
#define ZC_WAVE_SLACK 0.0         // share of a wave that may spill over without counting as one more
#define ZC_MANY_WAVES 1.2         // from this many waves of 4-per-SM CTAs on, the narrow build is used

// Device-side description of the cache buffer.  One "unit" = (batch, KV head).
// Per unit, at byte offsets from base + unit * unit_stride:
//   off_tiles[c]   cap_tiles[c] tiles of class c (0 = salient bits, 1 = regular bits)
//   off_fac        max_runs factor blocks (run = segment * 2 + class)
//   off_cmax       scratch of the quantiser, as ordered uint keys  [class][3][128]: channel maxima of
//                  |K| (channelwise keys: of K), of |V|, and channel minima of K (channelwise keys)
//   off_tailK/V    window x d elements of the input type
//   off_colsum     window floats: attention mass collected on probe steps
//   off_sync       ZC_EPOCH_CALLS arrival counters of the decode kernel's CTAs (zero between calls)
//   off_scores     normalised scores of the latest compression
//   off_idx        token index lists: segment 0 (salient then regular), then one
//                  window-sized slot per re-compressed window
// A tile of class c holds 64 tokens as four sub-blocks of 16 tokens, each
//   [K codes 16 x 16*bits B, canonical nibble/crumb order per token row]
//   [V codes of the 16 tokens in MMA fragment order (see zc_layout.cuh)]
//   [params 16 x (K scale, K zero, V scale, V zero) f32; channelwise keys: 16 x (V scale, V zero)]
struct ZcLayout {
  int units, G, n_kv, window, dtype;
  int out_f32;            // decode outputs are stored as fp32 (ZC_FLAG_OUT_F32)
  int kch;                // keys are quantised channelwise (ZC_K_CHANNEL): no per-token key parameters
  int p16;                // ZC_FLAG_PARAMS_F16: per-token parameters as (fp16 scale, int16 zero) pairs
  int grp_all;            // ZC_FLAG_GROUP_ALL_HEADS: a token's (s, z) over the channels of all KV heads of its batch row
  int bits[2];
  int tile_bytes[2];
  int cap_tiles[2];
  int max_runs;
  int idx_cap0;
  long long unit_stride;
  long long off_tiles[2], off_fac, off_cmax, off_tailK, off_tailV, off_colsum, off_sync, off_scores,
      off_idx, off_tokmm;   // off_tokmm: [tokens of a subset] x (min K, max K, min V, max V) of y = x / c over all heads (grp_all; kept by the row's first unit)
};

// Where the rows to compress come from (caller tensors at prefill, the tail at a flush).
struct ZcSrc {
  const void* K;
  const void* V;
  long long sb, sh, sl;  // element strides of (batch, kv head, token)
  int l;                 // rows per (batch, kv head)
};

// One segment's two subsets.
struct ZcSeg {
  int n_tok[2];    // tokens per class
  int tile0[2];    // first tile per class
  int idx_off;     // offset (ints) of this segment's index lists in the idx region
  int run0;        // factor-block index of class 0 (class 1 = run0 + 1)
};

// Re-compression of the window by the decode call that completes it (Alg. 3).
struct ZcFlushArgs {
  int on;
  ZcSeg seg;                             // the segment the window becomes
  unsigned char nnz[ZC_MAX_WINDOW];      // per tail token: probe steps that saw it
};
static_assert(ZC_MAX_WINDOW <= 255, "probe-step counts are kept in bytes");

// Split-K plan of one decode call (identical for every unit).
struct ZcDecodePlan {
  int n_seg;
  int n0[2], nw[2];        // tokens per class: segment 0, re-compressed windows
  int tiles0[2], tilesw[2];
  int split0[2];           // items covering segment 0, per class
  int spi0[2];             // 16-token sub-tiles per item, per class
  int n_tail;
  int ctas_per_sm;         // build of the decode kernel: 3 (wide rings) or 4 (narrow rings)
  int items;               // items per unit
  int cta_items;           // consecutive items one CTA works through
  int fold_tail;           // the tail is attended by the unit's first item CTA, not by a CTA of its own
  int chain_free;          // ZC_FLAG_OVERLAP_CALLS: working CTAs do not wait for the previous kernel
  int l0;
};

// Where in a stream's sequence of decode calls a cache was last changed (a stored tail row,
// a re-compressed window); see zc_order.h.
struct ZcFence {
  int rec;          // stream record, -1: none
  unsigned tag;     // epoch
  int e;            // calls of that epoch that must have completed
  int capturing;
};

struct zc_cache {
  zc_config cfg;
  ZcLayout lay;
  char* base;
  size_t bytes;
  size_t ws_bytes;
  int l0;          // prefill length, -1 before prefill
  int n0[2];
  int nw[2];
  int n_seg;       // 1 + number of re-compressed windows
  int n_tail;
  int step_i;      // decode steps taken in the current window
  int fresh;       // a token was appended since the last decode call (that call takes a step of Alg. 3)
  int n_new;       // tokens appended since prefill
  int tail_nnz[ZC_MAX_WINDOW];
  int last_scores_n;
  int n_sm;
  long long launches;
  // deferred append: the row at tail index n_tail - 1 still lives in the caller's buffers
  const void* pend_k;
  const void* pend_v;
  cudaStream_t pend_stream;
  // the cache's last change by a decode call (a stored tail row, a re-compressed window): its next call waits for it
  ZcFence fence;
};

__host__ __device__ static inline int zc_ceil_div(int a, int b) { return (a + b - 1) / b; }

// Bounds-checked build (-DZC_DEBUG, `python -m paper_2405_14256_b200.build --debug`): index
// arithmetic of the kernels is checked where a tile, a row or a partial is addressed; a check
// that fails records its code (first failure wins) in a word that zc_device_status reports as
// 100 + code, and the access is skipped.  Nothing traps.  In the normal build the macro is empty.
#ifdef ZC_DEBUG
#define ZC_CHECKED(ok, code) (zc_debug_check((ok), (code)))
#else
#define ZC_CHECKED(ok, code) (true)
#endif
enum {
  ZC_DBG_QUANT_ROW = 1,     // quantiser: a gathered token index outside [0, l)
  ZC_DBG_QUANT_TILE = 2,    // quantiser: a tile beyond the class's capacity
  ZC_DBG_DECODE_ITEM = 3,   // decode: an item's sub-tiles beyond the class's capacity
  ZC_DBG_DECODE_PART = 4,   // decode: a partial beyond the workspace region
  ZC_DBG_TAIL_ROW = 5,      // append / decode: a tail row beyond the window
  ZC_DBG_FLUSH_TILE = 6,    // window re-compression: a tile beyond the class's capacity
  ZC_DBG_TOPK_INDEX = 7,    // split: an index list entry beyond its list
};

ZcSeg zc_segment(const zc_cache* c, int seg);
ZcDecodePlan zc_make_plan(const zc_cache* c);

// ---- launchers (each returns a cudaError_t as int) ----
// qp_ws / qp_bytes: room for a dense copy of the probe rows (batch * n_q_heads * n_probe rows of
// 256 bytes, 16-byte aligned); used when large enough.
// lse_rows: non-null = every row's log-sum-exp [batch][n_q_heads][l] is known already (from
// zc_launch_prefill_attention): pass 1 is replaced by a gather of the probe rows' values.
int zc_launch_probe_scores(zc_cache* c, const void* Q, const void* K, int l,
                           const int64_t* qs, const int64_t* ks, const int32_t* P_dev,
                           int n_probe, float* lse_ws, void* qp_ws, size_t qp_bytes,
                           const float* lse_rows, cudaStream_t st);
// Causal attention output O [batch][n_q_heads][l][128] and row log-sum-exp lse [batch][n_q_heads][l].
int zc_launch_prefill_attention(zc_cache* c, const void* Q, const void* K, const void* V, int l,
                                const int64_t* qs, const int64_t* ks, void* O, float* lse, cudaStream_t st);
int zc_launch_gather_probe_lse(zc_cache* c, const float* lse_rows, const int32_t* P_dev, int n_probe, int l,
                               float* lse_probe, cudaStream_t st);
int zc_attention_error_code(int* out);   // 0 or 1: a bounded wait in the prefill attention kernel ran out
int zc_launch_topk(zc_cache* c, int n, int n_s, int idx_off, const int32_t* given_sal,
                   cudaStream_t st);
int zc_launch_quantize(zc_cache* c, const ZcSrc& src, const ZcSeg& seg, cudaStream_t st);
int zc_launch_share_scores(zc_cache* c, int n, cudaStream_t st);
int zc_launch_window_scores(zc_cache* c, const ZcFlushArgs& fl, cudaStream_t st);
int zc_launch_append(zc_cache* c, const void* k_new, const void* v_new, int pos,
                     cudaStream_t st);
// k_new / v_new non-null: the newest tail row is read from them and stored into the tail.
// Calls that may be in flight together on a stream take consecutive regions of ws.
int zc_launch_decode(zc_cache* c, const ZcDecodePlan& plan, const void* q, void* out, int collect,
                     char* ws, size_t ws_bytes, const void* k_new, const void* v_new,
                     const ZcFlushArgs* flush, cudaStream_t st);
// Bytes of ws one call of `items` items per unit takes.
size_t zc_decode_scratch_bytes(const zc_cache* c, int items);
int zc_device_error_code(int* out);
int zc_debug_code_compress(int* out);   // bounds-checked build: first failed check of the compression kernels (0: none)
int zc_debug_code_decode(int* out);     // ... of the append / decode kernels
int zc_probe_error_code(int* out);   // 0 or 1: a bounded wait in a probe-score kernel ran out
// Device address of the per-stream ordering words on the current device (looked up once per
// device; pass nullptr to only perform the look-up).
int zc_order_words(unsigned** ptr);
// Device address of the built-in scratch buffer on the current device (looked up once per device).
int zc_static_scratch(void** ptr);
int zc_launch_export_scores(zc_cache* c, float* out, int n, cudaStream_t st);
int zc_launch_export_segment(zc_cache* c, const ZcSeg& seg, int tensor, int subset,
                             int32_t* idx, uint8_t* codes, float* sz, float* cf,
                             cudaStream_t st);
