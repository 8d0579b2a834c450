/*
 * zipcache.h -- C ABI of the B200 (sm_100a) quantize-and-attend library.
 *
 * The library implements the mixed-precision KV-cache path of ZipCache:
 *   prefill:  probe attention (Eq. 9) -> normalised attention score (Eq. 8)
 *             -> split by saliency ratio (Alg. 2) -> channel-separable tokenwise
 *             quantisation (Alg. 1, Eq. 5, Eq. 6) -> packed 4-bit / 2-bit codes;
 *   decode:   append of the new token at full precision (Eq. 3, Alg. 3),
 *             single-query attention over the whole cache with in-kernel
 *             dequantisation (Eq. 4, Alg. 3), probe-row collection and the
 *             re-compression of every `window` generated tokens (Alg. 3).
 *
 * Conventions
 *   - "unit" = one (batch, KV head).  Query head h reads KV head h / G,
 *     G = n_q_heads / n_kv_heads.
 *   - Every pointer is tagged [host] or [device].  The library never allocates
 *     or frees device memory and never creates streams: the caller owns the
 *     cache buffer and the workspace, and all work is enqueued on the stream
 *     passed in.  Inputs may be released once the stream has passed the call.
 *   - Every function returns 0 (ZC_OK) or a negative status; nothing throws
 *     and device code never traps.  NaN / Inf in inputs give undefined values
 *     but no fault.
 *   - Device pointers must be 16-byte aligned (ZC_EALIGN otherwise).
 */
#ifndef ZIPCACHE_H_
#define ZIPCACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* zc_stream_t; /* a cudaStream_t */

enum { ZC_F16 = 0, ZC_BF16 = 1 };
/* How keys are quantised (values always by CSTQuant, Alg. 1).  ZC_K_CHANNEL is the paper's own
 * setting (Sec. 4.1, Table 1 last row, Alg. 2 "ChannelQuant"): Eq. 5 with minimum and maximum
 * taken over the tokens of a subset, one (s, z) pair per channel and none per token, which
 * saves 8 bytes per cached token. */
enum { ZC_K_CST = 0, ZC_K_CHANNEL = 1 };
/* Who shares a saliency decision (Sec. 4.2 speaks of the saliency "of each token"; the paper
 * does not say how heads are combined).  ZC_SCOPE_KV_HEAD: one decision per (batch row, KV head)
 * from that head's own normalised scores (Eq. 8 over its query heads).  ZC_SCOPE_TOKEN: one
 * decision per token of a batch row, shared by all its KV heads: the token's score is the mean
 * of its per-KV-head normalised scores, in the prompt and in every re-compressed window, so
 * every head of the row keeps the same tokens at the higher precision.  With ZC_SCOPE_TOKEN the
 * window is re-compressed by kernels of its own that follow the decode kernel of the call that
 * completes it (the heads' statistics must meet first), so it cannot be combined with
 * ZC_FLAG_OVERLAP_CALLS (zc_cache_bytes / zc_cache_init return ZC_EINVAL). */
enum { ZC_SCOPE_KV_HEAD = 0, ZC_SCOPE_TOKEN = 1 };

enum {
  ZC_OK = 0,
  ZC_EINVAL = -1,    /* bad shape / ratio / bit-width / stride / probe list */
  ZC_ECAPACITY = -2, /* more tokens than the cache or workspace was sized for */
  ZC_ESTATE = -3,    /* call out of order (e.g. decode before prefill) */
  ZC_EALIGN = -4,    /* pointer not 16-byte aligned */
  ZC_ECUDA = -5,     /* a CUDA runtime call or launch failed */
  ZC_ESCRATCH = -6   /* zc_decode_attention_noalloc: the call needs more scratch than the
                        library's built-in buffer holds */
};

#define ZC_MAX_WINDOW 128

/* zc_config.flags.  With ZC_FLAG_DEFER_APPEND, zc_append enqueues nothing: the new row is
 * taken straight from k_new / v_new by the next zc_decode_attention on the same cache and
 * stream, which also stores it into the tail (Alg. 3's concat and attention as one step: one
 * launch less and no wait between the two).  The caller then promises that k_new and v_new
 * stay valid and unchanged until the stream has passed that zc_decode_attention call.  Any
 * other call on the cache first performs the pending append as its own launch. */
#define ZC_FLAG_DEFER_APPEND 1
/* With ZC_FLAG_OVERLAP_CALLS the caller PROMISES that, on the stream it passes, a decode call of
 * this cache is preceded only by work that has completed or by other zc_decode_attention /
 * zc_append calls of this library (the layers of a benchmark, caches of independent requests),
 * with no kernel of another library between them.  The decode kernel then does not wait for the
 * kernel before it: consecutive calls run side by side on the GPU, ordered among themselves only
 * where their buffers require it (see zc_decode_attention), and a call is cut into few large
 * work items, which is best when several calls share the GPU.
 * Without the flag (the default) every decode kernel waits for everything that precedes it on
 * the stream before it reads q, k_new, v_new or the cache -- also when the kernel before it is
 * one that lets its successors start early (programmatic dependent launch), e.g. the projection
 * that produces q -- and a call is cut into items sized for a call that has the GPU to itself. */
#define ZC_FLAG_OVERLAP_CALLS 2
/* With ZC_FLAG_OUT_F32 zc_decode_attention stores its result as fp32 (out [device]
 * b x h_q x d floats) instead of rounding it to cfg.dtype.  A 16-bit output cannot be closer
 * to the exact result than half a unit in its last place (bf16: 2e-3 from |o| = 0.25 on), so
 * this is the form in which the kernel's own arithmetic (Eq. 4 over the dequantised cache)
 * can be compared with a reference at a tolerance below that. */
#define ZC_FLAG_OUT_F32 4
/* With ZC_FLAG_PARAMS_F16 the quantisation parameters are stored in 16 bits each, as Appendix A
 * counts them: the channel factors and the token scales as fp16 values, ROUNDED UP before the
 * codes are formed (a scale rounded down would no longer cover its token's range), the zero
 * points as 16-bit integers; a cached token then takes 8 bytes of parameters instead of 16.
 * For CSTQuant on keys and values (ZC_K_CST) at 2 or 4 bits; the window is re-compressed by
 * kernels of their own behind the decode kernel of the call that completes it, so the flag
 * cannot be combined with ZC_FLAG_OVERLAP_CALLS (ZC_EINVAL for either violation). */
#define ZC_FLAG_PARAMS_F16 8
/* With ZC_FLAG_GROUP_ALL_HEADS a token's scale and zero point are taken over the channels of ALL
 * KV heads of its batch row (Alg. 1 as printed: X in R^{l x hd}; Sec. 4.1 counts 2bl token
 * parameters per tensor), not over one head's head_dim channels; every head's tiles carry the
 * row's shared pair.  The heads must agree on the subsets, so it needs ZC_SCOPE_TOKEN (and with
 * it no ZC_FLAG_OVERLAP_CALLS); 16-bit classes are not admitted (ZC_EINVAL otherwise).
 * Channelwise keys have no token parameters: with ZC_K_CHANNEL only the values are grouped. */
#define ZC_FLAG_GROUP_ALL_HEADS 16

/* Plain-data configuration; set struct_size = sizeof(zc_config). */
typedef struct {
  int32_t struct_size;
  int32_t dtype;          /* ZC_F16 | ZC_BF16: type of Q, K, V, q, k, v, out */
  int32_t batch;          /* b */
  int32_t n_q_heads;      /* h_q, multiple of n_kv_heads, G <= 8 */
  int32_t n_kv_heads;     /* h_kv */
  int32_t head_dim;       /* d, must be 128 */
  int32_t max_prefill;    /* largest l accepted by zc_prefill_compress */
  int32_t max_new_tokens; /* decode capacity (tokens appended after prefill) */
  int32_t window;         /* tokens kept at full precision before re-compression
                             (Alg. 3 uses 100); 8 <= window <= ZC_MAX_WINDOW */
  int32_t bits_hi;        /* bit-width of salient tokens: 8, 4, 2, or 16 (kept as they are: the
                             "16/16" and "16/2" settings of Table 3) */
  int32_t bits_lo;        /* bit-width of regular tokens: 8, 4, 2 or 16; a cache with an 8-bit
                             class cannot also have a 16-bit one (ZC_EINVAL) */
  int32_t flags;          /* 0 or an OR of the ZC_FLAG_* values above */
  double saliency_ratio;  /* r in [0,1]; n_salient = floor(r * n) */
  int32_t k_scheme;       /* quantiser of the keys: ZC_K_CST (Alg. 1 on K and V) or ZC_K_CHANNEL
                             (channelwise keys, Sec. 4.1 last paragraph / Alg. 2; values stay CST) */
  int32_t scope;          /* ZC_SCOPE_KV_HEAD (0) or ZC_SCOPE_TOKEN: who shares a saliency decision */
} zc_config;

typedef struct zc_cache zc_cache; /* small host-side handle */

/* Sizes [host].  cache_bytes: device buffer for the compressed cache;
 * workspace_bytes: device scratch shared by all calls (in prefill: probe positions, probe-row
 * statistics and a dense copy of the probe rows; in decode: split-K partial results, with room
 * for 16 calls in flight together).  Either out pointer may be NULL. */
int zc_cache_bytes(const zc_config* cfg, size_t* cache_bytes, size_t* workspace_bytes);

/* Create a handle over caller-owned device memory `dev_mem` [device, >= cache_bytes,
 * 256-byte aligned].  No device work is enqueued.  *out is freed with zc_cache_free,
 * which releases the host handle only. */
int zc_cache_init(void* dev_mem, size_t bytes, const zc_config* cfg, zc_cache** out);
void zc_cache_free(zc_cache* c);

/* Probe selection (Sec. 4.3 "random+recent"): ascending positions made of the last
 * max(1, floor(rho_recent*l)) tokens plus floor(rho_random*l) of the others, drawn by a
 * partial Fisher-Yates shuffle driven by splitmix64(seed).  out [host] must hold
 * zc_probe_count(l, ...) entries; *n_out receives the count. */
int zc_probe_count(int l, double rho_recent, double rho_random);
int zc_default_probes(int l, double rho_recent, double rho_random, uint64_t seed,
                      int32_t* out, int* n_out);

/* Prefill compression (Alg. 2 without its attention-output line).
 *   Q [device] b x h_q x l x d, K, V [device] b x h_kv x l x d, element type cfg.dtype,
 *   d contiguous; q_strides / kv_strides [host] = strides of (batch, head, token) in
 *   ELEMENTS (multiples of 8).
 *   probe_pos [host] n_probe ascending token positions, the last one equal to l-1
 *   (Eq. 9's probe rows); ignored when salient_idx is given.
 *   salient_idx [device or NULL]: test hook -- b x h_kv x floor(r*l) ascending token
 *   indices to use as the salient set instead of computing Eq. 8 / the split.
 *   workspace [device] >= workspace_bytes from zc_cache_bytes.
 * Resets the cache to one compressed segment of l tokens and an empty tail. */
int zc_prefill_compress(zc_cache* c, const void* Q, const void* K, const void* V, int l,
                        const int64_t q_strides[3], const int64_t kv_strides[3],
                        const int32_t* probe_pos, int n_probe, const int32_t* salient_idx,
                        void* workspace, size_t workspace_bytes, zc_stream_t stream);

/* Prefill attention output (Eq. 2 with the causal mask; Alg. 2's line "O = FlashAttention(Q, K,
 * V)", Appendix B): O [device] b x h_q x l x d (contiguous, cfg.dtype) = Softmax(Q K^T /
 * sqrt(d)) V, row i over keys j <= i, and row_lse [device] b x h_q x l floats, every row's
 * base-2 log-sum-exp of its scaled logits (log2 sum_j 2^(q_i.k_j log2(e) / sqrt(d))).  Q, K, V and
 * their strides as for zc_prefill_compress.  The cache is not touched (the handle supplies the
 * shapes).  Needs the driver's tensor-map entry point (ZC_ECUDA "not supported" without it). */
int zc_prefill_attention(zc_cache* c, const void* Q, const void* K, const void* V, int l,
                         const int64_t q_strides[3], const int64_t kv_strides[3], void* O,
                         float* row_lse, zc_stream_t stream);

/* zc_prefill_compress for a caller that has just run zc_prefill_attention on the same Q and K:
 * row_lse [device] (that call's output) stands in for the first of the two probe-score passes
 * (Eq. 9's row statistics), which is then not run; everything else, and the resulting cache, is
 * the same. */
int zc_prefill_compress_lse(zc_cache* c, const void* Q, const void* K, const void* V, int l,
                            const int64_t q_strides[3], const int64_t kv_strides[3],
                            const int32_t* probe_pos, int n_probe, const float* row_lse,
                            void* workspace, size_t workspace_bytes, zc_stream_t stream);

/* Append (Eq. 3, Alg. 3): k_new, v_new [device] b x h_kv x d, contiguous, are copied
 * verbatim into the full-precision tail.  ZC_ECAPACITY beyond max_new_tokens.  With
 * ZC_FLAG_DEFER_APPEND the copy happens inside the next zc_decode_attention (see the flag). */
int zc_append(zc_cache* c, const void* k_new, const void* v_new, zc_stream_t stream);

/* Decode attention (Eq. 4, Alg. 3): q [device] b x h_q x d -> out [device] b x h_q x d,
 * softmax(q K^T / sqrt(d)) V over every cached token, codes dequantised in the kernel.
 * The step counter of the current window advances; on a probe step (is_probe_step != 0,
 * or one of the last five steps of a window) this step's attention over the tail's
 * tokens is added to the window statistics; the call that takes the window's last step
 * also re-compresses the tail into a new segment, inside the same kernel (no further launch,
 * no host synchronisation); with ZC_SCOPE_TOKEN or ZC_FLAG_PARAMS_F16 by five or six small kernels
 * launched behind it on the same stream (still no host synchronisation).
 * Only a call that follows a zc_append takes a step of Alg. 3; a further call on the same tail
 * (the same token queried again) attends the cache as it is and leaves the window's counters,
 * statistics and segments alone.
 * Ordering.  Default: the call's kernel starts its work after everything issued before it on
 * the stream has completed, whoever launched it.  With ZC_FLAG_OVERLAP_CALLS: consecutive calls
 * on one stream may run at the same time on the GPU; the library orders a call after the
 * earlier ones whenever it reads or overwrites one of their outputs, overwrites one of their
 * inputs, or updates the same cache's window statistics; it cannot see other aliasing, so q,
 * k_new, v_new and out of calls issued back to back must not overlap buffers that an earlier
 * call of the stream still uses in any other way, and (the flag's promise) no kernel of another
 * library may sit between the calls.  In both modes the workspace must not be used by calls on
 * another stream at the same time, and CUDA graphs captured from one stream must not be
 * replayed at the same time on several streams (the calls of a capture share one ordering
 * word per captured stream). */
int zc_decode_attention(zc_cache* c, const void* q, void* out, int is_probe_step,
                        void* workspace, size_t workspace_bytes, zc_stream_t stream);

/* ---- parity / export: canonical layouts written to caller buffers [device] ---- */
/* Normalised scores (Eq. 8) of the most recent compression: p_tilde b x h_kv x n floats,
 * n = l after prefill, window after a re-compression. */
int zc_export_scores(zc_cache* c, float* p_tilde, zc_stream_t stream);
/* Number of tokens in (segment, subset); subset 0 = salient, 1 = regular. */
int zc_segment_tokens(const zc_cache* c, int segment, int subset);
int zc_num_segments(const zc_cache* c);
int zc_tail_tokens(const zc_cache* c);
/* One subset of one segment, all units: idx b x h_kv x n int32 (ascending positions
 * within the segment); codes b x h_kv x n x (d*bits/8) bytes in canonical packing
 * (4-bit: element 2m low nibble, 2m+1 high nibble of byte m; 2-bit: element 4m+j in
 * bits [2j,2j+1] of byte m); sz b x h_kv x n x 2 floats (scale, zero point);
 * cf b x h_kv x d floats (channel factors).  tensor 0 = K, 1 = V.  Any out may be NULL.
 * A subset kept at 16 bits exports its rows' bytes as codes (256 per token) and nothing else.
 * Keys under ZC_K_CHANNEL have no per-token parameters and no channel factors: for tensor 0,
 * sz then receives b x h_kv x d x 2 floats, the (scale, zero point) of every channel, and cf
 * is left untouched. */
int zc_export_segment(zc_cache* c, int segment, int tensor, int subset, int32_t* idx,
                      uint8_t* codes, float* sz, float* cf, zc_stream_t stream);

/* Size of the scratch buffer built into the library for zc_decode_attention_noalloc. */
#define ZC_NOALLOC_SCRATCH_BYTES (4u << 20)

/* The paper has no counterpart for this entry point; it exists for integration reasons.
 * Same operation, arguments and state changes as zc_decode_attention, for callers that have
 * no way to hand the library a workspace: code that runs where device allocation is not
 * allowed or not possible -- a plug-in inside a serving process whose memory pool owns the
 * whole device and forbids further cudaMalloc calls, a latency-critical loop that must not
 * enter the allocator, a caller that has already given away its memory budget.  The split-K
 * partial results go to a fixed buffer of ZC_NOALLOC_SCRATCH_BYTES that is
 * part of the library image (every GPU that loads the library carries it until the process
 * ends); the caller still owns q [device] and out [device].  The call allocates and frees
 * nothing.
 *   - ZC_ESCRATCH, with nothing enqueued, when the cache's shape needs more than the
 *     built-in buffer (about batch * n_q_heads * (items + 8) * 528 bytes, items = split-K
 *     pieces per KV head, 8 = tiles of the full-precision tail; use zc_decode_attention with a
 *     caller workspace then).
 *   - The buffer's device address is looked up once per device (a synchronous runtime
 *     query), by zc_cache_init when a device is current there, else by the first call of
 *     this entry point on the device: that first call then belongs outside any stream capture.
 *   - All calls share the one buffer, whatever cache they work on.  Calls that follow one
 *     another in ONE stream get separate parts of it or are ordered by the library; calls in
 *     different streams, or from several host threads, that may run at the same time on the
 *     GPU overwrite each other's partial results.  Nothing in the buffer has to survive between calls and nothing in it
 *     has to be cleared: each call rewrites every word it later reads. */
int zc_decode_attention_noalloc(zc_cache* c, const void* q, void* out, int is_probe_step,
                                zc_stream_t stream);

/* Algorithmic bytes one zc_decode_attention call must read in the cache's current
 * state (packed codes + per-token parameters + tail + channel factors + q and out). */
int64_t zc_decode_bytes(const zc_cache* c);
/* Kernel launches enqueued by this library since the handle was created. */
int64_t zc_launch_count(const zc_cache* c);

/* Synchronises the device and reads the library's device-side error word into *code
 * [host]: 0 = none, 1 = a bounded wait on an asynchronous copy inside the decode kernel
 * ran out, 2 = a bounded wait for an earlier decode call of the stream ran out, 3 = a bounded wait
 * on the tensor cores inside a probe-score or prefill-attention kernel ran out (outputs are then invalid).  Device code never traps or spins forever. */
int zc_device_status(int* code);

/* Host-only model of the ordering the library applies to zc_decode_attention calls issued on
 * one stream (the contract stated at zc_decode_attention): what each call's kernel waits for
 * before it reads its inputs and before it writes.  These two functions make no CUDA call,
 * need no device and keep a table of their own, apart from the one real calls use; they exist
 * so that the rules can be checked on any machine.  Not thread-safe.
 *
 * zc_order_model_reset forgets every stream and cache of the model.
 *
 * zc_order_model_call books one call.  stream_id: any integer naming the stream; cache_id in
 * [0, 16) names the cache; addr [host] = the addresses of q, k_new, v_new, out as integers
 * (k_new = v_new = 0: the call changes nothing in the cache), of io_bytes (q, out) and kv_bytes (k_new,
 * v_new); collect = is_probe_step; ws_addr / ws_bytes = the workspace, need = the bytes one
 * call uses of it; capture_id = 0 outside stream capture, else the capture's id.
 * result [host, 8 ints] = {epoch_start (1: launched without early start, everything issued
 * before it on the stream has completed), e (index of the call in its epoch), need_start
 * (the first need_start calls of the epoch have completed before this one reads its inputs;
 * <= 0: none), need_end (likewise before it writes anything), slot (workspace region and
 * arrival counter), tag (12-bit epoch number), record (stream record used), drain (1: the
 * record was taken from another stream, which a real call drains first)}.
 * Returns ZC_OK, or ZC_EINVAL (null pointer, cache_id out of range, need = 0 or > ws_bytes).
 */
void zc_order_model_reset(void);
int zc_order_model_call(uint64_t stream_id, int cache_id, const uint64_t addr[4], uint64_t io_bytes,
                        uint64_t kv_bytes, int collect, uint64_t ws_addr, uint64_t ws_bytes,
                        uint64_t need, uint64_t capture_id, int result[8]);

const char* zc_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* ZIPCACHE_H_ */
