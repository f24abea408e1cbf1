/*
 * logquant -- decode-time hot path of LogQuant (arXiv 2503.19950) for NVIDIA B200 (sm_100a).
 *
 * A mixed KV cache per (layer, batch row, KV head):
 *   - a full-precision (bf16) store holding at most 3W tokens, maintained by the log-based
 *     filter of the paper's Algorithm 1 (Sec. 2.5), and
 *   - a 2-bit store that receives the W tokens the filter removes at every window overflow,
 *     quantised with asymmetric min/max groups of G values: keys grouped per channel over G
 *     consecutive removed tokens ("Key-per-channel strategy", Sec. 2.5), values grouped per
 *     token over G consecutive channels, scale and zero stored as bf16.
 * Decode attention (Eq. 2, with the 1/sqrt(d) of the appendix) runs directly on both stores,
 * dequantising in registers; the two stores and the split-K partitions are visited in an
 * arbitrary order and merged with an online-softmax (m, l) reduction, which Eq. 3
 * (position-agnostic attention, Sec. 2.4) permits.
 *
 * Conventions for every call
 *   - Pointers named k, v, q, out are DEVICE pointers unless the name ends in _host.  They are
 *     borrowed: they must stay valid until `stream` has executed the call's work.
 *   - Layout of k, v: [batch, kv_head, token, head_dim] contiguous bf16.  q, out:
 *     [batch, q_head, head_dim].  Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Calls enqueue work and return without synchronising (lq_export and the *_host entry
 *     points synchronise).  Argument and state errors are detected on the host and leave the
 *     cache unchanged; every length is a function of the number of appended tokens, so the
 *     host never has to read one back from the device.
 *   - No call throws, aborts or traps.  One cache must not be used from two threads at once.
 *   - All layers of a cache share one split-K workspace (partial records, arrival counters, sums), and
 *     the kernels rely on stream order to hand it from one launch to the next: every call on one
 *     cache must be enqueued on the same stream, or the caller must order the streams with events.
 *     Calls for different layers on different, unordered streams race on that workspace and give
 *     wrong results without any error.  Different caches are independent.
 *   - There is no CPU implementation: without a CUDA device lq_cache_create fails, except for
 *     the bookkeeping-only mode device == LQ_DEVICE_NONE in which the compute calls return
 *     LQ_ERR_UNSUPPORTED.
 */
#ifndef LQ_H_
#define LQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lq_cache lq_cache_t; /* opaque; owns every device byte it allocates */

typedef enum {
  LQ_OK = 0,
  LQ_ERR_INVALID_ARG = 1, /* null pointer, index out of range, empty cache for attention        */
  LQ_ERR_UNSUPPORTED = 2, /* configuration outside what the kernels implement                   */
  LQ_ERR_OOM = 3,         /* device allocation failed                                           */
  LQ_ERR_WINDOW_FULL = 4, /* lq_append would exceed 3W full-precision tokens (auto_compress=0)  */
  LQ_ERR_NOT_FULL = 5,    /* lq_compress on a layer that holds fewer than 3W full-precision tokens */
  LQ_ERR_CAPACITY = 6,    /* max_tokens would be exceeded, or a size beyond a fixed scratch     */
  LQ_ERR_CUDA = 7         /* a CUDA runtime call or a kernel launch failed                      */
} lq_status_t;

#define LQ_DEVICE_NONE (-1)

/* decode-attention kernel selection */
#define LQ_KERNEL_AUTO 0   /* the tensor-core kernel                                             */
#define LQ_KERNEL_SCALAR 1 /* plain fp32 FMA kernel (slow; kept as an independent cross-check)   */
#define LQ_KERNEL_MMA 2    /* mma.sync tensor-core kernel with bulk-copy staging                 */
#define LQ_KERNEL_UMMA 3   /* tcgen05 kernel: codes unpacked into tensor memory, accumulators in tensor memory
                              (bits = 2 only; the cache then uses the device layout made for it)  */

/* Which tokens an overflow step removes from the 3W full-precision tokens (in age order A[0..3W)):
 *   LQ_FILTER_LOG     Algorithm 1: A[1], A[3], ..., A[2W-1]; kept tokens thin out with distance.
 *   LQ_FILTER_RECENT  comparator, not the paper's method: the W oldest, A[0..W), so that only a recent
 *                     window stays at full precision (the retention rule of the sliding-window
 *                     quantisers the paper compares with, Sec. 2.2-2.3), same memory as LQ_FILTER_LOG. */
#define LQ_FILTER_LOG 0
#define LQ_FILTER_RECENT 1

/* lq_config_t.flags.
 *   LQ_FLAG_OVERLAP_DECODE  Decode-attention launches of DIFFERENT layers of this cache that follow one another
 *     on a stream may overlap: the later launch streams its own layer's stores while the earlier one is still
 *     merging its partials, and waits for it only before it touches the shared split-K workspace (programmatic
 *     dependent launch with the dependency wait moved behind the main loop).  The library applies this only when
 *     its own previous call on the cache was a decode call for another layer on the same stream; what it cannot
 *     see is work the CALLER enqueues in between.  The flag is therefore a promise: between two lq decode calls
 *     for different layers the caller enqueues on that stream either nothing, or only kernels that were launched
 *     without the programmatic-stream-serialization attribute and do not trigger dependents early (plain launches,
 *     which is what frameworks issue by default): then q, k and v are complete before the decode launch starts.
 *     (A launch whose layer got a row from an earlier fused lq_append_decode_attn launch overlaps only once that
 *     launch is known to be complete, which the library derives from the launches enqueued since.)
 *     Without the flag every launch waits for its predecessor before it reads anything. */
#define LQ_FLAG_OVERLAP_DECODE 1

typedef struct {
  int32_t n_layers;      /* independent stacked layer caches, >= 1                               */
  int32_t batch;         /* B: sequences; all share one length                                   */
  int32_t n_q_heads;     /* Hq; Hq % Hkv == 0 and Hq / Hkv <= 8                                  */
  int32_t n_kv_heads;    /* Hkv                                                                  */
  int32_t head_dim;      /* D; only 128 is implemented                                           */
  int32_t window;        /* W of Algorithm 1, <= 512.  W % G != 0 (the paper's W = 42 or 85 with G = 64): removed
                            tokens wait at full precision, in removal order, until G of them form a key group */
  int32_t group;         /* G: quantisation group size, 32 or 64                                 */
  int32_t bits;          /* 2, or 4 (the paper's second precision, Table 3; not with LQ_KERNEL_UMMA) */
  int64_t max_tokens;    /* capacity per sequence (tokens ever appended)                         */
  int32_t auto_compress; /* 1: lq_append runs the overflow step itself when the window is full   */
  int32_t device;        /* CUDA device ordinal, or LQ_DEVICE_NONE for bookkeeping only          */
  int32_t kernel;        /* LQ_KERNEL_*                                                          */
  int32_t n_splits;      /* split-K CTAs per (batch row, KV head); 0 = chosen by the library     */
  int32_t filter;        /* LQ_FILTER_*: which W tokens leave the full-precision store on overflow */
  int32_t flags;         /* LQ_FLAG_* bits, 0 = none                                             */
  /* Optional device allocator (all three NULL / 0: cudaMalloc and cudaFree).  dev_alloc returns device memory of
     at least `bytes` bytes, 256-byte aligned, on `device`, or NULL on failure (the call that needed it then gives
     LQ_ERR_OOM); every block is handed back to dev_free by lq_destroy (or at once when creation fails).  Both
     are called on the host, from the thread that calls into the library, with alloc_ctx passed through. */
  void* (*dev_alloc)(size_t bytes, void* alloc_ctx);
  void (*dev_free)(void* ptr, void* alloc_ctx);
  void* alloc_ctx;
} lq_config_t;

typedef struct {
  int64_t n_seen;   /* tokens appended so far                                                    */
  int64_t n_fp;     /* tokens in the full-precision store (2W < n_fp <= 3W after the first event; up to
                       3W + G - 1 when W % G != 0: those waiting for a full key group count)       */
  int64_t n_quant;  /* tokens in the quantised store (a multiple of G)                           */
  int64_t n_events; /* window overflows processed                                                */
  int64_t bytes_device;        /* device bytes owned by the whole cache (all layers + workspace) */
  int64_t bytes_decode_step;   /* algorithmic bytes one lq_decode_attn on this layer has to read:
                                  B*Hkv*(n_quant*bytes_quant_per_token + n_fp*4*D); q/out excluded */
  int64_t bytes_quant_per_token; /* per KV head: codes + amortised scale/zero (96 at G=32, 80 at G=64) */
  int32_t n_splits;            /* split-K partial records per (batch row, KV head) the next
                                  lq_decode_attn would use                                        */
  int32_t n_ctas;              /* CTAs of its attention kernel (tensor-core kernel; else 0)      */
  int64_t n_kernel_launches;   /* kernels this cache has launched so far (all layers)            */
  int32_t n_ctas_overlapped;   /* CTAs of an attention launch that overlaps the launch before it
                                  (LQ_FLAG_OVERLAP_DECODE: a third of the resident wave; else 0)  */
  int32_t n_launches_overlapped; /* attention launches of this cache so far (all layers) that did overlap the
                                    launch before them                                               */
} lq_info_t;

/*
 * Canonical image of one layer (host buffers supplied by the caller; a null member is skipped).
 * Sizes use n_fp, n_quant from lq_cache_info.  This is the format parity is checked on; the
 * device-side layout is private.
 *   kept_ids  [n_fp]    int32, ascending: ids (append order, from 0) of the full-precision tokens
 *   quant_ids [n_quant] int32, in store order: event order, then age order inside an event
 *   k_codes, v_codes [B][Hkv][n_quant][D/4] uint8: channel 4j+i of a token in bits [2i+1:2i] of byte j
 *                    (bits = 4: [..][D/2], channel 2j+i in bits [4i+3:4i] of byte j)
 *   k_scale, k_zero  [B][Hkv][n_quant/G][D] uint16 (bf16 bit patterns)
 *   v_scale, v_zero  [B][Hkv][n_quant][D/G] uint16
 *   fp_k, fp_v       [B][Hkv][n_fp][D] uint16, rows in kept_ids order
 */
typedef struct {
  int32_t* kept_ids;
  int32_t* quant_ids;
  uint8_t* k_codes;
  uint8_t* v_codes;
  uint16_t* k_scale;
  uint16_t* k_zero;
  uint16_t* v_scale;
  uint16_t* v_zero;
  uint16_t* fp_k;
  uint16_t* fp_v;
} lq_image_t;

/* Create a cache.  Validates the configuration (LQ_ERR_INVALID_ARG / LQ_ERR_UNSUPPORTED),
 * selects cfg->device and allocates both stores and the split-K workspace with cudaMalloc
 * (LQ_ERR_OOM).  *out is written only on success.  (Problem statement: window W of Sec. 2.5,
 * group size G and INT2 of Sec. 3.1.) */
lq_status_t lq_cache_create(const lq_config_t* cfg, lq_cache_t** out);

/* Free the cache and its device memory.  NULL is a no-op.  The caller must have synchronised
 * every stream that still has work of this cache in flight. */
lq_status_t lq_destroy(lq_cache_t* cache);

/* Append n_tokens new tokens (Algorithm 1, the "length(A) < 3W" branch) to one layer.
 * k, v: device, bf16, [B, Hkv, n_tokens, D].  A prompt of n tokens is equivalent to n single
 * appends.  auto_compress = 0: LQ_ERR_WINDOW_FULL if the tokens do not fit below 3W (nothing is
 * appended).  auto_compress = 1: the call is split into fill-to-3W / overflow step / continue;
 * when the layer is still empty and n_tokens > 3W (a prompt), or the layer is in use, n_tokens >= 2W
 * and the window overflows on the way (a chunk of a prompt), the same
 * result -- the same image -- is produced by one kernel launch from the kept/removed sets that
 * Algorithm 1 fixes in advance (the index lists of that launch are copied from pageable host memory
 * on `stream`; calls that ingest prompts must share one stream or be ordered by the caller). */
lq_status_t lq_append(lq_cache_t* cache, int32_t layer, const void* k, const void* v,
                      int32_t n_tokens, void* stream);

/* Window-overflow step (Algorithm 1, else-branch; Fig. 5): of the 3W full-precision tokens in
 * age order A, the W tokens A[1], A[3], ..., A[2W-1] are 2-bit quantised (keys per channel over
 * blocks of G of these tokens in age order, values per token over blocks of G channels; group
 * min/max by warp-shuffle reductions), bit-packed and appended to the 2-bit store; A[0:2W:2] and
 * A[2W:3W] stay.  layer = -1 processes every layer that is full (others are skipped);
 * a single layer that is not full gives LQ_ERR_NOT_FULL. */
lq_status_t lq_compress(lq_cache_t* cache, int32_t layer, void* stream);

/* One-token decode attention over the whole mixed cache of one layer (Eq. 2; order of the two
 * stores and of the split-K partitions is free by Eq. 3).  q: device bf16 [B, Hq, D];
 * sm_scale <= 0 selects 1/sqrt(D); out: device [B, Hq, D], out_dtype 0 = fp32, 1 = bf16.
 * Accumulation is fp32.  The result is reproducible bit for bit from call to call, except when more than
 * 12 CTAs share one (batch row, KV head) -- long contexts with few such pairs --, where the partial results
 * are summed in arrival order.  An empty cache gives LQ_ERR_INVALID_ARG.  Range: any finite bf16 keys, queries
 * and values with up to 4 query heads per KV head; with 5 to 8 the quantised values pass through fp16
 * operands, so value zero-points and scales must lie within fp16 range (|v| < 65504). */
lq_status_t lq_decode_attn(lq_cache_t* cache, int32_t layer, const void* q, float sm_scale,
                           void* out, int32_t out_dtype, void* stream);

/* The same over the full-precision store only: the result of the eviction variants the paper compares
 * with in Sec. 2.3 (tokens the filter removes are dropped instead of quantised).  A comparator for accuracy
 * measurements; the quantised store is still maintained, this call just leaves it out. */
lq_status_t lq_decode_attn_fp_only(lq_cache_t* cache, int32_t layer, const void* q, float sm_scale,
                                   void* out, int32_t out_dtype, void* stream);

/* Left padding of a ragged batch.  pad: HOST array of `batch` int32 >= 0, copied by the call; the first pad[b]
 * token positions of sequence b are padding in every layer.  Padding tokens are appended, filtered and
 * quantised like any token (Algorithm 1 and the quantiser only look at positions), but every decode
 * attention call leaves them out: sequence b attends to its tokens pad[b], pad[b] + 1, ...  Leading key
 * groups of the quantised store that hold nothing but padding of a sequence are not even read for it.
 * May be called at any time and takes effect from the next decode call; NULL clears all padding.  A decode
 * call gives LQ_ERR_INVALID_ARG while some sequence has pad[b] >= the tokens appended to that layer.
 * The masks (about max_tokens / 8 bytes per sequence and layer) are allocated by the first call
 * (LQ_ERR_OOM if that fails) and re-derived on the host and uploaded on the decode call's stream after every
 * overflow step or prompt ingestion of a layer.  The tensor-core kernel shares its CTAs out over the
 * sequences in proportion to the tokens each has left (config n_splits then only caps the share of one
 * (batch row, KV head)).  lq_decode_attn_image_static knows no padding. */
lq_status_t lq_set_padding(lq_cache_t* cache, const int32_t* pad);

/* lq_append of ONE token followed by lq_decode_attn, in one launch: the attention kernel takes the
 * new row from k, v ([B, Hkv, 1, D] bf16, device) where it belongs in its pass over the cache and
 * writes it to the full-precision store on the way (Algorithm 1's append and Eq. 2 of the same
 * step; the result is the one of the two separate calls).  When the window is full (the overflow
 * step has to run in between; auto_compress = 0 then gives LQ_ERR_WINDOW_FULL), the plain kernel
 * is selected, or the cache is so large that the saved launch no longer pays (only without
 * LQ_FLAG_OVERLAP_DECODE: with it a separate append would cost the overlap), the call simply makes
 * the two calls.  Errors leave the cache unchanged. */
lq_status_t lq_append_decode_attn(lq_cache_t* cache, int32_t layer, const void* k, const void* v,
                                  const void* q, float sm_scale, void* out, int32_t out_dtype,
                                  void* stream);

/* One decode step of one layer with HOST buffers: copies k_host, v_host ([B,Hkv,1,D] bf16) and
 * q_host ([B,Hq,D] bf16) to the device, appends (running the overflow step first when the window
 * is full, whatever auto_compress says), runs decode attention and copies the fp32 result to
 * out_host ([B,Hq,D]).  sync != 0: synchronises `stream` before returning.  sync == 0: everything
 * is only enqueued (the host buffers must be pinned and must stay untouched, and out_host is
 * valid, once the caller has synchronised the stream); each layer has its own staging buffers,
 * so steps of different layers may be enqueued back to back.  When k_host, v_host and out_host are
 * page-locked, device-addressable (cudaHostAlloc / cudaHostRegister, as reported by
 * cudaPointerGetAttributes) and 16-byte aligned -- all four buffers --, the kernels read the inputs
 * from and write the result to host memory directly, in the single launch of lq_append_decode_attn (every CTA
 * fetches the query rows of its pair from host memory, about 1 KB; consecutive layers overlap under
 * LQ_FLAG_OVERLAP_DECODE); otherwise every buffer is copied through device staging memory. */
lq_status_t lq_decode_step_host(lq_cache_t* cache, int32_t layer, const void* k_host,
                                const void* v_host, const void* q_host, float sm_scale,
                                float* out_host, int32_t sync, void* stream);

/* Kernel timing for benchmarks.  While enabled, every lq_decode_attn brackets its split-K
 * attention kernel with a pair of CUDA events on the call's stream (at most 8192 pairs are kept;
 * later launches are not timed).  lq_profile_read synchronises the device and returns the summed
 * duration in milliseconds and the number of timed launches since profiling was enabled. */
lq_status_t lq_profile_enable(lq_cache_t* cache, int32_t on);
lq_status_t lq_profile_read(lq_cache_t* cache, double* total_ms, int64_t* n_launches);

/* Device status word of the cache: 0 = healthy; bit 0 = a bounded wait inside a kernel gave up
 * (its output is then invalid).  Kernels never trap or spin for ever; they record the failure
 * here.  Synchronises the device. */
lq_status_t lq_kernel_status(lq_cache_t* cache, int32_t* status_word);

/* Set the status word back to 0 (after the caller has dealt with a failure).  Synchronises the device. */
lq_status_t lq_reset_kernel_status(lq_cache_t* cache);

/* Test hook for the failure path (no counterpart in the paper): the next decode-attention launch of this cache
 * on a tensor-core kernel arms the barrier of its query copy, issues no copy and polls a few hundred times only,
 * so that its bounded wait runs out.  That launch must set bit 0 of the status word, write nothing to `out` and
 * return normally; the cache and the CUDA context stay usable.  Nothing on the GPU faults, traps or hangs. */
lq_status_t lq_debug_stall_next_decode(lq_cache_t* cache);

/* Test hook of the index-check build (library compiled with -DLQ_DEBUG_BOUNDS, where every index that comes from
 * the host's bookkeeping is checked in the kernels; no counterpart in the paper): the next lq_append launches
 * its kernel with a first slot beyond the full-precision store.  The checks must refuse every row, set bit 2
 * of the status word and write nothing.  The normal build returns LQ_ERR_UNSUPPORTED and changes nothing.
 * The cache's contents are undefined after the hooked append (its bookkeeping counts rows that were not
 * written): destroy it. */
lq_status_t lq_debug_bad_slot_next_append(lq_cache_t* cache);

/* Guard words: every device block a cache allocates (through cudaMalloc or the caller's allocator) is
 * followed by 256 guard bytes of a fixed pattern that no kernel may touch.  lq_check_guards synchronises the
 * device, reads them back and stores the number of blocks whose guard was overwritten in *n_damaged
 * (0 = intact): a cheap stand-in for a memory checker that the tests call on every cache they close. */
lq_status_t lq_check_guards(lq_cache_t* cache, int32_t* n_damaged);

/* Introspection (host-side bookkeeping only; never synchronises). */
lq_status_t lq_cache_info(const lq_cache_t* cache, int32_t layer, lq_info_t* info);

/* Copy the canonical image of one layer into the caller's HOST buffers.  Synchronises the device. */
lq_status_t lq_export(const lq_cache_t* cache, int32_t layer, lq_image_t* image_host);

/* Load a canonical image (as lq_export wrote it; HOST buffers) into a layer that is still EMPTY: the inverse of
 * lq_export, for checkpoint / resume (no counterpart in the paper).  n_seen = tokens the exported layer had seen
 * (lq_info_t.n_seen), n_fp and n_quant = its sizes.  Algorithm 1 never looks at the data, so the library
 * rebuilds its bookkeeping by replaying n_seen appends on token ids and then writes both stores from the image
 * in its private layout; decode and further appends continue exactly as on the exported cache.  The cache must
 * have the exporting cache's batch, heads, window, group, bits and filter (its kernel, hence its device layout,
 * may differ); image->kept_ids and image->quant_ids, when not NULL, are compared with the replayed lists.
 * LQ_ERR_INVALID_ARG: layer not empty, sizes or id lists that are not those of this configuration after n_seen
 * tokens, or a missing array; nothing changes then.  Synchronises the device. */
lq_status_t lq_import(lq_cache_t* cache, int32_t layer, const lq_image_t* image_host, int64_t n_seen, int64_t n_fp,
                      int64_t n_quant);

/* Host-side bookkeeping only (works in LQ_DEVICE_NONE mode): ids of the tokens the next
 * lq_compress on `layer` would remove, in removal order (W entries; LQ_ERR_NOT_FULL if the
 * layer holds fewer than 3W full-precision tokens). */
lq_status_t lq_next_evicted_ids(const lq_cache_t* cache, int32_t layer, int32_t* ids_host);

/*
 * Device-resident canonical image of one layer: the same arrays and layouts as lq_image_t, but the
 * pointers are DEVICE pointers into memory the caller owns (ids are not needed for attention).
 */
typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, head_dim, group;
  int32_t bits;      /* code width of k_codes / v_codes: 2 or 4 (anything else: LQ_ERR_INVALID_ARG)  */
  int32_t n_fp;      /* rows of fp_k / fp_v per (batch row, KV head)                              */
  int64_t n_quant;   /* quantised tokens per (batch row, KV head); a multiple of group            */
  const uint16_t* fp_k;    /* [B][Hkv][n_fp][D] bf16 bits                                          */
  const uint16_t* fp_v;
  const uint8_t* k_codes;  /* [B][Hkv][n_quant][D/4] (bits = 2) or [..][D/2] (bits = 4)                */
  const uint8_t* v_codes;
  const uint16_t* k_scale; /* [B][Hkv][n_quant/G][D]                                               */
  const uint16_t* k_zero;
  const uint16_t* v_scale; /* [B][Hkv][n_quant][D/G]                                               */
  const uint16_t* v_zero;
} lq_device_image_t;

/*
 * Decode attention that allocates nothing (the paper has no counterpart: this entry point exists for
 * callers, not for the method).  For processes that may not call cudaMalloc -- a server that handed
 * its whole memory budget to a fixed arena at start-up, code running under another component's
 * allocator policy, or code called while a stream is being captured -- lq_cache_create is out of
 * reach, because it allocates the stores and the split-K workspace.  Here the caller keeps the cache
 * itself, as a canonical image in its own device memory, and passes q ([B,Hq,D] bf16, device) and
 * out ([B,Hq,D] fp32, device); the only scratch, the split-K partials, lives in a fixed 4.06 MiB
 * array inside the library image (held by every GPU that loads the library until the process exits).
 * The result equals lq_decode_attn on the same cache content (plain fp32 kernel, same tolerance).
 *
 * Limits and rules:
 *   - batch * n_q_heads <= 8192 (LQ_ERR_CAPACITY otherwise: the scratch holds 8192 partial records);
 *     head_dim 128, group 32 or 64, n_q_heads / n_kv_heads <= 8 (LQ_ERR_UNSUPPORTED otherwise); bits 2 or 4,
 *     which must be the width the codes of the image were packed with (LQ_ERR_INVALID_ARG for other values).
 *   - No cudaMalloc, cudaFree or other allocating call is made, ever.  The first call on each device
 *     looks up the scratch's device address (cudaGetSymbolAddress) with that device current; make
 *     that first call before any stream capture begins.
 *   - All calls on a device share the one scratch array.  Nothing in it needs clearing (every record a
 *     call reads, it has written first), but two calls whose kernels overlap on the GPU -- different
 *     streams, or the same image from two threads -- race on it: serialise them.
 *   - Enqueues two kernels on `stream` and returns without synchronising.
 */
lq_status_t lq_decode_attn_image_static(const lq_device_image_t* image, const void* q, float sm_scale,
                                        float* out, void* stream);

const char* lq_status_str(lq_status_t status);

/* Sticky description of the last CUDA error seen by this cache ("" if none). */
const char* lq_last_error(const lq_cache_t* cache);

#ifdef __cplusplus
}
#endif
#endif /* LQ_H_ */
