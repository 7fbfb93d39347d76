/*
 * kvp.h - C ABI of the composed-cache query-prefill library (KV Packet serving path) for NVIDIA B200.
 *
 * The paper's serving step (Section 3.1; Section 3.2 step 4): N document KV caches ("packets"), each
 * computed offline and wrapped in header/trailer soft-token adapters (Eq. 2), are re-aligned to their
 * positions in the request by one RoPE rotation per key (Eq. 1), concatenated without recomputation,
 * and the query tokens then attend causally over everything before them (Fig. 2(d)).
 *
 * Conventions
 *   - every call returns a kvp_status (0 = KVP_OK); nothing throws, aborts or traps the device;
 *   - all argument checking happens on the host before any kernel is launched;
 *   - kernels are enqueued on the caller's stream (a cudaStream_t passed as void*; NULL = default
 *     stream) and the call returns without synchronising unless stated;
 *   - "device" pointers are CUDA device addresses on the context's GPU, "host" pointers are ordinary
 *     host addresses; the library never allocates device memory: the caller lends it a pool and a
 *     workspace at kvp_create and keeps them alive until kvp_destroy;
 *   - ids are dense int32 counted from 0 in registration order;
 *   - element type is the context's dtype (float32 or bfloat16) for every K/V/Q/out buffer.
 */
#ifndef KVP_H_
#define KVP_H_

#include <stdint.h>

#if defined(__GNUC__)
#define KVP_API __attribute__((visibility("default")))
#else
#define KVP_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum kvp_status {
    KVP_OK = 0,
    KVP_ERR_INVALID = 1,      /* bad argument (null pointer, out-of-range value, bad CSR)          */
    KVP_ERR_CAPACITY = 2,     /* pool, workspace or a configured maximum would be exceeded         */
    KVP_ERR_NOT_FOUND = 3,    /* unknown packet / adapter / assembly id                            */
    KVP_ERR_STATE = 4,        /* call not possible in this state (e.g. host-only context)          */
    KVP_ERR_UNSUPPORTED = 5,  /* valid request that this build has no kernel for                   */
    KVP_ERR_CUDA = 6,         /* a CUDA runtime/driver call failed (text in kvp_last_error)        */
    KVP_ERR_TIMEOUT = 7       /* a bounded device-side wait ran out (see kvp_status_word)          */
} kvp_status;

enum { KVP_DTYPE_F32 = 0, KVP_DTYPE_BF16 = 1 };

/* kvp_assemble flags */
enum {
    KVP_REBASE = 1u,          /* rotate every cached key from its cache-time position to its slot (Eq. 1) */
    KVP_MATERIALIZE = 2u      /* also copy the whole composed prefix into the workspace cache             */
};

/* kvp_query_prefill flags */
enum {
    KVP_ROPE_QUERY = 1u,      /* q and k_new are raw: rotate them at positions prefix_len[b] + i        */
    KVP_FORCE_SIMPLE = 2u,    /* use the plain fp32 CUDA-core kernel (cross-check path, any dtype)      */
    KVP_CONTINUE = 4u,        /* the q_len tokens follow the rows this layer's earlier calls appended   */
    KVP_PRECISE_QK = 8u,      /* tcgen05 path: carry the re-based operand of q.k in two bf16 numbers    */
    KVP_PARTIAL = 16u,        /* `out` receives un-normalised partial results (see kvp_merge_partials)  */
    KVP_SKIP_QUERY_BLOCK = 32u /* with KVP_PARTIAL: leave the query's own keys to another rank           */
};

typedef struct kvp_ctx kvp_ctx;

typedef struct kvp_config {
    int32_t struct_bytes;       /* = sizeof(kvp_config)                                               */
    int32_t device;             /* CUDA device ordinal; -1 = host-only planning context: registration
                                   records sizes, kvp_assemble/kvp_export_plan work, nothing can run  */
    int32_t n_layers;
    int32_t n_q_heads;
    int32_t n_kv_heads;         /* must divide n_q_heads; q head h reads kv head h / (Hq/Hkv)         */
    int32_t head_dim;           /* 64 or 128                                                          */
    int32_t dtype;              /* KVP_DTYPE_*                                                        */
    int32_t rope_pairing;       /* 0: pairs (i, i + d/2);  1: pairs (2i, 2i + 1)                      */
    double rope_theta;          /* theta_i = rope_theta^(-2i/d), i < d/2                              */
    const double *inv_freq;     /* optional host array [head_dim/2] overriding rope_theta; copied     */
    double softmax_scale;       /* 0 -> 1/sqrt(head_dim)                                              */
    void *pool;                 /* device; K/V store for registered packets and adapters              */
    uint64_t pool_bytes;        /* capacity in tokens = pool_bytes / kvp_token_bytes(cfg)             */
    void *workspace;            /* device; plans, staged rows, appended query K/V, split partials     */
    uint64_t workspace_bytes;   /* at least kvp_workspace_bytes(cfg)                                  */
    int32_t max_packets;
    int32_t max_adapters;
    int32_t max_batch;          /* requests per assembly                                              */
    int32_t max_slots;          /* packets per assembly, summed over its requests                     */
    int32_t max_prefix_tokens;  /* composed prefix length of one request                              */
    int32_t max_query_tokens;   /* q_len                                                              */
    int32_t max_ws_rows;        /* workspace K/V rows per assembly: sum over requests of
                                   (adapter tokens + max_query_tokens), or with KVP_MATERIALIZE of
                                   (prefix tokens + max_query_tokens)                                  */
    int32_t max_assemblies;     /* assemblies alive at once (ring; ids older than this are dropped)   */
    int32_t max_compressed;     /* compressed packets one assembly may use (0: none; sizes the per-layer
                                   tile lists and the table of kept counts)                            */
} kvp_config;

/* Bytes of pool one token occupies (K and V, all layers and kv heads).  0 if cfg is invalid. */
KVP_API uint64_t kvp_token_bytes(const kvp_config *cfg);

/* Workspace size the configuration needs.  0 if cfg is invalid. */
KVP_API uint64_t kvp_workspace_bytes(const kvp_config *cfg);

/*
 * Create a context on cfg->device.  The pool and the workspace are borrowed, must be 1024-byte
 * aligned, and are zero-filled here (stream 0, synchronised before return).  Errors: KVP_ERR_INVALID
 * (shape/dtype/alignment), KVP_ERR_CAPACITY (workspace too small), KVP_ERR_CUDA.
 */
KVP_API int32_t kvp_create(const kvp_config *cfg, kvp_ctx **out);

/* Free host resources.  Device memory belongs to the caller; synchronises the device first. */
KVP_API int32_t kvp_destroy(kvp_ctx *ctx);

/*
 * Register one packet: the per-layer K/V of a document as it was computed offline for the
 * wrapped document (Section 3.1).  k, v: device, layout [n_layers][n_tokens][n_kv_heads][head_dim];
 * k is post-RoPE for positions cache_pos0 + t.  The rows are copied into the pool (kv-head-major
 * planes) on `stream`; the source may be freed once the stream has passed this point.  Pool rows are
 * assigned densely in registration order.  In a host-only context k, v may be NULL.
 * Errors: INVALID (n_tokens <= 0, null pointers), CAPACITY (max_packets or pool full), CUDA.
 */
KVP_API int32_t kvp_register_packet(kvp_ctx *ctx, const void *k, const void *v, int32_t n_tokens,
                            int32_t cache_pos0, void *stream, int32_t *packet_id);

/*
 * Register one packet whose K/V stay in host memory until a request uses it (the CPU-to-GPU cache transfer
 * that the paper counts inside time-to-first-token, Section 4.3).  Pool rows are reserved now; nothing is copied.
 * The first kvp_assemble that names the packet enqueues the copy on a stream the context owns, layer by layer,
 * and kvp_query_prefill(layer) makes its stream wait for that layer only: the transfer of layer l+1 runs while
 * layer l is attended to.  After that the packet is resident like any other, until kvp_evict_packet.
 *   k_host, v_host   host, layout [n_layers][n_kv_heads][n_tokens][head_dim] (the pool's own plane order, so a
 *                    layer of a packet is one strided copy); k post-RoPE for positions cache_pos0 + t.  The
 *                    buffers stay with the caller and must remain valid while the packet is registered; pinned
 *                    memory is needed for the copies to overlap anything.
 * In a host-only context the pointers may be NULL.  Not available for compressed packets.
 * Errors: INVALID, CAPACITY (max_packets or pool full).
 */
KVP_API int32_t kvp_register_packet_host(kvp_ctx *ctx, const void *k_host, const void *v_host, int32_t n_tokens,
                                 int32_t cache_pos0, int32_t *packet_id);

/*
 * Mark a packet registered with kvp_register_packet_host as no longer on the device: the next kvp_assemble
 * that names it copies it in again (into the same pool rows).  Eviction frees no pool capacity: the packet keeps
 * its rows reserved and no other packet can take them; it only forces the copy to happen again (a packet whose
 * host copy changed, a transfer to be timed).  The caller must not evict a packet that work already enqueued
 * still reads, other than on the stream it passes to that next kvp_assemble.
 * Errors: NOT_FOUND, STATE (the packet has no host copy).
 */
KVP_API int32_t kvp_evict_packet(kvp_ctx *ctx, int32_t packet_id);

/*
 * Register one compressed packet: a document cache after unstructured KV pruning (Section 4.3,
 * "Compatibility with KV Compression": compressors keep a different token subset per layer - and, for
 * many of them, per head - and the method composes such caches as opaque units).  Layer l, kv head h keeps
 * kept[l * n_kv_heads + h] of the document's n_tokens keys and values (>= 1 each); which tokens is the
 * compressor's business: every key carries the rotation of the position it was cached at and the packet
 * keeps those positions, so it still takes one offset Delta, and its extent in a request stays n_tokens
 * positions (the next segment starts n_tokens further on).
 *   k, v   device; for (l, h) in that order, kept[l][h] rows of head_dim elements, the runs back to back
 *   kept   host [n_layers][n_kv_heads]
 * The packet occupies max(kept) pool rows.  Needs cfg.max_compressed > 0.  Assemblies that use a
 * compressed packet cannot be materialised (KVP_MATERIALIZE) or exported with kvp_export_cache: those
 * return KVP_ERR_UNSUPPORTED.
 * Errors: INVALID, CAPACITY (max_packets, pool), STATE (max_compressed == 0), CUDA.
 */
KVP_API int32_t kvp_register_packet_compressed(kvp_ctx *ctx, const void *k, const void *v, int32_t n_tokens,
                                               int32_t cache_pos0, const int32_t *kept, void *stream,
                                               int32_t *packet_id);

/*
 * Register one adapter: K/V of N_h header and N_t trailer soft tokens (Section 3.1, phi = {H, T}),
 * same layout as a packet with n_tokens = n_header / n_trailer; either count may be 0 (pointers then
 * ignored).  Header rows are stored first, trailer rows after them.  header_pos0 / trailer_pos0 are
 * the positions at which those keys were cached.
 */
KVP_API int32_t kvp_register_adapter(kvp_ctx *ctx, const void *hk, const void *hv, int32_t n_header,
                             int32_t header_pos0, const void *tk, const void *tv, int32_t n_trailer,
                             int32_t trailer_pos0, void *stream, int32_t *adapter_id);

/*
 * Compose a batch of requests (Section 3.2 step 4: re-align by Eq. 1, then concatenate).
 * Request b uses slots [slot_offsets[b], slot_offsets[b+1]); slot s is  header(adapter_ids[s]) |
 * packet_ids[s] | trailer(adapter_ids[s])  in Eq. 2 order, adapter_ids[s] = -1 for "no adapter".
 * Positions are dense from 0; a segment cached at p0 and placed at slot offset t gets Delta = t - p0
 * (0 for every segment when KVP_REBASE is not set).  All three index arrays are host arrays.
 *
 * Host work: validation, segment table, tile list, cos/sin of Delta*theta_i in double precision.
 * Device work on `stream`: one plan upload and one gather kernel that copies + re-bases either the
 * adapter tokens only (default: documents are read in place by kvp_query_prefill) or, with
 * KVP_MATERIALIZE, the whole prefix into the workspace cache.
 * prefix_len (host, [batch]) is written before return.  Errors: INVALID, NOT_FOUND, CAPACITY, CUDA.
 */
KVP_API int32_t kvp_assemble(kvp_ctx *ctx, int32_t batch, const int32_t *slot_offsets,
                     const int32_t *packet_ids, const int32_t *adapter_ids, uint32_t flags,
                     void *stream, int32_t *prefix_len, int32_t *assembly_id);

/*
 * The same composition for one shard of a request whose packets are spread over several GPUs (the paper scales
 * context by adding packets - the long-context settings of Section 4.3 - and a request's packets are independent
 * units, Section 3.1, so a rank can hold any subset of them).  Request b's slots here are a contiguous part of
 * its full slot list; pos_base[b] (host, [batch], >= 0) is the position at which that part starts in the full
 * composed sequence, i.e. the total length of the slots before it, adapters included.  Every key is re-based to
 * its position in the full sequence: Delta = pos_base[b] + offset within this part - cache position (Eq. 1).
 * prefix_len[b] receives the number of tokens of this part.  Everything else as kvp_assemble.  On such an
 * assembly kvp_query_prefill refuses KVP_ROPE_QUERY (the query's position is not prefix_len[b]).
 */
KVP_API int32_t kvp_assemble_at(kvp_ctx *ctx, int32_t batch, const int32_t *slot_offsets,
                        const int32_t *packet_ids, const int32_t *adapter_ids, const int32_t *pos_base,
                        uint32_t flags, void *stream, int32_t *prefix_len, int32_t *assembly_id);

/*
 * Query prefill of one layer over an assembly (Section 3.2 step 4; Fig. 2(d)): query token i of
 * request b attends to all prefix_len[b] composed tokens and to query tokens <= i, softmax in fp32,
 * q head h using kv head h / (Hq/Hkv).  k_new / v_new are appended to the request's cache at rows
 * prefix_len[b] + i (readable through kvp_export_cache).
 *   q      device [batch][q_len][n_q_heads][head_dim]
 *   k_new  device [batch][q_len][n_kv_heads][head_dim]   (v_new likewise)
 *   out    device [batch][q_len][n_q_heads][head_dim]
 *   lse    device float [batch][n_q_heads][q_len] or NULL: natural-log sum of exp(scaled scores)
 * By default q and k_new are already rotated for positions prefix_len[b] + i; KVP_ROPE_QUERY makes
 * the library rotate them.
 * KVP_PRECISE_QK: the tcgen05 kernel applies Eq. 1 to the query side of q.k (a document's keys stay as they
 * were cached) and rounds the rotated query to bf16 once per document - the rounding any bf16 cache of
 * re-based keys carries, 2^-9 relative per term of the dot product.  With this flag the rotated query is
 * kept as value + rounding remainder (two bf16 numbers) and both are multiplied with the keys, which removes
 * that rounding from the scores at 1.5x the Q.K tensor work on document tiles.  Meant for caches with
 * outlier channels, where the plain rounding, multiplied by values of magnitude 10 and more, shows in the
 * output.  No effect on the CUDA-core kernel (fp32 throughout) or on a materialised cache (its keys are
 * stored re-based and rounded).
 * KVP_CONTINUE (the step after the prefill - decoding with q_len = 1 - or a prefill fed in chunks): the
 * rows appended by the earlier calls for this layer since kvp_assemble stay; with n of them, token i of
 * this call sits at position prefix_len[b] + n + i, attends to the prefix, to those n rows and to this
 * call's tokens <= i, and is appended behind them.  n + q_len may not exceed max_query_tokens.  Without
 * the flag a call starts again at prefix_len[b].  Errors: INVALID, NOT_FOUND, CAPACITY (q_len > max_query_tokens),
 * STATE (host-only context), UNSUPPORTED, CUDA.  The call returns KVP_OK once the kernels are enqueued: a
 * device-side wait that ran out (the launch then gave up and its output is not valid) shows only in
 * kvp_status_word, which a caller that needs to know must read after synchronising the stream.
 */
KVP_API int32_t kvp_query_prefill(kvp_ctx *ctx, int32_t assembly_id, int32_t layer, const void *q,
                          const void *k_new, const void *v_new, int32_t q_len, uint32_t flags,
                          void *out, float *lse, void *stream);

/* Size in bytes of the buffer a KVP_PARTIAL prefill of `batch` requests x `q_len` tokens writes.  0 if invalid. */
KVP_API uint64_t kvp_partial_bytes(kvp_ctx *ctx, int32_t batch, int32_t q_len);

/*
 * Combine the partial results of the ranks of a prefix-sharded request into the attention output: per query row
 * M = max m_r, L = sum_r l_r 2^((m_r - M) c), O = sum_r O_r 2^((m_r - M) c) / L - softmax attention over the union
 * of the ranks' keys (Section 3.2 step 4 over the whole composed sequence).
 *   parts   device: n_parts buffers of kvp_partial_bytes(ctx, batch, q_len) bytes back to back (what an
 *           all-gather of the ranks' buffers delivers), 16-byte aligned, all in this GPU's memory
 *   out     device [batch][q_len][n_q_heads][head_dim], lse device float [batch][n_q_heads][q_len] or NULL
 * Errors: INVALID, CAPACITY (batch / q_len beyond the context's maxima), STATE, UNSUPPORTED (not bf16 / 128), CUDA.
 */
KVP_API int32_t kvp_merge_partials(kvp_ctx *ctx, const void *parts, int32_t n_parts, int32_t batch, int32_t q_len,
                           void *out, float *lse, void *stream);

/*
 * The same for a batch whose requests bring query chunks of different lengths (a serving batch rarely has equal
 * ones; the paper's Section 3.2 is per request).  q, k_new, v_new, out, lse have the layout of kvp_query_prefill
 * with q_len_max as the token stride; request b uses its first q_lens[b] tokens (1 <= q_lens[b] <= q_len_max).
 * Rows of out / lse beyond a request's length are not written; the padding rows of q, k_new, v_new are never
 * used in a result but are read, so they must hold finite numbers (zeros will do).
 *   q_lens   host [batch]
 * Runs on the two-stream tcgen05 kernel with its own append only (bf16, head_dim 128, sm_100a; 16-byte aligned
 * k_new / v_new): KVP_ERR_UNSUPPORTED otherwise; no flags.  The appended rows differ per request, so this
 * layer of the assembly cannot be continued (KVP_CONTINUE), exported with query rows or given to
 * kvp_segment_mass afterwards.
 * Errors: as kvp_query_prefill, INVALID (a length outside [1, q_len_max]).
 */
KVP_API int32_t kvp_query_prefill_ragged(kvp_ctx *ctx, int32_t assembly_id, int32_t layer, const void *q, const void *k_new,
                                 const void *v_new, int32_t q_len_max, const int32_t *q_lens, void *out, float *lse,
                                 void *stream);

/* ---- inspection helpers (not on the hot path) -------------------------------------------------- */

/*
 * The composed sequence of request b, as host arrays (any may be NULL):
 *   src_row [prefix_len]  pool row each composed position is read from
 *   delta   [prefix_len]  rotation offset applied to that key
 *   seg_table [4 * n_segments]  per segment: src_row0, length, dst_pos0, delta
 *   n_segments  number of (non-empty) segments
 */
KVP_API int32_t kvp_export_plan(kvp_ctx *ctx, int32_t assembly_id, int32_t b, int32_t *src_row,
                        int32_t *delta, int32_t *seg_table, int32_t *n_segments);

/*
 * Logical composed cache of (layer, request b): rows [0, prefix_len) re-based prefix, then the rows
 * appended by the last kvp_query_prefill of that layer.  k_out, v_out: device,
 * [n_rows][n_kv_heads][head_dim]; n_rows = prefix_len + n_query_rows.  k_as_f32 != 0 writes k_out as
 * float32 (the rotation result before narrowing to the stored dtype); v_out always has the stored dtype.
 */
KVP_API int32_t kvp_export_cache(kvp_ctx *ctx, int32_t assembly_id, int32_t layer, int32_t b,
                         int32_t n_query_rows, void *k_out, void *v_out, int32_t k_as_f32,
                         void *stream);

/*
 * The work list the tensor-core attention kernel would use for `q_len` query tokens over this assembly
 * (host arrays, any may be NULL; works in a host-only context).  The kernel is persistent: CTA c runs
 * pieces [cta_begin[c], cta_begin[c+1]).  A piece is 8 ints {request, kv head, first packed query row
 * of its unit, mode, first key tile, number of key tiles, partial slot of stream 0, of stream 1};
 * a unit is <= 256 packed rows (query token, head-in-group) of one request and kv head, its key tiles
 * numbered with the causal tiles of the query's own keys first and the request's prefix tiles after
 * them; mode 0 = two 128-row query tiles over every key tile, mode 1 = one query tile whose key tiles
 * alternate between the CTA's two streams; slot -1 = the piece covers the unit's whole key range and
 * writes the output directly.  A merge item is 8 ints {request, kv head, first packed row, first
 * partial slot, number of slots, 0, 0, 0}.  counts (4 ints): CTAs, pieces, merge items, partial slots.
 * Errors: NOT_FOUND, INVALID, CAPACITY (an output array is too small; counts is still written).
 */
KVP_API int32_t kvp_export_schedule(kvp_ctx *ctx, int32_t assembly_id, int32_t q_len, int32_t *cta_begin,
                                    int32_t cta_cap, int32_t *works, int32_t work_cap, int32_t *merges,
                                    int32_t merge_cap, int32_t *counts);

/*
 * Attention mass per segment (the quantity behind the paper's attention maps, Section 4.4 / Fig. 5: how
 * much of a query token's attention the header and trailer soft tokens of each packet absorb).  For query
 * token i of request b and q head h:  mass[s] = sum over the keys j of segment s of exp(score_j - lse),
 * with score_j = scale * q . R_Delta k_j (Eq. 1 applied to the cached key) and lse the value
 * kvp_query_prefill returned for that row, so that the columns of a row add up to 1.
 * Call it after kvp_query_prefill of the same layer with the same q, q_len and flags; the keys of the
 * query block are the rows that call (and, with KVP_CONTINUE, the calls before it) appended.
 *   q     device [batch][q_len][n_q_heads][head_dim]   (with KVP_ROPE_QUERY: ignored, the rotated copy
 *                                                        the prefill made is used)
 *   lse   device float [batch][n_q_heads][q_len]
 *   mass  device float [batch][q_len][n_q_heads][n_cols]: column s < n_segments(b) is segment s of the
 *         request in Eq. 2 order (header, document, trailer per slot; kvp_export_plan lists them), column
 *         n_segments(b) the query block, further columns 0.  n_cols > largest n_segments.
 * A diagnostic on CUDA cores, not part of the hot path.  Errors: INVALID, NOT_FOUND, STATE, CAPACITY
 * (n_cols too small), CUDA.
 */
KVP_API int32_t kvp_segment_mass(kvp_ctx *ctx, int32_t assembly_id, int32_t layer, const void *q, const float *lse,
                                 int32_t q_len, uint32_t flags, float *mass, int32_t n_cols, void *stream);

/* Synchronises the device and returns the device-side status word (0 = no bounded wait ran out;
   otherwise a code identifying the wait) in *device_status, then clears it. */
KVP_API int32_t kvp_status_word(kvp_ctx *ctx, int32_t *device_status);

/* How the last kvp_query_prefill was launched (host ints, any may be NULL): kernel kind
   (0 = fp32 CUDA-core kernel, 1 = bf16 tcgen05 kernel), CTAs, key splits, kernels launched. */
KVP_API int32_t kvp_last_launch(kvp_ctx *ctx, int32_t *kind, int32_t *ctas, int32_t *splits, int32_t *launches);

/* Launch tuning (not needed for correctness).  key KVP_TUNE_SPLIT_TARGET_CTAS: the tcgen05 path
   splits each request's keys until about `value` CTAs exist (0 = default, 4 per SM);
   key KVP_TUNE_FORCE_SPLITS: 1 = no unit's key range is split (0 = automatic);
   key KVP_TUNE_FUSED_APPEND: 1 (default) = on the plain prefill path (no KVP_ROPE_QUERY, no KVP_CONTINUE) the
   tcgen05 kernel reads the query block's keys and values straight from k_new / v_new and appends them itself,
   0 = always run the separate append kernel first;
   key KVP_TUNE_TIME_KERNELS: value p >= 1 brackets every p-th attention kernel and every p-th gather kernel
   with CUDA events on the caller's stream (up to 4096 timed launches between two kvp_kernel_times calls; the
   events between back-to-back launches cost a little, hence the period), 0 = off. */
enum { KVP_TUNE_SPLIT_TARGET_CTAS = 1, KVP_TUNE_FORCE_SPLITS = 2, KVP_TUNE_TIME_KERNELS = 3, KVP_TUNE_FUSED_APPEND = 5 };
KVP_API int32_t kvp_tune(kvp_ctx *ctx, int32_t key, int32_t value);

/* Device durations, in milliseconds, of the kernels launched since the last call with this `which`
   (0 = main attention kernel of kvp_query_prefill, 1 = gather kernel of kvp_assemble), oldest first;
   needs KVP_TUNE_TIME_KERNELS.  Synchronises on the recorded events.  ms: host array of `cap`
   floats; *n receives the number written. */
KVP_API int32_t kvp_kernel_times(kvp_ctx *ctx, int32_t which, float *ms, int32_t cap, int32_t *n);

/*
 * Gather + re-base of one request's segments with NO allocation anywhere (the paper has no
 * counterpart of this call; it exists for integration).  It is the gather kernel of kvp_assemble
 * for callers that cannot provide a workspace and must not trigger any allocation: code that runs
 * after the process's device heap has been frozen, plugins that receive raw device pointers but no
 * allocator, callbacks that may not enter the CUDA allocator.  It needs no kvp_ctx.
 *
 * Segment s (pool rows [src_row0[s], src_row0[s] + seg_len[s]) of every plane) is copied behind
 * segment s-1 into the cache, starting at cache row 0; its keys are rotated by delta[s] positions
 * (Eq. 1; theta_i = rope_theta^(-2i/d); angles in double precision on the device), its values are
 * byte copies.  A plane is one (layer, kv head): pool_k/pool_v are [n_planes][pool_rows][head_dim],
 * cache_k/cache_v are [n_planes][cache_rows][head_dim], all device pointers the caller owns, 16-byte
 * aligned.  src_row0, seg_len, delta are host arrays, read before the call returns.
 *
 * Scratch: the per-segment records and cos/sin tables live in a fixed array inside the library image,
 * 50,688 bytes on every GPU that loads the library, sized for KVP_NOALLOC_MAX_SEGMENTS segments per
 * call; more segments are refused with KVP_ERR_CAPACITY (split the request into several calls with
 * cache pointers advanced by the rows already written).  The array is shared by all calls on a device
 * and keeps the previous call's contents; every record a call reads is rewritten by that call first,
 * so nothing depends on its old contents, but calls whose kernels can overlap on the GPU (different
 * streams or threads) race on it and must be serialised by the caller.
 *
 * The first call on each device looks up the array's device address (the device must be current) and
 * makes the CUDA runtime load this library's kernels, which the driver may serve with allocations of
 * its own: make one warm-up call per device while allocation is still allowed (before the heap is
 * frozen) and outside any stream capture.  Two kernels are enqueued on `stream`; the call does not
 * synchronise.  The library itself calls no cudaMalloc/cudaFree or other allocating routine here.
 * err (optional, err_cap bytes) receives a message on failure.
 * Errors: INVALID (null or misaligned pointer, bad shape/dtype, segment outside the pool), CAPACITY
 * (too many segments, or more rows than cache_rows or than 2^31 - 1), CUDA.
 */
#define KVP_NOALLOC_MAX_SEGMENTS 96
KVP_API int32_t kvp_compose_noalloc(const void *pool_k, const void *pool_v, int64_t pool_rows, int32_t n_planes,
                                    int32_t head_dim, int32_t dtype, int32_t rope_pairing, double rope_theta,
                                    int32_t n_segments, const int32_t *src_row0, const int32_t *seg_len,
                                    const int32_t *delta, void *cache_k, void *cache_v, int64_t cache_rows,
                                    void *stream, char *err, int32_t err_cap);

/* Text of the last error on this context (owned by ctx; "" if none).  With ctx == NULL: the reason
   the last kvp_create on this thread failed. */
KVP_API const char *kvp_last_error(kvp_ctx *ctx);

/* Library version, major*10000 + minor*100 + patch. */
KVP_API int32_t kvp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KVP_H_ */
