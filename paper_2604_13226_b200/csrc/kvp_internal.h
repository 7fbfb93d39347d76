// Internal declarations shared by the host planner and the CUDA kernels.
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/kvp.h"

#define KVP_TILE_KEYS 128      // keys per attention tile (one TMA box of K or V rows)
#define KVP_TILE_ROWS 128      // packed query rows per CTA tile (MMA M)
#define KVP_CHUNK_ROWS 32      // rows per gather work item
#define KVP_MAX_SPLIT_UNITS 2048   // partial slots (128 query rows each) in the workspace

// ---- device-visible plan records (written by the host planner, uploaded once per assembly) -----

struct kvp_tile {              // one run of <= 128 consecutive key rows sharing one rotation offset
    int32_t row0;              // first row, in the pool (src 0) or in the workspace rows (src 1)
    int16_t n_keys;            // 1..128
    int16_t src;               // 0 pool, 1 workspace
    int32_t rope;              // rope-table index of the offset still to be applied to these keys (0 = none)
    int32_t pad;
};

struct kvp_chunk {             // gather work item: <= 32 rows copied pool -> workspace, keys rotated
    int32_t src_row0;
    int32_t dst_row0;
    int32_t n_rows;
    int32_t rope;              // rope-table index (0 = identity: byte copy)
};

struct kvp_seg {               // one segment of a composed request (header, document or trailer)
    int32_t src_row0;
    int32_t len;
    int32_t dst_pos0;
    int32_t delta;
    int32_t rope;
    int32_t pad[3];
};

struct kvp_item {              // one request of the batch
    int32_t prefix_len;
    int32_t tile_begin, tile_end;      // its prefix tiles in the tile array
    int32_t seg_begin, seg_end;        // its segments
    int32_t tail_row0;                 // workspace row where its query K/V rows are appended
    int32_t cache_row0;                // workspace row of composed position 0 (materialised), else -1
    int32_t pad;
};

// One piece of work of the two-stream attention kernel: a contiguous range of one unit's key tiles.
// A unit is up to 256 packed query rows of one (request, kv head).  Its key tiles are numbered: the
// causal tiles of the query's own keys first, then the request's prefix tiles in plan order.
//   mode 0: two 128-row query tiles ("streams"), each visiting every key tile of the range;
//   mode 1: one 128-row query tile; the key tiles alternate between the two streams and the two
//           partial results are combined inside the CTA.
// slot >= 0: un-normalised fp32 partial written to that partial slot (the unit's key range is shared
// by several pieces); slot < 0: this piece covers the whole range and writes the output rows.
struct kvp_work {
    int32_t b, hk;
    int32_t row_base;          // first packed query row of the unit
    int32_t mode;
    int32_t tile_lo, n_tiles;  // range in the unit's tile numbering
    int32_t slot0, slot1;      // stream 0 / stream 1 (mode 1 uses slot0 only)
    // copied from the request's plan item, so that a CTA's first look-up is one memory round trip, not two
    int32_t tile_begin;        // first prefix tile of the (request, plane) in the plan's tile array
    int32_t tail_row0;         // workspace row where the request's query K/V rows are appended
    int32_t pad[2];
};
static_assert(sizeof(kvp_work) == 48, "three 16-byte words");

struct kvp_merge_item {        // 128 packed rows whose result is spread over n_slots partial slots
    int32_t b, hk;
    int32_t row_base;
    int32_t slot0, n_slots;
    int32_t pad[3];            // pad[0]: the request's own query length (0: the call's q_len)
};

// Offsets (bytes) of the arrays inside one plan blob; identical on host and device.
struct kvp_plan_layout {
    uint64_t items, tiles, chunks, segs, rope, kept, total;
    int32_t max_items, max_tiles, max_chunks, max_segs, max_rope;
};

// Pointers into a device-resident plan, passed to kernels by value.
struct kvp_plan_dev {
    const kvp_item *items;
    const kvp_tile *tiles;
    const kvp_chunk *chunks;
    const kvp_seg *segs;
    const float2 *rope;        // [n_rope][head_dim/2] (cos, sin) of delta * theta_i
    const int32_t *kept;       // [compressed packets of the assembly][n_layers * n_kv_heads] kept rows per plane
    int32_t item_stride;       // 0: one item / tile list for all planes; batch: items[(layer * n_kv_heads + kv head) * batch + b]
    int32_t n_planes;
};

struct kvp_shape {
    int32_t n_layers, n_q_heads, n_kv_heads, head_dim, group, dtype, pairing, elem_bytes;
    float scale;               // softmax scale
    int64_t pool_rows;         // rows per (layer, kv head) plane in the pool
    int64_t ws_rows;           // rows per plane in one assembly's workspace rows
};

// ---- host-side context -----------------------------------------------------------------------

struct kvp_segment_host {
    int32_t row0, n, pos0;             // first pool row, positions covered, position it was cached at
    std::vector<int32_t> kept;         // compressed packets: rows kept per plane (layer, kv head); else empty
};

struct kvp_assembly_host {
    int32_t id = -1;
    uint32_t flags = 0;
    int32_t batch = 0;
    std::vector<kvp_item> items;
    std::vector<kvp_seg> segs;
    std::vector<kvp_tile> tiles;
    int32_t n_chunks = 0, n_rope = 0;
    int32_t item_stride = 0;               // batch when the assembly has a tile list per (layer, kv head) (compressed packets)
    int32_t last_q_len = 0;
    std::vector<int32_t> appended;         // per layer: query rows appended so far (KVP_CONTINUE)
    bool shard = false;                    // made by kvp_assemble_at: positions start at a caller-given base
    bool ragged = false;                   // a kvp_query_prefill_ragged call has appended a different number of rows per request
    bool waits_loads = false;              // uses packets that came from host memory: wait for the layer's load event
    // work lists of the two-stream kernel (one, or one per layer when the tile lists differ per layer), each
    // built for q_len query tokens at offset q_pos0 (q_len 0 = none yet)
    struct sched_state { int32_t q_len = 0, q_pos0 = 0, ctas = 0, works = 0, merges = 0, slots = 0; uint32_t opts = 0; std::vector<int32_t> q_lens; };
    std::vector<sched_state> sched;
};

struct kvp_ctx {
    kvp_config cfg;
    kvp_shape shape;
    bool host_only = false;
    std::vector<double> inv_freq;
    std::vector<kvp_segment_host> packets;
    // packets whose K/V wait in host memory until a request uses them (parallel to `packets`, grown on demand)
    struct host_src { const char *k = nullptr, *v = nullptr; bool from_host = false, resident = true; };
    std::vector<host_src> packet_src;
    cudaStream_t load_stream = nullptr;             // host -> pool copies, layer by layer
    cudaEvent_t load_fence = nullptr;               // the caller's stream at the assemble that starts a load
    std::vector<cudaEvent_t> load_done;             // [layer]: the loads enqueued so far have landed for this layer
    bool loads_recorded = false;
    std::vector<kvp_segment_host> adapter_h, adapter_t;
    int64_t pool_rows_used = 0;

    // device memory carved out of the caller's buffers
    char *pool_k = nullptr, *pool_v = nullptr;
    int32_t *status_dev = nullptr;
    kvp_plan_layout pl;
    std::vector<char *> slot_plan_dev;     // per assembly slot
    std::vector<char *> slot_k, slot_v;    // per assembly slot: workspace rows
    std::vector<char *> slot_sched_dev;    // per assembly slot: cta ranges, work list, merge list
    std::vector<char *> slot_sched_host;   // pinned staging of the same
    std::vector<cudaEvent_t> sched_event;
    uint64_t sched_off_works = 0, sched_off_merges = 0, sched_bytes = 0;
    int32_t sched_max_works = 0, sched_max_merges = 0;
    int32_t fused_append = 1;              // plain prefill: the attention kernel reads k_new / v_new itself and appends them
    void *encode_tiled = nullptr;          // cuTensorMapEncodeTiled
    float *partial_o = nullptr;            // [units][128][head_dim]
    float2 *partial_ml = nullptr;          // [units][128] (running max, running sum)
    char *q_scratch = nullptr;
    float2 *q_rope = nullptr;              // [max_batch*max_query][head_dim/2] for KVP_ROPE_QUERY

    // pinned host staging (one per slot) and the event guarding its reuse
    std::vector<char *> slot_plan_host;
    std::vector<cudaEvent_t> slot_event;
    std::vector<kvp_assembly_host> slots;
    int32_t next_assembly = 0;

    // TMA descriptors (bf16, head_dim 128 only)
    bool have_tma = false;
    CUtensorMap tm_pool_k, tm_pool_v;
    std::vector<CUtensorMap> tm_ws_k, tm_ws_v;

    int32_t sm_count = 148;
    int32_t split_target_ctas = 0, force_splits = 0;
    // optional CUDA-event timing of the attention (0) and gather (1) kernels, for roofline reports
    int32_t time_kernels = 0;             // 0: off; p >= 1: every p-th attention / gather kernel is bracketed by events
    int32_t tev_seen[2] = {0, 0};
    bool tev_open[2] = {false, false};
    std::vector<cudaEvent_t> tev[2][2];
    int32_t tev_n[2] = {0, 0};
    int32_t last_kind = -1, last_ctas = 0, last_splits = 0, last_launches = 0;
    std::string err;
};

// ---- kernel launchers (kvp_kernels.cu, kvp_attn_sm100.cu) ---------------------------------------

cudaError_t kvp_launch_store_rows(const kvp_shape &sh, const void *src, char *dst_plane0, int64_t plane_rows,
                                  int64_t dst_row0, int32_t n_tokens, cudaStream_t st);
cudaError_t kvp_launch_gather(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t n_chunks,
                              const char *pool_k, const char *pool_v, char *ws_k, char *ws_v, cudaStream_t st);
cudaError_t kvp_launch_append(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t batch, int32_t q_len,
                              int32_t q_pos0, const void *q, const void *k_new, const void *v_new, char *ws_k, char *ws_v,
                              int32_t layer, int32_t rope_query, const double *inv_freq_dev, void *q_rot,
                              cudaStream_t st);
cudaError_t kvp_launch_export(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t b, int32_t layer,
                              int32_t prefix_len, int32_t n_query_rows, const char *pool_k, const char *pool_v,
                              const char *ws_k, const char *ws_v, void *k_out, void *v_out, int32_t k_as_f32,
                              cudaStream_t st);
cudaError_t kvp_launch_segment_mass(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t batch, int32_t q_len,
                                    int32_t q_pos0, int32_t layer, const void *q, const float *lse, const char *pool_k,
                                    const char *ws_k, float *mass, int32_t n_cols, cudaStream_t st);
cudaError_t kvp_launch_attn_simple(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t batch, int32_t q_len,
                                   int32_t q_pos0, int32_t layer, const void *q, const char *pool_k, const char *pool_v,
                                   const char *ws_k, const char *ws_v, void *out, float *lse, int32_t *ctas,
                                   cudaStream_t st);

struct kvp_attn2_args {
    kvp_plan_dev plan;
    int32_t q_len, q_pos0, layer, n_ctas;
    const int32_t *cta_begin;      // [n_ctas + 1] ranges into works
    const kvp_work *works;
    const void *q;
    void *out;
    float *lse;
    float *partial_o;
    float2 *partial_ml;
    int32_t *status;
    // tail_direct: the query block's K/V tiles are loaded from k_new / v_new ([batch][q_len][Hkv][d]) through
    // tm_knew / tm_vnew and the kernel copies those rows into the workspace rows itself
    int32_t tail_direct;
    int32_t precise;               // KVP_PRECISE_QK
    int32_t l2_prefetch;           // the launch has at most two 256-row units per (request, kv head)
    const void *k_new, *v_new;
    char *ws_k, *ws_v;
    CUtensorMap tm_knew, tm_vnew;
};
cudaError_t kvp_attn_sm100_prepare(void);
cudaError_t kvp_launch_attn_sm100(const kvp_shape &sh, const kvp_attn2_args &a, const CUtensorMap &tm_pool_k,
                                  const CUtensorMap &tm_pool_v, const CUtensorMap &tm_ws_k,
                                  const CUtensorMap &tm_ws_v, cudaStream_t st);
// part_out != nullptr: the merged tiles stay partials and go to a rank buffer of part_tiles query tiles
cudaError_t kvp_launch_merge_list(const kvp_shape &sh, int32_t q_len, int32_t n_merges, const kvp_merge_item *merges,
                                  const float *partial_o, const float2 *partial_ml, void *out, float *lse,
                                  void *part_out, int64_t part_tiles, cudaStream_t st);
// n_parts rank buffers back to back -> final output rows
cudaError_t kvp_launch_merge_ranks(const kvp_shape &sh, int32_t batch, int32_t q_len, const void *parts, int32_t n_parts,
                                   void *out, float *lse, cudaStream_t st);
