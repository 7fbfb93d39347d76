// C ABI + host planner of the composed-cache query-prefill library.
//
// The planner turns a batch of requests into (i) a segment table - header | document | trailer per
// slot, Eq. 2 order, dense positions, Delta = slot offset - cache position (Eq. 1) - and (ii) the tile
// list the attention kernels walk: runs of <= 128 key rows that share one rotation offset, read in
// place from the pool (documents) or from the workspace (staged adapter rows, materialised cache).
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <map>

#include "kvp_internal.h"

namespace {

constexpr uint64_t kAlign = 1024;
inline uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

struct ws_layout {
    uint64_t status, inv_freq, slots, slot_stride, slot_plan, slot_sched, slot_k, slot_v, partial_o, partial_ml, q_scratch, total;
    uint64_t rows_bytes;
};

constexpr int kMaxCtas = 256;          // upper bound on persistent CTAs (one per SM)

// Work list of the two-stream attention kernel: [cta_begin: kMaxCtas + 1 ints][works][merge items].
struct sched_layout {
    uint64_t works, merges, total;
    int32_t max_works, max_merges;
};

sched_layout schedule_layout(const kvp_config *c)
{
    sched_layout s;
    const int group = c->n_q_heads / c->n_kv_heads;
    const int64_t tiles_q = ((int64_t)group * c->max_query_tokens + KVP_TILE_ROWS - 1) / KVP_TILE_ROWS;
    const int64_t units = (int64_t)c->max_batch * c->n_kv_heads * tiles_q;
    s.max_works = (int32_t)std::min<int64_t>(units + kMaxCtas, 1 << 24);
    s.max_merges = 2 * kMaxCtas + 8 + (int32_t)std::min<int64_t>(units, KVP_MAX_SPLIT_UNITS);   // every unit has one with KVP_PARTIAL
    s.works = round_up(4 * (kMaxCtas + 1), 256);
    s.merges = round_up(s.works + sizeof(kvp_work) * (uint64_t)s.max_works, 256);
    s.total = round_up(s.merges + sizeof(kvp_merge_item) * (uint64_t)s.max_merges, 256);
    return s;
}

bool valid_cfg(const kvp_config *c)
{
    if (!c || c->struct_bytes != (int32_t)sizeof(kvp_config)) return false;
    if (c->n_layers <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0) return false;
    if (c->n_q_heads % c->n_kv_heads) return false;
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->dtype != KVP_DTYPE_F32 && c->dtype != KVP_DTYPE_BF16) return false;
    if (c->rope_pairing != 0 && c->rope_pairing != 1) return false;
    if (c->max_packets <= 0 || c->max_adapters < 0 || c->max_batch <= 0 || c->max_slots <= 0) return false;
    if (c->max_prefix_tokens <= 0 || c->max_query_tokens <= 0 || c->max_ws_rows <= 0 || c->max_assemblies <= 0)
        return false;
    if (!c->inv_freq && !(c->rope_theta > 0.0)) return false;
    if (c->max_compressed < 0) return false;
    return true;
}

kvp_plan_layout plan_layout(const kvp_config *c)
{
    kvp_plan_layout p;
    // with compressed packets every (layer, kv head) has its own item records and tile list
    const int64_t lists = c->max_compressed > 0 ? (int64_t)c->n_layers * c->n_kv_heads : 1;
    p.max_segs = 3 * c->max_slots;
    p.max_rope = p.max_segs + 1;
    p.max_items = (int32_t)(c->max_batch * lists);
    p.max_tiles = (int32_t)((c->max_batch * ((int64_t)c->max_prefix_tokens / KVP_TILE_KEYS + 2) + c->max_slots +
                             c->max_ws_rows / KVP_TILE_KEYS + 8) * lists);
    p.max_chunks = c->max_ws_rows / KVP_CHUNK_ROWS + p.max_segs + 8;
    uint64_t o = 0;
    p.items = o;  o = round_up(o + sizeof(kvp_item) * p.max_items, 256);
    p.tiles = o;  o = round_up(o + sizeof(kvp_tile) * (uint64_t)p.max_tiles, 256);
    p.chunks = o; o = round_up(o + sizeof(kvp_chunk) * p.max_chunks, 256);
    p.segs = o;   o = round_up(o + sizeof(kvp_seg) * p.max_segs, 256);
    p.rope = o;   o = round_up(o + sizeof(float2) * (uint64_t)p.max_rope * (c->head_dim / 2), 256);
    p.kept = o;   o = round_up(o + 4ull * c->max_compressed * c->n_layers * c->n_kv_heads, 256);
    p.total = o;
    return p;
}

ws_layout workspace_layout(const kvp_config *c)
{
    ws_layout w;
    const uint64_t e = c->dtype == KVP_DTYPE_BF16 ? 2 : 4;
    const kvp_plan_layout p = plan_layout(c);
    uint64_t o = 0;
    w.status = o;   o += 256;
    w.inv_freq = o; o = round_up(o + 8 * 64, kAlign);
    w.rows_bytes = round_up((uint64_t)c->n_layers * c->n_kv_heads * c->max_ws_rows * c->head_dim * e, kAlign);
    w.slot_plan = 0;
    w.slot_sched = round_up(p.total, kAlign);
    w.slot_k = round_up(w.slot_sched + schedule_layout(c).total * (c->max_compressed > 0 ? c->n_layers : 1), kAlign);
    w.slot_v = w.slot_k + w.rows_bytes;
    w.slot_stride = w.slot_v + w.rows_bytes;
    w.slots = o;    o += w.slot_stride * c->max_assemblies;
    w.partial_o = o;  o = round_up(o + (uint64_t)KVP_MAX_SPLIT_UNITS * KVP_TILE_ROWS * c->head_dim * 4, kAlign);
    w.partial_ml = o; o = round_up(o + (uint64_t)KVP_MAX_SPLIT_UNITS * KVP_TILE_ROWS * 8, kAlign);
    w.q_scratch = o;  o = round_up(o + (uint64_t)c->max_batch * c->max_query_tokens * c->n_q_heads * c->head_dim * e, kAlign);
    w.total = o;
    return w;
}

int32_t fail(kvp_ctx *ctx, int32_t code, const char *fmt, ...) __attribute__((format(printf, 3, 4)));
int32_t fail(kvp_ctx *ctx, int32_t code, const char *fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (ctx) ctx->err = buf;
    return code;
}

#define KVP_CUDA(ctx, call)                                                                              \
    do {                                                                                                 \
        cudaError_t e_ = (call);                                                                         \
        if (e_ != cudaSuccess) return fail(ctx, KVP_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_));  \
    } while (0)

typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// One K or V plane set as a 3-D bf16 tensor (head_dim, rows, layer*kv_head); box = 64 columns x 128
// rows with the 128-byte swizzle the MMA descriptors expect; out-of-range rows read as zero.
bool make_tensor_map(encode_tiled_fn enc, CUtensorMap *tm, void *base, int head_dim, int64_t rows, int planes)
{
    const cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)rows, (cuuint64_t)planes};
    const cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)rows * head_dim * 2};
    const cuuint32_t box[3] = {64, KVP_TILE_KEYS, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The caller's k_new or v_new, [batch][q_len][Hkv][d] bf16, as a 4-D tensor (d, Hkv, q_len, batch); box = 64
// columns x 1 head x 128 tokens, the same shared-memory tile as a pool box.  Tokens past q_len read as zero.
bool make_query_tensor_map(encode_tiled_fn enc, CUtensorMap *tm, const void *base, int head_dim, int n_kv, int q_len, int batch)
{
    const cuuint64_t dims[4] = {(cuuint64_t)head_dim, (cuuint64_t)n_kv, (cuuint64_t)q_len, (cuuint64_t)batch};
    const cuuint64_t strides[3] = {(cuuint64_t)head_dim * 2, (cuuint64_t)n_kv * head_dim * 2, (cuuint64_t)q_len * n_kv * head_dim * 2};
    const cuuint32_t box[4] = {64, 1, KVP_TILE_KEYS, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kMaxTimed = 4096;

// Record an event before (edge 0) / after (edge 1) a timed kernel; events are created on first use.  With a
// period p only every p-th kernel of its kind is bracketed.
cudaError_t time_edge(kvp_ctx *ctx, int which, int edge, cudaStream_t st)
{
    if (!ctx->time_kernels || ctx->tev_n[which] >= kMaxTimed) return cudaSuccess;
    if (edge == 0) ctx->tev_open[which] = (ctx->tev_seen[which]++ % ctx->time_kernels) == 0;
    if (!ctx->tev_open[which]) return cudaSuccess;
    std::vector<cudaEvent_t> &v = ctx->tev[which][edge];
    const int i = ctx->tev_n[which];
    if ((int)v.size() <= i) {
        cudaEvent_t e;
        cudaError_t rc = cudaEventCreate(&e);
        if (rc != cudaSuccess) return rc;
        v.push_back(e);
    }
    cudaError_t rc = cudaEventRecord(v[i], st);
    if (rc == cudaSuccess && edge == 1) ++ctx->tev_n[which];
    return rc;
}

kvp_plan_dev plan_dev(const kvp_ctx *ctx, int slot)
{
    char *base = ctx->slot_plan_dev[slot];
    kvp_plan_dev p;
    p.items = reinterpret_cast<const kvp_item *>(base + ctx->pl.items);
    p.tiles = reinterpret_cast<const kvp_tile *>(base + ctx->pl.tiles);
    p.chunks = reinterpret_cast<const kvp_chunk *>(base + ctx->pl.chunks);
    p.segs = reinterpret_cast<const kvp_seg *>(base + ctx->pl.segs);
    p.rope = reinterpret_cast<const float2 *>(base + ctx->pl.rope);
    p.kept = reinterpret_cast<const int32_t *>(base + ctx->pl.kept);
    p.item_stride = ctx->slots[slot].item_stride;
    p.n_planes = ctx->shape.n_layers * ctx->shape.n_kv_heads;
    return p;
}

int find_slot(kvp_ctx *ctx, int32_t assembly_id)
{
    if (assembly_id < 0) return -1;
    const int slot = assembly_id % ctx->cfg.max_assemblies;
    return ctx->slots[slot].id == assembly_id ? slot : -1;
}

// Work list of the two-stream kernel for one assembly and query length.  Units (<= 256 packed query
// rows of one request and kv head) are laid end to end, each weighted by the tensor-core work of its
// key tiles, and the line is cut into equal shares, one per CTA; a cut closer than two tiles to a unit
// boundary moves onto it.  A unit that ends up in several pieces gets partial slots and merge items.
// Start-up and write-out of a piece (first Q tile, pipeline fill, epilogue) cost about as much as two
// two-stream key tiles (measured: 7,000 cycles per piece against 3,500-4,000 per tile pair, from the
// per-CTA durations of a config-3 launch); the unit weights carry it so that CTAs with more pieces get
// fewer tiles.  Counted in single-stream tiles.
constexpr int kPieceCost = 4;

struct schedule_t {
    std::vector<int32_t> cta_begin;
    std::vector<kvp_work> works;
    std::vector<kvp_merge_item> merges;
    int32_t n_ctas = 0, n_slots = 0, max_pieces = 1;
};

// q_lens: nullptr, or one query length per request (<= q_len, the stride of the padded tensors); a request's
// work records and merge items then carry its own length.
// opts: KVP_PARTIAL - every unit writes partial slots and gets merge items (even with one piece or none);
// KVP_SKIP_QUERY_BLOCK - a unit's range starts behind the causal tiles of the query's own keys.
int32_t plan_schedule(kvp_ctx *ctx, const kvp_assembly_host &as, int layer, int q_len, int q_pos0, const int32_t *q_lens,
                      uint32_t opts, schedule_t &out)
{
    const kvp_shape &sh = ctx->shape;
    const bool force_partial = (opts & KVP_PARTIAL) != 0, skip_tail = (opts & KVP_SKIP_QUERY_BLOCK) != 0;
    struct unit_t { int32_t b, hk, row_base, mode, n_all, first_piece, n_pieces, q_len, t_first, tile_begin, tail_row0, n_tail; };
    std::vector<unit_t> units;
    const int max_rows = sh.group * q_len;
    int64_t total = 0;
    // Row blocks outermost: the units of one (request, kv head) - which stream the same K/V - then lie a
    // whole number of CTA shares apart on the line (when their count divides the CTA count), so the CTAs
    // that hold them reach the same key tiles at the same time and all but the first find them in L2.
    for (int row_base = 0; row_base < max_rows; row_base += 2 * KVP_TILE_ROWS)
        for (int b = 0; b < as.batch; ++b) {
            const int n_rows = sh.group * (q_lens ? q_lens[b] : q_len);
            if (row_base >= n_rows) continue;
            for (int hk = 0; hk < sh.n_kv_heads; ++hk) {
                const kvp_item &item = as.items[(as.item_stride ? (layer * sh.n_kv_heads + hk) * as.item_stride : 0) + b];
                const int n_prefix = item.tile_end - item.tile_begin;
                unit_t u;
                u.q_len = q_lens ? q_lens[b] : 0;
                u.b = b; u.hk = hk; u.row_base = row_base;
                u.mode = (n_rows - row_base <= KVP_TILE_ROWS) ? 1 : 0;
                const int last = std::min(n_rows - 1, row_base + (u.mode ? 1 : 2) * KVP_TILE_ROWS - 1);
                const int n_tail = (q_pos0 + last / sh.group) / KVP_TILE_KEYS + 1;
                u.n_all = n_tail + n_prefix;
                u.t_first = skip_tail ? n_tail : 0;
                u.n_tail = n_tail;
                u.tile_begin = item.tile_begin;
                u.tail_row0 = item.tail_row0;
                u.first_piece = u.n_pieces = 0;
                units.push_back(u);
                total += (int64_t)(u.n_all - u.t_first) * (u.mode ? 1 : 2) + kPieceCost;
            }
        }
    int G = std::min(ctx->sm_count, kMaxCtas);
    if (ctx->split_target_ctas > 0) G = std::min(ctx->split_target_ctas, kMaxCtas);
    const bool no_split = ctx->force_splits == 1;               // cuts only between units

    // Cut positions (unit, tile), non-decreasing.  A run of units is dealt out to g CTAs one after the other, each
    // taking its even share of what is left (the work still to hand out divided by the CTAs still to fill, but
    // not less than a minimum that keeps tiny launches on few CTAs); every piece pays kPieceCost on top of its
    // tiles, a piece is at least two tiles long (or the whole unit), and without splitting a unit goes to the CTA
    // that holds its larger part.  The last CTA of the run takes all that is left, so g CTAs always suffice.
    struct cut_t { int32_t u, t; };
    std::vector<cut_t> cuts;
    const int64_t min_budget = 8 + kPieceCost;
    auto fill = [&](size_t u_begin, size_t u_end, int g, std::vector<cut_t> *rec) -> int {
        std::vector<int64_t> after(u_end - u_begin + 1, 0);           // weight of the units behind unit u
        for (size_t u = u_end; u > u_begin; --u) {
            const unit_t &x = units[u - 1];
            const int64_t wgt = x.n_all == x.t_first ? 0 : (int64_t)(x.n_all - x.t_first) * (x.mode ? 1 : 2) + kPieceCost;
            after[u - 1 - u_begin] = after[u - u_begin] + wgt;
        }
        int used = 0;
        size_t u = u_begin;
        while (u < u_end && units[u].n_all == units[u].t_first) ++u;      // units without a key tile get no piece
        int32_t t = u < u_end ? units[u].t_first : 0;
        while (u < u_end) {
            const int64_t left_all = after[u + 1 - u_begin] + (int64_t)(units[u].n_all - t) * (units[u].mode ? 1 : 2) + kPieceCost;
            const int ctas_left = std::max(1, g - used);
            // every further CTA is likely to start inside a unit, i.e. to add a piece
            const int64_t to_share = left_all + (int64_t)kPieceCost * (ctas_left - 1);
            const int64_t budget = ctas_left == 1 ? left_all : std::max(min_budget, (to_share + ctas_left - 1) / ctas_left);
            ++used;
            if (rec) rec->push_back({(int32_t)u, t});
            int64_t cost = 0;
            while (u < u_end) {
                const int w = units[u].mode ? 1 : 2;
                const int32_t left = units[u].n_all - t;
                const int64_t room = budget - cost - kPieceCost;
                int32_t take = (int32_t)std::min<int64_t>(left, room > 0 ? room / w : 0);      // rounded down: the shares are re-dealt at every CTA
                if (no_split) take = (t == units[u].t_first && (2 * take >= left || cost == 0)) ? left : 0;
                if (left - take < 2) take = left;                 // do not leave a sliver behind
                if (take < 2 && take < left) take = 0;
                if (take == 0) {
                    if (cost > 0) break;                          // start the piece in the next CTA
                    take = no_split ? left : std::min<int32_t>(left, 2);
                    if (left - take < 2) take = left;
                }
                cost += kPieceCost + (int64_t)take * w;
                t += take;
                if (t == units[u].n_all) {
                    ++u;
                    while (u < u_end && units[u].n_all == units[u].t_first) ++u;
                    t = u < u_end ? units[u].t_first : 0;
                }
                if (cost >= budget) break;
            }
        }
        return used;
    };
    auto cut_range = [&](size_t u_begin, size_t u_end, int64_t weight, int g) {
        (void)weight;
        fill(u_begin, u_end, g, &cuts);
    };
    // Each row block gets its own run of CTAs, in proportion to its work, and is cut on its own: row blocks of
    // equal work then get the same cuts, so the CTAs of units that share K/V walk the same tiles in step.  With
    // more row blocks than half the CTAs (or when told not to split) the whole line is cut at once.
    std::vector<size_t> rb_begin;                                 // first unit of every row block
    std::vector<int64_t> rb_weight;
    for (size_t u = 0; u < units.size(); ++u) {
        if (u == 0 || units[u].row_base != units[u - 1].row_base) {
            rb_begin.push_back(u);
            rb_weight.push_back(0);
        }
        rb_weight.back() += (int64_t)(units[u].n_all - units[u].t_first) * (units[u].mode ? 1 : 2) + kPieceCost;
    }
    rb_begin.push_back(units.size());
    const int n_rb = (int)rb_weight.size();
    std::vector<int> rb_ctas(n_rb, 0);
    bool per_block = n_rb >= 2 && 2 * n_rb <= G && !no_split;
    if (per_block) {
        int given = 0;
        std::vector<std::pair<int64_t, int>> rem;
        for (int r = 0; r < n_rb; ++r) {
            const int64_t num = rb_weight[r] * G;
            rb_ctas[r] = (int)(num / total);
            rem.push_back({-(num % total), r});
            given += rb_ctas[r];
        }
        std::sort(rem.begin(), rem.end());
        for (int i = 0; given < G; ++i, ++given) ++rb_ctas[rem[i % n_rb].second];
        for (int r = 0; r < n_rb; ++r) per_block = per_block && rb_ctas[r] >= 1;
    }
    std::vector<int> rb_used(n_rb, 0);
    // Row blocks that differ only in a few causal tiles are cut at the same PREFIX tiles: one row block is dealt
    // out and its cuts, counted from the first prefix tile of a unit, are used for all of them.  The CTAs that
    // hold the same (request, kv head) then stay on the same K/V tiles for the whole launch instead of drifting
    // apart by the tail tiles they have more or less (drift beyond what L2 holds per CTA turns re-reads into DRAM
    // reads: config 5, 16 packets, q 256, batch 4 read 1.37x its K/V).
    bool aligned = per_block && !q_lens && G / n_rb >= 1 && (G - n_rb * (G / n_rb)) * 50 <= G;
    if (aligned) {
        const size_t n_u = rb_begin[1] - rb_begin[0];
        int tail_lo = INT32_MAX, tail_hi = 0, prefix_lo = INT32_MAX;
        for (int r = 0; r < n_rb && aligned; ++r) {
            aligned = rb_begin[r + 1] - rb_begin[r] == n_u;
            for (size_t i = 0; i < n_u && aligned; ++i) {
                const unit_t &a = units[rb_begin[0] + i], &x = units[rb_begin[r] + i];
                aligned = x.b == a.b && x.hk == a.hk && x.mode == units[0].mode && x.n_all - x.n_tail == a.n_all - a.n_tail;
                tail_lo = std::min(tail_lo, x.n_tail); tail_hi = std::max(tail_hi, x.n_tail);
                prefix_lo = std::min(prefix_lo, x.n_all - x.n_tail);
            }
        }
        aligned = aligned && (tail_hi - tail_lo) * 50 <= prefix_lo && prefix_lo >= 8;
    }
    if (aligned) {
        const int rm = n_rb - 1;                                  // the row block with the most causal tiles
        std::vector<cut_t> model;
        fill(rb_begin[rm], rb_begin[rm + 1], G / n_rb, &model);
        for (int r = 0; r < n_rb; ++r) {
            const size_t before = cuts.size();
            for (const cut_t &m : model) {
                const unit_t &um = units[m.u], &ur = units[rb_begin[r] + (m.u - rb_begin[rm])];
                cut_t c;
                c.u = (int32_t)(rb_begin[r] + (m.u - rb_begin[rm]));
                c.t = m.t == um.t_first ? ur.t_first : ur.n_tail + std::max(m.t - um.n_tail, 2);
                if (cuts.size() > before && cuts.back().u == c.u && cuts.back().t >= c.t) continue;
                cuts.push_back(c);
            }
            rb_used[r] = (int)(cuts.size() - before);
        }
    } else if (per_block) {
        for (int r = 0; r < n_rb; ++r) {
            const size_t before = cuts.size();
            cut_range(rb_begin[r], rb_begin[r + 1], rb_weight[r], rb_ctas[r]);
            rb_used[r] = (int)(cuts.size() - before);
        }
    } else {
        cut_range(0, units.size(), total, G);
    }
    cuts.push_back({(int32_t)units.size(), 0});

    std::vector<kvp_work> &works = out.works;
    std::vector<int32_t> &cta_begin = out.cta_begin;
    struct cta_rec { std::vector<kvp_work> ws; std::vector<int32_t> unit; };
    std::vector<cta_rec> recs;
    for (size_t c = 0; c + 1 < cuts.size(); ++c) {
        const cut_t a = cuts[c], z = cuts[c + 1];
        cta_rec rec;
        for (int32_t u = a.u; u <= z.u && u < (int32_t)units.size(); ++u) {
            const int32_t lo = (u == a.u) ? a.t : units[u].t_first;
            const int32_t hi = (u == z.u) ? z.t : units[u].n_all;
            if (hi <= lo) continue;
            kvp_work w;
            w.b = units[u].b; w.hk = units[u].hk; w.row_base = units[u].row_base;
            w.mode = units[u].mode | (units[u].q_len << 8);       // a request's own query length rides in the upper bits
            w.tile_lo = lo; w.n_tiles = hi - lo; w.slot0 = w.slot1 = -1;
            w.tile_begin = units[u].tile_begin; w.tail_row0 = units[u].tail_row0; w.pad[0] = w.pad[1] = 0;
            rec.ws.push_back(w);
            rec.unit.push_back(u);
        }
        recs.push_back(rec);
    }
    // emission order: the j-th CTAs of all row blocks next to each other
    std::vector<int> order;
    if (per_block) {
        std::vector<int> off(n_rb + 1, 0);
        for (int r = 0; r < n_rb; ++r) off[r + 1] = off[r] + rb_used[r];
        for (int j = 0; (int)order.size() < off[n_rb]; ++j)
            for (int r = 0; r < n_rb; ++r)
                if (j < rb_used[r]) order.push_back(off[r] + j);
    } else {
        for (size_t c = 0; c < recs.size(); ++c) order.push_back((int)c);
    }
    std::vector<std::vector<int32_t>> unit_pieces(units.size());
    for (int idx : order) {
        const cta_rec &rec = recs[idx];
        if (rec.ws.empty()) continue;
        cta_begin.push_back((int32_t)works.size());
        for (size_t i = 0; i < rec.ws.size(); ++i) {
            unit_pieces[rec.unit[i]].push_back((int32_t)works.size());
            works.push_back(rec.ws[i]);
        }
    }
    for (size_t u = 0; u < units.size(); ++u) units[u].n_pieces = (int32_t)unit_pieces[u].size();
    const int n_ctas = (int)cta_begin.size();
    cta_begin.push_back((int32_t)works.size());

    std::vector<kvp_merge_item> &merges = out.merges;
    int32_t n_slots = 0, max_pieces = 1;
    for (size_t ui = 0; ui < units.size(); ++ui) {
        const unit_t &u = units[ui];
        if (u.n_pieces <= 1 && !force_partial) continue;
        max_pieces = std::max(max_pieces, u.n_pieces);
        const int32_t base = n_slots;
        for (int i = 0; i < u.n_pieces; ++i) {
            kvp_work &w = works[unit_pieces[ui][i]];
            w.slot0 = base + i;
            if (u.mode == 0) w.slot1 = base + u.n_pieces + i;
        }
        kvp_merge_item m;
        memset(&m, 0, sizeof m);
        m.b = u.b; m.hk = u.hk; m.row_base = u.row_base; m.slot0 = base; m.n_slots = u.n_pieces;
        m.pad[0] = u.q_len;
        merges.push_back(m);
        n_slots += u.n_pieces;
        if (u.mode == 0) {
            m.row_base = u.row_base + KVP_TILE_ROWS;
            m.slot0 = base + u.n_pieces;
            merges.push_back(m);
            n_slots += u.n_pieces;
        }
    }
    if (n_ctas > kMaxCtas || (int)works.size() > ctx->sched_max_works || (int)merges.size() > ctx->sched_max_merges ||
        n_slots > KVP_MAX_SPLIT_UNITS)
        return fail(ctx, KVP_ERR_CAPACITY, "query_prefill: work list overflow (%d ctas, %zu pieces, %zu merges, %d slots)",
                    n_ctas, works.size(), merges.size(), n_slots);

    out.n_ctas = n_ctas;
    out.n_slots = n_slots;
    out.max_pieces = max_pieces;
    return KVP_OK;
}

int32_t build_schedule(kvp_ctx *ctx, kvp_assembly_host &as, int slot, int layer, int q_len, int q_pos0, const int32_t *q_lens,
                       uint32_t opts, cudaStream_t st)
{
    schedule_t sc;
    const int32_t rc = plan_schedule(ctx, as, layer, q_len, q_pos0, q_lens, opts, sc);
    if (rc != KVP_OK) return rc;
    const std::vector<int32_t> &cta_begin = sc.cta_begin;
    const std::vector<kvp_work> &works = sc.works;
    const std::vector<kvp_merge_item> &merges = sc.merges;
    const int n_ctas = sc.n_ctas;
    const int32_t max_pieces = sc.max_pieces;
    KVP_CUDA(ctx, cudaEventSynchronize(ctx->sched_event[slot]));          // staging buffer free again?
    char *h = ctx->slot_sched_host[slot];
    memcpy(h, cta_begin.data(), 4 * cta_begin.size());
    memcpy(h + ctx->sched_off_works, works.data(), sizeof(kvp_work) * works.size());
    memcpy(h + ctx->sched_off_merges, merges.data(), sizeof(kvp_merge_item) * merges.size());
    const int li = as.item_stride ? layer : 0;                   // which of the assembly's work lists
    char *d = ctx->slot_sched_dev[slot] + ctx->sched_bytes * li;
    KVP_CUDA(ctx, cudaMemcpyAsync(d, h, 4 * cta_begin.size(), cudaMemcpyHostToDevice, st));
    KVP_CUDA(ctx, cudaMemcpyAsync(d + ctx->sched_off_works, h + ctx->sched_off_works, sizeof(kvp_work) * works.size(),
                                  cudaMemcpyHostToDevice, st));
    if (!merges.empty())
        KVP_CUDA(ctx, cudaMemcpyAsync(d + ctx->sched_off_merges, h + ctx->sched_off_merges,
                                      sizeof(kvp_merge_item) * merges.size(), cudaMemcpyHostToDevice, st));
    KVP_CUDA(ctx, cudaEventRecord(ctx->sched_event[slot], st));
    kvp_assembly_host::sched_state &ss = as.sched[li];
    ss.q_len = q_len;
    ss.q_lens.assign(q_lens ? q_lens : nullptr, q_lens ? q_lens + as.batch : nullptr);
    ss.q_pos0 = q_pos0;
    ss.opts = opts;
    ss.ctas = n_ctas;
    ss.works = (int32_t)works.size();
    ss.merges = (int32_t)merges.size();
    ss.slots = max_pieces;
    return KVP_OK;
}

thread_local std::string g_create_error;

}  // namespace

extern "C" {

int32_t kvp_version(void) { return 100; }

uint64_t kvp_token_bytes(const kvp_config *cfg)
{
    if (!valid_cfg(cfg)) return 0;
    return 2ull * cfg->n_layers * cfg->n_kv_heads * cfg->head_dim * (cfg->dtype == KVP_DTYPE_BF16 ? 2 : 4);
}

uint64_t kvp_workspace_bytes(const kvp_config *cfg)
{
    if (!valid_cfg(cfg)) return 0;
    return workspace_layout(cfg).total;
}

const char *kvp_last_error(kvp_ctx *ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

int32_t kvp_create(const kvp_config *cfg, kvp_ctx **out)
{
    if (!out) return KVP_ERR_INVALID;
    *out = nullptr;
    if (!valid_cfg(cfg)) { g_create_error = "invalid configuration"; return KVP_ERR_INVALID; }
    g_create_error.clear();
    kvp_ctx *ctx = new kvp_ctx();
    ctx->cfg = *cfg;
    ctx->host_only = cfg->device < 0;
    kvp_shape &sh = ctx->shape;
    sh.n_layers = cfg->n_layers;
    sh.n_q_heads = cfg->n_q_heads;
    sh.n_kv_heads = cfg->n_kv_heads;
    sh.head_dim = cfg->head_dim;
    sh.group = cfg->n_q_heads / cfg->n_kv_heads;
    sh.dtype = cfg->dtype;
    sh.pairing = cfg->rope_pairing;
    sh.elem_bytes = cfg->dtype == KVP_DTYPE_BF16 ? 2 : 4;
    sh.scale = (float)(cfg->softmax_scale > 0.0 ? cfg->softmax_scale : 1.0 / sqrt((double)cfg->head_dim));
    sh.pool_rows = (int64_t)(cfg->pool_bytes / kvp_token_bytes(cfg));
    sh.ws_rows = cfg->max_ws_rows;
    ctx->inv_freq.resize(cfg->head_dim / 2);
    for (int i = 0; i < cfg->head_dim / 2; ++i)
        ctx->inv_freq[i] = cfg->inv_freq ? cfg->inv_freq[i] : pow(cfg->rope_theta, -2.0 * i / cfg->head_dim);
    ctx->cfg.inv_freq = nullptr;
    ctx->pl = plan_layout(cfg);
    {
        const sched_layout sl = schedule_layout(cfg);
        ctx->sched_off_works = sl.works;
        ctx->sched_off_merges = sl.merges;
        ctx->sched_bytes = sl.total;
        ctx->sched_max_works = sl.max_works;
        ctx->sched_max_merges = sl.max_merges;
    }
    ctx->slots.resize(cfg->max_assemblies);
    *out = ctx;
    if (ctx->host_only) {
        if (sh.pool_rows <= 0) sh.pool_rows = INT32_MAX;      // sizes only: no pool behind it
        return KVP_OK;
    }

    const ws_layout w = workspace_layout(cfg);
    auto bail = [&](int32_t code, const char *msg) {
        g_create_error = msg;
        delete ctx;
        *out = nullptr;
        return code;
    };
    if (!cfg->pool || !cfg->workspace || ((uintptr_t)cfg->pool % kAlign) || ((uintptr_t)cfg->workspace % kAlign))
        return bail(KVP_ERR_INVALID, "pool/workspace must be non-null and 1024-byte aligned");
    if (sh.pool_rows <= 0) return bail(KVP_ERR_CAPACITY, "pool smaller than one token");
    if (cfg->workspace_bytes < w.total) return bail(KVP_ERR_CAPACITY, "workspace too small");
    if (cudaSetDevice(cfg->device) != cudaSuccess) return bail(KVP_ERR_CUDA, "cudaSetDevice failed");
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return bail(KVP_ERR_CUDA, "no device properties");
    ctx->sm_count = prop.multiProcessorCount;

    const uint64_t plane_bytes = (uint64_t)sh.n_layers * sh.n_kv_heads * sh.pool_rows * sh.head_dim * sh.elem_bytes;
    ctx->pool_k = (char *)cfg->pool;
    ctx->pool_v = ctx->pool_k + plane_bytes;
    char *ws = (char *)cfg->workspace;
    ctx->status_dev = (int32_t *)(ws + w.status);
    for (int a = 0; a < cfg->max_assemblies; ++a) {
        char *s = ws + w.slots + w.slot_stride * a;
        ctx->slot_plan_dev.push_back(s + w.slot_plan);
        ctx->slot_sched_dev.push_back(s + w.slot_sched);
        ctx->slot_k.push_back(s + w.slot_k);
        ctx->slot_v.push_back(s + w.slot_v);
    }
    ctx->partial_o = (float *)(ws + w.partial_o);
    ctx->partial_ml = (float2 *)(ws + w.partial_ml);
    ctx->q_scratch = ws + w.q_scratch;

    if (cudaMemset(cfg->pool, 0, 2 * plane_bytes) != cudaSuccess ||
        cudaMemset(cfg->workspace, 0, w.total) != cudaSuccess ||
        cudaMemcpy(ws + w.inv_freq, ctx->inv_freq.data(), 8 * ctx->inv_freq.size(), cudaMemcpyHostToDevice) !=
            cudaSuccess ||
        cudaDeviceSynchronize() != cudaSuccess)
        return bail(KVP_ERR_CUDA, "clearing pool/workspace failed");

    for (int a = 0; a < cfg->max_assemblies; ++a) {
        char *h = nullptr;
        cudaEvent_t ev;
        if (cudaHostAlloc((void **)&h, ctx->pl.total, cudaHostAllocDefault) != cudaSuccess ||
            cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess)
            return bail(KVP_ERR_CUDA, "pinned staging allocation failed");
        ctx->slot_plan_host.push_back(h);
        ctx->slot_event.push_back(ev);
        char *hs = nullptr;
        cudaEvent_t evs;
        if (cudaHostAlloc((void **)&hs, ctx->sched_bytes, cudaHostAllocDefault) != cudaSuccess ||
            cudaEventCreateWithFlags(&evs, cudaEventDisableTiming) != cudaSuccess)
            return bail(KVP_ERR_CUDA, "pinned staging allocation failed");
        ctx->slot_sched_host.push_back(hs);
        ctx->sched_event.push_back(evs);
    }

    if (cudaStreamCreateWithFlags(&ctx->load_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->load_fence, cudaEventDisableTiming) != cudaSuccess)
        return bail(KVP_ERR_CUDA, "load stream creation failed");
    ctx->load_done.resize(sh.n_layers);
    for (int l = 0; l < sh.n_layers; ++l)
        if (cudaEventCreateWithFlags(&ctx->load_done[l], cudaEventDisableTiming) != cudaSuccess)
            return bail(KVP_ERR_CUDA, "load event creation failed");

    if (sh.dtype == KVP_DTYPE_BF16 && sh.head_dim == 128 && prop.major == 10) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess && fn &&
            qres == cudaDriverEntryPointSuccess) {
            encode_tiled_fn enc = (encode_tiled_fn)fn;
            ctx->encode_tiled = fn;
            const int planes = sh.n_layers * sh.n_kv_heads;
            bool ok = make_tensor_map(enc, &ctx->tm_pool_k, ctx->pool_k, sh.head_dim, sh.pool_rows, planes) &&
                      make_tensor_map(enc, &ctx->tm_pool_v, ctx->pool_v, sh.head_dim, sh.pool_rows, planes);
            ctx->tm_ws_k.resize(cfg->max_assemblies);
            ctx->tm_ws_v.resize(cfg->max_assemblies);
            for (int a = 0; ok && a < cfg->max_assemblies; ++a)
                ok = make_tensor_map(enc, &ctx->tm_ws_k[a], ctx->slot_k[a], sh.head_dim, sh.ws_rows, planes) &&
                     make_tensor_map(enc, &ctx->tm_ws_v[a], ctx->slot_v[a], sh.head_dim, sh.ws_rows, planes);
            if (!ok) return bail(KVP_ERR_CUDA, "cuTensorMapEncodeTiled failed");
            if (kvp_attn_sm100_prepare() != cudaSuccess)
                return bail(KVP_ERR_CUDA, "tcgen05 kernel attribute setup failed");
            ctx->have_tma = true;
        }
    }
    return KVP_OK;
}

int32_t kvp_destroy(kvp_ctx *ctx)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (!ctx->host_only) {
        cudaSetDevice(ctx->cfg.device);
        cudaDeviceSynchronize();
        for (char *h : ctx->slot_plan_host) cudaFreeHost(h);
        for (cudaEvent_t e : ctx->slot_event) cudaEventDestroy(e);
        for (char *h : ctx->slot_sched_host) cudaFreeHost(h);
        for (cudaEvent_t e : ctx->sched_event) cudaEventDestroy(e);
        for (auto &w : ctx->tev) for (auto &v : w) for (cudaEvent_t e : v) cudaEventDestroy(e);
        for (cudaEvent_t e : ctx->load_done) cudaEventDestroy(e);
        if (ctx->load_fence) cudaEventDestroy(ctx->load_fence);
        if (ctx->load_stream) cudaStreamDestroy(ctx->load_stream);
    }
    delete ctx;
    return KVP_OK;
}

static int32_t store_segment(kvp_ctx *ctx, const void *k, const void *v, int32_t n, cudaStream_t st)
{
    if (n == 0 || ctx->host_only) return KVP_OK;
    const kvp_shape &sh = ctx->shape;
    KVP_CUDA(ctx, kvp_launch_store_rows(sh, k, ctx->pool_k, sh.pool_rows, ctx->pool_rows_used, n, st));
    KVP_CUDA(ctx, kvp_launch_store_rows(sh, v, ctx->pool_v, sh.pool_rows, ctx->pool_rows_used, n, st));
    return KVP_OK;
}

int32_t kvp_register_packet(kvp_ctx *ctx, const void *k, const void *v, int32_t n_tokens, int32_t cache_pos0,
                            void *stream, int32_t *packet_id)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (!packet_id || n_tokens <= 0) return fail(ctx, KVP_ERR_INVALID, "register_packet: bad arguments");
    if (!ctx->host_only && (!k || !v)) return fail(ctx, KVP_ERR_INVALID, "register_packet: null K/V");
    if (((uintptr_t)k | (uintptr_t)v) & 15) return fail(ctx, KVP_ERR_INVALID, "register_packet: K/V must be 16-byte aligned");
    if ((int)ctx->packets.size() >= ctx->cfg.max_packets) return fail(ctx, KVP_ERR_CAPACITY, "max_packets reached");
    if (ctx->pool_rows_used + n_tokens > ctx->shape.pool_rows) return fail(ctx, KVP_ERR_CAPACITY, "pool full");
    const int32_t rc = store_segment(ctx, k, v, n_tokens, (cudaStream_t)stream);
    if (rc != KVP_OK) return rc;
    ctx->packets.push_back({(int32_t)ctx->pool_rows_used, n_tokens, cache_pos0, {}});
    ctx->pool_rows_used += n_tokens;
    *packet_id = (int32_t)ctx->packets.size() - 1;
    return KVP_OK;
}

int32_t kvp_register_packet_host(kvp_ctx *ctx, const void *k_host, const void *v_host, int32_t n_tokens,
                                 int32_t cache_pos0, int32_t *packet_id)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (!packet_id || n_tokens <= 0) return fail(ctx, KVP_ERR_INVALID, "register_packet_host: bad arguments");
    if (!ctx->host_only && (!k_host || !v_host)) return fail(ctx, KVP_ERR_INVALID, "register_packet_host: null K/V");
    if ((int)ctx->packets.size() >= ctx->cfg.max_packets) return fail(ctx, KVP_ERR_CAPACITY, "max_packets reached");
    if (ctx->pool_rows_used + n_tokens > ctx->shape.pool_rows) return fail(ctx, KVP_ERR_CAPACITY, "pool full");
    ctx->packets.push_back({(int32_t)ctx->pool_rows_used, n_tokens, cache_pos0, {}});
    ctx->pool_rows_used += n_tokens;
    ctx->packet_src.resize(ctx->packets.size());
    kvp_ctx::host_src &src = ctx->packet_src.back();
    src.k = (const char *)k_host;
    src.v = (const char *)v_host;
    src.from_host = true;
    src.resident = false;
    *packet_id = (int32_t)ctx->packets.size() - 1;
    return KVP_OK;
}

int32_t kvp_evict_packet(kvp_ctx *ctx, int32_t packet_id)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (packet_id < 0 || packet_id >= (int)ctx->packets.size()) return fail(ctx, KVP_ERR_NOT_FOUND, "evict_packet: unknown packet id %d", packet_id);
    if (packet_id >= (int)ctx->packet_src.size() || !ctx->packet_src[packet_id].from_host)
        return fail(ctx, KVP_ERR_STATE, "evict_packet: packet %d has no host copy to come back from", packet_id);
    ctx->packet_src[packet_id].resident = false;
    return KVP_OK;
}

// Host -> pool copies of the packets of an assembly that are not on the device yet, one layer after the other
// on the context's own stream, an event per layer.  Host layout [n_layers][n_kv_heads][n_tokens][head_dim]: a
// layer of a packet is n_kv_heads runs of n_tokens rows, one per plane, i.e. one 2-D copy for K and one for V.
static int32_t load_host_packets(kvp_ctx *ctx, const std::vector<int32_t> &ids, cudaStream_t st)
{
    const kvp_shape &sh = ctx->shape;
    const size_t row_bytes = (size_t)sh.head_dim * sh.elem_bytes;
    KVP_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    // the rows may still be read by work the caller enqueued before (a packet that was evicted)
    KVP_CUDA(ctx, cudaEventRecord(ctx->load_fence, st));
    KVP_CUDA(ctx, cudaStreamWaitEvent(ctx->load_stream, ctx->load_fence, 0));
    for (int l = 0; l < sh.n_layers; ++l) {
        for (int32_t id : ids) {
            const kvp_segment_host &pk = ctx->packets[id];
            const kvp_ctx::host_src &src = ctx->packet_src[id];
            const size_t run = (size_t)pk.n * row_bytes;
            const size_t dst = ((size_t)l * sh.n_kv_heads * sh.pool_rows + pk.row0) * row_bytes;
            const size_t from = (size_t)l * sh.n_kv_heads * run;
            KVP_CUDA(ctx, cudaMemcpy2DAsync(ctx->pool_k + dst, (size_t)sh.pool_rows * row_bytes, src.k + from, run, run,
                                            sh.n_kv_heads, cudaMemcpyHostToDevice, ctx->load_stream));
            KVP_CUDA(ctx, cudaMemcpy2DAsync(ctx->pool_v + dst, (size_t)sh.pool_rows * row_bytes, src.v + from, run, run,
                                            sh.n_kv_heads, cudaMemcpyHostToDevice, ctx->load_stream));
        }
        KVP_CUDA(ctx, cudaEventRecord(ctx->load_done[l], ctx->load_stream));
    }
    for (int32_t id : ids) ctx->packet_src[id].resident = true;
    ctx->loads_recorded = true;
    return KVP_OK;
}

int32_t kvp_register_packet_compressed(kvp_ctx *ctx, const void *k, const void *v, int32_t n_tokens,
                                       int32_t cache_pos0, const int32_t *kept, void *stream, int32_t *packet_id)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (!packet_id || !kept || n_tokens <= 0) return fail(ctx, KVP_ERR_INVALID, "register_packet_compressed: bad arguments");
    if (ctx->cfg.max_compressed <= 0) return fail(ctx, KVP_ERR_STATE, "register_packet_compressed: max_compressed is 0");
    if (!ctx->host_only && (!k || !v)) return fail(ctx, KVP_ERR_INVALID, "register_packet_compressed: null K/V");
    if ((int)ctx->packets.size() >= ctx->cfg.max_packets) return fail(ctx, KVP_ERR_CAPACITY, "max_packets reached");
    const kvp_shape &sh = ctx->shape;
    const int planes = sh.n_layers * sh.n_kv_heads;
    int32_t n_max = 0;
    for (int i = 0; i < planes; ++i) {
        if (kept[i] < 1 || kept[i] > n_tokens) return fail(ctx, KVP_ERR_INVALID, "register_packet_compressed: kept[%d] = %d", i, kept[i]);
        n_max = std::max(n_max, kept[i]);
    }
    if (ctx->pool_rows_used + n_max > sh.pool_rows) return fail(ctx, KVP_ERR_CAPACITY, "pool full");
    if (!ctx->host_only) {
        // plane (l, h) receives its run of kept rows; the runs lie back to back in the caller's buffers
        cudaStream_t st = (cudaStream_t)stream;
        KVP_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
        const size_t row_bytes = (size_t)sh.head_dim * sh.elem_bytes;
        size_t src_off = 0;
        for (int i = 0; i < planes; ++i) {
            const size_t dst_off = ((size_t)i * sh.pool_rows + ctx->pool_rows_used) * row_bytes;
            const size_t n = (size_t)kept[i] * row_bytes;
            KVP_CUDA(ctx, cudaMemcpyAsync(ctx->pool_k + dst_off, (const char *)k + src_off, n, cudaMemcpyDeviceToDevice, st));
            KVP_CUDA(ctx, cudaMemcpyAsync(ctx->pool_v + dst_off, (const char *)v + src_off, n, cudaMemcpyDeviceToDevice, st));
            src_off += n;
        }
    }
    ctx->packets.push_back({(int32_t)ctx->pool_rows_used, n_tokens, cache_pos0, std::vector<int32_t>(kept, kept + planes)});
    ctx->pool_rows_used += n_max;
    *packet_id = (int32_t)ctx->packets.size() - 1;
    return KVP_OK;
}

int32_t kvp_register_adapter(kvp_ctx *ctx, const void *hk, const void *hv, int32_t n_header, int32_t header_pos0,
                             const void *tk, const void *tv, int32_t n_trailer, int32_t trailer_pos0, void *stream,
                             int32_t *adapter_id)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (!adapter_id || n_header < 0 || n_trailer < 0) return fail(ctx, KVP_ERR_INVALID, "register_adapter: bad arguments");
    if (!ctx->host_only && ((n_header > 0 && (!hk || !hv)) || (n_trailer > 0 && (!tk || !tv))))
        return fail(ctx, KVP_ERR_INVALID, "register_adapter: null K/V");
    if (((n_header > 0 ? ((uintptr_t)hk | (uintptr_t)hv) : 0) | (n_trailer > 0 ? ((uintptr_t)tk | (uintptr_t)tv) : 0)) & 15)
        return fail(ctx, KVP_ERR_INVALID, "register_adapter: K/V must be 16-byte aligned");
    if ((int)ctx->adapter_h.size() >= ctx->cfg.max_adapters) return fail(ctx, KVP_ERR_CAPACITY, "max_adapters reached");
    if (ctx->pool_rows_used + n_header + n_trailer > ctx->shape.pool_rows) return fail(ctx, KVP_ERR_CAPACITY, "pool full");
    int32_t rc = store_segment(ctx, hk, hv, n_header, (cudaStream_t)stream);
    if (rc != KVP_OK) return rc;
    ctx->adapter_h.push_back({(int32_t)ctx->pool_rows_used, n_header, header_pos0, {}});
    ctx->pool_rows_used += n_header;
    rc = store_segment(ctx, tk, tv, n_trailer, (cudaStream_t)stream);
    if (rc != KVP_OK) { ctx->adapter_h.pop_back(); ctx->pool_rows_used -= n_header; return rc; }
    ctx->adapter_t.push_back({(int32_t)ctx->pool_rows_used, n_trailer, trailer_pos0, {}});
    ctx->pool_rows_used += n_trailer;
    *adapter_id = (int32_t)ctx->adapter_h.size() - 1;
    return KVP_OK;
}

static int32_t assemble_impl(kvp_ctx *ctx, int32_t batch, const int32_t *slot_offsets, const int32_t *packet_ids,
                             const int32_t *adapter_ids, const int32_t *pos_base, uint32_t flags, void *stream,
                             int32_t *prefix_len, int32_t *assembly_id)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (!slot_offsets || !packet_ids || !adapter_ids || !prefix_len || !assembly_id || batch <= 0)
        return fail(ctx, KVP_ERR_INVALID, "assemble: bad arguments");
    if (flags & ~(uint32_t)(KVP_REBASE | KVP_MATERIALIZE)) return fail(ctx, KVP_ERR_INVALID, "assemble: unknown flags");
    const kvp_config &cfg = ctx->cfg;
    if (batch > cfg.max_batch) return fail(ctx, KVP_ERR_CAPACITY, "assemble: batch > max_batch");
    if (slot_offsets[0] != 0) return fail(ctx, KVP_ERR_INVALID, "assemble: slot_offsets[0] != 0");
    for (int b = 0; b < batch; ++b)
        if (slot_offsets[b + 1] < slot_offsets[b]) return fail(ctx, KVP_ERR_INVALID, "assemble: slot_offsets not monotone");
    const int n_slots = slot_offsets[batch];
    if (n_slots > cfg.max_slots) return fail(ctx, KVP_ERR_CAPACITY, "assemble: more than max_slots slots");
    for (int s = 0; s < n_slots; ++s) {
        if (packet_ids[s] < 0 || packet_ids[s] >= (int)ctx->packets.size())
            return fail(ctx, KVP_ERR_NOT_FOUND, "assemble: unknown packet id %d", packet_ids[s]);
        if (adapter_ids[s] < -1 || adapter_ids[s] >= (int)ctx->adapter_h.size())
            return fail(ctx, KVP_ERR_NOT_FOUND, "assemble: unknown adapter id %d", adapter_ids[s]);
    }
    const bool rebase = flags & KVP_REBASE, mat = flags & KVP_MATERIALIZE;
    const int half = cfg.head_dim / 2;

    kvp_assembly_host as;
    as.flags = flags;
    as.batch = batch;
    as.shard = pos_base != nullptr;
    if (pos_base)
        for (int b = 0; b < batch; ++b)
            if (pos_base[b] < 0) return fail(ctx, KVP_ERR_INVALID, "assemble_at: pos_base[%d] < 0", b);
    // packets that still wait in host memory are brought in now, layer by layer, on the context's own stream
    std::vector<int32_t> to_load;
    bool host_origin = false;
    for (int s = 0; s < n_slots; ++s) {
        const int32_t id = packet_ids[s];
        if (id >= (int)ctx->packet_src.size() || !ctx->packet_src[id].from_host) continue;
        host_origin = true;
        if (!ctx->packet_src[id].resident && std::find(to_load.begin(), to_load.end(), id) == to_load.end()) to_load.push_back(id);
    }
    as.waits_loads = host_origin && !ctx->host_only && (ctx->loads_recorded || !to_load.empty());
    const bool waits_loads = as.waits_loads;
    std::map<int32_t, int32_t> rope_of;        // delta -> rope-table index (0 = identity)
    std::vector<int32_t> rope_delta(1, 0);
    rope_of[0] = 0;
    std::vector<kvp_chunk> chunks;
    int64_t ws_cursor = 0;

    auto add_chunks = [&](int32_t src, int32_t dst, int32_t n, int32_t rope) {
        for (int32_t o = 0; o < n; o += KVP_CHUNK_ROWS)
            chunks.push_back({src + o, dst + o, std::min<int32_t>(KVP_CHUNK_ROWS, n - o), rope});
    };
    auto add_tiles = [&](int16_t src, int32_t row0, int32_t n, int32_t rope) {
        for (int32_t o = 0; o < n; o += KVP_TILE_KEYS)
            as.tiles.push_back({row0 + o, (int16_t)std::min<int32_t>(KVP_TILE_KEYS, n - o), src, rope, 0});
    };
    std::map<int32_t, int32_t> kept_row_of;    // compressed packet id -> row of the kept table
    std::vector<int32_t> kept_packets;
    struct item_build { kvp_item it; int32_t stage0, staged; };
    std::vector<item_build> builds;

    for (int b = 0; b < batch; ++b) {
        kvp_item it;
        memset(&it, 0, sizeof it);
        it.seg_begin = (int32_t)as.segs.size();
        int64_t t = 0;
        int64_t staged = 0;
        for (int s = slot_offsets[b]; s < slot_offsets[b + 1]; ++s) {
            const kvp_segment_host *parts[3] = {nullptr, &ctx->packets[packet_ids[s]], nullptr};
            if (adapter_ids[s] >= 0) {
                parts[0] = &ctx->adapter_h[adapter_ids[s]];
                parts[2] = &ctx->adapter_t[adapter_ids[s]];
            }
            for (int k = 0; k < 3; ++k) {
                const kvp_segment_host *sg = parts[k];
                if (!sg || sg->n == 0) continue;
                kvp_seg e;
                memset(&e, 0, sizeof e);
                e.src_row0 = sg->row0;
                e.len = sg->n;
                e.dst_pos0 = (int32_t)t;
                e.delta = rebase ? (int32_t)(t + (pos_base ? pos_base[b] : 0) - sg->pos0) : 0;
                auto f = rope_of.find(e.delta);
                if (f == rope_of.end()) {
                    f = rope_of.emplace(e.delta, (int32_t)rope_delta.size()).first;
                    rope_delta.push_back(e.delta);
                }
                e.rope = f->second;
                e.pad[0] = -1;                   // workspace row of a staged copy, if any
                e.pad[1] = k;                    // 0 header, 1 document, 2 trailer
                e.pad[2] = -1;                   // row of the kept table (compressed document)
                if (k == 1 && !sg->kept.empty()) {
                    auto kr = kept_row_of.find(packet_ids[s]);
                    if (kr == kept_row_of.end()) {
                        kr = kept_row_of.emplace(packet_ids[s], (int32_t)kept_packets.size()).first;
                        kept_packets.push_back(packet_ids[s]);
                    }
                    e.pad[2] = kr->second;
                }
                if (!mat && k != 1) staged += sg->n;
                as.segs.push_back(e);
                t += sg->n;
            }
        }
        if (t > cfg.max_prefix_tokens) return fail(ctx, KVP_ERR_CAPACITY, "assemble: request %d prefix %lld > max_prefix_tokens", b, (long long)t);
        it.seg_end = (int32_t)as.segs.size();
        it.prefix_len = (int32_t)t;
        prefix_len[b] = (int32_t)t;
        if (mat) {
            if (!kept_packets.empty()) return fail(ctx, KVP_ERR_UNSUPPORTED, "assemble: compressed packets cannot be materialised");
            it.tile_begin = (int32_t)as.tiles.size();
            it.cache_row0 = (int32_t)ws_cursor;
            for (int s = it.seg_begin; s < it.seg_end; ++s) {
                kvp_seg &e = as.segs[s];
                add_chunks(e.src_row0, it.cache_row0 + e.dst_pos0, e.len, e.rope);
            }
            add_tiles(1, it.cache_row0, it.prefix_len, 0);
            it.tail_row0 = it.cache_row0 + it.prefix_len;
            it.tile_end = (int32_t)as.tiles.size();
            ws_cursor += (int64_t)it.prefix_len + cfg.max_query_tokens;
            builds.push_back({it, 0, 0});
        } else {
            it.cache_row0 = -1;
            const int32_t stage0 = (int32_t)ws_cursor;
            int32_t so = 0;
            for (int s = it.seg_begin; s < it.seg_end; ++s) {      // adapter tokens: staged, re-based
                kvp_seg &e = as.segs[s];
                if (e.pad[1] == 1) continue;
                e.pad[0] = stage0 + so;
                add_chunks(e.src_row0, e.pad[0], e.len, e.rope);
                so += e.len;
            }
            it.tail_row0 = stage0 + so;
            ws_cursor += (int64_t)so + cfg.max_query_tokens;
            builds.push_back({it, stage0, so});
        }
        if (ws_cursor > cfg.max_ws_rows) return fail(ctx, KVP_ERR_CAPACITY, "assemble: needs more than max_ws_rows workspace rows");
    }
    if ((int)kept_packets.size() > cfg.max_compressed)
        return fail(ctx, KVP_ERR_CAPACITY, "assemble: %zu compressed packets > max_compressed", kept_packets.size());
    // tile lists: one for all planes, or - when a compressed packet keeps a different number of rows per
    // (layer, kv head) - one per plane, so that a head walks exactly the tiles it holds (documents are read
    // in place; the staged adapter rows come first)
    const int n_lists = kept_packets.empty() ? 1 : cfg.n_layers * cfg.n_kv_heads;
    as.item_stride = kept_packets.empty() ? 0 : batch;
    for (int l = 0; l < n_lists; ++l)
        for (int b = 0; b < batch; ++b) {
            kvp_item it = builds[b].it;
            if (!mat) {
                it.tile_begin = (int32_t)as.tiles.size();
                add_tiles(1, builds[b].stage0, builds[b].staged, 0);
                for (int s = it.seg_begin; s < it.seg_end; ++s) {
                    const kvp_seg &e = as.segs[s];
                    if (e.pad[1] != 1) continue;
                    if (e.pad[2] < 0) {
                        add_tiles(0, e.src_row0, e.len, e.rope);
                    } else {
                        const std::vector<int32_t> &kept = ctx->packets[kept_packets[e.pad[2]]].kept;
                        add_tiles(0, e.src_row0, kept[l], e.rope);              // l = layer * n_kv_heads + kv head
                    }
                }
                it.tile_end = (int32_t)as.tiles.size();
            }
            as.items.push_back(it);
        }
    if ((int)as.tiles.size() > ctx->pl.max_tiles || (int)chunks.size() > ctx->pl.max_chunks ||
        (int)as.items.size() > ctx->pl.max_items ||
        (int)rope_delta.size() > ctx->pl.max_rope || (int)as.segs.size() > ctx->pl.max_segs)
        return fail(ctx, KVP_ERR_CAPACITY, "assemble: plan tables overflow");
    as.n_chunks = (int32_t)chunks.size();
    as.n_rope = (int32_t)rope_delta.size();

    const int32_t id = ctx->next_assembly++;
    const int slot = id % cfg.max_assemblies;
    as.id = id;
    if (!ctx->host_only) {
        cudaStream_t st = (cudaStream_t)stream;
        KVP_CUDA(ctx, cudaSetDevice(cfg.device));
        KVP_CUDA(ctx, cudaEventSynchronize(ctx->slot_event[slot]));      // staging buffer free again?
        char *h = ctx->slot_plan_host[slot];
        memcpy(h + ctx->pl.items, as.items.data(), sizeof(kvp_item) * as.items.size());
        memcpy(h + ctx->pl.tiles, as.tiles.data(), sizeof(kvp_tile) * as.tiles.size());
        memcpy(h + ctx->pl.chunks, chunks.data(), sizeof(kvp_chunk) * chunks.size());
        memcpy(h + ctx->pl.segs, as.segs.data(), sizeof(kvp_seg) * as.segs.size());
        float2 *rt = reinterpret_cast<float2 *>(h + ctx->pl.rope);
        for (size_t r = 0; r < rope_delta.size(); ++r)
            for (int i = 0; i < half; ++i) {
                const double a = (double)rope_delta[r] * ctx->inv_freq[i];      // angle in double: Delta reaches 1e5
                rt[r * half + i] = make_float2((float)cos(a), (float)sin(a));
            }
        const uint64_t used = ctx->pl.rope + sizeof(float2) * rope_delta.size() * half;
        KVP_CUDA(ctx, cudaMemcpyAsync(ctx->slot_plan_dev[slot], h, used, cudaMemcpyHostToDevice, st));
        if (!kept_packets.empty()) {
            const size_t planes = (size_t)cfg.n_layers * cfg.n_kv_heads;
            int32_t *kt = reinterpret_cast<int32_t *>(h + ctx->pl.kept);
            for (size_t r = 0; r < kept_packets.size(); ++r)
                memcpy(kt + r * planes, ctx->packets[kept_packets[r]].kept.data(), 4 * planes);
            KVP_CUDA(ctx, cudaMemcpyAsync(ctx->slot_plan_dev[slot] + ctx->pl.kept, kt, 4 * planes * kept_packets.size(),
                                          cudaMemcpyHostToDevice, st));
        }
        KVP_CUDA(ctx, cudaEventRecord(ctx->slot_event[slot], st));
    }
    const int32_t n_chunks = as.n_chunks;
    ctx->slots[slot] = std::move(as);
    *assembly_id = id;
    if (ctx->host_only) {
        for (int32_t id : to_load) ctx->packet_src[id].resident = true;
    } else {
        cudaStream_t st = (cudaStream_t)stream;
        if (!to_load.empty()) {
            const int32_t rc = load_host_packets(ctx, to_load, st);
            if (rc != KVP_OK) return rc;
        }
        if (mat && waits_loads)                                   // the gather reads every layer of the documents
            KVP_CUDA(ctx, cudaStreamWaitEvent(st, ctx->load_done[ctx->shape.n_layers - 1], 0));
        KVP_CUDA(ctx, time_edge(ctx, 1, 0, st));
        KVP_CUDA(ctx, kvp_launch_gather(ctx->shape, plan_dev(ctx, slot), n_chunks, ctx->pool_k, ctx->pool_v,
                                        ctx->slot_k[slot], ctx->slot_v[slot], st));
        KVP_CUDA(ctx, time_edge(ctx, 1, 1, st));
    }
    return KVP_OK;
}

int32_t kvp_assemble(kvp_ctx *ctx, int32_t batch, const int32_t *slot_offsets, const int32_t *packet_ids,
                     const int32_t *adapter_ids, uint32_t flags, void *stream, int32_t *prefix_len,
                     int32_t *assembly_id)
{
    return assemble_impl(ctx, batch, slot_offsets, packet_ids, adapter_ids, nullptr, flags, stream, prefix_len, assembly_id);
}

int32_t kvp_assemble_at(kvp_ctx *ctx, int32_t batch, const int32_t *slot_offsets, const int32_t *packet_ids,
                        const int32_t *adapter_ids, const int32_t *pos_base, uint32_t flags, void *stream,
                        int32_t *prefix_len, int32_t *assembly_id)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (!pos_base) return fail(ctx, KVP_ERR_INVALID, "assemble_at: pos_base is null");
    return assemble_impl(ctx, batch, slot_offsets, packet_ids, adapter_ids, pos_base, flags, stream, prefix_len, assembly_id);
}

int32_t kvp_export_plan(kvp_ctx *ctx, int32_t assembly_id, int32_t b, int32_t *src_row, int32_t *delta,
                        int32_t *seg_table, int32_t *n_segments)
{
    if (!ctx) return KVP_ERR_INVALID;
    const int slot = find_slot(ctx, assembly_id);
    if (slot < 0) return fail(ctx, KVP_ERR_NOT_FOUND, "export_plan: unknown assembly %d", assembly_id);
    const kvp_assembly_host &as = ctx->slots[slot];
    if (b < 0 || b >= as.batch) return fail(ctx, KVP_ERR_INVALID, "export_plan: bad request index");
    const kvp_item &it = as.items[b];
    if (n_segments) *n_segments = it.seg_end - it.seg_begin;
    for (int s = it.seg_begin; s < it.seg_end; ++s) {
        const kvp_seg &e = as.segs[s];
        if (seg_table) {
            int32_t *row = seg_table + 4 * (s - it.seg_begin);
            row[0] = e.src_row0; row[1] = e.len; row[2] = e.dst_pos0; row[3] = e.delta;
        }
        for (int o = 0; o < e.len; ++o) {
            if (src_row) src_row[e.dst_pos0 + o] = e.pad[2] >= 0 ? -1 : e.src_row0 + o;   // compressed: no row per position
            if (delta) delta[e.dst_pos0 + o] = e.delta;
        }
    }
    return KVP_OK;
}

int32_t kvp_export_cache(kvp_ctx *ctx, int32_t assembly_id, int32_t layer, int32_t b, int32_t n_query_rows,
                         void *k_out, void *v_out, int32_t k_as_f32, void *stream)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (ctx->host_only) return fail(ctx, KVP_ERR_STATE, "export_cache: host-only context");
    const int slot = find_slot(ctx, assembly_id);
    if (slot < 0) return fail(ctx, KVP_ERR_NOT_FOUND, "export_cache: unknown assembly %d", assembly_id);
    const kvp_assembly_host &as = ctx->slots[slot];
    if (as.item_stride) return fail(ctx, KVP_ERR_UNSUPPORTED, "export_cache: the assembly uses compressed packets");
    if (as.ragged && n_query_rows > 0)
        return fail(ctx, KVP_ERR_UNSUPPORTED, "export_cache: query rows after kvp_query_prefill_ragged differ per request");
    if (b < 0 || b >= as.batch || layer < 0 || layer >= ctx->cfg.n_layers || !k_out || !v_out || n_query_rows < 0 ||
        n_query_rows > ctx->cfg.max_query_tokens)
        return fail(ctx, KVP_ERR_INVALID, "export_cache: bad arguments");
    KVP_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    if (as.waits_loads) KVP_CUDA(ctx, cudaStreamWaitEvent((cudaStream_t)stream, ctx->load_done[layer], 0));
    KVP_CUDA(ctx, kvp_launch_export(ctx->shape, plan_dev(ctx, slot), b, layer, as.items[b].prefix_len, n_query_rows,
                                    ctx->pool_k, ctx->pool_v, ctx->slot_k[slot], ctx->slot_v[slot], k_out, v_out,
                                    k_as_f32, (cudaStream_t)stream));
    return KVP_OK;
}

static int32_t query_prefill_impl(kvp_ctx *ctx, int32_t assembly_id, int32_t layer, const void *q, const void *k_new,
                                  const void *v_new, int32_t q_len, const int32_t *q_lens, uint32_t flags, void *out,
                                  float *lse, void *stream)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (ctx->host_only) return fail(ctx, KVP_ERR_STATE, "query_prefill: host-only context has no device to run on");
    const int slot = find_slot(ctx, assembly_id);
    if (slot < 0) return fail(ctx, KVP_ERR_NOT_FOUND, "query_prefill: unknown assembly %d", assembly_id);
    if (!q || !k_new || !v_new || !out || layer < 0 || layer >= ctx->cfg.n_layers || q_len <= 0)
        return fail(ctx, KVP_ERR_INVALID, "query_prefill: bad arguments");
    if (flags & ~(uint32_t)(KVP_ROPE_QUERY | KVP_FORCE_SIMPLE | KVP_CONTINUE | KVP_PRECISE_QK | KVP_PARTIAL | KVP_SKIP_QUERY_BLOCK))
        return fail(ctx, KVP_ERR_INVALID, "query_prefill: unknown flags");
    const uint32_t part_opts = flags & (uint32_t)(KVP_PARTIAL | KVP_SKIP_QUERY_BLOCK);
    if ((flags & KVP_SKIP_QUERY_BLOCK) && !(flags & KVP_PARTIAL))
        return fail(ctx, KVP_ERR_INVALID, "query_prefill: KVP_SKIP_QUERY_BLOCK needs KVP_PARTIAL");
    if (part_opts && ((flags & (KVP_CONTINUE | KVP_ROPE_QUERY | KVP_FORCE_SIMPLE)) || q_lens || !ctx->have_tma))
        return fail(ctx, KVP_ERR_UNSUPPORTED, "query_prefill: KVP_PARTIAL runs on the tcgen05 kernel only, without KVP_CONTINUE, KVP_ROPE_QUERY or per-request lengths");
    {
        // every kernel reads whole elements; the tcgen05 path moves q and out 16 bytes at a time
        const uintptr_t all = (uintptr_t)q | (uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)out;
        if ((all & (uintptr_t)(ctx->shape.elem_bytes - 1)) || ((uintptr_t)lse & 3))
            return fail(ctx, KVP_ERR_INVALID, "query_prefill: q / k_new / v_new / out / lse not aligned to their element size");
        if (ctx->have_tma && !(flags & KVP_FORCE_SIMPLE) && ((((uintptr_t)q | (uintptr_t)out) & 15) != 0))
            return fail(ctx, KVP_ERR_INVALID, "query_prefill: q and out must be 16-byte aligned on the tcgen05 path (KVP_FORCE_SIMPLE takes any element-aligned pointer)");
    }
    if (q_len > ctx->cfg.max_query_tokens) return fail(ctx, KVP_ERR_CAPACITY, "query_prefill: q_len > max_query_tokens");
    kvp_assembly_host &as = ctx->slots[slot];
    const kvp_shape &sh = ctx->shape;
    cudaStream_t st = (cudaStream_t)stream;
    if ((int)as.appended.size() != ctx->cfg.n_layers) as.appended.assign(ctx->cfg.n_layers, 0);
    const int q_pos0 = (flags & KVP_CONTINUE) ? as.appended[layer] : 0;
    if (q_pos0 + q_len > ctx->cfg.max_query_tokens)
        return fail(ctx, KVP_ERR_CAPACITY, "query_prefill: %d rows appended + q_len %d > max_query_tokens", q_pos0, q_len);
    KVP_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    if (as.waits_loads) KVP_CUDA(ctx, cudaStreamWaitEvent(st, ctx->load_done[layer], 0));   // this layer's documents have landed
    const kvp_plan_dev plan = plan_dev(ctx, slot);
    const int rope_query = (flags & KVP_ROPE_QUERY) ? 1 : 0;
    if (rope_query && as.shard)
        return fail(ctx, KVP_ERR_UNSUPPORTED, "query_prefill: KVP_ROPE_QUERY on an assembly made by kvp_assemble_at (the query's position is not prefix_len)");
    const bool skip_block = (flags & KVP_SKIP_QUERY_BLOCK) != 0;
    const double *inv_freq_dev = reinterpret_cast<const double *>((char *)ctx->cfg.workspace + 256);

    int launches = 0;
    const bool fast = ctx->have_tma && !(flags & KVP_FORCE_SIMPLE);
    if (q_lens && !fast) return fail(ctx, KVP_ERR_UNSUPPORTED, "query_prefill_ragged: needs the tcgen05 kernel (bf16, head_dim 128, sm_100)");
    // plain prefill on the two-stream kernel: it reads the query block's K/V from k_new / v_new and appends them itself
    kvp_attn2_args a;
    a.tail_direct = 0;
    a.precise = (flags & KVP_PRECISE_QK) ? 1 : 0;
    if (fast && ctx->fused_append && !rope_query && q_pos0 == 0 && !skip_block &&
        (((uintptr_t)k_new | (uintptr_t)v_new) & 15) == 0 &&
        make_query_tensor_map((encode_tiled_fn)ctx->encode_tiled, &a.tm_knew, k_new, sh.head_dim, sh.n_kv_heads, q_len, as.batch) &&
        make_query_tensor_map((encode_tiled_fn)ctx->encode_tiled, &a.tm_vnew, v_new, sh.head_dim, sh.n_kv_heads, q_len, as.batch))
        a.tail_direct = 1;
    if (q_lens && !a.tail_direct)
        return fail(ctx, KVP_ERR_UNSUPPORTED, "query_prefill_ragged: needs the tcgen05 kernel with its own append (bf16, head_dim 128, 16-byte aligned k_new / v_new)");
    if (!a.tail_direct && !skip_block) {
        KVP_CUDA(ctx, kvp_launch_append(sh, plan, as.batch, q_len, q_pos0, q, k_new, v_new, ctx->slot_k[slot], ctx->slot_v[slot],
                                        layer, rope_query, inv_freq_dev, ctx->q_scratch, st));
        ++launches;
    }
    const void *q_used = rope_query ? (const void *)ctx->q_scratch : q;
    as.last_q_len = q_len;
    as.appended[layer] = (q_lens || skip_block) ? 0 : q_pos0 + q_len;       // after a ragged call the rows behind the prefixes differ per request
    if (q_lens) as.ragged = true;

    int32_t ctas = 0, splits = 1;
    if (!fast) {
        KVP_CUDA(ctx, time_edge(ctx, 0, 0, st));
        KVP_CUDA(ctx, kvp_launch_attn_simple(sh, plan, as.batch, q_len, q_pos0, layer, q_used, ctx->pool_k, ctx->pool_v,
                                             ctx->slot_k[slot], ctx->slot_v[slot], out, lse, &ctas, st));
        KVP_CUDA(ctx, time_edge(ctx, 0, 1, st));
        ++launches;
        ctx->last_kind = 0;
    } else {
        const int li = as.item_stride ? layer : 0;
        if (as.sched.empty()) as.sched.resize(as.item_stride ? ctx->cfg.n_layers : 1);
        const bool same_lens = q_lens ? (as.sched[li].q_lens.size() == (size_t)as.batch &&
                                          std::equal(q_lens, q_lens + as.batch, as.sched[li].q_lens.begin()))
                                       : as.sched[li].q_lens.empty();
        if (as.sched[li].q_len != q_len || as.sched[li].q_pos0 != q_pos0 || as.sched[li].ctas == 0 || !same_lens ||
            as.sched[li].opts != part_opts) {
            const int32_t rc = build_schedule(ctx, as, slot, layer, q_len, q_pos0, q_lens, part_opts, st);
            if (rc != KVP_OK) return rc;
        }
        const kvp_assembly_host::sched_state &ss = as.sched[li];
        const char *sd = ctx->slot_sched_dev[slot] + ctx->sched_bytes * li;
        a.k_new = k_new;
        a.v_new = v_new;
        a.ws_k = ctx->slot_k[slot];
        a.ws_v = ctx->slot_v[slot];
        a.plan = plan;
        a.l2_prefetch = (sh.group * q_len <= 4 * KVP_TILE_ROWS) ? 1 : 0;      // <= 2 units share a (request, kv head)'s K/V
        a.q_len = q_len;
        a.q_pos0 = q_pos0;
        a.layer = layer;
        a.n_ctas = ss.ctas;
        a.cta_begin = reinterpret_cast<const int32_t *>(sd);
        a.works = reinterpret_cast<const kvp_work *>(sd + ctx->sched_off_works);
        a.q = q_used;
        a.out = out;
        a.lse = lse;
        a.partial_o = ctx->partial_o;
        a.partial_ml = ctx->partial_ml;
        a.status = ctx->status_dev;
        if (ss.ctas > 0) {                                         // (a rank may hold no key of any request)
            KVP_CUDA(ctx, time_edge(ctx, 0, 0, st));
            KVP_CUDA(ctx, kvp_launch_attn_sm100(sh, a, ctx->tm_pool_k, ctx->tm_pool_v, ctx->tm_ws_k[slot], ctx->tm_ws_v[slot], st));
            KVP_CUDA(ctx, time_edge(ctx, 0, 1, st));
            ++launches;
        }
        if (ss.merges > 0) {
            const bool partial = (flags & KVP_PARTIAL) != 0;
            const int64_t n_rt = ((int64_t)sh.group * q_len + KVP_TILE_ROWS - 1) / KVP_TILE_ROWS;
            KVP_CUDA(ctx, kvp_launch_merge_list(sh, q_len, ss.merges,
                                                reinterpret_cast<const kvp_merge_item *>(sd + ctx->sched_off_merges),
                                                ctx->partial_o, ctx->partial_ml, out, lse, partial ? out : nullptr,
                                                (int64_t)as.batch * sh.n_kv_heads * n_rt, st));
            ++launches;
        }
        ctas = ss.ctas;
        splits = ss.slots;
        ctx->last_kind = 1;
    }
    ctx->last_ctas = ctas;
    ctx->last_splits = splits;
    ctx->last_launches = launches;
    return KVP_OK;
}

int32_t kvp_query_prefill(kvp_ctx *ctx, int32_t assembly_id, int32_t layer, const void *q, const void *k_new,
                          const void *v_new, int32_t q_len, uint32_t flags, void *out, float *lse, void *stream)
{
    return query_prefill_impl(ctx, assembly_id, layer, q, k_new, v_new, q_len, nullptr, flags, out, lse, stream);
}

int32_t kvp_query_prefill_ragged(kvp_ctx *ctx, int32_t assembly_id, int32_t layer, const void *q, const void *k_new,
                                 const void *v_new, int32_t q_len_max, const int32_t *q_lens, void *out, float *lse,
                                 void *stream)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (!q_lens) return fail(ctx, KVP_ERR_INVALID, "query_prefill_ragged: q_lens is null");
    const int slot = find_slot(ctx, assembly_id);
    if (slot < 0) return fail(ctx, KVP_ERR_NOT_FOUND, "query_prefill_ragged: unknown assembly %d", assembly_id);
    for (int b = 0; b < ctx->slots[slot].batch; ++b)
        if (q_lens[b] < 1 || q_lens[b] > q_len_max)
            return fail(ctx, KVP_ERR_INVALID, "query_prefill_ragged: q_lens[%d] = %d outside [1, %d]", b, q_lens[b], q_len_max);
    return query_prefill_impl(ctx, assembly_id, layer, q, k_new, v_new, q_len_max, q_lens, 0, out, lse, stream);
}

uint64_t kvp_partial_bytes(kvp_ctx *ctx, int32_t batch, int32_t q_len)
{
    if (!ctx || batch <= 0 || q_len <= 0) return 0;
    const kvp_shape &sh = ctx->shape;
    const uint64_t n_rt = ((uint64_t)sh.group * q_len + KVP_TILE_ROWS - 1) / KVP_TILE_ROWS;
    return (uint64_t)batch * sh.n_kv_heads * n_rt * (KVP_TILE_ROWS * ((uint64_t)sh.head_dim * 4 + 8));
}

int32_t kvp_merge_partials(kvp_ctx *ctx, const void *parts, int32_t n_parts, int32_t batch, int32_t q_len, void *out,
                           float *lse, void *stream)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (ctx->host_only) return fail(ctx, KVP_ERR_STATE, "merge_partials: host-only context");
    if (!parts || !out || n_parts <= 0 || batch <= 0 || q_len <= 0 || (((uintptr_t)parts | (uintptr_t)out) & 15) || ((uintptr_t)lse & 3))
        return fail(ctx, KVP_ERR_INVALID, "merge_partials: bad arguments (parts and out must be 16-byte aligned)");
    if (!ctx->have_tma) return fail(ctx, KVP_ERR_UNSUPPORTED, "merge_partials: bf16, head_dim 128, sm_100 only");
    if (batch > ctx->cfg.max_batch || q_len > ctx->cfg.max_query_tokens)
        return fail(ctx, KVP_ERR_CAPACITY, "merge_partials: batch or q_len beyond the context's maxima");
    KVP_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    KVP_CUDA(ctx, kvp_launch_merge_ranks(ctx->shape, batch, q_len, parts, n_parts, out, lse, (cudaStream_t)stream));
    return KVP_OK;
}

int32_t kvp_segment_mass(kvp_ctx *ctx, int32_t assembly_id, int32_t layer, const void *q, const float *lse,
                         int32_t q_len, uint32_t flags, float *mass, int32_t n_cols, void *stream)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (ctx->host_only) return fail(ctx, KVP_ERR_STATE, "segment_mass: host-only context");
    const int slot = find_slot(ctx, assembly_id);
    if (slot < 0) return fail(ctx, KVP_ERR_NOT_FOUND, "segment_mass: unknown assembly %d", assembly_id);
    if (!q || !lse || !mass || layer < 0 || layer >= ctx->cfg.n_layers || q_len <= 0)
        return fail(ctx, KVP_ERR_INVALID, "segment_mass: bad arguments");
    if (flags & ~(uint32_t)(KVP_ROPE_QUERY | KVP_CONTINUE | KVP_FORCE_SIMPLE | KVP_PRECISE_QK)) return fail(ctx, KVP_ERR_INVALID, "segment_mass: unknown flags");
    const kvp_assembly_host &as = ctx->slots[slot];
    if (ctx->shape.group > 8) return fail(ctx, KVP_ERR_UNSUPPORTED, "segment_mass: more than 8 q heads per kv head");
    if ((int)as.appended.size() != ctx->cfg.n_layers || as.appended[layer] < q_len)
        return fail(ctx, KVP_ERR_STATE, "segment_mass: call kvp_query_prefill for this layer first");
    if (as.flags & KVP_MATERIALIZE) return fail(ctx, KVP_ERR_UNSUPPORTED, "segment_mass: materialised assemblies keep no segment rows apart");
    int max_seg = 0;
    for (int b = 0; b < as.batch; ++b) max_seg = std::max(max_seg, as.items[b].seg_end - as.items[b].seg_begin);
    if (n_cols <= max_seg) return fail(ctx, KVP_ERR_CAPACITY, "segment_mass: n_cols %d <= %d segments", n_cols, max_seg);
    KVP_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    if (as.waits_loads) KVP_CUDA(ctx, cudaStreamWaitEvent((cudaStream_t)stream, ctx->load_done[layer], 0));
    const void *q_used = (flags & KVP_ROPE_QUERY) ? (const void *)ctx->q_scratch : q;
    KVP_CUDA(ctx, kvp_launch_segment_mass(ctx->shape, plan_dev(ctx, slot), as.batch, q_len, as.appended[layer] - q_len, layer,
                                          q_used, lse, ctx->pool_k, ctx->slot_k[slot], mass, n_cols, (cudaStream_t)stream));
    return KVP_OK;
}

int32_t kvp_status_word(kvp_ctx *ctx, int32_t *device_status)
{
    if (!ctx || !device_status) return KVP_ERR_INVALID;
    if (ctx->host_only) { *device_status = 0; return KVP_OK; }
    KVP_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    KVP_CUDA(ctx, cudaDeviceSynchronize());
    KVP_CUDA(ctx, cudaMemcpy(device_status, ctx->status_dev, 4, cudaMemcpyDeviceToHost));
    if (*device_status != 0) {
        KVP_CUDA(ctx, cudaMemset(ctx->status_dev, 0, 4));
        return fail(ctx, KVP_ERR_TIMEOUT, "device-side bounded wait ran out (code %d)", *device_status);
    }
    return KVP_OK;
}

int32_t kvp_last_launch(kvp_ctx *ctx, int32_t *kind, int32_t *ctas, int32_t *splits, int32_t *launches)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (kind) *kind = ctx->last_kind;
    if (ctas) *ctas = ctx->last_ctas;
    if (splits) *splits = ctx->last_splits;
    if (launches) *launches = ctx->last_launches;
    return KVP_OK;
}

int32_t kvp_export_schedule(kvp_ctx *ctx, int32_t assembly_id, int32_t q_len, int32_t *cta_begin, int32_t cta_cap,
                            int32_t *works, int32_t work_cap, int32_t *merges, int32_t merge_cap, int32_t *counts)
{
    if (!ctx || !counts) return KVP_ERR_INVALID;
    const int slot = find_slot(ctx, assembly_id);
    if (slot < 0) return fail(ctx, KVP_ERR_NOT_FOUND, "export_schedule: unknown assembly %d", assembly_id);
    if (q_len <= 0 || q_len > ctx->cfg.max_query_tokens) return fail(ctx, KVP_ERR_INVALID, "export_schedule: bad q_len");
    schedule_t sc;
    const int32_t rc = plan_schedule(ctx, ctx->slots[slot], 0, q_len, 0, nullptr, 0, sc);
    if (rc != KVP_OK) return rc;
    counts[0] = sc.n_ctas;
    counts[1] = (int32_t)sc.works.size();
    counts[2] = (int32_t)sc.merges.size();
    counts[3] = sc.n_slots;
    if ((cta_begin && cta_cap < sc.n_ctas + 1) || (works && work_cap < counts[1]) || (merges && merge_cap < counts[2]))
        return fail(ctx, KVP_ERR_CAPACITY, "export_schedule: output arrays too small");
    if (cta_begin) memcpy(cta_begin, sc.cta_begin.data(), 4 * sc.cta_begin.size());
    if (works)
        for (size_t i = 0; i < sc.works.size(); ++i) memcpy(works + 8 * i, &sc.works[i], 32);     // the 8 documented ints of a piece
    if (merges) memcpy(merges, sc.merges.data(), sizeof(kvp_merge_item) * sc.merges.size());
    return KVP_OK;
}

int32_t kvp_kernel_times(kvp_ctx *ctx, int32_t which, float *ms, int32_t cap, int32_t *n)
{
    if (!ctx || !n || which < 0 || which > 1 || (cap > 0 && !ms)) return KVP_ERR_INVALID;
    if (ctx->host_only) return fail(ctx, KVP_ERR_STATE, "kernel_times: host-only context");
    const int cnt = std::min(cap, ctx->tev_n[which]);
    for (int i = 0; i < cnt; ++i) {
        KVP_CUDA(ctx, cudaEventSynchronize(ctx->tev[which][1][i]));
        KVP_CUDA(ctx, cudaEventElapsedTime(&ms[i], ctx->tev[which][0][i], ctx->tev[which][1][i]));
    }
    *n = cnt;
    ctx->tev_n[which] = 0;
    return KVP_OK;
}

int32_t kvp_tune(kvp_ctx *ctx, int32_t key, int32_t value)
{
    if (!ctx) return KVP_ERR_INVALID;
    if (key == KVP_TUNE_SPLIT_TARGET_CTAS || key == KVP_TUNE_FORCE_SPLITS) {
        (key == KVP_TUNE_SPLIT_TARGET_CTAS ? ctx->split_target_ctas : ctx->force_splits) = value;
        for (kvp_assembly_host &as : ctx->slots) as.sched.clear();       // work lists are rebuilt on next use
    }
    else if (key == KVP_TUNE_FUSED_APPEND) ctx->fused_append = value != 0;
    else if (key == KVP_TUNE_TIME_KERNELS) {
        ctx->time_kernels = std::max(0, value);
        ctx->tev_n[0] = ctx->tev_n[1] = 0;
        ctx->tev_seen[0] = ctx->tev_seen[1] = 0;
    }
    else return fail(ctx, KVP_ERR_INVALID, "tune: unknown key %d", key);
    return KVP_OK;
}

}  // extern "C"
