// bf16 composed-cache attention for sm_100a: TMA-staged K/V tiles, tcgen05 MMA with TMEM accumulators,
// two query streams per CTA so that the tensor pipe works on one stream while the other is in softmax.
//
// A persistent CTA (one per SM) walks a host-built list of work pieces.  A piece is a contiguous range
// of the key tiles of one unit (<= 256 packed query rows - query token i, head-in-group - of one
// request and kv head).  Key tiles are numbered per unit: the causal tiles of the query's own keys
// first, then the prefix tiles of the plan (staged adapter rows, then documents read in place from
// the pool).  The two streams of a piece are
//   mode 0: query rows [0,128) and [128,256) of the unit, both visiting every key tile of the range;
//   mode 1: the same 128 query rows twice, stream s visiting tiles lo+s, lo+s+2, ...; the two partial
//           results are combined inside the CTA at the end of the piece.
//
//   warps 0-3 / 4-7   softmax of stream 0 / 1: one thread per query row.  S = Q K^T arrives in TMEM;
//                     the thread takes the row max, forms p = exp2((s - m) * scale*log2e), sums it in
//                     fp32, writes P as bf16 back into TMEM over S, and rescales O in TMEM when the
//                     running max moved by more than 2^8.  Both warpgroups run the same compact code
//                     (rolled 32-column chunk loops) so that it stays in the instruction cache.  At the end of a piece it normalises O and
//                     writes the output rows (or an fp32 partial when the unit's keys are split).
//   warps 8-11        Q producer.  Documents keep the keys they were cached with: instead of rotating
//                     every key by Delta (Eq. 1) the 128-row Q tile of a stream is counter-rotated by
//                     -Delta once per document, which leaves every score q.k unchanged.  Each stream has
//                     two Q buffers, so the next document's Q is written while the current one is in use.
//   warp 12           MMA issuer and TMEM owner.  Per stream and step: O += P V of the previous tile,
//                     then S = Q K^T of the next one; the two streams alternate.
//   warp 13           TMA producer: K and V tiles into a 3-stage ring (two 64-column boxes each,
//                     128-byte swizzle), in the order the MMA warp consumes them.
//   warps 14-15       with tail_direct: copy the query block's K/V rows behind the prefix (the append).
//
// Every mbarrier wait is bounded: when it runs out the CTA records a code in the status word, drains
// what it has in flight, frees TMEM and returns.
#include <cuda_bf16.h>

#include <type_traits>

#include "kvp_internal.h"

namespace {

constexpr int kStages = 3;
constexpr int kTileBytes = KVP_TILE_KEYS * 128 * 2;      // 32 KB: 128 rows x 128 bf16
constexpr int kHalfBytes = kTileBytes / 2;               // one 64-column box
constexpr int kThreads = 512;
constexpr int kTmemCols = 512;
constexpr uint32_t kColS = 0, kColO = 256;               // + 128 * stream

constexpr int kOffQ = 0;                                  // two 32 KB rotated-Q buffers per stream: [stream][epoch & 1]
constexpr int kOffRing = 4 * kTileBytes;                  // kStages x 32 KB
constexpr int kOffBar = kOffRing + kStages * kTileBytes;
constexpr int kOffMl = kOffBar + 256;                     // float2[128]: stream 1's (max, sum) in mode 1
constexpr int kSmemBytes = kOffMl + 1024 + 1024;          // + alignment slack


enum BarIdx { kKvFull = 0, kKvEmpty = kStages, kQFull = 2 * kStages, kQFree = kQFull + 4, kSFull = kQFree + 4,   // Q: [2 * stream + buffer]
              kPFull = kSFull + 2, kOFull = kPFull + 2, kOFree = kOFull + 2, kMlFull = kOFree + 2, kDrain = kMlFull + 1,
              kNumBars = kDrain + 1 };
static_assert(8 * kNumBars + 8 <= 256, "barrier block");

struct Params {
    kvp_plan_dev plan;
    int q_len, q_pos0, layer, n_q, n_kv, group, pairing;      // q_pos0: tail rows appended by earlier calls
    float scale, scale_log2;
    const int32_t *cta_begin;
    const kvp_work *works;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    float *lse;
    float *partial_o;
    float2 *partial_ml;
    int32_t *status;
    // tail_direct: the query block's tiles come from k_new / v_new ([batch][q_len][Hkv][d], through their own
    // tensor maps) and the kernel copies those rows into the workspace rows (the append) itself
    int tail_direct;
    // precise: the counter-rotated query is kept as value + rounding remainder (two bf16 tiles per stream, one
    // epoch buffer instead of two) and Q K^T of a rotated tile takes both
    int precise;
    // l2_prefetch: the K/V tiles of a unit are read by at most two units of the launch, i.e. they come from DRAM
    // rather than from L2: the TMA warp then asks L2 for each tile a few loads before it fetches it
    int l2_prefetch;
    const uint4 *k_new, *v_new;
    uint4 *ws_k, *ws_v;
    long long ws_rows;
};

// ---- PTX wrappers ---------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false when another role has aborted or after ~2 s (then the status word and
// the CTA's abort flag are set).  `code` identifies the wait.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                            int32_t *status, int code)
{
    const uint64_t t0 = global_ns();
    uint32_t it = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++it & 63u) == 0) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > 2000000000ull) {
                atomicCAS(status, 0, code);
                *abort_flag = 1;
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          int32_t *status, int code)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status, code);
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, int w, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// The MMA warp runs convergently; one elected lane issues each tcgen05.mma / tcgen05.commit.
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile(
        "{\n\t.reg .pred e;\n\telect.sync _|e, 0xffffffff;\n\t"
        "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 64-bit shared-memory matrix descriptors are kept as a constant high word and a low word (start
// address and leading-dimension offset, in 16-byte units) that advances by an immediate per K-step.
__device__ __forceinline__ uint64_t desc64(uint32_t lo, uint32_t hi)
{
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}
// D[tmem] (+)= A[smem] * B[smem]
template <int ACC>
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p, e;\n\telect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d), "l"(a), "l"(b), "r"(idesc), "n"(ACC)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p, e;\n\telect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc)
        : "memory");
}
template <int ACC>
__device__ __forceinline__ void mma_ts_c(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p, e;\n\telect.sync _|e, 0xffffffff;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d), "r"(a), "l"(b), "r"(idesc), "n"(ACC)
        : "memory");
}

#define KVP_R8(r, o) "=r"(r[o]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), "=r"(r[o + 7])
#define KVP_W8(r, o) "r"(r[o]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]), "r"(r[o + 7])

// 32 TMEM lanes (this warp's) x 32 consecutive 32-bit columns -> 32 registers per thread
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t *r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : KVP_R8(r, 0), KVP_R8(r, 8), KVP_R8(r, 16), KVP_R8(r, 24)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t *r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), KVP_W8(r, 0), KVP_W8(r, 8), KVP_W8(r, 16), KVP_W8(r, 24)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t *r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), KVP_W8(r, 0), KVP_W8(r, 8)
        : "memory");
}

// tcgen05.ld fills its destination registers asynchronously, until tcgen05.wait::ld.  This empty
// statement, placed after the wait, makes the compiler treat the 32 registers as written there, so that
// no copy of them taken between the load and the wait can be used afterwards.
#define KVP_RW8(r, o) "+r"(r[o]), "+r"(r[o + 1]), "+r"(r[o + 2]), "+r"(r[o + 3]), "+r"(r[o + 4]), "+r"(r[o + 5]), "+r"(r[o + 6]), "+r"(r[o + 7])
__device__ __forceinline__ void landed32(uint32_t *r)
{
    asm volatile("" : KVP_RW8(r, 0), KVP_RW8(r, 8), KVP_RW8(r, 16), KVP_RW8(r, 24)::"memory");
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart.
//   K-major operand (Q, K): rows are 128-byte lines; the leading-dimension field is unused (1).
//   MN-major operand (V):   the second 64-column block lies `lbo_bytes` further on.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // stride 1024 B, sm_100 version, SWIZZLE_128B
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes)
{
    return ((addr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = n, A K-major, B K-major or MN-major.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, uint32_t b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// ---- work pieces and tiles ---------------------------------------------------------------------------

struct Work {
    int b, hk, row_base, mode, lo, n, slot0, slot1;
    int n_tail, tile_begin, tail_row0, plane;
    int steps0, steps1;
    int q_len;                 // query tokens of this request (the call's q_len unless the work record carries its own)
};

__device__ __forceinline__ Work load_work(const Params &p, int wi)
{
    const int4 *w4 = reinterpret_cast<const int4 *>(p.works + wi);
    const int4 a = __ldg(w4), c = __ldg(w4 + 1), e = __ldg(w4 + 2);
    Work w;
    w.b = a.x; w.hk = a.y; w.row_base = a.z; w.mode = a.w & 0xff;
    w.q_len = (a.w >> 8) ? (a.w >> 8) : p.q_len;
    w.lo = c.x; w.n = c.y; w.slot0 = c.z; w.slot1 = c.w;
    w.tile_begin = e.x;                                       // the plan item's entries, carried in the work record
    w.tail_row0 = e.y;
    const int n_rows = p.group * w.q_len;
    const int last = min(n_rows - 1, w.row_base + (w.mode ? KVP_TILE_ROWS : 2 * KVP_TILE_ROWS) - 1);
    w.n_tail = (p.q_pos0 + last / p.group) / KVP_TILE_KEYS + 1;
    w.plane = p.layer * p.n_kv + w.hk;
    w.steps0 = w.mode ? (w.n + 1) >> 1 : w.n;
    w.steps1 = w.mode ? w.n >> 1 : w.n;
    return w;
}

struct Tile {
    int row0, n_keys, src, rope, qoff;
};

// tile j of the unit's numbering
__device__ __forceinline__ Tile get_tile(const Params &p, const Work &w, int j)
{
    Tile t;
    if (j < w.n_tail) {
        t.row0 = p.tail_direct ? j * KVP_TILE_KEYS : w.tail_row0 + j * KVP_TILE_KEYS;
        t.n_keys = min(KVP_TILE_KEYS, p.q_pos0 + w.q_len - j * KVP_TILE_KEYS);
        t.src = p.tail_direct ? 2 : 1;               // 2: rows of the caller's k_new / v_new, by query token
        t.rope = 0;
        t.qoff = j * KVP_TILE_KEYS;
    } else {
        const int4 g = __ldg(reinterpret_cast<const int4 *>(p.plan.tiles + w.tile_begin + (j - w.n_tail)));
        t.row0 = g.x;
        t.n_keys = g.y & 0xFFFF;
        t.src = g.y >> 16;
        t.rope = g.z;
        t.qoff = -1;
    }
    return t;
}
// unit tile number of step k of stream s
__device__ __forceinline__ int stream_tile(const Work &w, int s, int k) { return w.lo + (w.mode ? 2 * k + s : k); }

// Position of a K (kv = 0) or V (kv = 1) tile, r-th of the piece, in the piece's load order.
//   mode 0: K0 V0 K1 V1 ...        mode 1: K0 K1 V0 K2 V1 K3 V2 ... V(n-1)
__device__ __forceinline__ int load_seq(int mode, int n, int r, int kv)
{
    if (mode == 0) return 2 * r + kv;
    if (kv == 0) return r == 0 ? 0 : 2 * r - 1;
    return r <= n - 2 ? 2 * r + 2 : 2 * n - 1;
}

// The Q producer (128 threads) writes one 128-row query tile, counter-rotated by the offset of rope-table row
// `rope` - q' = R(-Delta) q, which leaves q'.k = q.(R(Delta) k), Eq. 1 moved onto Q - into a rotated-Q buffer
// in the K-major 128-byte-swizzled layout (two 64-column halves of 128 rows x 128 bytes).  Thread t owns
// the 16-byte chunks c = t & 7 and c + 8 (the rotation partners when pairs are (i, i + 64)) of rows
// t >> 3, + 16, + 32, ...  The raw rows go to their place in the buffer by asynchronous copies, all in flight
// together (one memory round trip for the tile, eight threads per 128-byte line); the thread then rotates
// its own chunks in place.
// With `qrem` (precise mode) the remainders r - bf16(r) of the rotated values go, as bf16, to the same places of
// a second tile: q' = hi + rem to about 2^-17, so that the rounding of the re-based operand leaves the scores.
__device__ __forceinline__ void produce_q_tile(const Params &p, char *qbuf, char *qrem, int t, const __nv_bfloat16 *q_b, int hk,
                                               int row_base, int n_rows, int rope)
{
    const int c = t & 7, r0 = t >> 3;
    char *mine = qbuf + r0 * 128 + ((c ^ (r0 & 7)) << 4);                       // row & 7 == r0 & 7 for all of its rows
    float4 w4[4];
    if (rope != 0) {
        const float4 *cs = reinterpret_cast<const float4 *>(p.plan.rope + (size_t)rope * 64);   // (cos, sin) pairs
#pragma unroll
        for (int j = 0; j < 4; ++j)
            w4[j] = __ldg(p.pairing == 0 ? cs + c * 4 + j : cs + (c + 8 * (j >> 1)) * 2 + (j & 1));
    }
#pragma unroll 1
    for (int i = 0; i < 8; ++i) {
        const int r = row_base + r0 + 16 * i;
        char *lo = mine + i * (16 * 128);
        if (r < n_rows) {
            const uint4 *src = reinterpret_cast<const uint4 *>(q_b + ((long long)(r / p.group) * p.n_q + hk * p.group + r % p.group) * 128);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(lo)), "l"(src + c) : "memory");
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(lo + kHalfBytes)), "l"(src + c + 8) : "memory");
        } else {
            *reinterpret_cast<uint4 *>(lo) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4 *>(lo + kHalfBytes) = make_uint4(0, 0, 0, 0);
        }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (rope == 0) return;
    auto lo_f = [](uint32_t u) { return __uint_as_float(u << 16); };
    auto hi_f = [](uint32_t u) { return __uint_as_float(u & 0xffff0000u); };
#pragma unroll 1
    for (int i = 0; i < 8; ++i) {
        if (row_base + r0 + 16 * i >= n_rows) break;
        char *lo = mine + i * (16 * 128);
        uint4 qa = *reinterpret_cast<uint4 *>(lo), qb = *reinterpret_cast<uint4 *>(lo + kHalfBytes);
        uint32_t *a = reinterpret_cast<uint32_t *>(&qa);
        uint32_t *b = reinterpret_cast<uint32_t *>(&qb);
        uint4 ra, rb;                                            // remainders (precise mode)
        uint32_t *ar = reinterpret_cast<uint32_t *>(&ra);
        uint32_t *br = reinterpret_cast<uint32_t *>(&rb);
        // word = bf16 pair of (x, y); rem = bf16 pair of what the rounding of the word dropped
        auto put = [&](uint32_t &word, uint32_t &rem, float x, float y) {
            word = pack_bf16(x, y);
            rem = pack_bf16(x - lo_f(word), y - hi_f(word));
        };
        if (p.pairing == 0) {
            // pairs (i, i + 64): word j of chunk c holds elements 8c+2j, 8c+2j+1; partners in chunk c+8
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float4 w = w4[j];                          // cos, sin of pair 8c+2j; cos, sin of pair 8c+2j+1
                const float a0 = lo_f(a[j]), a1 = hi_f(a[j]), b0 = lo_f(b[j]), b1 = hi_f(b[j]);
                put(a[j], ar[j], a0 * w.x + b0 * w.y, a1 * w.z + b1 * w.w);     // R(-Delta): cos same, sin negated
                put(b[j], br[j], b0 * w.x - a0 * w.y, b1 * w.z - a1 * w.w);
            }
        } else {
            // pairs (2i, 2i+1): one word each; chunk c holds pairs 4c..4c+3 (w4[0], w4[1]), chunk c+8 w4[2], w4[3]
#pragma unroll
            for (int j = 0; j < 4; j += 2) {
                float4 w = w4[j >> 1];
                float x0 = lo_f(a[j]), y0 = hi_f(a[j]), x1 = lo_f(a[j + 1]), y1 = hi_f(a[j + 1]);
                put(a[j], ar[j], x0 * w.x + y0 * w.y, y0 * w.x - x0 * w.y);
                put(a[j + 1], ar[j + 1], x1 * w.z + y1 * w.w, y1 * w.z - x1 * w.w);
                w = w4[2 + (j >> 1)];
                x0 = lo_f(b[j]); y0 = hi_f(b[j]); x1 = lo_f(b[j + 1]); y1 = hi_f(b[j + 1]);
                put(b[j], br[j], x0 * w.x + y0 * w.y, y0 * w.x - x0 * w.y);
                put(b[j + 1], br[j + 1], x1 * w.z + y1 * w.w, y1 * w.z - x1 * w.w);
            }
        }
        *reinterpret_cast<uint4 *>(lo) = qa;
        *reinterpret_cast<uint4 *>(lo + kHalfBytes) = qb;
        if (qrem != nullptr) {
            char *rl = qrem + (lo - qbuf);
            *reinterpret_cast<uint4 *>(rl) = ra;
            *reinterpret_cast<uint4 *>(rl + kHalfBytes) = rb;
        }
    }
}

struct Cta {
    char *smem;
    uint32_t smem_base, bar0, tmem;
    volatile uint32_t *abort_flag;
    int item_begin, item_end;
    __device__ __forceinline__ uint32_t bar(int i) const { return bar0 + 8u * i; }
};

// ---- softmax / correction / epilogue of stream S -------------------------------------------------------
// One thread per query row.  S is read from TMEM in 32-column chunks, once; the chunk loop is rolled and
// shared by both streams so that the code stays resident in the instruction cache.
__device__ __forceinline__ float chunk_max(const uint32_t *v, float m)
{
    float m0 = m, m1 = m;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        m0 = fmax3(m0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
        m1 = fmax3(m1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
    }
    return fmaxf(m0, m1);
}
__device__ __forceinline__ void chunk_mask(uint32_t *v, int lim)
{
#pragma unroll
    for (int i = 0; i < 32; ++i)
        if (i >= lim) v[i] = 0xff800000u;                  // -inf
}
// ---- packed fp32 pairs (two lanes of the FMA pipe per instruction) --------------------------------------
__device__ __forceinline__ uint64_t pair(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpair(uint64_t r, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// p = exp2(s*c2 - mc) for 32 scores, packed as bf16 pairs into pk[16]; returns their fp32 sum.
// (Evaluating part of the exponentials by a polynomial on the FMA pipe was measured and lost: the
// extra issue slots cost more than the special-function unit saves.)
__device__ __forceinline__ float chunk_exp(const uint32_t *v, float c2, float mc, uint32_t *pk)
{
    const uint64_t c2p = pair(c2, c2), nmc = pair(-mc, -mc);
    uint64_t la = pair(0.f, 0.f), lb = pair(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        float x0, x1;
        unpair(fma2(pair(__uint_as_float(v[i]), __uint_as_float(v[i + 1])), c2p, nmc), x0, x1);
        const float p0 = ex2(x0), p1 = ex2(x1);
        if (i & 2) lb = add2(lb, pair(p0, p1)); else la = add2(la, pair(p0, p1));
        pk[i >> 1] = pack_bf16(p0, p1);
    }
    float s0, s1;
    unpair(add2(la, lb), s0, s1);
    return s0 + s1;
}

// Rare path of the softmax: the row's reference max moved up, so everything accumulated against the old
// one shrinks by alpha = 2^(old - new): O in TMEM (when a P V product has been accumulated) and the P
// chunks [0, n_chunks) of the current tile that were already written.  S of this step is complete, hence
// so is the P V product of the previous step: O is quiet.
__device__ __forceinline__ void rescale_row(uint32_t s_addr, uint32_t o_addr, float alpha, int n_chunks, bool with_o)
{
    uint32_t v[32];
    if (with_o) {
#pragma unroll 1
        for (int ch = 0; ch < 4; ++ch) {
            tmem_ld32(o_addr + ch * 32, v);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
            tmem_st32(o_addr + ch * 32, v);
        }
    }
    if (n_chunks > 0) tc_wait_st();                  // the P chunks this thread stored are read back below
#pragma unroll 1
    for (int ch = 0; ch < n_chunks; ++ch) {          // 16 columns of packed bf16 pairs per chunk
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
            "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
            : KVP_R8(v, 0), KVP_R8(v, 8)
            : "r"(s_addr + ch * 16)
            : "memory");
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; ++i)
            v[i] = pack_bf16(__uint_as_float(v[i] << 16) * alpha, __uint_as_float(v[i] & 0xffff0000u) * alpha);
        tmem_st16(s_addr + ch * 16, v);
    }
    tc_wait_st();
}

__device__ __forceinline__ void softmax_role(const Params &p, const Cta &c, const int S, const int t)
{
    const uint32_t lane_base = (uint32_t)((t >> 5) * 32) << 16;
    const uint32_t s_addr = c.tmem + lane_base + kColS + S * 128;
    const uint32_t o_addr = c.tmem + lane_base + kColO + S * 128;
    const float c2 = p.scale_log2;
    float2 *ml_smem = reinterpret_cast<float2 *>(c.smem + kOffMl);
    uint32_t nS = 0, nO = 0, nMl = 0;
    bool ok = true;

    for (int wi = c.item_begin; wi < c.item_end && ok; ++wi) {
        const Work w = load_work(p, wi);
        const int steps = S == 0 ? w.steps0 : w.steps1;
        if (steps == 0) continue;
        const int n_rows = p.group * w.q_len;
        const int r = w.row_base + (w.mode == 0 ? S * KVP_TILE_ROWS : 0) + t;
        const bool valid = r < n_rows;
        const int qi = valid ? r / p.group : w.q_len - 1;
        const int h = w.hk * p.group + (valid ? r % p.group : 0);

        float m_ref = -1e30f, l = 0.f;
        Tile nxt = get_tile(p, w, stream_tile(w, S, 0));
#pragma unroll 1
        for (int k = 0; k < steps; ++k) {
            const Tile tl = nxt;
            if (k + 1 < steps) nxt = get_tile(p, w, stream_tile(w, S, k + 1));
            ok = mbar_wait(c.bar(kSFull + S), nS & 1, c.abort_flag, p.status, 30 + S);
            ++nS;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();

            const bool full = (tl.n_keys == KVP_TILE_KEYS) && (tl.qoff < 0);
            const int lim = tl.qoff < 0 ? tl.n_keys : min(tl.n_keys, p.q_pos0 + qi - tl.qoff + 1);       // visible keys: [0, lim)
            uint32_t va[32];

            // One pass over S: the exponentials use the reference max carried over from earlier tiles; each
            // 32-column chunk's own max is checked first, and only if it exceeds the reference by more than
            // 2^8 (first tile of a piece, or a rare jump) are l, O and the P chunks already written rescaled.
            // The exponentials of a chunk are formed optimistically against the current reference while its
            // max is reduced alongside; the check comes last, so the two dependency chains overlap.
            auto process = [&](uint32_t *v, int ch) {
                if (!full) chunk_mask(v, lim - ch * 32);
                uint32_t pk[16];
                const float cm = chunk_max(v, -INFINITY);
                float ls = chunk_exp(v, c2, m_ref * c2, pk);
                const bool need = (cm - m_ref) * c2 > 8.0f;
                if (__any_sync(0xffffffffu, need)) {
                    const float m_new = need ? cm : m_ref;
                    const float alpha = need ? ex2((m_ref - m_new) * c2) : 1.f;
                    rescale_row(s_addr, o_addr, alpha, ch, k > 0);
                    l *= alpha;
                    m_ref = m_new;
                    tmem_ld32(s_addr + ch * 32, v);             // this chunk's scores again (P so far lies below them)
                    tc_wait_ld();
                    landed32(v);
                    if (!full) chunk_mask(v, lim - ch * 32);
                    ls = chunk_exp(v, c2, m_ref * c2, pk);
                }
                tmem_st16(s_addr + ch * 16, pk);
                l += ls;
            };
            // a short tile (the end of a document, staged adapter rows) needs P only for the columns P V will read
            const int n_ch = full ? 4 : max(1, (tl.n_keys + 31) >> 5);
#pragma unroll 1
            for (int ch = 0; ch < n_ch; ++ch) {
                tmem_ld32(s_addr + ch * 32, va);
                tc_wait_ld();
                landed32(va);
                process(va, ch);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(c.bar(kPFull + S));
        }
        if (!ok) break;

        // ---- end of the piece: O of this stream is complete once its last P V has landed ----------
        ok = mbar_wait(c.bar(kOFull + S), nO & 1, c.abort_flag, p.status, 32 + S);
        ++nO;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();

        if (w.mode == 1 && S == 1) {
            ml_smem[t] = make_float2(m_ref, l);
            mbar_arrive(c.bar(kMlFull));         // stream 0's warpgroup combines and writes
            continue;
        }
        float w0 = 1.f, w1 = 0.f;
        const bool both = (w.mode == 1) && (w.steps1 > 0);
        if (both) {
            ok = mbar_wait(c.bar(kMlFull), nMl & 1, c.abort_flag, p.status, 34);
            ++nMl;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float2 o = ml_smem[t];
            const float M = fmaxf(m_ref, o.x);
            w0 = ex2((m_ref - M) * c2);
            w1 = ex2((o.x - M) * c2);
            l = w0 * l + w1 * o.y;
            m_ref = M;
        }
        const int slot = S == 0 ? w.slot0 : w.slot1;
        const bool direct = slot < 0;
        if (direct) {
            const float inv = 1.f / l;
            w0 *= inv;
            w1 *= inv;
        }
        // un-normalised (partial slot) or normalised (output rows) O = w0 O_s (+ w1 O_1)
        uint4 *orow_bf = (direct && valid) ? reinterpret_cast<uint4 *>(p.out + (((long long)w.b * p.q_len + qi) * p.n_q + h) * 128) : nullptr;
        // partial slot layout: [32 float4 columns][128 rows], so that a warp's store covers 512 contiguous bytes
        uint4 *orow_f = direct ? nullptr : reinterpret_cast<uint4 *>(p.partial_o) + (long long)slot * (32 * KVP_TILE_ROWS) + t;
#pragma unroll 1
        for (int ch = 0; ch < 4; ++ch) {
            uint32_t a[32];
            tmem_ld32(o_addr + ch * 32, a);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) a[i] = __float_as_uint(__uint_as_float(a[i]) * w0);
            if (both) {
                uint32_t b2[32];
                tmem_ld32(o_addr + 128 + ch * 32, b2);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) a[i] = __float_as_uint(fmaf(__uint_as_float(b2[i]), w1, __uint_as_float(a[i])));
            }
            if (orow_bf != nullptr) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 u;
                    u.x = pack_bf16(__uint_as_float(a[8 * i + 0]), __uint_as_float(a[8 * i + 1]));
                    u.y = pack_bf16(__uint_as_float(a[8 * i + 2]), __uint_as_float(a[8 * i + 3]));
                    u.z = pack_bf16(__uint_as_float(a[8 * i + 4]), __uint_as_float(a[8 * i + 5]));
                    u.w = pack_bf16(__uint_as_float(a[8 * i + 6]), __uint_as_float(a[8 * i + 7]));
                    orow_bf[ch * 4 + i] = u;
                }
            } else if (orow_f != nullptr) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    orow_f[(ch * 8 + i) * KVP_TILE_ROWS] = make_uint4(a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
            }
        }
        if (direct) {
            if (valid && p.lse != nullptr)
                p.lse[((long long)w.b * p.n_q + h) * p.q_len + qi] = m_ref * p.scale + logf(l);
        } else {
            p.partial_ml[(long long)slot * KVP_TILE_ROWS + t] = make_float2(m_ref, l);
        }
        tc_fence_before();
        mbar_arrive(c.bar(kOFree + S));
        if (both) mbar_arrive(c.bar(kOFree + 1));
    }
}

// ---- Q producer -----------------------------------------------------------------------------------------
__device__ __forceinline__ void producer_role(const Params &p, const Cta &c, const int t)
{
    uint32_t nEp0 = 0, nEp1 = 0;
    bool ok = true;
    for (int wi = c.item_begin; wi < c.item_end && ok; ++wi) {
        const Work w = load_work(p, wi);
        const int n_rows = p.group * w.q_len;
        const int max_steps = max(w.steps0, w.steps1);
        int prev0 = 0, prev1 = 0;
        auto produce = [&](int s, int rope, uint32_t &nEp) {
            // two buffers per stream taken in turn; in precise mode one (value, remainder) pair, rewritten once
            // the last Q K^T of the epoch before has run
            const int buf = p.precise ? 0 : (nEp & 1);
            const uint32_t back = p.precise ? 1u : 2u;      // the epoch that used this buffer last
            if (nEp >= back) {
                const uint32_t par = p.precise ? (nEp - 1) & 1 : ((nEp >> 1) - 1) & 1;
                ok = mbar_wait(c.bar(kQFree + 2 * s + buf), par, c.abort_flag, p.status, 40 + s);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) return;
            }
            char *qb = c.smem + kOffQ + (2 * s + buf) * kTileBytes;
            produce_q_tile(p, qb, p.precise ? qb + kTileBytes : nullptr, t, p.q + (long long)w.b * p.q_len * p.n_q * 128,
                           w.hk, w.row_base + (w.mode == 0 ? s * KVP_TILE_ROWS : 0), n_rows, rope);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(c.bar(kQFull + 2 * s + buf));
            ++nEp;
        };
        for (int k = 0; k < max_steps && ok; ++k) {
            if (k < w.steps0) {
                const int rope = get_tile(p, w, stream_tile(w, 0, k)).rope;
                if (k == 0 || rope != prev0) produce(0, rope, nEp0);
                prev0 = rope;
            }
            if (ok && k < w.steps1) {
                const int rope = get_tile(p, w, stream_tile(w, 1, k)).rope;
                if (k == 0 || rope != prev1) produce(1, rope, nEp1);
                prev1 = rope;
            }
        }
    }
}

// ---- append (the two spare warps) -------------------------------------------------------------------------------
// With tail_direct the attention reads the query block's K/V from the caller's tensors; the rows are also copied
// behind the prefix in the workspace, for later calls.  Every unit copies the query tokens whose first packed row
// it holds (for its kv head), in the piece that starts the unit, so the copy is spread over all CTAs; four
// 16-byte words of K and of V are in flight per thread.  Nothing in this launch waits for the copy.
__device__ __forceinline__ void append_role(const Params &p, const Cta &c, const int t)
{
    if (!p.tail_direct) return;
    for (int wi = c.item_begin; wi < c.item_end; ++wi) {
        const Work w = load_work(p, wi);
        if (w.lo != 0) continue;
        const int n_rows = p.group * w.q_len;
        const int row_end = min(n_rows, w.row_base + (w.mode ? KVP_TILE_ROWS : 2 * KVP_TILE_ROWS));
        const int i0 = (w.row_base + p.group - 1) / p.group, i1 = (row_end + p.group - 1) / p.group;   // tokens [i0, i1)
        const long long src0 = (((long long)w.b * p.q_len + i0) * p.n_kv + w.hk) * 16;     // 16-byte words; a token's row is 16
        const long long dst0 = ((long long)w.plane * p.ws_rows + w.tail_row0 + i0) * 16;
        const int n_words = (i1 - i0) * 16;
        for (int base = 0; base < n_words; base += 64 * 4) {
            uint4 k[4], v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = base + j * 64 + t;
                if (i < n_words) {
                    const long long src = src0 + (long long)(i >> 4) * p.n_kv * 16 + (i & 15);
                    k[j] = __ldg(p.k_new + src);
                    v[j] = __ldg(p.v_new + src);
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = base + j * 64 + t;
                if (i < n_words) {
                    p.ws_k[dst0 + i] = k[j];
                    p.ws_v[dst0 + i] = v[j];
                }
            }
        }
    }
}

// ---- TMA producer (whole warp; lane 0 issues) ----------------------------------------------------------
__device__ __forceinline__ void tma_role(const Params &p, const Cta &c, const int lane, const CUtensorMap *tm_pool_k,
                                         const CUtensorMap *tm_pool_v, const CUtensorMap *tm_ws_k,
                                         const CUtensorMap *tm_ws_v, const CUtensorMap *tm_knew,
                                         const CUtensorMap *tm_vnew)
{
    uint32_t ring_n = 0;                                   // loads issued before this piece
    bool ok = true;
    for (int wi = c.item_begin; wi < c.item_end && ok; ++wi) {
        const Work w = load_work(p, wi);
        const int n_loads = 2 * w.n;
        for (int q0 = 0; q0 < n_loads && ok; q0 += 32) {
            // lane i looks up the tile of load q0 + i
            const int q = q0 + lane;
            int r = 0, kv = 0;
            if (w.mode == 0) { r = q >> 1; kv = q & 1; }
            else if (q == 0) { r = 0; kv = 0; }
            else if (q == n_loads - 1) { r = w.n - 1; kv = 1; }
            else if (q & 1) { r = (q + 1) >> 1; kv = 0; }
            else { r = (q - 2) >> 1; kv = 1; }
            int row0 = 0, src = 0;
            if (q < n_loads) {
                const Tile tl = get_tile(p, w, w.lo + r);
                row0 = tl.row0;
                src = tl.src;
            }
            const int cnt = min(32, n_loads - q0);
            for (int i = 0; i < cnt && ok; ++i) {
                const int row0_i = __shfl_sync(0xffffffffu, row0, i);
                const int src_i = __shfl_sync(0xffffffffu, src, i);
                const int kv_i = __shfl_sync(0xffffffffu, kv, i);
                if (p.l2_prefetch && w.mode == 0) {      // tiles that come from DRAM: ask L2 for the one four loads ahead
                    constexpr int KVP_L2_PREFETCH = 4;
                    const int j = min(i + KVP_L2_PREFETCH, 31);
                    const int row0_j = __shfl_sync(0xffffffffu, row0, j);
                    const int src_j = __shfl_sync(0xffffffffu, src, j);
                    const int kv_j = __shfl_sync(0xffffffffu, kv, j);
                    if (lane == 0 && i + KVP_L2_PREFETCH < cnt && src_j != 2) {
                        const CUtensorMap *tm = src_j == 0 ? (kv_j ? tm_pool_v : tm_pool_k) : (kv_j ? tm_ws_v : tm_ws_k);
                        asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(tm), "r"(0), "r"(row0_j), "r"(w.plane) : "memory");
                        asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(tm), "r"(64), "r"(row0_j), "r"(w.plane) : "memory");
                    }
                }
                if (lane == 0) {
                    const uint32_t g = ring_n + (uint32_t)(q0 + i);
                    const uint32_t stage = g % kStages, use = g / kStages;
                    if (use > 0) ok = mbar_wait(c.bar(kKvEmpty + stage), (use - 1) & 1, c.abort_flag, p.status, 10 + stage);
                    if (ok) {
                        const uint32_t dst = c.smem_base + kOffRing + stage * kTileBytes;
                        mbar_expect_tx(c.bar(kKvFull + stage), kTileBytes);
                        if (src_i == 2) {
                            const CUtensorMap *tm = kv_i ? tm_vnew : tm_knew;
                            tma_load_4d(dst, tm, 0, w.hk, row0_i, w.b, c.bar(kKvFull + stage));
                            tma_load_4d(dst + kHalfBytes, tm, 64, w.hk, row0_i, w.b, c.bar(kKvFull + stage));
                        } else {
                            const CUtensorMap *tm = src_i == 0 ? (kv_i ? tm_pool_v : tm_pool_k) : (kv_i ? tm_ws_v : tm_ws_k);
                            tma_load_3d(dst, tm, 0, row0_i, w.plane, c.bar(kKvFull + stage));
                            tma_load_3d(dst + kHalfBytes, tm, 64, row0_i, w.plane, c.bar(kKvFull + stage));
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            }
        }
        ring_n += (uint32_t)n_loads;
    }
}

// ---- MMA issuer (whole warp, convergent; one elected lane issues) ----------------------------------------------------------------------------
struct MmaStream {
    uint32_t nP, nEpoch, nItems, qbuf;
    int prev_rope, prev_keys;
    Tile cur, nxt;
};

__device__ __forceinline__ void mma_role(const Params &p, const Cta &c)
{
    const uint32_t idesc_pv = instr_desc(128, 1);
    MmaStream st[2];
    st[0].nP = st[0].nEpoch = st[0].nItems = st[0].qbuf = 0;
    st[1].nP = st[1].nEpoch = st[1].nItems = st[1].qbuf = 0;
    uint32_t ring_n = 0;
    bool ok = true;

    // ---- S_s = Q_s K^T of step k of piece wq (whose loads start at ring position `base`) ----------------
    auto issue_qk = [&](auto s_c, const Work &wq, uint32_t base, int k) {
        constexpr int s = decltype(s_c)::value;
        MmaStream &ms = st[s];
        const int n_steps = s == 0 ? wq.steps0 : wq.steps1;
        const bool shared_stage = (wq.mode == 0);                 // mode 0: both streams read the same K/V stage
        if (k == 0) {
            ms.prev_rope = 0;
            ms.cur = get_tile(p, wq, stream_tile(wq, s, 0));
            ms.nxt = n_steps > 1 ? get_tile(p, wq, stream_tile(wq, s, 1)) : ms.cur;
        }
        const Tile tl = ms.cur;
        if (k == 0 || tl.rope != ms.prev_rope) {                  // first tile of a document: its own Q buffer
            ms.qbuf = p.precise ? 0 : (ms.nEpoch & 1);
            ok = mbar_wait(c.bar(kQFull + 2 * s + ms.qbuf), (p.precise ? ms.nEpoch : ms.nEpoch >> 1) & 1, c.abort_flag, p.status, 20 + s);
            ++ms.nEpoch;
        }
        const int r = wq.mode ? 2 * k + s : k;
        const uint32_t g = base + (uint32_t)load_seq(wq.mode, wq.n, r, 0);
        const uint32_t stage = g % kStages, par = (g / kStages) & 1;
        if (ok && !(shared_stage && s == 1)) ok = mbar_wait(c.bar(kKvFull + stage), par, c.abort_flag, p.status, 22);
        ok = __all_sync(0xffffffffu, ok);                         // the lanes stay together
        if (!ok) return;
        tc_fence_after();
        const uint32_t n16 = max(16u, (uint32_t)(tl.n_keys + 15) & ~15u);
        const uint32_t idesc = instr_desc(n16, 0);
        const uint32_t q_lo = desc_lo(c.smem_base + kOffQ + (2 * s + ms.qbuf) * kTileBytes, 16);
        const uint32_t k_lo = desc_lo(c.smem_base + kOffRing + stage * kTileBytes, 16);
        const uint32_t d = c.tmem + kColS + s * 128;
        mma_ss<0>(d, desc64(q_lo, kDescHi), desc64(k_lo, kDescHi), idesc);
#pragma unroll
        for (int kk = 1; kk < 8; ++kk) {                         // 16 columns per step: 32 bytes, second half 16 KB on
            constexpr uint32_t kHalf16 = kHalfBytes >> 4;
            const uint32_t off = (kk >> 2) * kHalf16 + (kk & 3) * 2;
            mma_ss<1>(d, desc64(q_lo + off, kDescHi), desc64(k_lo + off, kDescHi), idesc);
        }
        if (p.precise && tl.rope != 0) {                         // + (rounding remainder of the rotated Q) K^T
            constexpr uint32_t kRem16 = kTileBytes >> 4;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                constexpr uint32_t kHalf16 = kHalfBytes >> 4;
                const uint32_t off = (kk >> 2) * kHalf16 + (kk & 3) * 2;
                mma_ss<1>(d, desc64(q_lo + kRem16 + off, kDescHi), desc64(k_lo + off, kDescHi), idesc);
            }
        }
        tc_commit(c.bar(kSFull + s));
        if (!shared_stage || s == 1) tc_commit(c.bar(kKvEmpty + stage));
        const bool last = (k + 1 == n_steps) || (ms.nxt.rope != tl.rope);
        if (last) tc_commit(c.bar(kQFree + 2 * s + ms.qbuf));
        ms.prev_rope = tl.rope;
        ms.prev_keys = tl.n_keys;
        ms.cur = ms.nxt;
        if (k + 2 < n_steps) ms.nxt = get_tile(p, wq, stream_tile(wq, s, k + 2));
    };

    // ---- a piece in mode 0: both streams take every tile; loads arrive K(0) V(0) K(1) V(1) ... -----------------
    // This is the tensor-bound path, and the issuing warp's own instruction time is what bounds it, so
    // the loop is kept short: tile facts (key count, document) are fetched 32 tiles at a time, one per
    // lane, and handed round by shuffle; ring stages advance incrementally; all waits of a block come
    // first, with one vote and one fence.
    const int lane = threadIdx.x & 31;
    auto piece_mode0 = [&](const Work &w) {
        const int n = w.n;
        uint32_t stK = ring_n % kStages, parK = (ring_n / kStages) & 1;                 // K(k), used at step k
        uint32_t stV = (ring_n + 1) % kStages, parV = ((ring_n + 1) / kStages) & 1;     // V(k - 1), used at step k
        auto advance = [](uint32_t &st_, uint32_t &par_) {                              // two loads further on
            if (st_ == 0) st_ = 2; else { st_ -= 1; par_ ^= 1; }
        };
        int b0 = 0, nk_l = 0, rope_l = 0;
        auto refill = [&](int from) {
            b0 = from;
            if (from + lane < n) {
                const Tile t = get_tile(p, w, w.lo + from + lane);
                nk_l = t.n_keys;
                rope_l = t.rope;
            }
        };
        refill(0);
        int prev_nk = 0, prev_rope = 0;
        for (int k = 0; k <= n && ok; ++k) {
            if (k - b0 == 31) refill(k);                          // tile k + 1 stays inside the batch
            const int nk = __shfl_sync(0xffffffffu, nk_l, k - b0);
            const int rope = __shfl_sync(0xffffffffu, rope_l, k - b0);
            const int rope_n = __shfl_sync(0xffffffffu, rope_l, (k + 1 - b0) & 31);
            const bool newq = (k == 0) || rope != prev_rope;      // first tile of a document: its own Q buffer
            const bool lastq = (k + 1 >= n) || rope_n != rope;
            auto step = [&](auto s_c) {
                constexpr int s = decltype(s_c)::value;
                MmaStream &ms = st[s];
                // ---- waits of the block ---------------------------------------------------------
                if (s == 0) {                                 // the tiles first: they land while P is being formed
                    if (k >= 1) ok = mbar_wait(c.bar(kKvFull + stV), parV, c.abort_flag, p.status, 23);
                    if (k < n && ok) ok = mbar_wait(c.bar(kKvFull + stK), parK, c.abort_flag, p.status, 22);
                }
                if (k >= 1) {
                    if (ok) ok = mbar_wait(c.bar(kPFull + s), ms.nP & 1, c.abort_flag, p.status, 24 + s);
                    ++ms.nP;
                    if (ok && k == 1 && ms.nItems > 0)
                        ok = mbar_wait(c.bar(kOFree + s), (ms.nItems - 1) & 1, c.abort_flag, p.status, 26 + s);
                }
                if (k < n) {
                    if (newq) {
                        ms.qbuf = p.precise ? 0 : (ms.nEpoch & 1);
                        if (ok) ok = mbar_wait(c.bar(kQFull + 2 * s + ms.qbuf), (p.precise ? ms.nEpoch : ms.nEpoch >> 1) & 1, c.abort_flag, p.status, 20 + s);
                        ++ms.nEpoch;
                    }
                }
                ok = __all_sync(0xffffffffu, ok);                 // the lanes stay together
                if (!ok) return;
                tc_fence_after();
                if (k >= 1) {
                    // ---- O_s += P_s V of step k-1 ---------------------------------------------------
                    const uint32_t v_lo = desc_lo(c.smem_base + kOffRing + stV * kTileBytes, kHalfBytes);
                    const uint32_t pa = c.tmem + kColS + s * 128;
                    const uint32_t oa = c.tmem + kColO + s * 128;
                    if (prev_nk == KVP_TILE_KEYS && k > 1) {
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)           // 16 keys per step: P advances 8 columns, V 2048 bytes
                            mma_ts_c<1>(oa, pa + kk * 8, desc64(v_lo + kk * 128, kDescHi), idesc_pv);
                    } else {
                        const int ksteps = max(1, (prev_nk + 15) >> 4);    // an empty tile still initialises O (P = 0)
                        for (int kk = 0; kk < ksteps; ++kk)
                            mma_ts(oa, pa + kk * 8, desc64(v_lo + kk * 128, kDescHi), idesc_pv, (k > 1 || kk > 0));
                    }
                    if (s == 1) tc_commit(c.bar(kKvEmpty + stV));
                    if (k == n) {
                        tc_commit(c.bar(kOFull + s));
                        ++ms.nItems;
                    }
                }
                if (k < n) {
                    // ---- S_s = Q_s K^T of step k ----------------------------------------------------
                    const uint32_t n16 = max(16u, (uint32_t)(nk + 15) & ~15u);   
                    const uint32_t idesc = instr_desc(n16, 0);
                    const uint32_t q_lo = desc_lo(c.smem_base + kOffQ + (2 * s + ms.qbuf) * kTileBytes, 16);
                    const uint32_t k_lo = desc_lo(c.smem_base + kOffRing + stK * kTileBytes, 16);
                    const uint32_t d = c.tmem + kColS + s * 128;
                    mma_ss<0>(d, desc64(q_lo, kDescHi), desc64(k_lo, kDescHi), idesc);
#pragma unroll
                    for (int kk = 1; kk < 8; ++kk) {             // 16 columns per step: 32 bytes, second half 16 KB on
                        constexpr uint32_t kHalf16 = kHalfBytes >> 4;
                        const uint32_t off = (kk >> 2) * kHalf16 + (kk & 3) * 2;
                        mma_ss<1>(d, desc64(q_lo + off, kDescHi), desc64(k_lo + off, kDescHi), idesc);
                    }
                    if (p.precise && rope != 0) {                // + (rounding remainder of the rotated Q) K^T
                        constexpr uint32_t kRem16 = kTileBytes >> 4;
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            constexpr uint32_t kHalf16 = kHalfBytes >> 4;
                            const uint32_t off = (kk >> 2) * kHalf16 + (kk & 3) * 2;
                            mma_ss<1>(d, desc64(q_lo + kRem16 + off, kDescHi), desc64(k_lo + off, kDescHi), idesc);
                        }
                    }
                    tc_commit(c.bar(kSFull + s));
                    if (s == 1) tc_commit(c.bar(kKvEmpty + stK));
                    if (lastq) tc_commit(c.bar(kQFree + 2 * s + ms.qbuf));
                }
            };
            step(std::integral_constant<int, 0>{});
            if (ok) step(std::integral_constant<int, 1>{});
            if (k >= 1) advance(stV, parV);
            if (k < n) advance(stK, parK);
            prev_nk = nk;
            prev_rope = rope;
        }
    };

    for (int wi = c.item_begin; wi < c.item_end && ok; ++wi) {
        const Work w = load_work(p, wi);
        if (w.mode == 0) {
            piece_mode0(w);
            ring_n += 2u * (uint32_t)w.n;
            continue;
        }
        const int steps[2] = {w.steps0, w.steps1};
        const int max_steps = max(w.steps0, w.steps1);
        auto block = [&](auto s_c, int k) {
            constexpr int s = decltype(s_c)::value;
            MmaStream &ms = st[s];
            const bool shared_stage = (w.mode == 0);
            if (k >= 1 && k <= steps[s]) {
                // ---- O_s += P_s V of step k-1 -------------------------------------------------------
                const int r = w.mode ? 2 * (k - 1) + s : k - 1;
                const uint32_t g = ring_n + (uint32_t)load_seq(w.mode, w.n, r, 1);
                const uint32_t stage = g % kStages, par = (g / kStages) & 1;
                if (!(shared_stage && s == 1)) ok = mbar_wait(c.bar(kKvFull + stage), par, c.abort_flag, p.status, 23);
                if (ok) ok = mbar_wait(c.bar(kPFull + s), ms.nP & 1, c.abort_flag, p.status, 24 + s);
                ++ms.nP;
                if (ok && k == 1 && ms.nItems > 0)
                    ok = mbar_wait(c.bar(kOFree + s), (ms.nItems - 1) & 1, c.abort_flag, p.status, 26 + s);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) return;
                tc_fence_after();
                const uint32_t v_lo = desc_lo(c.smem_base + kOffRing + stage * kTileBytes, kHalfBytes);
                const uint32_t pa = c.tmem + kColS + s * 128;
                const uint32_t oa = c.tmem + kColO + s * 128;
                if (ms.prev_keys == KVP_TILE_KEYS && k > 1) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)               // 16 keys per step: P advances 8 columns, V 2048 bytes
                        mma_ts_c<1>(oa, pa + kk * 8, desc64(v_lo + kk * 128, kDescHi), idesc_pv);
                } else {
                    const int ksteps = max(1, (ms.prev_keys + 15) >> 4);   // an empty tile still initialises O (P = 0)
                    for (int kk = 0; kk < ksteps; ++kk)
                        mma_ts(oa, pa + kk * 8, desc64(v_lo + kk * 128, kDescHi), idesc_pv, (k > 1 || kk > 0));
                }
                if (!shared_stage || s == 1) tc_commit(c.bar(kKvEmpty + stage));
                if (k == steps[s]) {
                    tc_commit(c.bar(kOFull + s));
                    ++ms.nItems;
                }
            }
            if (k < steps[s]) issue_qk(s_c, w, ring_n, k);
        };
        for (int k = 0; k <= max_steps && ok; ++k) {
            block(std::integral_constant<int, 0>{}, k);
            if (ok) block(std::integral_constant<int, 1>{}, k);
        }
        ring_n += 2u * (uint32_t)w.n;
    }
    __syncwarp();
    if (!ok) {                      // drain whatever was issued before giving TMEM back
        tc_commit(c.bar(kDrain));
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(c.bar(kDrain), 0) && global_ns() - t0 < 100000000ull) {}
    }
}

__global__ void __launch_bounds__(kThreads, 1)
attn_sm100_kernel(const __grid_constant__ CUtensorMap tm_pool_k, const __grid_constant__ CUtensorMap tm_pool_v,
                  const __grid_constant__ CUtensorMap tm_ws_k, const __grid_constant__ CUtensorMap tm_ws_v,
                  const __grid_constant__ CUtensorMap tm_knew, const __grid_constant__ CUtensorMap tm_vnew,
                  const Params p)
{
    extern __shared__ char smem_raw[];
    Cta c;
    c.smem = reinterpret_cast<char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    c.smem_base = smem_u32(c.smem);
    c.bar0 = c.smem_base + kOffBar;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(c.smem + kOffBar + 8 * kNumBars);
    c.abort_flag = tmem_slot + 1;
    c.item_begin = __ldg(p.cta_begin + blockIdx.x);
    c.item_end = __ldg(p.cta_begin + blockIdx.x + 1);
    if (c.item_begin >= c.item_end) return;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(c.bar(kKvFull + s), 1);
            mbar_init(c.bar(kKvEmpty + s), 1);
        }
        for (int s = 0; s < 4; ++s) {
            mbar_init(c.bar(kQFull + s), 128);
            mbar_init(c.bar(kQFree + s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(c.bar(kSFull + s), 1);
            mbar_init(c.bar(kPFull + s), 128);
            mbar_init(c.bar(kOFull + s), 1);
            mbar_init(c.bar(kOFree + s), 128);
        }
        mbar_init(c.bar(kMlFull), 128);
        mbar_init(c.bar(kDrain), 1);
        *c.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 12) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    c.tmem = *tmem_slot;

    if (warp < 8) {
        softmax_role(p, c, warp >> 2, tid & 127);
    } else if (warp < 12) {
        producer_role(p, c, tid - 256);
    } else {
        if (warp == 12) {
            mma_role(p, c);
        } else if (warp == 13) {
            tma_role(p, c, lane, &tm_pool_k, &tm_pool_v, &tm_ws_k, &tm_ws_v, &tm_knew, &tm_vnew);
        } else {
            append_role(p, c, tid - 448);
        }
    }

    // ---- teardown ------------------------------------------------------------------------------
    if (*c.abort_flag) {                    // let copies still in flight land before the CTA goes away
        const uint64_t t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 12) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(c.tmem), "r"(kTmemCols) : "memory");
    }
}

// ---- merge of partial results -------------------------------------------------------------------------------
// A partial holds, per 128-row query tile: un-normalised O (fp32, stored [32 float4 columns][128 rows]), the
// running max m of the raw scores and the sum l of exp2((s - m) * c).  Block = 32 rows of one query tile; lanes
// run along rows while reading (coalesced).  The partials of a tile are `n` blocks `stride` apart (the slots of
// a unit cut into pieces: consecutive; the same tile on every rank of a prefix-sharded request: one rank buffer
// apart).  The result is either final - normalised, turned through shared memory so that bf16 output rows are
// written 256 contiguous bytes at a time - or again a partial, in the canonical order of a rank buffer
// [request][kv head][row tile] (KVP_PARTIAL: what a rank hands to the exchange).
struct MergeOut {
    __nv_bfloat16 *out;         // final: [batch][q_len][n_q][128]
    float *lse;
    float4 *part_o;             // or partial: [tiles][32][128] float4 ...
    float2 *part_ml;            // ... and [tiles][128] (m, l)
};

__device__ __forceinline__ void merge_tile(int b, int hk, int row_base, int item_q_len, const float4 *po, const float2 *pml,
                                           int n, long long stride_o, long long stride_ml, int q_len, int n_q, int n_kv,
                                           int group, float scale, const MergeOut &mo)
{
    __shared__ uint2 tile[32][33];
    const int lane = threadIdx.x & 31, wv = threadIdx.x >> 5;
    const int row = blockIdx.y * 32 + lane;                     // row of the 128-row query tile
    const int n_rows = group * (item_q_len ? item_q_len : q_len);       // q_len stays the stride of the padded tensors
    const float c2 = scale * 1.4426950408889634f;
    float M = -INFINITY;
    float L = 0.f;
    float4 o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) o[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < n; ++s) {
        const float2 ml = pml[s * stride_ml + row];
        if (ml.y > 0.f) M = fmaxf(M, ml.x);
    }
    for (int s = 0; s < n; ++s) {
        const float2 ml = pml[s * stride_ml + row];
        if (!(ml.y > 0.f)) continue;                        // an empty partial: nothing was visible to this row
        const float w = exp2f((ml.x - M) * c2);
        L += w * ml.y;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 a = po[s * stride_o + (wv + 8 * j) * KVP_TILE_ROWS + row];
            o[j].x += w * a.x; o[j].y += w * a.y; o[j].z += w * a.z; o[j].w += w * a.w;
        }
    }
    if (mo.part_o != nullptr) {                                 // stays a partial: un-normalised, against the max M
        const long long c = ((long long)b * n_kv + hk) * ((group * q_len + KVP_TILE_ROWS - 1) / KVP_TILE_ROWS) + row_base / KVP_TILE_ROWS;
#pragma unroll
        for (int j = 0; j < 4; ++j) mo.part_o[(c * 32 + wv + 8 * j) * KVP_TILE_ROWS + row] = o[j];
        if (wv == 0) mo.part_ml[c * KVP_TILE_ROWS + row] = make_float2(L > 0.f ? M : -1e30f, L);
        return;
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint2 u;
        u.x = pack_bf16(o[j].x * inv, o[j].y * inv);
        u.y = pack_bf16(o[j].z * inv, o[j].w * inv);
        tile[lane][wv + 8 * j] = u;
    }
    const int r = row_base + row;
    if (wv == 0 && r < n_rows && mo.lse != nullptr)
        mo.lse[((long long)b * n_q + hk * group + r % group) * q_len + r / group] = M * scale + logf(L);
    __syncthreads();
    // 8 threads per output row, 32 bytes each
    const int orow = threadIdx.x >> 3, j8 = threadIdx.x & 7;
    const int r2 = row_base + blockIdx.y * 32 + orow;
    if (r2 < n_rows) {
        const int i = r2 / group, h = hk * group + r2 % group;
        uint4 *dst = reinterpret_cast<uint4 *>(mo.out + (((long long)b * q_len + i) * n_q + h) * 128) + 2 * j8;
        const uint2 a0 = tile[orow][4 * j8], a1 = tile[orow][4 * j8 + 1], a2 = tile[orow][4 * j8 + 2], a3 = tile[orow][4 * j8 + 3];
        dst[0] = make_uint4(a0.x, a0.y, a1.x, a1.y);
        dst[1] = make_uint4(a2.x, a2.y, a3.x, a3.y);
    }
}

// The partial slots of the units of one launch.  Grid (merge item, 4).
__global__ void __launch_bounds__(256)
merge_list_kernel(const kvp_merge_item *__restrict__ merges, int q_len, int n_q, int n_kv, int group, float scale,
                  const float *__restrict__ part_o, const float2 *__restrict__ part_ml, MergeOut mo)
{
    const kvp_merge_item mi = merges[blockIdx.x];
    merge_tile(mi.b, mi.hk, mi.row_base, mi.pad[0], reinterpret_cast<const float4 *>(part_o) + (long long)mi.slot0 * (32 * KVP_TILE_ROWS),
               part_ml + (long long)mi.slot0 * KVP_TILE_ROWS, mi.n_slots, 32 * KVP_TILE_ROWS, KVP_TILE_ROWS, q_len, n_q, n_kv,
               group, scale, mo);
}

// The rank buffers of a prefix-sharded request, `n_parts` of them `part_bytes` apart.  Grid (query tile, 4), query
// tiles in the canonical order [request][kv head][row tile].
__global__ void __launch_bounds__(256)
merge_ranks_kernel(const char *__restrict__ parts, int n_parts, long long part_bytes, long long ml_offset, int n_rt, int q_len,
                   int n_q, int n_kv, int group, float scale, MergeOut mo)
{
    const int c = blockIdx.x;
    const int rt = c % n_rt, hk = (c / n_rt) % n_kv, b = c / (n_rt * n_kv);
    merge_tile(b, hk, rt * KVP_TILE_ROWS, 0, reinterpret_cast<const float4 *>(parts) + (long long)c * (32 * KVP_TILE_ROWS),
               reinterpret_cast<const float2 *>(parts + ml_offset) + (long long)c * KVP_TILE_ROWS, n_parts, part_bytes / 16,
               part_bytes / 8, q_len, n_q, n_kv, group, scale, mo);
}

}  // namespace

cudaError_t kvp_attn_sm100_prepare(void)
{
    return cudaFuncSetAttribute(attn_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

cudaError_t kvp_launch_attn_sm100(const kvp_shape &sh, const kvp_attn2_args &a, const CUtensorMap &tm_pool_k,
                                  const CUtensorMap &tm_pool_v, const CUtensorMap &tm_ws_k,
                                  const CUtensorMap &tm_ws_v, cudaStream_t st)
{
    Params p;
    p.plan = a.plan;
    p.q_len = a.q_len;
    p.q_pos0 = a.q_pos0;
    p.layer = a.layer;
    p.n_q = sh.n_q_heads;
    p.n_kv = sh.n_kv_heads;
    p.group = sh.group;
    p.pairing = sh.pairing;
    p.scale = sh.scale;
    p.scale_log2 = sh.scale * 1.4426950408889634f;
    p.cta_begin = a.cta_begin;
    p.works = a.works;
    p.q = (const __nv_bfloat16 *)a.q;
    p.out = (__nv_bfloat16 *)a.out;
    p.lse = a.lse;
    p.partial_o = a.partial_o;
    p.partial_ml = a.partial_ml;
    p.status = a.status;
    p.tail_direct = a.tail_direct;
    p.precise = a.precise;
    p.l2_prefetch = a.l2_prefetch;
    p.k_new = (const uint4 *)a.k_new;
    p.v_new = (const uint4 *)a.v_new;
    p.ws_k = (uint4 *)a.ws_k;
    p.ws_v = (uint4 *)a.ws_v;
    p.ws_rows = sh.ws_rows;
    // without tail_direct the two query maps are never dereferenced: any valid map will do
    attn_sm100_kernel<<<a.n_ctas, kThreads, kSmemBytes, st>>>(tm_pool_k, tm_pool_v, tm_ws_k, tm_ws_v,
                                                              a.tail_direct ? a.tm_knew : tm_ws_k,
                                                              a.tail_direct ? a.tm_vnew : tm_ws_v, p);
    return cudaGetLastError();
}

cudaError_t kvp_launch_merge_list(const kvp_shape &sh, int32_t q_len, int32_t n_merges, const kvp_merge_item *merges,
                                  const float *partial_o, const float2 *partial_ml, void *out, float *lse,
                                  void *part_out, int64_t part_tiles, cudaStream_t st)
{
    if (n_merges <= 0) return cudaSuccess;
    MergeOut mo;
    mo.out = (__nv_bfloat16 *)out;
    mo.lse = lse;
    mo.part_o = nullptr;
    mo.part_ml = nullptr;
    if (part_out != nullptr) {                                   // KVP_PARTIAL: `out` stays untouched
        mo.part_o = reinterpret_cast<float4 *>(part_out);
        mo.part_ml = reinterpret_cast<float2 *>((char *)part_out + (uint64_t)part_tiles * (32ull * KVP_TILE_ROWS * 16));
    }
    merge_list_kernel<<<dim3(n_merges, KVP_TILE_ROWS / 32), 256, 0, st>>>(merges, q_len, sh.n_q_heads, sh.n_kv_heads, sh.group,
                                                                        sh.scale, partial_o, partial_ml, mo);
    return cudaGetLastError();
}

cudaError_t kvp_launch_merge_ranks(const kvp_shape &sh, int32_t batch, int32_t q_len, const void *parts, int32_t n_parts,
                                   void *out, float *lse, cudaStream_t st)
{
    const int n_rt = (sh.group * q_len + KVP_TILE_ROWS - 1) / KVP_TILE_ROWS;
    const uint64_t tiles = (uint64_t)batch * sh.n_kv_heads * n_rt;
    MergeOut mo;
    mo.out = (__nv_bfloat16 *)out;
    mo.lse = lse;
    mo.part_o = nullptr;
    mo.part_ml = nullptr;
    merge_ranks_kernel<<<dim3((unsigned)tiles, KVP_TILE_ROWS / 32), 256, 0, st>>>(
        (const char *)parts, n_parts, (long long)(tiles * (32ull * KVP_TILE_ROWS * 16 + KVP_TILE_ROWS * 8)),
        (long long)(tiles * (32ull * KVP_TILE_ROWS * 16)), n_rt, q_len, sh.n_q_heads, sh.n_kv_heads, sh.group, sh.scale, mo);
    return cudaGetLastError();
}
