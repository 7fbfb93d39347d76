// bf16 composed-cache attention for sm_100a: TMA-staged K/V tiles, tcgen05 MMA with TMEM accumulators.
//
// One CTA owns 128 packed query rows (query token i, head-in-group) of one (request, kv head) and a
// contiguous range of that request's key tiles: first the causal tiles of the query's own keys, then
// the prefix tiles of the plan (staged adapter rows, then documents read in place from the pool).
//
//   warps 0-3  softmax: one thread per query row.  S = Q K^T arrives in TMEM; the thread takes the row
//              max, forms p = exp2((s - m) * scale*log2e), sums it in fp32, writes P as bf16 back into
//              TMEM over S, and rescales O in TMEM when the running max moved by more than 2^8.
//              They also produce the Q operand: documents keep the keys they were cached with, so
//              instead of rotating every key by Delta (Eq. 1) the Q tile is counter-rotated by -Delta
//              once per document, which leaves every score q.k unchanged.
//   warp 4     TMA producer: K then V of each tile into a 4-stage ring (two 64-column boxes each,
//              128-byte swizzle).
//   warp 5     MMA issuer: QK^T (both operands K-major in shared memory) into one of two S buffers,
//              P V (P from TMEM, V MN-major in shared memory) accumulating into O; owns TMEM.
//
// Every mbarrier wait is bounded: when it runs out the CTA records a code in the status word, drains
// what it has in flight, frees TMEM and returns.
#include <cuda_bf16.h>

#include "kvp_internal.h"

namespace {

constexpr int kStages = 4;
constexpr int kTileBytes = KVP_TILE_KEYS * 128 * 2;      // 32 KB: 128 rows x 128 bf16
constexpr int kHalfBytes = kTileBytes / 2;               // one 64-column box
constexpr int kThreads = 192;
constexpr int kTmemCols = 512;
constexpr uint32_t kColS0 = 0, kColS1 = 128, kColO = 256;

constexpr int kOffQ = 0;                                  // 2 x 32 KB rotated-Q buffers
constexpr int kOffRing = 2 * kTileBytes;                  // kStages x 32 KB
constexpr int kOffBar = kOffRing + kStages * kTileBytes;
constexpr int kSmemBytes = kOffBar + 256 + 1024;          // + barrier block + alignment slack

enum BarIdx { kKvFull = 0, kKvEmpty = kStages, kQFull = 2 * kStages, kSFull = kQFull + 2, kPFull = kSFull + 2,
              kPvDone = kPFull + 2, kDrain = kPvDone + 2, kNumBars = kDrain + 1 };

struct Params {
    kvp_plan_dev plan;
    int batch, q_len, layer, n_splits, n_mtiles, n_q, n_kv, group, pairing;
    float scale, scale_log2;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    float *lse;
    float *partial_o;
    float2 *partial_ml;
    int32_t *status;
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

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc)
        : "memory");
}

#define KVP_R8(r, o) "=r"(r[o]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), "=r"(r[o + 6]), "=r"(r[o + 7])
#define KVP_W8(r, o) "r"(r[o]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]), "r"(r[o + 6]), "r"(r[o + 7])

// 32 TMEM lanes (this warp's) x 32 consecutive 32-bit columns -> 32 registers per thread
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : KVP_R8(r, 0), KVP_R8(r, 8), KVP_R8(r, 16), KVP_R8(r, 24)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), KVP_W8(r, 0), KVP_W8(r, 8), KVP_W8(r, 16), KVP_W8(r, 24)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), KVP_W8(r, 0), KVP_W8(r, 8)
        : "memory");
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
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
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes)
{
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= 1ull << 46;                    // descriptor version for sm_100
    d |= 2ull << 61;                    // SWIZZLE_128B
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = n, A K-major, B K-major or MN-major.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, uint32_t b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

struct Tile {
    int row0, n_keys, src, rope, qoff;
};

__device__ __forceinline__ Tile get_tile(const Params &p, const kvp_item &it, int n_tail, int idx)
{
    Tile t;
    if (idx < n_tail) {
        t.row0 = it.tail_row0 + idx * KVP_TILE_KEYS;
        t.n_keys = min(KVP_TILE_KEYS, p.q_len - idx * KVP_TILE_KEYS);
        t.src = 1;
        t.rope = 0;
        t.qoff = idx * KVP_TILE_KEYS;
    } else {
        const kvp_tile g = p.plan.tiles[it.tile_begin + idx - n_tail];
        t.row0 = g.row0;
        t.n_keys = g.n_keys;
        t.src = g.src;
        t.rope = g.rope;
        t.qoff = -1;
    }
    return t;
}

// Write this thread's query row, counter-rotated by the offset of rope-table row `rope`, into a
// rotated-Q buffer in the K-major 128-byte-swizzled layout (two 64-column halves of 128 x 128 bytes).
__device__ __forceinline__ void produce_q_row(const Params &p, char *qbuf, int t, const __nv_bfloat16 *qrow, int rope)
{
    const int sw = t & 7;
    char *row_lo = qbuf + t * 128;
    char *row_hi = row_lo + kHalfBytes;
    if (qrow == nullptr) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            *reinterpret_cast<uint4 *>(row_lo + ((c ^ sw) << 4)) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4 *>(row_hi + ((c ^ sw) << 4)) = make_uint4(0, 0, 0, 0);
        }
        return;
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(qrow);
    const float2 *cs = p.plan.rope + (size_t)rope * 64;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        union { uint4 u; __nv_bfloat16 e[8]; } lo, hi;
        lo.u = __ldg(src + c);
        hi.u = __ldg(src + c + 8);
        if (rope != 0) {
            if (p.pairing == 0) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float2 w = __ldg(cs + c * 8 + k);
                    const float a = __bfloat162float(lo.e[k]), b = __bfloat162float(hi.e[k]);
                    lo.e[k] = __float2bfloat16_rn(a * w.x + b * w.y);        // R(-Delta): cos same, sin negated
                    hi.e[k] = __float2bfloat16_rn(b * w.x - a * w.y);
                }
            } else {
#pragma unroll
                for (int k = 0; k < 8; k += 2) {
                    float2 w = __ldg(cs + (c * 8 + k) / 2);
                    float a = __bfloat162float(lo.e[k]), b = __bfloat162float(lo.e[k + 1]);
                    lo.e[k] = __float2bfloat16_rn(a * w.x + b * w.y);
                    lo.e[k + 1] = __float2bfloat16_rn(b * w.x - a * w.y);
                    w = __ldg(cs + ((c + 8) * 8 + k) / 2);
                    a = __bfloat162float(hi.e[k]);
                    b = __bfloat162float(hi.e[k + 1]);
                    hi.e[k] = __float2bfloat16_rn(a * w.x + b * w.y);
                    hi.e[k + 1] = __float2bfloat16_rn(b * w.x - a * w.y);
                }
            }
        }
        *reinterpret_cast<uint4 *>(row_lo + ((c ^ sw) << 4)) = lo.u;
        *reinterpret_cast<uint4 *>(row_hi + ((c ^ sw) << 4)) = hi.u;
    }
}

__global__ void __launch_bounds__(kThreads, 1)
attn_sm100_single_kernel(const __grid_constant__ CUtensorMap tm_pool_k, const __grid_constant__ CUtensorMap tm_pool_v,
                  const __grid_constant__ CUtensorMap tm_ws_k, const __grid_constant__ CUtensorMap tm_ws_v,
                  const Params p)
{
    extern __shared__ char smem_raw[];
    char *smem = reinterpret_cast<char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar0 = smem_base + kOffBar;
    auto bar = [&](int i) { return bar0 + 8u * i; };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + kOffBar + 8 * kNumBars);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- which unit of work --------------------------------------------------------------------
    int x = blockIdx.x;
    const int split = x % p.n_splits;  x /= p.n_splits;
    const int mt = x % p.n_mtiles;     x /= p.n_mtiles;
    const int hk = x % p.n_kv;
    const int b = x / p.n_kv;
    const kvp_item it = p.plan.items[b];
    const int n_rows = p.group * p.q_len;
    const int row_base = mt * KVP_TILE_ROWS;
    const int i_max = min(n_rows - 1, row_base + KVP_TILE_ROWS - 1) / p.group;
    const int n_tail = i_max / KVP_TILE_KEYS + 1;
    const int n_all = n_tail + (it.tile_end - it.tile_begin);
    const int lo = (int)((long long)n_all * split / p.n_splits);
    const int n_my = (int)((long long)n_all * (split + 1) / p.n_splits) - lo;
    const int plane = p.layer * p.n_kv + hk;
    const long long unit = (long long)blockIdx.x;

    if (n_my <= 0) {                       // nothing to do for this split: an empty partial
        if (tid < KVP_TILE_ROWS && p.n_splits > 1) {
            p.partial_ml[unit * KVP_TILE_ROWS + tid] = make_float2(-1e30f, 0.f);
            float4 *o = reinterpret_cast<float4 *>(p.partial_o + (unit * KVP_TILE_ROWS + tid) * 128);
            for (int c = 0; c < 32; ++c) o[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        return;
    }

    // ---- set-up --------------------------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar(kKvFull + s), 1);
            mbar_init(bar(kKvEmpty + s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kQFull + s), 128);
            mbar_init(bar(kSFull + s), 1);
            mbar_init(bar(kPFull + s), 128);
            mbar_init(bar(kPvDone + s), 1);
        }
        mbar_init(bar(kDrain), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        // ================================ TMA producer ==========================================
        if (lane == 0) {
            for (int j = 0; j < n_my; ++j) {
                const Tile tl = get_tile(p, it, n_tail, lo + j);
                bool ok = true;
                for (int kv = 0; kv < 2 && ok; ++kv) {
                    const int n = 2 * j + kv, stage = n % kStages, use = n / kStages;
                    if (use > 0) ok = mbar_wait(bar(kKvEmpty + stage), (use - 1) & 1, abort_flag, p.status, 10 + stage);
                    if (!ok) break;
                    const CUtensorMap *tm = tl.src == 0 ? (kv ? &tm_pool_v : &tm_pool_k) : (kv ? &tm_ws_v : &tm_ws_k);
                    const uint32_t dst = smem_base + kOffRing + stage * kTileBytes;
                    mbar_expect_tx(bar(kKvFull + stage), kTileBytes);
                    tma_load_3d(dst, tm, 0, tl.row0, plane, bar(kKvFull + stage));
                    tma_load_3d(dst + kHalfBytes, tm, 64, tl.row0, plane, bar(kKvFull + stage));
                }
                if (!ok) break;
            }
        }
    } else if (warp == 5) {
        // ================================ MMA issuer ============================================
        if (lane == 0) {
            const uint32_t idesc_pv = instr_desc(128, 1);
            int ep = 0, prev_rope = 0;
            bool ok = true;
            auto issue_qk = [&](int j) {
                const Tile tl = get_tile(p, it, n_tail, lo + j);
                bool fresh = (j == 0);
                if (j > 0 && tl.rope != prev_rope) { ++ep; fresh = true; }
                prev_rope = tl.rope;
                if (fresh) ok = mbar_wait(bar(kQFull + (ep & 1)), (ep >> 1) & 1, abort_flag, p.status, 20);
                const int n = 2 * j, stage = n % kStages, sb = j & 1;
                if (ok) ok = mbar_wait(bar(kKvFull + stage), (n / kStages) & 1, abort_flag, p.status, 21);
                if (ok && j >= 2) ok = mbar_wait(bar(kPvDone + sb), ((j - 2) >> 1) & 1, abort_flag, p.status, 22);
                if (!ok) return;
                tc_fence_after();
                const uint32_t n16 = (uint32_t)(tl.n_keys + 15) & ~15u;
                const uint32_t idesc = instr_desc(n16, 0);
                const uint32_t qa = smem_base + kOffQ + (ep & 1) * kTileBytes;
                const uint32_t ka = smem_base + kOffRing + stage * kTileBytes;
                const uint32_t d = tmem + (sb ? kColS1 : kColS0);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint32_t off = (k >> 2) * kHalfBytes + (k & 3) * 32;
                    mma_ss(d, smem_desc(qa + off, 16), smem_desc(ka + off, 16), idesc, k > 0);
                }
                tc_commit(bar(kKvEmpty + stage));
                tc_commit(bar(kSFull + sb));
            };
            auto issue_pv = [&](int j) {
                const Tile tl = get_tile(p, it, n_tail, lo + j);
                const int n = 2 * j + 1, stage = n % kStages, sb = j & 1;
                ok = mbar_wait(bar(kKvFull + stage), (n / kStages) & 1, abort_flag, p.status, 23);
                if (ok) ok = mbar_wait(bar(kPFull + sb), (j >> 1) & 1, abort_flag, p.status, 24);
                if (!ok) return;
                tc_fence_after();
                const uint32_t va = smem_base + kOffRing + stage * kTileBytes;
                const uint32_t pa = tmem + (sb ? kColS1 : kColS0);
                const int ksteps = (tl.n_keys + 15) >> 4;
                for (int k = 0; k < ksteps; ++k)
                    mma_ts(tmem + kColO, pa + k * 8, smem_desc(va + k * 2048, kHalfBytes), idesc_pv, (j > 0 || k > 0));
                tc_commit(bar(kKvEmpty + stage));
                tc_commit(bar(kPvDone + sb));
            };
            issue_qk(0);
            for (int j = 0; j < n_my && ok; ++j) {
                if (j + 1 < n_my) issue_qk(j + 1);
                if (ok) issue_pv(j);
            }
            if (!ok) {                      // drain whatever was issued before giving TMEM back
                tc_commit(bar(kDrain));
                const uint64_t t0 = global_ns();
                while (!mbar_try_wait(bar(kDrain), 0) && global_ns() - t0 < 100000000ull) {}
            }
        }
    } else {
        // ================================ softmax / correction / epilogue ========================
        const int r = row_base + tid;
        const bool valid = r < n_rows;
        const int qi = valid ? r / p.group : p.q_len - 1;
        const int h = hk * p.group + (valid ? r % p.group : 0);
        const __nv_bfloat16 *qrow = valid ? p.q + (((long long)b * p.q_len + qi) * p.n_q + h) * 128 : nullptr;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const float c2 = p.scale_log2;

        int ep = 0, prev_rope = 0;
        {
            const Tile t0 = get_tile(p, it, n_tail, lo);
            prev_rope = t0.rope;
            produce_q_row(p, smem + kOffQ, tid, qrow, t0.rope);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive(bar(kQFull + 0));
        }
        float m_ref = -1e30f, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_my && ok; ++j) {
            const Tile tl = get_tile(p, it, n_tail, lo + j);
            const int sb = j & 1;
            bool fresh = (j == 0);
            if (j > 0 && tl.rope != prev_rope) { ++ep; fresh = true; }
            prev_rope = tl.rope;
            ok = mbar_wait(bar(kSFull + sb), (j >> 1) & 1, abort_flag, p.status, 30);
            if (!ok) break;
            tc_fence_after();
            if (fresh) {
                // first tile of a rotation epoch: prepare the next epoch's Q in the other buffer
                // (its previous user's QK^T MMAs have all completed by now)
                int nxt = -1;
                for (int jj = j + 1; jj < n_my; ++jj) {
                    const int rp = get_tile(p, it, n_tail, lo + jj).rope;
                    if (rp != tl.rope) { nxt = rp; break; }
                }
                if (nxt >= 0) {
                    produce_q_row(p, smem + kOffQ + ((ep + 1) & 1) * kTileBytes, tid, qrow, nxt);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    mbar_arrive(bar(kQFull + ((ep + 1) & 1)));
                }
            }
            const uint32_t s_addr = tmem + lane_base + (sb ? kColS1 : kColS0);
            const int n_chunks = (tl.n_keys + 31) >> 5;
            const bool full = (tl.n_keys == KVP_TILE_KEYS) && (tl.qoff < 0);
            const int lim = tl.qoff < 0 ? tl.n_keys : min(tl.n_keys, qi - tl.qoff + 1);   // visible keys: [0, lim)

            // pass 1: row max
            float mx = -INFINITY;
            for (int ch = 0; ch < n_chunks; ++ch) {
                uint32_t v[32];
                tmem_ld32(s_addr + ch * 32, v);
                tc_wait_ld();
                if (full) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) mx = fmaxf(mx, __uint_as_float(v[c]));
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (ch * 32 + c < lim) mx = fmaxf(mx, __uint_as_float(v[c]));
                }
            }
            const float m_new = fmaxf(m_ref, mx);
            if (j == 0) {
                m_ref = m_new;
            } else {
                const bool need = (m_new - m_ref) * c2 > 8.0f;
                if (__any_sync(0xffffffffu, need)) {
                    // O is about to change scale: the previous P V product must have landed first
                    ok = mbar_wait(bar(kPvDone + ((j - 1) & 1)), ((j - 1) >> 1) & 1, abort_flag, p.status, 31);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const float alpha = ex2((m_ref - m_new) * c2);
                    m_ref = m_new;
                    l *= alpha;
                    for (int ch = 0; ch < 4; ++ch) {
                        uint32_t v[32];
                        tmem_ld32(tmem + lane_base + kColO + ch * 32, v);
                        tc_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) v[c] = __float_as_uint(__uint_as_float(v[c]) * alpha);
                        tmem_st32(tmem + lane_base + kColO + ch * 32, v);
                    }
                }
            }
            // pass 2: p = exp2((s - m) c), written over S as packed bf16 (chunk ch -> columns 16ch..16ch+15)
            const float mc = m_ref * c2;
            float lsum = 0.f;
            for (int ch = 0; ch < n_chunks; ++ch) {
                uint32_t v[32], w[16];
                tmem_ld32(s_addr + ch * 32, v);
                tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                    float p0 = ex2(fmaf(__uint_as_float(v[c]), c2, -mc));
                    float p1 = ex2(fmaf(__uint_as_float(v[c + 1]), c2, -mc));
                    if (!full) {
                        if (ch * 32 + c >= lim) p0 = 0.f;
                        if (ch * 32 + c + 1 >= lim) p1 = 0.f;
                    }
                    lsum += p0 + p1;
                    w[c >> 1] = pack_bf16(p0, p1);
                }
                tmem_st16(s_addr + ch * 16, w);
            }
            l += lsum;
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bar(kPFull + sb));
        }

        if (ok) ok = mbar_wait(bar(kPvDone + ((n_my - 1) & 1)), ((n_my - 1) >> 1) & 1, abort_flag, p.status, 32);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after();
            if (p.n_splits == 1) {
                const float inv = 1.f / l;
                uint4 *orow = valid ? reinterpret_cast<uint4 *>(p.out + (((long long)b * p.q_len + qi) * p.n_q + h) * 128) : nullptr;
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_base + kColO + ch * 32, v);
                    tc_wait_ld();
                    if (valid) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint4 u;
                            u.x = pack_bf16(__uint_as_float(v[8 * c + 0]) * inv, __uint_as_float(v[8 * c + 1]) * inv);
                            u.y = pack_bf16(__uint_as_float(v[8 * c + 2]) * inv, __uint_as_float(v[8 * c + 3]) * inv);
                            u.z = pack_bf16(__uint_as_float(v[8 * c + 4]) * inv, __uint_as_float(v[8 * c + 5]) * inv);
                            u.w = pack_bf16(__uint_as_float(v[8 * c + 6]) * inv, __uint_as_float(v[8 * c + 7]) * inv);
                            orow[ch * 4 + c] = u;
                        }
                    }
                }
                if (valid && p.lse != nullptr)
                    p.lse[((long long)b * p.n_q + h) * p.q_len + qi] = m_ref * p.scale + logf(l);
            } else {
                p.partial_ml[unit * KVP_TILE_ROWS + tid] = make_float2(m_ref, l);
                uint4 *orow = reinterpret_cast<uint4 *>(p.partial_o + (unit * KVP_TILE_ROWS + tid) * 128);
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_base + kColO + ch * 32, v);
                    tc_wait_ld();
#pragma unroll
                    for (int c = 0; c < 8; ++c) orow[ch * 8 + c] = make_uint4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                }
            }
        }
    }

    // ---- teardown ------------------------------------------------------------------------------
    if (*abort_flag) {                      // let copies still in flight land before the CTA goes away
        const uint64_t t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

cudaError_t kvp_attn_sm100_single_prepare(void)
{
    return cudaFuncSetAttribute(attn_sm100_single_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

cudaError_t kvp_launch_attn_sm100_single(const kvp_shape &sh, const kvp_attn_sm100_args &a, const CUtensorMap &tm_pool_k,
                                  const CUtensorMap &tm_pool_v, const CUtensorMap &tm_ws_k,
                                  const CUtensorMap &tm_ws_v, int32_t *ctas, cudaStream_t st)
{
    Params p;
    p.plan = a.plan;
    p.batch = a.batch;
    p.q_len = a.q_len;
    p.layer = a.layer;
    p.n_splits = a.n_splits;
    p.n_mtiles = a.n_mtiles;
    p.n_q = sh.n_q_heads;
    p.n_kv = sh.n_kv_heads;
    p.group = sh.group;
    p.pairing = sh.pairing;
    p.scale = sh.scale;
    p.scale_log2 = sh.scale * 1.4426950408889634f;
    p.q = (const __nv_bfloat16 *)a.q;
    p.out = (__nv_bfloat16 *)a.out;
    p.lse = a.lse;
    p.partial_o = a.partial_o;
    p.partial_ml = a.partial_ml;
    p.status = a.status;
    const int grid = a.batch * sh.n_kv_heads * a.n_mtiles * a.n_splits;
    if (ctas) *ctas = grid;
    attn_sm100_single_kernel<<<grid, kThreads, kSmemBytes, st>>>(tm_pool_k, tm_pool_v, tm_ws_k, tm_ws_v, p);
    return cudaGetLastError();
}
