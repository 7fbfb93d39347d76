// CUDA-core kernels of the composed-cache path: packet registration (layout change), gather with
// RoPE re-basing (Eq. 1), query K/V append, cache export, a plain fp32 attention kernel that reads
// packets in place through the tile list, and the split-KV merge.
#include <cuda_bf16.h>

#include "kvp_internal.h"

namespace {

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kPerVec = 4;
    __device__ static float to_f32(float x) { return x; }
    __device__ static float from_f32(float x) { return x; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    __device__ static float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
    __device__ static __nv_bfloat16 from_f32(float x) { return __float2bfloat16_rn(x); }
};

template <typename T> union Vec16 {
    uint4 u;
    T e[Elem<T>::kPerVec];
};

// Eq. 1 for one pair: (a, b) -> (a cos - b sin, a sin + b cos), fp32.
__device__ __forceinline__ void rotate_pair(float &a, float &b, float c, float s)
{
    const float ra = a * c - b * s;
    const float rb = a * s + b * c;
    a = ra;
    b = rb;
}

// Rotate the two 16-byte vectors a thread owns.  Half-split pairing: lo holds elements
// [c*EV, c*EV+EV) and hi the partners d/2 further on; interleaved pairing: each vector holds its
// own pairs (2i, 2i+1).  cs points at the (cos, sin) row of this offset.
template <typename T>
__device__ __forceinline__ void rotate_vec_pair(Vec16<T> &lo, Vec16<T> &hi, const float2 *cs, int c, int half_vecs,
                                                int pairing)
{
    constexpr int EV = Elem<T>::kPerVec;
    if (pairing == 0) {
#pragma unroll
        for (int k = 0; k < EV; ++k) {
            const float2 w = cs[c * EV + k];
            float a = Elem<T>::to_f32(lo.e[k]), b = Elem<T>::to_f32(hi.e[k]);
            rotate_pair(a, b, w.x, w.y);
            lo.e[k] = Elem<T>::from_f32(a);
            hi.e[k] = Elem<T>::from_f32(b);
        }
    } else {
#pragma unroll
        for (int k = 0; k < EV; k += 2) {
            float2 w = cs[(c * EV + k) / 2];
            float a = Elem<T>::to_f32(lo.e[k]), b = Elem<T>::to_f32(lo.e[k + 1]);
            rotate_pair(a, b, w.x, w.y);
            lo.e[k] = Elem<T>::from_f32(a);
            lo.e[k + 1] = Elem<T>::from_f32(b);
            w = cs[((c + half_vecs) * EV + k) / 2];
            a = Elem<T>::to_f32(hi.e[k]);
            b = Elem<T>::to_f32(hi.e[k + 1]);
            rotate_pair(a, b, w.x, w.y);
            hi.e[k] = Elem<T>::from_f32(a);
            hi.e[k + 1] = Elem<T>::from_f32(b);
        }
    }
}

// ---- registration: [L][n][Hkv][d] -> plane (l, hk), rows dst_row0 + t ----------------------------
__global__ void store_rows_kernel(const uint4 *__restrict__ src, char *__restrict__ dst, int64_t plane_rows,
                                  int64_t dst_row0, int n_tokens, int n_layers, int n_kv, int vecs_per_row)
{
    const int64_t total = (int64_t)n_layers * n_tokens * n_kv * vecs_per_row;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(idx % vecs_per_row);
        int64_t r = idx / vecs_per_row;
        const int hk = (int)(r % n_kv);
        r /= n_kv;
        const int t = (int)(r % n_tokens);
        const int l = (int)(r / n_tokens);
        const int64_t drow = ((int64_t)(l * n_kv + hk)) * plane_rows + dst_row0 + t;
        reinterpret_cast<uint4 *>(dst)[drow * vecs_per_row + c] = src[idx];
    }
}

// ---- gather + re-base: pool rows -> workspace rows, all layers and kv heads ------------------------
// grid (n_chunks, L*Hkv); one thread per (row, pair of 16-byte vectors); V is a byte copy, K is a byte
// copy when the chunk's offset is 0 and an fp32 rotation otherwise.
template <typename T>
__global__ void gather_kernel(kvp_plan_dev plan, const char *__restrict__ pool_k, const char *__restrict__ pool_v,
                              char *__restrict__ ws_k, char *__restrict__ ws_v, int64_t pool_rows, int64_t ws_rows,
                              int vecs_per_row, int half_dim, int pairing)
{
    const kvp_chunk ch = plan.chunks[blockIdx.x];
    const int plane = blockIdx.y;
    const int half_vecs = vecs_per_row / 2;
    const float2 *cs = plan.rope + (size_t)ch.rope * half_dim;
    const uint4 *sk = reinterpret_cast<const uint4 *>(pool_k) + ((int64_t)plane * pool_rows + ch.src_row0) * vecs_per_row;
    const uint4 *sv = reinterpret_cast<const uint4 *>(pool_v) + ((int64_t)plane * pool_rows + ch.src_row0) * vecs_per_row;
    uint4 *dk = reinterpret_cast<uint4 *>(ws_k) + ((int64_t)plane * ws_rows + ch.dst_row0) * vecs_per_row;
    uint4 *dv = reinterpret_cast<uint4 *>(ws_v) + ((int64_t)plane * ws_rows + ch.dst_row0) * vecs_per_row;
    for (int w = threadIdx.x; w < ch.n_rows * half_vecs; w += blockDim.x) {
        const int row = w / half_vecs, c = w % half_vecs;
        const int o = row * vecs_per_row + c;
        Vec16<T> lo, hi;
        lo.u = __ldg(sk + o);
        hi.u = __ldg(sk + o + half_vecs);
        if (ch.rope != 0) rotate_vec_pair<T>(lo, hi, cs, c, half_vecs, pairing);
        dk[o] = lo.u;
        dk[o + half_vecs] = hi.u;
        dv[o] = __ldg(sv + o);
        dv[o + half_vecs] = __ldg(sv + o + half_vecs);
    }
}

// ---- append: the query chunk's own K/V rows go behind the prefix (Section 3.2 step 4) --------------
// grid (batch*q_len); the rows go behind the q_pos0 rows appended earlier; with rope_query the raw
// k_new and q are first rotated to positions prefix_len + q_pos0 + i, angles formed in double precision.
template <typename T>
__global__ void append_kernel(kvp_plan_dev plan, int q_len, int q_pos0, const T *__restrict__ q, const T *__restrict__ k_new,
                              const T *__restrict__ v_new, char *__restrict__ ws_k, char *__restrict__ ws_v,
                              int64_t ws_rows, int layer, int n_q, int n_kv, int d, int pairing, int rope_query,
                              const double *__restrict__ inv_freq, T *__restrict__ q_rot)
{
    __shared__ float2 cs[64];
    const int b = blockIdx.x / q_len, i = blockIdx.x % q_len;
    const kvp_item it = plan.items[b];
    const int half = d / 2;
    if (rope_query) {
        for (int p = threadIdx.x; p < half; p += blockDim.x) {
            double s, c;
            sincos((double)(it.prefix_len + q_pos0 + i) * inv_freq[p], &s, &c);
            cs[p] = make_float2((float)c, (float)s);
        }
        __syncthreads();
    }
    const int64_t tok = (int64_t)b * q_len + i;
    // keys and values: one thread per (kv head, pair)
    for (int w = threadIdx.x; w < n_kv * half; w += blockDim.x) {
        const int hk = w / half, p = w % half;
        const int ia = pairing ? 2 * p : p, ib = pairing ? 2 * p + 1 : p + half;
        const T *ks = k_new + (tok * n_kv + hk) * d;
        const T *vs = v_new + (tok * n_kv + hk) * d;
        const int64_t drow = ((int64_t)(layer * n_kv + hk)) * ws_rows + it.tail_row0 + q_pos0 + i;
        T *kd = reinterpret_cast<T *>(ws_k) + drow * d;
        T *vd = reinterpret_cast<T *>(ws_v) + drow * d;
        float a = Elem<T>::to_f32(ks[ia]), bb = Elem<T>::to_f32(ks[ib]);
        if (rope_query) {
            rotate_pair(a, bb, cs[p].x, cs[p].y);
            kd[ia] = Elem<T>::from_f32(a);
            kd[ib] = Elem<T>::from_f32(bb);
        } else {
            kd[ia] = ks[ia];
            kd[ib] = ks[ib];
        }
        vd[ia] = vs[ia];
        vd[ib] = vs[ib];
    }
    if (rope_query) {
        for (int w = threadIdx.x; w < n_q * half; w += blockDim.x) {
            const int h = w / half, p = w % half;
            const int ia = pairing ? 2 * p : p, ib = pairing ? 2 * p + 1 : p + half;
            const T *qs = q + (tok * n_q + h) * d;
            T *qd = q_rot + (tok * n_q + h) * d;
            float a = Elem<T>::to_f32(qs[ia]), bb = Elem<T>::to_f32(qs[ib]);
            rotate_pair(a, bb, cs[p].x, cs[p].y);
            qd[ia] = Elem<T>::from_f32(a);
            qd[ib] = Elem<T>::from_f32(bb);
        }
    }
}

// ---- export of the logical composed cache of one (layer, request) ---------------------------------
// grid (n_rows, Hkv), one thread per pair.  Prefix rows come from where attention reads them: the
// materialised cache or the staged adapter rows (already re-based), else the pool (rotated here).
template <typename T>
__global__ void export_kernel(kvp_plan_dev plan, int b, int layer, int prefix_len, const char *__restrict__ pool_k,
                              const char *__restrict__ pool_v, const char *__restrict__ ws_k,
                              const char *__restrict__ ws_v, int64_t pool_rows, int64_t ws_rows, int n_kv, int d,
                              int pairing, void *__restrict__ k_out, T *__restrict__ v_out, int k_as_f32)
{
    const int t = blockIdx.x, hk = blockIdx.y;
    const kvp_item it = plan.items[b];
    const int half = d / 2;
    const int plane = layer * n_kv + hk;
    const T *ks, *vs;
    int rope = 0;
    if (t >= prefix_len) {
        const int64_t r = (int64_t)plane * ws_rows + it.tail_row0 + (t - prefix_len);
        ks = reinterpret_cast<const T *>(ws_k) + r * d;
        vs = reinterpret_cast<const T *>(ws_v) + r * d;
    } else if (it.cache_row0 >= 0) {
        const int64_t r = (int64_t)plane * ws_rows + it.cache_row0 + t;
        ks = reinterpret_cast<const T *>(ws_k) + r * d;
        vs = reinterpret_cast<const T *>(ws_v) + r * d;
    } else {
        int lo = it.seg_begin, hi = it.seg_end - 1;      // last segment with dst_pos0 <= t
        while (lo < hi) {
            const int mid = (lo + hi + 1) / 2;
            if (plan.segs[mid].dst_pos0 <= t) lo = mid; else hi = mid - 1;
        }
        const kvp_seg sg = plan.segs[lo];
        const int off = t - sg.dst_pos0;
        if (sg.pad[0] >= 0) {                            // staged in the workspace, already re-based
            const int64_t r = (int64_t)plane * ws_rows + sg.pad[0] + off;
            ks = reinterpret_cast<const T *>(ws_k) + r * d;
            vs = reinterpret_cast<const T *>(ws_v) + r * d;
        } else {
            const int64_t r = (int64_t)plane * pool_rows + sg.src_row0 + off;
            ks = reinterpret_cast<const T *>(pool_k) + r * d;
            vs = reinterpret_cast<const T *>(pool_v) + r * d;
            rope = sg.rope;
        }
    }
    const float2 *cs = plan.rope + (size_t)rope * half;
    const int64_t orow = ((int64_t)t * n_kv + hk) * d;
    for (int p = threadIdx.x; p < half; p += blockDim.x) {
        const int ia = pairing ? 2 * p : p, ib = pairing ? 2 * p + 1 : p + half;
        float a = Elem<T>::to_f32(ks[ia]), bb = Elem<T>::to_f32(ks[ib]);
        if (rope != 0) rotate_pair(a, bb, cs[p].x, cs[p].y);
        if (k_as_f32) {
            reinterpret_cast<float *>(k_out)[orow + ia] = a;
            reinterpret_cast<float *>(k_out)[orow + ib] = bb;
        } else if (rope != 0) {
            reinterpret_cast<T *>(k_out)[orow + ia] = Elem<T>::from_f32(a);
            reinterpret_cast<T *>(k_out)[orow + ib] = Elem<T>::from_f32(bb);
        } else {
            reinterpret_cast<T *>(k_out)[orow + ia] = ks[ia];
            reinterpret_cast<T *>(k_out)[orow + ib] = ks[ib];
        }
        v_out[orow + ia] = vs[ia];
        v_out[orow + ib] = vs[ib];
    }
}

// ---- plain fp32 attention over [tail tiles | prefix tiles] -----------------------------------------
// 16 packed rows (query token i, head-in-group) per CTA, 32 keys per step, online softmax in fp32.
// Keys still carrying an offset are rotated here as Eq. 1 states it (on K, in fp32).
template <typename T, int D>
__global__ void __launch_bounds__(128)
attn_simple_kernel(kvp_plan_dev plan, int q_len, int q_pos0, int layer, const T *__restrict__ q, const char *__restrict__ pool_k,
                   const char *__restrict__ pool_v, const char *__restrict__ ws_k, const char *__restrict__ ws_v,
                   int64_t pool_rows, int64_t ws_rows, int n_q, int n_kv, int group, int pairing, float scale,
                   T *__restrict__ out, float *__restrict__ lse)
{
    constexpr int RB = 16, KC = 32, HALF = D / 2;
    __shared__ float Qs[RB][D];
    __shared__ float Ks[KC][D + 1];
    __shared__ float Vs[KC][D];
    __shared__ float Ps[RB][KC];

    const int hk = blockIdx.y, b = blockIdx.z;
    const kvp_item it = plan.items[(layer * n_kv + hk) * plan.item_stride + b];
    const int n_rows = group * q_len;
    const int row = threadIdx.x / 8, sub = threadIdx.x % 8;
    const int r = blockIdx.x * RB + row;
    const bool valid = r < n_rows;
    const int i = valid ? r / group : q_len - 1;
    const int h = hk * group + (valid ? r % group : 0);
    const int plane = layer * n_kv + hk;

    for (int w = threadIdx.x; w < RB * D; w += blockDim.x) {
        const int rr = blockIdx.x * RB + w / D, c = w % D;
        float x = 0.f;
        if (rr < n_rows) x = Elem<T>::to_f32(q[(((int64_t)b * q_len + rr / group) * n_q + hk * group + rr % group) * D + c]);
        Qs[w / D][c] = x;
    }

    const int last_row = min(n_rows - 1, blockIdx.x * RB + RB - 1);
    const int i_max = last_row / group;
    const int n_tail = (q_pos0 + i_max) / KVP_TILE_KEYS + 1;      // tail keys: rows appended earlier, then this call's
    const int n_tiles = n_tail + (it.tile_end - it.tile_begin);

    float m = -1e30f, l = 0.f;
    float acc[D / 8];
#pragma unroll
    for (int e = 0; e < D / 8; ++e) acc[e] = 0.f;

    for (int tt = 0; tt < n_tiles; ++tt) {
        kvp_tile tl;
        int qoff = -1;
        if (tt < n_tail) {
            tl.row0 = it.tail_row0 + tt * KVP_TILE_KEYS;
            tl.n_keys = (int16_t)min(KVP_TILE_KEYS, q_pos0 + q_len - tt * KVP_TILE_KEYS);
            tl.src = 1;
            tl.rope = 0;
            qoff = tt * KVP_TILE_KEYS;
        } else {
            tl = plan.tiles[it.tile_begin + tt - n_tail];
        }
        const int64_t prow = (tl.src == 0) ? (int64_t)plane * pool_rows : (int64_t)plane * ws_rows;
        const T *kb = reinterpret_cast<const T *>(tl.src == 0 ? pool_k : ws_k) + (prow + tl.row0) * D;
        const T *vb = reinterpret_cast<const T *>(tl.src == 0 ? pool_v : ws_v) + (prow + tl.row0) * D;
        const float2 *cs = plan.rope + (size_t)tl.rope * HALF;

        for (int k0 = 0; k0 < tl.n_keys; k0 += KC) {
            const int nk = min(KC, tl.n_keys - k0);
            __syncthreads();
            for (int w = threadIdx.x; w < KC * HALF; w += blockDim.x) {
                const int kk = w / HALF, p = w % HALF;
                const int ia = pairing ? 2 * p : p, ib = pairing ? 2 * p + 1 : p + HALF;
                float a = 0.f, bb = 0.f, va = 0.f, vb2 = 0.f;
                if (kk < nk) {
                    const T *kr = kb + (int64_t)(k0 + kk) * D;
                    const T *vr = vb + (int64_t)(k0 + kk) * D;
                    a = Elem<T>::to_f32(kr[ia]);
                    bb = Elem<T>::to_f32(kr[ib]);
                    va = Elem<T>::to_f32(vr[ia]);
                    vb2 = Elem<T>::to_f32(vr[ib]);
                    if (tl.rope != 0) rotate_pair(a, bb, cs[p].x, cs[p].y);
                }
                Ks[kk][ia] = a;
                Ks[kk][ib] = bb;
                Vs[kk][ia] = va;
                Vs[kk][ib] = vb2;
            }
            __syncthreads();

            float s[4];
            float mx = -INFINITY;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int kk = sub + 8 * u;
                float a = 0.f;
#pragma unroll 8
                for (int c = 0; c < D; ++c) a += Qs[row][c] * Ks[kk][c];
                const bool vis = kk < nk && (qoff < 0 || qoff + k0 + kk <= q_pos0 + i);
                s[u] = vis ? a * scale : -INFINITY;
                mx = fmaxf(mx, s[u]);
            }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            const float m_new = fmaxf(m, mx);
            const float alpha = expf(m - m_new);
            float ps = 0.f;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float p = expf(s[u] - m_new);      // exp(-inf) = 0 for masked keys
                Ps[row][sub + 8 * u] = p;
                ps += p;
            }
            ps += __shfl_xor_sync(0xffffffffu, ps, 1);
            ps += __shfl_xor_sync(0xffffffffu, ps, 2);
            ps += __shfl_xor_sync(0xffffffffu, ps, 4);
            l = l * alpha + ps;
            m = m_new;
            __syncwarp();
#pragma unroll
            for (int e = 0; e < D / 8; ++e) acc[e] *= alpha;
            for (int kk = 0; kk < KC; ++kk) {
                const float p = Ps[row][kk];
#pragma unroll
                for (int e = 0; e < D / 8; ++e) acc[e] += p * Vs[kk][sub + 8 * e];
            }
            __syncwarp();
        }
    }
    if (valid) {
        const float inv = 1.f / l;
        T *o = out + (((int64_t)b * q_len + i) * n_q + h) * D;
#pragma unroll
        for (int e = 0; e < D / 8; ++e) o[sub + 8 * e] = Elem<T>::from_f32(acc[e] * inv);
        if (lse != nullptr && sub == 0) lse[((int64_t)b * n_q + h) * q_len + i] = m + logf(l);
    }
}

// ---- attention mass per segment (diagnostic) ----------------------------------------------------------
// grid (batch * q_len, Hkv), 256 threads = 8 warps.  The block holds the group's q rows in fp32; each warp
// takes every eighth key of a segment, each lane two rotation pairs of the key (Eq. 1 in fp32, as the
// CUDA-core attention kernel does), scores by warp reduction, p = exp(scale * q.k' - lse) summed per head.
template <typename T, int D>
__global__ void __launch_bounds__(256)
segment_mass_kernel(kvp_plan_dev plan, int q_len, int q_pos0, int layer, const T *__restrict__ q,
                    const float *__restrict__ lse, const char *__restrict__ pool_k, const char *__restrict__ ws_k,
                    int64_t pool_rows, int64_t ws_rows, int n_q, int n_kv, int group, int pairing, float scale,
                    float *__restrict__ mass, int n_cols)
{
    constexpr int HALF = D / 2, PPL = HALF / 32;            // rotation pairs per lane
    extern __shared__ float sm[];                            // [group][D] q rows, [8][group] partial sums, [group] lse
    float *qs = sm, *part = sm + group * D, *ls = part + 8 * group;
    const int b = blockIdx.x / q_len, i = blockIdx.x % q_len, hk = blockIdx.y;
    const kvp_item it = plan.items[(layer * n_kv + hk) * plan.item_stride + b];
    const int plane = layer * n_kv + hk;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int w = threadIdx.x; w < group * D; w += blockDim.x)
        qs[w] = Elem<T>::to_f32(q[(((int64_t)b * q_len + i) * n_q + hk * group + w / D) * D + w % D]);
    for (int w = threadIdx.x; w < group; w += blockDim.x) ls[w] = lse[((int64_t)b * n_q + hk * group + w) * q_len + i];
    __syncthreads();
    float *out = mass + (((int64_t)b * q_len + i) * n_q + hk * group) * n_cols;
    const int n_seg = it.seg_end - it.seg_begin;
    for (int s = 0; s <= n_seg; ++s) {
        // segment s, or (s == n_seg) the query block: appended rows 0 .. q_pos0 + i
        const T *kb;
        int n_keys, rope = 0;
        if (s < n_seg) {
            const kvp_seg sg = plan.segs[it.seg_begin + s];
            kb = reinterpret_cast<const T *>(pool_k) + ((int64_t)plane * pool_rows + sg.src_row0) * D;
            n_keys = sg.pad[2] >= 0 ? plan.kept[sg.pad[2] * plan.n_planes + plane] : sg.len;
            rope = sg.rope;
        } else {
            kb = reinterpret_cast<const T *>(ws_k) + ((int64_t)plane * ws_rows + it.tail_row0) * D;
            n_keys = q_pos0 + i + 1;
        }
        const float2 *cs = plan.rope + (size_t)rope * HALF;
        float acc[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) acc[h] = 0.f;
        for (int j = warp; j < n_keys; j += 8) {
            const T *kr = kb + (int64_t)j * D;
            float ka[PPL], kc[PPL];
            int ia[PPL], ib[PPL];
#pragma unroll
            for (int u = 0; u < PPL; ++u) {
                const int pr = lane + 32 * u;
                ia[u] = pairing ? 2 * pr : pr;
                ib[u] = pairing ? 2 * pr + 1 : pr + HALF;
                ka[u] = Elem<T>::to_f32(kr[ia[u]]);
                kc[u] = Elem<T>::to_f32(kr[ib[u]]);
                if (rope != 0) rotate_pair(ka[u], kc[u], cs[pr].x, cs[pr].y);
            }
            for (int h = 0; h < group; ++h) {
                float d = 0.f;
#pragma unroll
                for (int u = 0; u < PPL; ++u) d += qs[h * D + ia[u]] * ka[u] + qs[h * D + ib[u]] * kc[u];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
                if (h < 8) acc[h] += expf(d * scale - ls[h]);
            }
        }
        if (lane == 0)
            for (int h = 0; h < group && h < 8; ++h) part[warp * group + h] = acc[h];
        __syncthreads();
        if (threadIdx.x < group) {
            float t = 0.f;
            for (int w = 0; w < 8; ++w) t += part[w * group + threadIdx.x];
            out[(int64_t)threadIdx.x * n_cols + s] = t;
        }
        __syncthreads();
    }
    for (int w = threadIdx.x; w < group * (n_cols - n_seg - 1); w += blockDim.x)
        out[(int64_t)(w / (n_cols - n_seg - 1)) * n_cols + n_seg + 1 + w % (n_cols - n_seg - 1)] = 0.f;
}

}  // namespace

// ---- launchers ------------------------------------------------------------------------------------

cudaError_t kvp_launch_store_rows(const kvp_shape &sh, const void *src, char *dst_plane0, int64_t plane_rows,
                                  int64_t dst_row0, int32_t n_tokens, cudaStream_t st)
{
    const int vecs = sh.head_dim * sh.elem_bytes / 16;
    const int64_t total = (int64_t)sh.n_layers * n_tokens * sh.n_kv_heads * vecs;
    const int grid = (int)((total + 255) / 256 > 65535 * 8 ? 65535 * 8 : (total + 255) / 256);
    store_rows_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const uint4 *>(src), dst_plane0, plane_rows, dst_row0,
                                            n_tokens, sh.n_layers, sh.n_kv_heads, vecs);
    return cudaGetLastError();
}

cudaError_t kvp_launch_gather(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t n_chunks, const char *pool_k,
                              const char *pool_v, char *ws_k, char *ws_v, cudaStream_t st)
{
    if (n_chunks <= 0) return cudaSuccess;
    const int vecs = sh.head_dim * sh.elem_bytes / 16;
    const dim3 grid(n_chunks, sh.n_layers * sh.n_kv_heads);
    const int threads = KVP_CHUNK_ROWS * (vecs / 2);
    if (sh.dtype == KVP_DTYPE_BF16)
        gather_kernel<__nv_bfloat16><<<grid, threads, 0, st>>>(plan, pool_k, pool_v, ws_k, ws_v, sh.pool_rows,
                                                              sh.ws_rows, vecs, sh.head_dim / 2, sh.pairing);
    else
        gather_kernel<float><<<grid, threads, 0, st>>>(plan, pool_k, pool_v, ws_k, ws_v, sh.pool_rows, sh.ws_rows,
                                                      vecs, sh.head_dim / 2, sh.pairing);
    return cudaGetLastError();
}

cudaError_t kvp_launch_append(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t batch, int32_t q_len,
                              int32_t q_pos0, const void *q, const void *k_new, const void *v_new, char *ws_k, char *ws_v,
                              int32_t layer, int32_t rope_query, const double *inv_freq_dev, void *q_rot,
                              cudaStream_t st)
{
    const int grid = batch * q_len;
    if (sh.dtype == KVP_DTYPE_BF16)
        append_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(
            plan, q_len, q_pos0, (const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k_new, (const __nv_bfloat16 *)v_new, ws_k,
            ws_v, sh.ws_rows, layer, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.pairing, rope_query, inv_freq_dev,
            (__nv_bfloat16 *)q_rot);
    else
        append_kernel<float><<<grid, 256, 0, st>>>(plan, q_len, q_pos0, (const float *)q, (const float *)k_new,
                                                   (const float *)v_new, ws_k, ws_v, sh.ws_rows, layer, sh.n_q_heads,
                                                   sh.n_kv_heads, sh.head_dim, sh.pairing, rope_query, inv_freq_dev,
                                                   (float *)q_rot);
    return cudaGetLastError();
}

cudaError_t kvp_launch_export(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t b, int32_t layer,
                              int32_t prefix_len, int32_t n_query_rows, const char *pool_k, const char *pool_v,
                              const char *ws_k, const char *ws_v, void *k_out, void *v_out, int32_t k_as_f32,
                              cudaStream_t st)
{
    const int n_rows = prefix_len + n_query_rows;
    if (n_rows <= 0) return cudaSuccess;
    const dim3 grid(n_rows, sh.n_kv_heads);
    if (sh.dtype == KVP_DTYPE_BF16)
        export_kernel<__nv_bfloat16><<<grid, 64, 0, st>>>(plan, b, layer, prefix_len, pool_k, pool_v, ws_k, ws_v,
                                                         sh.pool_rows, sh.ws_rows, sh.n_kv_heads, sh.head_dim,
                                                         sh.pairing, k_out, (__nv_bfloat16 *)v_out, k_as_f32);
    else
        export_kernel<float><<<grid, 64, 0, st>>>(plan, b, layer, prefix_len, pool_k, pool_v, ws_k, ws_v, sh.pool_rows,
                                                 sh.ws_rows, sh.n_kv_heads, sh.head_dim, sh.pairing, k_out,
                                                 (float *)v_out, k_as_f32);
    return cudaGetLastError();
}

cudaError_t kvp_launch_segment_mass(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t batch, int32_t q_len,
                                    int32_t q_pos0, int32_t layer, const void *q, const float *lse, const char *pool_k,
                                    const char *ws_k, float *mass, int32_t n_cols, cudaStream_t st)
{
    const dim3 grid(batch * q_len, sh.n_kv_heads);
    const size_t smem = sizeof(float) * ((size_t)sh.group * sh.head_dim + 9 * sh.group);
#define KVP_MASS(T, D)                                                                                              \
    segment_mass_kernel<T, D><<<grid, 256, smem, st>>>(plan, q_len, q_pos0, layer, (const T *)q, lse, pool_k, ws_k,  \
                                                       sh.pool_rows, sh.ws_rows, sh.n_q_heads, sh.n_kv_heads,       \
                                                       sh.group, sh.pairing, sh.scale, mass, n_cols)
    if (sh.dtype == KVP_DTYPE_BF16) {
        if (sh.head_dim == 128) KVP_MASS(__nv_bfloat16, 128); else KVP_MASS(__nv_bfloat16, 64);
    } else {
        if (sh.head_dim == 128) KVP_MASS(float, 128); else KVP_MASS(float, 64);
    }
#undef KVP_MASS
    return cudaGetLastError();
}

cudaError_t kvp_launch_attn_simple(const kvp_shape &sh, const kvp_plan_dev &plan, int32_t batch, int32_t q_len,
                                   int32_t q_pos0, int32_t layer, const void *q, const char *pool_k, const char *pool_v,
                                   const char *ws_k, const char *ws_v, void *out, float *lse, int32_t *ctas,
                                   cudaStream_t st)
{
    const dim3 grid((sh.group * q_len + 15) / 16, sh.n_kv_heads, batch);
    if (ctas) *ctas = (int32_t)(grid.x * grid.y * grid.z);
#define KVP_SIMPLE(T, D)                                                                                             \
    attn_simple_kernel<T, D><<<grid, 128, 0, st>>>(plan, q_len, q_pos0, layer, (const T *)q, pool_k, pool_v, ws_k, ws_v,     \
                                                   sh.pool_rows, sh.ws_rows, sh.n_q_heads, sh.n_kv_heads, sh.group,  \
                                                   sh.pairing, sh.scale, (T *)out, lse)
    if (sh.dtype == KVP_DTYPE_BF16) {
        if (sh.head_dim == 128) KVP_SIMPLE(__nv_bfloat16, 128); else KVP_SIMPLE(__nv_bfloat16, 64);
    } else {
        if (sh.head_dim == 128) KVP_SIMPLE(float, 128); else KVP_SIMPLE(float, 64);
    }
#undef KVP_SIMPLE
    return cudaGetLastError();
}
