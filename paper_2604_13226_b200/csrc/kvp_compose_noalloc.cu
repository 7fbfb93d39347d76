// kvp_compose_noalloc: gather + re-base of one request's segments for callers that cannot allocate.
//
// The regular path (kvp_assemble) keeps its gather plan - segment records and the cos/sin table of
// every rotation offset - in a workspace the caller allocated, and stages it through pinned host
// memory the library allocated.  Some callers can do neither: code running inside a memory-frozen
// region (a serving process after its allocator has been sealed, a plugin that is handed raw device
// pointers but no allocator, an interrupt-style callback that must not touch the CUDA heap).  For
// them this file carries the same gather kernel with its scratch in a fixed device array that is
// part of the library image.
//
// The array is shared by every call on a device and keeps whatever the previous call left in it.
// Nothing in it has to start at zero: each call overwrites every record it will read before the
// gather kernel runs (stream order).  Two calls whose kernels overlap on the GPU (different streams,
// or different host threads) race on the array; callers must serialise them.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include <mutex>

#include "../../include/kvp.h"

namespace {

constexpr int kMaxSeg = KVP_NOALLOC_MAX_SEGMENTS;
constexpr int kHalfMax = 64;                       // head_dim <= 128
constexpr int kChunkRows = 32;

struct SegRecord {                                  // one segment as the gather kernel reads it
    int32_t src_row0, len, dst_row0, delta;
};
struct Scratch {
    float2 rope[kMaxSeg][kHalfMax];                 // (cos, sin) of delta * theta_i
    SegRecord seg[kMaxSeg];
};

// The scratch itself: 96 x (64 x 8 + 16) bytes = 50688 bytes of device memory that every GPU which
// loads this library holds until the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress - it is not a device address and must never be passed to a kernel.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(Scratch)];

struct SegParams {                                  // travels to the set-up kernel by value
    int32_t n;
    int32_t src_row0[kMaxSeg], len[kMaxSeg], dst_row0[kMaxSeg], delta[kMaxSeg];
};

// Fill the scratch for this call: one block per segment; angles and frequencies in double precision.
__global__ void noalloc_setup_kernel(Scratch *sc, const SegParams sp, double theta, int head_dim)
{
    const int s = blockIdx.x;
    const int half = head_dim / 2;
    if (threadIdx.x == 0) sc->seg[s] = SegRecord{sp.src_row0[s], sp.len[s], sp.dst_row0[s], sp.delta[s]};
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        const double inv_freq = pow(theta, -2.0 * (double)i / (double)head_dim);
        double sn, cs;
        sincos((double)sp.delta[s] * inv_freq, &sn, &cs);
        sc->rope[s][i] = make_float2((float)cs, (float)sn);
    }
}

template <typename T> struct El;
template <> struct El<float> {
    static constexpr int kPerVec = 4;
    __device__ static float ld(float x) { return x; }
    __device__ static float st(float x) { return x; }
};
template <> struct El<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    __device__ static float ld(__nv_bfloat16 x) { return __bfloat162float(x); }
    __device__ static __nv_bfloat16 st(float x) { return __float2bfloat16_rn(x); }
};

// Gather: grid (row chunks, segments, planes).  V rows and keys with offset 0 are byte copies; other
// keys are rotated pair by pair in fp32: (a, b) -> (a cos - b sin, a sin + b cos)  (Eq. 1).
template <typename T>
__global__ void noalloc_gather_kernel(const Scratch *sc, const uint4 *__restrict__ pool_k,
                                      const uint4 *__restrict__ pool_v, uint4 *__restrict__ cache_k,
                                      uint4 *__restrict__ cache_v, int64_t pool_rows, int64_t cache_rows,
                                      int vecs_per_row, int pairing)
{
    constexpr int EV = El<T>::kPerVec;
    const SegRecord sg = sc->seg[blockIdx.y];
    const int row_begin = blockIdx.x * kChunkRows;
    if (row_begin >= sg.len) return;
    const int n_rows = min(kChunkRows, sg.len - row_begin);
    const int plane = blockIdx.z;
    const int half_vecs = vecs_per_row / 2;
    const float2 *cs = sc->rope[blockIdx.y];
    const int64_t so = ((int64_t)plane * pool_rows + sg.src_row0 + row_begin) * vecs_per_row;
    const int64_t dofs = ((int64_t)plane * cache_rows + sg.dst_row0 + row_begin) * vecs_per_row;
    for (int w = threadIdx.x; w < n_rows * half_vecs; w += blockDim.x) {
        const int row = w / half_vecs, c = w % half_vecs;
        const int o = row * vecs_per_row + c;
        union { uint4 u; T e[EV]; } lo, hi;
        lo.u = __ldg(pool_k + so + o);
        hi.u = __ldg(pool_k + so + o + half_vecs);
        if (sg.delta != 0) {
            if (pairing == 0) {
#pragma unroll
                for (int k = 0; k < EV; ++k) {
                    const float2 t = cs[c * EV + k];
                    const float a = El<T>::ld(lo.e[k]), b = El<T>::ld(hi.e[k]);
                    lo.e[k] = El<T>::st(a * t.x - b * t.y);
                    hi.e[k] = El<T>::st(a * t.y + b * t.x);
                }
            } else {
#pragma unroll
                for (int k = 0; k < EV; k += 2) {
                    float2 t = cs[(c * EV + k) / 2];
                    float a = El<T>::ld(lo.e[k]), b = El<T>::ld(lo.e[k + 1]);
                    lo.e[k] = El<T>::st(a * t.x - b * t.y);
                    lo.e[k + 1] = El<T>::st(a * t.y + b * t.x);
                    t = cs[((c + half_vecs) * EV + k) / 2];
                    a = El<T>::ld(hi.e[k]);
                    b = El<T>::ld(hi.e[k + 1]);
                    hi.e[k] = El<T>::st(a * t.x - b * t.y);
                    hi.e[k + 1] = El<T>::st(a * t.y + b * t.x);
                }
            }
        }
        cache_k[dofs + o] = lo.u;
        cache_k[dofs + o + half_vecs] = hi.u;
        cache_v[dofs + o] = __ldg(pool_v + so + o);
        cache_v[dofs + o + half_vecs] = __ldg(pool_v + so + o + half_vecs);
    }
}

// Device address of the scratch array on the current device, looked up once per device.
std::mutex g_mu;
void *g_scratch_addr[64] = {};

cudaError_t scratch_on_current_device(Scratch **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_addr[dev] == nullptr) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);        // resolves the symbol for the current device
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    *out = static_cast<Scratch *>(g_scratch_addr[dev]);
    return cudaSuccess;
}

int32_t report(char *err, int32_t cap, int32_t code, const char *msg)
{
    if (err && cap > 0) snprintf(err, (size_t)cap, "%s", msg);
    return code;
}

}  // namespace

extern "C" int32_t kvp_compose_noalloc(const void *pool_k, const void *pool_v, int64_t pool_rows, int32_t n_planes,
                                       int32_t head_dim, int32_t dtype, int32_t rope_pairing, double rope_theta,
                                       int32_t n_segments, const int32_t *src_row0, const int32_t *seg_len,
                                       const int32_t *delta, void *cache_k, void *cache_v, int64_t cache_rows,
                                       void *stream, char *err, int32_t err_cap)
{
    if (err && err_cap > 0) err[0] = 0;
    if (!pool_k || !pool_v || !cache_k || !cache_v || !src_row0 || !seg_len || !delta)
        return report(err, err_cap, KVP_ERR_INVALID, "compose_noalloc: null pointer");
    if (((uintptr_t)pool_k | (uintptr_t)pool_v | (uintptr_t)cache_k | (uintptr_t)cache_v) & 15)
        return report(err, err_cap, KVP_ERR_INVALID, "compose_noalloc: pool and cache pointers must be 16-byte aligned");
    if (n_segments <= 0) return report(err, err_cap, KVP_ERR_INVALID, "compose_noalloc: n_segments must be positive");
    if (n_segments > kMaxSeg) {
        char msg[160];
        snprintf(msg, sizeof msg, "compose_noalloc: %d segments exceed the fixed scratch (max %d per call)", n_segments,
                 kMaxSeg);
        return report(err, err_cap, KVP_ERR_CAPACITY, msg);
    }
    if ((head_dim != 64 && head_dim != 128) || (dtype != KVP_DTYPE_F32 && dtype != KVP_DTYPE_BF16) ||
        (rope_pairing != 0 && rope_pairing != 1) || !(rope_theta > 0.0) || n_planes <= 0 || n_planes > 65535 ||
        pool_rows <= 0 || cache_rows <= 0)
        return report(err, err_cap, KVP_ERR_INVALID, "compose_noalloc: bad shape, dtype, pairing or theta");
    SegParams sp;
    sp.n = n_segments;
    int64_t dst = 0;
    int32_t max_len = 0;
    for (int s = 0; s < n_segments; ++s) {
        if (seg_len[s] <= 0 || src_row0[s] < 0 || (int64_t)src_row0[s] + seg_len[s] > pool_rows)
            return report(err, err_cap, KVP_ERR_INVALID, "compose_noalloc: segment outside the pool");
        if (dst + seg_len[s] > cache_rows || dst + seg_len[s] > (int64_t)INT32_MAX)     // before dst is narrowed below
            return report(err, err_cap, KVP_ERR_CAPACITY, "compose_noalloc: segments do not fit in cache_rows");
        sp.src_row0[s] = src_row0[s];
        sp.len[s] = seg_len[s];
        sp.dst_row0[s] = (int32_t)dst;
        sp.delta[s] = delta[s];
        dst += seg_len[s];
        if (seg_len[s] > max_len) max_len = seg_len[s];
    }

    Scratch *sc = nullptr;
    cudaError_t e = scratch_on_current_device(&sc);
    if (e != cudaSuccess) return report(err, err_cap, KVP_ERR_CUDA, cudaGetErrorString(e));
    cudaStream_t st = (cudaStream_t)stream;
    noalloc_setup_kernel<<<n_segments, 64, 0, st>>>(sc, sp, rope_theta, head_dim);
    const int elem = dtype == KVP_DTYPE_BF16 ? 2 : 4;
    const int vecs = head_dim * elem / 16;
    const dim3 grid((max_len + kChunkRows - 1) / kChunkRows, n_segments, n_planes);
    const int threads = kChunkRows * (vecs / 2);
    if (dtype == KVP_DTYPE_BF16)
        noalloc_gather_kernel<__nv_bfloat16><<<grid, threads, 0, st>>>(
            sc, (const uint4 *)pool_k, (const uint4 *)pool_v, (uint4 *)cache_k, (uint4 *)cache_v, pool_rows, cache_rows,
            vecs, rope_pairing);
    else
        noalloc_gather_kernel<float><<<grid, threads, 0, st>>>(sc, (const uint4 *)pool_k, (const uint4 *)pool_v,
                                                               (uint4 *)cache_k, (uint4 *)cache_v, pool_rows,
                                                               cache_rows, vecs, rope_pairing);
    e = cudaGetLastError();
    if (e != cudaSuccess) return report(err, err_cap, KVP_ERR_CUDA, cudaGetErrorString(e));
    return KVP_OK;
}
