// Bucket-streamed AdamW (OffloadStreamAdamW, Algorithm 4): host-resident fp32 state, a fused fp32 update + bf16
// refresh kernel, and a three-stream pipeline over staging slots in device memory.  See stream_adamw.h.
//
// The kernel is bound by device memory traffic (16 B read, 14 B written per parameter) and the pipeline by the
// host link (16 B in, 12 B out per parameter), three orders of magnitude apart: the update hides behind the copies.

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <new>
#include <vector>

#include "stream_adamw.h"
#include "vp_ce.h"

namespace {

struct AdamScalars {
    float decay;        // 1 - lr * weight_decay
    float beta1, one_minus_beta1, beta2, one_minus_beta2;
    float inv_bc2;      // 1 / (1 - beta2^t)
    float step_size;    // lr / (1 - beta1^t)
    float eps;
};

__device__ __forceinline__ void adam_one(float& p, float& m, float& v, float g, const AdamScalars& s) {
    p = p * s.decay;
    m = s.beta1 * m + s.one_minus_beta1 * g;
    v = s.beta2 * v + s.one_minus_beta2 * (g * g);
    const float denom = sqrtf(v * s.inv_bc2) + s.eps;
    p = p - s.step_size * (m / denom);
}

// One thread per 4 consecutive parameters (128-bit loads and stores), grid-stride; the tail runs scalar.
__global__ void __launch_bounds__(256)
osadamw_kernel(float* __restrict__ p, float* __restrict__ m, float* __restrict__ v, const float* __restrict__ g,
               __nv_bfloat16* __restrict__ w, long n, const AdamScalars s) {
    const long n4 = n >> 2;
    const long stride = static_cast<long>(gridDim.x) * blockDim.x;
    for (long i = static_cast<long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 pp = __ldcs(reinterpret_cast<const float4*>(p) + i);       // streamed: every byte is touched once
        float4 mm = __ldcs(reinterpret_cast<const float4*>(m) + i);
        float4 vv = __ldcs(reinterpret_cast<const float4*>(v) + i);
        const float4 gg = __ldcs(reinterpret_cast<const float4*>(g) + i);
        adam_one(pp.x, mm.x, vv.x, gg.x, s);
        adam_one(pp.y, mm.y, vv.y, gg.y, s);
        adam_one(pp.z, mm.z, vv.z, gg.z, s);
        adam_one(pp.w, mm.w, vv.w, gg.w, s);
        __stcs(reinterpret_cast<float4*>(p) + i, pp);
        __stcs(reinterpret_cast<float4*>(m) + i, mm);
        __stcs(reinterpret_cast<float4*>(v) + i, vv);
        const __nv_bfloat162 lo = __floats2bfloat162_rn(pp.x, pp.y), hi = __floats2bfloat162_rn(pp.z, pp.w);
        uint2 o;
        o.x = *reinterpret_cast<const uint32_t*>(&lo);
        o.y = *reinterpret_cast<const uint32_t*>(&hi);
        *(reinterpret_cast<uint2*>(w) + i) = o;                            // the working weight stays cached for its readers
    }
    const long tail0 = n4 << 2;
    for (long i = tail0 + static_cast<long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) {
        float pp = p[i], mm = m[i], vv = v[i];
        adam_one(pp, mm, vv, g[i], s);
        p[i] = pp; m[i] = mm; v[i] = vv;
        w[i] = __float2bfloat16_rn(pp);
    }
}

bool make_scalars(AdamScalars* s, float lr, float beta1, float beta2, float eps, float wd, int64_t step) {
    if (step < 1 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f)) return false;
    const double bc1 = 1.0 - std::pow(static_cast<double>(beta1), static_cast<double>(step));
    const double bc2 = 1.0 - std::pow(static_cast<double>(beta2), static_cast<double>(step));
    s->decay = static_cast<float>(1.0 - static_cast<double>(lr) * static_cast<double>(wd));
    s->beta1 = beta1; s->one_minus_beta1 = static_cast<float>(1.0 - static_cast<double>(beta1));
    s->beta2 = beta2; s->one_minus_beta2 = static_cast<float>(1.0 - static_cast<double>(beta2));
    s->inv_bc2 = static_cast<float>(1.0 / bc2);
    s->step_size = static_cast<float>(static_cast<double>(lr) / bc1);
    s->eps = eps;
    return true;
}

int grid_for(long n) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long blocks_needed = ((n >> 2) + 255) / 256 + 1;
    const long cap = static_cast<long>(sms) * 8;            // 8 resident blocks of 256 threads per SM
    return static_cast<int>(blocks_needed < cap ? blocks_needed : cap);
}

cudaError_t launch_update(float* p, float* m, float* v, const float* g, void* w, long n, const AdamScalars& s,
                          cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    osadamw_kernel<<<grid_for(n), 256, 0, st>>>(p, m, v, g, static_cast<__nv_bfloat16*>(w), n, s);
    return cudaGetLastError();
}

inline size_t slot_floats(int64_t bucket) { return (static_cast<size_t>(bucket) + 63) / 64 * 64; }   // 256-byte arrays

}  // namespace

struct osadamw_ctx {
    int dev;
    int64_t bucket;
    int slots;
    float* staging;
    cudaStream_t s_in, s_upd, s_out;
    std::vector<cudaEvent_t> loaded, updated, written;
    std::vector<char> used;
    cudaEvent_t ev_entry, ev_last_update;
};

extern "C" {

size_t osadamw_staging_bytes(int64_t bucket_params, int slots) {
    if (bucket_params <= 0 || slots <= 0 || slots > 64) return 0;
    return static_cast<size_t>(slots) * 4 * slot_floats(bucket_params) * sizeof(float);
}

int osadamw_create(osadamw_ctx** out, int64_t bucket_params, int slots, void* staging, size_t staging_bytes) {
    if (!out || !staging) return VPCE_INVALID_ARG;
    const size_t need = osadamw_staging_bytes(bucket_params, slots);
    if (need == 0) return VPCE_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(staging) & 255u) return VPCE_UNSUPPORTED;
    if (staging_bytes < need) return VPCE_WORKSPACE_TOO_SMALL;
    osadamw_ctx* c = new (std::nothrow) osadamw_ctx();
    if (!c) return VPCE_CUDA_ERROR;
    c->bucket = bucket_params; c->slots = slots; c->staging = static_cast<float*>(staging);
    c->s_in = c->s_upd = c->s_out = nullptr; c->ev_entry = c->ev_last_update = nullptr;
    bool ok = cudaGetDevice(&c->dev) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->s_in, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->s_upd, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_entry, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_last_update, cudaEventDisableTiming) == cudaSuccess;
    for (int k = 0; ok && k < slots; ++k) {
        cudaEvent_t a = nullptr, b = nullptr, w = nullptr;
        ok = cudaEventCreateWithFlags(&a, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&b, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&w, cudaEventDisableTiming) == cudaSuccess;
        c->loaded.push_back(a); c->updated.push_back(b); c->written.push_back(w);
    }
    c->used.assign(slots, 0);
    if (!ok) { osadamw_destroy(c); return VPCE_CUDA_ERROR; }
    *out = c;
    return VPCE_OK;
}

int osadamw_destroy(osadamw_ctx* c) {
    if (!c) return VPCE_OK;
    if (c->s_in) { cudaStreamSynchronize(c->s_in); cudaStreamDestroy(c->s_in); }
    if (c->s_upd) { cudaStreamSynchronize(c->s_upd); cudaStreamDestroy(c->s_upd); }
    if (c->s_out) { cudaStreamSynchronize(c->s_out); cudaStreamDestroy(c->s_out); }
    for (auto e : c->loaded) if (e) cudaEventDestroy(e);
    for (auto e : c->updated) if (e) cudaEventDestroy(e);
    for (auto e : c->written) if (e) cudaEventDestroy(e);
    if (c->ev_entry) cudaEventDestroy(c->ev_entry);
    if (c->ev_last_update) cudaEventDestroy(c->ev_last_update);
    delete c;
    return VPCE_OK;
}

int osadamw_step(osadamw_ctx* c, float* master, float* m, float* v, const float* grad, void* w_bf16, int64_t n,
                 const int64_t* bucket_offsets, int64_t n_buckets, float lr, float beta1, float beta2, float eps,
                 float weight_decay, int64_t step, void* user_stream) {
    if (!c || n < 0) return VPCE_INVALID_ARG;
    if (n == 0) return VPCE_OK;
    if (!master || !m || !v || !grad || !w_bf16) return VPCE_INVALID_ARG;
    AdamScalars sc;
    if (!make_scalars(&sc, lr, beta1, beta2, eps, weight_decay, step)) return VPCE_INVALID_ARG;
    if (bucket_offsets) {
        if (n_buckets < 1 || bucket_offsets[0] != 0 || bucket_offsets[n_buckets] != n) return VPCE_INVALID_ARG;
        for (int64_t b = 0; b < n_buckets; ++b) {
            const int64_t len = bucket_offsets[b + 1] - bucket_offsets[b];
            if (len <= 0 || len > c->bucket) return VPCE_INVALID_ARG;
            // the slot arrays are read with 128-bit loads from their start; the working weight is written at the
            // bucket's offset with 64-bit stores
            if (bucket_offsets[b] % 4) return VPCE_UNSUPPORTED;
        }
    } else {
        if (c->bucket % 4) return VPCE_UNSUPPORTED;
        n_buckets = (n + c->bucket - 1) / c->bucket;
    }
    if (reinterpret_cast<uintptr_t>(w_bf16) & 7u) return VPCE_UNSUPPORTED;
    cudaStream_t us = static_cast<cudaStream_t>(user_stream);
    // everything the caller enqueued so far comes first
    if (cudaEventRecord(c->ev_entry, us) != cudaSuccess || cudaStreamWaitEvent(c->s_in, c->ev_entry, 0) != cudaSuccess ||
        cudaStreamWaitEvent(c->s_upd, c->ev_entry, 0) != cudaSuccess)
        return VPCE_CUDA_ERROR;
    const size_t sf = slot_floats(c->bucket);
    for (int64_t b = 0; b < n_buckets; ++b) {
        const int64_t a0 = bucket_offsets ? bucket_offsets[b] : b * c->bucket;
        const int64_t a1 = bucket_offsets ? bucket_offsets[b + 1] : (a0 + c->bucket < n ? a0 + c->bucket : n);
        const size_t len = static_cast<size_t>(a1 - a0);
        const int k = static_cast<int>(b % c->slots);
        float* sp = c->staging + static_cast<size_t>(k) * 4 * sf;
        float *sm = sp + sf, *sv = sp + 2 * sf, *sg = sp + 3 * sf;
        // (i) a slot is free again once its write-back has completed (Algorithm 4: "wait for a free staging slot")
        if (c->used[k] && cudaStreamWaitEvent(c->s_in, c->written[k], 0) != cudaSuccess) return VPCE_CUDA_ERROR;
        c->used[k] = 1;
        // Inside a bucket the three stages run piece by piece (up to 8 pieces of at least 4 Mi parameters), so the update
        // and the write-back of a large bucket start when its first piece has arrived, not when all of it has: filling
        // and draining the pipeline then costs a piece, not a bucket.  An event may be recorded again while an earlier
        // wait on it is pending: a wait refers to the record that was current when the wait was enqueued.
        size_t piece = (len + 7) / 8;
        if (piece < (4u << 20)) piece = 4u << 20;
        piece = (piece + 3) / 4 * 4;
        for (size_t o = 0; o < len; o += piece) {
            const size_t l = len - o < piece ? len - o : piece, bytes = l * sizeof(float);
            const int64_t g0 = a0 + static_cast<int64_t>(o);
            if (cudaMemcpyAsync(sp + o, master + g0, bytes, cudaMemcpyHostToDevice, c->s_in) != cudaSuccess ||
                cudaMemcpyAsync(sm + o, m + g0, bytes, cudaMemcpyHostToDevice, c->s_in) != cudaSuccess ||
                cudaMemcpyAsync(sv + o, v + g0, bytes, cudaMemcpyHostToDevice, c->s_in) != cudaSuccess ||
                cudaMemcpyAsync(sg + o, grad + g0, bytes, cudaMemcpyHostToDevice, c->s_in) != cudaSuccess ||
                cudaEventRecord(c->loaded[k], c->s_in) != cudaSuccess)
                return VPCE_CUDA_ERROR;
            // (ii) fused update + bf16 refresh
            if (cudaStreamWaitEvent(c->s_upd, c->loaded[k], 0) != cudaSuccess ||
                launch_update(sp + o, sm + o, sv + o, sg + o, static_cast<__nv_bfloat16*>(w_bf16) + g0, static_cast<long>(l), sc,
                              c->s_upd) != cudaSuccess ||
                cudaEventRecord(c->updated[k], c->s_upd) != cudaSuccess)
                return VPCE_CUDA_ERROR;
            // (iii) write the fp32 state back
            if (cudaStreamWaitEvent(c->s_out, c->updated[k], 0) != cudaSuccess ||
                cudaMemcpyAsync(master + g0, sp + o, bytes, cudaMemcpyDeviceToHost, c->s_out) != cudaSuccess ||
                cudaMemcpyAsync(m + g0, sm + o, bytes, cudaMemcpyDeviceToHost, c->s_out) != cudaSuccess ||
                cudaMemcpyAsync(v + g0, sv + o, bytes, cudaMemcpyDeviceToHost, c->s_out) != cudaSuccess ||
                cudaEventRecord(c->written[k], c->s_out) != cudaSuccess)
                return VPCE_CUDA_ERROR;
        }
    }
    // later work on the caller's stream sees the refreshed working weight
    if (cudaEventRecord(c->ev_last_update, c->s_upd) != cudaSuccess ||
        cudaStreamWaitEvent(us, c->ev_last_update, 0) != cudaSuccess)
        return VPCE_CUDA_ERROR;
    return VPCE_OK;
}

int osadamw_wait(osadamw_ctx* c) {
    if (!c) return VPCE_INVALID_ARG;
    if (cudaStreamSynchronize(c->s_out) != cudaSuccess || cudaStreamSynchronize(c->s_upd) != cudaSuccess)
        return VPCE_CUDA_ERROR;
    return VPCE_OK;
}

int osadamw_update_device(float* p, float* m, float* v, const float* g, void* w_bf16, int64_t n, float lr, float beta1,
                          float beta2, float eps, float weight_decay, int64_t step, void* stream) {
    if (n < 0) return VPCE_INVALID_ARG;
    if (n == 0) return VPCE_OK;
    if (!p || !m || !v || !g || !w_bf16) return VPCE_INVALID_ARG;
    AdamScalars sc;
    if (!make_scalars(&sc, lr, beta1, beta2, eps, weight_decay, step)) return VPCE_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(p) | reinterpret_cast<uintptr_t>(m) | reinterpret_cast<uintptr_t>(v) |
         reinterpret_cast<uintptr_t>(g)) & 15u)
        return VPCE_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(w_bf16) & 7u) return VPCE_UNSUPPORTED;
    return launch_update(p, m, v, g, w_bf16, static_cast<long>(n), sc, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? VPCE_OK : VPCE_CUDA_ERROR;
}

}  // extern "C"
