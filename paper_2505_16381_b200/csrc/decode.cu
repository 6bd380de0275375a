// Decoding step with an in-place key cache (paper Sec. 3.4).
//
// The cache holds kc_j = H_{t-1} ... H_{j+1} k_j for every past position, in float32: when token t arrives every
// cached key gets kc_j <- H_t kc_j = kc_j - beta_t w_t (w_t . kc_j), then (k_t, v_t) are appended untouched, and the
// step's output is plain softmax attention of q_t over the cache.  The update and the attention are one pass over the
// cache (each key row is read once, updated, written back and used for its logit while still in registers), so the
// step is bound by memory bandwidth: 2 * 4 d bytes per cached key plus 2 d for its value.  The cache is float32
// because it is rewritten at every step: a bf16 cache would be rounded t times.
//
// One warp handles one cached key at a time, the head dimension spread over its lanes; a CTA covers 256 consecutive
// positions of one (batch, head) slice and leaves a partial softmax state (max, sum, weighted values), which a small
// second kernel merges over the CTAs of the slice.
#include "common.cuh"

namespace path {

namespace {

constexpr int kKeysPerCta = 256, kWarps = 8, kInFlight = 1;   // positions a warp has in flight at once

template <int E>
__device__ __forceinline__ void load_bf16(const __nv_bfloat16* p, int lane, float (&x)[E]) {
    if (E == 2) {
        const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p + lane * 2));
        x[0] = f.x; x[1] = f.y;
    } else {
        const uint2 u = *reinterpret_cast<const uint2*>(p + lane * 4);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
        x[0] = a.x; x[1] = a.y; x[E - 2] = b.x; x[E - 1] = b.y;
    }
}
template <int E>
__device__ __forceinline__ void load_f32(const float* p, int lane, float (&x)[E]) {
    if (E == 2) {
        const float2 f = *reinterpret_cast<const float2*>(p + lane * 2);
        x[0] = f.x; x[1] = f.y;
    } else {
        const float4 f = *reinterpret_cast<const float4*>(p + lane * 4);
        x[0] = f.x; x[1] = f.y; x[E - 2] = f.z; x[E - 1] = f.w;
    }
}
template <int E>
__device__ __forceinline__ void store_f32(float* p, int lane, const float (&x)[E]) {
    if (E == 2) *reinterpret_cast<float2*>(p + lane * 2) = make_float2(x[0], x[1]);
    else *reinterpret_cast<float4*>(p + lane * 4) = make_float4(x[0], x[1], x[E - 2], x[E - 1]);
}
__device__ __forceinline__ float warp_sum(float a) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
    return a;
}

// part: [S][nsplit][HD + 2] = (max, sum, weighted values) of each CTA's positions
template <int HD>
__global__ void __launch_bounds__(32 * kWarps) decode_update_kernel(
    const __nv_bfloat16* __restrict__ q_t, const __nv_bfloat16* __restrict__ k_t, const __nv_bfloat16* __restrict__ v_t,
    const __nv_bfloat16* __restrict__ w_t, const float* __restrict__ beta_t, const float* __restrict__ log_f_t, float* kc,
    __nv_bfloat16* vc, float* gc, int t, int cap, float scale, float* __restrict__ part) {
    constexpr int E = HD / 32;
    __shared__ float sm_m[kWarps], sm_l[kWarps], sm_acc[kWarps][HD];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int s = blockIdx.y, nsplit = gridDim.x;
    const int lo = blockIdx.x * kKeysPerCta, hi = min(lo + kKeysPerCta, t + 1);
    float q[E], w[E];
    load_bf16<E>(q_t + (size_t)s * HD, lane, q);
    load_bf16<E>(w_t + (size_t)s * HD, lane, w);
    const float b = beta_t[s];
    float qw = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) qw = fmaf(q[e], w[e], qw);
    qw = warp_sum(qw);
    const float Gt = gc ? ((t > 0 ? gc[(size_t)s * cap + t - 1] : 0.f) + log_f_t[s]) : 0.f;
    float* kcs = kc + (size_t)s * cap * HD;
    __nv_bfloat16* vcs = vc + (size_t)s * cap * HD;
    float m = -INFINITY, l = 0.f, acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;

    // several positions per iteration, so that a warp has that many rows of keys and values in flight
    for (int i0 = lo + warp; i0 < hi; i0 += kInFlight * kWarps) {
        float kk[kInFlight][E], vv[kInFlight][E], Gi[kInFlight], sc[kInFlight];
        bool live[kInFlight];
#pragma unroll
        for (int x = 0; x < kInFlight; ++x) {
            const int i = i0 + x * kWarps;
            live[x] = i < hi;
            Gi[x] = 0.f;
            if (!live[x]) continue;
            if (i < t) {
                load_f32<E>(kcs + (size_t)i * HD, lane, kk[x]);
                load_bf16<E>(vcs + (size_t)i * HD, lane, vv[x]);
                if (gc) Gi[x] = gc[(size_t)s * cap + i];
            } else {   // the new token: appended as it is
                load_bf16<E>(k_t + (size_t)s * HD, lane, kk[x]);
                load_bf16<E>(v_t + (size_t)s * HD, lane, vv[x]);
            }
        }
#pragma unroll
        for (int x = 0; x < kInFlight; ++x) {
            if (!live[x]) continue;
            const int i = i0 + x * kWarps;
            float a = 0.f, c = 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                a = fmaf(q[e], kk[x][e], a);
                c = fmaf(w[e], kk[x][e], c);
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
                a += __shfl_xor_sync(0xffffffffu, a, off);
                c += __shfl_xor_sync(0xffffffffu, c, off);
            }
            if (i < t) {   // kc_i <- H_t kc_i; its logit follows from the two dot products already known
                const float coef = b * c;
#pragma unroll
                for (int e = 0; e < E; ++e) kk[x][e] = fmaf(-coef, w[e], kk[x][e]);
                store_f32<E>(kcs + (size_t)i * HD, lane, kk[x]);
                sc[x] = fmaf(scale, a - coef * qw, Gt - Gi[x]);
            } else {
                store_f32<E>(kcs + (size_t)i * HD, lane, kk[x]);
                if (E == 2) {
                    *reinterpret_cast<__nv_bfloat162*>(vcs + (size_t)i * HD + lane * 2) = __floats2bfloat162_rn(vv[x][0], vv[x][1]);
                } else {
                    __nv_bfloat162 p0 = __floats2bfloat162_rn(vv[x][0], vv[x][1]), p1 = __floats2bfloat162_rn(vv[x][E - 2], vv[x][E - 1]);
                    uint2 u;
                    u.x = *reinterpret_cast<uint32_t*>(&p0); u.y = *reinterpret_cast<uint32_t*>(&p1);
                    *reinterpret_cast<uint2*>(vcs + (size_t)i * HD + lane * 4) = u;
                }
                if (gc && lane == 0) gc[(size_t)s * cap + i] = Gt;
                sc[x] = scale * a;
            }
            if (sc[x] > m) {   // warp-uniform
                const float r = expf(m - sc[x]);
                l *= r;
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] *= r;
                m = sc[x];
            }
            const float pj = expf(sc[x] - m);
            l += pj;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] = fmaf(pj, vv[x][e], acc[e]);
        }
    }
    // merge the warps of the CTA
    if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; }
#pragma unroll
    for (int e = 0; e < E; ++e) sm_acc[warp][lane * E + e] = acc[e];
    __syncthreads();
    float M = -INFINITY;
#pragma unroll
    for (int x = 0; x < kWarps; ++x) M = fmaxf(M, sm_m[x]);
    float* out = part + ((size_t)s * nsplit + blockIdx.x) * (HD + 2);
    if (threadIdx.x < HD) {
        float a = 0.f;
#pragma unroll
        for (int x = 0; x < kWarps; ++x) a += sm_acc[x][threadIdx.x] * expf(sm_m[x] - M);   // an idle warp has max = -inf: factor 0
        out[2 + threadIdx.x] = a;
    }
    if (threadIdx.x == 0) {
        float a = 0.f;
#pragma unroll
        for (int x = 0; x < kWarps; ++x) a += sm_l[x] * expf(sm_m[x] - M);
        out[0] = M; out[1] = a;
    }
}

template <int HD>
__global__ void __launch_bounds__(HD) decode_merge_kernel(const float* __restrict__ part, int nsplit, __nv_bfloat16* __restrict__ o_t,
                                                         float* __restrict__ lse_t) {
    const int s = blockIdx.x;
    const float* p = part + (size_t)s * nsplit * (HD + 2);
    float M = -INFINITY;
    for (int c = 0; c < nsplit; ++c) M = fmaxf(M, p[(size_t)c * (HD + 2)]);
    float l = 0.f, a = 0.f;
    for (int c = 0; c < nsplit; ++c) {
        const float f = expf(p[(size_t)c * (HD + 2)] - M);
        l += p[(size_t)c * (HD + 2) + 1] * f;
        a += p[(size_t)c * (HD + 2) + 2 + threadIdx.x] * f;
    }
    o_t[(size_t)s * HD + threadIdx.x] = __float2bfloat16_rn(a / l);
    if (threadIdx.x == 0) lse_t[s] = M + logf(l);
}

}  // namespace

size_t decode_partials_bytes(int S, int cap, int hd) {
    const size_t nsplit = ((size_t)cap + kKeysPerCta - 1) / kKeysPerCta;
    return (size_t)S * nsplit * (hd + 2) * sizeof(float);
}

cudaError_t launch_decode_step(const void* q_t, const void* k_t, const void* v_t, const void* w_t, const float* beta_t,
                               const float* log_f_t, float* kc, void* vc, float* gc, int t, int cap, void* o_t, float* lse_t,
                               int S, int hd, float scale, float* part, cudaStream_t st) {
    typedef __nv_bfloat16 bf;
    const int nsplit = (t + 1 + kKeysPerCta - 1) / kKeysPerCta;
    const dim3 grid(nsplit, S);
    if (hd == 64) {
        decode_update_kernel<64><<<grid, 32 * kWarps, 0, st>>>((const bf*)q_t, (const bf*)k_t, (const bf*)v_t, (const bf*)w_t, beta_t,
                                                               log_f_t, kc, (bf*)vc, gc, t, cap, scale, part);
        decode_merge_kernel<64><<<S, 64, 0, st>>>(part, nsplit, (bf*)o_t, lse_t);
    } else {
        decode_update_kernel<128><<<grid, 32 * kWarps, 0, st>>>((const bf*)q_t, (const bf*)k_t, (const bf*)v_t, (const bf*)w_t, beta_t,
                                                                log_f_t, kc, (bf*)vc, gc, t, cap, scale, part);
        decode_merge_kernel<128><<<S, 128, 0, st>>>(part, nsplit, (bf*)o_t, lse_t);
    }
    return cudaGetLastError();
}

}  // namespace path
