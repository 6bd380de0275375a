// Decoding step with an in-place key cache (paper Sec. 3.4).
//
// The cache holds kc_j = H_{t-1} ... H_{j+1} k_j for every past position, in float32: when token t arrives every
// cached key gets kc_j <- H_t kc_j = kc_j - beta_t w_t (w_t . kc_j), then (k_t, v_t) are appended untouched, and the
// step's output is plain softmax attention of q_t over the cache.  The update and the attention are one pass over the
// cache (each key row is read once, updated, written back and used for its logit while still in registers), so the
// step is bound by memory bandwidth: 2 * 4 d bytes per cached key plus 2 d for its value.  The cache is float32
// because it is rewritten at every step: a bf16 cache would be rounded t times.
//
// One half-warp handles one cached key at a time, the head dimension spread over its 16 lanes; a CTA covers 256
// consecutive positions of one (batch, head) slice and leaves a partial softmax state (max, sum, weighted values), which
// a small second kernel merges over the CTAs of the slice.
#include "common.cuh"

namespace path {

namespace {

constexpr int kKeysPerCta = 256, kWarps = 8;

// part: [S][nsplit][HD + 2] = (max, sum, weighted values) of each CTA's positions
//
// A half-warp (16 lanes) owns one cached position at a time: lane j of the half holds the elements
// [4j, 4j+4) of every 64-element panel of the row (16-byte loads, a half-warp covers 256 contiguous bytes per
// instruction), so a warp has two key rows and two value rows in flight.
template <int HD>
__global__ void __launch_bounds__(32 * kWarps, 4) decode_update_kernel(
    const __nv_bfloat16* __restrict__ q_t, const __nv_bfloat16* __restrict__ k_t, const __nv_bfloat16* __restrict__ v_t,
    const __nv_bfloat16* __restrict__ w_t, const float* __restrict__ beta_t, const float* __restrict__ log_f_t, float* kc,
    __nv_bfloat16* vc, float* gc, int t, int cap, float scale, float* __restrict__ part) {
    constexpr int NP = HD / 64;          // 64-element panels per row
    constexpr int NH = 2 * kWarps;       // half-warps per CTA
    __shared__ float sm_m[NH], sm_l[NH], sm_acc[NH][HD];
    const int lane = threadIdx.x & 31, hl = lane & 15, hw = threadIdx.x >> 4;   // lane in the half-warp, half-warp in the CTA
    const int s = blockIdx.y, nsplit = gridDim.x;
    const int lo = blockIdx.x * kKeysPerCta, hi = min(lo + kKeysPerCta, t + 1);
    auto ld_bf16 = [&](const __nv_bfloat16* row, float (&x)[NP][4]) {
#pragma unroll
        for (int pn = 0; pn < NP; ++pn) {
            const uint2 u = *reinterpret_cast<const uint2*>(row + pn * 64 + hl * 4);
            const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
            const float2 b2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
            x[pn][0] = a.x; x[pn][1] = a.y; x[pn][2] = b2.x; x[pn][3] = b2.y;
        }
    };
    float q[NP][4], w[NP][4];
    ld_bf16(q_t + (size_t)s * HD, q);
    ld_bf16(w_t + (size_t)s * HD, w);
    const float b = beta_t[s];
    float qw = 0.f;
#pragma unroll
    for (int pn = 0; pn < NP; ++pn)
#pragma unroll
        for (int e = 0; e < 4; ++e) qw = fmaf(q[pn][e], w[pn][e], qw);
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) qw += __shfl_xor_sync(0xffffffffu, qw, off);
    const float Gt = gc ? ((t > 0 ? gc[(size_t)s * cap + t - 1] : 0.f) + log_f_t[s]) : 0.f;
    float* kcs = kc + (size_t)s * cap * HD;
    __nv_bfloat16* vcs = vc + (size_t)s * cap * HD;
    float m = -INFINITY, l = 0.f, acc[NP][4];
#pragma unroll
    for (int pn = 0; pn < NP; ++pn)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[pn][e] = 0.f;

    // both halves of a warp run the same number of iterations (the shuffles below name all 32 lanes)
    for (int i0 = lo; i0 < hi; i0 += NH) {
        const int i = i0 + hw;
        const bool live = i < hi;
        float kk[NP][4], vv[NP][4], Gi = 0.f;
        if (live) {
            if (i < t) {
#pragma unroll
                for (int pn = 0; pn < NP; ++pn) {
                    const float4 f = *reinterpret_cast<const float4*>(kcs + (size_t)i * HD + pn * 64 + hl * 4);
                    kk[pn][0] = f.x; kk[pn][1] = f.y; kk[pn][2] = f.z; kk[pn][3] = f.w;
                }
                ld_bf16(vcs + (size_t)i * HD, vv);
                if (gc) Gi = gc[(size_t)s * cap + i];
            } else {   // the new token: appended as it is
                ld_bf16(k_t + (size_t)s * HD, kk);
                ld_bf16(v_t + (size_t)s * HD, vv);
            }
        } else {
#pragma unroll
            for (int pn = 0; pn < NP; ++pn)
#pragma unroll
                for (int e = 0; e < 4; ++e) kk[pn][e] = vv[pn][e] = 0.f;
        }
        float a = 0.f, c = 0.f;
#pragma unroll
        for (int pn = 0; pn < NP; ++pn)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                a = fmaf(q[pn][e], kk[pn][e], a);
                c = fmaf(w[pn][e], kk[pn][e], c);
            }
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) {   // within the half-warp
            a += __shfl_xor_sync(0xffffffffu, a, off);
            c += __shfl_xor_sync(0xffffffffu, c, off);
        }
        if (!live) continue;
        float sc;
        if (i < t) {   // kc_i <- H_t kc_i; its logit follows from the two dot products already known
            const float coef = b * c;
#pragma unroll
            for (int pn = 0; pn < NP; ++pn) {
                float4 f;
                f.x = fmaf(-coef, w[pn][0], kk[pn][0]); f.y = fmaf(-coef, w[pn][1], kk[pn][1]);
                f.z = fmaf(-coef, w[pn][2], kk[pn][2]); f.w = fmaf(-coef, w[pn][3], kk[pn][3]);
                *reinterpret_cast<float4*>(kcs + (size_t)i * HD + pn * 64 + hl * 4) = f;
            }
            sc = fmaf(scale, a - coef * qw, Gt - Gi);
        } else {
#pragma unroll
            for (int pn = 0; pn < NP; ++pn) {
                *reinterpret_cast<float4*>(kcs + (size_t)i * HD + pn * 64 + hl * 4) =
                    make_float4(kk[pn][0], kk[pn][1], kk[pn][2], kk[pn][3]);
                __nv_bfloat162 p0 = __floats2bfloat162_rn(vv[pn][0], vv[pn][1]), p1 = __floats2bfloat162_rn(vv[pn][2], vv[pn][3]);
                uint2 u;
                u.x = *reinterpret_cast<uint32_t*>(&p0); u.y = *reinterpret_cast<uint32_t*>(&p1);
                *reinterpret_cast<uint2*>(vcs + (size_t)i * HD + pn * 64 + hl * 4) = u;
            }
            if (gc && hl == 0) gc[(size_t)s * cap + i] = Gt;
            sc = scale * a;
        }
        if (sc > m) {   // uniform over the half-warp
            const float r = expf(m - sc);
            l *= r;
#pragma unroll
            for (int pn = 0; pn < NP; ++pn)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[pn][e] *= r;
            m = sc;
        }
        const float pj = expf(sc - m);
        l += pj;
#pragma unroll
        for (int pn = 0; pn < NP; ++pn)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[pn][e] = fmaf(pj, vv[pn][e], acc[pn][e]);
    }
    // merge the half-warps of the CTA
    if (hl == 0) { sm_m[hw] = m; sm_l[hw] = l; }
#pragma unroll
    for (int pn = 0; pn < NP; ++pn)
#pragma unroll
        for (int e = 0; e < 4; ++e) sm_acc[hw][pn * 64 + hl * 4 + e] = acc[pn][e];
    __syncthreads();
    float M = -INFINITY;
#pragma unroll
    for (int x = 0; x < NH; ++x) M = fmaxf(M, sm_m[x]);
    float* out = part + ((size_t)s * nsplit + blockIdx.x) * (HD + 2);
    if (threadIdx.x < HD) {
        float a = 0.f;
#pragma unroll
        for (int x = 0; x < NH; ++x) a += sm_acc[x][threadIdx.x] * expf(sm_m[x] - M);   // an idle half-warp has max = -inf: factor 0
        out[2 + threadIdx.x] = a;
    }
    if (threadIdx.x == 0) {
        float a = 0.f;
#pragma unroll
        for (int x = 0; x < NH; ++x) a += sm_l[x] * expf(sm_m[x] - M);
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
