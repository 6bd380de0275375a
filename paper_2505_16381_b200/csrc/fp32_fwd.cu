// Forward pass for float32 tensors (PATH_FP32): the definition itself, in float32 on the CUDA cores.
//
// One warp owns one query position i and walks the keys j = i, i-1, ..., 0 carrying u_{i,j} = H_{j+1} ... H_i q_i
// (paper Sec. 2.2: logit s_ij = scale * k_j . u_{i,j} + G_i - G_j, then u <- u - beta_j w_j (w_j . u)), with an online
// softmax over j.  The head dimension is spread over the lanes; the two dot products of a step are reduced together
// by one butterfly.  O(L^2 d) work with a serial chain per row: this is the accuracy path for float32 inputs (logits
// good to float32 rounding, where the bf16 tensor-core path would round the inputs), not a fast one.
#include "common.cuh"

namespace path {

namespace {

constexpr int kRowsPerCta = 8;

template <int HD>
__global__ void __launch_bounds__(32 * kRowsPerCta) fp32_fwd_kernel(const float* __restrict__ q, const float* __restrict__ k,
                                                                   const float* __restrict__ v, const float* __restrict__ w,
                                                                   const float* __restrict__ beta, const float* __restrict__ G,
                                                                   float* __restrict__ o, float* __restrict__ lse, int S, int L,
                                                                   int ldG, float scale) {
    constexpr int E = HD / 32;   // elements per lane
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nblk = (L + kRowsPerCta - 1) / kRowsPerCta;
    // long rows first, the slices of one row block side by side
    const int slice = blockIdx.x % S, blk = nblk - 1 - blockIdx.x / S;
    const int i = blk * kRowsPerCta + warp;
    if (i >= L) return;
    const size_t base = (size_t)slice * L;
    auto load = [&](const float* p, int pos, float (&x)[E]) {
        const float* r = p + (base + pos) * HD + lane * E;
        if (E == 2) {
            const float2 t = *reinterpret_cast<const float2*>(r);
            x[0] = t.x; x[1] = t.y;
        } else {
            const float4 t = *reinterpret_cast<const float4*>(r);
            x[0] = t.x; x[1] = t.y; x[E - 2] = t.z; x[E - 1] = t.w;
        }
    };
    float u[E], acc[E], kj[E], wj[E], vj[E];
    load(q, i, u);
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    const float Gi = G ? G[(size_t)slice * ldG + i] : 0.f;
    float m = -INFINITY, l = 0.f;
    load(k, i, kj); load(w, i, wj); load(v, i, vj);
    float bj = beta[base + i], Gj = Gi;
    for (int j = i; j >= 0; --j) {
        // the next key's row is requested before this step's reductions
        float kn[E], wn[E], vn[E], bn = 0.f, Gn = 0.f;
        if (j > 0) {
            load(k, j - 1, kn); load(w, j - 1, wn); load(v, j - 1, vn);
            bn = beta[base + j - 1];
            Gn = G ? G[(size_t)slice * ldG + j - 1] : 0.f;
        }
        float a = 0.f, t = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            a = fmaf(u[e], kj[e], a);
            t = fmaf(u[e], wj[e], t);
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, off);
            t += __shfl_xor_sync(0xffffffffu, t, off);
        }
        const float s = fmaf(scale, a, Gi - Gj);
        if (s > m) {   // warp-uniform: every lane holds the same s
            const float c = expf(m - s);
            l *= c;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] *= c;
            m = s;
        }
        const float pj = expf(s - m);
        l += pj;
        const float bt = bj * t;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            acc[e] = fmaf(pj, vj[e], acc[e]);
            u[e] = fmaf(-bt, wj[e], u[e]);
        }
        if (j > 0) {
#pragma unroll
            for (int e = 0; e < E; ++e) { kj[e] = kn[e]; wj[e] = wn[e]; vj[e] = vn[e]; }
            bj = bn; Gj = Gn;
        }
    }
    const float inv = 1.f / l;
    float* orow = o + (base + i) * HD + lane * E;
    if (E == 2) {
        *reinterpret_cast<float2*>(orow) = make_float2(acc[0] * inv, acc[1] * inv);
    } else {
        *reinterpret_cast<float4*>(orow) = make_float4(acc[0] * inv, acc[1] * inv, acc[E - 2] * inv, acc[E - 1] * inv);
    }
    if (lane == 0) lse[base + i] = m + logf(l);
}

}  // namespace

cudaError_t launch_fp32_fwd(const float* q, const float* k, const float* v, const float* w, const float* beta, const float* G,
                            float* o, float* lse, int S, int L, int ldG, int hd, float scale, cudaStream_t st) {
    const int nblk = (L + kRowsPerCta - 1) / kRowsPerCta;
    const dim3 grid((unsigned)((size_t)S * nblk));
    if (hd == 64)
        fp32_fwd_kernel<64><<<grid, 32 * kRowsPerCta, 0, st>>>(q, k, v, w, beta, G, o, lse, S, L, ldG, scale);
    else
        fp32_fwd_kernel<128><<<grid, 32 * kRowsPerCta, 0, st>>>(q, k, v, w, beta, G, o, lse, S, L, ldG, scale);
    return cudaGetLastError();
}

}  // namespace path
