// Layer front-end of the operator (paper Sec. 2.2, footnote to the definition of H_t; gate of Sec. 2.4):
//   w_t    = L2-normalise( short convolution, 3 taps, of z_t )      z = output of the low-rank linear layer (a library GEMM)
//   beta_t = 2 sigmoid(beta_logit_t),   log f_t = log sigmoid(gate_logit_t)
// and its backward.  The convolution is causal and depthwise (tap j multiplies z_{t-2+j}, zeros before the sequence), the
// normalisation is per head over its d channels with eps under the root.  Everything here is elementwise work with a
// 2-row halo, bound by memory bandwidth: each kernel reads its inputs once and also does the [B,L,H*d] -> [B,H,L,d]
// change of layout that the operator wants, so no separate transpose pass exists.
//
// Work split.  A lane holds 8 adjacent channels of a row (one 16-byte load), so a row of a head takes d/8 lanes and a
// warp holds 32/(d/8) lane groups.  Each group walks over R consecutive positions (5 or 8, see FwdR / BwdR) with the
// filter's window in registers.  The rows a lane will need are fetched by 16-byte asynchronous copies into a slot of
// shared memory that only this lane reads back (a per-lane queue, so no barrier is involved: the lane waits for its own
// copy group), one position block ahead of the one being computed: the bytes in flight, which is what a
// bandwidth-bound kernel lives on, sit in shared memory instead of registers.  A CTA is 4 warps = 4 * (256 / d) * R
// consecutive positions of one head; CTAs are numbered with the head fastest, so the CTAs that run at the same time
// read whole contiguous rows of z between them, and each loops over the position blocks of its head with a stride (the
// backward keeps its filter-gradient sums in registers across that loop and adds them to global memory once).
#include "common.cuh"

namespace path {

namespace {

constexpr int kWarps = 4;   // warps per CTA

template <int HD, int R>   // R = consecutive positions per lane group
struct Geo {
    static constexpr int LPR = HD / 8;        // lanes per row
    static constexpr int G = 32 / LPR;        // lane groups per warp
    static constexpr int ROWS_W = G * R;      // positions per warp
    static constexpr int ROWS_CTA = kWarps * ROWS_W;
    static_assert(ROWS_W <= 32, "one lane per position fetches its scalars");
};
// Positions per lane group, by measurement (TB/s of algorithmic bytes at B=32 H=32 L=4096 d=64 / B=8 H=32 L=8192 d=128):
// forward d = 64: 5.3 / 5.7 / 4.9 at 4 / 5 / 8;  forward d = 128: 5.5 / 5.9 / 5.8 at 5 / 6 / 8;
// backward d = 64: 3.4 / 3.9 / 4.2 at 5 / 6 / 8;  backward d = 128: 3.7 / 4.0 / 4.0 at 5 / 8 / 10.
template <int HD> struct FwdR { static constexpr int value = HD == 64 ? 5 : 8; };
template <int HD> struct BwdR { static constexpr int value = 8; };

// 16-byte asynchronous copy global -> shared; copies nothing and writes zeros when `valid` is false
__device__ __forceinline__ void cp_async16(uint4* dst, const void* src, bool valid) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src),
                 "r"(valid ? 16 : 0)
                 : "memory");
}
// 4-byte flavour for the per-position scalars
__device__ __forceinline__ void cp_async4(float* dst, const float* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// Two float32 lanes per instruction (fma.rn.f32x2 and friends): this kernel's arithmetic is all elementwise on 8
// channels per lane, and at d/8 lanes per row the instruction issue rate, not the memory, would otherwise set the pace.
typedef unsigned long long u64;
__device__ __forceinline__ u64 pk(float2 v) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(v.x), "f"(v.y));
    return r;
}
__device__ __forceinline__ float2 upk(u64 r) {
    float2 v;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(v.x), "=f"(v.y) : "l"(r));
    return v;
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(pk(a)), "l"(pk(b)), "l"(pk(c)));
    return upk(d);
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
    u64 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pk(a)), "l"(pk(b)));
    return upk(d);
}
__device__ __forceinline__ float2 bc(float x) { return make_float2(x, x); }

__device__ __forceinline__ void unpack8(const uint4& r, float2 (&x)[4]) {
    const uint32_t u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) x[i] = make_float2(__uint_as_float(u[i] << 16), __uint_as_float(u[i] & 0xffff0000u));
}
__device__ __forceinline__ void st16(__nv_bfloat16* p, const float2 (&x)[4]) {
    uint32_t r[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(x[i].x, x[i].y);
        r[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(r[0], r[1], r[2], r[3]);
}
__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + expf(-x)); }

constexpr int kThreads = 32 * kWarps;
constexpr int kFwdStages = 2, kBwdStages = 2;
__host__ __device__ constexpr int fwd_rows(int R) { return R + 2; }               // z rows t0-2 .. t0+R-1 per lane and block
__host__ __device__ constexpr int bwd_rows(int R) { return (R + 4) + (R + 2); }   // z rows t0-2 .. t0+R+1, then dw rows t0 .. t0+R+1

template <int HD>
__global__ void __launch_bounds__(kThreads, 4) frontend_fwd_kernel(
    const __nv_bfloat16* __restrict__ z, const float* __restrict__ cw, const float* __restrict__ bl, const float* __restrict__ gl,
    __nv_bfloat16* __restrict__ w, float* __restrict__ beta, float* __restrict__ logf, int B, int H, int L, int nblk, float eps) {
    constexpr int kR = FwdR<HD>::value, kFwdRows = fwd_rows(kR);
    typedef Geo<HD, kR> Ge;
    extern __shared__ uint4 queue[];   // [stage][row][thread]: every slot is written and read by the same thread
    float* lq = reinterpret_cast<float*>(queue + kFwdStages * kFwdRows * kThreads);   // [stage][beta, gate logit][thread]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, grp = lane / Ge::LPR, li = lane % Ge::LPR;
    const int h = blockIdx.x % H, W = gridDim.x / H, nitems = B * nblk, first = blockIdx.x / H;
    const size_t C = (size_t)H * HD;
    float2 c[4][3];   // taps of the lane's 8 channels, channel pairs packed
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            const float* cp = cw + ((size_t)h * HD + li * 8 + 2 * e) * 3 + j;
            c[e][j] = make_float2(cp[0], cp[3]);
        }
    // requests the rows of block `blk` into `stage`; always closes a copy group so that every thread counts alike
    auto request = [&](int blk, int stage) {
        if (blk < nitems) {
            const int b = blk / nblk, t0 = (blk % nblk) * Ge::ROWS_CTA + warp * Ge::ROWS_W + grp * kR;
            const __nv_bfloat16* zp = z + (size_t)b * L * C + (size_t)h * HD + li * 8;
#pragma unroll
            for (int i = 0; i < kFwdRows; ++i) {
                const int t = t0 - 2 + i;
                const bool in = t >= 0 && t < L;
                cp_async16(&queue[(stage * kFwdRows + i) * kThreads + threadIdx.x], in ? zp + (size_t)t * C : z, in);
            }
            const int t = t0 - grp * kR + lane;   // lane i of a warp also fetches the two logits of the warp's i-th position
            if (lane < Ge::ROWS_W && t < L) {
                const size_t src = ((size_t)b * L + t) * H + h;
                cp_async4(&lq[(stage * 2 + 0) * kThreads + threadIdx.x], bl + src);
                if (gl) cp_async4(&lq[(stage * 2 + 1) * kThreads + threadIdx.x], gl + src);
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < kFwdStages - 1; ++s) request(first + s * W, s);
    int it = 0;
    for (int blk = first; blk < nitems; blk += W, ++it) {
        request(blk + (kFwdStages - 1) * W, (it + kFwdStages - 1) % kFwdStages);
        cp_async_wait<kFwdStages - 1>();
        const uint4* rows = &queue[((it % kFwdStages) * kFwdRows) * kThreads + threadIdx.x];
        const int b = blk / nblk, tw = (blk % nblk) * Ge::ROWS_CTA + warp * Ge::ROWS_W;   // the warp's first position
        if (tw >= L) continue;
        const int bh = b * H + h, t0 = tw + grp * kR;                                     // the group's first position
        __nv_bfloat16* wp = w + (size_t)bh * L * HD + li * 8;
        float2 a0[4], a1[4], a2[4];
        unpack8(rows[0], a0);
        unpack8(rows[kThreads], a1);
#pragma unroll
        for (int i = 0; i < kR; ++i) {
            const int t = t0 + i;
            unpack8(rows[(i + 2) * kThreads], a2);
            float2 y[4], ss2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                y[e] = fma2(c[e][2], a2[e], fma2(c[e][1], a1[e], mul2(c[e][0], a0[e])));
                ss2 = fma2(y[e], y[e], ss2);
            }
            float ss = ss2.x + ss2.y;
#pragma unroll
            for (int off = Ge::LPR / 2; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
            const float2 r = bc(rsqrtf(ss + eps));
#pragma unroll
            for (int e = 0; e < 4; ++e) y[e] = mul2(y[e], r);
            if (t < L) st16(wp + (size_t)t * HD, y);   // rows past the end were computed from zeros and are dropped
#pragma unroll
            for (int e = 0; e < 4; ++e) { a0[e] = a1[e]; a1[e] = a2[e]; }
        }
        if (lane < Ge::ROWS_W && tw + lane < L) {   // the two scalars of each position, logits [b, t, h] -> [b, h, t]
            const size_t dst = (size_t)bh * L + tw + lane;
            const float* lg = &lq[((it % kFwdStages) * 2) * kThreads + threadIdx.x];
            beta[dst] = 2.f * sigmoidf_(lg[0]);
            if (gl) {
                const float x = lg[kThreads];
                logf[dst] = fminf(x, 0.f) - log1pf(expf(-fabsf(x)));
            }
        }
    }
    cp_async_wait<0>();
}

// Backward.  dy_s = r_s dw_s - r_s^3 y_s (y_s . dw_s) needs y_s again, which is recomputed from z; dz_t collects dy_t,
// dy_{t+1}, dy_{t+2}, so a group runs two positions past its own 8 (their dy only feeds its own dz rows).  The filter
// gradient counts every position once, in the group that owns it; the sums stay in registers over the CTA's whole loop,
// are then added up over the CTA's groups in shared memory and leave as one float32 atomic per (channel, tap) per CTA.
template <int HD>
__global__ void __launch_bounds__(kThreads, 2) frontend_bwd_kernel(
    const __nv_bfloat16* __restrict__ z, const float* __restrict__ cw, const float* __restrict__ bl, const float* __restrict__ gl,
    const __nv_bfloat16* __restrict__ dw, const float* __restrict__ dbeta, const float* __restrict__ dlogf,
    __nv_bfloat16* __restrict__ dz, float* dcw, float* __restrict__ dbl, float* __restrict__ dgl, int B, int H, int L, int nblk,
    float eps) {
    constexpr int kR = BwdR<HD>::value, kBwdRows = bwd_rows(kR);
    typedef Geo<HD, kR> Ge;
    extern __shared__ uint4 queue[];   // [stage][row][thread]; reused for the reduction of the filter gradient at the end
    float* lq = reinterpret_cast<float*>(queue + kBwdStages * kBwdRows * kThreads);   // [stage][4 scalars][thread]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, grp = lane / Ge::LPR, li = lane % Ge::LPR;
    const int h = blockIdx.x % H, W = gridDim.x / H, nitems = B * nblk, first = blockIdx.x / H;
    const size_t C = (size_t)H * HD;
    float2 c[4][3], gcw[4][3];   // taps and their gradient sums for the lane's 8 channels, channel pairs packed
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            const float* cp = cw + ((size_t)h * HD + li * 8 + 2 * e) * 3 + j;
            c[e][j] = make_float2(cp[0], cp[3]);
            gcw[e][j] = make_float2(0.f, 0.f);
        }
    auto request = [&](int blk, int stage) {
        if (blk < nitems) {
            const int b = blk / nblk, t0 = (blk % nblk) * Ge::ROWS_CTA + warp * Ge::ROWS_W + grp * kR;
            const __nv_bfloat16* zp = z + (size_t)b * L * C + (size_t)h * HD + li * 8;
            const __nv_bfloat16* gp = dw + (size_t)(b * H + h) * L * HD + li * 8;
            uint4* q = &queue[(stage * kBwdRows) * kThreads + threadIdx.x];
#pragma unroll
            for (int i = 0; i < kR + 4; ++i) {
                const int t = t0 - 2 + i;
                const bool in = t >= 0 && t < L;
                cp_async16(q + i * kThreads, in ? zp + (size_t)t * C : z, in);
            }
#pragma unroll
            for (int i = 0; i < kR + 2; ++i) {
                const int t = t0 + i;
                const bool in = t < L;
                cp_async16(q + (kR + 4 + i) * kThreads, in ? gp + (size_t)t * HD : dw, in);
            }
            const int t = t0 - grp * kR + lane;   // lane i of a warp also fetches the scalars of the warp's i-th position
            if (lane < Ge::ROWS_W && t < L) {
                const size_t lsrc = ((size_t)b * L + t) * H + h, gsrc = (size_t)(b * H + h) * L + t;
                float* lg = &lq[(stage * 4) * kThreads + threadIdx.x];
                cp_async4(lg, bl + lsrc);
                cp_async4(lg + kThreads, dbeta + gsrc);
                if (gl) {
                    cp_async4(lg + 2 * kThreads, gl + lsrc);
                    cp_async4(lg + 3 * kThreads, dlogf + gsrc);
                }
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < kBwdStages - 1; ++s) request(first + s * W, s);
    int it = 0;
    for (int blk = first; blk < nitems; blk += W, ++it) {
        request(blk + (kBwdStages - 1) * W, (it + kBwdStages - 1) % kBwdStages);
        cp_async_wait<kBwdStages - 1>();
        const uint4* rows = &queue[((it % kBwdStages) * kBwdRows) * kThreads + threadIdx.x];
        const uint4* grows = rows + (kR + 4) * kThreads;
        const int b = blk / nblk, tw = (blk % nblk) * Ge::ROWS_CTA + warp * Ge::ROWS_W;
        if (tw >= L) continue;
        const int t0 = tw + grp * kR;
        __nv_bfloat16* dzp = dz + (size_t)b * L * C + (size_t)h * HD + li * 8;
        float2 a0[4], a1[4], a2[4], dy0[4], dy1[4], dy2[4];
        unpack8(rows[0], a0);
        unpack8(rows[kThreads], a1);
#pragma unroll
        for (int e = 0; e < 4; ++e) dy0[e] = dy1[e] = make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < kR + 2; ++i) {
            const int s = t0 + i;
            float2 y[4], g[4], ss2 = make_float2(0.f, 0.f), dot2 = make_float2(0.f, 0.f);
            unpack8(rows[(i + 2) * kThreads], a2);
            unpack8(grows[i * kThreads], g);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                y[e] = fma2(c[e][2], a2[e], fma2(c[e][1], a1[e], mul2(c[e][0], a0[e])));
                ss2 = fma2(y[e], y[e], ss2);
                dot2 = fma2(y[e], g[e], dot2);
            }
            float ss = ss2.x + ss2.y, dot = dot2.x + dot2.y;
#pragma unroll
            for (int off = Ge::LPR / 2; off >= 1; off >>= 1) {
                ss += __shfl_xor_sync(0xffffffffu, ss, off);
                dot += __shfl_xor_sync(0xffffffffu, dot, off);
            }
            // positions past the end contribute nothing (their r may be inf when eps = 0): r = 0 makes dy = 0
            const float r = s < L ? rsqrtf(ss + eps) : 0.f;
            const float2 r2 = bc(r), nr3d = bc(-(r * r * r * dot));
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                dy2[e] = fma2(r2, g[e], mul2(nr3d, y[e]));
                if (i < kR) {
                    gcw[e][0] = fma2(dy2[e], a0[e], gcw[e][0]);
                    gcw[e][1] = fma2(dy2[e], a1[e], gcw[e][1]);
                    gcw[e][2] = fma2(dy2[e], a2[e], gcw[e][2]);
                }
            }
            if (i >= 2 && s - 2 < L) {   // dz_{s-2} = cw2 dy_{s-2} + cw1 dy_{s-1} + cw0 dy_s
                float2 o[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) o[e] = fma2(c[e][0], dy2[e], fma2(c[e][1], dy1[e], mul2(c[e][2], dy0[e])));
                st16(dzp + (size_t)(s - 2) * C, o);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) { dy0[e] = dy1[e]; dy1[e] = dy2[e]; a0[e] = a1[e]; a1[e] = a2[e]; }
        }
        if (lane < Ge::ROWS_W && tw + lane < L) {
            const size_t dst = ((size_t)b * L + tw + lane) * H + h;
            const float* lg = &lq[((it % kBwdStages) * 4) * kThreads + threadIdx.x];
            const float sg = sigmoidf_(lg[0]);
            dbl[dst] = lg[kThreads] * 2.f * sg * (1.f - sg);
            if (gl) dgl[dst] = lg[3 * kThreads] * sigmoidf_(-lg[2 * kThreads]);
        }
    }
    cp_async_wait<0>();
    __syncthreads();   // the queue is free: [group][channel][tap] partial sums
    float* sred = reinterpret_cast<float*>(queue);
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            float* dst = sred + (warp * Ge::G + grp) * HD * 3 + (li * 8 + 2 * e) * 3 + j;
            dst[0] = gcw[e][j].x;
            dst[3] = gcw[e][j].y;
        }
    __syncthreads();
    for (int idx = threadIdx.x; idx < HD * 3; idx += kThreads) {
        float a = 0.f;
#pragma unroll
        for (int x = 0; x < kWarps * Ge::G; ++x) a += sred[x * HD * 3 + idx];
        atomicAdd(dcw + (size_t)h * HD * 3 + idx, a);
    }
}

// CTAs per head: as many as fit on the device at once at `per_sm` resident CTAs per SM (rounded down: one CTA too
// many would run alone in a second wave and double the time), at least one, never more than there are blocks
cudaError_t ctas_per_head(int B, int H, int nblk, int per_sm, int* out) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    long long want = (long long)sms * per_sm / H;
    if (want < 1) want = 1;
    const long long items = (long long)B * nblk;
    *out = (int)(items < want ? items : want);
    return cudaSuccess;
}

}  // namespace

cudaError_t launch_frontend_fwd(const void* z, const float* cw, const float* bl, const float* gl, void* w, float* beta,
                                float* logf, int B, int H, int L, int hd, float eps, cudaStream_t st) {
    typedef __nv_bfloat16 bf;
    const int rows = hd == 64 ? Geo<64, FwdR<64>::value>::ROWS_CTA : Geo<128, FwdR<128>::value>::ROWS_CTA;
    const int nblk = (L + rows - 1) / rows;
    int W = 1;
    cudaError_t e = ctas_per_head(B, H, nblk, 4, &W);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)((size_t)H * W));
    auto smem_of = [](int R) { return kFwdStages * (fwd_rows(R) * (int)sizeof(uint4) + 2 * (int)sizeof(float)) * kThreads; };
    const int smem = smem_of(hd == 64 ? FwdR<64>::value : FwdR<128>::value);
    if (hd == 64) {
        e = cudaFuncSetAttribute(frontend_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        frontend_fwd_kernel<64><<<grid, kThreads, smem, st>>>((const bf*)z, cw, bl, gl, (bf*)w, beta, logf, B, H, L, nblk, eps);
    } else {
        e = cudaFuncSetAttribute(frontend_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        frontend_fwd_kernel<128><<<grid, kThreads, smem, st>>>((const bf*)z, cw, bl, gl, (bf*)w, beta, logf, B, H, L, nblk, eps);
    }
    return cudaGetLastError();
}

cudaError_t launch_frontend_bwd(const void* z, const float* cw, const float* bl, const float* gl, const void* dw,
                                const float* dbeta, const float* dlogf, void* dz, float* dcw, float* dbl, float* dgl, int B,
                                int H, int L, int hd, float eps, cudaStream_t st) {
    typedef __nv_bfloat16 bf;
    const int rows = hd == 64 ? Geo<64, BwdR<64>::value>::ROWS_CTA : Geo<128, BwdR<128>::value>::ROWS_CTA;
    const int nblk = (L + rows - 1) / rows;
    int W = 1;
    cudaError_t e = ctas_per_head(B, H, nblk, 2, &W);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)((size_t)H * W));
    auto smem_of = [](int R) { return kBwdStages * (bwd_rows(R) * (int)sizeof(uint4) + 4 * (int)sizeof(float)) * kThreads; };
    const int smem = smem_of(hd == 64 ? BwdR<64>::value : BwdR<128>::value);
    static_assert(kBwdStages * bwd_rows(1) * (int)sizeof(uint4) * kThreads >= kWarps * 4 * 64 * 3 * (int)sizeof(float) &&
                      kBwdStages * bwd_rows(1) * (int)sizeof(uint4) * kThreads >= kWarps * 2 * 128 * 3 * (int)sizeof(float),
                  "the queue also holds the filter-gradient partials");
    if (hd == 64) {
        e = cudaFuncSetAttribute(frontend_bwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        frontend_bwd_kernel<64><<<grid, kThreads, smem, st>>>((const bf*)z, cw, bl, gl, (const bf*)dw, dbeta, dlogf, (bf*)dz, dcw,
                                                           dbl, dgl, B, H, L, nblk, eps);
    } else {
        e = cudaFuncSetAttribute(frontend_bwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        frontend_bwd_kernel<128><<<grid, kThreads, smem, st>>>((const bf*)z, cw, bl, gl, (const bf*)dw, dbeta, dlogf, (bf*)dz, dcw,
                                                            dbl, dgl, B, H, L, nblk, eps);
    }
    return cudaGetLastError();
}

}  // namespace path
