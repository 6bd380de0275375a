// Memory-bound helpers: zero-padding of ragged inputs, prefix sum of the log gate (PaTH-FoX, paper Sec. 2.2),
// suffix sum of its gradient, row sums of the diagonal-chunk dS.
#include "linear.cuh"
#include "tc5.cuh"

namespace path {

namespace {

__global__ void pad_rows_kernel(const void* __restrict__ src, void* __restrict__ dst, int L, int Lp, int rowbytes16) {
    // one 16-byte vector per thread; grid.y = slice, grid.x covers Lp * rowbytes16
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    const long total = (long)Lp * rowbytes16;
    if (i >= total) return;
    const long row = i / rowbytes16, col = i % rowbytes16;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < L) v = ((const uint4*)src)[((long)blockIdx.y * L + row) * rowbytes16 + col];
    ((uint4*)dst)[((long)blockIdx.y * Lp + row) * rowbytes16 + col] = v;
}

__global__ void pad_vec_kernel(const float* __restrict__ src, float* __restrict__ dst, int L, int Lp) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < Lp) dst[(size_t)blockIdx.y * Lp + i] = (i < L) ? src[(size_t)blockIdx.y * L + i] : 0.f;
}

// One CTA (1024 threads) per slice: each thread scans a contiguous segment, then a block scan of the segment sums.
__global__ void __launch_bounds__(1024) gate_prefix_kernel(const float* __restrict__ g, float* __restrict__ G, int L,
                                                           int Lp) {
    __shared__ float part[1024];
    const int tid = threadIdx.x;
    const int seg = (Lp + 1023) / 1024;
    const int lo = tid * seg, hi = min(lo + seg, Lp);
    const float* gs = g + (size_t)blockIdx.x * L;
    float* Gs = G + (size_t)blockIdx.x * Lp;
    float acc = 0.f;
    for (int i = lo; i < hi; ++i) acc += (i < L) ? gs[i] : 0.f;
    part[tid] = acc;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        float v = (tid >= off) ? part[tid - off] : 0.f;
        __syncthreads();
        part[tid] += v;
        __syncthreads();
    }
    acc = (tid > 0) ? part[tid - 1] : 0.f;
    for (int i = lo; i < hi; ++i) {
        acc += (i < L) ? gs[i] : 0.f;
        Gs[i] = acc;
    }
}

// rs[chunk*128 + i] = sum_k dsd[chunk][i][k]; one warp per row (a lane reads four adjacent entries), four rows in flight.
__global__ void __launch_bounds__(256) dsd_rowsum_kernel(const float* __restrict__ dsd, float* __restrict__ rs) {
    const float4* base = reinterpret_cast<const float4*>(dsd + (size_t)blockIdx.x * CHUNK * CHUNK);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll 1
    for (int r0 = warp * 16; r0 < warp * 16 + 16; r0 += 4) {
        float4 v[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) v[x] = base[(r0 + x) * (CHUNK / 4) + lane];
        float acc[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) acc[x] = (v[x].x + v[x].y) + (v[x].z + v[x].w);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1)
#pragma unroll
            for (int x = 0; x < 4; ++x) acc[x] += __shfl_xor_sync(0xffffffffu, acc[x], off);
        if (lane < 4)
            rs[(size_t)blockIdx.x * CHUNK + r0 + lane] = lane == 0 ? acc[0] : lane == 1 ? acc[1] : lane == 2 ? acc[2] : acc[3];
    }
}

// dlog_f[t] = sum_{m >= t} (dGa + dGb + dGc)[m]: reverse inclusive scan per slice (inputs [S][Lp], output [S][L]).
__global__ void __launch_bounds__(1024) gate_suffix_kernel(const float* __restrict__ dGa, const float* __restrict__ dGb,
                                                           const float* __restrict__ dGc, float* __restrict__ out, int L,
                                                           int Lp) {
    __shared__ float part[1024];
    const int tid = threadIdx.x;
    const int seg = (L + 1023) / 1024;
    const int hi = L - tid * seg, lo = max(hi - seg, 0);  // this thread owns positions [lo, hi), scanning downwards
    const size_t so = (size_t)blockIdx.x * Lp;
    float* os = out + (size_t)blockIdx.x * L;
    float acc = 0.f;
    for (int i = hi - 1; i >= lo; --i) acc += (dGa[so + i] + dGb[so + i]) + dGc[so + i];
    part[tid] = acc;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        float v = (tid >= off) ? part[tid - off] : 0.f;
        __syncthreads();
        part[tid] += v;
        __syncthreads();
    }
    acc = (tid > 0) ? part[tid - 1] : 0.f;
    for (int i = hi - 1; i >= lo; --i) {
        acc += (dGa[so + i] + dGb[so + i]) + dGc[so + i];
        os[i] = acc;
    }
}

// ---- block skipping for gated problems (the paper notes that PaTH-FoX keeps FoX's pruning of negligible blocks)
//
// |k_j^T (H_{j+1} ... H_i) q_i| <= |k_j| |q_i| prod_s max(1, |1 - beta_s |w_s|^2|)   (each factor bounds the 2-norm of H_s;
// it is 1 whenever 0 <= beta_s |w_s|^2 <= 2), and every row's largest logit is at least its own diagonal one,
// s_ii = scale q_i . k_i.  So if for a pair of chunks (I, J)
//     |scale| max_I|q| max_J|k| exp(sum of the log factors over chunks J..I) + max_I G - min_J G  <  min_I s_ii - kSkipMargin
// every probability of the pair is below exp(-kSkipMargin) of its row's normaliser and the pair can be left out.  A
// query chunk keeps the key chunks up to the farthest one that fails this test.
constexpr float kSkipMargin = 30.f;   // exp(-30) ~ 1e-13 per logit, far below bf16 resolution even summed over a long row

// stats[tile] = {max|q|, max|k|, max G, min G, min s_ii over real rows, sum of log factors, 0, 0}
// A row takes hd/8 lanes (16-byte loads), so a warp works on 2 (hd = 128) or 4 (hd = 64) rows at a time.
__global__ void __launch_bounds__(256) tile_stats_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                                                        const __nv_bfloat16* __restrict__ w, const float* __restrict__ beta,
                                                        const float* __restrict__ G, float* __restrict__ stats, int L, int Lp,
                                                        int hd, float scale) {
    __shared__ float red[8][6];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lpr = hd / 8, grp = lane / lpr, li = lane % lpr, rows_w = 32 / lpr;
    const int N = Lp / CHUNK, sl = blockIdx.x / N, c = blockIdx.x % N;
    float qn = 0.f, kn = 0.f, gmax = -INFINITY, gmin = INFINITY, mlo = INFINITY, gam = 0.f;
    auto dot8 = [](const uint4& a, const uint4& b) {
        const uint32_t x[4] = {a.x, a.y, a.z, a.w}, y[4] = {b.x, b.y, b.z, b.w};
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc = fmaf(__uint_as_float(x[i] << 16), __uint_as_float(y[i] << 16), acc);
            acc = fmaf(__uint_as_float(x[i] & 0xffff0000u), __uint_as_float(y[i] & 0xffff0000u), acc);
        }
        return acc;
    };
    for (int r = warp * rows_w + grp; r < CHUNK; r += 8 * rows_w) {
        const int t = c * CHUNK + r;
        const size_t row = (size_t)sl * Lp + t;
        const uint4 a = *reinterpret_cast<const uint4*>(q + row * hd + li * 8);
        const uint4 b = *reinterpret_cast<const uint4*>(k + row * hd + li * 8);
        const uint4 x = *reinterpret_cast<const uint4*>(w + row * hd + li * 8);
        float qq = dot8(a, a), kk = dot8(b, b), qk = dot8(a, b), ww = dot8(x, x);
        for (int off = lpr / 2; off >= 1; off >>= 1) {
            qq += __shfl_xor_sync(0xffffffffu, qq, off); kk += __shfl_xor_sync(0xffffffffu, kk, off);
            qk += __shfl_xor_sync(0xffffffffu, qk, off); ww += __shfl_xor_sync(0xffffffffu, ww, off);
        }
        const float g = G[row];
        qn = fmaxf(qn, sqrtf(qq)); kn = fmaxf(kn, sqrtf(kk));
        gmax = fmaxf(gmax, g); gmin = fminf(gmin, g);
        if (t < L) mlo = fminf(mlo, scale * qk);
        gam += logf(fmaxf(1.f, fabsf(1.f - beta[row] * ww)));
    }
    // the lanes of a group hold the same values; combine the groups of the warp (the growth sum counts each group once)
    for (int off = lpr; off < 32; off <<= 1) {
        qn = fmaxf(qn, __shfl_xor_sync(0xffffffffu, qn, off)); kn = fmaxf(kn, __shfl_xor_sync(0xffffffffu, kn, off));
        gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, off)); gmin = fminf(gmin, __shfl_xor_sync(0xffffffffu, gmin, off));
        mlo = fminf(mlo, __shfl_xor_sync(0xffffffffu, mlo, off)); gam += __shfl_xor_sync(0xffffffffu, gam, off);
    }
    if (lane == 0) {
        red[warp][0] = qn; red[warp][1] = kn; red[warp][2] = gmax;
        red[warp][3] = gmin; red[warp][4] = mlo; red[warp][5] = gam;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int x = 1; x < 8; ++x) {
            qn = fmaxf(qn, red[x][0]); kn = fmaxf(kn, red[x][1]); gmax = fmaxf(gmax, red[x][2]); gmin = fminf(gmin, red[x][3]);
            mlo = fminf(mlo, red[x][4]); gam += red[x][5];
        }
        float* o = stats + (size_t)blockIdx.x * 8;
        // the norms and the growth go up, the row maximum goes down by a rounding margin: the test must err towards keeping
        o[0] = qn * 1.001f; o[1] = kn * 1.001f; o[2] = gmax; o[3] = gmin;
        o[4] = mlo - 1e-3f * fabsf(mlo); o[5] = gam * 1.001f + 1e-6f;
        o[6] = o[7] = 0.f;
    }
}

__global__ void __launch_bounds__(128) tile_keep_kernel(const float* __restrict__ stats, int* __restrict__ nkeep, int S, int N,
                                                       float ascale) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= S * N) return;
    const int sl = idx / N, I = idx % N;
    const float* me = stats + (size_t)idx * 8;
    const float qn = me[0], gmax = me[2], need = me[4] - kSkipMargin;
    float acc = 0.f;
    int keep = 1;
    for (int n = 0; n <= I; ++n) {
        const float* o = stats + ((size_t)sl * N + I - n) * 8;
        acc += o[5];
        const float bound = ascale * qn * o[1] * expf(acc) + gmax - o[3];
        if (!(bound < need)) keep = n + 1;   // also keeps everything when a NaN or an infinity is around
    }
    nkeep[idx] = keep;
}

// One CTA per slice.  First the kept ranges are made a staircase: the first kept key chunk of a query chunk never lies
// after that of a later query chunk (ranges only grow, which is always safe).  Then "key chunk J is kept by query chunk I"
// holds for exactly the I in J .. far(J), so the key-major sweep of the backward (nvisit[J] = far(J) - J + 1 query chunks)
// computes the same pairs as the query-major sweeps, and every version a sweep asks for lies within the levels its chunk
// reaches.  Also counts the kept pairs.
__global__ void __launch_bounds__(128) tile_stair_kernel(int* __restrict__ nkeep, int* __restrict__ nvisit,
                                                        unsigned long long* counters, int S, int N) {
    // one CTA per slice; the two serial scans run on a copy in shared memory when it fits (N <= kStairMax chunks, i.e.
    // sequences up to a million tokens), else directly on global memory
    constexpr int kStairMax = 8192;
    __shared__ int snk[kStairMax];
    const int sl = blockIdx.x;
    int* gk = nkeep + (size_t)sl * N;
    int* gv = nvisit + (size_t)sl * N;
    const bool in_smem = N <= kStairMax;
    if (in_smem) {
        for (int i = threadIdx.x; i < N; i += blockDim.x) snk[i] = gk[i];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        int* nk = in_smem ? snk : gk;
        unsigned long long kept = 0;
        int start = N;
        for (int I = N - 1; I >= 0; --I) {
            start = min(start, I - nk[I] + 1);
            nk[I] = I - start + 1;
            kept += (unsigned long long)nk[I];
        }
        if (in_smem) {   // nvisit is written below by all threads from the staircase
            atomicAdd(&counters[0], kept);
        } else {
            int far = 0;
            for (int J = 0; J < N; ++J) {
                far = max(far, J);
                while (far + 1 < N && far + 1 - nk[far + 1] + 1 <= J) ++far;
                gv[J] = far - J + 1;
            }
            atomicAdd(&counters[0], kept);
        }
        atomicAdd(&counters[1], (unsigned long long)N * (N + 1) / 2);
    }
    if (!in_smem) return;
    __syncthreads();
    // far(J) = the last I whose first kept key chunk I - nk[I] + 1 is <= J; those first chunks do not decrease with I, so a
    // binary search per J finds it
    for (int J = threadIdx.x; J < N; J += blockDim.x) {
        int lo = J, hi = N - 1;   // invariant: chunk lo keeps J (a chunk always keeps itself)
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (mid - snk[mid] + 1 <= J) lo = mid; else hi = mid - 1;
        }
        gv[J] = lo - J + 1;
        gk[J] = snk[J];
    }
}

// ---- context-parallel path: gate terms of a segment, merge of partial softmax results
__global__ void cp_gate_kernel(const float* __restrict__ G, float* __restrict__ gq, float* __restrict__ gk,
                               float* __restrict__ gtot, int L, int Lp) {
    const int s = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    const float tot = G ? G[(size_t)s * Lp + L - 1] : 0.f;
    if (i == 0) gtot[s] = tot;
    if (i >= Lp) return;
    const float g = G ? G[(size_t)s * Lp + i] : 0.f;
    gq[(size_t)s * Lp + i] = i < L ? g : 0.f;
    gk[(size_t)s * Lp + i] = i < L ? g - tot : 1e30f;
}
// one thread per 4 outputs of a row
__global__ void cp_merge_kernel(float* __restrict__ o_acc, float* __restrict__ lse_acc, const float* __restrict__ o_t,
                                const float* __restrict__ lse_t, size_t rows, int hd4) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * hd4) return;
    const size_t r = i / hd4;
    const float la = lse_acc[r], lt = lse_t[r];
    const float m = fmaxf(la, lt);
    const float wa = __expf(la - m), wt = __expf(lt - m), inv = 1.f / (wa + wt);
    const float4 a = reinterpret_cast<const float4*>(o_acc)[i], t = reinterpret_cast<const float4*>(o_t)[i];
    reinterpret_cast<float4*>(o_acc)[i] = make_float4((a.x * wa + t.x * wt) * inv, (a.y * wa + t.y * wt) * inv,
                                                      (a.z * wa + t.z * wt) * inv, (a.w * wa + t.w * wt) * inv);
    __syncwarp();   // (the lanes of a row read lse_acc before one of them replaces it: a row's hd4 lanes sit in one warp)
    if (i % hd4 == 0) lse_acc[r] = m + __logf(wa + wt);
}
__global__ void cp_finish_kernel(const float* __restrict__ o_acc, const float* __restrict__ lse_acc, __nv_bfloat16* __restrict__ o,
                                 float* __restrict__ lse, size_t rows, int hd4) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * hd4) return;
    const float4 a = reinterpret_cast<const float4*>(o_acc)[i];
    __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
    reinterpret_cast<uint2*>(o)[i] = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
    if (i % hd4 == 0) lse[i / hd4] = lse_acc[i / hd4];
}

// ---- forward-state record and the wait self-test
__global__ void state_write_kernel(StateRecord* dst, const StateRecord rec) {
    if (threadIdx.x == 0) *dst = rec;
}
__global__ void state_check_kernel(const StateRecord* have, const StateRecord want, uint32_t* status) {
    if (threadIdx.x != 0) return;
    const StateRecord h = *have;
    const bool same = h.magic == want.magic && h.q == want.q && h.k == want.k && h.v == want.v && h.w == want.w &&
                      h.beta == want.beta && h.log_f == want.log_f && h.B == want.B && h.H == want.H && h.L == want.L &&
                      h.d == want.d && h.gate == want.gate && (!want.gate || h.scale == want.scale);
    if (!same) atomicCAS(status, 0u, (uint32_t)ST_STATE);
}
// The same bounded wait every kernel of the library uses, on a barrier that never completes: after `ticks` cycles it
// gives up, raises the CTA's abort flag with its code, and the kernel forwards the flag to the status word and returns.
__global__ void selftest_wait_kernel(uint32_t* status, long long ticks) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_word;
    volatile uint32_t* abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        tc5::mbar_init(&bar, 1);
        *abort_flag = 0;
        tc5::mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        bool ok = tc5::mbar_try_wait(&bar, 0);
        if (!ok) ok = tc5::mbar_wait_slow(&bar, 0, abort_flag, ST_SELFTEST, ticks);
        if (!ok && *abort_flag != 0) atomicCAS(status, 0u, *abort_flag);
    }
}

}  // namespace

cudaError_t launch_gate_suffix(const float* dGa, const float* dGb, const float* dGc, float* out, int S, int L, int Lp,
                               cudaStream_t st) {
    gate_suffix_kernel<<<S, 1024, 0, st>>>(dGa, dGb, dGc, out, L, Lp);
    return cudaGetLastError();
}
cudaError_t launch_dsd_rowsum(const float* dsd, float* rs, int nchunks, cudaStream_t st) {
    dsd_rowsum_kernel<<<nchunks, 256, 0, st>>>(dsd, rs);
    return cudaGetLastError();
}

cudaError_t launch_pad_rows(const void* src, void* dst, int S, int L, int Lp, int d, int f32, cudaStream_t st) {
    const int rowbytes16 = d * (f32 ? 4 : 2) / 16;
    const long total = (long)Lp * rowbytes16;
    dim3 grid((unsigned)((total + 255) / 256), S);
    pad_rows_kernel<<<grid, 256, 0, st>>>(src, dst, L, Lp, rowbytes16);
    return cudaGetLastError();
}

cudaError_t launch_pad_vec(const float* src, float* dst, int S, int L, int Lp, cudaStream_t st) {
    dim3 grid((Lp + 255) / 256, S);
    pad_vec_kernel<<<grid, 256, 0, st>>>(src, dst, L, Lp);
    return cudaGetLastError();
}

cudaError_t launch_gate_prefix(const float* g, float* G, int S, int L, int Lp, cudaStream_t st) {
    gate_prefix_kernel<<<S, 1024, 0, st>>>(g, G, L, Lp);
    return cudaGetLastError();
}

cudaError_t launch_gate_skip(const void* q, const void* k, const void* w, const float* beta, const float* G, float* stats,
                             int* nkeep, int* nvisit, unsigned long long* counters, int S, int L, int Lp, int hd, float scale,
                             cudaStream_t st) {
    typedef __nv_bfloat16 bf;
    const int N = Lp / CHUNK;
    tile_stats_kernel<<<S * N, 256, 0, st>>>((const bf*)q, (const bf*)k, (const bf*)w, beta, G, stats, L, Lp, hd, scale);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    tile_keep_kernel<<<(S * N + 127) / 128, 128, 0, st>>>(stats, nkeep, S, N, fabsf(scale));
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    tile_stair_kernel<<<S, 128, 0, st>>>(nkeep, nvisit, counters, S, N);
    return cudaGetLastError();
}

cudaError_t launch_cp_gate(const float* G, float* gq, float* gk, float* gtot, int S, int L, int Lp, cudaStream_t st) {
    cp_gate_kernel<<<dim3((Lp + 255) / 256, S), 256, 0, st>>>(G, gq, gk, gtot, L, Lp);
    return cudaGetLastError();
}
cudaError_t launch_cp_merge(float* o_acc, float* lse_acc, const float* o_t, const float* lse_t, size_t rows, int hd,
                            cudaStream_t st) {
    const size_t n = rows * (hd / 4);
    cp_merge_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(o_acc, lse_acc, o_t, lse_t, rows, hd / 4);
    return cudaGetLastError();
}
cudaError_t launch_cp_finish(const float* o_acc, const float* lse_acc, void* o, float* lse, size_t rows, int hd,
                             cudaStream_t st) {
    const size_t n = rows * (hd / 4);
    cp_finish_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(o_acc, lse_acc, (__nv_bfloat16*)o, lse, rows, hd / 4);
    return cudaGetLastError();
}

cudaError_t launch_state_write(void* record, const StateRecord& rec, cudaStream_t st) {
    state_write_kernel<<<1, 32, 0, st>>>((StateRecord*)record, rec);
    return cudaGetLastError();
}
cudaError_t launch_state_check(const void* record, const StateRecord& want, uint32_t* status, cudaStream_t st) {
    state_check_kernel<<<1, 32, 0, st>>>((const StateRecord*)record, want, status);
    return cudaGetLastError();
}
cudaError_t launch_selftest_wait(uint32_t* status, long long ticks, cudaStream_t st) {
    selftest_wait_kernel<<<1, 32, 0, st>>>(status, ticks);
    return cudaGetLastError();
}

}  // namespace path
