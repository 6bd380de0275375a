// Chunk-level kernels of PaTH attention: everything that is linear in the sequence length.
//  - gemm_kernel: batched C = mask(alpha A B + gamma D + I) on mma.sync tensor cores (bf16 products, float
//    accumulation; float operands optionally split into two bf16 terms), 64 x 64 tile per CTA.
//  - tri_inverse_kernel: the inverse in the UT transform (paper Sec. 3.1), T^-1 = (I + strictLower(D W W^T))^-1 D.
//  - pad / gate-prefix helpers.
#include "linear.cuh"

namespace path {

namespace {

constexpr int TM = 64, TN = 64, TK = 32, LDS = TK + 8;  // smem row stride in bf16 elements

__device__ __forceinline__ const void* adv(const void* p, long elems, int f32) {
    return (const char*)p + elems * (f32 ? 4 : 2);
}
__device__ __forceinline__ void* adv(void* p, long elems, int f32) {
    return (char*)p + elems * (f32 ? 4 : 2);
}
__device__ __forceinline__ float ld_elem(const void* p, long idx, int f32) {
    return f32 ? ((const float*)p)[idx] : __bfloat162float(((const __nv_bfloat16*)p)[idx]);
}

// Loads a [64 (mn) x 32 (k)] tile of an operand into shared memory as bf16 hi (+ lo) parts, k contiguous.
__device__ __forceinline__ void load_tile(const Operand& op, int mn0, int MN, int k0, int K, __nv_bfloat16* hi,
                                          __nv_bfloat16* lo, bool split) {
    const int tid = threadIdx.x;
    const bool k_fast = (op.s_k == 1);
#pragma unroll 4
    for (int i = 0; i < (TM * TK) / 128; ++i) {
        const int idx = tid + i * 128;
        const int kk = k_fast ? (idx & (TK - 1)) : (idx >> 6);
        const int mn = k_fast ? (idx >> 5) : (idx & 63);
        float v = 0.f;
        if (mn0 + mn < MN && k0 + kk < K) v = ld_elem(op.p, (long)(mn0 + mn) * op.s_mn + (long)(k0 + kk) * op.s_k, op.f32);
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi[mn * LDS + kk] = h;
        if (split) lo[mn * LDS + kk] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

__device__ __forceinline__ void load_frag_a(const __nv_bfloat16* s, int row0, int kk, int lane, uint32_t (&a)[4]) {
    const int r = row0 + (lane >> 2), c = kk + (lane & 3) * 2;
    a[0] = *reinterpret_cast<const uint32_t*>(&s[r * LDS + c]);
    a[1] = *reinterpret_cast<const uint32_t*>(&s[(r + 8) * LDS + c]);
    a[2] = *reinterpret_cast<const uint32_t*>(&s[r * LDS + c + 8]);
    a[3] = *reinterpret_cast<const uint32_t*>(&s[(r + 8) * LDS + c + 8]);
}
__device__ __forceinline__ void load_frag_b(const __nv_bfloat16* s, int n0, int kk, int lane, uint32_t (&b)[2]) {
    const int n = n0 + (lane >> 2), c = kk + (lane & 3) * 2;
    b[0] = *reinterpret_cast<const uint32_t*>(&s[n * LDS + c]);
    b[1] = *reinterpret_cast<const uint32_t*>(&s[n * LDS + c + 8]);
}

struct Resolved {
    Operand A, B;
    int M, N, K;
    void* C; void* C2; const void* D;
    int c2_rows;
};

__device__ __forceinline__ bool resolve(const GemmProblem& g, const AffineBatch& b, int z, Resolved& r) {
    const long z0 = z / b.nb1, z1 = z % b.nb1;
    r.A = g.A; r.B = g.B; r.M = g.M; r.N = g.N; r.K = g.K;
    r.A.p = adv(g.A.p, z0 * b.a0 + z1 * b.a1, g.A.f32);
    r.B.p = adv(g.B.p, z0 * b.b0 + z1 * b.b1, g.B.f32);
    r.C = g.C ? adv(g.C, z0 * b.c0 + z1 * b.c1, g.c_f32) : nullptr;
    r.C2 = g.C2 ? adv(g.C2, z0 * b.c20 + z1 * b.c21, 0) : nullptr;
    r.D = g.D ? adv(g.D, z0 * b.d0 + z1 * b.d1, g.d_f32) : nullptr;
    r.c2_rows = g.c2_rows;
    if (b.rows_total > 0) {
        const long left = (long)b.rows_total - z1 * CHUNK;
        r.c2_rows = left < CHUNK ? (left > 0 ? (int)left : 0) : CHUNK;
    }
    return true;
}

// Fills the per-batch operands of a version-chain step; returns false if chunk `c` of this level has no such step.
__device__ __forceinline__ bool resolve(GemmProblem& g, const VersionBatch& v, int z, Resolved& r) {
    const int s = z / v.N, c = z % v.N;
    const int l2 = v.l2;
    int l1, b, src;
    if (!v.is_key) {
        const unsigned low = (unsigned)c & ((1u << l2) - 1u);
        if (!((c >> l2) & 1) || low == 0) return false;
        l1 = msb32(low);
        b = ((c >> l2) << l2) >> l1;
        src = qslot(l1, c);
    } else {
        const unsigned lowz = ~(unsigned)c & ((1u << l2) - 1u);
        if (((c >> l2) & 1) || lowz == 0) return false;
        if ((((c >> l2) + 1) << l2) > v.N - 1) return false;
        l1 = msb32(lowz);
        b = (c >> l1) + 1;
        src = kslot(l1, c);
    }
    const long d = v.d, dd = d * d;
    const long row_src = ((long)src * v.S + s) * v.Lp + (long)c * CHUNK;
    const long row_dst = ((long)l2 * v.S + s) * v.Lp + (long)c * CHUNK;
    const long dy_idx = v.lv.dy_off[l1] + ((long)s * v.lv.dy_cnt[l1] + b) * dd;
    const bool dy_transposed = (v.mode == 0) ? (v.is_key != 0) : (v.is_key == 0);
    g.split = 1; g.alpha = 1.f; g.alpha2 = 1.f; g.gamma = 1.f; g.mask = MASK_NONE; g.identity = 0;
    g.D = nullptr; g.C2 = nullptr; g.c_f32 = 1; g.c2_trans = 0;
    r.D = nullptr; r.C2 = nullptr; r.c2_rows = 1 << 30;
    if (v.mode == 0 || v.mode == 1) {
        r.A = (v.mode == 0) ? Operand{v.xv + row_src * d, d, 1, 0} : Operand{v.dxv + row_dst * d, d, 1, 1};
        r.B = dy_transposed ? Operand{v.dy + dy_idx, d, 1, 1} : Operand{v.dy + dy_idx, 1, d, 1};
        r.M = CHUNK; r.N = (int)d; r.K = (int)d;
        g.ldc = d;
        if (v.mode == 0) {
            r.C = v.out16 + row_dst * d;
            g.c_f32 = 0;
            g.accumulate = ACC_NONE;
        } else {
            r.C = v.dxv + row_src * d;
            g.accumulate = ACC_ADD;
        }
    } else {
        const __nv_bfloat16* x = v.xv + row_src * d;
        const float* gup = v.dxv + row_dst * d;
        if (!v.is_key) { r.A = Operand{x, 1, d, 0}; r.B = Operand{gup, 1, d, 1}; }
        else           { r.A = Operand{gup, 1, d, 1}; r.B = Operand{x, 1, d, 0}; }
        r.M = (int)d; r.N = (int)d; r.K = CHUNK;
        r.C = v.ddy + dy_idx;
        g.ldc = d;
        g.accumulate = ACC_ATOMIC;
    }
    g.C = r.C;
    return true;
}

template <class Batch>
__global__ void __launch_bounds__(128) gemm_kernel(GemmProblem g, const Batch batch) {
    __shared__ __align__(16) __nv_bfloat16 sAh[TM * LDS], sAl[TM * LDS], sBh[TN * LDS], sBl[TN * LDS];
    Resolved r;
    if (!resolve(g, batch, (int)blockIdx.x, r)) return;
    const int m0 = blockIdx.z * TM, n0 = blockIdx.y * TN;
    if (m0 >= r.M || n0 >= r.N) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wm = (warp >> 1) * 32, wn = (warp & 1) * 32;
    const bool split_a = g.split && r.A.f32, split_b = g.split && r.B.f32;

    float acc[2][4][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int x = 0; x < 4; ++x) acc[i][j][x] = 0.f;

    for (int k0 = 0; k0 < r.K; k0 += TK) {
        load_tile(r.A, m0, r.M, k0, r.K, sAh, sAl, split_a);
        load_tile(r.B, n0, r.N, k0, r.K, sBh, sBl, split_b);
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; kk += 16) {
            uint32_t ah[2][4], al[2][4], bh[4][2], bl[4][2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                load_frag_a(sAh, wm + i * 16, kk, lane, ah[i]);
                if (split_a) load_frag_a(sAl, wm + i * 16, kk, lane, al[i]);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                load_frag_b(sBh, wn + j * 8, kk, lane, bh[j]);
                if (split_b) load_frag_b(sBl, wn + j * 8, kk, lane, bl[j]);
            }
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (split_b) mma16816(acc[i][j], ah[i], bl[j]);
                    if (split_a) mma16816(acc[i][j], al[i], bh[j]);
                    mma16816(acc[i][j], ah[i], bh[j]);
                }
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int m = m0 + wm + i * 16 + (lane >> 2) + ((x >> 1) << 3);
                const int n = n0 + wn + j * 8 + (lane & 3) * 2 + (x & 1);
                if (m >= r.M || n >= r.N) continue;
                float v = g.alpha * acc[i][j][x];
                if (r.D) v += g.gamma * ld_elem(r.D, (long)m * g.ldd + n, g.d_f32);
                if (g.identity && m == n) v += 1.f;
                if ((g.mask == MASK_LOWER && n > m) || (g.mask == MASK_STRICT && n >= m)) v = 0.f;
                if (r.C) {
                    const long ci = (long)m * g.ldc + n;
                    if (g.c_f32) {
                        float* C = (float*)r.C;
                        if (g.accumulate == ACC_ATOMIC) { atomicAdd(&C[ci], v); }
                        else { if (g.accumulate == ACC_ADD) v += C[ci]; C[ci] = v; }
                    } else {
                        __nv_bfloat16* C = (__nv_bfloat16*)r.C;
                        if (g.accumulate == ACC_ADD) v += __bfloat162float(C[ci]);
                        C[ci] = __float2bfloat16_rn(v);
                    }
                }
                if (r.C2 && m < r.c2_rows) {
                    const long ci = g.c2_trans ? (long)n * g.ldc2 + m : (long)m * g.ldc2 + n;
                    ((__nv_bfloat16*)r.C2)[ci] = __float2bfloat16_rn(g.alpha2 * v);
                }
            }
}

// ---------------------------------------------------------------------------------------------- UT inverse
// One CTA per chunk, 256 threads.  X = (I + Nl)^-1 with Nl = strictLower(beta_r * Gm[r][c]), by 16-row panels:
// the 16 x 16 diagonal blocks by forward substitution, then panel bi: X[bi, <bi] = -X[bi,bi] (Nl[bi, <bi] X[<bi, <bi]).
constexpr int TRI_LD = CHUNK + 1;
constexpr size_t kTriSmem = (size_t)(2 * CHUNK * TRI_LD + 16 * CHUNK + CHUNK) * sizeof(float);

__global__ void __launch_bounds__(256) tri_inverse_kernel(const float* __restrict__ Gm, const float* __restrict__ beta,
                                                          float* __restrict__ Ainv, float* __restrict__ Tt) {
    extern __shared__ float tsm[];
    float* Nl = tsm;
    float* X = Nl + CHUNK * TRI_LD;
    float* Z = X + CHUNK * TRI_LD;
    float* bt = Z + 16 * CHUNK;
    const int tid = threadIdx.x;
    const size_t base = (size_t)blockIdx.x * CHUNK * CHUNK;
    if (tid < CHUNK) bt[tid] = beta[(size_t)blockIdx.x * CHUNK + tid];
    __syncthreads();
    for (int idx = tid; idx < CHUNK * CHUNK; idx += 256) {
        const int r = idx >> 7, c = idx & 127;
        Nl[r * TRI_LD + c] = (c < r) ? bt[r] * Gm[base + idx] : 0.f;
        X[r * TRI_LD + c] = 0.f;
    }
    __syncthreads();
    {   // diagonal blocks: warp w owns block w, lane j < 16 owns column j of the block
        const int w = tid >> 5, j = tid & 31;
        if (j < 16) {
            const int o = w * 16;
            for (int r = j; r < 16; ++r) {
                float v = (r == j) ? 1.f : 0.f;
                for (int c = j; c < r; ++c) v -= Nl[(o + r) * TRI_LD + o + c] * X[(o + c) * TRI_LD + o + j];
                X[(o + r) * TRI_LD + o + j] = v;
            }
        }
    }
    __syncthreads();
    for (int bi = 1; bi < CHUNK / 16; ++bi) {
        const int R = bi * 16, W = bi * 16;
        for (int idx = tid; idx < 16 * W; idx += 256) {
            const int r = idx / W, c = idx % W;
            float z = 0.f;
            for (int k = (c & ~15); k < W; ++k) z += Nl[(R + r) * TRI_LD + k] * X[k * TRI_LD + c];
            Z[r * CHUNK + c] = z;
        }
        __syncthreads();
        for (int idx = tid; idx < 16 * W; idx += 256) {
            const int r = idx / W, c = idx % W;
            float v = 0.f;
            for (int k = 0; k <= r; ++k) v -= X[(R + r) * TRI_LD + R + k] * Z[k * CHUNK + c];
            X[(R + r) * TRI_LD + c] = v;
        }
        __syncthreads();
    }
    for (int idx = tid; idx < CHUNK * CHUNK; idx += 256) {
        const int r = idx >> 7, c = idx & 127;
        const float x = X[r * TRI_LD + c];
        if (Ainv) Ainv[base + idx] = x;
        Tt[base + idx] = x * bt[c];
    }
}

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

// dbeta term 1 and the column scaling of dT (per chunk, 128 threads = columns):
//   t1[c] = sum_r Ainv[r][c] dT[r][c];   dT[r][c] *= beta[c]   (in place: dT becomes dT D)
__global__ void __launch_bounds__(128) beta_cols_kernel(const float* __restrict__ Ainv, float* __restrict__ dT,
                                                        const float* __restrict__ beta, float* __restrict__ t1) {
    const size_t base = (size_t)blockIdx.x * CHUNK * CHUNK;
    const int c = threadIdx.x;
    const float b = beta[(size_t)blockIdx.x * CHUNK + c];
    float acc = 0.f;
    for (int r = 0; r < CHUNK; ++r) {
        const float t = dT[base + r * CHUNK + c];
        acc += Ainv[base + r * CHUNK + c] * t;
        dT[base + r * CHUNK + c] = t * b;
    }
    t1[(size_t)blockIdx.x * CHUNK + c] = acc;
}

// dbeta term 2 and the row scaling of dA (per chunk, one warp per row):
//   dbeta[r] = t1[r] + sum_c dA[r][c] Gm[r][c];   dA[r][c] *= beta[r]   (in place: dA becomes dGm)
__global__ void __launch_bounds__(256) beta_rows_kernel(float* __restrict__ dA, const float* __restrict__ Gm,
                                                        const float* __restrict__ beta, const float* __restrict__ t1,
                                                        float* __restrict__ dbeta, int N, int L) {
    const size_t base = (size_t)blockIdx.x * CHUNK * CHUNK;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int s = blockIdx.x / N, ch = blockIdx.x % N;
    for (int r = warp; r < CHUNK; r += 8) {
        const float b = beta[(size_t)blockIdx.x * CHUNK + r];
        float acc = 0.f;
        for (int c = lane; c < CHUNK; c += 32) {
            const float a = dA[base + r * CHUNK + c];
            acc += a * Gm[base + r * CHUNK + c];
            dA[base + r * CHUNK + c] = a * b;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        const int pos = ch * CHUNK + r;
        if (lane == 0 && pos < L) dbeta[(size_t)s * L + pos] = acc + t1[(size_t)blockIdx.x * CHUNK + r];
    }
}

// rs[chunk*128 + i] = sum_k dsd[chunk][i][k]; one warp per row.
__global__ void __launch_bounds__(256) dsd_rowsum_kernel(const float* __restrict__ dsd, float* __restrict__ rs) {
    const size_t base = (size_t)blockIdx.x * CHUNK * CHUNK;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = warp; r < CHUNK; r += 8) {
        float acc = 0.f;
        for (int c = lane; c < CHUNK; c += 32) acc += dsd[base + r * CHUNK + c];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) rs[(size_t)blockIdx.x * CHUNK + r] = acc;
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

}  // namespace

cudaError_t launch_beta_cols(const float* Ainv, float* dT, const float* beta, float* t1, int nchunks, cudaStream_t st) {
    beta_cols_kernel<<<nchunks, 128, 0, st>>>(Ainv, dT, beta, t1);
    return cudaGetLastError();
}
cudaError_t launch_beta_rows(float* dA, const float* Gm, const float* beta, const float* t1, float* dbeta, int S, int N,
                             int L, cudaStream_t st) {
    beta_rows_kernel<<<S * N, 256, 0, st>>>(dA, Gm, beta, t1, dbeta, N, L);
    return cudaGetLastError();
}
cudaError_t launch_gate_suffix(const float* dGa, const float* dGb, const float* dGc, float* out, int S, int L, int Lp,
                               cudaStream_t st) {
    gate_suffix_kernel<<<S, 1024, 0, st>>>(dGa, dGb, dGc, out, L, Lp);
    return cudaGetLastError();
}
cudaError_t launch_dsd_rowsum(const float* dsd, float* rs, int nchunks, cudaStream_t st) {
    dsd_rowsum_kernel<<<nchunks, 256, 0, st>>>(dsd, rs);
    return cudaGetLastError();
}

cudaError_t launch_gemm(const GemmProblem& g, const AffineBatch& b, int nbatch, cudaStream_t st) {
    if (nbatch <= 0) return cudaSuccess;
    dim3 grid(nbatch, (g.N + TN - 1) / TN, (g.M + TM - 1) / TM);
    gemm_kernel<AffineBatch><<<grid, 128, 0, st>>>(g, b);
    return cudaGetLastError();
}

cudaError_t launch_gemm_version(const VersionBatch& v, cudaStream_t st) {
    GemmProblem g{};
    const int md = (v.mode == 2) ? v.d : CHUNK;
    dim3 grid(v.S * v.N, (v.d + TN - 1) / TN, (md + TM - 1) / TM);
    gemm_kernel<VersionBatch><<<grid, 128, 0, st>>>(g, v);
    return cudaGetLastError();
}

cudaError_t launch_tri_inverse(const float* Gm, const float* beta, float* Ainv, float* Tt, int nchunks,
                               cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(tri_inverse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kTriSmem);
    if (e != cudaSuccess) return e;
    tri_inverse_kernel<<<nchunks, 256, kTriSmem, st>>>(Gm, beta, Ainv, Tt);
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

}  // namespace path
