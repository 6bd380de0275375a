// Per-chunk compact representation of the Householder product (paper Sec. 3.1 UT transform) and the
// boundary-adjusted queries / keys and chunk product built from it (Sec. 3.3), fused into one kernel.
//
// One CTA owns one 128-token chunk.  With W, Q, K the chunk's rows and D = diag(beta):
//   Gm = W W^T,  Xq = lower(Q W^T),  Xk = strictLower(W K^T)                      (MMA group 1)
//   T~ = (I + strictLower(D Gm))^-1 D                                             (float32, blocked substitution)
//   U = T~ W,  Y = T~ Xk                                                          (MMA group 2)
//   Qleft = Q - Xq U,  Kright = K - Y^T W,  P = I - W^T U                          (MMA group 3)
// and the bf16 operands of the diagonal-chunk correction of the attention sweep, Xqn = -Xq and Yt = Y^T.
//
// Every product is a 128 x 128 x {64,128} tcgen05 MMA whose operands sit in shared memory as row-major
// 128-byte-swizzled tiles; whether a tile enters as X, X^T, on the left or on the right is only a matter of
// the descriptor's major-ness, so nothing is ever transposed in memory.  Accumulators live in tensor memory and
// are read back one row per thread.  T~ is kept as a bf16 pair (hi + lo) because everything downstream
// depends on it; the other intermediates are rounded to bf16 once, like the tiles the attention sweep consumes.
#include <type_traits>
#include "tileops.cuh"

namespace path {
using namespace tc5;

namespace {

using namespace tile;
constexpr int kLd = kT + 4;  // row stride of the float32 triangular buffer (rows stay 16-byte aligned)

// Seven 32 KB tile slots.  0: W.  1, 2: Q, K -> T~ hi, lo -> U hi, lo.  3..6: float32 triangular buffer and its
// scratch -> Xq hi, lo, Xk hi, lo -> (5, 6) Y hi, lo.
struct PrepSmem {
    static constexpr uint32_t offW = 0;
    static constexpr uint32_t offQK = kTileB;
    static constexpr uint32_t offBig = 3 * kTileB;
    static constexpr uint32_t offDiag = offBig + ((kT * kLd * 4 + 1023) / 1024) * 1024;   // [8][16][17] float
    static constexpr uint32_t offZ = offDiag + 8 * 16 * 17 * 4;                            // [16][128] float
    static constexpr uint32_t offBeta = offZ + 16 * kT * 4;                                // [128] float
    static constexpr uint32_t offBar = 7 * kTileB;
    static constexpr uint32_t total = offBar + 64;
    static constexpr uint32_t alloc = total + 1024;
    static_assert(offBeta + kT * 4 <= offBar, "scratch must fit in the tile slots it aliases");
};

template <int HD, bool SAVE>
__global__ void __launch_bounds__(256, 1) chunk_prep_kernel(const __grid_constant__ PrepTensorMaps tm, const PrepParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sW = smem + PrepSmem::offW;
    uint8_t* sQK = smem + PrepSmem::offQK;
    uint8_t* sBig = smem + PrepSmem::offBig;
    float* Xb = (float*)sBig;
    float* diagX = (float*)(smem + PrepSmem::offDiag);
    float* Z = (float*)(smem + PrepSmem::offZ);
    float* bt = (float*)(smem + PrepSmem::offBeta);
    uint64_t* bars = (uint64_t*)(smem + PrepSmem::offBar);  // [0] loads, [1] MMA groups
    uint32_t* tmem_slot = (uint32_t*)(bars + 2);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int chunk = blockIdx.x;                 // flattened (slice, chunk): rows chunk*128 .. +127 of the padded arrays
    const int row = (warp & 3) * 32 + lane;       // accumulator row (TMEM lane) of this thread
    const int half = warp >> 2;                   // which half of the accumulator's columns
    const size_t grow = (size_t)chunk * kT + row; // global row

    if (tid == 0) {
        mbar_init(&bars[0], 1);
        mbar_init(&bars[1], 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, 512);
    if (tid < kT) bt[tid] = p.beta[(size_t)chunk * kT + tid];
    if (HD == 64) {  // second panel of W must read as zeros when W^T is used with M = 128
        for (int i = tid; i < (int)(kPanelB / 16); i += 256) reinterpret_cast<uint4*>(sW + kPanelB)[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t aW = smem_u32(sW), aQ = smem_u32(sQK), aK = smem_u32(sQK + kTileB), aBig = smem_u32(sBig);
    constexpr int KS = HD / 16;  // k-steps over the head dimension
    bool ok = true;
    uint32_t r[32];
    float v[32];
    uint4 pre_q[HD / 64][4], pre_k[HD / 64][4];

    if (tid == 0) {
        mbar_expect_tx(&bars[0], 3 * kT * HD * 2);
        for (int h = 0; h < HD / 64; ++h) {
            tma_load_2d(sW + h * kPanelB, &tm.w, &bars[0], h * 64, chunk * kT);
            tma_load_2d(sQK + h * kPanelB, &tm.q, &bars[0], h * 64, chunk * kT);
            tma_load_2d(sQK + kTileB + h * kPanelB, &tm.k, &bars[0], h * 64, chunk * kT);
        }
        if (!mbar_wait(&bars[0], 0, abort_flag, ST_PREP)) ok = false;
        tc_fence_after_sync();
        if (ok) {   // group 1: Gm -> col 0, Xq -> col 128, Xk -> col 256
            mma(tmem + 0, aW, OP_K, aW, OP_K, KS, 128, false);
            mma(tmem + 128, aQ, OP_K, aW, OP_K, KS, 128, false);
            mma(tmem + 256, aW, OP_K, aK, OP_K, KS, 128, false);
            umma_commit(&bars[1]);
        }
    }
    __syncwarp();  // lanes 1-31 of the issuing warp block here instead of spinning against lane 0
    if (!mbar_wait(&bars[1], 0, abort_flag, ST_PREP)) ok = false;
    ok = __syncthreads_and(ok);
    tc_fence_after_sync();
    if (!ok) goto done;

    // ---- E1: Gm -> strictLower(D Gm) in the float32 buffer
    for (int c = 0; c < 2; ++c) {
        const int c0 = half * 64 + c * 32;
        tmem_ld32(tl + 0 + c0, r);
        tmem_ld_wait();
        const float b = bt[row];
#pragma unroll
        for (int x = 0; x < 32; ++x) v[x] = (c0 + x < row) ? b * __uint_as_float(r[x]) : 0.f;
#pragma unroll
        for (int x = 0; x < 8; ++x)
            *reinterpret_cast<float4*>(Xb + row * kLd + c0 + 4 * x) = make_float4(v[4 * x], v[4 * x + 1], v[4 * x + 2], v[4 * x + 3]);
    }
    __syncthreads();

    // ---- (I + Nl)^-1 in place, 16-row panels
    if (lane < 16) {   // diagonal blocks: warp w inverts block w by forward substitution, lane j keeps column j in registers
        const int o = warp * 16, j = lane;
        float* dx = diagX + warp * 16 * 17;
        float x[16];
#pragma unroll
        for (int rr = 0; rr < 16; ++rr) {
            float acc = (rr == j) ? 1.f : 0.f;
#pragma unroll
            for (int c = 0; c < rr; ++c) acc -= Xb[(o + rr) * kLd + o + c] * x[c];
            x[rr] = (rr >= j) ? acc : 0.f;
            dx[rr * 17 + j] = x[rr];
        }
    }
    __syncthreads();
    for (int bi = 0; bi < kT / 16; ++bi) {   // inverted diagonal blocks into place (their upper triangles are zero)
        const int rr = tid >> 4, k = tid & 15;
        Xb[(bi * 16 + rr) * kLd + bi * 16 + k] = diagX[bi * 16 * 17 + rr * 17 + k];
    }
    __syncthreads();
    // Three merge levels on blocks of NB = 16, 32, 64 rows:  [[A,0],[C,B]]^-1 = [[A^-1,0],[-B^-1 C A^-1, B^-1]].
    // Every level has 64 x NB entries of C blocks in total; each thread owns an (NB/16) x 4 tile of them.
    // T = C A^-1 goes through the scratch area (the diagonal-block buffer is dead by now), M = -B^-1 T replaces C.
    {
        float* T = diagX;   // [64][64]
        auto merge = [&](auto nb_tag) {
            constexpr int NB = decltype(nb_tag)::value, RT = NB / 16;
            const int pr = tid / (4 * NB), u = tid % (4 * NB);
            const int i0 = (u / (NB / 4)) * RT, j0 = (u % (NB / 4)) * 4, base = pr * 2 * NB;
            const float* Cp = Xb + (base + NB + i0) * kLd + base;          // rows i0.. of C
            float acc[RT][4];
#pragma unroll
            for (int r_ = 0; r_ < RT; ++r_)
#pragma unroll
                for (int x = 0; x < 4; ++x) acc[r_][x] = 0.f;
            // T[i][j] = sum_{k >= j} C[i][k] A^-1[k][j]   (A^-1 is lower triangular: rows k < j0 contribute nothing)
#pragma unroll 4
            for (int k = j0; k < NB; ++k) {
                const float4 a4 = *reinterpret_cast<const float4*>(Xb + (base + k) * kLd + base + j0);
#pragma unroll
                for (int r_ = 0; r_ < RT; ++r_) {
                    const float ck = Cp[r_ * kLd + k];
                    acc[r_][0] += ck * a4.x; acc[r_][1] += ck * a4.y; acc[r_][2] += ck * a4.z; acc[r_][3] += ck * a4.w;
                }
            }
#pragma unroll
            for (int r_ = 0; r_ < RT; ++r_)
                *reinterpret_cast<float4*>(T + (pr * NB + i0 + r_) * 64 + j0) =
                    make_float4(acc[r_][0], acc[r_][1], acc[r_][2], acc[r_][3]);
            __syncthreads();
            // M[i][j] = -sum_{k <= i} B^-1[i][k] T[k][j]
#pragma unroll
            for (int r_ = 0; r_ < RT; ++r_)
#pragma unroll
                for (int x = 0; x < 4; ++x) acc[r_][x] = 0.f;
            const float* Bp = Xb + (base + NB + i0) * kLd + base + NB;     // rows i0.. of B^-1
            const float* Tp = T + (pr * NB) * 64 + j0;
#pragma unroll 4
            for (int k = 0; k < i0 + RT; ++k) {                            // B^-1[i][k] = 0 for k > i
                const float4 t4 = *reinterpret_cast<const float4*>(Tp + k * 64);
#pragma unroll
                for (int r_ = 0; r_ < RT; ++r_) {
                    const float bk = Bp[r_ * kLd + k];
                    acc[r_][0] -= bk * t4.x; acc[r_][1] -= bk * t4.y; acc[r_][2] -= bk * t4.z; acc[r_][3] -= bk * t4.w;
                }
            }
#pragma unroll
            for (int r_ = 0; r_ < RT; ++r_)
                *reinterpret_cast<float4*>(Xb + (base + NB + i0 + r_) * kLd + base + j0) =
                    make_float4(acc[r_][0], acc[r_][1], acc[r_][2], acc[r_][3]);
            __syncthreads();
        };
        merge(std::integral_constant<int, 16>{});
        merge(std::integral_constant<int, 32>{});
        merge(std::integral_constant<int, 64>{});
    }

    // ---- T~ = X D as a bf16 pair into the Q / K tiles' space (group 1 has finished with them)
    for (int c = 0; c < 2; ++c) {
        const int c0 = half * 64 + c * 32;
        float hi[32], lo[32];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const float4 f = *reinterpret_cast<const float4*>(Xb + row * kLd + c0 + 4 * x);
            v[4 * x] = f.x; v[4 * x + 1] = f.y; v[4 * x + 2] = f.z; v[4 * x + 3] = f.w;
        }
#pragma unroll
        for (int x = 0; x < 32; ++x) {
            const float xv = v[x];
            const float t = xv * bt[c0 + x];
            v[x] = xv;
            hi[x] = __bfloat162float(__float2bfloat16_rn(t));
            lo[x] = t - hi[x];
        }
        tile_store32(sQK, row, c0, hi);
        tile_store32(sQK + kTileB, row, c0, lo);
        if (SAVE) {
            gstore_bf16x32(p.sTh + grow * kT + c0, hi);
            gstore_bf16x32(p.sTl + grow * kT + c0, lo);
#pragma unroll
            for (int x = 0; x < 32; ++x) {
                hi[x] = __bfloat162float(__float2bfloat16_rn(v[x]));
                lo[x] = v[x] - hi[x];
            }
            gstore_bf16x32(p.sAh + grow * kT + c0, hi);
            gstore_bf16x32(p.sAl + grow * kT + c0, lo);
        }
    }
    __syncthreads();  // everyone has read the float32 buffer; it now becomes the Xq / Xk tiles

    // ---- E1b: Xq = lower(.), Xk = strictLower(.) -> bf16 hi / lo tiles (slots 3..6); Xqn = -Xq -> global
    for (int c = 0; c < 2; ++c) {
        const int c0 = half * 64 + c * 32;
        float lo[32];
        tmem_ld32(tl + 128 + c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 32; ++x) {
            const float t = (c0 + x <= row) ? __uint_as_float(r[x]) : 0.f;
            v[x] = __bfloat162float(__float2bfloat16_rn(t));
            lo[x] = t - v[x];
        }
        tile_store32(sBig, row, c0, v);
        tile_store32(sBig + kTileB, row, c0, lo);
        if (SAVE) gstore_bf16x32(p.sXq + grow * kT + c0, v);
#pragma unroll
        for (int x = 0; x < 32; ++x) v[x] = -v[x];
        gstore_bf16x32(p.Xqn + grow * kT + c0, v);
        tmem_ld32(tl + 256 + c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 32; ++x) {
            const float t = (c0 + x < row) ? __uint_as_float(r[x]) : 0.f;
            v[x] = __bfloat162float(__float2bfloat16_rn(t));
            lo[x] = t - v[x];
        }
        tile_store32(sBig + 2 * kTileB, row, c0, v);
        tile_store32(sBig + 3 * kTileB, row, c0, lo);
        if (SAVE) gstore_bf16x32(p.sXk + grow * kT + c0, v);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {   // group 2: U = T~ W -> col 0, Y = T~ Xk -> col 128 (lo x lo terms dropped)
        tc_fence_after_sync();
        mma(tmem + 0, aQ, OP_K, aW, OP_MN, 8, HD, false);
        mma(tmem + 0, aK, OP_K, aW, OP_MN, 8, HD, true);
        mma(tmem + 128, aQ, OP_K, aBig + 2 * kTileB, OP_MN, 8, 128, false);
        mma(tmem + 128, aK, OP_K, aBig + 2 * kTileB, OP_MN, 8, 128, true);
        mma(tmem + 128, aQ, OP_K, aBig + 3 * kTileB, OP_MN, 8, 128, true);
        umma_commit(&bars[1]);
    }
    __syncwarp();
    if (!mbar_wait(&bars[1], 1, abort_flag, ST_PREP)) ok = false;
    ok = __syncthreads_and(ok);
    tc_fence_after_sync();
    if (!ok) goto done;

    // ---- E2: U -> hi / lo tiles over T~ (slots 1, 2); Y -> hi / lo tiles over Xk (slots 5, 6); Yt = Y^T -> global
    for (int c = 0; c < HD / 64; ++c) {
        const int c0 = half * (HD / 2) + c * 32;
        float lo[32];
        tmem_ld32(tl + 0 + c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 32; ++x) {
            const float t = __uint_as_float(r[x]);
            v[x] = __bfloat162float(__float2bfloat16_rn(t));
            lo[x] = t - v[x];
        }
        tile_store32(sQK, row, c0, v);
        tile_store32(sQK + kTileB, row, c0, lo);
        if (SAVE) gstore_bf16x32(p.sU + grow * HD + c0, v);
    }
    for (int c = 0; c < 2; ++c) {
        const int c0 = half * 64 + c * 32;
        float lo[32];
        tmem_ld32(tl + 128 + c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 32; ++x) {
            const float t = __uint_as_float(r[x]);
            v[x] = __bfloat162float(__float2bfloat16_rn(t));
            lo[x] = t - v[x];
        }
        tile_store32(sBig + 2 * kTileB, row, c0, v);
        tile_store32(sBig + 3 * kTileB, row, c0, lo);
        if (SAVE) gstore_bf16x32(p.sY + grow * kT + c0, v);
        __nv_bfloat16* yt = p.Yt + ((size_t)chunk * kT + c0) * kT + row;
#pragma unroll
        for (int x = 0; x < 32; ++x) yt[(size_t)x * kT] = __float2bfloat16_rn(v[x]);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {   // group 3: Xq U -> col 256, Y^T W -> col 384, W^T U -> col 0
        tc_fence_after_sync();
        mma(tmem + 256, aBig, OP_K, aQ, OP_MN, 8, HD, false);
        mma(tmem + 256, aBig + kTileB, OP_K, aQ, OP_MN, 8, HD, true);
        mma(tmem + 256, aBig, OP_K, aK, OP_MN, 8, HD, true);
        mma(tmem + 384, aBig + 2 * kTileB, OP_MN, aW, OP_MN, 8, HD, false);
        mma(tmem + 384, aBig + 3 * kTileB, OP_MN, aW, OP_MN, 8, HD, true);
        mma(tmem + 0, aW, OP_MN, aQ, OP_MN, 8, HD, false);
        mma(tmem + 0, aW, OP_MN, aK, OP_MN, 8, HD, true);
        umma_commit(&bars[1]);
    }
    __syncwarp();
    // the q / k rows of the final subtraction are fetched while the MMAs run
#pragma unroll
    for (int c = 0; c < HD / 64; ++c) {
        const int c0 = half * (HD / 2) + c * 32;
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            pre_q[c][x] = reinterpret_cast<const uint4*>(p.q + grow * HD + c0)[x];
            pre_k[c][x] = reinterpret_cast<const uint4*>(p.k + grow * HD + c0)[x];
        }
    }
    if (!mbar_wait(&bars[1], 0, abort_flag, ST_PREP)) ok = false;
    ok = __syncthreads_and(ok);
    tc_fence_after_sync();
    if (!ok) goto done;

    // ---- E3: Qleft = Q - Xq U, Kright = K - Y^T W, P = I - W^T U
    for (int c = 0; c < HD / 64; ++c) {
        const int c0 = half * (HD / 2) + c * 32;
        float in[32];
        tmem_ld32(tl + 256 + c0, r);
        tmem_ld_wait();
        unpack_bf16x32(pre_q[c], in);
#pragma unroll
        for (int x = 0; x < 32; ++x) v[x] = in[x] - __uint_as_float(r[x]);
        gstore_bf16x32(p.ql + grow * HD + c0, v);
        tmem_ld32(tl + 384 + c0, r);
        tmem_ld_wait();
        unpack_bf16x32(pre_k[c], in);
#pragma unroll
        for (int x = 0; x < 32; ++x) v[x] = in[x] - __uint_as_float(r[x]);
        gstore_bf16x32(p.kr + grow * HD + c0, v);
        tmem_ld32(tl + 0 + c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 32; ++x) {
            v[x] = ((c0 + x == row) ? 1.f : 0.f) - __uint_as_float(r[x]);
            in[x] = __bfloat162float(__float2bfloat16_rn(v[x]));
            v[x] -= in[x];
        }
        gstore_bf16x32(p.Ph + ((size_t)chunk * HD + row) * HD + c0, in, row < HD);
        gstore_bf16x32(p.Pl + ((size_t)chunk * HD + row) * HD + c0, v, row < HD);
    }

done:
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && *abort_flag != 0) atomicCAS(p.status, 0u, *abort_flag);
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, 512);
    }
}

}  // namespace

cudaError_t launch_chunk_prep(const PrepTensorMaps& tm, const PrepParams& p, int hd, int save, int nchunks,
                              cudaStream_t st) {
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PrepSmem::alloc);
        if (e != cudaSuccess) return e;
        kern<<<nchunks, 256, PrepSmem::alloc, st>>>(tm, p);
        return cudaGetLastError();
    };
    if (hd == 64) return save ? go(chunk_prep_kernel<64, true>) : go(chunk_prep_kernel<64, false>);
    return save ? go(chunk_prep_kernel<128, true>) : go(chunk_prep_kernel<128, false>);
}

}  // namespace path
