// Per-chunk compact representation of the Householder product (paper Sec. 3.1 UT transform) and the
// boundary-adjusted queries / keys and chunk product built from it (Sec. 3.3), fused into one kernel.
//
// With W, Q, K the rows of one 128-token chunk and D = diag(beta):
//   Gm = W W^T,  Xq = lower(Q W^T),  Xk = strictLower(W K^T)
//   T~ = (I + strictLower(D Gm))^-1 D        (float32 blocked substitution up to 64-row blocks; the last merge level is two
//                                             64 x 64 x 64 products of bf16 pairs on the tensor cores)
//   U = T~ W,  Y = T~ Xk
//   Qleft = Q - Xq U,  Kright = K - Y^T W,  P = I - W^T U
// and the bf16 operands of the diagonal-chunk correction of the attention sweep, Xqn = -Xq and Yt = Y^T.
//
// Every product is a 128 x 128 x {64,128} tcgen05 MMA whose operands sit in shared memory as row-major
// 128-byte-swizzled tiles; whether a tile enters as X, X^T, on the left or on the right is only a matter of
// the descriptor's major-ness, so nothing is ever transposed in memory.  Accumulators live in tensor memory and
// are read back one row per thread.  T~ is kept as a bf16 pair (hi + lo) because everything downstream
// depends on it; the other intermediates are rounded to bf16 once, like the tiles the attention sweep consumes.
//
// The kernel is persistent: one CTA per SM walks over chunks.  Eight worker warps do the element-wise work (the
// triangular inverse, accumulator read-outs, conversions, global stores); a ninth warp's first lane issues the TMA
// loads and every product as soon as its operands are published, so the products run underneath the workers'
// next phase and the first product of the next chunk is already finished when the workers get there.
#include <type_traits>
#include "tileops.cuh"

namespace path {
using namespace tc5;

namespace {

using namespace tile;
constexpr int kLd = kT + 4;  // row stride of the float32 triangular buffer (rows stay 16-byte aligned)
constexpr uint32_t kInvTileB = 8192;   // a [64 x 64] bf16 operand tile of the inverse's last merge level

// Seven 32 KB tile slots.  0: W.  1, 2: Q, K -> operands of the inverse's last merge level -> T~ hi, lo -> U hi, lo.  3..6: float32 triangular buffer and its
// scratch -> Xq hi, lo, Xk hi, lo -> (5, 6) Y hi, lo.
struct PrepSmem {
    static constexpr uint32_t offW = 0;
    static constexpr uint32_t offQK = kTileB;
    static constexpr uint32_t offBig = 3 * kTileB;
    static constexpr uint32_t offDiag = offBig + ((kT * kLd * 4 + 1023) / 1024) * 1024;   // [64][64] float scratch
    static constexpr uint32_t offBar = 7 * kTileB;
    static constexpr uint32_t offBeta = offBar + 256;                                      // [128] float
    static constexpr uint32_t total = offBeta + kT * 4;
    static constexpr uint32_t alloc = total + 1024;
    static_assert(offDiag + 64 * 64 * 4 <= offBar, "scratch must fit in the tile slots it aliases");
};

// mbarriers.  Issuer -> workers: one per group of products (and the TMA load, which only the issuer waits for).
// Workers -> issuer (256 arrivals): operands published / accumulators drained.  Each completes once per chunk.
enum { B_LOAD = 0, B_GM, B_XQK, B_M1, B_M2, B_U, B_Y, B_G3A, B_G3B, R_TT, R_M1, R_M2, R_XK, R_U, R_Y, R_E3, B_COUNT };
constexpr int kWorkers = 256, kThreads = 384;   // warps 8..11: the issuer's warpgroup (one active lane)

// Barriers over the eight worker warps.  bar.sync / bar.red are warp-aligned instructions: a warp whose lanes left a
// loop at different times must reconverge first, or the part that runs ahead is taken for the whole warp.
__device__ __forceinline__ void wsync() {
    __syncwarp();
    asm volatile("bar.sync 1, 256;" ::: "memory");
}
__device__ __forceinline__ bool wsync_and(bool ok) {   // barrier over the worker warps + AND of `ok`
    uint32_t r;
    __syncwarp();
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, 256, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)ok)
        : "memory");
    return r != 0;
}

// MODE: PREP_FWD = everything the forward needs; PREP_SAVE = also keeps the tiles of the chain rule (the backward's instance);
// PREP_KEYS = the key side only (prompt key cache: Kright and the chunk products; no query is involved, so Xq, Xq U,
// Qleft and the diagonal-correction operands are left out and q is not even loaded).
template <int HD, int MODE>
__global__ void __launch_bounds__(kThreads, 1) chunk_prep_kernel(const __grid_constant__ PrepTensorMaps tm, const PrepParams p,
                                                                      const int nchunks) {
    constexpr bool SAVE = MODE == PREP_SAVE, KEYS = MODE == PREP_KEYS;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sW = smem + PrepSmem::offW;
    uint8_t* sQK = smem + PrepSmem::offQK;
    uint8_t* sBig = smem + PrepSmem::offBig;
    float* Xb = (float*)sBig;
    float* diagX = (float*)(smem + PrepSmem::offDiag);
    float* bt = (float*)(smem + PrepSmem::offBeta);
    uint64_t* bars = (uint64_t*)(smem + PrepSmem::offBar);
    uint32_t* tmem_slot = (uint32_t*)(bars + B_COUNT);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row = (warp & 3) * 32 + lane;       // accumulator row (TMEM lane) of a worker thread
    const int half = (warp >> 2) & 1;             // which half of the accumulator's columns

    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) mbar_init(&bars[i], i >= R_TT ? (uint32_t)kWorkers : 1u);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, 512);
    if (tid < kT && (int)blockIdx.x < nchunks) bt[tid] = p.beta[(size_t)blockIdx.x * kT + tid];
    if (HD == 64) {  // second panel of W must read as zeros when W^T is used with M = 128
        for (int i = tid; i < (int)(kPanelB / 16); i += kThreads) reinterpret_cast<uint4*>(sW + kPanelB)[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t aW_ = smem_u32(sW), aQ_ = smem_u32(sQK), aK_ = smem_u32(sQK + kTileB), aBig_ = smem_u32(sBig);
    constexpr int KS = HD / 16;  // k-steps over the head dimension
    // tensor-memory columns:  0: Gm -> the inverse's last merge level (0: C A^-1, 64: B^-1 C A^-1) -> U   128: Xq -> W^T U
    //                         256: Xk -> Xq U   384: Y -> Y^T W

    if (warp >= kWorkers / 32) {
        // ------------------------------------------------------------------ issuer
        asm volatile("setmaxnreg.dec.sync.aligned.u32 96;");
        if (tid == kWorkers) {
            auto wait = [&](int b, uint32_t par) { return mbar_wait(&bars[b], par, abort_flag, ST_PREP); };
            auto load = [&](int chunk) {
                mbar_expect_tx(&bars[B_LOAD], (KEYS ? 2 : 3) * kT * HD * 2);
                for (int h = 0; h < HD / 64; ++h) {
                    tma_load_2d(sW + h * kPanelB, &tm.w, &bars[B_LOAD], h * 64, chunk * kT);
                    if (!KEYS) tma_load_2d(sQK + h * kPanelB, &tm.q, &bars[B_LOAD], h * 64, chunk * kT);
                    tma_load_2d(sQK + kTileB + h * kPanelB, &tm.k, &bars[B_LOAD], h * 64, chunk * kT);
                }
            };
            auto store = [&](const CUtensorMap* m, const uint8_t* tile_, int ncols, int chunk_) {
                for (int h = 0; h < ncols / 64; ++h) tma_store_2d(m, tile_ + h * kPanelB, h * 64, chunk_ * kT);
            };
            int chunk = blockIdx.x;
            bool ok = chunk < nchunks;
            if (ok) {
                load(chunk);
                ok = wait(B_LOAD, 0);
                if (ok) {
                    tc_fence_after_sync();
                    mma_small(tmem + 0, aW_, OP_K, aW_, OP_K, KS, 128, false);
                    umma_commit(&bars[B_GM]);
                }
            }
            for (uint32_t it = 0; ok && chunk < nchunks; ++it, chunk += gridDim.x) {
                const uint32_t par = it & 1;
                // (the tile addresses are made opaque once per chunk: otherwise every descriptor of every product is
                // hoisted out of this loop and the thread's small register allotment spills)
                uint32_t aW = aW_, aQ = aQ_, aK = aK_, aBig = aBig_;
                asm volatile("" : "+r"(aW), "+r"(aQ), "+r"(aK), "+r"(aBig));
                // Xq, Xk: their columns held the previous chunk's W^T U and Xq U
                if (it > 0 && !wait(R_E3, par ^ 1)) break;
                tc_fence_after_sync();
                if (!KEYS) mma_small(tmem + 128, aQ, OP_K, aW, OP_K, KS, 128, false);
                mma_small(tmem + 256, aW, OP_K, aK, OP_K, KS, 128, false);
                umma_commit(&bars[B_XQK]);
                // last merge level of the triangular inverse: T = C A^-1, then B^-1 T, as bf16 pairs (64 x 64 x 64 each; the
                // eight 8 KB operand tiles sit in the Q / K slots, whose products have retired by then)
                if (!wait(R_M1, par)) break;
                tc_fence_after_sync();
                mma_small(tmem + 0, aQ, OP_K, aQ + 2 * kInvTileB, OP_MN, 4, 64, false);
                mma_small(tmem + 0, aQ, OP_K, aQ + 3 * kInvTileB, OP_MN, 4, 64, true);
                mma_small(tmem + 0, aQ + kInvTileB, OP_K, aQ + 2 * kInvTileB, OP_MN, 4, 64, true);
                umma_commit(&bars[B_M1]);
                if (!wait(R_M2, par)) break;
                tc_fence_after_sync();
                mma_small(tmem + 64, aQ + 4 * kInvTileB, OP_K, aQ + 6 * kInvTileB, OP_MN, 4, 64, false);
                mma_small(tmem + 64, aQ + 4 * kInvTileB, OP_K, aQ + 7 * kInvTileB, OP_MN, 4, 64, true);
                mma_small(tmem + 64, aQ + 5 * kInvTileB, OP_K, aQ + 6 * kInvTileB, OP_MN, 4, 64, true);
                umma_commit(&bars[B_M2]);
                // U = T~ W  (lo x lo terms are dropped everywhere)
                if (!wait(R_TT, par)) break;
                tc_fence_after_sync();
                mma_small(tmem + 0, aQ, OP_K, aW, OP_MN, 8, HD, false);
                mma_small(tmem + 0, aK, OP_K, aW, OP_MN, 8, HD, true);
                umma_commit(&bars[B_U]);
                if (SAVE) {   // the tiles kept for the chain rule leave through TMA stores, straight from the operand slots
                    store(&tm.th, sQK, kT, chunk);
                    store(&tm.tl, sQK + kTileB, kT, chunk);
                }
                // Y = T~ Xk
                if (!wait(R_XK, par)) break;
                tc_fence_after_sync();
                if (SAVE) {   // (requested before the products are issued: the issue takes as long as the store's reads)
                    store(&tm.xk, sBig + 2 * kTileB, kT, chunk);
                    tma_store_commit();
                }
                mma_small(tmem + 384, aQ, OP_K, aBig + 2 * kTileB, OP_MN, 8, 128, false);
                mma_small(tmem + 384, aK, OP_K, aBig + 2 * kTileB, OP_MN, 8, 128, true);
                mma_small(tmem + 384, aQ, OP_K, aBig + 3 * kTileB, OP_MN, 8, 128, true);
                // B_Y lets the workers overwrite T~ (with U) and Xk (with Y): the stores must have read them
                if (SAVE) tma_store_wait_read();
                umma_commit(&bars[B_Y]);
                // Xq U and W^T U
                if (!wait(R_U, par)) break;
                tc_fence_after_sync();
                if (!KEYS) {
                    mma_small(tmem + 256, aBig, OP_K, aQ, OP_MN, 8, HD, false);
                    mma_small(tmem + 256, aBig + kTileB, OP_K, aQ, OP_MN, 8, HD, true);
                    mma_small(tmem + 256, aBig, OP_K, aK, OP_MN, 8, HD, true);
                }
                mma_small(tmem + 128, aW, OP_MN, aQ, OP_MN, 8, HD, false);
                mma_small(tmem + 128, aW, OP_MN, aK, OP_MN, 8, HD, true);
                umma_commit(&bars[B_G3A]);
                if (SAVE) {
                    store(&tm.u, sQK, HD, chunk);
                    tma_store_commit();
                }
                // Y^T W
                if (!wait(R_Y, par)) break;
                tc_fence_after_sync();
                mma_small(tmem + 384, aBig + 2 * kTileB, OP_MN, aW, OP_MN, 8, HD, false);
                mma_small(tmem + 384, aBig + 3 * kTileB, OP_MN, aW, OP_MN, 8, HD, true);
                umma_commit(&bars[B_G3B]);
                // next chunk: once this chunk's last product has retired every tile slot is free
                const int next = chunk + (int)gridDim.x;
                if (next < nchunks) {
                    if (!wait(B_G3B, par)) break;
                    if (SAVE) tma_store_wait_read();   // the U tile: the loads overwrite it
                    load(next);
                    if (!wait(B_LOAD, par ^ 1)) break;
                    tc_fence_after_sync();
                    mma_small(tmem + 0, aW, OP_K, aW, OP_K, KS, 128, false);
                    umma_commit(&bars[B_GM]);
                }
            }
            if (SAVE) tma_store_wait_all();
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ workers
        asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
        bool ok = true;
        uint32_t r[32];
        float v[32];
        uint32_t hi[16], lo[16];
        // lane 0 of every warp waits; the vote that follows is also the barrier that releases the other lanes
        auto wwait = [&](int b, uint32_t par) {
            bool good = true;
            if (lane == 0) good = mbar_wait(&bars[b], par, abort_flag, ST_PREP);
            good = wsync_and(good);
            tc_fence_after_sync();
            return good;
        };
        int chunk = blockIdx.x;
        for (uint32_t it = 0; chunk < nchunks; ++it, chunk += gridDim.x) {
            const uint32_t par = it & 1;
            const size_t grow = (size_t)chunk * kT + row;   // global row
            if (!(ok = wwait(B_GM, par))) break;

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
            wsync();

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
            wsync();
            for (int bi = 0; bi < kT / 16; ++bi) {   // inverted diagonal blocks into place (their upper triangles are zero)
                const int rr = tid >> 4, k = tid & 15;
                Xb[(bi * 16 + rr) * kLd + bi * 16 + k] = diagX[bi * 16 * 17 + rr * 17 + k];
            }
            wsync();
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
                    // T[i][j] = sum_k C[i][k] A^-1[k][j].  A^-1 is lower triangular with its zeros stored, so the rows k < j0
                    // could be skipped, but a loop that starts at the lane's own j0 puts every lane of a warp on a different
                    // row at the same time (no broadcast, bank conflicts: measured 6x slower than the full loop)
#pragma unroll 4
                    for (int k = 0; k < NB; ++k) {
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
                    wsync();
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
                    wsync();
                };
                merge(std::integral_constant<int, 16>{});
                merge(std::integral_constant<int, 32>{});
            }
            // Last level (64-row blocks) on the tensor cores: both products are 64 x 64 x 64, which the CUDA cores take
            // ten thousand cycles for (the triangular second product keeps only the warps with the long rows busy).  The
            // operands go as bf16 pairs (hi hi + hi lo + lo hi), the precision T~ itself is kept in afterwards.
            if (!(ok = wwait(B_XQK, par))) break;   // the products that read the Q and K tiles have retired
            {
                const int r_ = tid >> 2, seg = tid & 3;   // this thread: 16 columns of one row of C, A^-1 and B^-1
                const float* src[3] = {Xb + (64 + r_) * kLd + seg * 16, Xb + r_ * kLd + seg * 16, Xb + (64 + r_) * kLd + 64 + seg * 16};
#pragma unroll
                for (int m = 0; m < 3; ++m) {
                    uint32_t h8[8], l8[8];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const float4 f = *reinterpret_cast<const float4*>(src[m] + 4 * x);
                        const uint32_t a = pack_bf16(f.x, f.y), b = pack_bf16(f.z, f.w);
                        h8[2 * x] = a;
                        h8[2 * x + 1] = b;
                        l8[2 * x] = pack_bf16(f.x - __uint_as_float(a << 16), f.y - __uint_as_float(a & 0xffff0000u));
                        l8[2 * x + 1] = pack_bf16(f.z - __uint_as_float(b << 16), f.w - __uint_as_float(b & 0xffff0000u));
                    }
                    uint8_t* th_ = sQK + (2 * m) * kInvTileB;
                    uint8_t* tl_ = th_ + kInvTileB;
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        const uint32_t off = sw128_off((uint32_t)r_, (uint32_t)(seg * 2 + c));
                        *reinterpret_cast<uint4*>(th_ + off) = make_uint4(h8[4 * c], h8[4 * c + 1], h8[4 * c + 2], h8[4 * c + 3]);
                        *reinterpret_cast<uint4*>(tl_ + off) = make_uint4(l8[4 * c], l8[4 * c + 1], l8[4 * c + 2], l8[4 * c + 3]);
                    }
                }
                fence_proxy_async_smem();
                tc_fence_before_sync();
                mbar_arrive(&bars[R_M1]);
                if (!(ok = wwait(B_M1, par))) break;
                if (row < 64) {   // T: rows 0..63 of the accumulator -> bf16 pair, the right-hand operand of the second product
                    tmem_ld32(tl + 0 + half * 32, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int x = 0; x < 32; ++x) v[x] = __uint_as_float(r[x]);
                    split32(v, hi, lo);
                    tile_store_w16(sQK + 6 * kInvTileB, row, half * 32, hi);
                    tile_store_w16(sQK + 7 * kInvTileB, row, half * 32, lo);
                }
                fence_proxy_async_smem();
                tc_fence_before_sync();
                mbar_arrive(&bars[R_M2]);
                if (!(ok = wwait(B_M2, par))) break;
                if (row < 64) {   // -B^-1 T replaces C
                    tmem_ld32(tl + 64 + half * 32, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int x = 0; x < 8; ++x)
                        *reinterpret_cast<float4*>(Xb + (64 + row) * kLd + half * 32 + 4 * x) =
                            make_float4(-__uint_as_float(r[4 * x]), -__uint_as_float(r[4 * x + 1]), -__uint_as_float(r[4 * x + 2]),
                                        -__uint_as_float(r[4 * x + 3]));
                }
                tc_fence_before_sync();
                wsync();
            }

            // ---- T~ = X D as a bf16 pair into the Q / K tiles' space
            for (int c = 0; c < 2; ++c) {
                const int c0 = half * 64 + c * 32;
                float t[32];
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const float4 f = *reinterpret_cast<const float4*>(Xb + row * kLd + c0 + 4 * x);
                    v[4 * x] = f.x; v[4 * x + 1] = f.y; v[4 * x + 2] = f.z; v[4 * x + 3] = f.w;
                }
#pragma unroll
                for (int x = 0; x < 32; ++x) t[x] = v[x] * bt[c0 + x];
                split32(t, hi, lo);
                tile_store_w16(sQK, row, c0, hi);
                tile_store_w16(sQK + kTileB, row, c0, lo);
                if (SAVE) {
                    split32(v, hi, lo);
                    gstore_bf16_w16(p.sAh + grow * kT + c0, hi);
                    gstore_bf16_w16(p.sAl + grow * kT + c0, lo);
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(&bars[R_TT]);
            wsync();  // everyone has read the float32 buffer; it now becomes the Xq / Xk tiles

            // ---- E1b: Xk = strictLower(.) -> bf16 hi / lo tiles (slots 5, 6), then Xq = lower(.) (slots 3, 4); Xqn = -Xq -> global
            for (int c = 0; c < 2; ++c) {
                const int c0 = half * 64 + c * 32;
                tmem_ld32(tl + 256 + c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 32; ++x) v[x] = (c0 + x < row) ? __uint_as_float(r[x]) : 0.f;
                split32(v, hi, lo);
                tile_store_w16(sBig + 2 * kTileB, row, c0, hi);
                tile_store_w16(sBig + 3 * kTileB, row, c0, lo);
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars[R_XK]);
            for (int c = 0; c < (KEYS ? 0 : 2); ++c) {
                const int c0 = half * 64 + c * 32;
                tmem_ld32(tl + 128 + c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 32; ++x) v[x] = (c0 + x <= row) ? __uint_as_float(r[x]) : 0.f;
                split32(v, hi, lo);
                tile_store_w16(sBig, row, c0, hi);
                tile_store_w16(sBig + kTileB, row, c0, lo);
#pragma unroll
                for (int x = 0; x < 16; ++x) hi[x] ^= 0x80008000u;   // -Xq
                gstore_bf16_w16(p.Xqn + grow * kT + c0, hi);
            }

            // ---- E2: U -> hi / lo tiles over T~ (slots 1, 2) once Y = T~ Xk has retired; Y -> hi / lo tiles over Xk
            // (slots 5, 6); Yt = Y^T -> global
            if (!(ok = wwait(B_U, par))) break;
            uint32_t uh[HD / 64][16], ul[HD / 64][16];
#pragma unroll
            for (int c = 0; c < HD / 64; ++c) {
                const int c0 = half * (HD / 2) + c * 32;
                tmem_ld32(tl + 0 + c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 32; ++x) v[x] = __uint_as_float(r[x]);
                split32(v, uh[c], ul[c]);
            }
            if (!(ok = wwait(B_Y, par))) break;
#pragma unroll
            for (int c = 0; c < HD / 64; ++c) {
                const int c0 = half * (HD / 2) + c * 32;
                tile_store_w16(sQK, row, c0, uh[c]);
                tile_store_w16(sQK + kTileB, row, c0, ul[c]);
            }
            fence_proxy_async_smem();   // also covers the Xq tiles written above
            tc_fence_before_sync();
            mbar_arrive(&bars[R_U]);
            uint32_t yh[2][16];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int c0 = half * 64 + c * 32;
                tmem_ld32(tl + 384 + c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 32; ++x) v[x] = __uint_as_float(r[x]);
                split32(v, yh[c], lo);
                tile_store_w16(sBig + 2 * kTileB, row, c0, yh[c]);
                tile_store_w16(sBig + 3 * kTileB, row, c0, lo);
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars[R_Y]);
            if (!KEYS) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    unsigned short* yt = reinterpret_cast<unsigned short*>(p.Yt) + ((size_t)chunk * kT + half * 64 + c * 32) * kT + row;
#pragma unroll
                    for (int x = 0; x < 16; ++x) {
                        yt[(size_t)(2 * x) * kT] = (unsigned short)(yh[c][x] & 0xffffu);
                        yt[(size_t)(2 * x + 1) * kT] = (unsigned short)(yh[c][x] >> 16);
                    }
                }
            }

            // ---- E3: Qleft = Q - Xq U, P = I - W^T U, then Kright = K - Y^T W; the q / k rows are fetched while the
            // products run
            // At d = 128 a thread's half row is one 128-byte line: four lanes fetch four lines together, a quarter of each per
            // instruction (whole lines per request instead of 32 scattered pieces, which also hold up the products' operand reads)
            uint32_t rq[4][8], rk[4][8];
            uint4 pre_q[4], pre_k[4];
            {
                const __nv_bfloat16* gq = p.q + grow * HD + half * (HD / 2);
                const __nv_bfloat16* gk = p.k + grow * HD + half * (HD / 2);
                if (HD == 128) {
                    if (!KEYS) gload_f32x32_issue(reinterpret_cast<const float*>(gq), rq);
                    gload_f32x32_issue(reinterpret_cast<const float*>(gk), rk);
                } else {
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        if (!KEYS) pre_q[x] = reinterpret_cast<const uint4*>(gq)[x];
                        pre_k[x] = reinterpret_cast<const uint4*>(gk)[x];
                    }
                }
            }
            // in[] <- columns c * 32 .. + 31 of a fetched half row (`words`: the whole half row at d = 128, two bf16 per word)
            auto row_part = [&](const float (&words)[32], const uint4 (&pre)[4], int c, float (&in)[32]) {
                if (HD == 128) {
#pragma unroll
                    for (int x = 0; x < 16; ++x) {
                        const uint32_t u = __float_as_uint(words[16 * c + x]);
                        in[2 * x] = __uint_as_float(u << 16);
                        in[2 * x + 1] = __uint_as_float(u & 0xffff0000u);
                    }
                } else {
                    unpack_bf16x32(pre, in);
                }
            };
            const int next = chunk + (int)gridDim.x;
            float next_beta = 0.f;
            if (tid < kT && next < nchunks) next_beta = p.beta[(size_t)next * kT + tid];
            if (!(ok = wwait(B_G3A, par))) break;
            float words[32];
            if (HD == 128 && !KEYS) gload_f32x32_finish(rq, words);
#pragma unroll
            for (int c = 0; c < HD / 64; ++c) {
                const int c0 = half * (HD / 2) + c * 32;
                if (!KEYS) {
                    float in[32];
                    tmem_ld32(tl + 256 + c0, r);
                    tmem_ld_wait();
                    row_part(words, pre_q, c, in);
#pragma unroll
                    for (int x = 0; x < 32; ++x) v[x] = in[x] - __uint_as_float(r[x]);
                    gstore_bf16x32(p.ql + grow * HD + c0, v);
                }
                tmem_ld32(tl + 128 + c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 32; ++x) v[x] = ((c0 + x == row) ? 1.f : 0.f) - __uint_as_float(r[x]);
                split32(v, hi, lo);
                gstore_bf16_w16(p.Ph + ((size_t)chunk * HD + row) * HD + c0, hi, row < HD);
                gstore_bf16_w16(p.Pl + ((size_t)chunk * HD + row) * HD + c0, lo, row < HD);
            }
            if (!(ok = wwait(B_G3B, par))) break;
            if (HD == 128) gload_f32x32_finish(rk, words);
#pragma unroll
            for (int c = 0; c < HD / 64; ++c) {
                const int c0 = half * (HD / 2) + c * 32;
                float in[32];
                tmem_ld32(tl + 384 + c0, r);
                tmem_ld_wait();
                row_part(words, pre_k, c, in);
#pragma unroll
                for (int x = 0; x < 32; ++x) v[x] = in[x] - __uint_as_float(r[x]);
                gstore_bf16x32(p.kr + grow * HD + c0, v);
            }
            if (tid < kT) bt[tid] = next_beta;   // read again only after the next chunk's first wait (a worker barrier)
            tc_fence_before_sync();
            mbar_arrive(&bars[R_E3]);
        }
    }

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
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int grid = nchunks < sms ? nchunks : sms;
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e2 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PrepSmem::alloc);
        if (e2 != cudaSuccess) return e2;
        kern<<<grid, kThreads, PrepSmem::alloc, st>>>(tm, p, nchunks);
        return cudaGetLastError();
    };
    if (save == PREP_KEYS) return hd == 64 ? go(chunk_prep_kernel<64, PREP_KEYS>) : go(chunk_prep_kernel<128, PREP_KEYS>);
    if (hd == 64) return save ? go(chunk_prep_kernel<64, PREP_SAVE>) : go(chunk_prep_kernel<64, PREP_FWD>);
    return save ? go(chunk_prep_kernel<128, PREP_SAVE>) : go(chunk_prep_kernel<128, PREP_FWD>);
}

}  // namespace path
