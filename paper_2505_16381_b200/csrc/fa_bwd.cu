// Backward of the attention sweep (the paper gives no backward; this is the FlashAttention-2 style
// recomputation applied to the dyadic query / key versions of fa_fwd.cu).
//
//   P = exp(S - LSE),  dP = dO V^T,  dS = P o (dP - delta),  delta_i = dO_i . O_i
//   dV_J  = sum_I P^T dO_I                       dKv[l][J] = scale sum_{I at level l} dS^T Qv[l][I]
//   dQv[l][I] = scale sum_{J at level l} dS Kv[l][J]
//   gate prefix:  dG_m = sum_j dS_mj - sum_i dS_im  (row sums are written by dq_kernel, column sums by dkv_kernel;
//                 the row sums vanish in exact arithmetic but cancel the rounding of delta in the suffix sums)
//   diagonal chunk: dSd = lower(dS) (unscaled) is stored for the per-chunk chain rule.
//
// Two kernels so that every accumulator stays in tensor memory and nothing is added atomically:
//   dkv_kernel: one CTA per key chunk J, sweeps the query chunks I = J..N-1 with transposed tiles
//               (TMEM lanes = keys): S^T = K Q^T, dP^T = V dO^T, dV += P^T dO, dK += dS^T Q.
//   dq_kernel : one CTA per query chunk I, sweeps J = I-1..0: S = Q K^T, dP = dO V^T, dQ += dS K.
// The accumulator of a version is flushed to global memory when the sweep crosses into the next level.
// P^T / dS^T (dkv) and dS (dq) never touch shared memory: they overwrite the first half of the columns their thread
// read, as packed bf16, and enter the second products as tensor-memory A operands.  The shared memory this frees
// double-buffers the per-step tiles.
// Warps: 0 = TMA producer, 1 = tcgen05 MMA issuer, 2-9 = elementwise math (two warps per TMEM lane quadrant, each
// taking 64 of the 128 columns of a row).
#include "common.cuh"
#include "tc5.cuh"

namespace path {
using namespace tc5;

namespace {

constexpr int kTile = 128;
constexpr uint32_t kSlotBytes = 32768;
constexpr uint32_t kPanelBytes = 16384;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// D[tmem] (+)= A B^T with both operands K-major [rows][kdim] tiles (two 64-column panels per 128 of kdim).
__device__ __forceinline__ void mma_kk(uint32_t d_tmem, uint32_t a0, uint32_t b0, int kdim, uint32_t idesc, bool acc) {
    for (int kk = 0; kk < kdim / 16; ++kk) {
        const uint32_t off = (kk >> 2) * kPanelBytes + (kk & 3) * 32;
        umma_ss(d_tmem, umma_desc(a0 + off, 16, 1024), umma_desc(b0 + off, 16, 1024), idesc, (acc || kk > 0) ? 1u : 0u);
    }
}
// D[tmem] (+)= A B with A in tensor memory (packed bf16: the 64 contraction indices [64h, 64h+64) of a row sit in the
// 32 columns starting at a_col + 64h) and B MN-major [128 (k)][HD] in shared memory.
__device__ __forceinline__ void mma_tn(uint32_t d_tmem, uint32_t a_col, uint32_t b0, uint32_t idesc, bool acc) {
    for (int kk = 0; kk < kTile / 16; ++kk)
        umma_ts(d_tmem, a_col + (kk >> 2) * 64 + (kk & 3) * 8, umma_desc(b0 + kk * 2048, kPanelBytes, 1024), idesc,
                (acc || kk > 0) ? 1u : 0u);
}

__device__ __forceinline__ void tma_tile(uint8_t* dst, const CUtensorMap* m, uint64_t* bar, int kdim, int row0) {
    for (int h = 0; h < kdim / 64; ++h) tma_load_2d(dst + h * kPanelBytes, m, bar, h * 64, row0);
}

// ------------------------------------------------------------------------------------------------ dK, dV
enum { K_KFULL = 0, K_KEMPTY, K_VFULL, K_QFULL, K_QEMPTY = K_QFULL + 2, K_DOFULL = K_QEMPTY + 2,
       K_DOEMPTY = K_DOFULL + 2, K_SFULL = K_DOEMPTY + 2, K_PFULL, K_FINAL, K_COUNT };

template <int HD, bool GATE>
__global__ void __launch_bounds__(320, 1) dkv_kernel(const __grid_constant__ BwdTensorMaps tm, const BwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sK = smem;
    uint8_t* sV = sK + kSlotBytes;
    uint8_t* sQ = sV + kSlotBytes;          // 2 slots: rawQ, Xqn, then Q of step t >= 1 in slot (t + 1) & 1
    uint8_t* sDO = sQ + 2 * kSlotBytes;     // 2 slots: dO(0), Yt, then dO of step t >= 1 in slot (t + 1) & 1
    uint64_t* bars = (uint64_t*)(sDO + 2 * kSlotBytes);
    uint32_t* tmem_slot = (uint32_t*)(bars + K_COUNT);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    float* rowstat = (float*)(smem + 6 * kSlotBytes + 256);  // [2][3][128]: lse2, delta, G of the query chunk
    float* dsum_x = rowstat + 2 * 3 * kTile;                 // [128] exchange of the gate row sums

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int J = blockIdx.x, s = blockIdx.y;
    const int T = p.N - J;

    if (threadIdx.x == 0) {
        for (int i = 0; i < K_COUNT; ++i) mbar_init(&bars[i], i == K_PFULL ? 256u : 1u);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    constexpr uint32_t colS = 0, colDP = 128, colDV = 256, colDK = 384;
    const int rowJ = s * p.Lp + J * kTile;
    auto ver_row = [&](int slot, int chunk) { return (slot * p.S + s) * p.Lp + chunk * kTile; };
    auto level = [&](int t) { return t == 0 ? -1 : msb32((unsigned)((J + t) ^ J)); };

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int nk = 0;
            auto wait_empty = [&](int bar, int use) {
                if (ok && !mbar_wait(&bars[bar], (use & 1) ^ 1, abort_flag, ST_DKV_PRODUCER)) ok = false;
            };
            auto ring_load = [&](uint8_t* base, int bfull, int bempty, int item, const CUtensorMap* m, int kdim, int row0) {
                const int slot = item & 1;
                wait_empty(bempty + slot, item >> 1);
                if (!ok) return;
                mbar_expect_tx(&bars[bfull + slot], (uint32_t)(kTile * kdim * 2));
                tma_tile(base + slot * kSlotBytes, m, &bars[bfull + slot], kdim, row0);
            };
            for (int t = 0; t < T && ok; ++t) {
                const int I = J + t, l = level(t);
                if (t == 0 || l != level(t - 1)) {
                    wait_empty(K_KEMPTY, nk);
                    if (!ok) break;
                    mbar_expect_tx(&bars[K_KFULL], kTile * HD * 2);
                    if (t == 0) tma_tile(sK, &tm.k_raw, &bars[K_KFULL], HD, rowJ);
                    else tma_tile(sK, &tm.kv, &bars[K_KFULL], HD, ver_row(kslot(l, J), J));
                    ++nk;
                }
                if (t == 0) {
                    mbar_expect_tx(&bars[K_VFULL], kTile * HD * 2);
                    tma_tile(sV, &tm.v, &bars[K_VFULL], HD, rowJ);
                    ring_load(sQ, K_QFULL, K_QEMPTY, 0, &tm.q_raw, HD, rowJ);
                    ring_load(sDO, K_DOFULL, K_DOEMPTY, 0, &tm.d_o, HD, rowJ);
                    ring_load(sQ, K_QFULL, K_QEMPTY, 1, &tm.xqn, kTile, rowJ);
                    ring_load(sDO, K_DOFULL, K_DOEMPTY, 1, &tm.yt, kTile, rowJ);
                } else {
                    ring_load(sQ, K_QFULL, K_QEMPTY, t + 1, &tm.qv, HD, ver_row(qslot(l, I), I));
                    ring_load(sDO, K_DOFULL, K_DOEMPTY, t + 1, &tm.d_o, HD, s * p.Lp + I * kTile);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idescT = umma_idesc(128, 128, 0, 0);
            constexpr uint32_t idescD = umma_idesc(128, HD, 0, 1);
            bool ok = true;
            int nk = 0;
            auto wait = [&](int bar, int parity) {
                if (ok && !mbar_wait(&bars[bar], parity & 1, abort_flag, ST_DKV_MMA)) ok = false;
            };
            for (int t = 0; t < T && ok; ++t) {
                const int l = level(t);
                const int item = (t == 0) ? 0 : t + 1, slot = item & 1;
                const uint32_t aQ = smem_u32(sQ + slot * kSlotBytes), aDO = smem_u32(sDO + slot * kSlotBytes);
                if (t == 0 || l != level(t - 1)) { wait(K_KFULL, nk); ++nk; }
                wait(K_QFULL + slot, item >> 1);
                wait(K_DOFULL + slot, item >> 1);
                if (t == 0) { wait(K_VFULL, 0); wait(K_QFULL + 1, 0); wait(K_DOFULL + 1, 0); }
                tc_fence_after_sync();
                if (!ok) break;
                mma_kk(tmem + colS, smem_u32(sK), aQ, HD, idescT, false);
                if (t == 0) mma_kk(tmem + colS, smem_u32(sDO + kSlotBytes), smem_u32(sQ + kSlotBytes), kTile, idescT, true);
                mma_kk(tmem + colDP, smem_u32(sV), aDO, HD, idescT, false);
                umma_commit(&bars[K_SFULL]);
                if (t == 0) {   // raw q and the two correction operands are only needed by the products above
                    umma_commit(&bars[K_QEMPTY + 0]);
                    umma_commit(&bars[K_QEMPTY + 1]);
                    umma_commit(&bars[K_DOEMPTY + 1]);
                }
                if (t + 1 < T && level(t + 1) != l) umma_commit(&bars[K_KEMPTY]);
                wait(K_PFULL, t);
                tc_fence_after_sync();
                if (!ok) break;
                mma_tn(tmem + colDV, tmem + colS, aDO, idescD, t > 0);
                if (t > 0) {
                    mma_tn(tmem + colDK, tmem + colDP, aQ, idescD, !(t == 1 || l != level(t - 1)));
                    umma_commit(&bars[K_QEMPTY + slot]);
                }
                umma_commit(&bars[K_DOEMPTY + slot]);
                if (t == T - 1) umma_commit(&bars[K_FINAL]);
            }
        }
    } else {
        const int q4 = warp & 3, h = (warp - 2) >> 2, row = q4 * 32 + lane;
        const int tid = threadIdx.x - 64;       // 0..255
        const uint32_t tlane = tmem + ((uint32_t)(q4 * 32) << 16);
        const int kj = J * kTile + row;          // key position of this thread's row
        const float sl2 = p.scale * kLog2e;
        float gj2 = 0.f, dsum = 0.f;
        if (GATE) gj2 = p.G[(size_t)s * p.Lp + kj] * kLog2e;
        bool ok = true;
        uint32_t rs[32], rp[32];
        constexpr int CW = HD / 2;               // accumulator columns per thread when flushing
        auto flush_dk = [&](int lvl) {
            float* dst = p.dkv + ((size_t)ver_row(kslot(lvl, J), J) + row) * HD + h * CW;
            for (int c = 0; c < CW / 32; ++c) {
                tmem_ld32(tlane + colDK + h * CW + c * 32, rs);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 8; ++x)
                    reinterpret_cast<float4*>(dst + c * 32)[x] =
                        make_float4(__uint_as_float(rs[4 * x]) * p.scale, __uint_as_float(rs[4 * x + 1]) * p.scale,
                                    __uint_as_float(rs[4 * x + 2]) * p.scale, __uint_as_float(rs[4 * x + 3]) * p.scale);
            }
        };
        for (int t = 0; t < T; ++t) {
            const int I = J + t, b = t & 1;
            float* st_ = rowstat + b * 3 * kTile;
            if (tid < kTile) {
                const size_t gi = (size_t)s * p.Lp + I * kTile + tid;
                st_[tid] = p.lse2[gi];
                st_[kTile + tid] = p.delta[gi];
                if (GATE) st_[2 * kTile + tid] = p.G[gi] * kLog2e;
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (ok && !mbar_wait(&bars[K_SFULL], t & 1, abort_flag, ST_DKV_COMPUTE)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after_sync();
            if (ok) {
                // S^T / dP^T ready means every earlier product has retired: dK of the finished level can be flushed
                if (t >= 2 && level(t) != level(t - 1)) flush_dk(level(t - 1));
                uint32_t pkP[32], pkS[32];
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int c0 = h * 64 + c * 32;      // query columns of this pass
                    tmem_ld32(tlane + colS + c0, rs);
                    tmem_ld32(tlane + colDP + c0, rp);
                    tmem_ld_wait();
                    float dsv[32];
#pragma unroll
                    for (int x = 0; x < 32; ++x) {
                        const int col = c0 + x;
                        float v = __uint_as_float(rs[x]) * sl2 - st_[col];
                        if (GATE) v += st_[2 * kTile + col] - gj2;
                        float pr = ex2(v);
                        if (t == 0 && col < row) pr = 0.f;
                        const float ds = pr * (__uint_as_float(rp[x]) - st_[kTile + col]);
                        dsum += ds;
                        dsv[x] = ds;
                        rs[x] = __float_as_uint(pr);
                    }
#pragma unroll
                    for (int x = 0; x < 32; x += 2) {
                        pkP[c * 16 + (x >> 1)] = pack_bf16(__uint_as_float(rs[x]), __uint_as_float(rs[x + 1]));
                        pkS[c * 16 + (x >> 1)] = pack_bf16(dsv[x], dsv[x + 1]);
                    }
                    if (t == 0) {
                        float* dsd = p.dsd + ((size_t)(s * p.N + J) * kTile) * kTile;
#pragma unroll
                        for (int x = 0; x < 32; ++x) dsd[(size_t)(c0 + x) * kTile + row] = dsv[x];
                    }
                }
                tmem_st32(tlane + colS + h * 64, pkP);
                tmem_st32(tlane + colDP + h * 64, pkS);
                tmem_st_wait();
            }
            tc_fence_before_sync();
            mbar_arrive(&bars[K_PFULL]);
        }
        if (ok && !mbar_wait(&bars[K_FINAL], 0, abort_flag, ST_DKV_COMPUTE)) ok = false;
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after_sync();
        if (GATE) {   // the two threads of a key row add their halves of the column sum
            if (h == 1) dsum_x[row] = dsum;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (h == 0 && ok) p.dG[(size_t)s * p.Lp + kj] = -(dsum + dsum_x[row]);
        }
        if (ok) {
            if (T > 1) flush_dk(level(T - 1));
            else {  // last chunk: no later query chunk, the boundary-adjusted keys get a zero gradient from the sweep
                float4* dst = reinterpret_cast<float4*>(p.dkv + ((size_t)ver_row(0, J) + row) * HD + h * CW);
                for (int x = 0; x < CW / 4; ++x) dst[x] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            for (int c = 0; c < CW / 32; ++c) {
                tmem_ld32(tlane + colDV + h * CW + c * 32, rs);
                tmem_ld_wait();
                if (kj < p.L) {
                    uint4* dst = reinterpret_cast<uint4*>((__nv_bfloat16*)p.dv + ((size_t)s * p.L + kj) * HD + h * CW + c * 32);
#pragma unroll
                    for (int x = 0; x < 4; ++x)
                        dst[x] = make_uint4(pack_bf16(__uint_as_float(rs[8 * x]), __uint_as_float(rs[8 * x + 1])),
                                            pack_bf16(__uint_as_float(rs[8 * x + 2]), __uint_as_float(rs[8 * x + 3])),
                                            pack_bf16(__uint_as_float(rs[8 * x + 4]), __uint_as_float(rs[8 * x + 5])),
                                            pack_bf16(__uint_as_float(rs[8 * x + 6]), __uint_as_float(rs[8 * x + 7])));
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag != 0) atomicCAS(p.status, 0u, *abort_flag);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, 512);
    }
}

// ------------------------------------------------------------------------------------------------ dQ
enum { Q_QFULL = 0, Q_QEMPTY, Q_DOFULL, Q_KFULL, Q_KEMPTY = Q_KFULL + 2, Q_VFULL = Q_KEMPTY + 2,
       Q_VEMPTY = Q_VFULL + 2, Q_SFULL = Q_VEMPTY + 2, Q_DSFULL, Q_FINAL, Q_COUNT };

template <int HD, bool GATE>
__global__ void __launch_bounds__(320, 1) dq_kernel(const __grid_constant__ BwdTensorMaps tm, const BwdParams p) {
    const int I = (int)gridDim.x - 1 - (int)blockIdx.x, s = blockIdx.y;
    if (I == 0) {  // chunk 0 has no earlier keys: its boundary-adjusted queries get a zero gradient from the sweep
        float4* dst = reinterpret_cast<float4*>(p.dqv + (size_t)s * p.Lp * HD);
        for (int i = threadIdx.x; i < kTile * HD / 4; i += blockDim.x) dst[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;
    uint8_t* sDO = sQ + kSlotBytes;
    uint8_t* sK = sDO + kSlotBytes;        // 2 slots
    uint8_t* sV = sK + 2 * kSlotBytes;     // 2 slots
    uint64_t* bars = (uint64_t*)(sV + 2 * kSlotBytes);
    uint32_t* tmem_slot = (uint32_t*)(bars + Q_COUNT);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    float* gk = (float*)(smem + 6 * kSlotBytes + 256);  // [2][128] gate prefix of the key chunk
    float* dsum_x = gk + 2 * kTile;                     // [128]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = I;  // steps t = 0..I-1, J = I-1-t

    if (threadIdx.x == 0) {
        for (int i = 0; i < Q_COUNT; ++i) mbar_init(&bars[i], i == Q_DSFULL ? 256u : 1u);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    constexpr uint32_t colS = 0, colDP = 128, colDQ = 256;
    auto ver_row = [&](int slot, int chunk) { return (slot * p.S + s) * p.Lp + chunk * kTile; };
    auto level = [&](int t) { return msb32((unsigned)(I ^ (I - 1 - t))); };

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int nq = 0;
            auto wait_empty = [&](int bar, int parity) {
                if (ok && !mbar_wait(&bars[bar], parity & 1, abort_flag, ST_DQ_PRODUCER)) ok = false;
            };
            mbar_expect_tx(&bars[Q_DOFULL], kTile * HD * 2);
            tma_tile(sDO, &tm.d_o, &bars[Q_DOFULL], HD, s * p.Lp + I * kTile);
            for (int t = 0; t < T && ok; ++t) {
                const int J = I - 1 - t, l = level(t), slot = t & 1;
                if (t == 0 || l != level(t - 1)) {
                    wait_empty(Q_QEMPTY, (nq & 1) ^ 1);
                    if (!ok) break;
                    mbar_expect_tx(&bars[Q_QFULL], kTile * HD * 2);
                    tma_tile(sQ, &tm.qv, &bars[Q_QFULL], HD, ver_row(qslot(l, I), I));
                    ++nq;
                }
                wait_empty(Q_KEMPTY + slot, ((t >> 1) & 1) ^ 1);
                if (!ok) break;
                mbar_expect_tx(&bars[Q_KFULL + slot], kTile * HD * 2);
                tma_tile(sK + slot * kSlotBytes, &tm.kv, &bars[Q_KFULL + slot], HD, ver_row(kslot(l, J), J));
                wait_empty(Q_VEMPTY + slot, ((t >> 1) & 1) ^ 1);
                if (!ok) break;
                mbar_expect_tx(&bars[Q_VFULL + slot], kTile * HD * 2);
                tma_tile(sV + slot * kSlotBytes, &tm.v, &bars[Q_VFULL + slot], HD, s * p.Lp + J * kTile);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idescS = umma_idesc(128, 128, 0, 0);
            constexpr uint32_t idescD = umma_idesc(128, HD, 0, 1);
            bool ok = true;
            int nq = 0;
            auto wait = [&](int bar, int parity) {
                if (ok && !mbar_wait(&bars[bar], parity & 1, abort_flag, ST_DQ_MMA)) ok = false;
            };
            wait(Q_DOFULL, 0);
            for (int t = 0; t < T && ok; ++t) {
                const int l = level(t), slot = t & 1;
                if (t == 0 || l != level(t - 1)) { wait(Q_QFULL, nq); ++nq; }
                wait(Q_KFULL + slot, t >> 1);
                wait(Q_VFULL + slot, t >> 1);
                tc_fence_after_sync();
                if (!ok) break;
                // these overwrite S and dS of the previous step: in-order execution puts them after its dQ product,
                // and that product was only issued once every thread had finished reading (Q_DSFULL)
                mma_kk(tmem + colS, smem_u32(sQ), smem_u32(sK + slot * kSlotBytes), HD, idescS, false);
                mma_kk(tmem + colDP, smem_u32(sDO), smem_u32(sV + slot * kSlotBytes), HD, idescS, false);
                umma_commit(&bars[Q_SFULL]);
                umma_commit(&bars[Q_VEMPTY + slot]);
                if (t + 1 < T && level(t + 1) != l) umma_commit(&bars[Q_QEMPTY]);
                wait(Q_DSFULL, t);
                tc_fence_after_sync();
                if (!ok) break;
                mma_tn(tmem + colDQ, tmem + colDP, smem_u32(sK + slot * kSlotBytes), idescD, !(t == 0 || l != level(t - 1)));
                umma_commit(&bars[Q_KEMPTY + slot]);
                if (t == T - 1) umma_commit(&bars[Q_FINAL]);
            }
        }
    } else {
        const int q4 = warp & 3, h = (warp - 2) >> 2, row = q4 * 32 + lane;
        const int tid = threadIdx.x - 64;
        const uint32_t tlane = tmem + ((uint32_t)(q4 * 32) << 16);
        const size_t qi = (size_t)s * p.Lp + I * kTile + row;
        const float sl2 = p.scale * kLog2e;
        const float lse2 = p.lse2[qi], delta = p.delta[qi];
        float gi2 = 0.f, dsum = 0.f;
        if (GATE) gi2 = p.G[qi] * kLog2e;
        bool ok = true;
        uint32_t rs[32], rp[32];
        constexpr int CW = HD / 2;
        auto flush_dq = [&](int lvl) {
            float* dst = p.dqv + ((size_t)ver_row(qslot(lvl, I), I) + row) * HD + h * CW;
            for (int c = 0; c < CW / 32; ++c) {
                tmem_ld32(tlane + colDQ + h * CW + c * 32, rs);
                tmem_ld_wait();
#pragma unroll
                for (int x = 0; x < 8; ++x)
                    reinterpret_cast<float4*>(dst + c * 32)[x] =
                        make_float4(__uint_as_float(rs[4 * x]) * p.scale, __uint_as_float(rs[4 * x + 1]) * p.scale,
                                    __uint_as_float(rs[4 * x + 2]) * p.scale, __uint_as_float(rs[4 * x + 3]) * p.scale);
            }
        };
        for (int t = 0; t < T; ++t) {
            const int J = I - 1 - t, b = t & 1;
            if (GATE) {
                if (tid < kTile) gk[b * kTile + tid] = p.G[(size_t)s * p.Lp + J * kTile + tid] * kLog2e;
                asm volatile("bar.sync 1, 256;" ::: "memory");
            }
            if (ok && !mbar_wait(&bars[Q_SFULL], t & 1, abort_flag, ST_DQ_COMPUTE)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after_sync();
            if (ok) {
                if (t >= 1 && level(t) != level(t - 1)) flush_dq(level(t - 1));
                uint32_t pk[32];
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int c0 = h * 64 + c * 32;   // key columns of this pass
                    tmem_ld32(tlane + colS + c0, rs);
                    tmem_ld32(tlane + colDP + c0, rp);
                    tmem_ld_wait();
#pragma unroll
                    for (int x = 0; x < 32; x += 2) {
                        float v0 = __uint_as_float(rs[x]) * sl2 - lse2, v1 = __uint_as_float(rs[x + 1]) * sl2 - lse2;
                        if (GATE) {
                            v0 += gi2 - gk[b * kTile + c0 + x];
                            v1 += gi2 - gk[b * kTile + c0 + x + 1];
                        }
                        const float d0 = ex2(v0) * (__uint_as_float(rp[x]) - delta);
                        const float d1 = ex2(v1) * (__uint_as_float(rp[x + 1]) - delta);
                        if (GATE) dsum += d0 + d1;
                        pk[c * 16 + (x >> 1)] = pack_bf16(d0, d1);
                    }
                }
                tmem_st32(tlane + colDP + h * 64, pk);
                tmem_st_wait();
            }
            tc_fence_before_sync();
            mbar_arrive(&bars[Q_DSFULL]);
        }
        if (ok && !mbar_wait(&bars[Q_FINAL], 0, abort_flag, ST_DQ_COMPUTE)) ok = false;
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after_sync();
        if (GATE) {
            if (h == 1) dsum_x[row] = dsum;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (h == 0 && ok) p.dGrow[qi] = dsum + dsum_x[row];
        }
        if (ok) flush_dq(level(T - 1));
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag != 0) atomicCAS(p.status, 0u, *abort_flag);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, 512);
    }
}

// delta_i = dO_i . O_i and lse2_i = lse_i * log2(e), padded to Lp (tail rows: 0).  One warp per row.
template <int HD>
__global__ void rowstats_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                                const float* __restrict__ lse, float* __restrict__ delta, float* __restrict__ lse2,
                                int L, int Lp) {
    const int s = blockIdx.y;
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (i >= Lp) return;
    float acc = 0.f;
    if (i < L) {
        const size_t base = ((size_t)s * L + i) * HD;
        for (int x = lane * 2; x < HD; x += 64) {
            const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(o + base + x));
            const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(d_o + base + x));
            acc += a.x * b.x + a.y * b.y;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) {
        delta[(size_t)s * Lp + i] = acc;
        lse2[(size_t)s * Lp + i] = (i < L) ? lse[(size_t)s * L + i] * kLog2e : 0.f;
    }
}

template <class K>
cudaError_t set_smem(K kern, int bytes) {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

constexpr int kDkvSmem = 6 * kSlotBytes + 256 + (2 * 3 + 1) * kTile * 4 + 1024;
constexpr int kDqSmem = 6 * kSlotBytes + 256 + 3 * kTile * 4 + 1024;

template <int HD, bool GATE>
cudaError_t launch_one(const BwdTensorMaps& tm, const BwdParams& p, int which, cudaStream_t st) {
    if (which == 0) {
        cudaError_t e = set_smem(dkv_kernel<HD, GATE>, kDkvSmem);
        if (e != cudaSuccess) return e;
        dkv_kernel<HD, GATE><<<dim3(p.N, p.S), 320, kDkvSmem, st>>>(tm, p);
    } else {
        cudaError_t e = set_smem(dq_kernel<HD, GATE>, kDqSmem);
        if (e != cudaSuccess) return e;
        dq_kernel<HD, GATE><<<dim3(p.N, p.S), 320, kDqSmem, st>>>(tm, p);
    }
    return cudaGetLastError();
}

}  // namespace

// which = 0: dK/dV sweep, which = 1: dQ sweep.
cudaError_t launch_fa_bwd(const BwdTensorMaps& tm, const BwdParams& p, int hd, int which, cudaStream_t st) {
    if (hd == 64) return p.G ? launch_one<64, true>(tm, p, which, st) : launch_one<64, false>(tm, p, which, st);
    return p.G ? launch_one<128, true>(tm, p, which, st) : launch_one<128, false>(tm, p, which, st);
}

cudaError_t launch_rowstats(const void* o, const void* d_o, const float* lse, float* delta, float* lse2, int S, int L,
                            int Lp, int hd, cudaStream_t st) {
    dim3 grid((Lp + 7) / 8, S);
    if (hd == 64)
        rowstats_kernel<64><<<grid, 256, 0, st>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)d_o, lse, delta, lse2, L, Lp);
    else
        rowstats_kernel<128><<<grid, 256, 0, st>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)d_o, lse, delta, lse2, L, Lp);
    return cudaGetLastError();
}

}  // namespace path
