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
// read, as packed bf16, and enter the second products as tensor-memory A operands.
//
// The elementwise work of a step is split in two so that it overlaps the tensor pipe: part A turns S into P (the
// exponentials) as soon as S is there, while the dP product still runs; part B forms dS once dP has arrived.  The
// products are issued in the order  dV(t), S(t+1), dK(t), dP(t+1)  (dkv) and  dQ(t), dP(t+1), S(t+2)  (dq, which has
// room for two S tiles), so the pipe always has the next step's logits in flight.
// Warps: 0 = TMA producer, 1 = tcgen05 MMA issuer, 2-3 idle (their registers go to the others), 4-11 = elementwise
// math (two warps per TMEM lane quadrant, each taking 64 of the 128 columns of a row).
#include <type_traits>
#include "common.cuh"
#include "tc5.cuh"
#include "tileops.cuh"

namespace path {
using namespace tc5;

namespace {

constexpr int kTile = 128;
constexpr uint32_t kSlotBytes = 32768;
constexpr uint32_t kPanelBytes = 16384;
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kSmemAlloc = 232448;   // everything an SM offers one CTA

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Two-wide float arithmetic on register pairs.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// A warp writes its 32 accumulator rows as bf16: lane L holds CW consecutive columns of row L, scaled by `mul`; `dst`
// is the first of them in the lane's own row.  One 32-column piece at a time (this runs inside the sweeps' hot loops).
template <int CW>
__device__ __forceinline__ void store_acc_bf16(__nv_bfloat16* dst, uint32_t tcol, float mul) {
#pragma unroll 1
    for (int c = 0; c < CW / 32; ++c) {
        uint32_t r[32], w[16];
        tmem_ld32(tcol + c * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 16; ++x) w[x] = pack_bf16(__uint_as_float(r[2 * x]) * mul, __uint_as_float(r[2 * x + 1]) * mul);
        tile::gstore_bf16_w16(dst + c * 32, w);
    }
}

// Plain (untiled) bulk copy global -> shared, completion counted in bytes on `bar`; 16-byte aligned, size % 16 == 0.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
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

// D[tmem] (+)= A B^T with both operands K-major [rows][kdim] tiles (two 64-column panels per 128 of kdim).  Descriptors
// advance by their low word only (32 bytes per step, the next panel after four steps).
__device__ __forceinline__ void mma_kk(uint32_t d_tmem, uint32_t a0, uint32_t b0, int kdim, uint32_t idesc, bool acc) {
    uint32_t a_lo = umma_desc_lo(a0, 16), b_lo = umma_desc_lo(b0, 16);
#pragma unroll
    for (int kk = 0; kk < kdim / 16; ++kk) {
        umma_ss(d_tmem, umma_desc_join(a_lo), umma_desc_join(b_lo), idesc, (acc || kk > 0) ? 1u : 0u);
        const uint32_t step = (kk & 3) == 3 ? (kPanelBytes - 96u) >> 4 : 2u;
        a_lo += step;
        b_lo += step;
    }
}
// D[tmem] (+)= A B with A in tensor memory (packed bf16: the 64 contraction indices [64h, 64h+64) of a row sit in the
// 32 columns starting at a_col + 64h) and B MN-major [128 (k)][HD] in shared memory (2048 bytes per step).
__device__ __forceinline__ void mma_tn(uint32_t d_tmem, uint32_t a_col, uint32_t b0, uint32_t idesc, bool acc) {
    uint32_t b_lo = umma_desc_lo(b0, kPanelBytes);
#pragma unroll
    for (int kk = 0; kk < kTile / 16; ++kk) {
        umma_ts(d_tmem, a_col + (kk >> 2) * 64 + (kk & 3) * 8, umma_desc_join(b_lo), idesc, (acc || kk > 0) ? 1u : 0u);
        b_lo += 128u;
    }
}

__device__ __forceinline__ void tma_tile(uint8_t* dst, const CUtensorMap* m, uint64_t* bar, int kdim, int row0) {
    for (int h = 0; h < kdim / 64; ++h) tma_load_2d(dst + h * kPanelBytes, m, bar, h * 64, row0);
}

// ------------------------------------------------------------------------------------------------ dK, dV
// Persistent: the work items (one key chunk of one slice each) are listed slice after slice as pairs (longest,
// shortest), (second longest, second shortest), ...; CTA c takes the pairs c, c + gridDim.x, ...  Every ring and phase
// counter runs on across items, so the loads and the first products of the next item overlap the write-out of the
// current one.
enum { K_KFULL = 0, K_KEMPTY, K_VFULL, K_VEMPTY, K_QFULL, K_QEMPTY = K_QFULL + 3, K_DOFULL = K_QEMPTY + 3,
       K_DOEMPTY = K_DOFULL + 2, K_SFULL = K_DOEMPTY + 2, K_DPFULL, K_PFULL, K_DSFULL, K_ACCFULL, K_ACCFREE,
       K_STFULL, K_STEMPTY = K_STFULL + 2, K_COUNT = K_STEMPTY + 2 };
constexpr uint32_t kDkvStat = 7 * kSlotBytes + 256;           // [2][2][128] floats: -lse2 (plus gate), -delta
constexpr uint32_t kDkvTotal = kDkvStat + 2 * 2 * kTile * 4 + kTile * 4;   // + [128] exchange of the gate column sums

template <int HD, bool GATE>
__global__ void __launch_bounds__(384, 1) dkv_kernel(const __grid_constant__ BwdTensorMaps tm, const BwdParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    if ((uint32_t)(smem - smem_raw) + kDkvTotal > kSmemAlloc) {   // uniform over the CTA
        if (threadIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)ST_DKV_PRODUCER);
        return;
    }
    uint8_t* sK = smem;
    uint8_t* sV = sK + kSlotBytes;
    uint8_t* sQ = sV + kSlotBytes;          // ring of 3; per item: rawQ, Xqn, then Q of step t >= 1 (entry t + 1)
    uint8_t* sDO = sQ + 3 * kSlotBytes;     // ring of 2; per item: Yt, then dO of step t (entry t + 1)
    uint64_t* bars = (uint64_t*)(smem + 7 * kSlotBytes);
    uint32_t* tmem_slot = (uint32_t*)(bars + K_COUNT);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    float* rowstat = (float*)(smem + kDkvStat);
    float* dsum_x = rowstat + 2 * 2 * kTile;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int items = p.N * p.S;

    if (threadIdx.x == 0) {
        for (int i = 0; i < K_COUNT; ++i)
            mbar_init(&bars[i], (i == K_PFULL || i == K_DSFULL || i == K_ACCFREE || i == K_STEMPTY || i == K_STEMPTY + 1)
                                    ? 256u : 1u);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 2 && lane < 8) tma_prefetch_desc(reinterpret_cast<const CUtensorMap*>(&tm) + lane);
    if (warp == 1) tmem_alloc(tmem_slot, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    constexpr uint32_t colS = 0, colDP = 128, colDV = 256, colDK = 384;
    // k-th work item of this CTA
    auto item_of = [&](int k, int& J, int& s) {
        const int w = 2 * ((int)blockIdx.x + (k >> 1) * (int)gridDim.x) + (k & 1);
        if (w >= items) return false;
        s = w / p.N;
        const int j = w % p.N;
        J = (j & 1) ? p.N - 1 - (j >> 1) : (j >> 1);
        return true;
    };
    int J = 0, s = 0;   // current item of this thread's role
    auto qrow = [&](int lvl, int chunk) { return qver_row(p.vl, s, lvl, chunk); };   // first row of a version tile
    auto krow = [&](int lvl, int chunk) { return kver_row(p.vl, s, lvl, chunk); };
    auto row0 = [&](int chunk) { return (long)s * p.Lp + (long)chunk * kTile; };      // plane 0
    auto level = [&](int t) { return t == 0 ? -1 : msb32((unsigned)((J + t) ^ J)); };
    // query chunks this key chunk meets (I = J .. J + T - 1): all later ones, or fewer when the gate has made the far
    // pairs negligible (every warp role reads the same precomputed number)
    auto steps_of = [&](int J, int s) { return p.nvisit ? min(p.N - J, p.nvisit[s * p.N + J]) : p.N - J; };

    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
        if (warp == 0 && lane == 0) {
            bool ok = true;
            int nk = 0, nv = 0, qn = 0, dn = 0, sn = 0;   // fills so far: K, V, Q ring, dO ring, statistics ring
            auto wait_empty = [&](int bar, int use) {
                if (ok && !mbar_wait(&bars[bar], (use & 1) ^ 1, abort_flag, ST_DKV_PRODUCER)) ok = false;
            };
            auto load_q = [&](const CUtensorMap* m, int kdim, int row0) {
                const int slot = qn % 3;
                wait_empty(K_QEMPTY + slot, qn / 3);
                if (!ok) return;
                mbar_expect_tx(&bars[K_QFULL + slot], (uint32_t)(kTile * kdim * 2));
                tma_tile(sQ + slot * kSlotBytes, m, &bars[K_QFULL + slot], kdim, row0);
                ++qn;
            };
            auto load_do = [&](const CUtensorMap* m, int kdim, int row0) {
                const int slot = dn & 1;
                wait_empty(K_DOEMPTY + slot, dn >> 1);
                if (!ok) return;
                mbar_expect_tx(&bars[K_DOFULL + slot], (uint32_t)(kTile * kdim * 2));
                tma_tile(sDO + slot * kSlotBytes, m, &bars[K_DOFULL + slot], kdim, row0);
                ++dn;
            };
#pragma unroll 1
            for (int it = 0; ok && item_of(it, J, s); ++it) {
                const int T = steps_of(J, s), rowJ = s * p.Lp + J * kTile;
#pragma unroll 1
                for (int t = 0; t < T && ok; ++t) {
                    const int I = J + t, l = level(t);
                    if (t == 0 || l != level(t - 1)) {
                        wait_empty(K_KEMPTY, nk);
                        if (!ok) break;
                        mbar_expect_tx(&bars[K_KFULL], kTile * HD * 2);
                        if (t == 0) tma_tile(sK, &tm.k_raw, &bars[K_KFULL], HD, rowJ);
                        else tma_tile(sK, &tm.kv, &bars[K_KFULL], HD, (int)krow(l, J));
                        ++nk;
                    }
                    if (t == 0) {
                        load_q(&tm.q_raw, HD, rowJ);
                        load_q(&tm.xqn, kTile, rowJ);
                        load_do(&tm.yt, kTile, rowJ);
                        wait_empty(K_VEMPTY, nv);
                        if (!ok) break;
                        mbar_expect_tx(&bars[K_VFULL], kTile * HD * 2);
                        tma_tile(sV, &tm.v, &bars[K_VFULL], HD, rowJ);
                        ++nv;
                        load_do(&tm.d_o, HD, rowJ);
                    } else {
                        load_q(&tm.qv, HD, (int)qrow(l, I));
                        load_do(&tm.d_o, HD, s * p.Lp + I * kTile);
                    }
                    // per-query statistics of the step
                    wait_empty(K_STEMPTY + (sn & 1), sn >> 1);
                    if (!ok) break;
                    mbar_expect_tx(&bars[K_STFULL + (sn & 1)], 2 * kTile * 4);
                    const size_t gi = (size_t)s * p.Lp + I * kTile;
                    bulk_load(rowstat + (sn & 1) * 2 * kTile, p.lse2 + gi, kTile * 4, &bars[K_STFULL + (sn & 1)]);
                    bulk_load(rowstat + (sn & 1) * 2 * kTile + kTile, p.delta + gi, kTile * 4, &bars[K_STFULL + (sn & 1)]);
                    ++sn;
                }
            }
        } else if (warp == 1 && lane == 0) {
            constexpr uint32_t idescT = umma_idesc(128, 128, 0, 0);
            constexpr uint32_t idescD = umma_idesc(128, HD, 0, 1);
            bool ok = true;
            int nk = 0, nv = 0, qb = 0, db = 0, g = 0;   // K / V fills consumed; ring entries and steps before this item
            auto wait = [&](int bar, int parity) {
                if (ok && !mbar_wait(&bars[bar], parity & 1, abort_flag, ST_DKV_MMA)) ok = false;
            };
            auto q_wait = [&](int e) { wait(K_QFULL + e % 3, e / 3); };
            auto do_wait = [&](int e) { wait(K_DOFULL + (e & 1), e >> 1); };
            auto q_addr = [&](int e) { return smem_u32(sQ + (e % 3) * kSlotBytes); };
            auto do_addr = [&](int e) { return smem_u32(sDO + (e & 1) * kSlotBytes); };
#pragma unroll 1
            for (int it = 0; ok && item_of(it, J, s); ++it) {
                const int T = steps_of(J, s);
                // step 0: S^T of the diagonal chunk (two contractions) and its dP^T
                wait(K_KFULL, nk); ++nk;
                q_wait(qb);
                q_wait(qb + 1);
                do_wait(db);
                tc_fence_after_sync();
                if (!ok) break;
                mma_kk(tmem + colS, smem_u32(sK), q_addr(qb), HD, idescT, false);
                mma_kk(tmem + colS, do_addr(db), q_addr(qb + 1), kTile, idescT, true);
                umma_commit(&bars[K_SFULL]);
                umma_commit(&bars[K_QEMPTY + qb % 3]);         // raw q and the two correction operands are only needed here
                umma_commit(&bars[K_QEMPTY + (qb + 1) % 3]);
                umma_commit(&bars[K_DOEMPTY + (db & 1)]);
                umma_commit(&bars[K_KEMPTY]);                  // raw k as well: step 1 uses a key version
                wait(K_VFULL, nv); ++nv;
                do_wait(db + 1);
                tc_fence_after_sync();
                if (!ok) break;
                mma_kk(tmem + colDP, smem_u32(sV), do_addr(db + 1), HD, idescT, false);
                umma_commit(&bars[K_DPFULL]);
                if (T == 1) umma_commit(&bars[K_VEMPTY]);
#pragma unroll 1
                for (int t = 0; t < T && ok; ++t) {
                    const int l = level(t);
                    const int qe = qb + (t == 0 ? 0 : t + 1), de = db + 1 + t;
                    // dV += P^T dO; the first product of an item overwrites the accumulators the previous item's
                    // write-out must have read
                    wait(K_PFULL, g + t);
                    if (t == 0 && it > 0) wait(K_ACCFREE, it - 1);
                    tc_fence_after_sync();
                    if (!ok) break;
                    mma_tn(tmem + colDV, tmem + colS, do_addr(de), idescD, t > 0);
                    umma_commit(&bars[K_DOEMPTY + (de & 1)]);
                    // S^T of the next step overwrites P^T: in-order execution puts it after the product above
                    if (t + 1 < T) {
                        const int l1 = level(t + 1);
                        if (l1 != l) { wait(K_KFULL, nk); ++nk; }
                        q_wait(qb + t + 2);
                        tc_fence_after_sync();
                        if (!ok) break;
                        mma_kk(tmem + colS, smem_u32(sK), q_addr(qb + t + 2), HD, idescT, false);
                        umma_commit(&bars[K_SFULL]);
                        if (t + 2 >= T || level(t + 2) != l1) umma_commit(&bars[K_KEMPTY]);
                    }
                    // dK += dS^T Q
                    wait(K_DSFULL, g + t);
                    tc_fence_after_sync();
                    if (!ok) break;
                    if (t > 0) {
                        mma_tn(tmem + colDK, tmem + colDP, q_addr(qe), idescD, !(t == 1 || l != level(t - 1)));
                        umma_commit(&bars[K_QEMPTY + qe % 3]);
                    }
                    if (t + 1 < T) {
                        do_wait(de + 1);
                        tc_fence_after_sync();
                        if (!ok) break;
                        mma_kk(tmem + colDP, smem_u32(sV), do_addr(de + 1), HD, idescT, false);
                        umma_commit(&bars[K_DPFULL]);
                        if (t + 2 == T) umma_commit(&bars[K_VEMPTY]);   // that was the item's last use of V
                    } else {
                        umma_commit(&bars[K_ACCFULL]);
                    }
                }
                g += T; qb += T + 1; db += T + 1;
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        const int q4 = warp & 3, h = (warp - 4) >> 2, row = q4 * 32 + lane;
        const uint32_t tlane = tmem + ((uint32_t)(q4 * 32) << 16);
        const float sl2 = p.scale * kLog2e;
        const uint64_t sl2x2 = pack2(sl2, sl2);
        uint64_t ngj2 = 0;
        float dsum = 0.f;
        bool ok = true;
        int g = 0;                               // steps before the current item
        constexpr int CW = HD / 2;               // accumulator columns per thread when flushing
        auto flush_dk = [&](int lvl) {   // the version's gradient leaves as bf16, the form the version chain rule multiplies
            store_acc_bf16<CW>(p.dkv + ((size_t)krow(lvl, J) + row) * HD + h * CW, tlane + colDK + h * CW, p.scale);
        };
        auto step = [&](auto first_tag, const int t) {
            constexpr bool FIRST = decltype(first_tag)::value;   // the diagonal chunk: causal mask, dSd written out
            const int gs = g + t;                                // running step number: ring slot and phase
            const float* st_ = rowstat + (gs & 1) * 2 * kTile;   // [0,128): -lse2 (+gate), [128,256): -delta of the queries
            const int c0 = h * 64;               // query columns of this thread
            uint32_t pr[2][32];                  // S^T, then P^T (float bits)
            // ---- part A: P^T = exp2(S^T * scale - lse)
            if (ok && !mbar_wait(&bars[K_STFULL + (gs & 1)], (gs >> 1) & 1, abort_flag, ST_DKV_COMPUTE)) ok = false;
            if (ok && !mbar_wait(&bars[K_SFULL], gs & 1, abort_flag, ST_DKV_COMPUTE)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after_sync();
            if (ok) {
                tmem_ld32(tlane + colS + c0, pr[0]);
                tmem_ld32(tlane + colS + c0 + 32, pr[1]);
                tmem_ld_wait();
                uint32_t pk[32];
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int x = 0; x < 32; x += 4) {
                        const float4 ls = *reinterpret_cast<const float4*>(st_ + c0 + c * 32 + x);
                        uint64_t v01 = fma2(pack2(__uint_as_float(pr[c][x]), __uint_as_float(pr[c][x + 1])), sl2x2, pack2(ls.x, ls.y));
                        uint64_t v23 = fma2(pack2(__uint_as_float(pr[c][x + 2]), __uint_as_float(pr[c][x + 3])), sl2x2, pack2(ls.z, ls.w));
                        if (GATE) { v01 = add2(v01, ngj2); v23 = add2(v23, ngj2); }
                        float e[4];
                        unpack2(v01, e[0], e[1]);
                        unpack2(v23, e[2], e[3]);
#pragma unroll
                        for (int y = 0; y < 4; ++y) {
                            e[y] = ex2(e[y]);
                            if (FIRST && c0 + c * 32 + x + y < row) e[y] = 0.f;
                            pr[c][x + y] = __float_as_uint(e[y]);
                        }
                        pk[c * 16 + (x >> 1)] = pack_bf16(e[0], e[1]);
                        pk[c * 16 + (x >> 1) + 1] = pack_bf16(e[2], e[3]);
                    }
                tmem_st32(tlane + colS + c0, pk);
                tmem_st_wait();
            }
            tc_fence_before_sync();
            mbar_arrive(&bars[K_PFULL]);
            // ---- part B: dS^T = P^T o (dP^T - delta)
            if (ok && !mbar_wait(&bars[K_DPFULL], gs & 1, abort_flag, ST_DKV_COMPUTE)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after_sync();
            // dP^T ready means every product issued before it has retired: dK of a finished level can be flushed
            if (!FIRST && ok && t >= 2 && level(t) != level(t - 1)) flush_dk(level(t - 1));
            uint32_t dsw[FIRST ? 32 : 1];   // this thread's 64 entries of the transposed diagonal tile
            if (ok) {
                const float* dl_ = st_ + kTile;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t dp[32], pk[16];
                    tmem_ld32(tlane + colDP + c0 + c * 32, dp);
                    tmem_ld_wait();
#pragma unroll
                    for (int x = 0; x < 32; x += 4) {
                        const float4 dl = *reinterpret_cast<const float4*>(dl_ + c0 + c * 32 + x);
                        const uint64_t d01 = mul2(pack2(__uint_as_float(pr[c][x]), __uint_as_float(pr[c][x + 1])),
                                                  add2(pack2(__uint_as_float(dp[x]), __uint_as_float(dp[x + 1])), pack2(dl.x, dl.y)));
                        const uint64_t d23 = mul2(pack2(__uint_as_float(pr[c][x + 2]), __uint_as_float(pr[c][x + 3])),
                                                  add2(pack2(__uint_as_float(dp[x + 2]), __uint_as_float(dp[x + 3])), pack2(dl.z, dl.w)));
                        float d[4];
                        unpack2(d01, d[0], d[1]);
                        unpack2(d23, d[2], d[3]);
                        if (GATE) dsum += (d[0] + d[1]) + (d[2] + d[3]);
                        pk[x >> 1] = pack_bf16(d[0], d[1]);
                        pk[(x >> 1) + 1] = pack_bf16(d[2], d[3]);
                        if (FIRST) {   // (scale * dS)^T of the diagonal chunk for the chain rule; unscaled float copy if gated
                            dsw[c * 16 + (x >> 1)] = pack_bf16(d[0] * p.scale, d[1] * p.scale);
                            dsw[c * 16 + (x >> 1) + 1] = pack_bf16(d[2] * p.scale, d[3] * p.scale);
                            if (GATE) {
#pragma unroll
                                for (int y = 0; y < 4; ++y) dp[x + y] = __float_as_uint(d[y]);
                            }
                        }
                    }
                    tmem_st16(tlane + colDP + c0 + c * 16, pk);
                    if (FIRST && GATE) {
                        float* dsd = p.dsd + ((size_t)(s * p.N + J) * kTile) * kTile;
#pragma unroll
                        for (int x = 0; x < 32; ++x) dsd[(size_t)(c0 + c * 32 + x) * kTile + row] = __uint_as_float(dp[x]);
                    }
                }
                tmem_st_wait();
            }
            tc_fence_before_sync();
            mbar_arrive(&bars[K_DSFULL]);
            mbar_arrive(&bars[K_STEMPTY + (gs & 1)]);
            if constexpr (FIRST) {   // rows = keys (this warp's 32 lanes), 64 query columns = 128 bytes per row
                if (ok)
                    warp_store_rows128(p.dsdt + ((size_t)(s * p.N + J) * kTile + q4 * 32) * kTile + h * 64, (size_t)kTile * 2,
                                       dsw);
            }
        };
#pragma unroll 1
        for (int it = 0; item_of(it, J, s); ++it) {
            const int T = steps_of(J, s);
            const int kj = J * kTile + row;          // key position of this thread's row
            if (GATE) {
                const float gj2 = p.G[(size_t)s * p.Lp + kj] * kLog2e;
                ngj2 = pack2(-gj2, -gj2);
                dsum = 0.f;
            }
            step(std::true_type{}, 0);
#pragma unroll 1
            for (int t = 1; t < T; ++t) step(std::false_type{}, t);
            g += T;
            if (ok && !mbar_wait(&bars[K_ACCFULL], it & 1, abort_flag, ST_DKV_COMPUTE)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after_sync();
            if (GATE) {   // the two threads of a key row add their halves of the column sum
                if (h == 1) dsum_x[row] = dsum;
                { __syncwarp(); asm volatile("bar.sync 1, 256;" ::: "memory"); }
                if (h == 0 && ok) p.dG[(size_t)s * p.Lp + kj] = -(dsum + dsum_x[row]);
                { __syncwarp(); asm volatile("bar.sync 1, 256;" ::: "memory"); }
            }
            if (!ok) {
                mbar_arrive(&bars[K_ACCFREE]);
                break;
            }
            auto zero_dk = [&](int slot) {
                uint4* dst = reinterpret_cast<uint4*>(p.dkv + ((size_t)row0(J) + row) * HD + h * CW);
                for (int x = 0; x < CW / 8; ++x) dst[x] = make_uint4(0u, 0u, 0u, 0u);
            };
            if (T > 1) flush_dk(level(T - 1));
            else zero_dk(0);   // no later query chunk met: the boundary-adjusted keys get a zero gradient from the sweep
            // (levels that a sweep shortened by block skipping did not reach stay unwritten: the version chain rule starts
            // at the highest level reached)
            if (CW == 64) {   // 64 bf16 = one 128-byte line per row: coalesced exchange
                uint32_t r0[32], r1[32], w[32];
                tmem_ld32(tlane + colDV + h * CW, r0);
                tmem_ld32(tlane + colDV + h * CW + 32, r1);
                tmem_ld_wait();
                tc_fence_before_sync();
                mbar_arrive(&bars[K_ACCFREE]);   // both accumulators have been read
#pragma unroll
                for (int x = 0; x < 16; ++x) {
                    w[x] = pack_bf16(__uint_as_float(r0[2 * x]), __uint_as_float(r0[2 * x + 1]));
                    w[16 + x] = pack_bf16(__uint_as_float(r1[2 * x]), __uint_as_float(r1[2 * x + 1]));
                }
                const int row0 = J * kTile + q4 * 32;
                warp_store_rows128((__nv_bfloat16*)p.dv + ((size_t)s * p.L + row0) * HD + h * CW, (size_t)HD * 2, w,
                                   p.L - row0);
            } else {
                uint32_t r[32];
                tmem_ld32(tlane + colDV + h * CW, r);
                tmem_ld_wait();
                tc_fence_before_sync();
                mbar_arrive(&bars[K_ACCFREE]);
                if (kj < p.L) {
                    uint4* dst = reinterpret_cast<uint4*>((__nv_bfloat16*)p.dv + ((size_t)s * p.L + kj) * HD + h * CW);
#pragma unroll
                    for (int x = 0; x < 4; ++x)
                        dst[x] = make_uint4(pack_bf16(__uint_as_float(r[8 * x]), __uint_as_float(r[8 * x + 1])),
                                            pack_bf16(__uint_as_float(r[8 * x + 2]), __uint_as_float(r[8 * x + 3])),
                                            pack_bf16(__uint_as_float(r[8 * x + 4]), __uint_as_float(r[8 * x + 5])),
                                            pack_bf16(__uint_as_float(r[8 * x + 6]), __uint_as_float(r[8 * x + 7])));
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
// Persistent like the dK/dV sweep: items are the query chunks of a slice, paired (longest, shortest).
enum { Q_QFULL = 0, Q_QEMPTY, Q_DOFULL, Q_DOEMPTY, Q_KFULL, Q_KEMPTY = Q_KFULL + 3, Q_VFULL = Q_KEMPTY + 3,
       Q_VEMPTY = Q_VFULL + 2, Q_SFULL = Q_VEMPTY + 2, Q_DPFULL = Q_SFULL + 2, Q_DSFULL, Q_ACCFULL, Q_ACCFREE,
       Q_GKFULL, Q_GKEMPTY = Q_GKFULL + 2, Q_COUNT = Q_GKEMPTY + 2 };
constexpr uint32_t kDqGk = 7 * kSlotBytes + 256;              // [2][128] gate prefix of the key chunk, [128] exchange
constexpr uint32_t kDqTotal = kDqGk + 3 * kTile * 4;

template <int HD, bool GATE>
__global__ void __launch_bounds__(384, 1) dq_kernel(const __grid_constant__ BwdTensorMaps tm, const BwdParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    if ((uint32_t)(smem - smem_raw) + kDqTotal > kSmemAlloc) {   // uniform over the CTA
        if (threadIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)ST_DQ_PRODUCER);
        return;
    }
    uint8_t* sQ = smem;
    uint8_t* sDO = sQ + kSlotBytes;
    uint8_t* sK = sDO + kSlotBytes;        // ring of 3
    uint8_t* sV = sK + 3 * kSlotBytes;     // ring of 2
    uint64_t* bars = (uint64_t*)(smem + 7 * kSlotBytes);
    uint32_t* tmem_slot = (uint32_t*)(bars + Q_COUNT);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    float* gk = (float*)(smem + kDqGk);
    float* dsum_x = gk + 2 * kTile;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int items = p.N * p.S;

    if (threadIdx.x == 0) {
        for (int i = 0; i < Q_COUNT; ++i)
            mbar_init(&bars[i], (i == Q_DSFULL || i == Q_ACCFREE || i == Q_GKEMPTY || i == Q_GKEMPTY + 1) ? 256u : 1u);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 2 && lane < 8) tma_prefetch_desc(reinterpret_cast<const CUtensorMap*>(&tm) + lane);
    if (warp == 1) tmem_alloc(tmem_slot, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    constexpr uint32_t colS = 0, colDP = 256, colDQ = 384;   // two S tiles at 0 and 128
    // k-th work item of this CTA; query chunk I has I steps (t = 0..I-1, key chunk J = I-1-t)
    auto item_of = [&](int k, int& I, int& s) {
        const int w = 2 * ((int)blockIdx.x + (k >> 1) * (int)gridDim.x) + (k & 1);
        if (w >= items) return false;
        s = w / p.N;
        const int j = w % p.N;
        I = (j & 1) ? (j >> 1) : p.N - 1 - (j >> 1);
        return true;
    };
    int I = 0, s = 0;
    auto qrow = [&](int lvl, int chunk) { return qver_row(p.vl, s, lvl, chunk); };   // first row of a version tile
    auto krow = [&](int lvl, int chunk) { return kver_row(p.vl, s, lvl, chunk); };
    auto row0 = [&](int chunk) { return (long)s * p.Lp + (long)chunk * kTile; };      // plane 0
    auto level = [&](int t) { return msb32((unsigned)(I ^ (I - 1 - t))); };
    // earlier key chunks this query chunk visits (J = I-1 .. I-T): all of them, or fewer when the gate has made the far
    // ones negligible (every warp role reads the same precomputed number; the diagonal chunk is not part of this sweep)
    auto steps_of = [&](int I, int s) { return p.nkeep ? min(I, p.nkeep[s * p.N + I] - 1) : I; };

    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
        if (warp == 0 && lane == 0) {
            bool ok = true;
            int nq = 0, nd = 0, kn = 0, vn = 0;   // fills so far: Q, dO, K ring, V ring (= gate ring)
            auto wait_empty = [&](int bar, int use) {
                if (ok && !mbar_wait(&bars[bar], (use & 1) ^ 1, abort_flag, ST_DQ_PRODUCER)) ok = false;
            };
#pragma unroll 1
            for (int it = 0; ok && item_of(it, I, s); ++it) {
                const int T = steps_of(I, s);
                if (T == 0) continue;
                wait_empty(Q_DOEMPTY, nd);
                if (!ok) break;
                mbar_expect_tx(&bars[Q_DOFULL], kTile * HD * 2);
                tma_tile(sDO, &tm.d_o, &bars[Q_DOFULL], HD, s * p.Lp + I * kTile);
                ++nd;
#pragma unroll 1
                for (int t = 0; t < T && ok; ++t) {
                    const int J = I - 1 - t, l = level(t);
                    if (t == 0 || l != level(t - 1)) {
                        wait_empty(Q_QEMPTY, nq);
                        if (!ok) break;
                        mbar_expect_tx(&bars[Q_QFULL], kTile * HD * 2);
                        tma_tile(sQ, &tm.qv, &bars[Q_QFULL], HD, (int)qrow(l, I));
                        ++nq;
                    }
                    wait_empty(Q_KEMPTY + kn % 3, kn / 3);
                    if (!ok) break;
                    mbar_expect_tx(&bars[Q_KFULL + kn % 3], kTile * HD * 2);
                    tma_tile(sK + (kn % 3) * kSlotBytes, &tm.kv, &bars[Q_KFULL + kn % 3], HD, (int)krow(l, J));
                    ++kn;
                    wait_empty(Q_VEMPTY + (vn & 1), vn >> 1);
                    if (!ok) break;
                    mbar_expect_tx(&bars[Q_VFULL + (vn & 1)], kTile * HD * 2);
                    tma_tile(sV + (vn & 1) * kSlotBytes, &tm.v, &bars[Q_VFULL + (vn & 1)], HD, s * p.Lp + J * kTile);
                    if (GATE) {   // gate prefix of the key chunk
                        wait_empty(Q_GKEMPTY + (vn & 1), vn >> 1);
                        if (!ok) break;
                        mbar_expect_tx(&bars[Q_GKFULL + (vn & 1)], kTile * 4);
                        bulk_load(gk + (vn & 1) * kTile, p.G + (size_t)s * p.Lp + J * kTile, kTile * 4,
                                  &bars[Q_GKFULL + (vn & 1)]);
                    }
                    ++vn;
                }
            }
        } else if (warp == 1 && lane == 0) {
            constexpr uint32_t idescS = umma_idesc(128, 128, 0, 0);
            constexpr uint32_t idescD = umma_idesc(128, HD, 0, 1);
            bool ok = true;
            int nq = 0, nd = 0, g = 0, na = 0;   // Q / dO fills consumed, steps before this item, items with steps so far
            int T = 0;
            auto wait = [&](int bar, int parity) {
                if (ok && !mbar_wait(&bars[bar], parity & 1, abort_flag, ST_DQ_MMA)) ok = false;
            };
            auto issue_s = [&](int t) {      // S(t) into the tile of running step g + t
                const int gs = g + t;
                if (t == 0 || level(t) != level(t - 1)) { wait(Q_QFULL, nq); ++nq; }
                wait(Q_KFULL + gs % 3, gs / 3);
                tc_fence_after_sync();
                if (!ok) return;
                mma_kk(tmem + colS + (gs & 1) * 128, smem_u32(sQ), smem_u32(sK + (gs % 3) * kSlotBytes), HD, idescS, false);
                umma_commit(&bars[Q_SFULL + (gs & 1)]);
                if (t + 1 >= T || level(t + 1) != level(t)) umma_commit(&bars[Q_QEMPTY]);
            };
            auto issue_dp = [&](int t) {
                const int gs = g + t;
                wait(Q_VFULL + (gs & 1), gs >> 1);
                tc_fence_after_sync();
                if (!ok) return;
                mma_kk(tmem + colDP, smem_u32(sDO), smem_u32(sV + (gs & 1) * kSlotBytes), HD, idescS, false);
                umma_commit(&bars[Q_DPFULL]);
                umma_commit(&bars[Q_VEMPTY + (gs & 1)]);
                if (t + 1 >= T) umma_commit(&bars[Q_DOEMPTY]);   // the item's last use of dO
            };
#pragma unroll 1
            for (int it = 0; ok && item_of(it, I, s); ++it) {
                T = steps_of(I, s);
                if (T == 0) continue;
                wait(Q_DOFULL, nd); ++nd;
                issue_s(0);
                issue_dp(0);
                if (T > 1) issue_s(1);
#pragma unroll 1
                for (int t = 0; t < T && ok; ++t) {
                    const int gs = g + t;
                    // dQ += dS K.  dP of the next step overwrites dS, S(t+2) the tile whose P every thread has taken
                    // into registers before it delivered dS: in-order execution keeps both behind what they replace.
                    wait(Q_DSFULL, gs);
                    if (t == 0 && na > 0) wait(Q_ACCFREE, na - 1);   // the previous item's dQ has been read
                    tc_fence_after_sync();
                    if (!ok) break;
                    mma_tn(tmem + colDQ, tmem + colDP, smem_u32(sK + (gs % 3) * kSlotBytes), idescD,
                           !(t == 0 || level(t) != level(t - 1)));
                    umma_commit(&bars[Q_KEMPTY + gs % 3]);
                    if (t + 1 < T) issue_dp(t + 1);
                    if (t + 2 < T) issue_s(t + 2);
                    if (t == T - 1) umma_commit(&bars[Q_ACCFULL]);
                }
                g += T;
                ++na;
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        const int q4 = warp & 3, h = (warp - 4) >> 2, row = q4 * 32 + lane;
        const uint32_t tlane = tmem + ((uint32_t)(q4 * 32) << 16);
        const float sl2 = p.scale * kLog2e;
        const uint64_t sl2x2 = pack2(sl2, sl2), nlog2 = pack2(-kLog2e, -kLog2e);
        bool ok = true;
        int g = 0, na = 0;
        constexpr int CW = HD / 2;
        auto flush_dq = [&](int lvl) {
            store_acc_bf16<CW>(p.dqv + ((size_t)qrow(lvl, I) + row) * HD + h * CW, tlane + colDQ + h * CW, p.scale);
        };
#pragma unroll 1
        for (int it = 0; item_of(it, I, s); ++it) {
            const int T = steps_of(I, s);
            auto zero_dq = [&](int slot) {   // a whole [128 x HD] version gradient tile, by the 256 math threads
                uint4* dst = reinterpret_cast<uint4*>(p.dqv + (size_t)row0(I) * HD);
                for (int i = threadIdx.x - 128; i < kTile * HD / 8; i += 256) dst[i] = make_uint4(0u, 0u, 0u, 0u);
            };
            // no key chunk visited (chunk 0, or block skipping left only the diagonal): the boundary-adjusted queries get a
            // zero gradient from the sweep.  Levels that a shortened sweep does not reach stay unwritten: the version
            // chain rule starts at the highest level reached.
            if (T == 0) {
                zero_dq(0);
                continue;
            }
            const size_t qi = (size_t)s * p.Lp + I * kTile + row;
            const float ndelta = p.delta[qi];            // minus delta
            const float nl = p.lse2[qi];                 // minus lse2, plus the gate prefix of the row when gated
            const uint64_t nl2 = pack2(nl, nl), nd2 = pack2(ndelta, ndelta);
            float dsum = 0.f;
#pragma unroll 1
            for (int t = 0; t < T; ++t) {
                const int gs = g + t;
                const int c0 = h * 64;               // key columns of this thread
                uint32_t pr[2][32];                  // S, then P (float bits)
                // ---- part A: P = exp2(S * scale - lse)
                if (GATE && ok && !mbar_wait(&bars[Q_GKFULL + (gs & 1)], (gs >> 1) & 1, abort_flag, ST_DQ_COMPUTE)) ok = false;
                if (ok && !mbar_wait(&bars[Q_SFULL + (gs & 1)], (gs >> 1) & 1, abort_flag, ST_DQ_COMPUTE)) ok = false;
                ok = __all_sync(0xffffffffu, ok);
                tc_fence_after_sync();
                if (ok) {
                    tmem_ld32(tlane + colS + (gs & 1) * 128 + c0, pr[0]);
                    tmem_ld32(tlane + colS + (gs & 1) * 128 + c0 + 32, pr[1]);
                    tmem_ld_wait();
                    const float* g_ = gk + (gs & 1) * kTile + c0;
#pragma unroll
                    for (int c = 0; c < 2; ++c)
#pragma unroll
                        for (int x = 0; x < 32; x += 4) {
                            uint64_t v01 = fma2(pack2(__uint_as_float(pr[c][x]), __uint_as_float(pr[c][x + 1])), sl2x2, nl2);
                            uint64_t v23 = fma2(pack2(__uint_as_float(pr[c][x + 2]), __uint_as_float(pr[c][x + 3])), sl2x2, nl2);
                            if (GATE) {
                                const float4 g4 = *reinterpret_cast<const float4*>(g_ + c * 32 + x);
                                v01 = fma2(pack2(g4.x, g4.y), nlog2, v01);
                                v23 = fma2(pack2(g4.z, g4.w), nlog2, v23);
                            }
                            float e[4];
                            unpack2(v01, e[0], e[1]);
                            unpack2(v23, e[2], e[3]);
#pragma unroll
                            for (int y = 0; y < 4; ++y) pr[c][x + y] = __float_as_uint(ex2(e[y]));
                        }
                }
                // ---- part B: dS = P o (dP - delta)
                if (ok && !mbar_wait(&bars[Q_DPFULL], gs & 1, abort_flag, ST_DQ_COMPUTE)) ok = false;
                ok = __all_sync(0xffffffffu, ok);
                tc_fence_after_sync();
                // dP ready means every product issued before it has retired: dQ of a finished level can be flushed
                if (ok && t >= 1 && level(t) != level(t - 1)) flush_dq(level(t - 1));
                if (ok) {
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t dp[32], pk[16];
                        tmem_ld32(tlane + colDP + c0 + c * 32, dp);
                        tmem_ld_wait();
#pragma unroll
                        for (int x = 0; x < 32; x += 2) {
                            const uint64_t d01 = mul2(pack2(__uint_as_float(pr[c][x]), __uint_as_float(pr[c][x + 1])),
                                                      add2(pack2(__uint_as_float(dp[x]), __uint_as_float(dp[x + 1])), nd2));
                            float d0, d1;
                            unpack2(d01, d0, d1);
                            if (GATE) dsum += d0 + d1;
                            pk[x >> 1] = pack_bf16(d0, d1);
                        }
                        tmem_st16(tlane + colDP + c0 + c * 16, pk);
                    }
                    tmem_st_wait();
                }
                tc_fence_before_sync();
                mbar_arrive(&bars[Q_DSFULL]);
                if (GATE) mbar_arrive(&bars[Q_GKEMPTY + (gs & 1)]);
            }
            g += T;
            if (ok && !mbar_wait(&bars[Q_ACCFULL], na & 1, abort_flag, ST_DQ_COMPUTE)) ok = false;
            ++na;
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after_sync();
            if (GATE) {
                if (h == 1) dsum_x[row] = dsum;
                { __syncwarp(); asm volatile("bar.sync 1, 256;" ::: "memory"); }
                if (h == 0 && ok) p.dGrow[qi] = dsum + dsum_x[row];
                { __syncwarp(); asm volatile("bar.sync 1, 256;" ::: "memory"); }
            }
            if (ok) flush_dq(level(T - 1));
            tc_fence_before_sync();
            mbar_arrive(&bars[Q_ACCFREE]);
            if (!ok) break;
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

// Per-row constants of the backward sweeps, stored negated so that they enter as addends:
//   delta[i] = -(dO_i . O_i),   lse2[i] = (G_i - lse_i) * log2(e)   (G: gate prefix, absent = 0),
// padded to Lp (tail rows: delta 0, lse2 -1e30 so that their probabilities vanish).  One warp per row.
template <int HD>
__global__ void rowstats_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                                const float* __restrict__ lse, const float* __restrict__ G, float* __restrict__ delta,
                                float* __restrict__ lse2, int L, int Lp) {
    constexpr int TPR = HD / 8;                 // threads per row: 16 bytes (8 values) of o and of dO each
    const int s = blockIdx.y;
    const int i = blockIdx.x * (256 / TPR) + threadIdx.x / TPR;
    const int sub = threadIdx.x % TPR;
    float acc = 0.f;
    if (i < L) {
        const size_t base = ((size_t)s * L + i) * HD + sub * 8;
        const uint4 a = *reinterpret_cast<const uint4*>(o + base), b = *reinterpret_cast<const uint4*>(d_o + base);
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&aw[x]));
            const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[x]));
            acc += fa.x * fb.x + fa.y * fb.y;
        }
    }
#pragma unroll
    for (int off = TPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (sub == 0 && i < Lp) {
        delta[(size_t)s * Lp + i] = -acc;
        // rows of the zero-padded tail get a huge negative value: their probabilities must come out as exact zeros.  (A
        // plain 0 would do without a gate; with one, exp2(0 - G_j log2 e) of a strongly decayed key overflows and the
        // product with the row's zero dP - delta is a NaN.)
        float v = -1e30f;
        if (i < L) v = ((G ? G[(size_t)s * Lp + i] : 0.f) - lse[(size_t)s * L + i]) * kLog2e;
        lse2[(size_t)s * Lp + i] = v;
    }
}

template <class K>
cudaError_t set_smem(K kern, int bytes) {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

constexpr int kDkvSmem = kSmemAlloc;
constexpr int kDqSmem = kSmemAlloc;

template <int HD, bool GATE>
cudaError_t launch_one(const BwdTensorMaps& tm, const BwdParams& p, int which, cudaStream_t st) {
    if (which == 0) {
        cudaError_t e = set_smem(dkv_kernel<HD, GATE>, kDkvSmem);
        if (e != cudaSuccess) return e;
        int dev = 0, sms = 0;
        e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        const int pairs = (p.N * p.S + 1) / 2;
        dkv_kernel<HD, GATE><<<dim3(pairs < sms ? pairs : sms), 384, kDkvSmem, st>>>(tm, p);
    } else {
        cudaError_t e = set_smem(dq_kernel<HD, GATE>, kDqSmem);
        if (e != cudaSuccess) return e;
        int dev = 0, sms = 0;
        e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        const int pairs = (p.N * p.S + 1) / 2;
        dq_kernel<HD, GATE><<<dim3(pairs < sms ? pairs : sms), 384, kDqSmem, st>>>(tm, p);
    }
    return cudaGetLastError();
}

}  // namespace

// which = 0: dK/dV sweep, which = 1: dQ sweep.
cudaError_t launch_fa_bwd(const BwdTensorMaps& tm, const BwdParams& p, int hd, int which, cudaStream_t st) {
    if (hd == 64) return p.G ? launch_one<64, true>(tm, p, which, st) : launch_one<64, false>(tm, p, which, st);
    return p.G ? launch_one<128, true>(tm, p, which, st) : launch_one<128, false>(tm, p, which, st);
}

cudaError_t launch_rowstats(const void* o, const void* d_o, const float* lse, const float* G, float* delta, float* lse2,
                            int S, int L, int Lp, int hd, cudaStream_t st) {
    const int rows_per_cta = 256 / (hd / 8);
    dim3 grid((Lp + rows_per_cta - 1) / rows_per_cta, S);
    if (hd == 64)
        rowstats_kernel<64><<<grid, 256, 0, st>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)d_o, lse, G, delta, lse2, L, Lp);
    else
        rowstats_kernel<128><<<grid, 256, 0, st>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)d_o, lse, G, delta, lse2, L, Lp);
    return cudaGetLastError();
}

}  // namespace path
