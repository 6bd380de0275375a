// Fused forward sweep of PaTH attention (paper Sec. 3.3, the FlashAttention-style loop).
//
// A work item is one 128-row query chunk I of one (batch, head) slice; it walks the key chunks
// J = I, I-1, ..., 0.  The diagonal chunk uses the raw q, k plus the in-chunk Householder
// correction as a second contraction (Sec. 3.3, case i = j):
//     S = Q K^T + (-lower(Q W^T)) (T^-1 strictLower(W K^T))           [operands q_raw,k_raw,xqn,yt]
// Every earlier chunk J < I is an ordinary tile product of a query version and a key
// version that meet at the dyadic boundary of (I, J):  S = Qv[l][I] Kv[l][J]^T, l = msb(I xor J).
// The versions are prepared beforehand, so this loop contains no query update.
//
// The kernel is persistent: the work items are listed slice after slice, each slice as pairs (longest, shortest),
// (second longest, second shortest), ..., and CTA c takes the pairs c, c + gridDim.x, ...  Every pair has the same
// number of key chunks, CTAs that run together work on a few slices whose keys and values stay in L2, and the
// loads and the first logit tile of the next item are produced while the current item's result is written out.
//
// The key chunks are dealt alternately to two streams (n = I - J even / odd).  Each stream has its own
// softmax warpgroup (one query row per thread, the whole 128-wide logit row held in registers), its own S tile
// and O accumulator in tensor memory and its own running (max, sum); the two partial results are merged at
// the end like a split-KV attention.  While one warpgroup does its exponentials the tensor pipe works for the
// other stream.  P never touches shared memory: it overwrites the first half of its S tile as packed bf16 and
// enters O += P V as the tensor-memory A operand.
//
// Warps: 0 = TMA producer, 1 = tcgen05 MMA issuer, 2-3 idle (they give their registers to the softmax
// warps), 4-7 = softmax of stream 0, 8-11 = softmax of stream 1.
#include <type_traits>
#include "common.cuh"
#include "tc5.cuh"

namespace path {
using namespace tc5;

constexpr int kTile = 128;
constexpr uint32_t kSlotBytes = 32768;  // one [128 x 128] bf16 operand tile (two 64-column panels)
constexpr uint32_t kPanelBytes = 16384; // one [128 x 64] bf16 panel

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
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

// D[tmem] (+)= A[tmem, packed bf16, 8 columns per 16 elements of the contraction] * B[smem]
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

struct FwdSmem {
    static constexpr uint32_t offQ = 0;                       // 3 slots: ring of query operands
    static constexpr uint32_t offK = offQ + 3 * kSlotBytes;   // 2 slots: one per stream
    static constexpr uint32_t offV = offK + 2 * kSlotBytes;   // 2 slots: one per stream
    static constexpr uint32_t offBar = offV + 2 * kSlotBytes;
    // [2 streams][128] pairs: .x = gate prefix of the stream's current key chunk during the sweep; at the end of
    // a work item the pair is the stream's (running max, running sum)
    static constexpr uint32_t offStat = offBar + 256;
    static constexpr uint32_t total = offStat + 2 * kTile * 8;
    static constexpr uint32_t alloc = 232448;                 // everything an SM offers one CTA
    static_assert(total + 512 <= alloc, "no room left to align the base");
};

enum { B_QFULL = 0, B_QEMPTY = 3, B_KFULL = 6, B_KEMPTY = 8, B_VFULL = 10, B_VEMPTY = 12,
       B_SFULL = 14, B_PFULL = 16, B_OFULL = 18, B_OFREE = 20, B_COUNT = 21 };

// CROSS = true is the segment-against-segment variant used by the context-parallel path (paper Sec. 3.5): a work item is a
// query chunk of one segment, it visits EVERY key chunk of another (earlier) segment, there is no diagonal chunk and no
// causal mask, queries and keys come as one prepared tile each (tm.qv / tm.kv, no levels), the key-side gate terms are
// their own array (whose padded tail holds a huge value, which masks the padded keys), and the result is written
// normalised in float32 together with its LSE so that the caller can merge it into a running state.
template <int HD, bool GATE, bool CROSS = false>
__global__ void __launch_bounds__(384, 1)
fa_fwd_kernel(const __grid_constant__ FwdTensorMaps tm, const FwdParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    if ((uint32_t)(smem - smem_raw) + FwdSmem::total > FwdSmem::alloc) {   // uniform over the CTA
        if (threadIdx.x == 0) atomicCAS(p.status, 0u, (uint32_t)ST_FWD_PRODUCER);
        return;
    }
    uint8_t* sQ = smem + FwdSmem::offQ;
    uint8_t* sK = smem + FwdSmem::offK;
    uint8_t* sV = smem + FwdSmem::offV;
    uint64_t* bars = (uint64_t*)(smem + FwdSmem::offBar);
    uint32_t* tmem_slot = (uint32_t*)(bars + B_COUNT);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    float2* stat = (float2*)(smem + FwdSmem::offStat);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int items = p.N * p.S;

    if (threadIdx.x == 0) {
        for (int i = 0; i < B_COUNT; ++i)
            mbar_init(&bars[i], (i == B_PFULL || i == B_PFULL + 1) ? 128u : (i == B_OFREE ? 256u : 1u));
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 2 && lane < 7) {
        tma_prefetch_desc(reinterpret_cast<const CUtensorMap*>(&tm) + lane);   // the seven maps are contiguous
    }
    if (warp == 1) tmem_alloc(tmem_slot, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    // tensor memory columns: S of stream x at x*128 (P aliases its first 64 columns), O of stream x at 256 + x*128
    // k-th work item of this CTA: pairs (long, short) of one slice, slice after slice (keeps a slice's keys in L2)
    auto item_of = [&](int k, int& I, int& s) {
        const int w = 2 * ((int)blockIdx.x + (k >> 1) * (int)gridDim.x) + (k & 1);
        if (w >= items) return false;
        s = w / p.N;
        const int j = w % p.N;
        I = (j & 1) ? (j >> 1) : p.N - 1 - (j >> 1);
        return true;
    };
    // key chunks a work item visits, counted from the diagonal: all I + 1 of them, or fewer when the gate has made the
    // far ones negligible (every warp role reads the same precomputed number)
    auto steps_of = [&](int I, int s) {
        if (CROSS) return p.Nk;
        return p.nkeep ? min(I + 1, p.nkeep[s * p.N + I]) : I + 1;
    };


    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
        if (warp == 0 && lane == 0) {
            // ------------------------------------------------------------ TMA producer
            bool ok = true;
            int nq = 0;                       // query operands issued so far (all work items)
            uint32_t kf = 0, vf = 0;          // bit x: parity of the number of fills of K / V slot x so far
            auto wait_empty = [&](int bar, int use) {
                if (ok && !mbar_wait(&bars[bar], (use & 1) ^ 1, abort_flag, ST_FWD_PRODUCER)) ok = false;
            };
            auto load_q = [&](const CUtensorMap* m, int kdim, int row0) {
                const int slot = nq % 3;
                wait_empty(B_QEMPTY + slot, nq / 3);
                if (!ok) return;
                mbar_expect_tx(&bars[B_QFULL + slot], (uint32_t)(kTile * kdim * 2));
                for (int h = 0; h < kdim / 64; ++h)
                    tma_load_2d(sQ + slot * kSlotBytes + h * kPanelBytes, m, &bars[B_QFULL + slot], h * 64, row0);
                ++nq;
            };
            auto load_kv = [&](uint8_t* base, int bfull, int bempty, int slot, uint32_t& fills, const CUtensorMap* m,
                               int kdim, int row0) {
                wait_empty(bempty + slot, (int)((fills >> slot) & 1u));
                if (!ok) return;
                mbar_expect_tx(&bars[bfull + slot], (uint32_t)(kTile * kdim * 2));
                for (int h = 0; h < kdim / 64; ++h)
                    tma_load_2d(base + slot * kSlotBytes + h * kPanelBytes, m, &bars[bfull + slot], h * 64, row0);
                fills ^= 1u << slot;
            };
            int I, s;
            for (int it = 0; ok && item_of(it, I, s); ++it) {
                const int NS = steps_of(I, s);
                const int rowRaw = s * p.Lp + I * kTile;
                if (CROSS) {   // one query tile, then every key chunk of the other segment, last chunk first
                    load_q(&tm.qv, HD, rowRaw);
                    for (int n = 0; n < NS && ok; ++n) {
                        const int x = n & 1, rowK = s * p.Lkp + (NS - 1 - n) * kTile;
                        load_kv(sK, B_KFULL, B_KEMPTY, x, kf, &tm.kv, HD, rowK);
                        load_kv(sV, B_VFULL, B_VEMPTY, x, vf, &tm.v, HD, rowK);
                    }
                    continue;
                }
                // diagonal chunk: raw q, k and the correction operands (both K slots), V of chunk I
                load_q(&tm.q_raw, HD, rowRaw);
                load_kv(sK, B_KFULL, B_KEMPTY, 0, kf, &tm.k_raw, HD, rowRaw);
                load_q(&tm.xqn, kTile, rowRaw);
                load_kv(sV, B_VFULL, B_VEMPTY, 1, vf, &tm.yt, kTile, rowRaw);   // Yt borrows stream 1's V slot
                load_kv(sV, B_VFULL, B_VEMPTY, 0, vf, &tm.v, HD, rowRaw);
                int cur = -1;
                for (int n = 1; n < NS && ok; ++n) {
                    const int J = I - n, x = n & 1, l = msb32((unsigned)(I ^ J));   // l is non-decreasing in n
                    if (l != cur) {
                        load_q(&tm.qv, HD, (int)qver_row(p.vl, s, l, I));
                        cur = l;
                    }
                    load_kv(sK, B_KFULL, B_KEMPTY, x, kf, &tm.kv, HD, (int)kver_row(p.vl, s, l, J));
                    load_kv(sV, B_VFULL, B_VEMPTY, x, vf, &tm.v, HD, s * p.Lp + J * kTile);
                }
            }
        } else if (warp == 1 && lane == 0) {
            // ------------------------------------------------------------ MMA issuer
            // a negative scale is applied as a sign flip of the logits here (negate-A bit), its magnitude in the softmax
            const uint32_t idescS = umma_idesc(128, 128, 0, 0) | (p.scale < 0.f ? (1u << 13) : 0u);
            constexpr uint32_t idescO = umma_idesc(128, HD, 0, 1);
            bool ok = true;
            auto wait = [&](int bar, int parity) {
                if (ok && !mbar_wait(&bars[bar], parity & 1, abort_flag, ST_FWD_MMA)) ok = false;
            };
            auto issue_s = [&](int x, int qs, int ks, int kdim, bool acc) {   // ks >= 2: a V slot
                // (descriptors advance by their low word only: 32 bytes per step, the next panel after four steps)
                uint32_t a_lo = umma_desc_lo(smem_u32(sQ + qs * kSlotBytes), 16), b_lo = umma_desc_lo(smem_u32(sK + ks * kSlotBytes), 16);
                for (int kk = 0; kk < kdim / 16; ++kk) {
                    umma_ss(tmem + x * 128, umma_desc_join(a_lo), umma_desc_join(b_lo), idescS, (acc || kk > 0) ? 1u : 0u);
                    const uint32_t step = (kk & 3) == 3 ? (kPanelBytes - 96u) >> 4 : 2u;
                    a_lo += step;
                    b_lo += step;
                }
            };
            int qi_next = 0;                   // query operands waited for so far (all work items)
            int released = 0;                  // query operands [0, released) have been handed back to the producer
            uint32_t kc = 0, vc = 0, pc = 0;   // bit x: parity of the K / V fills and P tiles of stream x consumed so far
            int item = 0;
            auto take_q = [&]() {
                const int qi = qi_next++;
                wait(B_QFULL + qi % 3, qi / 3);
                return qi;
            };
            auto take_k = [&](int x) { wait(B_KFULL + x, (int)((kc >> x) & 1u)); kc ^= 1u << x; };
            auto release_q = [&](int upto) {
                for (; released < upto; ++released) umma_commit(&bars[B_QEMPTY + released % 3]);
            };
            int I, s_it;
            for (; ok && item_of(item, I, s_it); ++item) {
                const int NS = steps_of(I, s_it);
                int cur_level = -1;
                int q_of0, q_of1;              // operand index used by each stream's most recent S product
                auto advance_q = [&](int n) {  // operand index of step n >= 1 (waits for a newly needed one)
                    const int l = CROSS ? 0 : msb32((unsigned)(I ^ (I - n)));
                    if (l != cur_level) {
                        cur_level = l;
                        take_q();
                    }
                    return qi_next - 1;
                };
                if (CROSS) {   // S of step 0 (stream 0): an ordinary tile product; the one query operand serves every step
                    cur_level = 0;
                    const int q0 = take_q();
                    take_k(0);
                    tc_fence_after_sync();
                    if (!ok) break;
                    issue_s(0, q0 % 3, 0, HD, false);
                    umma_commit(&bars[B_SFULL + 0]);
                    umma_commit(&bars[B_KEMPTY + 0]);
                    q_of0 = q_of1 = q0;
                } else {
                // S of step 0 (diagonal, stream 0): two contractions
                const int q0 = take_q();
                take_k(0);
                tc_fence_after_sync();
                if (ok) issue_s(0, q0 % 3, 0, HD, false);
                const int q1 = take_q();
                wait(B_VFULL + 1, (int)((vc >> 1) & 1u)); vc ^= 2u;
                tc_fence_after_sync();
                if (!ok) break;
                issue_s(0, q1 % 3, 3, kTile, true);
                umma_commit(&bars[B_SFULL + 0]);
                umma_commit(&bars[B_KEMPTY + 0]);
                umma_commit(&bars[B_VEMPTY + 1]);
                release_q(q1 + 1);             // rawQ and Xqn go back once the diagonal products retire
                q_of0 = q_of1 = q1 + 1;
                }
                // S of step 1 (stream 1)
                if (NS > 1) {
                    q_of1 = advance_q(1);
                    take_k(1);
                    tc_fence_after_sync();
                    if (!ok) break;
                    issue_s(1, q_of1 % 3, 1, HD, false);
                    umma_commit(&bars[B_SFULL + 1]);
                    umma_commit(&bars[B_KEMPTY + 1]);
                }
                if (NS <= 2) release_q(qi_next);
                for (int n = 0; n < NS && ok; ++n) {
                    const int x = n & 1, t = n >> 1;
                    // O_x += P_x V_n; the first product of a work item overwrites O_x, which the previous item's
                    // epilogue must have read
                    wait(B_PFULL + x, (int)((pc >> x) & 1u)); pc ^= 1u << x;
                    wait(B_VFULL + x, (int)((vc >> x) & 1u)); vc ^= 1u << x;
                    if (t == 0 && item > 0) wait(B_OFREE, item - 1);
                    tc_fence_after_sync();
                    if (!ok) break;
                    {
                        uint32_t b_lo = umma_desc_lo(smem_u32(sV + x * kSlotBytes), kPanelBytes);
#pragma unroll
                        for (int kk = 0; kk < kTile / 16; ++kk) {
                            umma_ts(tmem + 256 + x * 128, tmem + x * 128 + kk * 8, umma_desc_join(b_lo), idescO,
                                    (t > 0 || kk > 0) ? 1u : 0u);
                            b_lo += 128u;
                        }
                        umma_commit(&bars[B_VEMPTY + x]);
                    }
                    // the stream's next S overwrites P; products issued by one thread execute in order, so it lands
                    // after the P V above has read P
                    if (n + 2 < NS) {
                        const int qi = advance_q(n + 2);
                        if (x) q_of1 = qi; else q_of0 = qi;
                        take_k(x);
                        tc_fence_after_sync();
                        if (!ok) break;
                        issue_s(x, qi % 3, x, HD, false);
                        umma_commit(&bars[B_SFULL + x]);
                        umma_commit(&bars[B_KEMPTY + x]);
                        // operands older than what either stream used last can go back to the producer
                        release_q(n + 3 == NS ? qi_next : min(qi, x ? q_of0 : q_of1));
                    } else {
                        umma_commit(&bars[B_OFULL + x]);
                    }
                }
                release_q(qi_next);
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // ------------------------------------------------------------ softmax warpgroups, one row per thread
        const int x = (warp - 4) >> 2;          // stream
        const int q4 = warp & 3;                // TMEM lane quadrant this warp may touch
        const int row = q4 * 32 + lane;
        const uint32_t tlane = tmem + ((uint32_t)(q4 * 32) << 16);
        const uint32_t colS = x * 128, colO = 256 + x * 128;
        const float kLog2e = 1.4426950408889634f;
        const float sl2 = fabsf(p.scale) * kLog2e;
        const uint64_t sl2x2 = pack2(sl2, sl2);
        bool ok = true;
        int sc = 0;                             // S tiles consumed so far by this stream (all work items)
        int o1 = 0;                             // work items so far in which stream 1 had steps
        int item = 0;
        float2* statx = stat + x * kTile;
        auto wg_sync = [&]() {
            __syncwarp();   // bar.sync is warp-aligned: reconverge first
            if (x == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
            else asm volatile("bar.sync 2, 128;" ::: "memory");
        };

        int I, s;
        for (; item_of(item, I, s); ++item) {
            const int NS = steps_of(I, s);
            const int qi = I * kTile + row;     // position within the slice (may be >= L in the ragged tail)
            const int TX = (NS - x + 1) >> 1;   // steps of this stream: n = 2t + x
            float gi2 = 0.f;
            if (GATE) gi2 = p.G[(size_t)s * p.Lp + qi] * kLog2e;
            float m = -INFINITY, l = 0.f;
            // the stat words are shared with the previous item's merge: every thread must have read them
            if (item > 0 && ok && !mbar_wait(&bars[B_OFREE], (item - 1) & 1, abort_flag, ST_FWD_SOFTMAX)) ok = false;

            auto softmax_step = [&](auto diag_tag, const int t) {
                constexpr bool DIAG = decltype(diag_tag)::value;   // the diagonal chunk (step 0): causal mask
                constexpr bool PRE = DIAG || GATE;                 // logits are scaled (and gated, masked) in place first
                const int n = 2 * t + x, J = CROSS ? NS - 1 - n : I - n;
                if (GATE) {
                    wg_sync();   // everyone is done with the previous chunk's values
                    statx[row].x = CROSS ? p.Gk[(size_t)s * p.Lkp + J * kTile + row] * kLog2e
                                         : p.G[(size_t)s * p.Lp + J * kTile + row] * kLog2e;
                    wg_sync();
                }
                if (ok && !mbar_wait(&bars[B_SFULL + x], sc & 1, abort_flag, ST_FWD_SOFTMAX)) ok = false;
                ++sc;
                ok = __all_sync(0xffffffffu, ok);  // keep the warp-collective TMEM accesses convergent
                tc_fence_after_sync();
                if (ok) {
                    uint32_t r[4][32];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld32(tlane + colS + c * 32, r[c]);
                    tmem_ld_wait();
                    if (PRE) {
#pragma unroll
                        for (int c = 0; c < 4; ++c)
#pragma unroll
                            for (int e = 0; e < 32; e += 2) {
                                float g0 = 0.f, g1 = 0.f;
                                if (GATE) { g0 = gi2 - statx[c * 32 + e].x; g1 = gi2 - statx[c * 32 + e + 1].x; }
                                const uint64_t v = fma2(pack2(__uint_as_float(r[c][e]), __uint_as_float(r[c][e + 1])), sl2x2,
                                                        pack2(g0, g1));
                                float a, b;
                                unpack2(v, a, b);
                                if (DIAG) {
                                    if (c * 32 + e > row) a = -INFINITY;
                                    if (c * 32 + e + 1 > row) b = -INFINITY;
                                }
                                r[c][e] = __float_as_uint(a);
                                r[c][e + 1] = __float_as_uint(b);
                            }
                    }
                    // row maximum of the scaled logits (log2 units)
                    float a4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int e = 0; e < 32; e += 2)
                            a4[(e >> 1) & 3] = max3(a4[(e >> 1) & 3], __uint_as_float(r[c][e]), __uint_as_float(r[c][e + 1]));
                    float mx = fmaxf(fmaxf(a4[0], a4[1]), fmaxf(a4[2], a4[3]));
                    if (!PRE) mx *= sl2;
                    // lazy rescaling: tolerate a stale maximum up to 2^8.  O of this stream is stable here: its S
                    // tile only becomes ready after the stream's previous P V has retired
                    float m_new = m;
                    const bool grow = mx > m + 8.f;
                    if (grow) m_new = mx;
                    if (__any_sync(0xffffffffu, grow)) {
                        const float alpha = ex2(m - m_new);
                        l *= alpha;
                        if (t > 0) {
#pragma unroll 1
                            for (int c = 0; c < HD / 16; ++c) {
                                uint32_t o[16];
                                tmem_ld16(tlane + colO + c * 16, o);
                                tmem_ld_wait();
#pragma unroll
                                for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                                tmem_st16(tlane + colO + c * 16, o);
                            }
                        }
                    }
                    m = m_new;
                    // probabilities -> packed bf16 over the first 64 columns of the S tile
                    const uint64_t nm2 = pack2(-m, -m);
                    const uint64_t mul2 = PRE ? pack2(1.f, 1.f) : sl2x2;
                    uint64_t lacc = pack2(0.f, 0.f);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t pk[16];
#pragma unroll
                        for (int e = 0; e < 32; e += 2) {
                            const uint64_t v = fma2(pack2(__uint_as_float(r[c][e]), __uint_as_float(r[c][e + 1])), mul2, nm2);
                            float a, b;
                            unpack2(v, a, b);
                            a = ex2(a);
                            b = ex2(b);
                            lacc = add2(lacc, pack2(a, b));
                            pk[e >> 1] = pack_bf16(a, b);
                        }
                        tmem_st16(tlane + colS + c * 16, pk);
                    }
                    float la, lb;
                    unpack2(lacc, la, lb);
                    l += la + lb;
                    tmem_st_wait();
                }
                tc_fence_before_sync();
                mbar_arrive(&bars[B_PFULL + x]);
            };
            {
                int t = 0;
                if (!CROSS && x == 0 && TX > 0) {
                    softmax_step(std::true_type{}, 0);
                    t = 1;
                }
#pragma unroll 1
                for (; t < TX; ++t) softmax_step(std::false_type{}, t);
            }
            // ---- merge the two streams and write O, LSE: warpgroup x handles columns [x*HD/2, (x+1)*HD/2)
            if (GATE) wg_sync();
            if (TX > 0) statx[row] = make_float2(m, l);
            __syncwarp();
            asm volatile("bar.sync 3, 256;" ::: "memory");
            const bool two = NS > 1;
            const float2 s0 = stat[row];
            const float2 s1 = two ? stat[kTile + row] : make_float2(-INFINITY, 0.f);
            if (ok && !mbar_wait(&bars[B_OFULL + 0], item & 1, abort_flag, ST_FWD_SOFTMAX)) ok = false;
            if (two) {
                if (ok && !mbar_wait(&bars[B_OFULL + 1], o1 & 1, abort_flag, ST_FWD_SOFTMAX)) ok = false;
                ++o1;
            }
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after_sync();
            if (!ok) break;
            constexpr int CW = HD / 2;            // columns per warpgroup
            const float mm = fmaxf(s0.x, s1.x);
            const float w0 = ex2(s0.x - mm), w1 = two ? ex2(s1.x - mm) : 0.f;
            const float lsum = s0.y * w0 + s1.y * w1;
            const float inv = 1.f / lsum;
            const float f0 = w0 * inv, f1 = w1 * inv;
            const bool live = qi < p.L;
            const size_t orow = ((size_t)s * p.L + (live ? qi : 0)) * HD;
            uint32_t wrow[CW == 64 ? 32 : 1];   // d = 128: this thread's 64 outputs as one 128-byte row piece
#pragma unroll
            for (int c = 0; c < CW / 32; ++c) {
                const int c0 = x * CW + c * 32;
                uint32_t oa[32], ob[32];
                tmem_ld32(tlane + 256 + c0, oa);
                if (two) tmem_ld32(tlane + 384 + c0, ob);
                tmem_ld_wait();
                if (c == CW / 32 - 1) {
                    tc_fence_before_sync();
                    mbar_arrive(&bars[B_OFREE]);      // O and the stat words may be overwritten
                }
                float o[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    float v = __uint_as_float(oa[e]) * f0;
                    if (two) v += __uint_as_float(ob[e]) * f1;
                    o[e] = v;
                }
                if (CW == 64 && !p.out_fp32) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) wrow[(CW == 64 ? c * 16 : 0) + (CW == 64 ? e : 0)] = pack_bf16(o[2 * e], o[2 * e + 1]);
                    continue;
                }
                if (!live) continue;
                if (p.out_fp32) {
                    float4* dst = reinterpret_cast<float4*>((float*)p.o + orow + c0);
#pragma unroll
                    for (int e = 0; e < 8; ++e) dst[e] = make_float4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
                } else {
                    uint4* dst = reinterpret_cast<uint4*>((__nv_bfloat16*)p.o + orow + c0);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        dst[e] = make_uint4(pack_bf16(o[8 * e], o[8 * e + 1]), pack_bf16(o[8 * e + 2], o[8 * e + 3]),
                                            pack_bf16(o[8 * e + 4], o[8 * e + 5]), pack_bf16(o[8 * e + 6], o[8 * e + 7]));
                }
            }
            if (CW == 64 && !p.out_fp32) {   // the warp's 32 rows, whole 128-byte pieces per store instruction
                const int row0 = I * kTile + q4 * 32;
                if (CW == 64)
                    warp_store_rows128((__nv_bfloat16*)p.o + ((size_t)s * p.L + row0) * HD + x * CW, (size_t)HD * 2,
                                       reinterpret_cast<uint32_t(&)[32]>(wrow), p.L - row0);
            }
            if (live) {
                if (x == 0) p.lse[(size_t)s * p.L + qi] = (mm + log2f(lsum)) * 0.6931471805599453f;
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

// Host-side launcher (called from the C-ABI translation unit).
template <int HD>
static cudaError_t launch_hd(const FwdTensorMaps& tm, const FwdParams& p, cudaStream_t st) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int pairs = (p.N * p.S + 1) / 2;
    dim3 grid(pairs < sms ? pairs : sms), block(384);
    if (p.G) {
        e = cudaFuncSetAttribute(fa_fwd_kernel<HD, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem::alloc);
        if (e != cudaSuccess) return e;
        fa_fwd_kernel<HD, true><<<grid, block, FwdSmem::alloc, st>>>(tm, p);
    } else {
        e = cudaFuncSetAttribute(fa_fwd_kernel<HD, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem::alloc);
        if (e != cudaSuccess) return e;
        fa_fwd_kernel<HD, false><<<grid, block, FwdSmem::alloc, st>>>(tm, p);
    }
    return cudaGetLastError();
}

cudaError_t launch_fa_fwd(const FwdTensorMaps& tm, const FwdParams& p, int hd, cudaStream_t st) {
    return hd == 64 ? launch_hd<64>(tm, p, st) : launch_hd<128>(tm, p, st);
}

template <int HD>
static cudaError_t launch_cross_hd(const FwdTensorMaps& tm, const FwdParams& p, cudaStream_t st) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (!p.G || !p.Gk || p.Nk < 1) return cudaErrorInvalidValue;
    const int pairs = (p.N * p.S + 1) / 2;
    e = cudaFuncSetAttribute(fa_fwd_kernel<HD, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem::alloc);
    if (e != cudaSuccess) return e;
    fa_fwd_kernel<HD, true, true><<<dim3(pairs < sms ? pairs : sms), 384, FwdSmem::alloc, st>>>(tm, p);
    return cudaGetLastError();
}

cudaError_t launch_fa_fwd_cross(const FwdTensorMaps& tm, const FwdParams& p, int hd, cudaStream_t st) {
    return hd == 64 ? launch_cross_hd<64>(tm, p, st) : launch_cross_hd<128>(tm, p, st);
}

}  // namespace path
