// Fused forward sweep of PaTH attention (paper Sec. 3.3, the FlashAttention-style loop).
//
// One CTA owns one 128-row query chunk I of one (batch, head) slice and walks the key chunks
// J = I, I-1, ..., 0.  The diagonal chunk uses the raw q, k plus the in-chunk Householder
// correction as a second contraction (Sec. 3.3, case i = j):
//     S = Q K^T + (-lower(Q W^T)) (T^-1 strictLower(W K^T))           [operands q_raw,k_raw,xqn,yt]
// Every earlier chunk J < I is an ordinary tile product of a query version and a key
// version that meet at the dyadic boundary of (I, J):  S = Qv[l][I] Kv[l][J]^T, l = msb(I xor J).
// The versions are prepared beforehand, so this loop contains no query update.
//
// The key chunks are dealt alternately to two streams (n = I - J even / odd).  Each stream has its own
// softmax warpgroup (one query row per thread), its own S tile and O accumulator in tensor memory and its own
// running (max, sum); the two partial results are merged at the end like a split-KV attention.  While one
// warpgroup does its exponentials the tensor pipe works for the other stream.  P never touches shared memory:
// it overwrites the first half of its S tile as packed bf16 and enters O += P V as the tensor-memory A operand.
//
// Warps: 0 = TMA producer, 1 = tcgen05 MMA issuer, 2-5 = softmax of stream 0, 6-9 = softmax of stream 1.
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
    static constexpr uint32_t offGk = offBar + 256;           // [2 streams][128] gate prefix of the current key chunk
    static constexpr uint32_t total = offGk + 2 * kTile * 4;
    static constexpr uint32_t alloc = total + 1024;           // slack to align the base to 1024 B
};

enum { B_QFULL = 0, B_QEMPTY = 3, B_KFULL = 6, B_KEMPTY = 8, B_VFULL = 10, B_VEMPTY = 12,
       B_SFULL = 14, B_PFULL = 16, B_OFINAL = 18, B_COUNT = 20 };

template <int HD, bool GATE>
__global__ void __launch_bounds__(320, 1)
fa_fwd_kernel(const __grid_constant__ FwdTensorMaps tm, const FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem + FwdSmem::offQ;
    uint8_t* sK = smem + FwdSmem::offK;
    uint8_t* sV = smem + FwdSmem::offV;
    uint64_t* bars = (uint64_t*)(smem + FwdSmem::offBar);
    uint32_t* tmem_slot = (uint32_t*)(bars + B_COUNT);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    float* gk = (float*)(smem + FwdSmem::offGk);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int I = (int)gridDim.x - 1 - (int)blockIdx.x;  // long tiles first
    const int s = blockIdx.y;
    const int NS = I + 1;                                 // steps n = 0..I: key chunk J = I - n, stream n & 1

    if (threadIdx.x == 0) {
        for (int i = 0; i < B_COUNT; ++i) mbar_init(&bars[i], (i == B_PFULL || i == B_PFULL + 1) ? 128u : 1u);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    // tensor memory columns: S of stream x at x*128 (P aliases its first 64 columns), O of stream x at 256 + x*128
    const int rowRaw = s * p.Lp + I * kTile;
    auto ver_row = [&](int slot, int chunk) { return (slot * p.S + s) * p.Lp + chunk * kTile; };
    auto level_of = [&](int n) { return msb32((unsigned)(I ^ (I - n))); };   // n >= 1; non-decreasing in n

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            bool ok = true;
            int nq = 0;   // query operands issued so far: rawQ, Xqn, then one version per level met
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
            auto load_kv = [&](uint8_t* base, int bfull, int bempty, int slot, int use, const CUtensorMap* m, int kdim,
                               int row0) {
                wait_empty(bempty + slot, use);
                if (!ok) return;
                mbar_expect_tx(&bars[bfull + slot], (uint32_t)(kTile * kdim * 2));
                for (int h = 0; h < kdim / 64; ++h)
                    tma_load_2d(base + slot * kSlotBytes + h * kPanelBytes, m, &bars[bfull + slot], h * 64, row0);
            };
            // diagonal chunk: raw q, k and the correction operands (both K slots), V of chunk I
            load_q(&tm.q_raw, HD, rowRaw);
            load_kv(sK, B_KFULL, B_KEMPTY, 0, 0, &tm.k_raw, HD, rowRaw);
            load_q(&tm.xqn, kTile, rowRaw);
            load_kv(sK, B_KFULL, B_KEMPTY, 1, 0, &tm.yt, kTile, rowRaw);
            load_kv(sV, B_VFULL, B_VEMPTY, 0, 0, &tm.v, HD, rowRaw);
            int cur = -1;
            for (int n = 1; n < NS && ok; ++n) {
                const int J = I - n, x = n & 1, l = level_of(n);
                if (l != cur) {
                    load_q(&tm.qv, HD, ver_row(qslot(l, I), I));
                    cur = l;
                }
                // K / V slot x belongs to stream x; K slot 1 also served the diagonal once
                const int kuse = (x == 0) ? (n >> 1) : (n >> 1) + 1;
                load_kv(sK, B_KFULL, B_KEMPTY, x, kuse, &tm.kv, HD, ver_row(kslot(l, J), J));
                load_kv(sV, B_VFULL, B_VEMPTY, x, n >> 1, &tm.v, HD, s * p.Lp + J * kTile);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idescS = umma_idesc(128, 128, 0, 0);
            constexpr uint32_t idescO = umma_idesc(128, HD, 0, 1);
            bool ok = true;
            auto wait = [&](int bar, int parity) {
                if (ok && !mbar_wait(&bars[bar], parity & 1, abort_flag, ST_FWD_MMA)) ok = false;
            };
            auto issue_s = [&](int x, int qs, int ks, int kdim, bool acc) {
                const uint32_t a0 = smem_u32(sQ + qs * kSlotBytes), b0 = smem_u32(sK + ks * kSlotBytes);
                for (int kk = 0; kk < kdim / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kPanelBytes + (kk & 3) * 32;
                    umma_ss(tmem + x * 128, umma_desc(a0 + off, 16, 1024), umma_desc(b0 + off, 16, 1024), idescS,
                            (acc || kk > 0) ? 1u : 0u);
                }
            };
            int qi_next = 2, cur_level = -1;   // next version operand index / level of the newest one
            int q_of[2] = {0, 0};              // operand index used by each stream's most recent S product
            int released = 0;                  // query operands [0, released) have been handed back to the producer
            auto advance_q = [&](int n) {      // operand index of step n >= 1 (waits for a newly needed one)
                const int l = level_of(n);
                if (l != cur_level) {
                    cur_level = l;
                    const int qi = qi_next++;
                    wait(B_QFULL + qi % 3, qi / 3);
                }
                return qi_next - 1;
            };
            auto release_q = [&](int upto) {
                for (; released < upto; ++released) umma_commit(&bars[B_QEMPTY + released % 3]);
            };
            // S of step 0 (diagonal, stream 0): two contractions
            wait(B_QFULL + 0, 0); wait(B_KFULL + 0, 0);
            tc_fence_after_sync();
            if (ok) issue_s(0, 0, 0, HD, false);
            wait(B_QFULL + 1, 0); wait(B_KFULL + 1, 0);
            tc_fence_after_sync();
            if (ok) {
                issue_s(0, 1, 1, kTile, true);
                umma_commit(&bars[B_SFULL + 0]);
                umma_commit(&bars[B_KEMPTY + 0]);
                umma_commit(&bars[B_KEMPTY + 1]);
                release_q(2);                  // rawQ and Xqn go back once the diagonal products retire
            }
            // S of step 1 (stream 1)
            if (NS > 1 && ok) {
                q_of[1] = advance_q(1);
                wait(B_KFULL + 1, 1);
                tc_fence_after_sync();
                if (ok) {
                    issue_s(1, q_of[1] % 3, 1, HD, false);
                    umma_commit(&bars[B_SFULL + 1]);
                    umma_commit(&bars[B_KEMPTY + 1]);
                }
            }
            for (int n = 0; n < NS && ok; ++n) {
                const int x = n & 1, t = n >> 1;
                // O_x += P_x V_n
                wait(B_PFULL + x, t);
                wait(B_VFULL + x, t);
                tc_fence_after_sync();
                if (!ok) break;
                {
                    const uint32_t b0 = smem_u32(sV + x * kSlotBytes);
                    for (int kk = 0; kk < kTile / 16; ++kk)
                        umma_ts(tmem + 256 + x * 128, tmem + x * 128 + kk * 8, umma_desc(b0 + kk * 2048, kPanelBytes, 1024),
                                idescO, (t > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(&bars[B_VEMPTY + x]);
                }
                // the stream's next S overwrites P; products issued by one thread execute in order, so it lands after
                // the P V above has read P
                if (n + 2 < NS) {
                    const int qi = advance_q(n + 2);
                    q_of[x] = qi;
                    const int kuse = (x == 0) ? ((n + 2) >> 1) : ((n + 2) >> 1) + 1;
                    wait(B_KFULL + x, kuse);
                    tc_fence_after_sync();
                    if (!ok) break;
                    issue_s(x, qi % 3, x, HD, false);
                    umma_commit(&bars[B_SFULL + x]);
                    umma_commit(&bars[B_KEMPTY + x]);
                    // operands older than what either stream used last can go back to the producer
                    release_q(min(qi, q_of[x ^ 1]));
                } else {
                    umma_commit(&bars[B_OFINAL + x]);
                }
            }
        }
    } else {
        // ------------------------------------------------------------ softmax warpgroups, one row per thread
        const int x = (warp - 2) >> 2;          // stream
        const int q4 = warp & 3;                // TMEM lane quadrant this warp may touch
        const int row = q4 * 32 + lane;
        const uint32_t tlane = tmem + ((uint32_t)(q4 * 32) << 16);
        const uint32_t colS = x * 128, colO = 256 + x * 128;
        const int qi = I * kTile + row;         // position within the slice (may be >= L in the ragged tail)
        const float kLog2e = 1.4426950408889634f;
        const float sl2 = p.scale * kLog2e;
        float gi2 = 0.f;
        if (GATE) gi2 = p.G[(size_t)s * p.Lp + qi] * kLog2e;
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        uint32_t r[32], r2[32];
        const int TX = (NS - x + 1) >> 1;       // steps of this stream: n = 2t + x
        float* gkx = gk + x * kTile;
        auto wg_sync = [&]() {
            if (x == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
            else asm volatile("bar.sync 2, 128;" ::: "memory");
        };

        for (int t = 0; t < TX; ++t) {
            const int n = 2 * t + x, J = I - n;
            if (GATE) {
                wg_sync();   // everyone is done with the previous chunk's values
                gkx[row] = p.G[(size_t)s * p.Lp + J * kTile + row] * kLog2e;
                wg_sync();
            }
            if (ok && !mbar_wait(&bars[B_SFULL + x], t & 1, abort_flag, ST_FWD_SOFTMAX)) ok = false;
            ok = __all_sync(0xffffffffu, ok);  // keep the warp-collective TMEM accesses convergent
            tc_fence_after_sync();
            if (ok) {
                // pass 1: row maximum of the scaled logits
                float mx = -INFINITY;
                for (int c = 0; c < 4; ++c) {
                    tmem_ld32(tlane + colS + c * 32, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        float v = __uint_as_float(r[e]) * sl2;
                        if (GATE) v += gi2 - gkx[c * 32 + e];
                        if (n == 0 && c * 32 + e > row) v = -INFINITY;
                        mx = fmaxf(mx, v);
                    }
                }
                // lazy rescaling: tolerate a stale maximum up to 2^8.  O of this stream is stable here: its S tile
                // only becomes ready after the stream's previous P V has retired
                float m_new = m;
                const bool grow = mx > m + 8.f;
                if (grow) m_new = mx;
                if (__any_sync(0xffffffffu, grow)) {
                    const float alpha = ex2(m - m_new);
                    l *= alpha;
                    if (t > 0) {
                        for (int c = 0; c < HD / 32; ++c) {
                            tmem_ld32(tlane + colO + c * 32, r);
                            tmem_ld_wait();
#pragma unroll
                            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                            tmem_st32(tlane + colO + c * 32, r);
                        }
                    }
                }
                m = m_new;
                // pass 2: probabilities -> packed bf16 over the first 64 columns of the S tile (64 keys per store)
                for (int hh = 0; hh < 2; ++hh) {
                    tmem_ld32(tlane + colS + hh * 64, r);
                    tmem_ld32(tlane + colS + hh * 64 + 32, r2);
                    tmem_ld_wait();
                    uint32_t pk[32];
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float v0 = __uint_as_float(r[e]) * sl2, v1 = __uint_as_float(r[e + 1]) * sl2;
                        float v2 = __uint_as_float(r2[e]) * sl2, v3 = __uint_as_float(r2[e + 1]) * sl2;
                        if (GATE) {
                            const float* g0 = gkx + hh * 64;
                            v0 += gi2 - g0[e]; v1 += gi2 - g0[e + 1]; v2 += gi2 - g0[32 + e]; v3 += gi2 - g0[32 + e + 1];
                        }
                        float p0 = ex2(v0 - m), p1 = ex2(v1 - m), p2 = ex2(v2 - m), p3 = ex2(v3 - m);
                        if (n == 0) {
                            const int c0 = hh * 64 + e;
                            if (c0 > row) p0 = 0.f;
                            if (c0 + 1 > row) p1 = 0.f;
                            if (c0 + 32 > row) p2 = 0.f;
                            if (c0 + 33 > row) p3 = 0.f;
                        }
                        l += (p0 + p1) + (p2 + p3);
                        pk[e >> 1] = pack_bf16(p0, p1);
                        pk[16 + (e >> 1)] = pack_bf16(p2, p3);
                    }
                    tmem_st32(tlane + colS + hh * 32, pk);
                }
                tmem_st_wait();
            }
            tc_fence_before_sync();
            mbar_arrive(&bars[B_PFULL + x]);
        }
        // ---- merge the two streams and write O, LSE: warpgroup x handles columns [x*HD/2, (x+1)*HD/2).
        // The (max, sum) pairs are exchanged through this stream's K slot, which is dead once its last product retired.
        if (ok && TX > 0 && !mbar_wait(&bars[B_OFINAL + x], 0, abort_flag, ST_FWD_SOFTMAX)) ok = false;
        float* stat = (float*)(sK + x * kSlotBytes);
        if (TX > 0) {   // a stream without steps must not touch its slot: the diagonal products may still read it
            stat[row] = m;
            stat[kTile + row] = l;
        }
        asm volatile("bar.sync 3, 256;" ::: "memory");
        if (ok && ((NS - (x ^ 1) + 1) >> 1) > 0 && !mbar_wait(&bars[B_OFINAL + (x ^ 1)], 0, abort_flag, ST_FWD_SOFTMAX))
            ok = false;
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after_sync();
        if (ok) {
            const float* st0 = (const float*)sK;
            const float* st1 = (const float*)(sK + kSlotBytes);
            const bool two = NS > 1;
            const float m0 = st0[row], l0 = st0[kTile + row];
            const float m1 = two ? st1[row] : -INFINITY, l1 = two ? st1[kTile + row] : 0.f;
            const float mm = fmaxf(m0, m1);
            const float w0 = ex2(m0 - mm), w1 = two ? ex2(m1 - mm) : 0.f;
            const float lsum = l0 * w0 + l1 * w1;
            const float inv = 1.f / lsum;
            const size_t orow = ((size_t)s * p.L + qi) * HD;
            constexpr int CW = HD / 2;            // columns per warpgroup
            for (int c = 0; c < CW / 32; ++c) {
                const int c0 = x * CW + c * 32;
                tmem_ld32(tlane + 256 + c0, r);
                if (two) tmem_ld32(tlane + 384 + c0, r2);
                tmem_ld_wait();
                float o[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    float v = __uint_as_float(r[e]) * w0;
                    if (two) v += __uint_as_float(r2[e]) * w1;
                    o[e] = v * inv;
                }
                if (qi >= p.L) continue;
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
            if (x == 0 && qi < p.L) p.lse[(size_t)s * p.L + qi] = (mm + log2f(lsum)) * 0.6931471805599453f;
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
    dim3 grid(p.N, p.S), block(320);
    cudaError_t e;
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

}  // namespace path
