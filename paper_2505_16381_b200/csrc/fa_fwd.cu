// Fused forward sweep of PaTH attention (paper Sec. 3.3, the FlashAttention-style loop).
//
// One CTA owns one 128-row query chunk I of one (batch, head) slice and walks the key chunks
// J = I, I-1, ..., 0.  The diagonal chunk uses the raw q, k plus the in-chunk Householder
// correction as a second contraction (Sec. 3.3, case i = j):
//     S = Q K^T + (-lower(Q W^T)) (T^-1 strictLower(W K^T))           [operands q_raw,k_raw,xqn,yt]
// Every earlier chunk J < I is an ordinary tile product of a query version and a key
// version that meet at the dyadic boundary of (I, J):  S = Qv[l][I] Kv[l][J]^T, l = msb(I xor J).
// The versions are prepared by the linear kernels, so this loop contains no query update.
//
// Warp roles: warp 0 = TMA producer, warp 1 = tcgen05 MMA issuer, warps 2-5 = online softmax
// (one query row per thread).  S is double-buffered in TMEM (2 x 128 columns), O accumulates
// in TMEM (HD columns); P goes through shared memory as the A operand of O += P V.
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

template <int HD>
struct FwdSmem {
    static constexpr uint32_t kVBytes = kTile * HD * 2;
    static constexpr uint32_t offA = 0;
    static constexpr uint32_t offK = offA + 2 * kSlotBytes;
    static constexpr uint32_t offV = offK + 2 * kSlotBytes;
    static constexpr uint32_t offP = offV + 2 * kVBytes;
    static constexpr uint32_t offBar = offP + kSlotBytes;
    static constexpr uint32_t offGk = offBar + 256;
    static constexpr uint32_t total = offGk + 2 * kTile * 4;
    static constexpr uint32_t alloc = total + 1024;  // slack to align the base to 1024 B
};

enum { B_AFULL = 0, B_AEMPTY = 2, B_KFULL = 4, B_KEMPTY = 6, B_VFULL = 8, B_VEMPTY = 10,
       B_SFULL = 12, B_SEMPTY = 14, B_PFULL = 16, B_PVDONE = 17, B_COUNT = 18 };

template <int HD, bool GATE>
__global__ void __launch_bounds__(192, 1)
fa_fwd_kernel(const __grid_constant__ FwdTensorMaps tm, const FwdParams p) {
    using SM = FwdSmem<HD>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sA = smem + SM::offA;
    uint8_t* sK = smem + SM::offK;
    uint8_t* sV = smem + SM::offV;
    uint8_t* sP = smem + SM::offP;
    uint64_t* bars = (uint64_t*)(smem + SM::offBar);
    uint32_t* tmem_slot = (uint32_t*)(bars + B_COUNT);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    float* gk = (float*)(smem + SM::offGk);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int I = (int)gridDim.x - 1 - (int)blockIdx.x;  // long tiles first
    const int s = blockIdx.y;
    const int T = I + 1;

    if (threadIdx.x == 0) {
        for (int i = 0; i < B_COUNT; ++i) {
            uint32_t cnt = (i == B_SEMPTY || i == B_SEMPTY + 1 || i == B_PFULL) ? 128u : 1u;
            mbar_init(&bars[i], cnt);
        }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    constexpr uint32_t colS = 0, colO = 256;

    const int rowRaw = s * p.Lp + I * kTile;
    auto ver_row = [&](int slot, int chunk) { return (slot * p.S + s) * p.Lp + chunk * kTile; };

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int na = 0, nk = 0, nv = 0;
            bool ok = true;
            auto load = [&](uint8_t* ring, uint32_t slot_bytes, int bfull, int bempty, int& n,
                            const CUtensorMap* m, int kdim, int row0) {
                if (!ok) return;
                const int slot = n & 1;
                if (!mbar_wait(&bars[bempty + slot], ((n >> 1) & 1) ^ 1, abort_flag, ST_FWD_PRODUCER)) {
                    ok = false;
                    return;
                }
                mbar_expect_tx(&bars[bfull + slot], (uint32_t)(kTile * kdim * 2));
                for (int h = 0; h < kdim / 64; ++h)
                    tma_load_2d(ring + slot * slot_bytes + h * kPanelBytes, m, &bars[bfull + slot], h * 64, row0);
                ++n;
            };
            load(sA, kSlotBytes, B_AFULL, B_AEMPTY, na, &tm.q_raw, HD, rowRaw);
            load(sK, kSlotBytes, B_KFULL, B_KEMPTY, nk, &tm.k_raw, HD, rowRaw);
            load(sA, kSlotBytes, B_AFULL, B_AEMPTY, na, &tm.xqn, kTile, rowRaw);
            load(sK, kSlotBytes, B_KFULL, B_KEMPTY, nk, &tm.yt, kTile, rowRaw);
            load(sV, SM::kVBytes, B_VFULL, B_VEMPTY, nv, &tm.v, HD, rowRaw);
            int cur = -1;
            for (int t = 1; t < T && ok; ++t) {
                const int J = I - t;
                const int l = msb32((unsigned)(I ^ J));
                if (l != cur) {
                    load(sA, kSlotBytes, B_AFULL, B_AEMPTY, na, &tm.qv, HD, ver_row(qslot(l, I), I));
                    cur = l;
                }
                load(sK, kSlotBytes, B_KFULL, B_KEMPTY, nk, &tm.kv, HD, ver_row(kslot(l, J), J));
                load(sV, SM::kVBytes, B_VFULL, B_VEMPTY, nv, &tm.v, HD, s * p.Lp + J * kTile);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idescS = umma_idesc(128, 128, 0, 0);
            constexpr uint32_t idescO = umma_idesc(128, HD, 0, 1);
            int na = 0, nk = 0;
            bool ok = true;
            auto wait_full = [&](int bfull, int n) {
                if (ok && !mbar_wait(&bars[bfull + (n & 1)], (n >> 1) & 1, abort_flag, ST_FWD_MMA)) ok = false;
            };
            // S[buf] (+)= A_slot * K_slot^T over kdim
            auto issue_s = [&](int buf, int aslot, int kslot_, int kdim, bool acc) {
                const uint32_t a0 = smem_u32(sA + aslot * kSlotBytes), b0 = smem_u32(sK + kslot_ * kSlotBytes);
                for (int kk = 0; kk < kdim / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kPanelBytes + (kk & 3) * 32;
                    umma_ss(tmem + colS + buf * 128, umma_desc(a0 + off, 16, 1024), umma_desc(b0 + off, 16, 1024),
                            idescS, (acc || kk > 0) ? 1u : 0u);
                }
            };
            // diagonal chunk: two contractions into S[0]
            wait_full(B_AFULL, 0); wait_full(B_KFULL, 0);
            tc_fence_after_sync();
            if (ok) issue_s(0, 0, 0, HD, false);
            wait_full(B_AFULL, 1); wait_full(B_KFULL, 1);
            tc_fence_after_sync();
            if (ok) {
                issue_s(0, 1, 1, kTile, true);
                umma_commit(&bars[B_SFULL + 0]);
                umma_commit(&bars[B_KEMPTY + 0]);
                umma_commit(&bars[B_KEMPTY + 1]);
                umma_commit(&bars[B_AEMPTY + 0]);
                umma_commit(&bars[B_AEMPTY + 1]);
            }
            na = 2; nk = 2;
            int cur = -1, cur_item = -1;
            for (int t = 0; t < T && ok; ++t) {
                if (t + 1 < T) {
                    const int J = I - (t + 1);
                    const int l = msb32((unsigned)(I ^ J));
                    if (l != cur) {
                        if (cur_item >= 0) umma_commit(&bars[B_AEMPTY + (cur_item & 1)]);
                        cur_item = na++;
                        cur = l;
                        wait_full(B_AFULL, cur_item);
                    }
                    const int buf = (t + 1) & 1, use = (t + 1) >> 1;
                    if (ok && !mbar_wait(&bars[B_SEMPTY + buf], (use & 1) ^ 1, abort_flag, ST_FWD_MMA)) ok = false;
                    wait_full(B_KFULL, nk);
                    tc_fence_after_sync();
                    if (ok) {
                        issue_s(buf, cur_item & 1, nk & 1, HD, false);
                        umma_commit(&bars[B_SFULL + buf]);
                        umma_commit(&bars[B_KEMPTY + (nk & 1)]);
                    }
                    ++nk;
                }
                // O += P V_t
                if (ok && !mbar_wait(&bars[B_PFULL], t & 1, abort_flag, ST_FWD_MMA)) ok = false;
                wait_full(B_VFULL, t);
                tc_fence_after_sync();
                if (ok) {
                    const uint32_t a0 = smem_u32(sP), b0 = smem_u32(sV + (t & 1) * SM::kVBytes);
                    for (int kk = 0; kk < kTile / 16; ++kk) {
                        const uint32_t aoff = (kk >> 2) * kPanelBytes + (kk & 3) * 32;
                        umma_ss(tmem + colO, umma_desc(a0 + aoff, 16, 1024),
                                umma_desc(b0 + kk * 2048, kPanelBytes, 1024), idescO, (t > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(&bars[B_PVDONE]);
                    umma_commit(&bars[B_VEMPTY + (t & 1)]);
                }
            }
        }
    } else {
        // ------------------------------------------------------------ online softmax, one row per thread
        const int q4 = warp & 3;
        const int row = q4 * 32 + lane;
        const int tid = threadIdx.x - 64;  // 0..127
        const uint32_t tlane = tmem + ((uint32_t)(q4 * 32) << 16);
        const int qi = I * kTile + row;  // position within the slice (may be >= L in the ragged tail)
        const float kLog2e = 1.4426950408889634f;
        const float sl2 = p.scale * kLog2e;
        float gi2 = 0.f;
        if (GATE) gi2 = p.G[(size_t)s * p.Lp + qi] * kLog2e;
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        uint32_t r[32];

        for (int t = 0; t < T; ++t) {
            const int b = t & 1;
            const int J = I - t;
            if (GATE) {
                gk[b * kTile + tid] = p.G[(size_t)s * p.Lp + J * kTile + tid] * kLog2e;
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
            if (ok && !mbar_wait(&bars[B_SFULL + b], (t >> 1) & 1, abort_flag, ST_FWD_SOFTMAX)) ok = false;
            ok = __all_sync(0xffffffffu, ok);  // keep the warp-collective TMEM accesses convergent
            tc_fence_after_sync();
            // pass 1: row maximum of the scaled logits
            float mx = -INFINITY;
            if (ok) {
                for (int c = 0; c < 4; ++c) {
                    tmem_ld32(tlane + colS + b * 128 + c * 32, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int x = 0; x < 32; ++x) {
                        float v = __uint_as_float(r[x]) * sl2;
                        if (GATE) v += gi2 - gk[b * kTile + c * 32 + x];
                        if (t == 0 && c * 32 + x > row) v = -INFINITY;
                        mx = fmaxf(mx, v);
                    }
                }
            }
            // the previous P V must be finished before P is overwritten or O rescaled
            if (t > 0 && ok && !mbar_wait(&bars[B_PVDONE], (t - 1) & 1, abort_flag, ST_FWD_SOFTMAX)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after_sync();
            float m_new = m;
            const bool grow = mx > m + 8.f;  // lazy rescaling: tolerate a stale maximum up to 2^8
            if (grow) m_new = mx;
            if (__any_sync(0xffffffffu, grow) && ok) {
                const float alpha = ex2(m - m_new);
                l *= alpha;
                if (t > 0) {
                    for (int c = 0; c < HD / 32; ++c) {
                        tmem_ld32(tlane + colO + c * 32, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int x = 0; x < 32; ++x) r[x] = __float_as_uint(__uint_as_float(r[x]) * alpha);
                        tmem_st32(tlane + colO + c * 32, r);
                    }
                    tmem_st_wait();
                }
            }
            m = m_new;
            // pass 2: probabilities -> bf16 -> swizzled shared-memory A operand
            if (ok) {
                for (int c = 0; c < 4; ++c) {
                    tmem_ld32(tlane + colS + b * 128 + c * 32, r);
                    tmem_ld_wait();
                    uint32_t pk[16];
#pragma unroll
                    for (int x = 0; x < 32; x += 2) {
                        float v0 = __uint_as_float(r[x]) * sl2, v1 = __uint_as_float(r[x + 1]) * sl2;
                        if (GATE) {
                            v0 += gi2 - gk[b * kTile + c * 32 + x];
                            v1 += gi2 - gk[b * kTile + c * 32 + x + 1];
                        }
                        float p0 = ex2(v0 - m), p1 = ex2(v1 - m);
                        if (t == 0) {
                            if (c * 32 + x > row) p0 = 0.f;
                            if (c * 32 + x + 1 > row) p1 = 0.f;
                        }
                        l += p0 + p1;
                        pk[x >> 1] = pack_bf16(p0, p1);
                    }
                    uint8_t* panel = sP + (c >> 1) * kPanelBytes;
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        uint4 val = make_uint4(pk[ch * 4], pk[ch * 4 + 1], pk[ch * 4 + 2], pk[ch * 4 + 3]);
                        *reinterpret_cast<uint4*>(panel + sw128_off((uint32_t)row, (uint32_t)((c & 1) * 4 + ch))) = val;
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&bars[B_SEMPTY + b]);
            fence_proxy_async_smem();
            mbar_arrive(&bars[B_PFULL]);
        }
        // epilogue: O / l, LSE
        if (ok && !mbar_wait(&bars[B_PVDONE], (T - 1) & 1, abort_flag, ST_FWD_SOFTMAX)) ok = false;
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after_sync();
        if (ok) {
            const float inv = 1.f / l;
            const size_t orow = ((size_t)s * p.L + qi) * HD;
            for (int c = 0; c < HD / 32; ++c) {
                tmem_ld32(tlane + colO + c * 32, r);  // warp-collective: rows of a ragged tail load too
                tmem_ld_wait();
                if (qi >= p.L) continue;
                if (p.out_fp32) {
                    float4* dst = reinterpret_cast<float4*>((float*)p.o + orow + c * 32);
#pragma unroll
                    for (int x = 0; x < 8; ++x)
                        dst[x] = make_float4(__uint_as_float(r[4 * x]) * inv, __uint_as_float(r[4 * x + 1]) * inv,
                                             __uint_as_float(r[4 * x + 2]) * inv, __uint_as_float(r[4 * x + 3]) * inv);
                } else {
                    uint4* dst = reinterpret_cast<uint4*>((__nv_bfloat16*)p.o + orow + c * 32);
#pragma unroll
                    for (int x = 0; x < 4; ++x)
                        dst[x] = make_uint4(
                            pack_bf16(__uint_as_float(r[8 * x]) * inv, __uint_as_float(r[8 * x + 1]) * inv),
                            pack_bf16(__uint_as_float(r[8 * x + 2]) * inv, __uint_as_float(r[8 * x + 3]) * inv),
                            pack_bf16(__uint_as_float(r[8 * x + 4]) * inv, __uint_as_float(r[8 * x + 5]) * inv),
                            pack_bf16(__uint_as_float(r[8 * x + 6]) * inv, __uint_as_float(r[8 * x + 7]) * inv));
                }
            }
            if (qi < p.L) p.lse[(size_t)s * p.L + qi] = (m + log2f(l)) * 0.6931471805599453f;
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
    using SM = FwdSmem<HD>;
    dim3 grid(p.N, p.S), block(192);
    cudaError_t e;
    if (p.G) {
        e = cudaFuncSetAttribute(fa_fwd_kernel<HD, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::alloc);
        if (e != cudaSuccess) return e;
        fa_fwd_kernel<HD, true><<<grid, block, SM::alloc, st>>>(tm, p);
    } else {
        e = cudaFuncSetAttribute(fa_fwd_kernel<HD, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::alloc);
        if (e != cudaSuccess) return e;
        fa_fwd_kernel<HD, false><<<grid, block, SM::alloc, st>>>(tm, p);
    }
    return cudaGetLastError();
}

cudaError_t launch_fa_fwd(const FwdTensorMaps& tm, const FwdParams& p, int hd, cudaStream_t st) {
    return hd == 64 ? launch_hd<64>(tm, p, st) : launch_hd<128>(tm, p, st);
}

}  // namespace path
