// Dyadic run products and version chains (forward and backward), as tcgen05 tile kernels.
//
// The attention sweep never updates a query while it walks the keys (the paper's Sec. 3.3 loop does, once per
// key chunk).  Instead query chunk I and key chunk J < I meet at the dyadic boundary e = (I >> l) << l,
// l = msb(I xor J), which is the same logit by associativity (the key-advance identity of Sec. 3.4):
//     Qv[l][I] = Qleft_I  P_{I-1} ... P_e          Kv[l][J] = Kright_J P_{J+1}^T ... P_{e-1}^T
// Both follow from products of aligned runs of chunk matrices, Dy[l][b] = P_{(b+1) 2^l - 1} ... P_{b 2^l}:
//     Dy[l+1][b] = Dy[l][2b+1] Dy[l][2b]                                                (dyadic_fwd)
//     Qv[l2][I]  = Qv[l1][I] Dy[l1][(I >> l2 << l2) >> l1]      l1 < l2 consecutive set bits of I     (version_fwd)
//     Kv[l2][J]  = Kv[l1][J] Dy[l1][(J >> l1) + 1]^T            l1 < l2 consecutive clear bits of J
// and the backward kernels apply the chain rule to exactly these products.  Run products are stored as bf16
// hi + lo pairs (they are multiplied up to log2(N) times); versions are bf16, the values the sweep consumes.
#include "tileops.cuh"

namespace path {
using namespace tile;

namespace {

struct Ctx {
    uint8_t* smem;
    uint64_t* bars;
    volatile uint32_t* abort_flag;
    uint32_t tmem, tl;
    int tid, warp, lane, row, half;
    uint32_t ph_load, ph_mma;
    bool ok;
};

template <int NCOLS>
__device__ __forceinline__ void setup(Ctx& c, uint8_t* smem_raw, uint32_t bar_off) {
    c.smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    c.bars = (uint64_t*)(c.smem + bar_off);
    uint32_t* tmem_slot = (uint32_t*)(c.bars + 2);
    c.abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    c.tid = threadIdx.x; c.warp = c.tid >> 5; c.lane = c.tid & 31;
    c.row = (c.warp & 3) * 32 + c.lane; c.half = c.warp >> 2;
    c.ph_load = c.ph_mma = 0; c.ok = true;
    if (c.tid == 0) {
        mbar_init(&c.bars[0], 1);
        mbar_init(&c.bars[1], 1);
        *c.abort_flag = 0;
        mbar_fence_init();
    }
    if (c.warp == 0) tmem_alloc(tmem_slot, NCOLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    c.tmem = *tmem_slot;
    c.tl = c.tmem + ((uint32_t)((c.warp & 3) * 32) << 16);
}
template <int NCOLS>
__device__ __forceinline__ void teardown(Ctx& c, uint32_t* status) {
    tc_fence_before_sync();
    __syncthreads();
    if (c.tid == 0 && *c.abort_flag != 0) atomicCAS(status, 0u, *c.abort_flag);
    if (c.warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(c.tmem, NCOLS);
    }
}
__device__ __forceinline__ void loads_wait(Ctx& c) {
    if (!mbar_wait(&c.bars[0], c.ph_load, c.abort_flag, ST_LEVELS)) c.ok = false;
    c.ph_load ^= 1;
}
__device__ __forceinline__ void publish() {
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
}
__device__ __forceinline__ void mma_wait(Ctx& c) {
    __syncwarp();
    if (!mbar_wait(&c.bars[1], c.ph_mma, c.abort_flag, ST_LEVELS)) c.ok = false;
    c.ph_mma ^= 1;
    c.ok = __syncthreads_and(c.ok);
    tc_fence_after_sync();
}
// float rows [nrows][ncols] of a global matrix -> bf16 tile (rows >= nrows are zero-filled)
__device__ __forceinline__ void conv(const Ctx& c, const float* src, int ncols, int nrows, uint8_t* dst) {
    const int per = ncols / 2;
    float v[32];
    for (int i = 0; i < per / 32; ++i) {
        const int c0 = c.half * per + i * 32;
        gload_f32x32(src + (size_t)c.row * ncols + c0, v, c.row < nrows);
        tile_store32(dst, c.row, c0, v);
    }
}
// accumulator rows -> global float matrix [nrows][ncols]: dst += acc (plain or atomic)
template <bool ATOMIC>
__device__ __forceinline__ void acc_add_global(const Ctx& c, uint32_t col, int ncols, int nrows, float* dst) {
    const int per = ncols / 2;
    float v[32];
    for (int i = 0; i < per / 32; ++i) {
        const int c0 = c.half * per + i * 32;
        tmem_row32(c.tl + col + c0, v);
        const bool live = c.row < nrows;
        float* d = dst + (size_t)c.row * ncols + c0;
        if (ATOMIC) {
            if (live) {
#pragma unroll
                for (int x = 0; x < 32; ++x) atomicAdd(d + x, v[x]);
            }
        } else {
            float o[32];
            gload_f32x32(d, o, live);
#pragma unroll
            for (int x = 0; x < 32; ++x) o[x] += v[x];
            gstore_f32x32(d, o, live);
        }
    }
}

// Resolves the version-chain step of chunk c at level l2.  Returns false if there is none.
__device__ __forceinline__ bool version_step(int is_key, int c, int l2, int N, int& l1, int& b, int& src_slot) {
    if (!is_key) {
        const unsigned low = (unsigned)c & ((1u << l2) - 1u);
        if (!((c >> l2) & 1) || low == 0) return false;
        l1 = msb32(low);
        b = ((c >> l2) << l2) >> l1;
        src_slot = qslot(l1, c);
    } else {
        const unsigned lowz = ~(unsigned)c & ((1u << l2) - 1u);
        if (((c >> l2) & 1) || lowz == 0) return false;
        if ((((c >> l2) + 1) << l2) > N - 1) return false;
        l1 = msb32(lowz);
        b = (c >> l1) + 1;
        src_slot = kslot(l1, c);
    }
    return true;
}

constexpr uint32_t kBar3 = 3 * kTileB, kBar4 = 4 * kTileB, kBar5 = 5 * kTileB;
constexpr uint32_t smem_bytes(uint32_t slots) { return slots * kTileB + 64 + 1024; }

// ---------------------------------------------------------------------------------------------- dyadic forward
// grid.x = S * cnt2.  Dy[l+1][b] = Dy[l][2b+1] Dy[l][2b] with hi/lo operands (three products).
template <int HD>
__global__ void __launch_bounds__(256, 1) dyadic_fwd_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<128>(c, smem_raw, kBar4);
    const int cnt2 = p.lv.dy_cnt[p.l + 1], cnt = p.lv.dy_cnt[p.l];
    const int s = blockIdx.x / cnt2, b = blockIdx.x % cnt2;
    const long mat_lo = p.lv.dy_off[p.l] / (HD * HD) + (long)s * cnt + 2 * b;        // right factor; left is +1
    const long mat_out = p.lv.dy_off[p.l + 1] / (HD * HD) + (long)s * cnt2 + b;
    uint8_t* sm = c.smem;
    if (c.tid == 0) {
        mbar_expect_tx(&c.bars[0], 4 * kT * HD * 2);
        tma_tile(sm + 0 * kTileB, &tm.dyh, &c.bars[0], HD, (int)((mat_lo + 1) * HD));
        tma_tile(sm + 1 * kTileB, &tm.dyl, &c.bars[0], HD, (int)((mat_lo + 1) * HD));
        tma_tile(sm + 2 * kTileB, &tm.dyh, &c.bars[0], HD, (int)(mat_lo * HD));
        tma_tile(sm + 3 * kTileB, &tm.dyl, &c.bars[0], HD, (int)(mat_lo * HD));
    }
    loads_wait(c);
    if (c.tid == 0 && c.ok) {
        tc_fence_after_sync();
        const uint32_t a = smem_u32(sm);
        mma(c.tmem, a, OP_K, a + 2 * kTileB, OP_MN, HD / 16, HD, false);
        mma(c.tmem, a, OP_K, a + 3 * kTileB, OP_MN, HD / 16, HD, true);
        mma(c.tmem, a + kTileB, OP_K, a + 2 * kTileB, OP_MN, HD / 16, HD, true);
        umma_commit(&c.bars[1]);
    }
    mma_wait(c);
    if (c.ok) {
        float v[32], hi[32];
        for (int i = 0; i < HD / 64; ++i) {
            const int c0 = c.half * (HD / 2) + i * 32;
            tmem_row32(c.tl + c0, v);
#pragma unroll
            for (int x = 0; x < 32; ++x) {
                hi[x] = __bfloat162float(__float2bfloat16_rn(v[x]));
                v[x] -= hi[x];
            }
            const size_t o = ((size_t)mat_out * HD + c.row) * HD + c0;
            gstore_bf16x32(p.dyh + o, hi, c.row < HD);
            gstore_bf16x32(p.dyl + o, v, c.row < HD);
        }
    }
    teardown<128>(c, p.status);
}

// ---------------------------------------------------------------------------------------------- version forward
// grid = (S * N, 2): y = 0 queries, y = 1 keys; p.l = number of levels.  One CTA walks the whole chain of its chunk,
// bottom level first:  Xv[l2] = Xv[l1] * Dy (queries) or Dy^T (keys).  The version just produced stays in shared
// memory as the next step's left operand (the same bf16 values that go to global memory).
// Highest dyadic level at which chunk `ch` of slice `s` takes part in a chunk pair the sweeps compute: every level for a
// plain problem; for a gated one the level of the farthest kept pair (0 = only level 0 or none: no version chain).
__device__ __forceinline__ int highest_level_reached(const LevelParams& p, int is_key, int s, int ch) {
    if (!p.nkeep) return 30;
    if (is_key) {
        const int T = min(p.N - ch, p.nvisit[s * p.N + ch]);          // query chunks ch .. ch + T - 1 meet this key chunk
        return T > 1 ? msb32((unsigned)((ch + T - 1) ^ ch)) : 0;
    }
    const int T = min(ch, p.nkeep[s * p.N + ch] - 1);                 // key chunks ch - 1 .. ch - T are visited
    return T > 0 ? msb32((unsigned)(ch ^ (ch - T))) : 0;
}

template <int HD>
__global__ void __launch_bounds__(256, 2) version_fwd_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    const int is_key = blockIdx.y, s = blockIdx.x / p.N, ch = blockIdx.x % p.N;
    // levels to build: all of them, or for a gated problem up to the highest one a kept chunk pair uses (see version_bwd)
    const int lim = min(p.l, highest_level_reached(p, is_key, s, ch) + 1);
    int l1, b, src, l2 = 1;
    for (; l2 < lim; ++l2)
        if (version_step(is_key, ch, l2, p.N, l1, b, src)) break;
    if (l2 >= lim) return;
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<128>(c, smem_raw, kBar3);
    uint8_t* sm = c.smem;   // slots: 0 current version, 1 Dy hi, 2 Dy lo
    bool first = true;
#pragma unroll 1
    for (; l2 < lim && c.ok; ++l2) {
        if (!version_step(is_key, ch, l2, p.N, l1, b, src)) continue;
        const long mat = p.lv.dy_off[l1] / (HD * HD) + (long)s * p.lv.dy_cnt[l1] + b;
        const long row_dst = ((long)l2 * p.S + s) * p.Lp + (long)ch * kT;
        if (c.tid == 0) {
            mbar_expect_tx(&c.bars[0], (first ? 3 : 2) * kT * HD * 2);
            if (first) {
                const long row_src = ((long)src * p.S + s) * p.Lp + (long)ch * kT;
                tma_tile(sm, is_key ? &tm.kv : &tm.qv, &c.bars[0], HD, (int)row_src);
            }
            tma_tile(sm + kTileB, &tm.dyh, &c.bars[0], HD, (int)(mat * HD));
            tma_tile(sm + 2 * kTileB, &tm.dyl, &c.bars[0], HD, (int)(mat * HD));
        }
        loads_wait(c);
        if (!first) publish();   // the left operand was written by this CTA's threads
        if (c.tid == 0 && c.ok) {
            tc_fence_after_sync();
            const uint32_t a = smem_u32(sm);
            const int bop = is_key ? OP_K : OP_MN;
            mma(c.tmem, a, OP_K, a + kTileB, bop, HD / 16, HD, false);
            mma(c.tmem, a, OP_K, a + 2 * kTileB, bop, HD / 16, HD, true);
            umma_commit(&c.bars[1]);
        }
        mma_wait(c);
        if (c.ok) {
            float v[32];
            __nv_bfloat16* out = (is_key ? p.kv : p.qv) + (size_t)row_dst * HD;
            for (int i = 0; i < HD / 64; ++i) {
                const int c0 = c.half * (HD / 2) + i * 32;
                tmem_row32(c.tl + c0, v);
                gstore_bf16x32(out + (size_t)c.row * HD + c0, v);
                tile_store32(sm, c.row, c0, v);
            }
        }
        first = false;
    }
    teardown<128>(c, p.status);
}

// ---------------------------------------------------------------------------------------------- version backward
// grid = (S * N, 2), p.l = number of levels.  One CTA walks the chain of its chunk top level first.  With
// g = dXv[l2][chunk] (what the sweeps wrote there plus what arrived from the level above, which stays in tensor memory):
//     dXv[l1][chunk] += g Dy^T (queries) or g Dy (keys);
//     dDy[l1][b]     += Xv[l1]^T g (queries) or g^T Xv[l1] (keys), atomically.
// The run products enter the backward as single bf16 operands (their hi plane), like every other operand of a gradient
// product; the lo plane only matters where products are chained (forward).  Gradients of the versions are bf16 (written
// by the sweeps).  Only the bottom of the chain (always slot 0) leaves the
// CTA: added in place to the slot-0 gradient, which the chunk chain rule then loads as a tile.  The next step's operands are fetched while the
// current one runs.
template <int HD>
__global__ void __launch_bounds__(256, 1) version_bwd_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    const int is_key = blockIdx.y, s = blockIdx.x / p.N, ch = blockIdx.x % p.N;
    int l1, b, src;
    auto next_step = [&](int from) {   // highest level <= from with a version step, 0 if none
        for (int l = from; l >= 1; --l)
            if (version_step(is_key, ch, l, p.N, l1, b, src)) return l;
        return 0;
    };
    // A sweep shortened by block skipping has written the gradients of the levels it reached only (the near ones); the
    // chain starts at the highest of them instead of the top (everything above would have been zero).
    const int top = min(p.l - 1, highest_level_reached(p, is_key, s, ch));
    int l2 = next_step(top);
    if (l2 == 0) return;   // no chain: what the sweeps left in slot 0 is final
    __nv_bfloat16* dxv = is_key ? p.dkv : p.dqv;
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<256>(c, smem_raw, 7 * kTileB);
    uint8_t* sm = c.smem;   // slot 0: g; two buffers of three slots: Dy (hi plane), -, Xv[l1]; a buffer is also the staging area
    auto issue_loads = [&](int buf, uint32_t more_bytes = 0) {   // operands of the step described by (l1, b, src)
        const long mat = p.lv.dy_off[l1] / (HD * HD) + (long)s * p.lv.dy_cnt[l1] + b;
        const long row_src = ((long)src * p.S + s) * p.Lp + (long)ch * kT;
        uint8_t* base = sm + (1 + 3 * buf) * kTileB;
        mbar_expect_tx(&c.bars[0], 2 * kT * HD * 2 + more_bytes);   // one arrival per phase: every byte is announced here
        tma_tile(base, &tm.dyh, &c.bars[0], HD, (int)(mat * HD));
        tma_tile(base + 2 * kTileB, is_key ? &tm.kv : &tm.qv, &c.bars[0], HD, (int)row_src);
    };
    // the top level's gradient needs nothing added: it goes into the g slot as a tile, next to the first operands
    if (c.tid == 0) {
        issue_loads(0, kT * HD * 2);
        tma_tile(sm, is_key ? &tm.dkv : &tm.dqv, &c.bars[0], HD, (int)(((long)l2 * p.S + s) * p.Lp + (long)ch * kT));
    }
    int buf = 0;
    bool have_acc = false;
    // The gradient stored in global memory at the level a step consumes is requested one step ahead (the first one
    // here), so that its latency hides behind the previous step's products and atomics.
    constexpr int NI = HD / 64;
    uint32_t pend[NI][2][8];   // 32 bf16 = 64 bytes per piece
    auto request = [&](long row0) {
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            const __nv_bfloat16* src = dxv + ((size_t)row0 + c.row) * HD + c.half * (HD / 2) + i * 32;
            ld_global_v8(src, pend[i][0]);
            ld_global_v8(src + 16, pend[i][1]);
        }
    };
    auto arrived = [&](int i, float (&v)[32]) {
#pragma unroll
        for (int x = 0; x < 16; ++x) {
            const uint32_t w = pend[i][x >> 3][x & 7];
            v[2 * x] = __uint_as_float(w << 16);
            v[2 * x + 1] = __uint_as_float(w & 0xffff0000u);
        }
    };

#pragma unroll 1
    while (l2 >= 1 && c.ok) {
        version_step(is_key, ch, l2, p.N, l1, b, src);
        const long mat = p.lv.dy_off[l1] / (HD * HD) + (long)s * p.lv.dy_cnt[l1] + b;
        const long row_src = ((long)src * p.S + s) * p.Lp + (long)ch * kT;
        // g = gradient stored at this level + the contribution from above -> bf16 tile (the first step's g is loaded as a tile)
        {
            if (have_acc) {
                float v[32], a[32];
#pragma unroll
                for (int i = 0; i < NI; ++i) {
                    const int c0 = c.half * (HD / 2) + i * 32;
                    arrived(i, v);
                    tmem_row32(c.tl + c0, a);
#pragma unroll
                    for (int x = 0; x < 32; ++x) v[x] += a[x];
                    tile_store32(sm, c.row, c0, v);
                }
            }
            // what is stored at the level this step contributes to: the next step's input, or the chain's final sum
            request(row_src);
        }
        // the step after this one (its description replaces l1, b, src only after this step's were copied above)
        const int l2n = next_step(l2 - 1);
        loads_wait(c);
        tma_store_wait_read();   // the previous step's reductions have read their staging area: the prefetch below refills it
        publish();
        if (c.tid == 0 && c.ok) {
            if (l2n >= 1) issue_loads(buf ^ 1);
            tc_fence_after_sync();
            const uint32_t g = smem_u32(sm), o = smem_u32(sm + (1 + 3 * buf) * kTileB);
            const int bop = is_key ? OP_MN : OP_K;
            mma(c.tmem, g, OP_K, o, bop, HD / 16, HD, false);
            if (!is_key) mma(c.tmem + 128, o + 2 * kTileB, OP_MN, g, OP_MN, 8, HD, false);
            else         mma(c.tmem + 128, g, OP_MN, o + 2 * kTileB, OP_MN, 8, HD, false);
            umma_commit(&c.bars[1]);
        }
        mma_wait(c);
        if (c.ok) {
            // run-product gradient: stage the [d][d] accumulator in this step's (now dead) operand slots
            constexpr int LDS = HD + 4;
            float* stage = (float*)(sm + (1 + 3 * buf) * kTileB);
            float v[32];
            for (int i = 0; i < HD / 64; ++i) {
                const int c0 = c.half * (HD / 2) + i * 32;
                tmem_row32(c.tl + 128 + c0, v);
                if (c.row < HD) {
#pragma unroll
                    for (int x = 0; x < 8; ++x)
                        *reinterpret_cast<float4*>(stage + c.row * LDS + c0 + 4 * x) =
                            make_float4(v[4 * x], v[4 * x + 1], v[4 * x + 2], v[4 * x + 3]);
                }
            }
            fence_proxy_async_smem();
            __syncthreads();
            // one bulk reduction per row: the adds happen at the memory side while this CTA goes on with its next step
            if (c.tid < HD) {
                bulk_reduce_add_f32(p.ddy + (size_t)mat * HD * HD + (size_t)c.tid * HD, stage + c.tid * LDS, HD * 4);
                tma_store_commit();
            }
        }
        have_acc = true;
        l2 = l2n;
        buf ^= 1;
    }
    if (c.ok && have_acc) {   // bottom of the chain: stored value + carried contribution
        float v[32], a[32];
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            const int c0 = c.half * (HD / 2) + i * 32;
            arrived(i, v);
            tmem_row32(c.tl + c0, a);
#pragma unroll
            for (int x = 0; x < 32; ++x) v[x] += a[x];
            // the chain's bottom is always slot 0: its rows now hold the final sum, which the chunk chain rule loads
            gstore_bf16x32(dxv + ((size_t)s * p.Lp + (size_t)ch * kT + c.row) * HD + c0, v);
        }
    }
    tma_store_wait_all();
    teardown<256>(c, p.status);
}

// ---------------------------------------------------------------------------------------------- dyadic backward
// grid.x = S * cnt(l).  With dC = dDy[l][b], A = Dy[l-1][2b+1], B = Dy[l-1][2b]:  dA += dC B^T,  dB += A^T dC
// (A, B: the hi planes of the run products).
template <int HD>
__global__ void __launch_bounds__(256, 1) dyadic_bwd_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<256>(c, smem_raw, kBar5);
    const int cnt = p.lv.dy_cnt[p.l], cntl = p.lv.dy_cnt[p.l - 1];
    const int s = blockIdx.x / cnt, b = blockIdx.x % cnt;
    const long mat_up = p.lv.dy_off[p.l] / (HD * HD) + (long)s * cnt + b;
    const long mat_lo = p.lv.dy_off[p.l - 1] / (HD * HD) + (long)s * cntl + 2 * b;   // B; A is +1
    uint8_t* sm = c.smem;   // slots: 0 dC, 1 A, 3 B (2 and 4 are only part of the staging area below)
    if (c.tid == 0) {
        mbar_expect_tx(&c.bars[0], 2 * kT * HD * 2);
        tma_tile(sm + 1 * kTileB, &tm.dyh, &c.bars[0], HD, (int)((mat_lo + 1) * HD));
        tma_tile(sm + 3 * kTileB, &tm.dyh, &c.bars[0], HD, (int)(mat_lo * HD));
    }
    conv(c, p.ddy + (size_t)mat_up * HD * HD, HD, HD, sm);
    constexpr int NI = HD / 64;
    loads_wait(c);
    publish();
    if (c.tid == 0 && c.ok) {
        tc_fence_after_sync();
        const uint32_t a = smem_u32(sm);
        mma(c.tmem, a, OP_K, a + 3 * kTileB, OP_K, HD / 16, HD, false);            // dC B^T
        mma(c.tmem + 128, a + 1 * kTileB, OP_MN, a, OP_MN, HD / 16, HD, false);    // A^T dC
        umma_commit(&c.bars[1]);
    }
    mma_wait(c);
    if (c.ok) {
        // both [d][d] accumulators are staged in the (now dead) operand slots and added to the gradients of the two
        // factors by bulk reductions, one per row: the adds happen at the memory side
        constexpr int LDS = HD + 4;
        float* stage = (float*)sm;
        float v[32];
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            const int c0 = c.half * (HD / 2) + i * 32;
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                tmem_row32(c.tl + m * 128 + c0, v);
                if (c.row < HD) {
#pragma unroll
                    for (int x = 0; x < 8; ++x)
                        *reinterpret_cast<float4*>(stage + (m * HD + c.row) * LDS + c0 + 4 * x) =
                            make_float4(v[4 * x], v[4 * x + 1], v[4 * x + 2], v[4 * x + 3]);
                }
            }
        }
        fence_proxy_async_smem();
        __syncthreads();
        if (c.tid < 2 * HD) {   // rows 0 .. d-1: dA (factor 2b+1), rows d .. 2d-1: dB (factor 2b)
            const int m = c.tid / HD, r = c.tid % HD;
            bulk_reduce_add_f32(p.ddy + (size_t)(mat_lo + 1 - m) * HD * HD + (size_t)r * HD, stage + c.tid * LDS, HD * 4);
            tma_store_commit();
            tma_store_wait_read();
        }
    }
    teardown<256>(c, p.status);
}

// ---------------------------------------------------------------------------------------------- key cache after a prefill
// grid = (S, d / 64).  Paper Sec. 3.4: after L tokens the cached key of position j is H_{L-1} ... H_{j+1} k_j.  In chunk
// form that is  kc_J = Kright_J R_J  with  R_J = P_{J+1}^T ... P_{N-1}^T,  so a CTA walks the chunks of its slice from the
// last to the first carrying R (bf16 hi + lo in shared memory):  kc_J = Kright_J R  (float32 out),  R <- P_J^T R.
// Both products act on the columns of R independently, so a CTA carries only 64 columns of R (and writes those columns
// of the cache): at d = 128 two CTAs share a slice (four with 32 columns each were no faster per step and, at 4096 tokens,
// more CTAs than SMs).
template <int HD>
__global__ void __launch_bounds__(256, 1) key_cache_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<256>(c, smem_raw, kBar5);
    constexpr int NC = 64;                      // columns of R per CTA
    const int s = blockIdx.x, col0 = blockIdx.y * NC;
    uint8_t* sm = c.smem;   // slots: 0 Kright_J, 1 P hi, 2 P lo, 3 R hi, 4 R lo ([d x 64] in the first panel)
    {   // R = I[:, col0 .. col0+63]; the tiles' unused parts read as zeros (P^T enters with M = 128: its second panel when d = 64)
        for (int i = c.tid; i < (int)(4 * kTileB / 16); i += 256) reinterpret_cast<uint4*>(sm + kTileB)[i] = make_uint4(0, 0, 0, 0);
        __syncthreads();
        if (c.tid < NC) {
            const uint32_t r = (uint32_t)(col0 + c.tid), j = (uint32_t)c.tid;
            *reinterpret_cast<__nv_bfloat16*>(sm + 3 * kTileB + sw128_off(r, j >> 3) + (j & 7) * 2) = __float2bfloat16_rn(1.f);
        }
        fence_proxy_async_smem();
        __syncthreads();
    }
    auto issue = [&](int J) {
        const long mat = p.lv.dy_off[0] / (HD * HD) + (long)s * p.lv.dy_cnt[0] + J;
        mbar_expect_tx(&c.bars[0], 3 * kT * HD * 2);
        tma_tile(sm, &tm.kv, &c.bars[0], HD, (int)((long)s * p.Lp + (long)J * kT));   // version slot 0 = Kright
        tma_tile(sm + kTileB, &tm.dyh, &c.bars[0], HD, (int)(mat * HD));
        tma_tile(sm + 2 * kTileB, &tm.dyl, &c.bars[0], HD, (int)(mat * HD));
    };
    if (c.tid == 0) issue(p.N - 1);
#pragma unroll 1
    for (int J = p.N - 1; J >= 0 && c.ok; --J) {
        loads_wait(c);
        publish();
        if (c.tid == 0 && c.ok) {
            tc_fence_after_sync();
            const uint32_t a = smem_u32(sm);
            mma(c.tmem, a, OP_K, a + 3 * kTileB, OP_MN, HD / 16, NC, false);                       // Kright R
            mma(c.tmem, a, OP_K, a + 4 * kTileB, OP_MN, HD / 16, NC, true);
            if (J > 0) {
                mma(c.tmem + 128, a + 1 * kTileB, OP_MN, a + 3 * kTileB, OP_MN, HD / 16, NC, false);   // P^T R
                mma(c.tmem + 128, a + 2 * kTileB, OP_MN, a + 3 * kTileB, OP_MN, HD / 16, NC, true);
                mma(c.tmem + 128, a + 1 * kTileB, OP_MN, a + 4 * kTileB, OP_MN, HD / 16, NC, true);
            }
            umma_commit(&c.bars[1]);
        }
        mma_wait(c);
        if (!c.ok) break;
        if (c.tid == 0 && J > 0) issue(J - 1);   // every product has retired: the operand slots are free again
        const int pos = J * kT + c.row, c0 = c.half * 32;
        float v[32];
        uint32_t hi[16], lo[16];
        tmem_row32(c.tl + c0, v);
        gstore_f32x32(p.kc + ((size_t)s * p.cap + pos) * HD + col0 + c0, v, pos < p.L);
        if (J > 0) {
            tmem_row32(c.tl + 128 + c0, v);
            if (c.row < HD) {
                split32(v, hi, lo);
                tile_store_w16(sm + 3 * kTileB, c.row, c0, hi);
                tile_store_w16(sm + 4 * kTileB, c.row, c0, lo);
            }
        }
    }
    teardown<256>(c, p.status);
}

template <class K>
cudaError_t launch(K kern, dim3 grid, uint32_t slots, const LevelTensorMaps& tm, const LevelParams& p, cudaStream_t st) {
    const uint32_t bytes = smem_bytes(slots);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return e;
    kern<<<grid, 256, bytes, st>>>(tm, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_level_kernel(int which, const LevelTensorMaps& tm, const LevelParams& p, int hd, cudaStream_t st) {
    switch (which) {
        case LEVEL_DYADIC_FWD: {
            dim3 g(p.S * p.lv.dy_cnt[p.l + 1]);
            return hd == 64 ? launch(dyadic_fwd_kernel<64>, g, 4, tm, p, st) : launch(dyadic_fwd_kernel<128>, g, 4, tm, p, st);
        }
        case LEVEL_VERSION_FWD: {
            dim3 g(p.S * p.N, 2);
            return hd == 64 ? launch(version_fwd_kernel<64>, g, 3, tm, p, st) : launch(version_fwd_kernel<128>, g, 3, tm, p, st);
        }
        case LEVEL_VERSION_BWD: {
            dim3 g(p.S * p.N, 2);
            return hd == 64 ? launch(version_bwd_kernel<64>, g, 7, tm, p, st) : launch(version_bwd_kernel<128>, g, 7, tm, p, st);
        }
        case LEVEL_KEY_CACHE: {
            dim3 g(p.S, hd / 64);
            return hd == 64 ? launch(key_cache_kernel<64>, g, 5, tm, p, st) : launch(key_cache_kernel<128>, g, 5, tm, p, st);
        }
        default: {
            dim3 g(p.S * p.lv.dy_cnt[p.l]);
            return hd == 64 ? launch(dyadic_bwd_kernel<64>, g, 5, tm, p, st) : launch(dyadic_bwd_kernel<128>, g, 5, tm, p, st);
        }
    }
}

}  // namespace path
